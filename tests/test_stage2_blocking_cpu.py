"""Host-side check of the blocked algebra stage 2 uses on the GPU (Section 3 Step 3; Algorithm 1 line 3).

The CUDA path does not follow the oracle's literal route (factor H~, invert, factor again): it factors
H~ = U~ U~^T backwards in outer panels with look-ahead, inverts the diagonal blocks as it goes, solves the
rows above a diagonal block with the block's explicit inverse, and then builds U = U~^-1 panel by panel.
This file replays exactly that sequence of block operations in numpy fp64 at small block sizes and checks
the result against the oracle's cholesky_inverse_upper, so that a wrong index range, a missing dependency
or a wrong triangle in the schedule is caught without a GPU.  It also pins the row-block form of the
triangular inverse, V[k, after] = -V_kk (T[k, after] V[after, after]).
"""
import numpy as np
import pytest

from oracle import gptq_oracle as O


def _spd(C, seed):
    rng = np.random.default_rng(seed)
    X = rng.normal(size=(3 * C, C)) * np.exp(rng.normal(size=C))
    H = 2.0 * X.T @ X
    Ht, _ = O.dampen(H, 0.01)
    return Ht


def _backward_cholesky_block(A):
    """T upper with A = T T^T (the factorisation run from the last row backwards)."""
    P = np.eye(A.shape[0])[::-1]
    L = np.linalg.cholesky(P @ A @ P)
    return P @ L @ P


def _stage2_blocked(Ht, NB2):
    """The schedule of the CUDA path with outer panels of NB2 columns: per panel J (last to first)
    C1 diagonal-block update, B1 update of the rows above, C2 factor D, C3 V = D^-1, C4 / B2 rows above
    = A V^T; then phase 2, U[0:j0, J] = -U[0:j0, 0:j0] (U~[0:j0, J] V_JJ).  Reads of the "finished factor"
    go through F, a separate copy that is written only where the CUDA path writes its split copies."""
    C = Ht.shape[0]
    U = np.triu(Ht).copy()
    F = np.zeros_like(U)
    n_outer = -(-C // NB2)
    for J in range(n_outer - 1, -1, -1):
        j0 = J * NB2
        wj = min(NB2, C - j0)
        rp = j0 + wj
        if rp < C:
            FJ = F[j0:rp, rp:]
            U[j0:rp, j0:rp] -= np.triu(FJ @ FJ.T)                      # C1 (upper part only)
            if j0 > 0:
                U[0:j0, j0:rp] -= F[0:j0, rp:] @ FJ.T                  # B1
        D = U[j0:rp, j0:rp]
        T = _backward_cholesky_block(np.triu(D) + np.triu(D, 1).T)      # C2
        V = np.linalg.inv(T)                                            # C3
        assert np.allclose(np.tril(V, -1), 0.0)
        U[j0:rp, j0:rp] = np.triu(V)
        if j0 == 0:
            continue
        r1 = j0 - NB2
        for lo, hi in ((0, r1), (r1, j0)):                              # B2, then C4
            if hi > lo:
                U[lo:hi, j0:rp] = U[lo:hi, j0:rp] @ V.T
                F[lo:hi, j0:rp] = U[lo:hi, j0:rp]
    for J in range(1, n_outer):                                         # phase 2
        j0 = J * NB2
        rp = min(C, j0 + NB2)
        if J == 1:
            F[0:NB2, 0:NB2] = U[0:NB2, 0:NB2]
        V = U[j0:rp, j0:rp]
        TT = V.T @ F[0:j0, j0:rp].T
        U[0:j0, j0:rp] = -np.triu(F[0:j0, 0:j0]) @ TT.T
        F[0:rp, j0:rp] = U[0:rp, j0:rp]
    return U


@pytest.mark.parametrize("C,NB2", [(8, 8), (12, 4), (24, 8), (40, 16), (33, 8), (64, 16)])
def test_lookahead_schedule_equals_literal_route(C, NB2):
    Ht = _spd(C, 100 + C)
    U_ref = O.cholesky_inverse_upper(Ht)
    U = _stage2_blocked(Ht, NB2)
    assert np.allclose(np.tril(U, -1), 0.0)
    assert np.linalg.norm(U - U_ref) <= 1e-9 * np.linalg.norm(U_ref)
    assert np.linalg.norm(U.T @ U @ Ht - np.eye(C)) <= 1e-8 * C


def test_row_block_form_of_the_triangular_inverse():
    """V = T^-1 for upper T, built from the last row block up: V_kk = T_kk^-1 and
    V[k, after] = -V_kk (T[k, after] V[after, after]) -- row block k of T is read only once, so the
    inverse can overwrite it while the factorisation goes on above it."""
    rng = np.random.default_rng(7)
    n, nb = 24, 4
    T = np.triu(rng.normal(size=(n, n))) + 4.0 * np.eye(n)
    V = np.zeros_like(T)
    for k0 in range(n - nb, -1, -nb):
        a = k0 + nb
        Vkk = np.linalg.inv(T[k0:a, k0:a])
        V[k0:a, k0:a] = Vkk
        if a < n:
            V[k0:a, a:] = -Vkk @ (T[k0:a, a:] @ V[a:, a:])
    assert np.allclose(V @ T, np.eye(n), atol=1e-12)
    assert np.allclose(np.tril(V, -1), 0.0)
