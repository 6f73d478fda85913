"""N > 1 host logic on CPU: two gloo ranks shard the units, agree on the slowest time, and -- rows and
layers being independent (Section 2) -- reproduce the single-process oracle result when their shares are joined."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import gptq_oracle as O
from paper_2210_17323_b200 import multi
from paper_2210_17323_b200.synth import workloads as WL


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # weak scaling: own copy of the layer set, own seeds
        wl = WL.workload(0)
        mine = multi.rank_layers(wl.layers, rank)
        assert mine[0].block_idx == rank and mine[0].seed(1) != wl.layers[0].seed(1) or rank == 0
        # strong scaling over rows of one layer: each rank solves its stripe with the shared U
        L = WL.Layer(7, 0, "q", 37, 64, 300)
        rows = multi.shard_units(L.R, world, rank)
        H = O.hessian_accumulate(np.zeros((L.C, L.C)), L.x_bits())
        U = O.cholesky_inverse_upper(O.dampen(H, 0.01)[0])
        part = O.quantize_layer(L.w(rows=np.arange(rows.start, rows.stop)), U, 4, 0, False, 32)
        np.save(os.path.join(out_dir, f"codes{rank}.npy"), part["codes"])
        # strong scaling of a whole layer: token-sharded Hessian + one all-reduce, factor on every rank, row stripes
        L2 = WL.Layer(7, 1, "k", 21, 32, 257)
        Xi = np.round(O.bf16_bits_to_f64(L2.x_bits()) * 4).clip(-64, 64)         # small integers: sums are exact in any order
        rows2, out2, H2, _ = multi.solve_layer_sharded(
            L2.n_tokens, L2.R, world, rank,
            hessian_of_tokens=lambda tr: torch.from_numpy(2.0 * Xi[tr.start:tr.stop].T @ Xi[tr.start:tr.stop]),
            factor_of=lambda H: O.cholesky_inverse_upper(O.dampen(H.numpy(), 0.01)[0]),
            quantize_rows=lambda rr, U: O.quantize_layer(L2.w(rows=np.arange(rr.start, rr.stop)), U, 3, 16, False, 16))
        assert np.array_equal(H2.numpy(), 2.0 * Xi.T @ Xi)                          # every rank holds the full Hessian
        np.save(os.path.join(out_dir, f"strong{rank}.npy"), out2["codes"])
        # timing reduction: the job's time is the slowest rank's; throughput sums
        assert multi.max_over_ranks(10.0 + rank) == 10.0 + world - 1
        assert multi.sum_over_ranks(float(len(rows))) == float(L.R)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_rows_and_reduce_timing(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    L = WL.Layer(7, 0, "q", 37, 64, 300)
    H = O.hessian_accumulate(np.zeros((L.C, L.C)), L.x_bits())
    U = O.cholesky_inverse_upper(O.dampen(H, 0.01)[0])
    full = O.quantize_layer(L.w(), U, 4, 0, False, 32)
    joined = np.concatenate([np.load(tmp_path / f"codes{r}.npy") for r in range(world)])
    assert np.array_equal(joined, full["codes"])
    L2 = WL.Layer(7, 1, "k", 21, 32, 257)
    Xi = np.round(O.bf16_bits_to_f64(L2.x_bits()) * 4).clip(-64, 64)
    U2 = O.cholesky_inverse_upper(O.dampen(2.0 * Xi.T @ Xi, 0.01)[0])
    full2 = O.quantize_layer(L2.w(), U2, 3, 16, False, 16)
    joined2 = np.concatenate([np.load(tmp_path / f"strong{r}.npy") for r in range(world)])
    assert np.array_equal(joined2, full2["codes"])


def test_shard_units_is_a_partition():
    for n in (0, 1, 5, 6, 72):
        for world in (1, 2, 4, 8):
            got = [i for r in range(world) for i in multi.shard_units(n, world, r)]
            assert got == list(range(n))
            sizes = [len(multi.shard_units(n, world, r)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    assert multi.max_over_ranks(3.5) == 3.5      # no process group: identity
