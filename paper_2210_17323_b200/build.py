"""Builds the CUDA libraries in-tree with nvcc for sm_100a (no GPU needed to compile).

    python -m paper_2210_17323_b200.build [--force] [--verbose]

Outputs (git-ignored, next to the sources so they travel with the tree):
    paper_2210_17323_b200/lib/libgptq_b200.so    the solver (C ABI of include/gptq_b200.h)
    paper_2210_17323_b200/lib/libgptq_synth.so   device-side filler for the seeded synthetic inputs
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
SYNTH = os.path.join(HERE, "synth")
LIB = os.path.join(HERE, "lib")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"] + os.environ.get("GPTQ_NVCC_EXTRA", "").split()

SOLVER_SOURCES = ["api.cu", "hessian.cu", "hessian_umma.cu", "hinv.cu", "quantize.cu", "solve_host.cu", "rtn.cu", "inference.cu"]


def _newest(paths):
    return max(os.path.getmtime(p) for p in paths)


def _compile(src, obj, verbose):
    cmd = [NVCC, *FLAGS, "-c", src, "-o", obj] + (["-Xptxas", "-v"] if verbose else [])
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed for {src}:\n{r.stdout}\n{r.stderr}")
    if verbose:
        sys.stderr.write(r.stderr)


def _build_lib(name, src_dir, sources, force, verbose):
    os.makedirs(LIB, exist_ok=True)
    out = os.path.join(LIB, name)
    srcs = [os.path.join(src_dir, s) for s in sources]
    deps = srcs + [os.path.join(src_dir, f) for f in os.listdir(src_dir) if f.endswith((".cuh", ".h"))]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "gptq_b200.h"))
    if not force and os.path.exists(out) and os.path.getmtime(out) >= _newest(deps):
        return out
    objs = [os.path.join(LIB, os.path.splitext(s)[0] + ".o") for s in sources]
    with ThreadPoolExecutor(8) as ex:
        list(ex.map(lambda so: _compile(so[0], so[1], verbose), zip(srcs, objs)))
    r = subprocess.run([NVCC, "-shared", "-o", out, *objs, "-lcudart"], capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed for {name}:\n{r.stdout}\n{r.stderr}")
    return out


def build(force=False, verbose=False):
    a = _build_lib("libgptq_b200.so", CSRC, SOLVER_SOURCES, force, verbose)
    b = _build_lib("libgptq_synth.so", SYNTH, ["synth_kernels.cu"], force, verbose)
    return a, b


if __name__ == "__main__":
    print(*build("--force" in sys.argv, "--verbose" in sys.argv), sep="\n")
