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


def test_shard_units_is_a_partition():
    for n in (0, 1, 5, 6, 72):
        for world in (1, 2, 4, 8):
            got = [i for r in range(world) for i in multi.shard_units(n, world, r)]
            assert got == list(range(n))
            sizes = [len(multi.shard_units(n, world, r)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    assert multi.max_over_ranks(3.5) == 3.5      # no process group: identity
