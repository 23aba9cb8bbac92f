"""Batch sharding over ranks (world size 2, gloo, CPU): slices are disjoint and complete, every rank
derives the same Phi from the seed, the gathered per-rank results equal the unsharded result, and the
timing reduction takes the maximum."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import csat_oracle as orc
from oracle import phi_oracle as pho
from paper_2507_02957_b200 import parallel, workloads as wl


def test_shard_range_partitions_every_total():
    for total in range(0, 23):
        for world in range(1, 9):
            got = []
            for rank in range(world):
                start, count = parallel.shard_range(total, world, rank)
                assert count in (total // world, total // world + 1)
                got.extend(range(start, start + count))
            assert got == list(range(total))
    with pytest.raises(ValueError):
        parallel.shard_range(4, 2, 2)
    with pytest.raises(ValueError):
        parallel.shard_range(4, 0, 0)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, outdir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = wl.shrink(wl.CONFIGS["c2"], B=5, H=2, n=48, n_q=48, m=16, d=8)
        inp = wl.make_inputs(w)                                   # the whole job's inputs, same on every rank
        phi = wl.round_to_storage(pho.phi_gaussian(w.H, w.m, w.n, w.phi_seed).astype(np.float32), w.dtype)
        start, count = parallel.shard_range(w.B, world, rank)
        D = np.broadcast_to(np.eye(w.d), (w.H, w.d, w.d))
        mine = orc.csat_forward(inp["Q"][start:start + count], inp["K"][start:start + count],
                                inp["V"][start:start + count], phi, T=3, lam=0.01, D=D)
        # no collective on the data path; the gather below only serves the check
        parts = [None] * world
        dist.all_gather_object(parts, (start, mine))
        t = parallel.max_over_ranks(1.0 + rank)
        if rank == 0:
            full = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi, T=3, lam=0.01, D=D)
            got = np.concatenate([p for _, p in sorted(parts, key=lambda sp: sp[0])], axis=0)
            np.save(os.path.join(outdir, "ok.npy"),
                    np.array([float(np.array_equal(got, full)), t, float(got.shape[0])]))
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_forward(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    ok, tmax, rows = np.load(tmp_path / "ok.npy")
    assert ok == 1.0 and tmax == 2.0 and rows == 5
