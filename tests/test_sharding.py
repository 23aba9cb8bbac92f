"""Sharding over ranks (world size 2, gloo, CPU).  Batch sharding: slices are disjoint and complete, every rank
derives the same Phi from the seed, the gathered per-rank results equal the unsharded result, and the
timing reduction takes the maximum.  Token sharding: the shards are aligned, disjoint and complete; the host logic
of parallel.sharded_forward (partial compression, one all-gather, fixed-order sum, local queries) is run with the
oracle's steps standing in for the kernels and must reproduce the unsharded oracle, with bit-identical K~|V~ on
both ranks."""
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


def test_token_shards_are_aligned_disjoint_and_complete():
    for n in (0, 1, 63, 64, 65, 197, 1568, 4096):
        for world in (1, 2, 3, 8):
            got = []
            for rank in range(world):
                start, count = parallel.token_shard_range(n, world, rank)
                assert count >= 0 and (count == 0 or start % 64 == 0)
                got.extend(range(start, start + count))
            assert got == list(range(n)), (n, world)


def _token_worker(rank, world, port, outdir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        B, H, n, nq, d, m, T, lam = 2, 2, 200, 37, 8, 24, 3, 0.01
        r = np.random.default_rng(123)                            # the whole job's inputs, same on every rank
        Q, K, V = r.standard_normal((B, H, nq, d)), r.standard_normal((B, H, n, d)), r.standard_normal((B, H, n, d))
        phi = pho.phi_gaussian(H, m, n, 7)
        D = np.broadcast_to(np.eye(d), (H, d, d))
        n0, n_len = parallel.token_shard_range(n, world, rank)
        q0, q_len = parallel.shard_range(nq, world, rank)
        state = {}

        def compress_partial(Ks, Vs, j0):
            Ks, Vs = Ks.numpy(), Vs.numpy()
            out = np.empty((B, H, m, 2 * d))
            for b in range(B):
                for h in range(H):
                    cols = phi[h][:, j0:j0 + Ks.shape[2]]
                    out[b, h] = np.concatenate([orc.compress(cols, Ks[b, h]), orc.compress(cols, Vs[b, h])], axis=1)
            return torch.from_numpy(out)

        def reduce_partials(stacked):
            acc = stacked[0].numpy().copy()
            for i in range(1, stacked.shape[0]):                  # rank order
                acc += stacked[i].numpy()
            state["kv"] = acc

        def attend(Ql):
            Ql = Ql.numpy()
            out = np.empty_like(Ql)
            for b in range(B):
                for h in range(H):
                    Kt, Vt = state["kv"][b, h][:, :d], state["kv"][b, h][:, d:]
                    Z = orc.compressed_output(orc.softmax_rows(orc.compressed_scores(Ql[b, h], Kt)), Vt)
                    S_dec, B_dec, theta, _ = orc.decoder_setup(D[h], lam)
                    out[b, h] = orc.reconstruct(orc.ista(Z, S_dec, B_dec, theta, T), None)
            return out

        mine = parallel.sharded_forward(
            torch.from_numpy(Q[:, :, q0:q0 + q_len].copy()), torch.from_numpy(K[:, :, n0:n0 + n_len].copy()),
            torch.from_numpy(V[:, :, n0:n0 + n_len].copy()), n0, compress_partial=compress_partial,
            zeros_partial=lambda: torch.zeros(B, H, m, 2 * d, dtype=torch.float64), reduce_partials=reduce_partials,
            attend=attend)
        parts = [None] * world
        dist.all_gather_object(parts, (q0, mine, state["kv"].tobytes()))
        if rank == 0:
            full = orc.csat_forward(Q, K, V, phi, T=T, lam=lam, D=D)
            got = np.concatenate([p for _, p, _ in sorted(parts, key=lambda sp: sp[0])], axis=2)
            same_kv = float(len({kvb for _, _, kvb in parts}) == 1)
            np.save(os.path.join(outdir, "tok.npy"),
                    np.array([float(np.abs(got - full).max()), float(np.abs(full).max()), same_kv, float(got.shape[2])]))
    finally:
        dist.destroy_process_group()


def test_two_ranks_token_sharded_forward_reproduces_the_oracle(tmp_path):
    world = 2
    mp.spawn(_token_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    err, ref_max, same_kv, rows = np.load(tmp_path / "tok.npy")
    assert ref_max > 0 and err <= 1e-12 * ref_max        # only the order of the token sum differs
    assert same_kv == 1.0                                # the fixed-order sum gives every rank the same bits
    assert rows == 37
