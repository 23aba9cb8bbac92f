"""Runs a few CSAT forwards of a given shape and prints the library's per-kernel CUDA-event times.

    python -m paper_2507_02957_b200.profile_case forward N M D B H T [--nq NQ] [--iters I] [--dtype bf16|fp32] [--untied]
    python -m paper_2507_02957_b200.profile_case workload c1|c2|c3|c4|c5 [--iters I]
    python -m paper_2507_02957_b200.profile_case ensembles N M D H        (regenerates Phi with every ensemble)
    python -m paper_2507_02957_b200.profile_case project N D B H DMODEL [--iters I]   (the Q, K, V projections)
    python -m paper_2507_02957_b200.profile_case backward c1|c2|c3|c4|c5 [--iters I]   (csat_backward on a workload)
    python -m paper_2507_02957_b200.profile_case hadamard N D B H [--iters I]   (compression of the structured Hadamard
                       ensemble, dense product against fast transform, for m / n in {1/16, 1/8, 1/4, 1/2})

A small driver to put under a profiler (ncu -k regex:<kernel> ...): 3 warm-up forwards, then I timed ones.
Inputs are seeded random tensors (N(0, 1/d) for `forward`, the workload's own recipe for `workload`).
--untied replaces the ISTA-derived decoder by random LISTA weights with one S_t, B_t per layer.
"""
from __future__ import annotations

import argparse
import time

import numpy as np
import torch

from . import binding, workloads as wl


def _timed_forwards(ctx, Q, K, V, iters):
    out = torch.empty_like(Q)
    for _ in range(3):
        ctx.forward(Q, K, V, out)
    torch.cuda.synchronize()
    binding.csat_set_i64(ctx.h, binding.CSAT_PROFILE, iters)
    for _ in range(iters):
        ctx.forward(Q, K, V, out)
    torch.cuda.synchronize()
    per = {}
    for i in range(iters):
        for kid, ms in binding.csat_get_profile(ctx.h, i):
            per.setdefault(binding.KERNEL_NAMES.get(kid, str(kid)), []).append(ms)
    return {k: round(float(np.median(v)), 5) for k, v in per.items()}


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="cmd", required=True)
    f = sub.add_parser("forward")
    for name in ("n", "m", "d", "B", "H", "T"):
        f.add_argument(name, type=int)
    f.add_argument("--nq", type=int, default=None)
    f.add_argument("--iters", type=int, default=5)
    f.add_argument("--dtype", default="bf16", choices=["bf16", "fp32"])
    f.add_argument("--untied", action="store_true")
    w_ = sub.add_parser("workload")
    w_.add_argument("name")
    w_.add_argument("--iters", type=int, default=5)
    e = sub.add_parser("ensembles")
    for name in ("n", "m", "d", "H"):
        e.add_argument(name, type=int)
    pj = sub.add_parser("project")
    for name in ("n", "d", "B", "H", "dm"):
        pj.add_argument(name, type=int)
    pj.add_argument("--iters", type=int, default=10)
    bw = sub.add_parser("backward")
    bw.add_argument("name")
    bw.add_argument("--iters", type=int, default=3)
    bw.add_argument("--weight-grads", action="store_true", help="also form the gradients of the decoder's parameters")
    bw.add_argument("--phi-grad", action="store_true", help="also time csat_backward_phi (reported separately)")
    bw.add_argument("--untied", action="store_true", help="one random S_t, B_t per layer instead of the ISTA-derived pair")
    bw.add_argument("--saved", action="store_true", help="time forward (saving for the backward) and backward separately")
    hd = sub.add_parser("hadamard")
    for name in ("n", "d", "B", "H"):
        hd.add_argument(name, type=int)
    hd.add_argument("--iters", type=int, default=10)
    a = ap.parse_args()

    if a.cmd == "forward":
        nq = a.nq or a.n
        dt = torch.bfloat16 if a.dtype == "bf16" else torch.float32
        g = torch.Generator(device="cuda")
        g.manual_seed(1)
        s = 1.0 / np.sqrt(a.d)
        Q = (torch.randn(a.B, a.H, nq, a.d, device="cuda", generator=g) * s).to(dt)
        K = (torch.randn(a.B, a.H, a.n, a.d, device="cuda", generator=g) * s).to(dt)
        V = (torch.randn(a.B, a.H, a.n, a.d, device="cuda", generator=g) * s).to(dt)
        ctx = binding.Csat(a.n, a.m, a.d, a.H, 0, B=a.B, n_q=nq, dtype=a.dtype, T=a.T, lam=0.05)
        if a.untied and a.T > 0:
            eye = torch.eye(a.d, device="cuda")
            S = (0.6 * eye + 0.4 * s * torch.randn(a.T, a.H, a.d, a.d, device="cuda", generator=g)).to(dt)
            Bm = (s * torch.randn(a.T, a.H, a.d, a.d, device="cuda", generator=g)).to(dt)
            ctx.set_lista_layer_weights(S, Bm, torch.full((a.T, a.H), 0.02, device="cuda"))
        print(vars(a), _timed_forwards(ctx, Q, K, V, a.iters))
        ctx.close()
    elif a.cmd == "workload":
        w = wl.CONFIGS[a.name]
        inp = wl.make_inputs(w)
        dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
        Q, K, V = (torch.from_numpy(inp[k]).cuda().to(dt) for k in "QKV")
        ctx = binding.Csat(w.n, w.m, w.d, w.H, w.phi_seed, B=w.B, n_q=w.n_q, dtype=w.dtype, T=w.T, lam=w.lam)
        if inp["Psi"] is not None:
            ctx.set_dictionary(torch.from_numpy(inp["Psi"]).cuda().to(dt))
        print(w.name, _timed_forwards(ctx, Q, K, V, a.iters))
        ctx.close()
    elif a.cmd == "backward":
        w = wl.CONFIGS[a.name]
        inp = wl.make_inputs(w)
        dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
        Q, K, V = (torch.from_numpy(inp[k]).cuda().to(dt) for k in "QKV")
        ctx = binding.Csat(w.n, w.m, w.d, w.H, w.phi_seed, B=w.B, n_q=w.n_q, dtype=w.dtype, T=w.T, lam=w.lam)
        if inp["Psi"] is not None:
            ctx.set_dictionary(torch.from_numpy(inp["Psi"]).cuda().to(dt))
        if a.weight_grads:
            binding.csat_set_i64(ctx.h, binding.CSAT_WEIGHT_GRADS, 1)
        if a.untied and w.T > 0:
            g = torch.Generator(device="cuda")
            g.manual_seed(1)
            sc = 1.0 / np.sqrt(w.d)
            S = (0.6 * torch.eye(w.d, device="cuda") + 0.4 * sc * torch.randn(w.T, w.H, w.d, w.d, device="cuda", generator=g)).to(dt)
            Bm = (sc * torch.randn(w.T, w.H, w.d, w.d, device="cuda", generator=g)).to(dt)
            ctx.set_lista_layer_weights(S, Bm, torch.full((w.T, w.H), 0.02, device="cuda"))
        G = torch.randn_like(Q)
        dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
        binding.csat_backward(ctx.h, Q, K, V, G, dQ, dK, dV)
        torch.cuda.synchronize()
        times = []
        for _ in range(a.iters):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            binding.csat_backward(ctx.h, Q, K, V, G, dQ, dK, dV)
            e1.record()
            e1.synchronize()
            times.append(e0.elapsed_time(e1))
        res = {"backward_ms": round(float(np.median(times)), 4), "weight_grads": bool(a.weight_grads), "untied": bool(a.untied)}
        if a.saved:
            binding.csat_set_i64(ctx.h, binding.CSAT_SAVE_FOR_BACKWARD, 1)
            out = torch.empty_like(Q)
            tf, tb = [], []
            for _ in range(a.iters + 1):
                e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                e0.record()
                ctx.forward(Q, K, V, out)
                e1.record()
                binding.csat_backward(ctx.h, Q, K, V, G, dQ, dK, dV)
                e2.record()
                e2.synchronize()
                tf.append(e0.elapsed_time(e1))
                tb.append(e1.elapsed_time(e2))
            res["saving_forward_ms"] = round(float(np.median(tf[1:])), 4)
            res["backward_after_saving_forward_ms"] = round(float(np.median(tb[1:])), 4)
        if a.phi_grad:
            dPhi = torch.empty(w.H, w.m, w.n, dtype=torch.float32, device="cuda")
            binding.csat_backward_phi(ctx.h, K, V, dPhi)
            torch.cuda.synchronize()
            tp = []
            for _ in range(a.iters):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                binding.csat_backward_phi(ctx.h, K, V, dPhi)
                e1.record()
                e1.synchronize()
                tp.append(e0.elapsed_time(e1))
            res["backward_phi_ms"] = round(float(np.median(tp)), 4)
        print(w.name, res)
        ctx.close()
    elif a.cmd == "hadamard":
        g = torch.Generator(device="cuda")
        g.manual_seed(1)
        s = 1.0 / np.sqrt(a.d)
        Q, K, V = ((torch.randn(a.B, a.H, a.n, a.d, device="cuda", generator=g) * s).to(torch.bfloat16) for _ in range(3))
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        for frac in (16, 8, 4, 2):
            ctx = binding.Csat(a.n, a.n // frac, a.d, a.H, 0, B=a.B, dtype="bf16", T=0)
            ctx.set(ensemble="hadamard")
            out = torch.empty_like(Q)
            row = {}
            for mode in ("dense", "transform"):
                ctx.set(hadamard_transform=(mode == "transform"))
                for _ in range(3):
                    ctx.forward(Q, K, V, out)
                torch.cuda.synchronize()
                binding.csat_set_i64(ctx.h, binding.CSAT_PROFILE, a.iters)
                for _ in range(a.iters):
                    flush.zero_()
                    ctx.forward(Q, K, V, out)
                torch.cuda.synchronize()
                ts = [ms for i in range(a.iters) for kid, ms in binding.csat_get_profile(ctx.h, i) if kid == 1]
                binding.csat_set_i64(ctx.h, binding.CSAT_PROFILE, 0)
                row[mode] = round(float(np.median(ts)), 5)
            print(f"n={a.n} d={a.d} B={a.B} H={a.H} m=n/{frac}={a.n // frac}: compress ms", row)
            ctx.close()
    elif a.cmd == "project":
        g = torch.Generator(device="cuda")
        g.manual_seed(1)
        X = torch.randn(a.B, a.n, a.dm, device="cuda", generator=g).to(torch.bfloat16)
        W = (torch.randn(a.dm, 3 * a.H * a.d, device="cuda", generator=g) / np.sqrt(a.dm)).to(torch.bfloat16)
        ctx = binding.Csat(a.n, min(64, a.n), a.d, a.H, 0, B=a.B, dtype="bf16", T=0)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        Q, K, V = (torch.empty(a.B, a.H, a.n, a.d, dtype=torch.bfloat16, device="cuda") for _ in range(3))
        for _ in range(3):
            binding.csat_project_qkv(ctx.h, X, X, W, a.dm, Q, K, V)
        times = []
        for _ in range(a.iters):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            binding.csat_project_qkv(ctx.h, X, X, W, a.dm, Q, K, V)
            e1.record()
            e1.synchronize()
            times.append(e0.elapsed_time(e1))
        ms = float(np.median(times))
        fl = 2.0 * a.B * a.n * a.dm * 3 * a.H * a.d
        print(vars(a), {"ms": round(ms, 4), "tflops": round(fl / ms / 1e9, 1)})
        ctx.close()
    else:
        ctx = binding.Csat(a.n, a.m, a.d, a.H, 0, dtype="bf16")
        for ens in ("rademacher", "gaussian", "hadamard", "gaussian", "rademacher"):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            ctx.set(ensemble=ens)
            torch.cuda.synchronize()
            print(ens, "regenerated (memset + kernel + synchronise):", round((time.perf_counter() - t0) * 1e3, 3), "ms")
        ctx.close()


if __name__ == "__main__":
    main()
