#!/usr/bin/env python
"""Benchmark of the CSAT forward (compressed-sensing attention) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--impl csat|reference]

A step is one whole forward (compression, compressed softmax attention, recovery iterations) over one
batch of synthetic input of the named workload.  One JSON line is printed by rank 0.

  value      query tokens per second, inputs resident in device memory, CUDA events around K steps
  e2e        same metric through csat_forward_host: pinned host buffers, copies inside the timed region
  roofline   dominant kernel: algorithmic flops / CUDA-event time against the measured bf16 peak
  cpu_baseline  the float64 CPU oracle timed on a bounded sample of the same workload (rank 0, N = 1)

With N > 1 (torchrun) every rank runs the same workload on its own batch (weak scaling, no collective on
the data path: every (batch, head) pair is independent and Phi is a function of the seed).
--impl reference times the CPU oracle instead (there is no other implementation of the paper).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2507_02957_b200 import workloads as wl  # noqa: E402

METRIC = "csat_forward_query_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu capture
# summarised under profiles/ (None until a capture of that kernel and workload exists)
NCU_TRAFFIC_BYTES = {
    # profiles/dram_traffic_c5_long.txt: 152.2 MB read + 86.0 MB written by the attention / recovery kernel (part of
    # the 134 MB output is still in L2 when the kernel ends); algorithmic: Q 134.2 + out 134.2 + K~|V~ B 16.8 MB
    ("attend_recover", "c5_long"): 238173952,
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


FFMA_LANES_PER_SM, SMS = 128, 148


def fp32_ffma_peak_tflops(peaks: dict) -> float:
    """Peak of the plain-ALU (FFMA) path, from the unit counts: SMs x fp32 lanes x 2 flop x the SM clock."""
    return SMS * FFMA_LANES_PER_SM * 2 * float(peaks.get("sm_max_mhz", 1965.0)) * 1e6 / 1e12


def choose_tensor_peak(peaks: dict, region_ms: float, clocks: dict | None) -> tuple[str, float]:
    """Burst or sustained bf16 peak, whichever matches how the kernel was timed: the burst figure for a short timed
    region at full clocks with no power cap, the sustained one for a long region or one that ran under the cap."""
    burst = float(peaks["bf16_tflops"])
    sustained = float(peaks.get("bf16_tflops_sustained") or burst)
    capped = bool(clocks) and "sw_power_cap" in (clocks.get("reasons") or [])
    slow = bool(clocks) and clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and clocks["sm_mhz"] < 0.95 * clocks["sm_max_mhz"]
    if region_ms > 500.0 or capped or slow:
        return "sustained", sustained
    return "burst", burst


def roofline_fractions(w: wl.Workload, ms: float, flop: float, peaks: dict) -> dict:
    """Achieved throughput of one whole forward against both rooflines (tensor or ALU, and HBM)."""
    es = 4 if w.dtype == "fp32" else 2
    bytes_alg = input_bytes(w) + w.H * w.m * w.n * es
    t = ms * 1e-3
    hbm = float(peaks["hbm_gbs"])
    out = {"hbm_gbs": bytes_alg / t / 1e9, "frac_hbm": bytes_alg / t / 1e9 / hbm}
    if w.dtype == "fp32":
        pk = fp32_ffma_peak_tflops(peaks)
        out.update(bound="alu", frac_alu_peak=flop / t / 1e12 / pk, peak_tflops=pk)
        t_roof = max(flop / (pk * 1e12), bytes_alg / (hbm * 1e9))
    else:
        burst, sus = float(peaks["bf16_tflops"]), float(peaks.get("bf16_tflops_sustained") or peaks["bf16_tflops"])
        out.update(bound="tensor", frac_burst=flop / t / 1e12 / burst, frac_sustained=flop / t / 1e12 / sus,
                   frac_nominal_2250=flop / t / 1e12 / 2250.0)
        t_roof = max(flop / (burst * 1e12), bytes_alg / (hbm * 1e9))
    out["roofline_us"] = t_roof * 1e6            # the slower of the two limits (burst peak, measured HBM)
    out["frac_of_roofline"] = t_roof / t
    return out


def workload_config(w: wl.Workload, n_gpus: int) -> dict:
    return {"workload": w.name, "B_per_gpu": w.B, "H": w.H, "n": w.n, "n_q": w.n_q, "d": w.d, "m": w.m,
            "T": w.T, "lambda": w.lam, "storage": w.dtype, "parallelism": f"batch-sharded x{n_gpus}",
            "l2": "inputs larger than L2" if input_bytes(w) > 126e6 else "L2 flushed between iterations"}


def input_bytes(w: wl.Workload) -> int:
    es = 4 if w.dtype == "fp32" else 2
    return (2 * w.B * w.H * w.n_q * w.d + 2 * w.B * w.H * w.n * w.d) * es


# ---------------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        import torch
        sel = str(device_index)
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            sel = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            pass
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", sel, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.tmp.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        self.tmp.close()
        os.unlink(self.tmp.name)
        # samples under load: the upper half (the sampler also sees idle time around the region)
        sm_sorted = sorted(sm)
        load = sm_sorted[len(sm_sorted) // 2:] if sm_sorted else []
        return {"sm_mhz": float(np.median(load)) if load else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------------
# the CPU oracle, timed (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------------------
def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 0) for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def oracle_step(w: wl.Workload, inp: dict, phi_by_head: dict, pairs) -> float:
    """One bounded step of the oracle: the listed (b, h) pairs in full.  Returns seconds."""
    from oracle import csat_oracle as orc
    t0 = time.perf_counter()
    for (b, h) in pairs:
        orc.csat_forward_head(inp["Q"][b, h], inp["K"][b, h], inp["V"][b, h], phi_by_head[h], T=w.T, lam=w.lam,
                              Psi=inp["Psi"])
    return time.perf_counter() - t0


def oracle_sample_plan(w: wl.Workload, inp: dict, budget_s: float):
    """Choose how many (b, h) pairs one oracle step covers so that a step costs about budget_s."""
    from oracle import phi_oracle as pho
    phi = {0: wl.round_to_storage(pho.phi_gaussian(w.H, w.m, w.n, w.phi_seed, heads=[0])[0].astype(np.float32),
                                  w.dtype).astype(np.float64)}
    t1 = oracle_step(w, inp, phi, [(0, 0)])
    total = w.B * w.H
    k = int(max(1, min(total, round(budget_s / max(t1, 1e-6)))))
    pairs = [(i // w.H, i % w.H) for i in range(k)]
    for h in sorted({h for _, h in pairs} - {0}):
        phi[h] = wl.round_to_storage(pho.phi_gaussian(w.H, w.m, w.n, w.phi_seed, heads=[h])[0].astype(np.float32),
                                     w.dtype).astype(np.float64)
    return pairs, phi


def oracle_tokens_per_s(w: wl.Workload, seconds: float, npairs: int) -> float:
    # a whole job is B*H pairs and B*n_q query tokens; scale the sampled pairs to it
    return (w.B * w.n_q) / (seconds * (w.B * w.H) / npairs)


def run_reference(args, w: wl.Workload) -> dict:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return {}
    inp = wl.make_inputs(w)
    per_step_budget = max(1.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    pairs, phi = oracle_sample_plan(w, inp, per_step_budget)
    for _ in range(args.warmup):
        oracle_step(w, inp, phi, pairs)
    t = 0.0
    for _ in range(args.steps):
        t += oracle_step(w, inp, phi, pairs)
    per = t / args.steps
    val = oracle_tokens_per_s(w, per, len(pairs))
    cores = blas_threads()
    sample = f"{len(pairs)} of {w.B * w.H} (batch, head) pairs per step, all {w.n_q} queries each, scaled to the whole job"
    return {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": per * 1e3 * (w.B * w.H) / len(pairs),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, args.gpus),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


# ---------------------------------------------------------------------------------------------------
# the CUDA library, timed
# ---------------------------------------------------------------------------------------------------
def device_tensors(w: wl.Workload, seed_shift: int = 0):
    """Host (pinned) and device copies of the workload's inputs in the storage dtype."""
    import torch
    from dataclasses import replace
    inp = wl.make_inputs(replace(w, data_seed=w.data_seed + seed_shift), rounded=False)
    dt = torch.float32 if w.dtype == "fp32" else torch.bfloat16
    host = {k: torch.from_numpy(inp[k]).to(dt).pin_memory() for k in "QKV"}     # round-to-nearest-even
    dev = {k: host[k].cuda(non_blocking=True) for k in "QKV"}
    psi = None if inp["Psi"] is None else torch.from_numpy(inp["Psi"]).to(dt).cuda()
    torch.cuda.synchronize()
    return host, dev, psi


def make_ctx(w: wl.Workload, psi):
    from paper_2507_02957_b200 import binding
    ctx = binding.Csat(w.n, w.m, w.d, w.H, w.phi_seed, B=w.B, n_q=w.n_q, dtype=w.dtype, T=w.T, lam=w.lam)
    if psi is not None:
        ctx.set_dictionary(psi)
    return ctx


def kernel_flops(w: wl.Workload) -> dict:
    f = wl.flops(w)
    return {"compress": f["compress"], "attend_recover": f["attend"] + f["recover"], "decoder_setup": 0}


def executed_attend_flops(w: wl.Workload, sms: int) -> int:
    """Flops the attention / recovery launch group really performs on the tensor cores.  The algorithmic count has
    T + 1 products of d x d per query (alpha^t S for t = 0 .. T-1 and z B); the kernel skips alpha^0 S = 0, and where
    the library folds B into the compressed values (ISTA-derived decoder, T >= 2, a positive threshold, at least
    2 tiles of 128 queries per SM at d = 128 and 8 at d = 64) the n_q products z B become the m products V~ B of the
    small kernel before it."""
    bh = w.B * w.H
    f = wl.flops(w)
    if w.T <= 0:
        return f["attend"]
    psi = f["recover"] - 2 * w.n_q * w.d * w.d * (w.T + 1) * bh
    ex = f["attend"] + 2 * w.n_q * w.d * w.d * w.T * bh + psi
    folded = (w.dtype == "bf16" and w.d in (64, 128) and w.T >= 2 and w.lam > 0
              and -(-w.n_q // 128) * bh >= (2 if w.d == 128 else 8) * sms)
    if folded:
        ex += (2 * w.m - 2 * w.n_q) * w.d * w.d * bh
    return ex


def time_small(w: wl.Workload, iters: int = 10, warmup: int = 3, untied: bool = False, peaks: dict | None = None,
               device_index: int = 0) -> dict:
    """Per-iteration CUDA-event timing with an L2 flush between iterations (workloads that fit in L2).
    untied: random LISTA weights with one S_t, B_t per layer instead of the ISTA-derived decoder."""
    import torch
    host, dev, psi = device_tensors(w)
    ctx = make_ctx(w, psi)
    if untied:
        g = torch.Generator(device="cuda")
        g.manual_seed(7)
        s = 1.0 / np.sqrt(w.d)
        dt = dev["Q"].dtype
        S = (0.6 * torch.eye(w.d, device="cuda") + 0.4 * s * torch.randn(w.T, w.H, w.d, w.d, device="cuda", generator=g)).to(dt)
        Bm = (s * torch.randn(w.T, w.H, w.d, w.d, device="cuda", generator=g)).to(dt)
        ctx.set_lista_layer_weights(S, Bm, torch.full((w.T, w.H), 0.02, device="cuda"))
    out = torch.empty_like(dev["Q"])
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(warmup):
        ctx.forward(dev["Q"], dev["K"], dev["V"], out)
    times = []
    # at least `iters` iterations and long enough (0.25 s) for the clock sampler to see the GPU under this load
    sampler = ClockSampler(device_index) if peaks is not None else None
    t_start = time.perf_counter()
    while len(times) < iters or (sampler is not None and time.perf_counter() - t_start < 0.25 and len(times) < 2000):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.forward(dev["Q"], dev["K"], dev["V"], out)
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
    clocks = sampler.stop() if sampler is not None else None
    ctx.close()
    ms = float(np.median(times))
    f = wl.flops(w)["total"]
    if untied:
        f += 2 * w.n_q * w.d * w.d * (w.T - 1) * w.B * w.H      # z B_t in every layer after the first
    res = {"ms": ms, "iters": len(times), "tokens_per_s": w.query_tokens / (ms * 1e-3), "tflops": f / (ms * 1e-3) / 1e12,
           "gflop": f / 1e9}
    if peaks is not None:
        res["roofline"] = roofline_fractions(w, ms, f, peaks)
        res["clocks"] = clocks
    return res


def time_projection(w: wl.Workload, iters: int = 10, warmup: int = 3) -> dict:
    """The Q, K, V projections in front of the path (csat_project_qkv) for the workload's shape, d_model = H d,
    self-attention form (one GEMM over 3 H d columns); L2 flushed between iterations."""
    import torch
    from paper_2507_02957_b200 import binding
    dm = w.H * w.d
    g = torch.Generator(device="cuda")
    g.manual_seed(11)
    X = torch.randn(w.B, w.n, dm, device="cuda", generator=g).to(torch.bfloat16)
    W = (torch.randn(dm, 3 * dm, device="cuda", generator=g) / np.sqrt(dm)).to(torch.bfloat16)
    ctx = binding.Csat(w.n, w.m, w.d, w.H, w.phi_seed, B=w.B, dtype="bf16", T=0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    Q, K, V = (torch.empty(w.B, w.H, w.n, w.d, dtype=torch.bfloat16, device="cuda") for _ in range(3))
    for _ in range(warmup):
        binding.csat_project_qkv(ctx.h, X, X, W, dm, Q, K, V)
    times = []
    for _ in range(iters):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        binding.csat_project_qkv(ctx.h, X, X, W, dm, Q, K, V)
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
    ctx.close()
    ms = float(np.median(times))
    f = 2.0 * w.B * w.n * dm * 3 * dm
    return {"ms": ms, "tflops": f / (ms * 1e-3) / 1e12, "gflop": f / 1e9, "d_model": dm}


def time_backward(w: wl.Workload, iters: int = 2, weight_grads: bool = False) -> dict:
    """csat_backward (gradients with respect to Q, K, V; with weight_grads also to the decoder's S, B, thresholds and
    dictionary) on a workload."""
    import torch
    from paper_2507_02957_b200 import binding
    host, dev, psi = device_tensors(w)
    ctx = make_ctx(w, psi)
    if weight_grads:
        binding.csat_set_i64(ctx.h, binding.CSAT_WEIGHT_GRADS, 1)
    G = torch.randn_like(dev["Q"])
    dQ, dK, dV = torch.empty_like(dev["Q"]), torch.empty_like(dev["K"]), torch.empty_like(dev["V"])
    binding.csat_backward(ctx.h, dev["Q"], dev["K"], dev["V"], G, dQ, dK, dV)
    torch.cuda.synchronize()
    times = []
    for _ in range(iters):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        binding.csat_backward(ctx.h, dev["Q"], dev["K"], dev["V"], G, dQ, dK, dV)
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
    phi_ms = None
    if w.dtype == "bf16" and w.d in (64, 128) and not weight_grads:
        # the gradient with respect to the measurement matrices, from the dK~|dV~ that call left
        dPhi = torch.empty(w.H, w.m, w.n, dtype=torch.float32, device="cuda")
        binding.csat_backward_phi(ctx.h, dev["K"], dev["V"], dPhi)
        torch.cuda.synchronize()
        tp = []
        for _ in range(iters):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            binding.csat_backward_phi(ctx.h, dev["K"], dev["V"], dPhi)
            e1.record()
            e1.synchronize()
            tp.append(e0.elapsed_time(e1))
        phi_ms = float(np.median(tp))
    saved = None
    if w.dtype == "bf16" and w.d in (64, 128) and not weight_grads:
        # the training pattern: a forward that saves for the backward, then a backward that reuses it
        binding.csat_set_i64(ctx.h, binding.CSAT_SAVE_FOR_BACKWARD, 1)
        out = torch.empty_like(dev["Q"])
        tf, tb = [], []
        for _ in range(iters + 1):
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            e0.record()
            binding.csat_forward(ctx.h, dev["Q"], dev["K"], dev["V"], out)
            e1.record()
            binding.csat_backward(ctx.h, dev["Q"], dev["K"], dev["V"], G, dQ, dK, dV)
            e2.record()
            e2.synchronize()
            tf.append(e0.elapsed_time(e1))
            tb.append(e1.elapsed_time(e2))
        saved = {"forward_ms": float(np.median(tf[1:])), "backward_ms": float(np.median(tb[1:]))}
    ctx.close()
    if weight_grads:
        return {"ms": float(np.median(times)), "kernels": "as backward, plus the iterates and dx_t kept as bf16, a tcgen05 "
                "contraction over them (dS, dB, dPsi) and a streaming sum (dtheta)"}
    return {"ms": float(np.median(times)), "backward_phi_ms": phi_ms, "with_save_for_backward": saved,
            "kernels": "bf16: every stage on tcgen05 (forward with decisions recorded, recurrence backward, dQ, dK~|dV~, "
                       "Phi^T); float32: ffma kernels"}


def run_csat(args, w: wl.Workload) -> dict:
    import torch
    import torch.distributed as dist
    from paper_2507_02957_b200 import binding, parallel

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the CSAT library has no CPU path")
    torch.cuda.set_device(local)
    under_torchrun = "RANK" in os.environ and "MASTER_ADDR" in os.environ
    if world > 1 or under_torchrun:
        # NCCL prints its version banner on stdout (NCCL_DEBUG=VERSION) when the communicator is created, i.e. at the
        # first collective; stdout carries the one JSON line, so file descriptor 1 points at stderr until then
        sys.stdout.flush()
        saved_fd = os.dup(1)
        os.dup2(2, 1)
        try:
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
            dist.barrier()
            torch.cuda.synchronize()
        finally:
            sys.stdout.flush()
            os.dup2(saved_fd, 1)
            os.close(saved_fd)

    def barrier():
        if dist.is_initialized():
            dist.barrier()
        torch.cuda.synchronize()

    peaks, peak_kind = load_peaks()
    host, dev, psi = device_tensors(w, seed_shift=rank)
    ctx = make_ctx(w, psi)
    out = torch.empty_like(dev["Q"])
    K, W = args.steps, max(args.warmup, 3)
    for _ in range(W):
        ctx.forward(dev["Q"], dev["K"], dev["V"], out)
    torch.cuda.synchronize()
    binding.csat_set_i64(ctx.h, binding.CSAT_PROFILE, K)

    sampler = ClockSampler(local) if rank == 0 else None
    launches = 0
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(K):
        ctx.forward(dev["Q"], dev["K"], dev["V"], out)
        launches += ctx.launches
    e1.record()
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop() if sampler else None
    ms_total = parallel.max_over_ranks(e0.elapsed_time(e1), device="cuda")
    ms_step = ms_total / K

    # per-kernel CUDA-event times recorded inside the timed region
    per = {}
    for i in range(K):
        for kid, ms in binding.csat_get_profile(ctx.h, i):
            name = binding.KERNEL_NAMES.get(kid, str(kid))
            a = per.setdefault(name, [0, 0.0])
            a[0] += 1
            a[1] += ms
    binding.csat_set_i64(ctx.h, binding.CSAT_PROFILE, 0)
    kf = kernel_flops(w)
    tot_ms = sum(v[1] for v in per.values()) or 1.0
    kernels = []
    for name, (cnt, ms) in sorted(per.items(), key=lambda kv: -kv[1][1]):
        avg = ms / cnt
        tf = kf.get(name, 0) / (avg * 1e-3) / 1e12
        kernels.append({"kernel": name, "launch_groups": cnt, "avg_ms": avg, "share": ms / tot_ms, "tflops": tf})
    top = kernels[0]
    burst_tf = float(peaks["bf16_tflops"])
    sustained_tf = float(peaks.get("bf16_tflops_sustained") or burst_tf)
    if w.dtype == "fp32":
        # FFMA path (no fp32 tensor-core kernel): plain ALU bound, peak from the unit counts and the clock
        peak_tf = fp32_ffma_peak_tflops(peaks)
        roofline = {"kernel": top["kernel"], "bound": "alu", "achieved": top["tflops"], "peak": peak_tf,
                    "unit": "TFLOP/s", "frac": top["tflops"] / peak_tf,
                    "peak_source": "148 SMs x 128 fp32 lanes x 2 flop x max SM clock", "traffic": None,
                    "flops_per_launch": kf.get(top["kernel"], 0), "avg_launch_ms": top["avg_ms"]}
    else:
        which, peak_tf = choose_tensor_peak(peaks, ms_total, clocks)
        roofline = {"kernel": top["kernel"], "bound": "tensor", "achieved": top["tflops"], "peak": peak_tf,
                    "unit": "TFLOP/s", "frac": top["tflops"] / peak_tf,
                    "peak_source": f"{peak_kind} bf16 {which} (timed region {ms_total:.0f} ms)",
                    "frac_burst": top["tflops"] / burst_tf, "frac_sustained": top["tflops"] / sustained_tf,
                    "frac_nominal_2250": top["tflops"] / 2250.0,
                    "traffic": NCU_TRAFFIC_BYTES.get((top["kernel"], w.name)),
                    "flops_per_launch": kf.get(top["kernel"], 0), "avg_launch_ms": top["avg_ms"]}
        if top["kernel"] == "attend_recover":
            # achieved / frac above count the algorithmic flops; these two count what the tensor cores really did
            ex = executed_attend_flops(w, torch.cuda.get_device_properties(local).multi_processor_count)
            roofline["flops_executed_per_launch"] = ex
            roofline["frac_executed"] = ex / (top["avg_ms"] * 1e-3) / 1e12 / peak_tf
        for k in kernels:
            k["frac_burst"] = k["tflops"] / burst_tf
            k["frac_sustained"] = k["tflops"] / sustained_tf

    # end to end through the host-buffer entry point (copies inside the timed region)
    oh = torch.empty_like(host["Q"]).pin_memory()
    ctx.forward_host(host["Q"], host["K"], host["V"], oh)
    barrier()
    t0 = time.perf_counter()
    for _ in range(K):
        ctx.forward_host(host["Q"], host["K"], host["V"], oh)
    torch.cuda.synchronize()
    e2e_s = parallel.max_over_ranks(time.perf_counter() - t0, device="cuda")
    h2d = sum(host[k].numel() * host[k].element_size() for k in "QKV")
    d2h = oh.numel() * oh.element_size()
    ctx.close()

    tokens = w.query_tokens * world
    fl = wl.flops(w)
    result = {
        "metric": METRIC, "value": tokens / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic", "config": workload_config(w, world),
        "tflops": fl["total"] * world / (ms_step * 1e-3) / 1e12,
        "frac_of_bf16_peak": {"measured_burst": fl["total"] / (ms_step * 1e-3) / 1e12 / burst_tf,
                              "measured_sustained": fl["total"] / (ms_step * 1e-3) / 1e12 / sustained_tf,
                              "nominal_2250": fl["total"] / (ms_step * 1e-3) / 1e12 / 2250.0},
        "hbm_gbs_algorithmic": (input_bytes(w) + w.H * w.m * w.n * (4 if w.dtype == "fp32" else 2))
        / (ms_step * 1e-3) / 1e9,
        "roofline": roofline, "kernels": kernels,
        "e2e": {"value": tokens / (e2e_s / K), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_s / K * 1e3},
        "gpu_launches": launches, "clocks": clocks,
    }

    if rank == 0 and world == 1:
        if not args.no_extra:
            extra = {}
            for key in ("c1", "c2", "c3", "c4"):
                extra[wl.CONFIGS[key].name] = time_small(wl.CONFIGS[key], peaks=peaks, device_index=local)
            for n in (2048, 4096, 8192, 16384):
                extra[f"c5_sweep_n{n}"] = time_small(wl.sweep_config(n), peaks=peaks, device_index=local)
            if w.T > 1 and w.dtype == "bf16":
                extra[f"{w.name}_untied_layers"] = time_small(w, untied=True)
            if w.dtype == "bf16" and w.n == w.n_q:
                extra[f"{w.name}_qkv_projection"] = time_projection(w)
            extra["backward"] = {wl.CONFIGS[k].name: time_backward(wl.CONFIGS[k], iters=1 if k == "c5" else 2)
                                 for k in ("c1", "c2", "c3", "c4", "c5")}
            extra["backward_with_weight_gradients"] = {
                wl.CONFIGS[k].name: time_backward(wl.CONFIGS[k], iters=1 if k == "c5" else 2, weight_grads=True)
                for k in ("c2", "c3", "c4", "c5")}
            result["other_workloads"] = extra
        if not args.no_cpu_baseline:
            inp = {k: host[k].float().numpy() for k in "QKV"}
            inp["Psi"] = None if psi is None else psi.float().cpu().numpy()
            pairs, phi = oracle_sample_plan(w, inp, 12.0)
            sec = oracle_step(w, inp, phi, pairs)
            result["cpu_baseline"] = {
                "value": oracle_tokens_per_s(w, sec, len(pairs)), "unit": UNIT, "cores": blas_threads(),
                "kind": "oracle", "seconds": sec,
                "sample": f"{len(pairs)} of {w.B * w.H} (batch, head) pairs in full, scaled to the whole job"}
    if dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()
    return result if rank == 0 else {}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c5", help="c1..c5 or c5_sweep_n<N>")
    ap.add_argument("--impl", default="csat", choices=["csat", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="skip the short timings of the other workloads")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.workload.startswith("c5_sweep_n"):
        w = wl.sweep_config(int(args.workload[len("c5_sweep_n"):]))
    else:
        w = wl.CONFIGS[args.workload]
    res = run_reference(args, w) if args.impl == "reference" else run_csat(args, w)
    if res:
        print(json.dumps(res))


if __name__ == "__main__":
    main()
