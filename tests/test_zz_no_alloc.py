"""csat_attend_noalloc: compressed attention for callers that must not allocate device memory.

Such callers (code running inside another framework's sealed memory plan, real-time loops that cannot
take cudaMalloc's implicit synchronisation, processes with a fixed memory budget) cannot use
csat_create/csat_forward, whose K~|V~ workspace is allocated.  The entry point keeps that scratch in a
fixed array inside the library.  This test calls it through the C-ABI twice in a row (the array is shared
and keeps the previous call's contents, so the second call must not be disturbed by the first) and checks
each result against csat_forward with recovery disabled on the same inputs and the same Phi, and (so that the
agreement of two CUDA paths is not the only evidence) against the float64 oracle's compressed attention.

The file name sorts last so that a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import csat_oracle as orc
from paper_2507_02957_b200 import binding, workloads as wl
from gpu_util import TOL, device_inputs, make_ctx, rel_err, to_np

pytestmark = pytest.mark.gpu

CASES = [
    wl.CONFIGS["c1"],                                                             # float32, 256 tokens
    wl.Workload("noalloc_ragged_bf16", 2, 3, 203, 67, 40, 41, "bf16", 0, 0.0, "iid", 91),
]


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    expected, got = [], []
    for w in CASES:
        inp = wl.make_inputs(w)
        Q, K, V, _ = device_inputs(w, inp)
        ctx = make_ctx(w, T=0)
        phi = ctx.get_phi()
        expected.append(ctx.forward(Q, K, V).clone())
        ctx.close()
        out = torch.full_like(Q, float("nan"))
        binding.csat_attend_noalloc(Q, K, V, phi, out)
        got.append((w, out, inp, to_np(phi)))
    torch.cuda.synchronize()
    for (w, out, inp, phi), ref in zip(got, expected):
        assert torch.isfinite(out).all()
        assert rel_err(to_np(out), to_np(ref)) <= TOL[w.dtype], w.name
        oracle = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi, T=0, lam=0.0)
        assert rel_err(to_np(out), oracle) <= TOL[w.dtype], w.name


def test_sizes_beyond_the_built_in_scratch_are_refused():
    d, m, H = 64, 1024, 40                       # 40 * 1024 * 128 * 2 bytes = 10 MiB > 8 MiB
    assert H * m * 2 * d * 2 > binding.NOALLOC_SCRATCH_BYTES
    Q = torch.zeros(1, H, 8, d, dtype=torch.bfloat16, device="cuda")
    K = torch.zeros(1, H, m, d, dtype=torch.bfloat16, device="cuda")
    phi = torch.zeros(H, m, m, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.CsatError) as ei:
        binding.csat_attend_noalloc(Q, K, K.clone(), phi, torch.empty_like(Q))
    assert ei.value.code == 2 and "scratch" in str(ei.value)
    # still usable afterwards
    w = CASES[1]
    inp = wl.make_inputs(w)
    Qd, Kd, Vd, _ = device_inputs(w, inp)
    ctx = make_ctx(w, T=0)
    phi = ctx.get_phi()
    ref = ctx.forward(Qd, Kd, Vd)
    out = binding.csat_attend_noalloc(Qd, Kd, Vd, phi, torch.empty_like(Qd))
    assert rel_err(to_np(out), to_np(ref)) <= TOL[w.dtype]
    ctx.close()
