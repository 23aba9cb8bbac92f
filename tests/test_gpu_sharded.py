"""GPU parity of the token-sharded forward (csat_compress_partial, csat_reduce_partials, csat_attend).

One GPU stands in for R ranks by running their steps one after the other on the same context (no kernel waits
for another): every shard's float32 partials, stacked in rank order, the fixed-order sum, then attention and
recovery for every rank's queries.  Checked against the float64 oracle (the parity bar) and against csat_forward
(only the order of the token sum differs: partial sums per shard instead of one running sum)."""
import numpy as np
import pytest
import torch

from oracle import csat_oracle as orc
from paper_2507_02957_b200 import binding, parallel, workloads as wl
from gpu_util import TOL, device_inputs, make_ctx, rel_err, to_np

pytestmark = pytest.mark.gpu
C = wl.CONFIGS

CASES = {
    "bf16_d64_two_batch_elements": (wl.shrink(C["c3"], B=2, H=2, n=784, n_q=300, m=128), 3),
    "bf16_d64_ragged_tokens": (wl.Workload("shard_ragged", 1, 3, 200, 150, 64, 64, "bf16", 4, 0.01, "iid", 61), 2),
    "bf16_d128": (wl.shrink(C["c5"], B=1, H=2, n=2048, n_q=700, m=128), 4),
    "fp32": (wl.shrink(C["c1"], B=2, H=1), 2),
    "fp32_more_ranks_than_shards": (wl.shrink(C["c1"], n=100, n_q=100, m=64), 3),
}


@pytest.mark.parametrize("name", sorted(CASES))
@pytest.mark.parametrize("separate", [False, True])
def test_sharded_forward_matches_oracle_and_unsharded(name, separate):
    w, R = CASES[name]
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w, lam=0.0 if w.name.startswith("c5") else w.lam)
    if separate:
        ctx.set(separate_phi=True)
    phi = to_np(ctx.get_phi())
    lam = binding.csat_get_f64(ctx.h, binding.CSAT_LAMBDA)
    unsharded = ctx.forward(Q, K, V).clone()
    kt_ref, vt_ref = (t.clone() for t in ctx.get_compressed())
    partials = []
    for rank in range(R):
        n0, n_len = parallel.token_shard_range(w.n, R, rank)
        if n_len == 0:
            partials.append(torch.zeros(w.B, w.H, w.m, 2 * w.d, dtype=torch.float32, device="cuda"))
            continue
        partials.append(ctx.compress_partial(K[:, :, n0:n0 + n_len].contiguous(), V[:, :, n0:n0 + n_len].contiguous(), n0))
    ctx.reduce_partials(torch.stack(partials))
    kt, vt = ctx.get_compressed()
    tol_kv = 8e-3 if w.dtype == "bf16" else 1e-5          # one rounding of a differently ordered sum
    assert rel_err(to_np(kt), to_np(kt_ref)) <= tol_kv and rel_err(to_np(vt), to_np(vt_ref)) <= tol_kv
    outs = []
    for rank in range(R):
        q0, q_len = parallel.shard_range(w.n_q, R, rank)
        ctx.set_n_q(q_len)
        outs.append(ctx.attend(Q[:, :, q0:q0 + q_len].contiguous()))
    got = torch.cat(outs, dim=2)
    ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi[:w.H], T=w.T, lam=lam,
                           Phi_V=phi[w.H:] if separate else None)
    assert np.abs(ref).max() > 0
    assert rel_err(to_np(got), ref) <= TOL[w.dtype], name
    assert rel_err(to_np(got), to_np(unsharded)) <= TOL[w.dtype], name
    # the same partials in the same order give the same bits
    ctx.reduce_partials(torch.stack(partials))
    kt2, vt2 = ctx.get_compressed()
    assert torch.equal(kt, kt2) and torch.equal(vt, vt2)
    ctx.close()


def test_sharded_entry_points_refuse_bad_calls():
    ctx = binding.Csat(256, 64, 64, 1, 0, dtype="bf16", T=0)
    K = torch.zeros(1, 1, 128, 64, dtype=torch.bfloat16, device="cuda")
    part = torch.zeros(1, 1, 64, 128, dtype=torch.float32, device="cuda")
    q = torch.zeros(1, 1, 256, 64, dtype=torch.bfloat16, device="cuda")
    lib = binding.load()
    s = torch.cuda.current_stream().cuda_stream
    assert lib.csat_attend(ctx.h, q.data_ptr(), torch.empty_like(q).data_ptr(), s) == 6           # empty workspace
    assert lib.csat_compress_partial(ctx.h, K.data_ptr(), K.data_ptr(), 192, 128, part.data_ptr(), s) == 2   # past n
    assert lib.csat_compress_partial(ctx.h, K.data_ptr(), K.data_ptr(), 4, 128, part.data_ptr(), s) == 2     # misaligned start
    assert lib.csat_reduce_partials(ctx.h, part.data_ptr(), 0, s) == 1
    ctx.compress_partial(K, K, 128)
    ctx.reduce_partials(part[None])
    ctx.attend(q)
    ctx.close()
