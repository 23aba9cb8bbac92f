"""The torch.autograd glue: loss.backward() through csat_attention gives csat_backward's gradients."""
import numpy as np
import pytest
import torch

from oracle import csat_oracle as orc
from paper_2507_02957_b200 import binding, workloads as wl
from gpu_util import TOL, device_inputs, make_ctx, rel_err, to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("save", [True, False], ids=["saving_forward", "recomputing_backward"])
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_autograd_function_matches_the_library_and_the_oracle(dtype, save):
    from paper_2507_02957_b200.autograd import csat_attention
    w = wl.shrink(wl.CONFIGS["c2"], B=2, H=2, n_q=150, lam=0.0) if dtype == "bf16" else wl.shrink(wl.CONFIGS["c1"], B=2, H=2, n=100, n_q=37, m=40, d=32, T=3, lam=0.0)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    q, k, v = (t.clone().requires_grad_(True) for t in (Q, K, V))
    out = csat_attention(ctx, q, k, v, save_for_backward=save)
    G = torch.randn(out.shape, device="cuda", generator=torch.Generator(device="cuda").manual_seed(3)).to(out.dtype)
    (out.float() * G.float()).sum().backward()
    # the same numbers as the library's own calls
    binding.csat_set_i64(ctx.h, binding.CSAT_SAVE_FOR_BACKWARD, 0)
    assert torch.equal(out.detach(), ctx.forward(Q, K, V)) or rel_err(to_np(out.detach()), to_np(ctx.forward(Q, K, V))) <= TOL[dtype]
    dQ, dK, dV = ctx.backward(Q, K, V, G)
    for a, b in zip((q.grad, k.grad, v.grad), (dQ, dK, dV)):
        assert torch.equal(a, b)
    # and the oracle's (lambda = 0: every shrinkage decision is |x| > 0 on both sides)
    ref = orc.csat_backward(inp["Q"], inp["K"], inp["V"], to_np(ctx.get_phi()), to_np(G), T=w.T, lam=0.0)
    for g, rf in zip((q.grad, k.grad, v.grad), ref):
        assert rel_err(to_np(g), rf) <= (2e-2 if dtype == "bf16" else 2e-5)
    ctx.close()


def test_module_owns_a_context():
    from paper_2507_02957_b200.autograd import CsatAttention
    mod = CsatAttention(256, 64, 64, 2, B=1, T=4, lam=0.01, seed=5)
    g = torch.Generator(device="cuda").manual_seed(1)
    Q, K, V = ((torch.randn(1, 2, 256, 64, device="cuda", generator=g) / 8).bfloat16().requires_grad_(True) for _ in range(3))
    out = mod(Q, K, V)
    assert out.shape == (1, 2, 256, 64) and torch.isfinite(out).all()
    out.float().sum().backward()
    assert all(t.grad is not None and torch.isfinite(t.grad).all() for t in (Q, K, V))
