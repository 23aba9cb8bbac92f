"""GPU tests of the library's behaviour around its compute kernels: the host-buffer forward with more batch
elements than it has pipeline events, and a context whose re-allocation failed."""
import pytest
import torch

from paper_2507_02957_b200 import binding, workloads as wl
from gpu_util import device_inputs, make_ctx

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,H", [(65, 1), (70, 3), (3, 50)])
def test_host_forward_with_more_pairs_than_pipeline_chunks(B, H):
    """The pipelined host-buffer forward cuts the job into at most 64 runs of (batch, head) pairs; with more batch
    elements than that a run spans several of them.  The call must return and equal csat_forward bit for bit."""
    w = wl.Workload("many_pairs", B, H, 128, 96, 64, 64, "bf16", 2, 0.01, "iid", 51)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    ref = ctx.forward(Q, K, V).cpu()
    Qh, Kh, Vh = (t.cpu().pin_memory() for t in (Q, K, V))
    oh = torch.full_like(Qh, float("nan")).pin_memory()
    ctx.forward_host(Qh, Kh, Vh, oh)
    assert torch.equal(oh, ref)
    ctx.close()


def test_failed_reallocation_is_refused_until_a_setter_succeeds():
    """A setter whose cudaMalloc fails must not leave a context that launches kernels on null buffers: compute calls
    and getters answer CSAT_ERR_STATE until a re-allocating setter succeeds.  The failure is injected on the host."""
    w = wl.Workload("realloc", 2, 2, 256, 256, 64, 64, "bf16", 3, 0.01, "iid", 52)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    ref = ctx.forward(Q, K, V).clone()
    lib = binding.load()
    s = torch.cuda.current_stream().cuda_stream
    out = torch.empty_like(Q)
    for key, bad_value, good_value in [(binding.CSAT_BATCH, 5, 2), (binding.CSAT_SEPARATE_PHI, 1, 0),
                                       (binding.CSAT_DTYPE, binding.CSAT_DTYPE_FP32, binding.CSAT_DTYPE_BF16)]:
        for countdown in (1, 2):
            assert binding.csat_debug_fail_alloc(countdown) == 0
            rc = lib.csat_set_i64(ctx.h, key, bad_value)
            binding.csat_debug_fail_alloc(0)
            if key == binding.CSAT_BATCH and countdown == 2:
                assert rc == 0                                        # that setter allocates once: nothing failed
            else:
                assert rc == 3, (key, countdown, rc)                  # CSAT_ERR_ALLOC
                assert lib.csat_forward(ctx.h, Q.data_ptr(), K.data_ptr(), V.data_ptr(), out.data_ptr(), s) == 6
                assert "re-allocate" in binding.csat_last_error(ctx.h)
                phi = torch.empty(2 * w.H, w.m, w.n, dtype=torch.float32, device="cuda")
                assert lib.csat_get_phi(ctx.h, phi.data_ptr(), s) == 6
                assert lib.csat_backward(ctx.h, *(t.data_ptr() for t in (Q, K, V, Q, out, out, out)), s) == 6
            binding.csat_set_i64(ctx.h, key, good_value)              # succeeds and repairs the context
            torch.cuda.synchronize()
            assert torch.equal(ctx.forward(Q, K, V), ref), (key, countdown)
    ctx.close()


@pytest.mark.parametrize("shape", [(1, 3, 131, 67, 64, 67), (2, 2, 203, 37, 128, 139), (3, 1, 392, 200, 64, 200),
                                   (1, 2, 100, 50, 40, 41)])
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_workspace_canary_finds_no_unwritten_row(shape, dtype):
    """CSAT_DEBUG_CANARY fills the K~|V~ workspace with NaN before every compression: on ragged shapes (measurement and
    token counts that are no multiples of the tiles, odd batches, both kernel families) the forward and the backward
    must stay finite and give the same bits as without the canary, i.e. every workspace row that is read was
    written by the same call."""
    B, H, n, nq, d, m = shape
    w = wl.Workload("canary", B, H, n, nq, d, m, dtype, 3, 0.01, "iid", 57)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    ref = ctx.forward(Q, K, V).clone()
    G = torch.randn_like(Q)
    gref = [t.clone() for t in ctx.backward(Q, K, V, G)]
    binding.csat_set_i64(ctx.h, binding.CSAT_DEBUG_CANARY, 1)
    assert binding.csat_get_i64(ctx.h, binding.CSAT_DEBUG_CANARY) == 1
    out = ctx.forward(Q, K, V)
    assert torch.isfinite(out).all() and torch.equal(out, ref)
    for a, b in zip(ctx.backward(Q, K, V, G), gref):
        assert torch.isfinite(a).all() and torch.equal(a, b)
    ctx.close()
