"""torch.autograd glue for the CSAT library: marshalling only.

`csat_attention(ctx, Q, K, V)` runs `csat_forward` through a `binding.Csat` context and, under autograd, registers
`csat_backward` as its backward, so that the compressed-sensing attention can sit inside a torch model.  With
`save_for_backward=True` (the default) the forward keeps what the backward needs (CSAT_SAVE_FOR_BACKWARD), and the
backward starts from it instead of recomputing.  Every step of the path runs in the library's kernels; nothing here
computes.

The gradients with respect to the decoder's parameters and to the measurement matrices are not torch leaves of this
function: after `loss.backward()` fetch them from the context (`ctx.weight_grads()` with CSAT_WEIGHT_GRADS set,
`ctx.backward_phi(K, V)`).
"""
import torch

from . import binding


class _CsatFunction(torch.autograd.Function):
    @staticmethod
    def forward(fn_ctx, csat, Q, K, V, save):
        Q, K, V = Q.contiguous(), K.contiguous(), V.contiguous()
        binding.csat_set_i64(csat.h, binding.CSAT_SAVE_FOR_BACKWARD, 1 if save else 0)
        out = csat.forward(Q, K, V)
        fn_ctx.csat = csat
        fn_ctx.save_for_backward(Q, K, V)
        return out

    @staticmethod
    def backward(fn_ctx, dOut):
        Q, K, V = fn_ctx.saved_tensors
        dQ, dK, dV = fn_ctx.csat.backward(Q, K, V, dOut.contiguous())
        return None, dQ, dK, dV, None


def csat_attention(csat, Q, K, V, save_for_backward=True):
    """Compressed-sensing attention of Q [B,H,n_q,d], K, V [B,H,n,d] through the context `csat` (a binding.Csat of that
    shape and dtype), differentiable with respect to Q, K, V.  One forward of a context may be in flight between this
    call and its backward (the context holds the saved state)."""
    return _CsatFunction.apply(csat, Q, K, V, save_for_backward)


class CsatAttention(torch.nn.Module):
    """The same as a module that owns its context: CsatAttention(n, m, d, H, B=..., n_q=..., T=..., lam=..., seed=...).
    forward(Q, K, V) -> [B,H,n_q,d]."""

    def __init__(self, n, m, d, H, *, B=1, n_q=None, T=10, lam=0.1, seed=0, dtype="bf16", save_for_backward=True):
        super().__init__()
        self.csat = binding.Csat(n, m, d, H, seed, B=B, n_q=n_q if n_q is not None else n, dtype=dtype, T=T, lam=lam)
        self.save = save_for_backward

    def forward(self, Q, K, V):
        return csat_attention(self.csat, Q, K, V, self.save)
