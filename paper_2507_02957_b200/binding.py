"""ctypes binding of libcsat.so: the same entry points as include/csat.h, argument marshalling only.

Every step of the CSAT forward runs inside the library's CUDA kernels.  PyTorch is used for
device memory and streams.  There is no CPU path: loading fails loudly if the library cannot be
found or built, and every call raises CsatError on a non-zero status.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

CSAT_OK = 0
ERR_NAMES = {1: "CSAT_ERR_INVALID_ARG", 2: "CSAT_ERR_SHAPE", 3: "CSAT_ERR_ALLOC", 4: "CSAT_ERR_CUDA",
             5: "CSAT_ERR_UNSUPPORTED", 6: "CSAT_ERR_STATE", 7: "CSAT_ERR_TIMEOUT"}
CSAT_BATCH, CSAT_NQ, CSAT_DTYPE, CSAT_T, CSAT_FORCE_SIMT, CSAT_PROFILE, CSAT_ENSEMBLE, CSAT_SEPARATE_PHI = 1, 2, 3, 4, 5, 6, 7, 8
CSAT_KEEP_MASKS = 9
CSAT_HADAMARD_TRANSFORM = 10
CSAT_DEBUG_CANARY = 11
CSAT_WEIGHT_GRADS = 12
CSAT_SAVE_FOR_BACKWARD = 13
CSAT_ENSEMBLE_GAUSSIAN, CSAT_ENSEMBLE_RADEMACHER, CSAT_ENSEMBLE_HADAMARD = 0, 1, 2
KERNEL_NAMES = {0: "decoder_setup", 1: "compress", 2: "attend_recover"}
CSAT_DTYPE_BF16, CSAT_DTYPE_FP32 = 0, 1
CSAT_LAMBDA, CSAT_STEP, CSAT_SCALE = 1, 2, 3

_DTYPES = {"bf16": (CSAT_DTYPE_BF16, torch.bfloat16), "fp32": (CSAT_DTYPE_FP32, torch.float32)}

# name -> (restype, argtypes); must list every symbol include/csat.h declares
_vp, _i64, _u64, _int, _dbl = C.c_void_p, C.c_int64, C.c_uint64, C.c_int, C.c_double
SIGNATURES = {
    "csat_create": (_vp, [_i64, _i64, _i64, _i64, _u64]),
    "csat_destroy": (_int, [_vp]),
    "csat_set_i64": (_int, [_vp, _int, _i64]),
    "csat_get_i64": (_int, [_vp, _int, C.POINTER(_i64)]),
    "csat_set_f64": (_int, [_vp, _int, _dbl]),
    "csat_get_f64": (_int, [_vp, _int, C.POINTER(_dbl)]),
    "csat_set_phi": (_int, [_vp, _vp, _vp]),
    "csat_get_phi": (_int, [_vp, _vp, _vp]),
    "csat_set_dictionary": (_int, [_vp, _vp, _int, _vp]),
    "csat_set_decoder_matrix": (_int, [_vp, _vp, _vp]),
    "csat_set_lista_weights": (_int, [_vp, _vp, _vp, _vp, _int, _vp]),
    "csat_set_lista_layer_weights": (_int, [_vp, _vp, _vp, _vp, _int, _vp]),
    "csat_project_qkv": (_int, [_vp, _vp, _vp, _vp, _i64, _vp, _vp, _vp, _vp]),
    "csat_forward": (_int, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "csat_compress_partial": (_int, [_vp, _vp, _vp, _i64, _i64, _vp, _vp]),
    "csat_reduce_partials": (_int, [_vp, _vp, _int, _vp]),
    "csat_attend": (_int, [_vp, _vp, _vp, _vp]),
    "csat_backward": (_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "csat_forward_host": (_int, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "csat_get_compressed": (_int, [_vp, _vp, _vp, _vp]),
    "csat_get_decoder": (_int, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "csat_get_backward_masks": (_int, [_vp, _vp, _vp]),
    "csat_get_weight_grads": (_int, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "csat_backward_phi": (_int, [_vp, _vp, _vp, _vp, _vp]),
    "csat_get_profile": (_int, [_vp, _i64, _int, C.POINTER(_int), C.POINTER(C.c_float), C.POINTER(_int)]),
    "csat_attend_noalloc": (_int, [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i64, _i64, _i64, _int, _dbl, _vp,
                                   C.c_char_p, C.c_size_t]),
    "csat_selftest_wait_timeout": (_int, [_vp, _i64, _vp]),
    "csat_clear_status": (_int, [_vp, C.POINTER(_int)]),
    "csat_debug_fail_alloc": (_int, [_int]),
    "csat_workspace_bytes": (C.c_size_t, [_vp]),
    "csat_last_launch_count": (_int, [_vp]),
    "csat_last_error": (C.c_char_p, [_vp]),
    "csat_version": (_int, []),
}

_lib = None


class CsatError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"{ERR_NAMES.get(code, code)}: {text}")
        self.code = code


def load() -> C.CDLL:
    """Load (building first if the sources are newer) the in-tree libcsat.so."""
    global _lib
    if _lib is not None:
        return _lib
    try:
        path = _build.build_library()
    except Exception as exc:  # no nvcc and no prebuilt library: there is nothing to fall back to
        if not os.path.exists(_build.LIB):
            raise RuntimeError(f"libcsat.so is missing and could not be built: {exc}") from exc
        path = _build.LIB
    lib = C.CDLL(path)
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(lib, name)          # AttributeError if the library lacks a declared symbol
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _ptr(t):
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to libcsat must be contiguous"
    return C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _check(handle, rc):
    if rc != CSAT_OK:
        raise CsatError(rc, (load().csat_last_error(handle) or b"").decode())


# ---- thin functions, one per C entry point -------------------------------------------------
def csat_version() -> int:
    return load().csat_version()


def csat_create(n, m, d, H, seed):
    h = load().csat_create(n, m, d, H, seed)
    if not h:
        raise CsatError(0, (load().csat_last_error(None) or b"").decode())
    return C.c_void_p(h)


def csat_destroy(h):
    _check(None, load().csat_destroy(h))


def csat_set_i64(h, key, v):
    _check(h, load().csat_set_i64(h, key, int(v)))


def csat_get_i64(h, key) -> int:
    out = _i64()
    _check(h, load().csat_get_i64(h, key, C.byref(out)))
    return out.value


def csat_set_f64(h, key, v):
    _check(h, load().csat_set_f64(h, key, float(v)))


def csat_get_f64(h, key) -> float:
    out = _dbl()
    _check(h, load().csat_get_f64(h, key, C.byref(out)))
    return out.value


def csat_set_phi(h, phi, stream=None):
    _check(h, load().csat_set_phi(h, _ptr(phi), _stream(stream)))


def csat_get_phi(h, phi_out, stream=None):
    _check(h, load().csat_get_phi(h, _ptr(phi_out), _stream(stream)))


def csat_set_dictionary(h, psi, per_head=False, stream=None):
    _check(h, load().csat_set_dictionary(h, _ptr(psi), int(per_head), _stream(stream)))


def csat_set_decoder_matrix(h, D, stream=None):
    _check(h, load().csat_set_decoder_matrix(h, _ptr(D), _stream(stream)))


def csat_set_lista_weights(h, S, Bm, theta, layers, stream=None):
    _check(h, load().csat_set_lista_weights(h, _ptr(S), _ptr(Bm), _ptr(theta), int(layers), _stream(stream)))


def csat_set_lista_layer_weights(h, S, Bm, theta, layers, stream=None):
    _check(h, load().csat_set_lista_layer_weights(h, _ptr(S), _ptr(Bm), _ptr(theta), int(layers), _stream(stream)))


def csat_project_qkv(h, Xq, Xkv, W, d_model, Q, K, V, stream=None):
    _check(h, load().csat_project_qkv(h, _ptr(Xq), _ptr(Xkv), _ptr(W), int(d_model), _ptr(Q), _ptr(K), _ptr(V),
                                      _stream(stream)))


def csat_forward(h, Q, K, V, out, stream=None):
    _check(h, load().csat_forward(h, _ptr(Q), _ptr(K), _ptr(V), _ptr(out), _stream(stream)))


def csat_compress_partial(h, K_shard, V_shard, n0, n_len, partial_out, stream=None):
    _check(h, load().csat_compress_partial(h, _ptr(K_shard), _ptr(V_shard), int(n0), int(n_len), _ptr(partial_out),
                                           _stream(stream)))


def csat_reduce_partials(h, partials, count, stream=None):
    _check(h, load().csat_reduce_partials(h, _ptr(partials), int(count), _stream(stream)))


def csat_attend(h, Q, out, stream=None):
    _check(h, load().csat_attend(h, _ptr(Q), _ptr(out), _stream(stream)))


def csat_backward(h, Q, K, V, dOut, dQ, dK, dV, stream=None):
    _check(h, load().csat_backward(h, _ptr(Q), _ptr(K), _ptr(V), _ptr(dOut), _ptr(dQ), _ptr(dK), _ptr(dV),
                                   _stream(stream)))


def csat_forward_host(h, Qh, Kh, Vh, outh, stream=None):
    _check(h, load().csat_forward_host(h, _ptr(Qh), _ptr(Kh), _ptr(Vh), _ptr(outh), _stream(stream)))


def csat_get_compressed(h, kt_out, vt_out, stream=None):
    _check(h, load().csat_get_compressed(h, _ptr(kt_out), _ptr(vt_out), _stream(stream)))


def csat_get_decoder(h, S_out, B_out, theta_out, mu_out, stream=None):
    _check(h, load().csat_get_decoder(h, _ptr(S_out), _ptr(B_out), _ptr(theta_out), _ptr(mu_out), _stream(stream)))


def csat_get_backward_masks(h, masks_out, stream=None):
    _check(h, load().csat_get_backward_masks(h, _ptr(masks_out), _stream(stream)))


def csat_get_weight_grads(h, dS, dB, dtheta, dPsi=None, stream=None):
    _check(h, load().csat_get_weight_grads(h, _ptr(dS), _ptr(dB), _ptr(dtheta), _ptr(dPsi) if dPsi is not None else None,
                                           _stream(stream)))


def csat_backward_phi(h, K, V, dPhi, stream=None):
    _check(h, load().csat_backward_phi(h, _ptr(K), _ptr(V), _ptr(dPhi), _stream(stream)))


def csat_get_profile(h, call_index):
    """[(kernel id, milliseconds), ...] of one recorded forward call."""
    cap = 8
    ids, ms, cnt = (_int * cap)(), (C.c_float * cap)(), _int()
    _check(h, load().csat_get_profile(h, call_index, cap, ids, ms, C.byref(cnt)))
    return [(ids[i], ms[i]) for i in range(min(cnt.value, cap))]


NOALLOC_SCRATCH_BYTES = 8 << 20


def csat_attend_noalloc(Q, K, V, phi, out, scale=0.0, stream=None):
    """Compressed attention with recovery disabled, for callers that must not allocate device memory:
    the K~|V~ scratch is a fixed array inside the library (see include/csat.h).  Shapes are read from
    the tensors: Q [B,H,n_q,d], K,V [B,H,n,d], phi [H,m,n], out [B,H,n_q,d]; nothing is allocated here."""
    B, H, nq, d = Q.shape
    n, m = K.shape[2], phi.shape[1]
    code = CSAT_DTYPE_FP32 if Q.dtype == torch.float32 else CSAT_DTYPE_BF16
    err = C.create_string_buffer(512)
    rc = load().csat_attend_noalloc(_ptr(Q), _ptr(K), _ptr(V), _ptr(phi), _ptr(out), B, H, n, nq, m, d, code,
                                    float(scale), _stream(stream), err, len(err))
    if rc != CSAT_OK:
        raise CsatError(rc, err.value.decode())
    return out


def csat_selftest_wait_timeout(h, limit_us, stream=None) -> int:
    """Returns the status code (CSAT_ERR_TIMEOUT = 7 when the bounded wait reported its time-out as it must)."""
    return load().csat_selftest_wait_timeout(h, int(limit_us), _stream(stream))


def csat_clear_status(h) -> int:
    code = _int()
    _check(h, load().csat_clear_status(h, C.byref(code)))
    return code.value


def csat_debug_fail_alloc(countdown: int) -> int:
    """Test aid: the countdown-th device allocation from now on fails (0 = off)."""
    return load().csat_debug_fail_alloc(int(countdown))


def csat_workspace_bytes(h) -> int:
    return load().csat_workspace_bytes(h)


def csat_last_launch_count(h) -> int:
    return load().csat_last_launch_count(h)


def csat_last_error(h) -> str:
    return (load().csat_last_error(h) or b"").decode()


# ---- convenience wrapper: owns a handle, allocates result tensors with torch ------------------
class Csat:
    """A CSAT context.  Tensors are torch CUDA tensors of the context's dtype."""

    def __init__(self, n, m, d, H, seed=0, *, B=1, n_q=None, dtype="bf16", T=10, lam=0.1, step=0.0, scale=0.0):
        if not torch.cuda.is_available():
            raise RuntimeError("libcsat needs a CUDA device (sm_100a); there is no CPU path")
        self.n, self.m, self.d, self.H, self.B = n, m, d, H, B
        self.n_q = n if n_q is None else n_q
        self.dtype_name = dtype
        self.code, self.torch_dtype = _DTYPES[dtype]
        self.h = csat_create(n, m, d, H, seed)
        try:
            if self.code != CSAT_DTYPE_BF16:
                csat_set_i64(self.h, CSAT_DTYPE, self.code)
            csat_set_i64(self.h, CSAT_BATCH, B)
            csat_set_i64(self.h, CSAT_NQ, self.n_q)
            csat_set_i64(self.h, CSAT_T, T)
            csat_set_f64(self.h, CSAT_LAMBDA, lam)
            csat_set_f64(self.h, CSAT_STEP, step)
            csat_set_f64(self.h, CSAT_SCALE, scale)
        except Exception:
            self.close()
            raise

    def close(self):
        if getattr(self, "h", None):
            csat_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set(self, *, T=None, lam=None, step=None, scale=None, force_simt=None, ensemble=None, separate_phi=None,
            hadamard_transform=None):
        if hadamard_transform is not None:
            csat_set_i64(self.h, CSAT_HADAMARD_TRANSFORM, int(bool(hadamard_transform)))
        if separate_phi is not None:
            csat_set_i64(self.h, CSAT_SEPARATE_PHI, int(bool(separate_phi)))
            self.phi_heads = self.H * (2 if separate_phi else 1)
        if ensemble is not None:
            csat_set_i64(self.h, CSAT_ENSEMBLE, {"gaussian": 0, "rademacher": 1, "hadamard": 2}[ensemble])
        if T is not None:
            csat_set_i64(self.h, CSAT_T, T)
        if lam is not None:
            csat_set_f64(self.h, CSAT_LAMBDA, lam)
        if step is not None:
            csat_set_f64(self.h, CSAT_STEP, step)
        if scale is not None:
            csat_set_f64(self.h, CSAT_SCALE, scale)
        if force_simt is not None:
            csat_set_i64(self.h, CSAT_FORCE_SIMT, int(force_simt))

    def _new(self, *shape, dtype=None):
        return torch.empty(*shape, dtype=dtype or self.torch_dtype, device="cuda")

    def forward(self, Q, K, V, out=None):
        assert Q.shape == (self.B, self.H, self.n_q, self.d) and Q.dtype == self.torch_dtype and Q.is_cuda
        assert K.shape == (self.B, self.H, self.n, self.d) and K.dtype == self.torch_dtype and K.is_cuda
        assert V.shape == K.shape and V.dtype == self.torch_dtype and V.is_cuda
        if out is None:
            out = self._new(self.B, self.H, self.n_q, self.d)
        csat_forward(self.h, Q, K, V, out)
        return out

    def forward_host(self, Qh, Kh, Vh, outh):
        for t in (Qh, Kh, Vh, outh):
            assert not t.is_cuda and t.dtype == self.torch_dtype
        csat_forward_host(self.h, Qh, Kh, Vh, outh)
        return outh

    def get_phi(self):
        phi = self._new(getattr(self, "phi_heads", self.H), self.m, self.n)
        csat_get_phi(self.h, phi)
        return phi

    def set_phi(self, phi):
        assert phi.shape == (getattr(self, "phi_heads", self.H), self.m, self.n) and phi.dtype == self.torch_dtype
        csat_set_phi(self.h, phi.contiguous())

    def set_dictionary(self, psi):
        if psi is None:
            csat_set_dictionary(self.h, None)
            return
        assert psi.dtype == self.torch_dtype and psi.shape[-2:] == (self.d, self.d)
        csat_set_dictionary(self.h, psi.contiguous(), per_head=(psi.dim() == 3))

    def set_decoder_matrix(self, D):
        if D is not None:
            assert D.shape == (self.H, self.d, self.d) and D.dtype == self.torch_dtype
            D = D.contiguous()
        csat_set_decoder_matrix(self.h, D)

    def set_lista_weights(self, S, Bm=None, theta=None):
        """Supplied LISTA weights: S, Bm [H,d,d] (context dtype), theta [layers,H] or [H] float32; S=None restores
        the ISTA-derived decoder."""
        self._per_layer_weights = False
        if S is None:
            csat_set_lista_weights(self.h, None, None, None, 1)
            return
        assert S.shape == (self.H, self.d, self.d) and Bm.shape == S.shape and S.dtype == self.torch_dtype == Bm.dtype
        theta = theta.reshape(-1, self.H).to(torch.float32).contiguous()
        csat_set_lista_weights(self.h, S.contiguous(), Bm.contiguous(), theta, theta.shape[0])

    def compress_partial(self, K_shard, V_shard, n0):
        """float32 partial sums [B,H,m,2d] of K~|V~ for the token shard that starts at token n0."""
        assert K_shard.shape == V_shard.shape and K_shard.shape[:2] == (self.B, self.H) and K_shard.shape[3] == self.d
        out = self._new(self.B, self.H, self.m, 2 * self.d, dtype=torch.float32)
        csat_compress_partial(self.h, K_shard, V_shard, n0, K_shard.shape[2], out)
        return out

    def reduce_partials(self, partials):
        """partials [count,B,H,m,2d] float32, summed in the order given into the workspace."""
        assert partials.dtype == torch.float32 and partials.shape[1:] == (self.B, self.H, self.m, 2 * self.d)
        csat_reduce_partials(self.h, partials.contiguous(), partials.shape[0])

    def attend(self, Q, out=None):
        """Attention and recovery for Q [B,H,n_q,d] against the K~|V~ in the workspace."""
        assert Q.shape == (self.B, self.H, self.n_q, self.d) and Q.dtype == self.torch_dtype and Q.is_cuda
        if out is None:
            out = self._new(self.B, self.H, self.n_q, self.d)
        csat_attend(self.h, Q, out)
        return out

    def set_n_q(self, n_q):
        csat_set_i64(self.h, CSAT_NQ, n_q)
        self.n_q = n_q

    def backward(self, Q, K, V, dOut):
        """Gradients of forward(Q, K, V) with respect to Q, K, V for the output gradient dOut."""
        dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
        csat_backward(self.h, Q, K, V, dOut, dQ, dK, dV)
        return dQ, dK, dV

    def backward_masks(self):
        """The shrinkage decisions of the most recent backward (CSAT_KEEP_MASKS = 1): int32 [B,H,n_q,d], bit t of a
        word = |x_t| > theta_t."""
        out = self._new(self.B, self.H, self.n_q, self.d, dtype=torch.int32)
        csat_get_backward_masks(self.h, out)
        return out

    def backward_phi(self, K, V):
        """Gradient with respect to the measurement matrices from the most recent backward's dK~, dV~ and the same K, V:
        float32 [H, m, n] ([2H, m, n] with separate Phi_K / Phi_V)."""
        heads = self.H * (2 if csat_get_i64(self.h, CSAT_SEPARATE_PHI) else 1)
        out = self._new(heads, self.m, self.n, dtype=torch.float32)
        csat_backward_phi(self.h, K, V, out)
        return out

    def weight_grads(self):
        """Gradients with respect to the decoder's parameters from the most recent backward (CSAT_WEIGHT_GRADS = 1):
        dS [H,d,d], dB [H,d,d] ([T,H,d,d] after set_lista_layer_weights), dtheta [T,H], dPsi [d,d] (float32)."""
        T = csat_get_i64(self.h, CSAT_T)
        lead = (T, self.H) if getattr(self, "_per_layer_weights", False) else (self.H,)
        dS = self._new(*lead, self.d, self.d, dtype=torch.float32)
        dB = self._new(*lead, self.d, self.d, dtype=torch.float32)
        dth = self._new(T, self.H, dtype=torch.float32)
        dPsi = self._new(self.d, self.d, dtype=torch.float32)
        csat_get_weight_grads(self.h, dS, dB, dth, dPsi)
        return dS, dB, dth, dPsi

    def project_qkv(self, X, W, Xkv=None):
        """Q, K, V [B,H,tokens,d] from tokens X [B,n_q,d_model] (and Xkv [B,n,d_model] for cross-attention; default X)
        and W [d_model, 3*H*d] = [W^Q heads | W^K heads | W^V heads]."""
        Xkv = X if Xkv is None else Xkv
        dm = X.shape[-1]
        assert X.shape == (self.B, self.n_q, dm) and Xkv.shape == (self.B, self.n, dm)
        assert W.shape == (dm, 3 * self.H * self.d) and X.dtype == self.torch_dtype == W.dtype == Xkv.dtype
        Q = self._new(self.B, self.H, self.n_q, self.d)
        K = self._new(self.B, self.H, self.n, self.d)
        V = self._new(self.B, self.H, self.n, self.d)
        csat_project_qkv(self.h, X, Xkv, W, dm, Q, K, V)
        return Q, K, V

    def set_lista_layer_weights(self, S, Bm, theta):
        """Untied layers: S, Bm [layers,H,d,d] (context dtype), theta [layers,H] float32."""
        L = S.shape[0]
        assert S.shape == (L, self.H, self.d, self.d) and Bm.shape == S.shape and S.dtype == self.torch_dtype == Bm.dtype
        theta = theta.to(torch.float32).contiguous()
        assert theta.shape == (L, self.H)
        csat_set_lista_layer_weights(self.h, S.contiguous(), Bm.contiguous(), theta, L)
        self._per_layer_weights = True

    def get_compressed(self):
        kt = self._new(self.B, self.H, self.m, self.d)
        vt = self._new(self.B, self.H, self.m, self.d)
        csat_get_compressed(self.h, kt, vt)
        return kt, vt

    def get_decoder(self):
        S = self._new(self.H, self.d, self.d, dtype=torch.float32)
        Bm = self._new(self.H, self.d, self.d, dtype=torch.float32)
        th = self._new(self.H, dtype=torch.float32)
        mu = self._new(self.H, dtype=torch.float32)
        csat_get_decoder(self.h, S, Bm, th, mu)
        return S, Bm, th, mu

    @property
    def launches(self) -> int:
        return csat_last_launch_count(self.h)

    @property
    def workspace_bytes(self) -> int:
        return csat_workspace_bytes(self.h)
