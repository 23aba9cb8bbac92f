"""Seeded synthetic inputs for the CSAT forward (shapes of the paper's workloads).

This module only draws random tensors and rounds them to the storage type. It
holds none of the method's arithmetic (no compression, softmax or recovery), so
both the CUDA path's tests and the CPU oracle may take their inputs from it.

The paper evaluates on image, video and text benchmarks (Experiments section);
those datasets are not used here.  Only their shapes are borrowed: 197 tokens
of a ViT-B/16 image (196 patches + CLS), 196 patches per video frame, 77 text
query tokens, sequence lengths up to 16k.

All arrays are numpy.  Storage types: "fp32" arrays are float32; "bf16" arrays
are returned as float32 arrays whose values are exactly representable in
bfloat16 (round-to-nearest-even), plus helpers to get the 16-bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    n: int          # key/value tokens
    n_q: int        # query tokens
    d: int          # head dimension (the paper's d_k)
    m: int          # measurements
    dtype: str      # "fp32" | "bf16"  (storage type)
    T: int          # recovery iterations
    lam: float      # LASSO weight lambda
    kind: str       # "iid" | "iid_scaled" | "video" | "crossmodal"
    data_seed: int
    phi_seed: int = 0
    frames: int = 1
    patches: int = 0
    sparsity: int = 0   # k of the k-sparse value rows ("crossmodal")
    psi_seed: int = 4242

    @property
    def query_tokens(self) -> int:
        return self.B * self.n_q


CONFIGS = {
    "c1": Workload("c1_tiny_fp32", 1, 1, 256, 256, 64, 64, "fp32", 10, 0.1, "iid", 1001),
    "c2": Workload("c2_vit_b16", 32, 12, 197, 197, 64, 64, "bf16", 10, 0.1, "iid_scaled", 1002),
    "c3": Workload("c3_video", 8, 12, 1568, 1568, 64, 256, "bf16", 20, 0.05, "video", 1003,
                   frames=8, patches=196),
    "c4": Workload("c4_text_to_video", 16, 8, 3136, 77, 64, 392, "bf16", 20, 0.05, "crossmodal", 1004,
                   frames=16, patches=196, sparsity=16),
    "c5": Workload("c5_long", 2, 16, 16384, 16384, 128, 1024, "bf16", 20, 0.05, "iid_scaled", 1005),
}


def sweep_config(n: int) -> Workload:
    """Length-sweep point of the long-sequence workload: m = n/16."""
    return replace(CONFIGS["c5"], name=f"c5_sweep_n{n}", n=n, n_q=n, m=n // 16)


def shrink(w: Workload, **kw) -> Workload:
    """A smaller instance of the same recipe (used by parity tests).  For the frame-structured
    workloads a new n keeps the patches per frame and changes the number of frames."""
    if "n" in kw and w.patches and "frames" not in kw:
        assert kw["n"] % w.patches == 0, "n must stay a whole number of frames"
        kw["frames"] = kw["n"] // w.patches
    return replace(w, **kw)


# ----------------------------------------------------------------------------
# storage rounding
# ----------------------------------------------------------------------------
def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round-to-nearest-even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = (u + 0x7FFF + lsb) >> 16
    # NaN stays NaN (not produced by the generators, kept for safety)
    nan = np.isnan(x)
    r = np.where(nan, 0x7FC0, r)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def round_to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round to the storage type and return the values as float32."""
    x = np.asarray(x, dtype=np.float32)
    if dtype == "fp32":
        return np.ascontiguousarray(x)
    if dtype == "bf16":
        return bf16_bits_to_f32(to_bf16_bits(x)).reshape(x.shape)
    raise ValueError(f"unknown storage dtype {dtype!r}")


# ----------------------------------------------------------------------------
# generators
# ----------------------------------------------------------------------------
def _normal(rng: np.random.Generator, shape, scale=1.0) -> np.ndarray:
    return (rng.standard_normal(shape, dtype=np.float32) * np.float32(scale)).astype(np.float32)


def orthonormal_basis(d: int, seed: int) -> np.ndarray:
    """Fixed random orthonormal d x d basis: Q factor of a Gaussian matrix, columns
    sign-fixed so that diag(R) > 0.  (A draw of a basis, not part of the method.)"""
    rng = np.random.Generator(np.random.PCG64(seed))
    a = rng.standard_normal((d, d))
    q, r = np.linalg.qr(a)
    q = q * np.sign(np.diag(r))[None, :]
    return q.astype(np.float32)


def _redundant_frames(rng, B, H, frames, patches, d) -> np.ndarray:
    """Temporal-redundancy model: one base vector per patch position, every frame
    repeats it with small additive noise.  Token index = frame * patches + patch."""
    base = _normal(rng, (B, H, 1, patches, d))
    noise = _normal(rng, (B, H, frames, patches, d), 0.1)
    return (base + noise).reshape(B, H, frames * patches, d)


def flops(w: Workload, with_psi: bool | None = None) -> dict:
    """Algorithmic floating-point operations of one forward (all B*H pairs), per stage."""
    bh = w.B * w.H
    psi = (w.kind == "crossmodal") if with_psi is None else with_psi
    compress = 4 * w.m * w.n * w.d * bh
    attend = 4 * w.n_q * w.m * w.d * bh
    recover = (2 * w.n_q * w.d * w.d * (w.T + 1) + (2 * w.n_q * w.d * w.d if psi else 0)) * bh if w.T > 0 else 0
    return {"compress": compress, "attend": attend, "recover": recover, "total": compress + attend + recover}


def make_inputs(w: Workload, rounded: bool = True) -> dict:
    """Draw Q, K, V (and Psi for the cross-modal workload) for a workload.

    Returns float32 arrays, rounded to the storage type unless rounded=False (a caller that
    converts with another round-to-nearest-even routine gets the same values):
      Q [B,H,n_q,d], K [B,H,n,d], V [B,H,n,d], Psi [d,d] or None.
    """
    if not rounded:
        w = replace(w, dtype="fp32")
    rng = np.random.Generator(np.random.PCG64(w.data_seed))
    B, H, n, nq, d = w.B, w.H, w.n, w.n_q, w.d
    psi = None
    if w.kind == "iid":
        Q = _normal(rng, (B, H, nq, d))
        K = _normal(rng, (B, H, n, d))
        V = _normal(rng, (B, H, n, d))
    elif w.kind == "iid_scaled":
        s = 1.0 / np.sqrt(d)
        Q = _normal(rng, (B, H, nq, d), s)
        K = _normal(rng, (B, H, n, d), s)
        V = _normal(rng, (B, H, n, d), s)
    elif w.kind == "video":
        assert w.frames * w.patches == n
        Q = _normal(rng, (B, H, nq, d))
        K = _redundant_frames(rng, B, H, w.frames, w.patches, d)
        V = _redundant_frames(rng, B, H, w.frames, w.patches, d)
    elif w.kind == "crossmodal":
        assert w.frames * w.patches == n
        Q = _normal(rng, (B, H, nq, d))
        K = _redundant_frames(rng, B, H, w.frames, w.patches, d)
        psi = orthonormal_basis(d, w.psi_seed)
        # V rows are exactly k-sparse in the basis Psi: V[j] = beta_j Psi^T
        k = w.sparsity
        beta = np.zeros((B * H * n, d), dtype=np.float32)
        keys = rng.random((B * H * n, d), dtype=np.float32)
        support = np.argpartition(keys, k, axis=1)[:, :k]        # uniform k-subsets
        vals = _normal(rng, (B * H * n, k))
        np.put_along_axis(beta, support, vals, axis=1)
        V = (beta @ psi.T).reshape(B, H, n, d).astype(np.float32)
        psi = round_to_storage(psi, w.dtype)
    else:
        raise ValueError(w.kind)
    return {
        "Q": round_to_storage(Q, w.dtype),
        "K": round_to_storage(K, w.dtype),
        "V": round_to_storage(V, w.dtype),
        "Psi": psi,
    }
