"""CPU oracle for the seeded Gaussian measurement matrix Phi.  TEST INFRASTRUCTURE.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this.

The paper draws Phi from a sub-Gaussian ensemble (Gaussian entries first among its examples; section
"Mathematical Framework", the sentence after the compression equation) and fixes
neither generator nor variance.  The reading implemented here (and, separately,
by the CUDA library):

  * entries i.i.d. N(0, 1/m), one Phi per head, Phi_K = Phi_V = Phi;
  * Philox4x32-10 (Salmon et al., SC'11), key = (seed low 32 bits, seed high 32 bits);
    element e = (h*m + r)*n + j uses the block with counter (q low, q high, 0, 0),
    q = e // 4, and takes Gaussian number e % 4 of that block;
  * the four 32-bit outputs u0..u3 become uniforms U = ((u >> 9) + 0.5) * 2^-23
    (exact in float32), Box-Muller on (U0,U1) gives g0 = r cos(2 pi U1), g1 = r sin(2 pi U1)
    with r = sqrt(-2 ln U0); (U2,U3) give g2, g3 likewise;
  * Phi[h,r,j] = g / sqrt(m), then rounded to the storage type by the caller.

Everything after the integer stage is float64 here.  The integer stage is pinned by the
published known-answer vectors of Philox4x32-10; the Gaussian stage by moment and
distribution tests.
"""
from __future__ import annotations

import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = np.uint64(0x9E3779B9)
_W1 = np.uint64(0xBB67AE85)
_MASK = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Philox4x32 with 10 rounds.  Inputs: arrays (or scalars) of 32-bit words held in uint64.
    Returns the four output words as uint64 arrays with values < 2^32."""
    c0, c1, c2, c3 = (np.asarray(c, dtype=np.uint64) & _MASK for c in (c0, c1, c2, c3))
    k0 = np.asarray(k0, dtype=np.uint64) & _MASK
    k1 = np.asarray(k1, dtype=np.uint64) & _MASK
    for rnd in range(10):
        p0 = _M0 * c0                      # 32x32 -> 64 bit products (fit in uint64)
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _S32, p0 & _MASK
        hi1, lo1 = p1 >> _S32, p1 & _MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0), lo1, (hi0 ^ c3 ^ k1), lo0
        if rnd != 9:
            k0 = (k0 + _W0) & _MASK
            k1 = (k1 + _W1) & _MASK
    return c0, c1, c2, c3


def _uniform23(u):
    """U = ((u >> 9) + 0.5) * 2^-23, strictly inside (0, 1)."""
    return ((u >> np.uint64(9)).astype(np.float64) + 0.5) * (2.0 ** -23)


def gaussian_block(q, seed: int):
    """The four standard normal numbers of Philox block q (q: uint64 array)."""
    q = np.asarray(q, dtype=np.uint64)
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    u0, u1, u2, u3 = philox4x32_10(q & _MASK, q >> _S32, 0, 0, seed & 0xFFFFFFFF, seed >> 32)
    out = []
    for ua, ub in ((u0, u1), (u2, u3)):
        r = np.sqrt(-2.0 * np.log(_uniform23(ua)))
        ang = 2.0 * np.pi * _uniform23(ub)
        out.append(r * np.cos(ang))
        out.append(r * np.sin(ang))
    return out  # [g0, g1, g2, g3]


def gaussian_elements(e, seed: int) -> np.ndarray:
    """Standard normal number assigned to flat element indices e (any shape)."""
    e = np.asarray(e, dtype=np.uint64)
    g = np.stack(gaussian_block(e >> np.uint64(2), seed), axis=-1)
    return np.take_along_axis(g, (e & np.uint64(3)).astype(np.int64)[..., None], axis=-1)[..., 0]


def phi_gaussian(H: int, m: int, n: int, seed: int, heads=None) -> np.ndarray:
    """Phi [H,m,n] float64 (unrounded): Phi[h,r,j] = g((h*m + r)*n + j) / sqrt(m)."""
    heads = range(H) if heads is None else heads
    out = np.empty((len(heads), m, n), dtype=np.float64)
    for i, h in enumerate(heads):
        e = (np.uint64(h) * np.uint64(m) * np.uint64(n)
             + np.arange(m * n, dtype=np.uint64)).reshape(m, n)
        out[i] = gaussian_elements(e, seed) / np.sqrt(np.float64(m))
    return out


def phi_rademacher(H: int, m: int, n: int, seed: int, heads=None) -> np.ndarray:
    """Rademacher ensemble (the paper's second example of a sub-Gaussian measurement matrix):
    Phi[h,r,j] = +-1/sqrt(m), float64 (unrounded).

    Reading (the paper fixes no generator): element e = (h*m + r)*n + j takes bit e % 32 of word (e // 32) % 4
    of the Philox4x32-10 block with counter (q low, q high, 1, 0), q = e // 128, key = seed; a set bit means
    -1/sqrt(m).  (The third counter word is 1 so that the stream differs from the Gaussian ensemble's.)
    """
    heads = range(H) if heads is None else heads
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    out = np.empty((len(heads), m, n), dtype=np.float64)
    for i, h in enumerate(heads):
        e = np.uint64(h) * np.uint64(m) * np.uint64(n) + np.arange(m * n, dtype=np.uint64)
        q = e >> np.uint64(7)
        words = np.stack(philox4x32_10(q & _MASK, q >> _S32, 1, 0, seed & 0xFFFFFFFF, seed >> 32), axis=-1)
        word = np.take_along_axis(words, ((e >> np.uint64(5)) & np.uint64(3)).astype(np.int64)[:, None], axis=-1)[:, 0]
        bit = (word >> (e & np.uint64(31))) & np.uint64(1)
        out[i] = ((1.0 - 2.0 * bit.astype(np.float64)) / np.sqrt(np.float64(m))).reshape(m, n)
    return out


def hadamard_rows(H: int, m: int, n: int, seed: int):
    """Row indices i_r of the subsampled Hadamard ensemble: N = smallest power of two >= n; for head h,
    i_r = (a r + b) mod N with a = 2 u0 + 1 (odd, so r -> i_r is injective for r < N) and b = u1, where u0, u1
    are the first two words of the Philox block with counter (h, 0, 3, 0).  Returns (N, rows [H, m])."""
    N = 1
    while N < n:
        N *= 2
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    rows = np.empty((H, m), dtype=np.int64)
    for h in range(H):
        u0, u1, _, _ = philox4x32_10(h, 0, 3, 0, seed & 0xFFFFFFFF, seed >> 32)
        a, b = 2 * int(u0) + 1, int(u1)
        rows[h] = [(a * r + b) % N for r in range(m)]
    return N, rows


def phi_hadamard(H: int, m: int, n: int, seed: int, heads=None) -> np.ndarray:
    """Structured Hadamard ensemble (the paper's third example): m rows of the N x N Sylvester-Hadamard matrix
    W (W[i,j] = (-1)^popcount(i & j)), columns truncated to n, with a random sign per column:
        Phi[h,r,j] = s[h,j] * W[i_r, j] / sqrt(m),   float64 (unrounded),
    rows i_r from hadamard_rows, column signs s[h,j] = -1 where bit e % 32 of word (e // 32) % 4 of the Philox
    block with counter (e // 128, 0, 2, 0) is set, e = h*n + j.  Needs m <= N."""
    heads = range(H) if heads is None else heads
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    N, rows = hadamard_rows(H, m, n, seed)
    assert m <= N
    out = np.empty((len(heads), m, n), dtype=np.float64)
    j = np.arange(n, dtype=np.uint64)
    for i, h in enumerate(heads):
        e = np.uint64(h) * np.uint64(n) + j
        q = e >> np.uint64(7)
        words = np.stack(philox4x32_10(q & _MASK, q >> _S32, 2, 0, seed & 0xFFFFFFFF, seed >> 32), axis=-1)
        word = np.take_along_axis(words, ((e >> np.uint64(5)) & np.uint64(3)).astype(np.int64)[:, None], axis=-1)[:, 0]
        s = 1.0 - 2.0 * ((word >> (e & np.uint64(31))) & np.uint64(1)).astype(np.float64)
        for r in range(m):
            x = np.uint64(rows[h, r]) & j
            par = np.zeros(n, dtype=np.uint64)
            for sh in range(40):                                    # parity of popcount, bit by bit
                par ^= (x >> np.uint64(sh)) & np.uint64(1)
            out[i, r] = s * (1.0 - 2.0 * par.astype(np.float64)) / np.sqrt(np.float64(m))
    return out
