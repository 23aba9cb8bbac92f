// Seeded Gaussian measurement matrices Phi_h in R^{m x n}, entries N(0, 1/m).
// Paper: compression equation and the sentence after it (Phi is drawn from a sub-Gaussian ensemble; Gaussian entries are the default).
// The paper fixes no generator: this library uses Philox4x32-10 (Salmon et al., SC'11) keyed by the
// 64-bit seed, counter = flat element index / 4, and Box-Muller on 23-bit uniforms.
#include "csat_internal.h"

namespace csat {
namespace {

struct U4 { uint32_t x, y, z, w; };

__device__ __forceinline__ U4 philox4x32_10(U4 c, uint32_t k0, uint32_t k1) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(M0, c.x), lo0 = M0 * c.x;
    const uint32_t hi1 = __umulhi(M1, c.z), lo1 = M1 * c.z;
    c = U4{hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0};
    k0 += W0;
    k1 += W1;
  }
  return c;
}

// U = ((u >> 9) + 0.5) * 2^-23 : exact in float, strictly inside (0,1)
__device__ __forceinline__ float uniform23(uint32_t u) {
  return (static_cast<float>(u >> 9) + 0.5f) * 1.1920928955078125e-07f;
}

__device__ __forceinline__ void box_muller(uint32_t ua, uint32_t ub, float& g0, float& g1) {
  const float r = sqrtf(-2.0f * logf(uniform23(ua)));
  float s, c;
  sincospif(2.0f * uniform23(ub), &s, &c);
  g0 = r * c;
  g1 = r * s;
}

template <typename T> __device__ __forceinline__ T to_storage(float v);
template <> __device__ __forceinline__ float to_storage<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 to_storage<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// One thread per Philox block = 4 consecutive elements of the UNPADDED index space e = (h*m + r)*n + j.
template <typename T>
__global__ void phi_gen_kernel(T* __restrict__ phi, int64_t total, int64_t n, int64_t n_pad, float inv_sqrt_m,
                               uint32_t k0, uint32_t k1) {
  const int64_t nblocks = (total + 3) >> 2;
  for (int64_t q = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; q < nblocks;
       q += (int64_t)gridDim.x * blockDim.x) {
    const U4 u = philox4x32_10(U4{(uint32_t)q, (uint32_t)(q >> 32), 0u, 0u}, k0, k1);
    float g[4];
    box_muller(u.x, u.y, g[0], g[1]);
    box_muller(u.z, u.w, g[2], g[3]);
    const int64_t e0 = q << 2;
    int64_t row = e0 / n;
    int64_t j = e0 - row * n;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (e0 + i < total) phi[row * n_pad + j] = to_storage<T>(g[i] * inv_sqrt_m);
      if (++j == n) { j = 0; ++row; }
    }
  }
}

// bf16 storage, n % 8 == 0: the same Philox stream and the same Box-Muller pairing, with arithmetic sized for a
// 16-bit result (the stored value has 8 bits of mantissa; everything below is accurate to ~1e-6 relative, so the
// rounded value differs from the exactly computed one only where that lies within 1e-6 of a rounding boundary):
//   radius  sqrt(-2 ln u / m) = sqrt.approx(c log2 u), c = -2 ln 2 / m (the 1/sqrt(m) scale folded in);
//   angle   x = 2 u in (0, 2) half-turns: k = nearest multiple of 1/2, f = x - k / 2 in [-1/4, 1/4] (exact),
//           sin(pi f), cos(pi f) by odd / even polynomials in y = pi f (relative accuracy also next to the zeros,
//           where the value is f itself), quadrant k selects and signs them.
// A thread produces eight consecutive elements (two Philox blocks) and writes them with one 16-byte store; rows
// are walked by stepping (one 64-bit division per thread, outside the loop).
// Cost: Philox4x32-10 alone is 20 wide multiplies, 20 three-input xors and 20 key additions per four elements, so
// the kernel is bound by integer arithmetic, not by the 2 bytes it writes per element.
// ((u >> 9) + 0.5) * 2^-23 without an integer-to-float conversion: 1 + k 2^-23 is the float with mantissa field k,
// and subtracting 1 - 2^-24 from it is exact
__device__ __forceinline__ float uniform23_bits(uint32_t u) {
  return __uint_as_float(0x3f800000u | (u >> 9)) - 0.99999994039535522461f;
}

__device__ __forceinline__ void box_muller_bf16(uint32_t ua, uint32_t ub, float c, float& g0, float& g1) {
  float r;
  {
    const float r2 = c * __log2f(uniform23_bits(ua));
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(r2));
  }
  const float x = 2.0f * uniform23_bits(ub);
  // k = nearest integer to 2 x (0 .. 4): the low mantissa bits of 2 x + 1.5 * 2^23 hold it
  const float tk = fmaf(2.0f, x, 12582912.f);
  const float kf = tk - 12582912.f;
  const uint32_t k = __float_as_uint(tk);
  const float y = 3.14159265358979f * fmaf(kf, -0.5f, x);
  const float y2 = y * y;
  float sn = fmaf(y2, -1.9841270e-4f, 8.3333333e-3f);
  sn = fmaf(sn, y2, -1.6666667e-1f);
  sn = fmaf(sn * y2, y, y);
  float cs = fmaf(y2, 2.4801587e-5f, -1.3888889e-3f);
  cs = fmaf(cs, y2, 4.1666667e-2f);
  cs = fmaf(cs, y2, -0.5f);
  cs = fmaf(cs, y2, 1.0f);
  const float sa = (k & 1u) ? cs : sn, ca = (k & 1u) ? sn : cs;
  // quadrant 0: (s, c); 1: (c, -s); 2: (-s, -c); 3: (-c, s): the sign bits come from bit 1 of k and of k + 1
  const float s_out = __uint_as_float(__float_as_uint(sa) ^ ((k & 2u) << 30));
  const float c_out = __uint_as_float(__float_as_uint(ca) ^ (((k + 1u) & 2u) << 30));
  g0 = r * c_out;
  g1 = r * s_out;
}

__global__ void phi_gen_bf16_vec_kernel(__nv_bfloat16* __restrict__ phi, int64_t total, int64_t n, int64_t n_pad, float c,
                                        uint32_t k0, uint32_t k1) {
  const int64_t noct = total >> 3;                       // total % 8 == 0
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int64_t o = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (o >= noct) return;
  int64_t row = (o << 3) / n, j = (o << 3) - row * n;
  const int64_t drow = (stride << 3) / n, dj = (stride << 3) - drow * n;
  for (; o < noct; o += stride) {
    uint32_t w[4];
#pragma unroll
    for (int b = 0; b < 2; ++b) {
      const int64_t q = 2 * o + b;
      const U4 u = philox4x32_10(U4{(uint32_t)q, (uint32_t)(q >> 32), 0u, 0u}, k0, k1);
      float g0, g1, g2, g3;
      box_muller_bf16(u.x, u.y, c, g0, g1);
      box_muller_bf16(u.z, u.w, c, g2, g3);
      __nv_bfloat162 p0 = __floats2bfloat162_rn(g0, g1), p1 = __floats2bfloat162_rn(g2, g3);
      w[2 * b] = *reinterpret_cast<uint32_t*>(&p0);
      w[2 * b + 1] = *reinterpret_cast<uint32_t*>(&p1);
    }
    *reinterpret_cast<uint4*>(phi + row * n_pad + j) = make_uint4(w[0], w[1], w[2], w[3]);
    row += drow;
    j += dj;
    if (j >= n) { j -= n; ++row; }
  }
}

// Rademacher ensemble: one sign bit per element of the unpadded index space, 128 elements per Philox block,
// counter (q, 0, 1, 0) as (low, high, third, fourth) words.  A warp takes 32 consecutive blocks (4096
// elements): lane l computes block l, and in step s the word (s % 4) of lane s / 4 is broadcast so that lane l
// writes element 32 s + l: consecutive lanes write consecutive elements.  Write-bound.
template <typename T>
__global__ void phi_rademacher_kernel(T* __restrict__ phi, int64_t total, int64_t n, int64_t n_pad, float inv_sqrt_m,
                                      uint32_t k0, uint32_t k1) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const int64_t nspans = (total + 4095) >> 12;
  const T pos = to_storage<T>(inv_sqrt_m), neg = to_storage<T>(-inv_sqrt_m);
  for (int64_t span = warp; span < nspans; span += nwarps) {
    const int64_t q = (span << 5) + lane;
    const U4 u = philox4x32_10(U4{(uint32_t)q, (uint32_t)(q >> 32), 1u, 0u}, k0, k1);
    int64_t e = (span << 12) + lane;
    int64_t row = e / n;
    int64_t j = e - row * n;
#pragma unroll 4
    for (int s = 0; s < 128; ++s) {
      const int w = s & 3;
      const uint32_t mine = w == 0 ? u.x : (w == 1 ? u.y : (w == 2 ? u.z : u.w));
      const uint32_t bits = __shfl_sync(0xffffffffu, mine, s >> 2);
      if (e < total) phi[row * n_pad + j] = ((bits >> lane) & 1u) ? neg : pos;
      e += 32;
      j += 32;
      while (j >= n) { j -= n; ++row; }
    }
  }
}

// Same stream, n % 8 == 0: every lane writes 8 consecutive elements (one 16-byte store for bf16, two for
// float) that never straddle a row.  A warp step covers 256 elements = 2 Philox blocks; lane l needs byte
// (l % 4) of word (l / 4) % 4 of block 2 s + l / 16.
template <typename T>
__global__ void phi_rademacher_vec_kernel(T* __restrict__ phi, int64_t total, int64_t n, int64_t n_pad,
                                          float inv_sqrt_m, uint32_t k0, uint32_t k1) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const int64_t nspans = (total + 4095) >> 12;
  const T pos = to_storage<T>(inv_sqrt_m), neg = to_storage<T>(-inv_sqrt_m);
  for (int64_t span = warp; span < nspans; span += nwarps) {
    const int64_t q = (span << 5) + lane;
    const U4 u = philox4x32_10(U4{(uint32_t)q, (uint32_t)(q >> 32), 1u, 0u}, k0, k1);
    int64_t e = (span << 12) + lane * 8;
    int64_t row = e / n;
    int64_t j = e - row * n;
#pragma unroll 4
    for (int s = 0; s < 16; ++s) {
      const int src = 2 * s + (lane >> 4);
      const uint32_t wx = __shfl_sync(0xffffffffu, u.x, src), wy = __shfl_sync(0xffffffffu, u.y, src);
      const uint32_t wz = __shfl_sync(0xffffffffu, u.z, src), ww = __shfl_sync(0xffffffffu, u.w, src);
      const int wi = (lane >> 2) & 3;
      const uint32_t word = wi == 0 ? wx : (wi == 1 ? wy : (wi == 2 ? wz : ww));
      const uint32_t byte = (word >> ((lane & 3) * 8)) & 0xffu;
      if (e < total) {                      // total % 8 == 0: all 8 elements exist
        alignas(16) T v[8];
#pragma unroll
        for (int b = 0; b < 8; ++b) v[b] = ((byte >> b) & 1u) ? neg : pos;
        T* dst = phi + row * n_pad + j;
        if (sizeof(T) == 2) {
          *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(v);
        } else {
          reinterpret_cast<uint4*>(dst)[0] = reinterpret_cast<const uint4*>(v)[0];
          reinterpret_cast<uint4*>(dst)[1] = reinterpret_cast<const uint4*>(v)[1];
        }
      }
      e += 256;
      j += 256;
      while (j >= n) { j -= n; ++row; }
    }
  }
}

// Structured Hadamard ensemble: Phi[h,r,j] = s[h,j] (-1)^popcount(i_r & j) / sqrt(m), i_r = (a r + b) mod N with
// a = 2 u0 + 1, b = u1 from the Philox block (h, 0, 3, 0); column sign s[h,j] from bit e % 32 of word (e / 32) % 4 of
// block (e / 128, 0, 2, 0), e = h n + j.  One thread per V consecutive columns of one row (V = 8 when n % 8 == 0:
// the eight sign bits are one byte of one word, and the store is one 16-byte vector for bf16).
template <typename T, int V>
__global__ void phi_hadamard_kernel(T* __restrict__ phi, int64_t n, int64_t n_pad, int64_t m, int64_t rows,
                                    uint32_t log2N, float inv_sqrt_m, uint32_t k0, uint32_t k1) {
  const int64_t j0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * V;
  if (j0 >= n) return;
  for (int64_t row = blockIdx.y; row < rows; row += gridDim.y) {     // row = h * m + r
  const int64_t h = row / m, r = row - h * m;
  const U4 ab = philox4x32_10(U4{(uint32_t)h, 0u, 3u, 0u}, k0, k1);
  const uint64_t a = 2ull * ab.x + 1ull, b = ab.y;
  const uint32_t ir = (uint32_t)((a * (uint64_t)r + b) & ((1ull << log2N) - 1ull));
  const int64_t e0 = h * n + j0;
  const U4 u = philox4x32_10(U4{(uint32_t)(e0 >> 7), (uint32_t)(e0 >> 39), 2u, 0u}, k0, k1);
  const uint32_t wi = (uint32_t)(e0 >> 5) & 3u;
  const uint32_t word = wi == 0 ? u.x : (wi == 1 ? u.y : (wi == 2 ? u.z : u.w));
  const T pos = to_storage<T>(inv_sqrt_m), neg = to_storage<T>(-inv_sqrt_m);
  alignas(16) T v[V];
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const uint32_t sbit = (word >> (((uint32_t)e0 & 31u) + i)) & 1u;          // V = 8: e0 % 8 == 0, the bits share a byte
    const uint32_t par = __popc(ir & (uint32_t)(j0 + i)) & 1u;
    v[i] = (sbit ^ par) ? neg : pos;
  }
  T* dst = phi + row * n_pad + j0;
  if (V == 8) {
    const uint4* src = reinterpret_cast<const uint4*>(v);
    reinterpret_cast<uint4*>(dst)[0] = src[0];
    if (sizeof(T) == 4) reinterpret_cast<uint4*>(dst)[1] = src[1];
  } else {
    dst[0] = v[0];
  }
  }
}

// word k of the column-sign stream = word k % 4 of the Philox block with counter (k / 4, 0, 2, 0); (u0, u1) of head h
// = the first two words of block (h, 0, 3, 0): the same blocks phi_hadamard_kernel draws from
__global__ void hadamard_tables_kernel(uint32_t* __restrict__ sign_words, uint32_t* __restrict__ ab, int64_t nwords,
                                       int heads, uint32_t k0, uint32_t k1) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  const int64_t nblocks = (nwords + 3) >> 2;
  if (i < nblocks) {
    const U4 u = philox4x32_10(U4{(uint32_t)i, (uint32_t)(i >> 32), 2u, 0u}, k0, k1);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
    for (int q = 0; q < 4; ++q)
      if (4 * i + q < nwords) sign_words[4 * i + q] = w[q];
  }
  if (i < heads) {
    const U4 u = philox4x32_10(U4{(uint32_t)i, 0u, 3u, 0u}, k0, k1);
    ab[2 * i] = u.x;
    ab[2 * i + 1] = u.y;
  }
}

template <typename T>
__global__ void phi_pack_kernel(T* __restrict__ dst, const T* __restrict__ src, int64_t rows, int64_t n,
                                int64_t n_pad, bool to_padded) {
  const int64_t total = rows * n;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / n, j = i - r * n;
    if (to_padded) dst[r * n_pad + j] = src[i];
    else dst[i] = src[r * n_pad + j];
  }
}

int grid_for(int64_t work, int block) {
  int64_t g = (work + block - 1) / block;
  const int64_t cap = 148LL * 16;   // a few waves of the 148 SMs; kernels use grid-stride loops
  return (int)(g < 1 ? 1 : (g > cap ? cap : g));
}

}  // namespace

size_t elt_size(int dtype) { return dtype == CSAT_DTYPE_FP32 ? 4 : 2; }

cudaError_t launch_phi_gen(void* phi, const Params& p, cudaStream_t s) {
  const int64_t total = p.H * p.m * p.n;
  cudaError_t e = cudaSuccess;
  if (p.n_pad != p.n)      // the padding columns must hold zeros; without padding every element is written below
    e = cudaMemsetAsync(phi, 0, (size_t)(p.H * p.m * p.n_pad) * elt_size(p.dtype), s);
  if (e != cudaSuccess) return e;
  const float inv = (float)(1.0 / sqrt((double)p.m));
  const uint32_t k0 = (uint32_t)(p.seed & 0xFFFFFFFFull), k1 = (uint32_t)(p.seed >> 32);
  if (p.ensemble == CSAT_ENSEMBLE_HADAMARD) {
    uint32_t log2N = 0;
    while (((int64_t)1 << log2N) < p.n) ++log2N;
    const int64_t rows = p.H * p.m;
    const bool vec = p.n % 8 == 0;
    const int64_t per_row = vec ? p.n / 8 : p.n;
    const dim3 grid((unsigned)((per_row + 127) / 128), (unsigned)(rows < 65535 ? rows : 65535));   // rows beyond: strided
#define CSAT_HAD(T, V) phi_hadamard_kernel<T, V><<<grid, 128, 0, s>>>((T*)phi, p.n, p.n_pad, p.m, rows, log2N, inv, k0, k1)
    if (p.dtype == CSAT_DTYPE_FP32) { if (vec) CSAT_HAD(float, 8); else CSAT_HAD(float, 1); }
    else { if (vec) CSAT_HAD(__nv_bfloat16, 8); else CSAT_HAD(__nv_bfloat16, 1); }
#undef CSAT_HAD
    return cudaGetLastError();
  }
  if (p.ensemble == CSAT_ENSEMBLE_RADEMACHER) {
    const int rb = 256, rg = grid_for((total + 127) / 128, rb);
    const bool vec = p.n % 8 == 0;
    if (p.dtype == CSAT_DTYPE_FP32) {
      if (vec) phi_rademacher_vec_kernel<float><<<rg, rb, 0, s>>>((float*)phi, total, p.n, p.n_pad, inv, k0, k1);
      else phi_rademacher_kernel<float><<<rg, rb, 0, s>>>((float*)phi, total, p.n, p.n_pad, inv, k0, k1);
    } else {
      if (vec)
        phi_rademacher_vec_kernel<__nv_bfloat16><<<rg, rb, 0, s>>>((__nv_bfloat16*)phi, total, p.n, p.n_pad, inv, k0, k1);
      else
        phi_rademacher_kernel<__nv_bfloat16><<<rg, rb, 0, s>>>((__nv_bfloat16*)phi, total, p.n, p.n_pad, inv, k0, k1);
    }
    return cudaGetLastError();
  }
  if (p.dtype == CSAT_DTYPE_BF16 && p.n % 8 == 0) {
    const int block = 256, grid = grid_for(total / 8, block);
    const float c = (float)(-2.0 * 0.6931471805599453 / (double)p.m);
    phi_gen_bf16_vec_kernel<<<grid, block, 0, s>>>((__nv_bfloat16*)phi, total, p.n, p.n_pad, c, k0, k1);
    return cudaGetLastError();
  }
  const int block = 256, grid = grid_for((total + 3) / 4, block);
  if (p.dtype == CSAT_DTYPE_FP32)
    phi_gen_kernel<float><<<grid, block, 0, s>>>((float*)phi, total, p.n, p.n_pad, inv, k0, k1);
  else
    phi_gen_kernel<__nv_bfloat16><<<grid, block, 0, s>>>((__nv_bfloat16*)phi, total, p.n, p.n_pad, inv, k0, k1);
  return cudaGetLastError();
}

cudaError_t launch_hadamard_tables(uint32_t* sign_words, uint32_t* ab, const Params& p, cudaStream_t s) {
  const int64_t nwords = (p.H * p.n + 31) / 32;            // p.H counts every generated matrix (2 H with separate Phi_V)
  const int64_t nblocks = (nwords + 3) / 4;
  const int64_t work = nblocks > p.H ? nblocks : p.H;
  const uint32_t k0 = (uint32_t)(p.seed & 0xFFFFFFFFull), k1 = (uint32_t)(p.seed >> 32);
  hadamard_tables_kernel<<<(unsigned)((work + 127) / 128), 128, 0, s>>>(sign_words, ab, nwords, (int)p.H, k0, k1);
  return cudaGetLastError();
}

static cudaError_t pack(void* dst, const void* src, const Params& p, cudaStream_t s, bool to_padded) {
  const int64_t rows = p.H * p.m;
  const int block = 256, grid = grid_for(rows * p.n, block);
  if (p.dtype == CSAT_DTYPE_FP32)
    phi_pack_kernel<float><<<grid, block, 0, s>>>((float*)dst, (const float*)src, rows, p.n, p.n_pad, to_padded);
  else
    phi_pack_kernel<__nv_bfloat16><<<grid, block, 0, s>>>((__nv_bfloat16*)dst, (const __nv_bfloat16*)src, rows, p.n,
                                                         p.n_pad, to_padded);
  return cudaGetLastError();
}

cudaError_t launch_phi_pack(void* phi_padded, const void* phi_dense, const Params& p, cudaStream_t s) {
  cudaError_t e = cudaMemsetAsync(phi_padded, 0, (size_t)(p.H * p.m * p.n_pad) * elt_size(p.dtype), s);
  if (e != cudaSuccess) return e;
  return pack(phi_padded, phi_dense, p, s, true);
}

cudaError_t launch_phi_unpack(void* phi_dense, const void* phi_padded, const Params& p, cudaStream_t s) {
  return pack(phi_dense, phi_padded, p, s, false);
}

}  // namespace csat
