// K~|V~ = Phi [K|V] for the structured Hadamard ensemble by a fast Walsh-Hadamard transform instead of a dense
// product (paper: the compression equation, with Phi drawn from the "structured Hadamard" family it lists).
//
// The ensemble (see phi_gen.cu): Phi[h,r,j] = s[h,j] (-1)^popcount(i_r & j) / sqrt(m), i_r = (a_h r + b_h) mod N, N the
// smallest power of two >= n.  Hence, column by column of K and V,
//     K~[r, c] = (1 / sqrt(m)) * ( H_N (s o K[:, c] padded with zeros to N) )[i_r] :
// one length-N transform (N log2 N additions) and a gather of m of its entries, instead of m n multiply-adds.
//
// One CTA transforms CG columns of K or V of one (batch, head) entirely in shared memory (float32, [CG][N] with
// one padding word per 32 so that strided butterflies spread over the banks):
//   load    every thread reads CG adjacent columns of its token rows (one vector load) and applies the sign s[h,j];
//   passes  radix-16 (four butterfly stages in registers per pass through shared memory), a smaller radix for the
//           remaining log2 N mod 4 stages;
//   gather  row r of the output is entry i_r of every transformed column, scaled, rounded to the storage type.
// The sign bits and (a_h, b_h) come from tables the generator writes when the ensemble is selected, so the kernel
// computes no Philox blocks.  The n_q x m score matrix etc. are untouched: only the compression stage changes.
#include "csat_internal.h"

namespace csat {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ int pad(int j) { return j + (j >> 5); }

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// CG consecutive elements as one aligned vector
template <typename T, int CG> struct alignas(sizeof(T) * CG < 16 ? sizeof(T) * CG : 16) Vec { T v[CG]; };

// one pass of radix 2^RLOG with stride 2^s over all CG columns
template <int RLOG, int CG>
__device__ __forceinline__ void fwht_pass(float* xs, int Np, int log2N, int s) {
  constexpr int R = 1 << RLOG;
  const int S = 1 << s;
  const int groups = 1 << (log2N - RLOG);                 // per column
  for (int idx = threadIdx.x; idx < groups * CG; idx += kThreads) {
    const int c = idx >> (log2N - RLOG), gi = idx & (groups - 1);
    const int lo = gi & (S - 1), hi = gi >> s;
    const int base = (hi << (s + RLOG)) + lo;
    float* col = xs + c * Np;
    float a[R];
#pragma unroll
    for (int k = 0; k < R; ++k) a[k] = col[pad(base + k * S)];
#pragma unroll
    for (int q = 1; q < R; q <<= 1) {
#pragma unroll
      for (int k = 0; k < R; ++k) {
        if ((k & q) == 0) {
          const float u = a[k], v = a[k | q];
          a[k] = u + v;
          a[k | q] = u - v;
        }
      }
    }
#pragma unroll
    for (int k = 0; k < R; ++k) col[pad(base + k * S)] = a[k];
  }
}

template <typename T, int CG>
__global__ void __launch_bounds__(kThreads) fwht_compress_kernel(T* __restrict__ kv, const T* __restrict__ K,
                                                                 const T* __restrict__ V,
                                                                 const uint32_t* __restrict__ sign_words,
                                                                 const uint32_t* __restrict__ ab, int64_t n, int log2N,
                                                                 int64_t m, int d, int H, int sep, float inv_sqrt_m) {
  extern __shared__ float xs[];                            // [CG][Np]
  const int N = 1 << log2N, Np = N + (N >> 5);
  const int bh = blockIdx.y, h = bh % H;
  const int col0 = blockIdx.x * CG;                        // column of K|V: [0, d) are K's, [d, 2d) are V's
  const bool is_v = col0 >= d;
  const T* src = (is_v ? V : K) + (int64_t)bh * n * d + (is_v ? col0 - d : col0);
  const int hp = (is_v && sep) ? H + h : h;                // the generator's head: Phi_V of head h is head H + h
  // four token rows per thread and step: the loads are independent and all in flight together
  constexpr int kU = 4;
  for (int j0 = threadIdx.x; j0 < N; j0 += kThreads * kU) {
    Vec<T, CG> in[kU];
    uint32_t sw[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int j = j0 + u * kThreads;
      if (j < n) {
        in[u] = *reinterpret_cast<const Vec<T, CG>*>(src + (int64_t)j * d);
        const int64_t e = (int64_t)hp * n + j;
        sw[u] = sign_words[e >> 5] >> (e & 31);
      }
    }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int j = j0 + u * kThreads;
      if (j >= N) continue;
      const bool live = j < n, neg = live && (sw[u] & 1u);
#pragma unroll
      for (int c = 0; c < CG; ++c) {
        const float x = live ? to_f<T>(in[u].v[c]) : 0.f;
        xs[c * Np + pad(j)] = neg ? -x : x;
      }
    }
  }
  __syncthreads();
  int s = 0;
  for (; s + 4 <= log2N; s += 4) {
    fwht_pass<4, CG>(xs, Np, log2N, s);
    __syncthreads();
  }
  const int rest = log2N - s;
  if (rest == 3) fwht_pass<3, CG>(xs, Np, log2N, s);
  else if (rest == 2) fwht_pass<2, CG>(xs, Np, log2N, s);
  else if (rest == 1) fwht_pass<1, CG>(xs, Np, log2N, s);
  if (rest) __syncthreads();
  // row r of the output = entry i_r of every transformed column
  const uint64_t a = 2ull * ab[2 * hp] + 1ull, b = ab[2 * hp + 1];
  T* dst = kv + (int64_t)bh * m * 2 * d + col0;
  for (int64_t r = threadIdx.x; r < m; r += kThreads) {
    const int i = (int)((a * (uint64_t)r + b) & (uint64_t)(N - 1));
    Vec<T, CG> out;
#pragma unroll
    for (int c = 0; c < CG; ++c) out.v[c] = from_f<T>(xs[c * Np + pad(i)] * inv_sqrt_m);
    *reinterpret_cast<Vec<T, CG>*>(dst + r * 2 * d) = out;
  }
}

template <typename T, int CG>
cudaError_t launch_cg(csat_ctx* c, const void* K, const void* V, cudaStream_t s, int log2N) {
  const Params& p = c->p;
  const int64_t N = (int64_t)1 << log2N;
  const size_t smem = (size_t)CG * (size_t)(N + (N >> 5)) * sizeof(float);
  cudaError_t e = cudaSuccess;
  if (smem > 48 * 1024)
    e = cudaFuncSetAttribute(fwht_compress_kernel<T, CG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const dim3 grid((unsigned)(2 * p.d / CG), (unsigned)(p.B * p.H));
  fwht_compress_kernel<T, CG><<<grid, kThreads, smem, s>>>((T*)c->kv, (const T*)K, (const T*)V, c->had_signs, c->had_ab,
                                                         p.n, log2N, p.m, (int)p.d, (int)p.H, p.separate_phi,
                                                         (float)(1.0 / sqrt((double)p.m)));
  return cudaGetLastError();
}

template <typename T>
cudaError_t launch_t(csat_ctx* c, const void* K, const void* V, cudaStream_t s, int log2N) {
  // columns per CTA: the CTA's [CG][N] float32 tile takes ~68 KB (three CTAs per SM), 136 KB at N = 16384
  if (log2N <= 11) return launch_cg<T, 8>(c, K, V, s, log2N);
  if (log2N == 12) return launch_cg<T, 4>(c, K, V, s, log2N);
  return launch_cg<T, 2>(c, K, V, s, log2N);
}

}  // namespace

bool fwht_compress_supported(const csat_ctx* c) {
  int log2N = 0;
  while (((int64_t)1 << log2N) < c->p.n) ++log2N;
  return c->p.ensemble == CSAT_ENSEMBLE_HADAMARD && c->phi_generated && c->had_signs != nullptr && log2N <= 14;
}

cudaError_t launch_fwht_compress(csat_ctx* c, const void* K, const void* V, cudaStream_t s, int* launches) {
  *launches += 1;
  int log2N = 0;
  while (((int64_t)1 << log2N) < c->p.n) ++log2N;
  return c->p.dtype == CSAT_DTYPE_FP32 ? launch_t<float>(c, K, V, s, log2N) : launch_t<__nv_bfloat16>(c, K, V, s, log2N);
}

}  // namespace csat
