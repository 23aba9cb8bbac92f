// Plain FFMA kernels for the CSAT forward: the float32 path (and bf16 storage with head sizes the
// tensor-core kernels do not cover).  Accumulation, softmax and the recovery iterates are float32.
//
// Paper equations, in order: K~ = Phi K, V~ = Phi V (compress_kernel); A~ = softmax(Q K~^T / sqrt(d_k)),
// Z = A~ V~, alpha^{t+1} = eta_theta(S alpha^t + B Z_i), C^_i = Psi alpha^_i (attend_recover_kernel).
// The n_q x m matrix A~ and the iterates alpha^t stay in registers / shared memory.
#include "csat_internal.h"

namespace csat {
namespace {

template <typename T> __device__ __forceinline__ float ldf(const T* p, int64_t i);
template <> __device__ __forceinline__ float ldf<float>(const float* p, int64_t i) { return p[i]; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p, int64_t i) {
  return __bfloat162float(p[i]);
}
template <typename T> __device__ __forceinline__ void stf(T* p, int64_t i, float v);
template <> __device__ __forceinline__ void stf<float>(float* p, int64_t i, float v) { p[i] = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16* p, int64_t i, float v) {
  p[i] = __float2bfloat16_rn(v);
}

// ---------------------------------------------------------------------------------------------
// K~|V~[b,h,r,:] = sum_j Phi[h,r,j] * [K|V][b,h,j,:]       (compression equation)
// block: 256 threads = 8 row groups x 32 column lanes; tile = 32 measurements x 2d columns;
// the token axis is walked in chunks of 16 staged in shared memory.
// ---------------------------------------------------------------------------------------------
constexpr int kCmpRows = 32, kCmpChunk = 16;

// Token-sharded use: K, V hold the n tokens [phi_j0, phi_j0 + n) of the sequence and the sums go out as float32
// partials (TO = float) that are added over the shards before anything reads them.
template <typename T, typename TO, int KC>   // KC = ceil(2d / 32) column slots per lane
__global__ void __launch_bounds__(256) compress_kernel(TO* __restrict__ kv, const T* __restrict__ phi,
                                                       const T* __restrict__ K, const T* __restrict__ V, int64_t n,
                                                       int64_t n_pad, int64_t m, int d, int H, int phi_v_head0,
                                                       int64_t phi_j0) {
  // phi_v_head0: index of the first Phi_V matrix in phi (0 when Phi_V = Phi_K, H when they are separate)
  extern __shared__ float smem[];
  float* phis = smem;                              // [2][32][17]: Phi_K tile, Phi_V tile
  float* phiv = smem + kCmpRows * (kCmpChunk + 1);
  float* kvs = smem + 2 * kCmpRows * (kCmpChunk + 1);  // [16][2d]
  const int d2 = 2 * d;
  const int bh = blockIdx.y, h = bh % H;
  const int64_t r0 = (int64_t)blockIdx.x * kCmpRows;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const T* Kb = K + (int64_t)bh * n * d;
  const T* Vb = V + (int64_t)bh * n * d;
  const T* Ph = phi + (int64_t)h * m * n_pad;
  const T* Pv = phi + (int64_t)(phi_v_head0 + h) * m * n_pad;
  float acc[4][KC];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int k = 0; k < KC; ++k) acc[i][k] = 0.f;

  for (int64_t j0 = 0; j0 < n; j0 += kCmpChunk) {
    for (int i = threadIdx.x; i < kCmpRows * kCmpChunk; i += 256) {
      const int rr = i / kCmpChunk, jj = i % kCmpChunk;
      const int64_t r = r0 + rr;
      const bool in = r < m && j0 + jj < n;              // a shard's last chunk must not reach into the next shard
      phis[rr * (kCmpChunk + 1) + jj] = in ? ldf(Ph, r * n_pad + phi_j0 + j0 + jj) : 0.f;
      phiv[rr * (kCmpChunk + 1) + jj] = in ? ldf(Pv, r * n_pad + phi_j0 + j0 + jj) : 0.f;
    }
    for (int i = threadIdx.x; i < kCmpChunk * d2; i += 256) {
      const int jj = i / d2, c = i % d2;
      const int64_t j = j0 + jj;
      float v = 0.f;
      if (j < n) v = (c < d) ? ldf(Kb, j * d + c) : ldf(Vb, j * d + (c - d));
      kvs[jj * d2 + c] = v;
    }
    __syncthreads();
#pragma unroll 4
    for (int jj = 0; jj < kCmpChunk; ++jj) {
      float a[4], av[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        a[i] = phis[(ty * 4 + i) * (kCmpChunk + 1) + jj];
        av[i] = phiv[(ty * 4 + i) * (kCmpChunk + 1) + jj];
      }
#pragma unroll
      for (int k = 0; k < KC; ++k) {
        const int c = tx + 32 * k;
        const float b = (c < d2) ? kvs[jj * d2 + c] : 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i][k] = fmaf(c < d ? a[i] : av[i], b, acc[i][k]);   // K columns, then V columns
      }
    }
    __syncthreads();
  }
  TO* dst = kv + (int64_t)bh * m * d2;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t r = r0 + ty * 4 + i;
    if (r >= m) continue;
#pragma unroll
    for (int k = 0; k < KC; ++k) {
      const int c = tx + 32 * k;
      if (c < d2) stf(dst, r * d2 + c, acc[i][k]);
    }
  }
}

// workspace[i] = sum over r < R of partials[r][i], added in the order r = 0, 1, ..., R-1 (the same on every rank
// and in every run), rounded once to the storage type
template <typename T>
__global__ void reduce_partials_kernel(T* __restrict__ kv, const float* __restrict__ partials, int64_t count, int R) {
  for (int64_t i = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) * 4; i < count; i += (int64_t)gridDim.x * blockDim.x * 4) {
    float4 a = *reinterpret_cast<const float4*>(partials + i);
    for (int r = 1; r < R; ++r) {
      const float4 b = *reinterpret_cast<const float4*>(partials + (int64_t)r * count + i);
      a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
    }
    stf(kv, i, a.x); stf(kv, i + 1, a.y); stf(kv, i + 2, a.z); stf(kv, i + 3, a.w);
  }
}

// ---------------------------------------------------------------------------------------------
// One warp per query row.  Scores: lane = measurement; softmax statistics by warp shuffles (online
// over chunks of 32 measurements); Z and the iterates: lane = feature column (col = lane + 32 j).
// ---------------------------------------------------------------------------------------------
constexpr int kAttWarps = 8;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float soft_threshold(float x, float theta) {
  return x - fminf(fmaxf(x, -theta), theta);   // = sign(x) max(|x| - theta, 0)
}

// y[col_j] = sum_k x_k * W[k*d + col_j]  with x distributed as x[j] <-> feature lane + 32 j
template <int DC>
__device__ __forceinline__ void row_times_matrix(const float (&x)[DC], float (&y)[DC], const float* __restrict__ W,
                                                 int d, int lane) {
#pragma unroll
  for (int j = 0; j < DC; ++j) y[j] = 0.f;
#pragma unroll
  for (int jk = 0; jk < DC; ++jk) {
    for (int l = 0; l < 32; ++l) {
      const int k = 32 * jk + l;
      const float xk = __shfl_sync(0xffffffffu, x[jk], l);
      if (k < d) {
#pragma unroll
        for (int j = 0; j < DC; ++j) {
          const int col = lane + 32 * j;
          if (col < d) y[j] = fmaf(xk, W[(int64_t)k * d + col], y[j]);
        }
      }
    }
  }
}

template <typename T, int DC>   // DC = ceil(d / 32)
__global__ void __launch_bounds__(kAttWarps * 32) attend_recover_kernel(
    T* __restrict__ out, const T* __restrict__ Q, const T* __restrict__ kv, const float* __restrict__ S_dec,
    const float* __restrict__ B_dec, int64_t layer_stride, const float* __restrict__ theta, int theta_stride,
    const float* __restrict__ psi_f32, int64_t nq, int64_t m, int d, int H, int T_iters, float scale) {
  extern __shared__ float smem[];
  const int d2 = 2 * d, ldk = d2 + 1;
  float* kvs = smem;                       // [32][2d+1]
  float* qs = smem + 32 * ldk;             // [warps][d]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, h = bh % H;
  const int64_t row = (int64_t)blockIdx.x * kAttWarps + warp;
  const bool live = row < nq;
  const T* Qr = Q + ((int64_t)bh * nq + (live ? row : 0)) * d;
  const T* kvb = kv + (int64_t)bh * m * d2;
  float* q = qs + warp * d;
  for (int c = lane; c < d; c += 32) q[c] = live ? ldf(Qr, c) : 0.f;

  float z[DC];
#pragma unroll
  for (int j = 0; j < DC; ++j) z[j] = 0.f;
  float run_max = -INFINITY, run_sum = 0.f;

  for (int64_t r0 = 0; r0 < m; r0 += 32) {
    __syncthreads();
    for (int i = threadIdx.x; i < 32 * d2; i += kAttWarps * 32) {
      const int rr = i / d2, c = i % d2;
      kvs[rr * ldk + c] = (r0 + rr < m) ? ldf(kvb, (r0 + rr) * d2 + c) : 0.f;
    }
    __syncthreads();
    float s = 0.f;
    const float* kr = kvs + lane * ldk;
    for (int c = 0; c < d; ++c) s = fmaf(q[c], kr[c], s);
    s = (r0 + lane < m) ? s * scale : -INFINITY;
    const float new_max = fmaxf(run_max, warp_max(s));      // finite: measurement r0 always exists
    const float corr = expf(run_max - new_max);             // 0 on the first chunk (run_max = -inf)
    const float p = expf(s - new_max);
    run_sum = run_sum * corr + warp_sum(p);
    run_max = new_max;
#pragma unroll
    for (int j = 0; j < DC; ++j) z[j] *= corr;
    for (int rr = 0; rr < 32; ++rr) {
      const float pr = __shfl_sync(0xffffffffu, p, rr);
      const float* vr = kvs + rr * ldk + d;
#pragma unroll
      for (int j = 0; j < DC; ++j) {
        const int col = lane + 32 * j;
        if (col < d) z[j] = fmaf(pr, vr[col], z[j]);
      }
    }
  }
  const float inv = 1.f / run_sum;
#pragma unroll
  for (int j = 0; j < DC; ++j) z[j] *= inv;

  float res[DC];
  if (T_iters == 0) {
#pragma unroll
    for (int j = 0; j < DC; ++j) res[j] = z[j];
  } else {
    // layer t reads theta[t * theta_stride + h] and the matrices at layer_stride * t (0: one S, B for all layers)
    const float* Sh = S_dec + (int64_t)h * d * d;
    const float* Bh = B_dec + (int64_t)h * d * d;
    float th = theta[h];
    float c[DC], a[DC], t[DC];
    row_times_matrix<DC>(z, c, Bh, d, lane);
#pragma unroll
    for (int j = 0; j < DC; ++j) a[j] = soft_threshold(c[j], th);   // alpha^1 = eta(0 S + z B)
    for (int it = 1; it < T_iters; ++it) {
      th = theta[(int64_t)it * theta_stride + h];
      if (layer_stride != 0) row_times_matrix<DC>(z, c, Bh + layer_stride * it, d, lane);   // z B_t
      row_times_matrix<DC>(a, t, Sh + layer_stride * it, d, lane);
#pragma unroll
      for (int j = 0; j < DC; ++j) a[j] = soft_threshold(t[j] + c[j], th);
    }
    if (psi_f32) {
      // out_c = sum_k alpha_k Psi[c][k]
      const float* Ph = psi_f32 + (int64_t)h * d * d;
#pragma unroll
      for (int j = 0; j < DC; ++j) res[j] = 0.f;
#pragma unroll
      for (int jk = 0; jk < DC; ++jk) {
        for (int l = 0; l < 32; ++l) {
          const int k = 32 * jk + l;
          const float ak = __shfl_sync(0xffffffffu, a[jk], l);
          if (k < d) {
#pragma unroll
            for (int j = 0; j < DC; ++j) {
              const int col = lane + 32 * j;
              if (col < d) res[j] = fmaf(ak, Ph[(int64_t)col * d + k], res[j]);
            }
          }
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < DC; ++j) res[j] = a[j];
    }
  }
  if (live) {
    T* o = out + ((int64_t)bh * nq + row) * d;
#pragma unroll
    for (int j = 0; j < DC; ++j) {
      const int col = lane + 32 * j;
      if (col < d) stf(o, col, res[j]);
    }
  }
}

template <typename T>
__global__ void split_kv_kernel(T* __restrict__ kt, T* __restrict__ vt, const T* __restrict__ kv, int64_t rows, int d) {
  const int64_t total = rows * 2 * d;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / (2 * d);
    const int c = (int)(i % (2 * d));
    if (c < d) { if (kt) kt[r * d + c] = kv[i]; }
    else       { if (vt) vt[r * d + (c - d)] = kv[i]; }
  }
}

template <typename T>
cudaError_t compress_t(csat_ctx* c, const void* K, const void* V, cudaStream_t s, int64_t phi_j0, int64_t n_len,
                       float* partial) {
  const Params& p = c->p;
  const int d = (int)p.d;
  const dim3 grid((unsigned)((p.m + kCmpRows - 1) / kCmpRows), (unsigned)(p.B * p.H));
  const size_t sm = (size_t)(2 * kCmpRows * (kCmpChunk + 1) + kCmpChunk * 2 * d) * sizeof(float);
  const int kc = (2 * d + 31) / 32;
#define CSAT_CMP(KC)                                                                                                  \
  do {                                                                                                                \
    if (partial)                                                                                                      \
      compress_kernel<T, float, KC><<<grid, 256, sm, s>>>(partial, (const T*)c->phi, (const T*)K, (const T*)V, n_len, \
                                                          p.n_pad, p.m, d, (int)p.H, p.separate_phi ? (int)p.H : 0,  \
                                                          phi_j0);                                                    \
    else                                                                                                              \
      compress_kernel<T, T, KC><<<grid, 256, sm, s>>>((T*)c->kv, (const T*)c->phi, (const T*)K, (const T*)V, n_len,  \
                                                      p.n_pad, p.m, d, (int)p.H, p.separate_phi ? (int)p.H : 0,      \
                                                      phi_j0);                                                        \
  } while (0)
  if (kc <= 4) CSAT_CMP(4);
  else if (kc <= 8) CSAT_CMP(8);
  else CSAT_CMP(16);
#undef CSAT_CMP
  return cudaGetLastError();
}

template <typename T>
cudaError_t attend_t(csat_ctx* c, const void* Q, void* out, cudaStream_t s) {
  const Params& p = c->p;
  const int d = (int)p.d;
  const dim3 grid((unsigned)((p.nq + kAttWarps - 1) / kAttWarps), (unsigned)(p.B * p.H));
  const size_t sm = (size_t)(32 * (2 * d + 1) + kAttWarps * d) * sizeof(float);
  const float scale = (float)(p.scale > 0.0 ? p.scale : 1.0 / sqrt((double)d));
  const int dc = (d + 31) / 32;
  cudaError_t e = cudaSuccess;
#define CSAT_ATT(DC)                                                                                              \
  do {                                                                                                            \
    if (sm > 48 * 1024)                                                                                           \
      e = cudaFuncSetAttribute(attend_recover_kernel<T, DC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm); \
    if (e == cudaSuccess)                                                                                         \
      attend_recover_kernel<T, DC><<<grid, kAttWarps * 32, sm, s>>>(                                              \
          (T*)out, (const T*)Q, (const T*)c->kv, c->w_untied ? c->Sl_dec : c->S_dec,                             \
          c->w_untied ? c->Bl_dec : c->B_dec, c->w_untied ? (int64_t)(p.H * p.d * p.d) : (int64_t)0, c->thr(),  \
          c->thr_stride(),                                                                                       \
          c->psi ? c->psi_f32 : nullptr,                                                                         \
          p.nq, p.m, d, (int)p.H, p.T, scale);                                                                    \
  } while (0)
  if (dc <= 2) CSAT_ATT(2);
  else if (dc <= 4) CSAT_ATT(4);
  else CSAT_ATT(8);
#undef CSAT_ATT
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

cudaError_t launch_simt_compress(csat_ctx* c, const void* K, const void* V, cudaStream_t s, int* launches,
                                 int64_t phi_j0, int64_t n_len, float* partial) {
  *launches += 1;
  if (n_len <= 0) n_len = c->p.n;
  return c->p.dtype == CSAT_DTYPE_FP32 ? compress_t<float>(c, K, V, s, phi_j0, n_len, partial)
                                       : compress_t<__nv_bfloat16>(c, K, V, s, phi_j0, n_len, partial);
}

cudaError_t launch_reduce_partials(csat_ctx* c, const float* partials, int R, cudaStream_t s, int* launches) {
  *launches += 1;
  const Params& p = c->p;
  const int64_t count = p.B * p.H * p.m * 2 * p.d;       // a multiple of 16 (d % 8 == 0)
  int64_t g = (count / 4 + 255) / 256;
  if (g > 148 * 16) g = 148 * 16;
  if (p.dtype == CSAT_DTYPE_FP32)
    reduce_partials_kernel<float><<<(unsigned)g, 256, 0, s>>>((float*)c->kv, partials, count, R);
  else
    reduce_partials_kernel<__nv_bfloat16><<<(unsigned)g, 256, 0, s>>>((__nv_bfloat16*)c->kv, partials, count, R);
  return cudaGetLastError();
}

cudaError_t launch_simt_attend_recover(csat_ctx* c, const void* Q, void* out, cudaStream_t s, int* launches) {
  *launches += 1;
  return c->p.dtype == CSAT_DTYPE_FP32 ? attend_t<float>(c, Q, out, s) : attend_t<__nv_bfloat16>(c, Q, out, s);
}

cudaError_t launch_split_kv(const csat_ctx* c, void* kt, void* vt, cudaStream_t s) {
  const Params& p = c->p;
  const int64_t rows = p.B * p.H * p.m;
  const int64_t work = rows * 2 * p.d;
  int64_t g = (work + 255) / 256;
  if (g > 148 * 16) g = 148 * 16;
  if (p.dtype == CSAT_DTYPE_FP32)
    split_kv_kernel<float><<<(unsigned)g, 256, 0, s>>>((float*)kt, (float*)vt, (const float*)c->kv, rows, (int)p.d);
  else
    split_kv_kernel<__nv_bfloat16><<<(unsigned)g, 256, 0, s>>>((__nv_bfloat16*)kt, (__nv_bfloat16*)vt,
                                                               (const __nv_bfloat16*)c->kv, rows, (int)p.d);
  return cudaGetLastError();
}

}  // namespace csat

// =============================================================================================
// csat_attend_noalloc: compressed attention (recovery disabled) for callers that cannot allocate.
// The K~|V~ scratch lives in a fixed array inside the library image instead of a cudaMalloc'd
// workspace.  See include/csat.h for who needs this and for the rules of use.
// =============================================================================================
#include <mutex>

namespace csat {
namespace {

// Scratch shared by every call on a device.  Resident on each GPU that loads the library, until exit.
static __device__ __align__(256) unsigned char g_noalloc_scratch[CSAT_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_noalloc_ptr[kMaxDevices] = {};   // device address of the array above, per device
std::mutex g_noalloc_mutex;

// Dense-Phi compression into the scratch: one thread per output element, tokens summed in index order
// (the same order, with the same fused multiply-adds, as compress_kernel).
template <typename T>
__global__ void compress_dense_phi_kernel(T* __restrict__ kv, const T* __restrict__ phi, const T* __restrict__ K,
                                          const T* __restrict__ V, int64_t n, int64_t m, int d, int H, int64_t total) {
  const int d2 = 2 * d;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int c = (int)(i % d2);
    const int64_t r = (i / d2) % m, bh = i / (d2 * m);
    const T* src = (c < d ? K : V) + bh * n * d + (c < d ? c : c - d);
    const T* ph = phi + ((bh % H) * m + r) * n;
    float acc = 0.f;
    for (int64_t j = 0; j < n; ++j) acc = fmaf(ldf(ph, j), ldf(src, j * d), acc);
    stf(kv, i, acc);
  }
}

void write_err(char* buf, size_t cap, const char* msg) {
  if (buf && cap) snprintf(buf, cap, "%s", msg);
}

template <typename T>
int attend_noalloc_t(const void* Q, const void* K, const void* V, const void* phi, void* out, void* scratch,
                     int64_t B, int64_t H, int64_t n, int64_t nq, int64_t m, int d, float scale, cudaStream_t s,
                     char* err, size_t cap) {
  const int64_t total = B * H * m * 2 * d;
  int64_t g = (total + 255) / 256;
  if (g > 148 * 32) g = 148 * 32;
  compress_dense_phi_kernel<T><<<(unsigned)g, 256, 0, s>>>((T*)scratch, (const T*)phi, (const T*)K, (const T*)V, n, m,
                                                          d, (int)H, total);
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) {
    const dim3 grid((unsigned)((nq + kAttWarps - 1) / kAttWarps), (unsigned)(B * H));
    const size_t sm = (size_t)(32 * (2 * d + 1) + kAttWarps * d) * sizeof(float);
    const int dc = (d + 31) / 32;
#define CSAT_NOALLOC_ATT(DC)                                                                                        \
  do {                                                                                                              \
    if (sm > 48 * 1024)                                                                                             \
      e = cudaFuncSetAttribute(attend_recover_kernel<T, DC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm); \
    if (e == cudaSuccess)                                                                                           \
      attend_recover_kernel<T, DC><<<grid, kAttWarps * 32, sm, s>>>((T*)out, (const T*)Q, (const T*)scratch,        \
                                                                    nullptr, nullptr, (int64_t)0, nullptr, 0,       \
                                                                    nullptr, nq, m, d,                              \
                                                                    (int)H, /*T_iters=*/0, scale);                  \
  } while (0)
    if (dc <= 2) CSAT_NOALLOC_ATT(2);
    else if (dc <= 4) CSAT_NOALLOC_ATT(4);
    else CSAT_NOALLOC_ATT(8);
#undef CSAT_NOALLOC_ATT
    if (e == cudaSuccess) e = cudaGetLastError();
  }
  if (e != cudaSuccess) {
    write_err(err, cap, cudaGetErrorString(e));
    return CSAT_ERR_CUDA;
  }
  return CSAT_OK;
}

}  // namespace
}  // namespace csat

extern "C" int csat_attend_noalloc(const void* Q, const void* K, const void* V, const void* phi, void* out, int64_t B,
                                   int64_t H, int64_t n, int64_t n_q, int64_t m, int64_t d, int dtype, double scale,
                                   void* stream, char* err_host, size_t err_cap) {
  using namespace csat;
  if (err_host && err_cap) err_host[0] = 0;
  if (!Q || !K || !V || !phi || !out) {
    write_err(err_host, err_cap, "csat_attend_noalloc: NULL tensor pointer");
    return CSAT_ERR_INVALID_ARG;
  }
  for (const void* p : {Q, K, V, phi, (const void*)out})
    if (reinterpret_cast<uintptr_t>(p) & 15u) {
      write_err(err_host, err_cap, "csat_attend_noalloc: tensor pointers must be 16-byte aligned");
      return CSAT_ERR_INVALID_ARG;
    }
  if (dtype != CSAT_DTYPE_BF16 && dtype != CSAT_DTYPE_FP32) {
    write_err(err_host, err_cap, "csat_attend_noalloc: unknown dtype");
    return CSAT_ERR_INVALID_ARG;
  }
  if (B < 1 || H < 1 || n < 1 || n_q < 1 || m < 1 || m > n || d < 8 || d > 256 || d % 8 != 0 || B * H > 65535 ||
      n > ((int64_t)1 << 31) || n_q > ((int64_t)1 << 31)) {
    write_err(err_host, err_cap, "csat_attend_noalloc: need B,H,n_q >= 1, 1 <= m <= n, 8 <= d <= 256, d % 8 == 0, B*H <= 65535");
    return CSAT_ERR_SHAPE;
  }
  const int64_t need = B * H * m * 2 * d * (int64_t)elt_size(dtype);
  if (need > (int64_t)CSAT_NOALLOC_SCRATCH_BYTES) {
    if (err_host && err_cap)
      snprintf(err_host, err_cap,
               "csat_attend_noalloc: K~|V~ needs %lld bytes (B*H*m*2d*elt) but the built-in scratch holds %lld; "
               "use csat_create/csat_forward for larger problems",
               (long long)need, (long long)CSAT_NOALLOC_SCRATCH_BYTES);
    return CSAT_ERR_SHAPE;
  }
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    write_err(err_host, err_cap, "csat_attend_noalloc: no usable current CUDA device");
    return CSAT_ERR_CUDA;
  }
  void* scratch = nullptr;
  {
    // once per device, with that device current: turn the host-side symbol into a device address
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
      void* p = nullptr;
      e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
      if (e != cudaSuccess || !p) {
        write_err(err_host, err_cap, cudaGetErrorString(e));
        return CSAT_ERR_CUDA;
      }
      g_noalloc_ptr[dev] = p;
    }
    scratch = g_noalloc_ptr[dev];
  }
  const float sc = (float)(scale > 0.0 ? scale : 1.0 / sqrt((double)d));
  cudaStream_t s = (cudaStream_t)stream;
  return dtype == CSAT_DTYPE_FP32
             ? attend_noalloc_t<float>(Q, K, V, phi, out, scratch, B, H, n, n_q, m, (int)d, sc, s, err_host, err_cap)
             : attend_noalloc_t<__nv_bfloat16>(Q, K, V, phi, out, scratch, B, H, n, n_q, m, (int)d, sc, s, err_host,
                                               err_cap);
}
