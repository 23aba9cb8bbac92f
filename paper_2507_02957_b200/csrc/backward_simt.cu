// Backward of the CSAT forward with respect to Q, K, V: the chain rule through the paper's equations, last to
// first (reconstruction C^ = Psi alpha, the unrolled recurrence alpha^{t+1} = eta_theta(alpha^t S + z B), the
// compressed output Z = A~ V~, the softmax, the scores S = Q K~^T / sqrt(d_k), the compression K~ = Phi K,
// V~ = Phi V).  The paper trains through the unrolled decoder but prints no backward pass; eta_theta has derivative
// 1 where |x| > theta and 0 elsewhere.
//
// First CUDA version: plain FFMA kernels, float32 arithmetic, nothing stored by the forward.  After the
// compression (the forward's own kernel) three kernels run:
//   transpose_kernel: float32 transposes of the decoder matrices S_t, B_t, so that every product below reads its
//                     matrix row by row (coalesced).
//   bwd_rows_kernel : one warp per query row.  Recomputes the row's scores, softmax statistics and Z, runs the
//                     recurrence forward keeping one bit per layer and column (|x_t| > theta_t), then backward:
//                     d alpha_T = G Psi, dx_t = d alpha_{t+1} o mask_t, dZ += dx_t B_t^T, d alpha_t = dx_t S_t^T
//                     (with one B for all layers dZ = (sum_t dx_t) B^T is a single product at the end).
//                     Stores dZ, L = log sum exp of the row's scores and D = <dZ, Z>, then sweeps K~|V~ again:
//                     p = exp(s - L), dS = p (dZ . V~_r - D), dQ = scale sum_r dS_r K~_r.
//   bwd_cols_kernel : one warp per measurement r, all query rows in turn (deterministic, no atomics):
//                     dK~_r = scale sum_i dS_ir Q_i,  dV~_r = sum_i p_ir dZ_i  (bf16 contexts with d in {64, 128}
//                     run this stage on the tensor cores instead: bwd_cols_sm100.cu).
//   bwd_phiT_kernel : dK = Phi^T dK~, dV = Phi_V^T dV~  (bf16 contexts with d in {64, 128} run this product on the
//                     tensor cores instead: phiT_sm100.cu, from a bf16 copy of dK~|dV~).
#include "csat_internal.h"

namespace csat {
namespace {

constexpr int kRowWarps = 8;
constexpr int kColWarps = 8;
constexpr int kColRows = 16;      // query rows staged per step of bwd_cols_kernel

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
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// lane owns columns lane + 32 j.  y[col] = sum_k x[k] W[k][col]
template <int DC>
__device__ __forceinline__ void row_times(const float (&x)[DC], float (&y)[DC], const float* __restrict__ W, int d, int lane) {
#pragma unroll
  for (int j = 0; j < DC; ++j) y[j] = 0.f;
#pragma unroll
  for (int jk = 0; jk < DC; ++jk)
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
// out[mat][a][b] = in[mat][b][a] for every d x d matrix
__global__ void transpose_kernel(float* __restrict__ out, const float* __restrict__ in, int d, int64_t mats) {
  const int64_t total = mats * d * d;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t mat = i / (d * d);
    const int a = (int)((i / d) % d), b = (int)(i % d);
    out[i] = in[mat * d * d + (int64_t)b * d + a];
  }
}

// out[(bh, row, c)] = sum over layers t of bit_t << t, from the forward kernel's record [bh][t][row][d / 32] in which
// column c is bit 31 - c % 32 of word c / 32
__global__ void expand_masks_kernel(uint32_t* __restrict__ out, const uint32_t* __restrict__ bits, int64_t total,
                                    int64_t nq, int d, int T) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int c = (int)(i % d);
  const int64_t row = (i / d) % nq, bh = i / (d * nq);
  uint32_t wv = 0;
  for (int t = 0; t < T; ++t) {
    const uint32_t m = bits[((bh * T + t) * nq + row) * (d / 32) + (c >> 5)];
    wv |= ((m >> (31 - (c & 31))) & 1u) << t;
  }
  out[i] = wv;
}

template <typename T, int DC>   // DC = ceil(d / 32)
__global__ void __launch_bounds__(kRowWarps * 32) bwd_rows_kernel(
    T* __restrict__ dQ, float* __restrict__ ws_dZ, __nv_bfloat16* __restrict__ ws_dZ16, float* __restrict__ ws_LD,
    const T* __restrict__ Q,
    const T* __restrict__ G, const T* __restrict__ kv, const float* __restrict__ S_dec, const float* __restrict__ B_dec,
    const float* __restrict__ S_decT, const float* __restrict__ B_decT, int64_t layer_stride, const float* __restrict__ theta, int theta_stride, const float* __restrict__ psi_f32,
    int64_t nq, int64_t m, int d, int H, int T_iters, float scale, uint32_t* __restrict__ ws_masks) {
  extern __shared__ float smem[];
  const int d2 = 2 * d, ldk = d2 + 1;
  float* kvs = smem;                               // [32][2d+1]
  float* qs = smem + 32 * ldk;                     // [warps][d]
  float* dzs = qs + kRowWarps * d;                 // [warps][d]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, h = bh % H;
  const int64_t row = (int64_t)blockIdx.x * kRowWarps + warp;
  const bool live = row < nq;
  const int64_t grow = (int64_t)bh * nq + (live ? row : 0);
  const T* kvb = kv + (int64_t)bh * m * d2;
  float* q = qs + warp * d;
  float* dzr = dzs + warp * d;
  for (int c = lane; c < d; c += 32) q[c] = live ? ldf(Q, grow * d + c) : 0.f;

  // ---- forward: scores, softmax statistics, Z ----
  float z[DC];
#pragma unroll
  for (int j = 0; j < DC; ++j) z[j] = 0.f;
  float run_max = -INFINITY, run_sum = 0.f;
  for (int64_t r0 = 0; r0 < m; r0 += 32) {
    __syncthreads();
    for (int i = threadIdx.x; i < 32 * d2; i += kRowWarps * 32) {
      const int rr = i / d2, c = i % d2;
      kvs[rr * ldk + c] = (r0 + rr < m) ? ldf(kvb, (r0 + rr) * d2 + c) : 0.f;
    }
    __syncthreads();
    float s = 0.f;
    const float* kr = kvs + lane * ldk;
    for (int c = 0; c < d; ++c) s = fmaf(q[c], kr[c], s);
    s = (r0 + lane < m) ? s * scale : -INFINITY;
    const float new_max = fmaxf(run_max, warp_max(s));
    const float corr = expf(run_max - new_max);
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
  const float L = run_max + logf(run_sum);          // log sum exp of the row's scaled scores

  // ---- recurrence forward (masks), then backward: dZ ----
  float g[DC], dz[DC];
#pragma unroll
  for (int j = 0; j < DC; ++j) {
    const int col = lane + 32 * j;
    g[j] = (live && col < d) ? ldf(G, grow * d + col) : 0.f;
  }
  if (T_iters == 0) {
#pragma unroll
    for (int j = 0; j < DC; ++j) dz[j] = g[j];
  } else {
    const float* Sh = S_dec + (int64_t)h * d * d;
    const float* Bh = B_dec + (int64_t)h * d * d;
    const float* ShT = S_decT + (int64_t)h * d * d;             // transposes: x W^T = row_times(x, W^T)
    const float* BhT = B_decT + (int64_t)h * d * d;
    uint32_t mask[DC];
    float a[DC], c[DC], t[DC];
#pragma unroll
    for (int j = 0; j < DC; ++j) { mask[j] = 0u; a[j] = 0.f; }
    for (int it = 0; it < T_iters; ++it) {
      const float th = theta[(int64_t)it * theta_stride + h];
      if (it == 0 || layer_stride != 0) row_times<DC>(z, c, Bh + layer_stride * it, d, lane);      // z B_t
      if (it > 0) row_times<DC>(a, t, Sh + layer_stride * it, d, lane);
#pragma unroll
      for (int j = 0; j < DC; ++j) {
        const float x = (it > 0 ? t[j] : 0.f) + c[j];
        if (fabsf(x) > th) mask[j] |= 1u << it;
        a[j] = x - fminf(fmaxf(x, -th), th);
      }
    }
    if (ws_masks && live) {
#pragma unroll
      for (int j = 0; j < DC; ++j) {
        const int col = lane + 32 * j;
        if (col < d) ws_masks[grow * d + col] = mask[j];          // bit t: |x_t| > theta_t
      }
    }
    float da[DC], dx[DC];
    if (psi_f32) row_times<DC>(g, da, psi_f32 + (int64_t)h * d * d, d, lane);     // d alpha_T = G Psi
    else {
#pragma unroll
      for (int j = 0; j < DC; ++j) da[j] = g[j];
    }
#pragma unroll
    for (int j = 0; j < DC; ++j) dz[j] = 0.f;
    for (int it = T_iters - 1; it >= 0; --it) {
#pragma unroll
      for (int j = 0; j < DC; ++j) dx[j] = ((mask[j] >> it) & 1u) ? da[j] : 0.f;
      if (layer_stride != 0) {
        row_times<DC>(dx, t, BhT + layer_stride * it, d, lane);                   // dZ += dx B_t^T
#pragma unroll
        for (int j = 0; j < DC; ++j) dz[j] += t[j];
      } else {
#pragma unroll
        for (int j = 0; j < DC; ++j) dz[j] += dx[j];                              // one B: sum the dx first
      }
      if (it > 0) row_times<DC>(dx, da, ShT + layer_stride * it, d, lane);        // d alpha_t = dx S_t^T
    }
    if (layer_stride == 0) {
#pragma unroll
      for (int j = 0; j < DC; ++j) dx[j] = dz[j];
      row_times<DC>(dx, dz, BhT, d, lane);                                        // dZ = (sum_t dx_t) B^T
    }
  }
  float part = 0.f;
#pragma unroll
  for (int j = 0; j < DC; ++j) part = fmaf(dz[j], z[j], part);
  const float Dr = warp_sum(part);                                                // <dZ, Z> = rowsum(dA o A)
#pragma unroll
  for (int j = 0; j < DC; ++j) {
    const int col = lane + 32 * j;
    if (col < d) {
      dzr[col] = dz[j];
      if (live) {
        ws_dZ[grow * d + col] = dz[j];
        if (ws_dZ16) ws_dZ16[grow * d + col] = __float2bfloat16_rn(dz[j]);     // operand of the tensor-core stage
      }
    }
  }
  if (live && lane == 0) { ws_LD[grow * 2] = L; ws_LD[grow * 2 + 1] = Dr; }

  // ---- second sweep: dS, dQ ----
  float dq[DC];
#pragma unroll
  for (int j = 0; j < DC; ++j) dq[j] = 0.f;
  for (int64_t r0 = 0; r0 < m; r0 += 32) {
    __syncthreads();
    for (int i = threadIdx.x; i < 32 * d2; i += kRowWarps * 32) {
      const int rr = i / d2, c = i % d2;
      kvs[rr * ldk + c] = (r0 + rr < m) ? ldf(kvb, (r0 + rr) * d2 + c) : 0.f;
    }
    __syncthreads();
    const float* kr = kvs + lane * ldk;
    float s = 0.f, dA = 0.f;
    for (int c = 0; c < d; ++c) {
      s = fmaf(q[c], kr[c], s);
      dA = fmaf(dzr[c], kr[d + c], dA);
    }
    const float p = (r0 + lane < m) ? expf(s * scale - L) : 0.f;
    const float dS = p * (dA - Dr);
    for (int rr = 0; rr < 32; ++rr) {
      const float ds = __shfl_sync(0xffffffffu, dS, rr);
      const float* krr = kvs + rr * ldk;
#pragma unroll
      for (int j = 0; j < DC; ++j) {
        const int col = lane + 32 * j;
        if (col < d) dq[j] = fmaf(ds, krr[col], dq[j]);
      }
    }
  }
  if (live) {
#pragma unroll
    for (int j = 0; j < DC; ++j) {
      const int col = lane + 32 * j;
      if (col < d) stf(dQ, grow * d + col, dq[j] * scale);
    }
  }
}

template <typename T, int DC>
__global__ void __launch_bounds__(kColWarps * 32) bwd_cols_kernel(
    float* __restrict__ ws_dKV, const T* __restrict__ Q, const T* __restrict__ kv, const float* __restrict__ ws_dZ,
    const float* __restrict__ ws_LD, int64_t nq, int64_t m, int d, float scale) {
  extern __shared__ float smem[];
  float* qt = smem;                                // [kColRows][d]
  float* dzt = qt + kColRows * d;                  // [kColRows][d]
  float* ldt = dzt + kColRows * d;                 // [kColRows][2]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y;
  const int64_t r = (int64_t)blockIdx.x * kColWarps + warp;
  const bool live = r < m;
  const T* kvr = kv + ((int64_t)bh * m + (live ? r : 0)) * 2 * d;
  float kr[DC], vr[DC], ak[DC], av[DC];
#pragma unroll
  for (int j = 0; j < DC; ++j) {
    const int col = lane + 32 * j;
    kr[j] = (col < d) ? ldf(kvr, col) : 0.f;
    vr[j] = (col < d) ? ldf(kvr, d + col) : 0.f;
    ak[j] = av[j] = 0.f;
  }
  for (int64_t i0 = 0; i0 < nq; i0 += kColRows) {
    __syncthreads();
    for (int i = threadIdx.x; i < kColRows * d; i += kColWarps * 32) {
      const int ii = i / d, c = i % d;
      const bool ok = i0 + ii < nq;
      const int64_t gi = (int64_t)bh * nq + i0 + ii;
      qt[i] = ok ? ldf(Q, gi * d + c) : 0.f;
      dzt[i] = ok ? ws_dZ[gi * d + c] : 0.f;
    }
    if (threadIdx.x < kColRows * 2) {
      const int ii = threadIdx.x >> 1;
      ldt[threadIdx.x] = (i0 + ii < nq) ? ws_LD[((int64_t)bh * nq + i0 + ii) * 2 + (threadIdx.x & 1)] : 0.f;
    }
    __syncthreads();
    const int cnt = (int)((nq - i0 < kColRows) ? nq - i0 : kColRows);
    for (int ii = 0; ii < cnt; ++ii) {
      float s = 0.f, dA = 0.f;
#pragma unroll
      for (int j = 0; j < DC; ++j) {
        const int col = lane + 32 * j;
        if (col < d) {
          s = fmaf(qt[ii * d + col], kr[j], s);
          dA = fmaf(dzt[ii * d + col], vr[j], dA);
        }
      }
      s = warp_sum(s);
      dA = warp_sum(dA);
      const float p = expf(s * scale - ldt[2 * ii]);
      const float dS = p * (dA - ldt[2 * ii + 1]);
#pragma unroll
      for (int j = 0; j < DC; ++j) {
        const int col = lane + 32 * j;
        if (col < d) {
          ak[j] = fmaf(dS, qt[ii * d + col], ak[j]);
          av[j] = fmaf(p, dzt[ii * d + col], av[j]);
        }
      }
    }
  }
  if (live) {
    float* o = ws_dKV + ((int64_t)bh * m + r) * 2 * d;
#pragma unroll
    for (int j = 0; j < DC; ++j) {
      const int col = lane + 32 * j;
      if (col < d) { o[col] = ak[j] * scale; o[d + col] = av[j]; }
    }
  }
}

// dK[j][c] = sum_r Phi_K[r][j] dK~[r][c],  dV[j][c] = sum_r Phi_V[r][j] dV~[r][c].
// Block = 64 tokens x 32 columns of K (blockIdx.z even) or V (odd); 256 threads, 4 tokens x 2 columns each;
// Phi and dK~|dV~ pass through shared memory 32 measurement rows at a time (Phi rows are read along the tokens).
constexpr int kPtTok = 64, kPtCol = 32, kPtRows = 32;
template <typename T>
__global__ void __launch_bounds__(256) bwd_phiT_kernel(T* __restrict__ dK, T* __restrict__ dV, const T* __restrict__ phi,
                                                       const float* __restrict__ ws_dKV, int64_t n, int64_t n_pad,
                                                       int64_t m, int d, int H, int phi_v_head0) {
  __shared__ float ps[kPtRows][kPtTok + 1];
  __shared__ float gs[kPtRows][kPtCol + 1];
  const int bh = blockIdx.z >> 1, is_v = blockIdx.z & 1, h = bh % H;
  const int64_t j0 = (int64_t)blockIdx.x * kPtTok;
  const int c0 = blockIdx.y * kPtCol;
  const T* ph = phi + (int64_t)((is_v ? phi_v_head0 : 0) + h) * m * n_pad;
  const float* g = ws_dKV + (int64_t)bh * m * 2 * d + (is_v ? d : 0);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;       // columns 2 tx, 2 tx + 1; tokens 4 ty .. 4 ty + 3
  float acc[4][2];
#pragma unroll
  for (int a = 0; a < 4; ++a) acc[a][0] = acc[a][1] = 0.f;
  for (int64_t r0 = 0; r0 < m; r0 += kPtRows) {
    __syncthreads();
    for (int i = threadIdx.x; i < kPtRows * kPtTok; i += 256) {
      const int rr = i / kPtTok, jj = i % kPtTok;
      ps[rr][jj] = (r0 + rr < m && j0 + jj < n) ? ldf(ph, (r0 + rr) * n_pad + j0 + jj) : 0.f;
    }
    for (int i = threadIdx.x; i < kPtRows * kPtCol; i += 256) {
      const int rr = i / kPtCol, cc = i % kPtCol;
      gs[rr][cc] = (r0 + rr < m && c0 + cc < d) ? g[(r0 + rr) * 2 * d + c0 + cc] : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int rr = 0; rr < kPtRows; ++rr) {
      const float g0 = gs[rr][2 * tx], g1 = gs[rr][2 * tx + 1];
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const float pv = ps[rr][4 * ty + a];
        acc[a][0] = fmaf(pv, g0, acc[a][0]);
        acc[a][1] = fmaf(pv, g1, acc[a][1]);
      }
    }
  }
  T* dst = is_v ? dV : dK;
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    const int64_t j = j0 + 4 * ty + a;
    if (j >= n) continue;
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int c = c0 + 2 * tx + u;
      if (c < d) stf(dst, ((int64_t)bh * n + j) * d + c, acc[a][u]);
    }
  }
}

template <typename T>
cudaError_t run(csat_ctx* c, const void* Q, const void* G, void* dQ, void* dK, void* dV, cudaStream_t s, int* launches) {
  const Params& p = c->p;
  const int d = (int)p.d, dc = (d + 31) / 32;
  const float scale = (float)(p.scale > 0.0 ? p.scale : 1.0 / sqrt((double)d));
  const unsigned BH = (unsigned)(p.B * p.H);
  const float* Sd = c->w_untied ? c->Sl_dec : c->S_dec;
  const float* Bd = c->w_untied ? c->Bl_dec : c->B_dec;
  const int64_t lstride = c->w_untied ? (int64_t)(p.H * p.d * p.d) : 0;
  cudaError_t e = cudaSuccess;
  // bf16 with d in {64, 128}: the stages after the per-row kernel run on the tensor cores
  const bool tc_stages = c->bw_dKV16 != nullptr && c->bw_dZ16 != nullptr && c->tmap_phi_valid && c->force_simt == 0;
  // ... and with one S, B for all layers the per-query stages too: the forward's attention phase leaves Z and the
  // rows' log sum exp, then the recurrence (forward with its decisions recorded, and backward) and dQ
  if (tc_stages && c->bw_Z16 != nullptr && (p.T == 0 || c->bw_maskbits != nullptr)) {
    const bool wg = c->weight_grads && p.T > 0 && c->bw_alpha16 != nullptr;
    if (!c->reuse_saved) {        // otherwise a csat_forward with CSAT_SAVE_FOR_BACKWARD has left all of it
      if (wg && (e = cudaMemsetAsync(c->bw_alpha16, 0, (size_t)(p.B * p.H * p.nq * p.d) * 2, s)) != cudaSuccess) return e;   // alpha^0
      if ((e = launch_sm100_attend_for_backward(c, Q, c->bw_Z16, c->bw_LD, 2, c->bw_maskbits, wg ? c->bw_alpha16 : nullptr,
                                                s, launches)) != cudaSuccess)
        return e;
    }
    if (c->bw_masks != nullptr && p.T > 0) {           // CSAT_KEEP_MASKS: the decisions in the exported layout
      const int64_t total = p.B * p.H * p.nq * p.d;
      expand_masks_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(c->bw_masks, c->bw_maskbits, total, p.nq, d, p.T);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
      *launches += 1;
    }
    if ((e = launch_sm100_bwd_recur(c, G, s, launches)) != cudaSuccess) return e;
    if (wg && (e = launch_sm100_wgrad(c, G, s, launches)) != cudaSuccess) return e;
    if ((e = launch_sm100_bwd_dq(c, Q, dQ, s, launches)) != cudaSuccess) return e;
    if ((e = launch_sm100_bwd_cols(c, Q, s, launches)) != cudaSuccess) return e;
    return launch_sm100_phiT(c, c->bw_dKV16, dK, dV, s, launches);
  }
  const int64_t mats = (c->w_untied ? c->w_layers : 1) * p.H;
  float* SdT = c->bw_WT;
  float* BdT = c->bw_WT + mats * d * d;
  if (p.T > 0) {
    const int64_t total = mats * d * d;
    const unsigned tg = (unsigned)((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
    transpose_kernel<<<tg, 256, 0, s>>>(SdT, Sd, d, mats);
    transpose_kernel<<<tg, 256, 0, s>>>(BdT, Bd, d, mats);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    *launches += 2;
  }
  {
    const dim3 grid((unsigned)((p.nq + kRowWarps - 1) / kRowWarps), BH);
    const size_t sm = (size_t)(32 * (2 * d + 1) + 2 * kRowWarps * d) * sizeof(float);
#define CSAT_BWD_ROWS(DC)                                                                                            \
  do {                                                                                                               \
    if (sm > 48 * 1024)                                                                                              \
      e = cudaFuncSetAttribute(bwd_rows_kernel<T, DC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);        \
    if (e == cudaSuccess)                                                                                            \
      bwd_rows_kernel<T, DC><<<grid, kRowWarps * 32, sm, s>>>(                                                       \
          (T*)dQ, c->bw_dZ, tc_stages ? c->bw_dZ16 : nullptr, c->bw_LD, (const T*)Q, (const T*)G, (const T*)c->kv, Sd, Bd, SdT, BdT, lstride, c->thr(), \
          c->thr_stride(), c->psi ? c->psi_f32 : nullptr, p.nq, p.m, d, (int)p.H, p.T, scale, c->bw_masks);          \
  } while (0)
    if (dc <= 2) CSAT_BWD_ROWS(2);
    else if (dc <= 4) CSAT_BWD_ROWS(4);
    else CSAT_BWD_ROWS(8);
#undef CSAT_BWD_ROWS
    if (e != cudaSuccess) return e;
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  if (tc_stages) {
    // dK~, dV~ and dK, dV on the tensor cores
    if ((e = launch_sm100_bwd_cols(c, Q, s, launches)) != cudaSuccess) return e;
    if ((e = launch_sm100_phiT(c, c->bw_dKV16, dK, dV, s, launches)) != cudaSuccess) return e;
    *launches += 1;
    return cudaSuccess;
  }
  {
    const dim3 grid((unsigned)((p.m + kColWarps - 1) / kColWarps), BH);
    const size_t sm = (size_t)(2 * kColRows * d + 2 * kColRows) * sizeof(float);
#define CSAT_BWD_COLS(DC)                                                                                            \
  bwd_cols_kernel<T, DC><<<grid, kColWarps * 32, sm, s>>>(c->bw_dKV, (const T*)Q, (const T*)c->kv, c->bw_dZ, c->bw_LD, \
                                                         p.nq, p.m, d, scale)
    if (dc <= 2) CSAT_BWD_COLS(2);
    else if (dc <= 4) CSAT_BWD_COLS(4);
    else CSAT_BWD_COLS(8);
#undef CSAT_BWD_COLS
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  {
    const dim3 grid((unsigned)((p.n + kPtTok - 1) / kPtTok), (unsigned)((d + kPtCol - 1) / kPtCol), BH * 2);
    bwd_phiT_kernel<T><<<grid, 256, 0, s>>>((T*)dK, (T*)dV, (const T*)c->phi, c->bw_dKV, p.n, p.n_pad, p.m, d,
                                                (int)p.H, p.separate_phi ? (int)p.H : 0);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  *launches += 3;
  return cudaSuccess;
}

}  // namespace

// K~|V~ must already be in the workspace (the forward's compression of the same K, V)
cudaError_t launch_backward(csat_ctx* c, const void* Q, const void* G, void* dQ, void* dK, void* dV, cudaStream_t s,
                            int* launches) {
  return c->p.dtype == CSAT_DTYPE_FP32 ? run<float>(c, Q, G, dQ, dK, dV, s, launches)
                                       : run<__nv_bfloat16>(c, Q, G, dQ, dK, dV, s, launches);
}

}  // namespace csat
