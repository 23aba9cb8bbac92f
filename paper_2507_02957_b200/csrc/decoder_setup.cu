// Decoder set-up, once per parameter change and per head (tiny: d x d matrices, float64 arithmetic).
// Paper: LISTA recurrence alpha^{t+1} = eta_theta(S alpha^t + B Z_i) with S, B, theta taken from ISTA
// (the paper names ISTA among the approximate solvers it allows) for the model Z_i = D Psi alpha_i:
//   M = D Psi, G = M^T M, L^ = max_a sum_b |G[a][b]|, mu = 1/L^ (or the caller's step),
//   S = I - mu G, B = mu M, theta = mu lambda.
// D defaults to the leading d x d block of the head's Phi (the paper decodes with the values' measurement matrix).
#include "csat_internal.h"

namespace csat {
namespace {

template <typename T> __device__ __forceinline__ double ld(const T* p, int64_t i);
template <> __device__ __forceinline__ double ld<float>(const float* p, int64_t i) { return (double)p[i]; }
template <> __device__ __forceinline__ double ld<__nv_bfloat16>(const __nv_bfloat16* p, int64_t i) {
  return (double)__bfloat162float(p[i]);
}

// M[h][a][b] = sum_k D[h][a][k] * Psi[h][k][b]
template <typename T>
__global__ void build_M_kernel(double* __restrict__ M, const T* __restrict__ phi, const T* __restrict__ dmat,
                               const T* __restrict__ psi, int psi_per_head, int d, int64_t m, int64_t n_pad, int phi_head0) {
  const int h = blockIdx.y;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= d * d) return;
  const int a = idx / d, b = idx % d;
  const T* Dh = dmat ? dmat + (int64_t)h * d * d : phi + (int64_t)(phi_head0 + h) * m * n_pad;   // block of Phi_V
  const int64_t ldD = dmat ? d : n_pad;
  double acc;
  if (psi) {
    const T* P = psi + (psi_per_head ? (int64_t)h * d * d : 0);
    acc = 0.0;
    for (int k = 0; k < d; ++k) acc += ld(Dh, a * ldD + k) * ld(P, (int64_t)k * d + b);
  } else {
    acc = ld(Dh, a * ldD + b);
  }
  M[(int64_t)h * d * d + idx] = acc;
}

// G[h][a][b] = sum_k M[h][k][a] * M[h][k][b]
__global__ void gram_kernel(double* __restrict__ G, const double* __restrict__ M, int d) {
  const int h = blockIdx.y;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= d * d) return;
  const int a = idx / d, b = idx % d;
  const double* Mh = M + (int64_t)h * d * d;
  double acc = 0.0;
  for (int k = 0; k < d; ++k) acc += Mh[k * d + a] * Mh[k * d + b];
  G[(int64_t)h * d * d + idx] = acc;
}

// one block per head; blockDim.x >= d (power of two <= 256)
template <typename T>
__global__ void finalize_kernel(float* __restrict__ S_dec, float* __restrict__ B_dec, float* __restrict__ theta,
                                float* __restrict__ mu_out, float* __restrict__ psi_f32, const double* __restrict__ G,
                                const double* __restrict__ M, const T* __restrict__ psi, int psi_per_head, int d,
                                double lambda, double step, __nv_bfloat16* __restrict__ mats_bf16) {
  __shared__ double red[256];
  const int h = blockIdx.x, t = threadIdx.x;
  const double* Gh = G + (int64_t)h * d * d;
  const double* Mh = M + (int64_t)h * d * d;
  double rs = 0.0;
  if (t < d)
    for (int b = 0; b < d; ++b) rs += fabs(Gh[t * d + b]);
  red[t] = rs;
  __syncthreads();
  for (int s = blockDim.x >> 1; s > 0; s >>= 1) {   // max is order-independent: deterministic
    if (t < s) red[t] = fmax(red[t], red[t + s]);
    __syncthreads();
  }
  const double L = red[0];
  const double mu = step > 0.0 ? step : (L > 0.0 ? 1.0 / L : 0.0);
  for (int i = t; i < d * d; i += blockDim.x) {
    const int a = i / d, b = i % d;
    S_dec[(int64_t)h * d * d + i] = (float)((a == b ? 1.0 : 0.0) - mu * Gh[i]);
    B_dec[(int64_t)h * d * d + i] = (float)(mu * Mh[i]);
    if (psi) psi_f32[(int64_t)h * d * d + i] = (float)ld(psi + (psi_per_head ? (int64_t)h * d * d : 0), i);
    if (mats_bf16) {
      // tensor-core operand copies, each stored [output column][k]: -mu G (symmetric), (mu M)^T, Psi
      __nv_bfloat16* mh = mats_bf16 + (int64_t)h * 3 * d * d;
      mh[i] = __float2bfloat16_rn((float)(-mu * Gh[i]));
      mh[d * d + i] = __float2bfloat16_rn((float)(mu * Mh[b * d + a]));
      mh[2 * d * d + i] =
          psi ? __float2bfloat16_rn((float)ld(psi + (psi_per_head ? (int64_t)h * d * d : 0), i)) : __float2bfloat16_rn(0.f);
    }
  }
  if (t == 0) {
    theta[h] = (float)(mu * lambda);
    mu_out[h] = (float)mu;
  }
}

// Supplied LISTA weights: S, B as given (float32 copies for the FFMA kernels), and the tensor-core operand
// copies, each stored [output column][k]: S - I (so that alpha S = alpha + alpha (S - I)), B, Psi.
template <typename T>
__global__ void weights_kernel(float* __restrict__ S_dec, float* __restrict__ B_dec, float* __restrict__ mu_out,
                               float* __restrict__ psi_f32, const T* __restrict__ S, const T* __restrict__ Bm,
                               const T* __restrict__ psi, int psi_per_head, int d,
                               __nv_bfloat16* __restrict__ mats_bf16) {
  const int h = blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= d * d) return;
  const int a = i / d, b = i % d;
  const int64_t base = (int64_t)h * d * d;
  S_dec[base + i] = (float)ld(S, base + i);
  B_dec[base + i] = (float)ld(Bm, base + i);
  const T* P = psi ? psi + (psi_per_head ? base : 0) : nullptr;
  if (P) psi_f32[base + i] = (float)ld(P, i);
  if (mats_bf16) {
    __nv_bfloat16* mh = mats_bf16 + base * 3;
    mh[i] = __float2bfloat16_rn((float)(ld(S, base + (int64_t)b * d + a) - (a == b ? 1.0 : 0.0)));   // (S - I)[b][a]
    mh[d * d + i] = __float2bfloat16_rn((float)ld(Bm, base + (int64_t)b * d + a));                    // B[b][a]
    mh[2 * d * d + i] = P ? __float2bfloat16_rn((float)ld(P, i)) : __float2bfloat16_rn(0.f);
  }
  if (i == 0) mu_out[h] = 0.f;
}

// Supplied LISTA weights with one S_t, B_t per layer (grid z = layer): float32 copies [L, H, d, d] for the FFMA
// kernels, and the tensor-core operands of head h at lmats[h][2t] = S_t - I and lmats[h][2t + 1] = B_t, each stored
// [output column][k] (layer t is the product [alpha^t | z] [S_t - I ; B_t], added to alpha^t), lmats[h][2L] = Psi.
// Layer 0 also goes to S_dec / B_dec (what csat_get_decoder returns).
template <typename T>
__global__ void layer_weights_kernel(float* __restrict__ Sl_dec, float* __restrict__ Bl_dec, float* __restrict__ S_dec,
                                     float* __restrict__ B_dec, float* __restrict__ mu_out, float* __restrict__ psi_f32,
                                     const T* __restrict__ S, const T* __restrict__ Bm, const T* __restrict__ psi,
                                     int psi_per_head, int d, int H, int L, __nv_bfloat16* __restrict__ lmats) {
  const int h = blockIdx.y, l = blockIdx.z;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= d * d) return;
  const int a = i / d, b = i % d;
  const int64_t dd = (int64_t)d * d;
  const int64_t src = ((int64_t)l * H + h) * dd;
  const float sv = (float)ld(S, src + i), bv = (float)ld(Bm, src + i);
  Sl_dec[src + i] = sv;
  Bl_dec[src + i] = bv;
  const T* P = psi ? psi + (psi_per_head ? (int64_t)h * dd : 0) : nullptr;
  if (l == 0) {
    S_dec[(int64_t)h * dd + i] = sv;
    B_dec[(int64_t)h * dd + i] = bv;
    if (P) psi_f32[(int64_t)h * dd + i] = (float)ld(P, i);
    if (i == 0) mu_out[h] = 0.f;
  }
  if (lmats) {
    __nv_bfloat16* mh = lmats + (int64_t)h * (2 * L + 1) * dd;
    mh[(int64_t)(2 * l) * dd + i] =
        __float2bfloat16_rn((float)(ld(S, src + (int64_t)b * d + a) - (a == b ? 1.0 : 0.0)));             // (S_t - I)[b][a]
    mh[(int64_t)(2 * l + 1) * dd + i] = __float2bfloat16_rn((float)ld(Bm, src + (int64_t)b * d + a));    // B_t[b][a]
    if (l == 0) mh[(int64_t)(2 * L) * dd + i] = P ? __float2bfloat16_rn((float)ld(P, i)) : __float2bfloat16_rn(0.f);
  }
}

template <typename T>
cudaError_t run(csat_ctx* c, cudaStream_t s, int* launches) {
  const Params& p = c->p;
  const int d = (int)p.d, H = (int)p.H;
  const dim3 grid((d * d + 255) / 256, H);
  if (c->w_S && c->w_untied) {
    const dim3 lgrid(grid.x, H, c->w_layers);
    layer_weights_kernel<T><<<lgrid, 256, 0, s>>>(c->Sl_dec, c->Bl_dec, c->S_dec, c->B_dec, c->mu, c->psi_f32,
                                                  (const T*)c->w_S, (const T*)c->w_B, (const T*)c->psi,
                                                  c->psi_per_head ? 1 : 0, d, H, c->w_layers, c->lmats_bf16);
    *launches += 1;
    return cudaGetLastError();
  }
  if (c->w_S) {
    weights_kernel<T><<<grid, 256, 0, s>>>(c->S_dec, c->B_dec, c->mu, c->psi_f32, (const T*)c->w_S, (const T*)c->w_B,
                                           (const T*)c->psi, c->psi_per_head ? 1 : 0, d, c->mats_bf16);
    *launches += 1;
    return cudaGetLastError();
  }
  build_M_kernel<T><<<grid, 256, 0, s>>>(c->Mf64, (const T*)c->phi, (const T*)c->dmat, (const T*)c->psi,
                                         c->psi_per_head ? 1 : 0, d, p.m, p.n_pad, p.separate_phi ? (int)p.H : 0);
  gram_kernel<<<grid, 256, 0, s>>>(c->Gf64, c->Mf64, d);
  finalize_kernel<T><<<H, 256, 0, s>>>(c->S_dec, c->B_dec, c->theta, c->mu, c->psi_f32, c->Gf64, c->Mf64,
                                       (const T*)c->psi, c->psi_per_head ? 1 : 0, d, p.lambda, p.step, c->mats_bf16);
  *launches += 3;
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decoder_setup(csat_ctx* c, cudaStream_t s, int* launches) {
  return c->p.dtype == CSAT_DTYPE_FP32 ? run<float>(c, s, launches) : run<__nv_bfloat16>(c, s, launches);
}

}  // namespace csat
