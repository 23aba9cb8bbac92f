// Gradients with respect to the decoder's parameters (paper: the sparse decoder is an unrolled network whose S, B,
// theta and dictionary Psi are trained by backpropagation; the paper prints no backward pass, this is the chain rule
// through x_t = alpha^t S + Z B, alpha^{t+1} = eta_theta(x_t), C^ = alpha^T Psi^T):
//   dS     = sum_t  (alpha^t)^T dx_t          dB = sum_t Z^T dx_t          (one S, B for all layers: summed over t)
//   dtheta_t = - sum  sign(x_t) o dx_t        (sign(x_t) = sign(alpha^{t+1}) wherever dx_t is not zero)
//   dPsi   = G^T alpha^T
// each summed over the queries and over the batch, per head (dPsi also over the heads: one dictionary).
// The forward kernel (run for the backward pass) leaves the iterates alpha^0 .. alpha^T and the recurrence kernel the
// dx_t, both bf16 [slot][B,H,n_q,d]; here they are only contracted:
//
// wgrad_gram_kernel: C = sum over a list of (slab pairs) of A1^T B and A2^T B, slabs = [n_q x d] bf16 matrices.
//   One CTA sums a range of (batch element, 128-row tile) units of one head over all layers: TMA brings the three
//   tiles (A1, A2, B) of a (unit, layer) into a ring stage; a tile of 128 rows x d with 128-byte rows is an
//   MN-major operand when its rows are the reduction index, so A1^T B needs no transposed copy.  d = 128: two
//   accumulators [128 x 128] in tensor memory; d = 64: A1 | A2 side by side form one M = 128 operand and one
//   accumulator [128 x 64] holds A1^T B over A2^T B.  The CTA's sums go to a partial buffer; a second kernel adds the
//   partials in a fixed order (no atomics: the result is the same bits on every run).
// dtheta_kernel / reduce kernels: plain loads and adds.
#include "csat_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace csat {
namespace {

using namespace ptx;

constexpr int kRows = 128;
constexpr int kThreads = 192;          // warps 0-3: epilogue (TMEM lane = row of C), warp 4: TMA, warp 5: MMA

template <int D> struct GCfg {
  static constexpr int kDBoxes = D / 64;
  static constexpr int kStages = (D == 64) ? 4 : 2;
  static constexpr uint32_t kBoxBytes = kRows * 128;                 // 128 rows x 64 columns
  static constexpr uint32_t kTileBytes = kDBoxes * kBoxBytes;
  static constexpr uint32_t kStageBytes = 3 * kTileBytes;            // A1 | A2 | B
  static constexpr uint32_t kOffBar = kStages * kStageBytes;
  static constexpr uint32_t kSmemBytes = kOffBar + 256 + 1024;
  static constexpr uint32_t kTmemCols = (D == 64) ? 64 : 256;
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
};

struct GBars {
  uint64_t full[4], empty[4], acc_done;
  uint32_t tmem_slot;
  int abort;
};

// slab of (batch element b, head h, layer t) in a [slot][B,H] tensor: off + t * tstride + b * H + h
struct SlabIndex { int off, tstride; };

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
wgrad_gram_kernel(const __grid_constant__ CUtensorMap tmap_a1, const __grid_constant__ CUtensorMap tmap_a2,
                  const __grid_constant__ CUtensorMap tmap_b, SlabIndex ia1, SlabIndex ia2, SlabIndex ib,
                  float* __restrict__ part, int nq, int H, int B, int nt, int units_per_cta, int* status) {
  using C = GCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  GBars* bars = reinterpret_cast<GBars*>(smem + C::kOffBar);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.y, split = blockIdx.x;
  const int ntiles = (nq + kRows - 1) / kRows;
  const int total = B * ntiles;
  const int u0 = split * units_per_cta, u1 = min(total, u0 + units_per_cta);
  const int steps = (u1 > u0 ? (u1 - u0) : 0) * nt;              // (unit, layer) pairs of this CTA

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_a1);
    prefetch_tmap(&tmap_a2);
    prefetch_tmap(&tmap_b);
    for (int s = 0; s < C::kStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
    mbar_init(&bars->acc_done, 1);
    bars->abort = 0;
    fence_mbar_init();
  }
  if (warp == 5) {
    tmem_alloc(&bars->tmem_slot, C::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_slot;

  if (warp == 4) {
    if (elect_one()) {
      bool ok = true;
      int issued = 0;
      for (int i = 0; i < steps && ok; ++i) {
        const int s = i % C::kStages;
        if (i >= C::kStages) ok = mbar_wait(&bars->empty[s], ((i / C::kStages) & 1) ^ 1, status, 701, &bars->abort);
        if (!ok) break;
        const int u = u0 + i / nt, t = (int)blockIdx.z + i % nt, b = u / ntiles, tile = u % ntiles;
        const int bh = b * H + h;
        uint8_t* st = smem + (uint32_t)s * C::kStageBytes;
        mbar_arrive_expect_tx(&bars->full[s], C::kStageBytes);
        for (int gx = 0; gx < C::kDBoxes; ++gx) {
          tma_load_3d(st + gx * C::kBoxBytes, &tmap_a1, &bars->full[s], gx * 64, tile * kRows, ia1.off + t * ia1.tstride + bh);
          tma_load_3d(st + C::kTileBytes + gx * C::kBoxBytes, &tmap_a2, &bars->full[s], gx * 64, tile * kRows,
                      ia2.off + t * ia2.tstride + bh);
          tma_load_3d(st + 2 * C::kTileBytes + gx * C::kBoxBytes, &tmap_b, &bars->full[s], gx * 64, tile * kRows,
                      ib.off + t * ib.tstride + bh);
        }
        ++issued;
      }
      if (!ok)                                     // gave up: let the copies in flight land before the CTA exits
        for (int i = issued > C::kStages ? issued - C::kStages : 0; i < issued; ++i)
          mbar_wait_drain(&bars->full[i % C::kStages], (i / C::kStages) & 1);
    }
  } else if (warp == 5) {
    if (elect_one()) {
      // both operands MN-major: rows = the reduction index; the next 64 elements along M / N start one box further;
      // 16 reduction rows = 2048 bytes.  d = 64: A1 | A2 are two adjacent boxes = one operand with M = 128
      constexpr uint32_t idesc = make_idesc_bf16(kRows, D, true, true);
      const uint64_t a0 = make_smem_desc(smem_u32(smem), C::kBoxBytes, 1024);
      constexpr uint64_t kStageStep = C::kStageBytes >> 4, kTileStep = C::kTileBytes >> 4;
      bool ok = true;
      for (int i = 0; i < steps && ok; ++i) {
        const int s = i % C::kStages;
        ok = mbar_wait(&bars->full[s], (i / C::kStages) & 1, status, 702, &bars->abort);
        if (!ok) break;
        tc_fence_after();
        const uint64_t d1 = a0 + (uint64_t)s * kStageStep, d2 = d1 + kTileStep, db = d1 + 2 * kTileStep;
#pragma unroll
        for (int k = 0; k < kRows / 16; ++k) {
          if (D == 64) {
            mma_f16_ss(tmem, d1 + (uint64_t)(k * 128), db + (uint64_t)(k * 128), idesc, (i | k) != 0);
          } else {
            mma_f16_ss(tmem, d1 + (uint64_t)(k * 128), db + (uint64_t)(k * 128), idesc, (i | k) != 0);
            mma_f16_ss(tmem + D, d2 + (uint64_t)(k * 128), db + (uint64_t)(k * 128), idesc, (i | k) != 0);
          }
        }
        mma_commit(&bars->empty[s]);
      }
      if (ok) mma_commit(&bars->acc_done);
    }
  } else {
    // epilogue: lane = row of C (d = 128: row i of A1^T B and of A2^T B; d = 64: rows 0-63 A1^T B, 64-127 A2^T B)
    const int row = warp * 32 + lane;
    const uint32_t tbase = tmem + ((uint32_t)(warp * 32) << 16);
    float* p1 = part + ((int64_t)((blockIdx.z * gridDim.x + split) * H + h) * 2) * D * D;       // [2][D][D]
    const bool have = steps > 0;
    bool ok = true;
    if (have) ok = mbar_wait(&bars->acc_done, 0, status, 703, &bars->abort) && *(volatile int*)&bars->abort == 0;
    ok = __all_sync(0xffffffffu, ok);
    if (have && ok) tc_fence_after();
    constexpr int kAccs = (D == 64) ? 1 : 2;
#pragma unroll 1
    for (int a = 0; a < kAccs; ++a) {
#pragma unroll 1
      for (int c0 = 0; c0 < D; c0 += 16) {
        uint32_t v[16];
        if (have && ok) {                          // uniform over the warp
          tmem_ld_32x32b_x16(tbase + a * D + c0, v);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int e = 0; e < 16; ++e) v[e] = 0u;   // a CTA without units contributes zeros
        }
        if (ok) {
          float* o = (D == 64) ? p1 + ((int64_t)(row >> 6) * D + (row & 63)) * D + c0 : p1 + ((int64_t)a * D + row) * D + c0;
#pragma unroll
          for (int e = 0; e < 16; e += 4)
            *reinterpret_cast<float4*>(o + e) = make_float4(__uint_as_float(v[e]), __uint_as_float(v[e + 1]),
                                                            __uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, C::kTmemCols);
}

// out[z][h][i] = sum over the splits, in order, of part[z][split][h][which][i]   (i over d*d; z = layer with one pair of
// matrices per layer, else 0); all heads into out[i] with `over_heads` (the dictionary is shared by the heads)
__global__ void wgrad_reduce_kernel(float* __restrict__ out, const float* __restrict__ part, int splits, int H, int Z,
                                    int which, int64_t dd, int over_heads) {
  const int64_t total = (over_heads ? 1 : (int64_t)Z * H) * dd;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t e = i % dd;
    float acc = 0.f;
    if (over_heads) {
      for (int h = 0; h < H; ++h)
        for (int s = 0; s < splits; ++s) acc += part[(((int64_t)s * H + h) * 2 + which) * dd + e];
    } else {
      const int64_t zh = i / dd, z = zh / H, h = zh % H;
      for (int s = 0; s < splits; ++s) acc += part[((((int64_t)z * splits + s) * H + h) * 2 + which) * dd + e];
    }
    out[i] = acc;
  }
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

// partial[chunk][t][h] = - sum over the chunk's share of (batch element, query, column) of sign(alpha^{t+1}) dx_t
// (sign taken from the stored iterate's sign bit; where the iterate is zero dx_t is zero too)
constexpr int kThThreads = 256;
__global__ void __launch_bounds__(kThThreads)
dtheta_partial_kernel(float* __restrict__ partial, const __nv_bfloat16* __restrict__ alpha,
                      const __nv_bfloat16* __restrict__ dx, int64_t slot, int64_t per_bh, int B, int H, int T) {
  const int h = blockIdx.y, t = blockIdx.z, chunk = blockIdx.x, chunks = gridDim.x;
  const int64_t vec_per_bh = per_bh / 8;                           // 8 bf16 = 16 bytes
  const int64_t total = (int64_t)B * vec_per_bh;
  float acc = 0.f;
  for (int64_t i = (int64_t)chunk * kThThreads + threadIdx.x; i < total; i += (int64_t)chunks * kThThreads) {
    const int64_t b = i / vec_per_bh, r = i % vec_per_bh;
    const int64_t off = ((b * H + h) * per_bh) + r * 8;
    const uint4 a = *reinterpret_cast<const uint4*>(alpha + (int64_t)(t + 1) * slot + off);
    const uint4 x = *reinterpret_cast<const uint4*>(dx + (int64_t)t * slot + off);
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, xw[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint32_t f = xw[q] ^ (aw[q] & 0x80008000u);            // dx with the iterate's sign applied
      acc += bf16_bits_to_float(f & 0xffffu) + bf16_bits_to_float(f >> 16);
    }
  }
  // fixed-order block sum
  __shared__ float sh[kThThreads];
  sh[threadIdx.x] = acc;
  __syncthreads();
  for (int w = kThThreads / 2; w > 0; w >>= 1) {
    if (threadIdx.x < w) sh[threadIdx.x] += sh[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) partial[((int64_t)chunk * T + t) * H + h] = -sh[0];
}

__global__ void dtheta_reduce_kernel(float* __restrict__ out, const float* __restrict__ partial, int chunks, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float acc = 0.f;
  for (int c = 0; c < chunks; ++c) acc += partial[(int64_t)c * n + i];
  out[i] = acc;
}

cudaError_t slab_map(CUtensorMap* m, const void* base, const Params& p, int64_t slabs) {
  const uint64_t dims[3] = {(uint64_t)p.d, (uint64_t)p.nq, (uint64_t)slabs};
  const uint64_t strides[2] = {(uint64_t)p.d * 2, (uint64_t)p.nq * p.d * 2};
  const uint32_t box[3] = {64, (uint32_t)kRows, 1};
  return make_tmap_bf16_3d(m, base, dims, strides, box);
}

template <int D>
cudaError_t launch_gram(csat_ctx* c, const CUtensorMap& a1, const CUtensorMap& a2, const CUtensorMap& b, SlabIndex ia1,
                        SlabIndex ia2, SlabIndex ib, int nt, int splits, int units_per_cta, cudaStream_t s, int layers_z = 1) {
  using C = GCfg<D>;
  static DeviceFlags smem_opt_in;
  cudaError_t e = ensure_dynamic_smem(wgrad_gram_kernel<D>, (int)C::kSmemBytes, c->device, smem_opt_in);
  if (e != cudaSuccess) return e;
  const Params& p = c->p;
  wgrad_gram_kernel<D><<<dim3((unsigned)splits, (unsigned)p.H, (unsigned)layers_z), kThreads, C::kSmemBytes, s>>>(
      a1, a2, b, ia1, ia2, ib, c->bw_wpart, (int)p.nq, (int)p.H, (int)p.B, nt, units_per_cta, c->status);
  return cudaGetLastError();
}

}  // namespace

int wgrad_splits(const csat_ctx* c) {
  const Params& p = c->p;
  const int64_t units = p.B * ((p.nq + kRows - 1) / kRows);
  // one wave: at most sms CTAs in all; with one pair of matrices per layer every (head, layer) has its own CTAs
  int64_t s = c->sms / (p.H * (c->w_untied && p.T > 0 ? p.T : 1));
  if (s > units) s = units;
  return (int)(s < 1 ? 1 : s);
}

// needs bw_alpha16 (slots 0 .. T, slot 0 cleared), bw_dx16 (slots 0 .. T-1), bw_Z16 and G; fills bw_wgrad:
// dS [H,d,d] | dB [H,d,d] | dPsi [d,d] | dtheta [T,H]
cudaError_t launch_sm100_wgrad(csat_ctx* c, const void* G, cudaStream_t s, int* launches) {
  const Params& p = c->p;
  const int64_t BH = p.B * p.H, dd = p.d * p.d;
  const int splits = wgrad_splits(c);
  const int64_t units = p.B * ((p.nq + kRows - 1) / kRows);
  const int upc = (int)((units + splits - 1) / splits);
  CUtensorMap ta, tx, tz, tg;
  cudaError_t e;
  if ((e = slab_map(&ta, c->bw_alpha16, p, (p.T + 1) * BH)) != cudaSuccess) return e;
  if ((e = slab_map(&tx, c->bw_dx16, p, p.T * BH)) != cudaSuccess) return e;
  if ((e = slab_map(&tz, c->bw_Z16, p, BH)) != cudaSuccess) return e;
  if ((e = slab_map(&tg, G, p, BH)) != cudaSuccess) return e;
  // dS [Z,H,d,d] | dB [Z,H,d,d] | dPsi [d,d] | dtheta [T,H]; Z = T with one S_t, B_t per layer, else 1
  const int Z = (c->w_untied && p.T > 0) ? p.T : 1;
  float* dS = c->bw_wgrad;
  float* dB = dS + (int64_t)Z * p.H * dd;
  float* dPsi = dB + (int64_t)Z * p.H * dd;
  float* dTh = dPsi + dd;
  const unsigned rblocks = (unsigned)(((int64_t)Z * p.H * dd + 255) / 256);
  // dS = sum_t (alpha^t)^T dx_t, dB = sum_t Z^T dx_t (per layer: no sum over t, the layer is the grid's z index)
  const SlabIndex ia{0, (int)BH}, iz{0, 0}, ix{0, (int)BH};
  const int nt = Z > 1 ? 1 : p.T;
  e = p.d == 64 ? launch_gram<64>(c, ta, tz, tx, ia, iz, ix, nt, splits, upc, s, Z)
                : launch_gram<128>(c, ta, tz, tx, ia, iz, ix, nt, splits, upc, s, Z);
  if (e != cudaSuccess) return e;
  wgrad_reduce_kernel<<<rblocks, 256, 0, s>>>(dS, c->bw_wpart, splits, (int)p.H, Z, 0, dd, 0);
  wgrad_reduce_kernel<<<rblocks, 256, 0, s>>>(dB, c->bw_wpart, splits, (int)p.H, Z, 1, dd, 0);
  *launches += 3;
  if (c->psi) {
    // dPsi = G^T alpha^T: A1 = A2 = G, B = slot T of the iterates, one "layer"
    const SlabIndex ig{0, 0}, iaT{(int)(p.T * BH), 0};
    e = p.d == 64 ? launch_gram<64>(c, tg, tg, ta, ig, ig, iaT, 1, splits, upc, s)
                  : launch_gram<128>(c, tg, tg, ta, ig, ig, iaT, 1, splits, upc, s);
    if (e != cudaSuccess) return e;
    wgrad_reduce_kernel<<<(unsigned)((dd + 255) / 256), 256, 0, s>>>(dPsi, c->bw_wpart, splits, (int)p.H, 1, 0, dd, 1);
    *launches += 2;
  } else {
    if ((e = cudaMemsetAsync(dPsi, 0, (size_t)dd * 4, s)) != cudaSuccess) return e;
  }
  // dtheta
  const int chunks = 64;
  dtheta_partial_kernel<<<dim3(chunks, (unsigned)p.H, (unsigned)p.T), kThThreads, 0, s>>>(
      c->bw_thpart, c->bw_alpha16, c->bw_dx16, BH * p.nq * p.d, p.nq * p.d, (int)p.B, (int)p.H, p.T);
  dtheta_reduce_kernel<<<(unsigned)((p.T * p.H + 255) / 256), 256, 0, s>>>(dTh, c->bw_thpart, chunks, (int)(p.T * p.H));
  *launches += 2;
  return cudaGetLastError();
}

}  // namespace csat
