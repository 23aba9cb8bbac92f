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
//   dtheta rides along: while a stage's tiles are in shared memory the four epilogue warps (one thread per row of
//   the tile) read their row of dx_t from it and the row's sign bits of x_t (recorded by the forward kernel, one bit
//   per column like the decisions), and add sign(x_t) o dx_t into per-layer sums; a stage is released by the MMA
//   commit and by these four warps.  The sums go to a partial buffer like the matrices.
// dtheta_partial_kernel (the same sum from the stored iterates' signs) serves depths beyond kMaxFusedLayers.
#include "csat_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace csat {
namespace {

using namespace ptx;

constexpr int kRows = 128;
constexpr int kThreads = 192;          // warps 0-3: epilogue (TMEM lane = row of C), warp 4: TMA, warp 5: MMA
constexpr int kMaxFusedLayers = 256;   // per-layer sums of sign(x_t) o dx_t kept in shared memory: [layers][4 warps]

template <int D> struct GCfg {
  static constexpr int kDBoxes = D / 64;
  static constexpr int kStages = (D == 64) ? 4 : 2;
  static constexpr uint32_t kBoxBytes = kRows * 128;                 // 128 rows x 64 columns
  static constexpr uint32_t kTileBytes = kDBoxes * kBoxBytes;
  static constexpr uint32_t kStageBytes = 3 * kTileBytes;            // A1 | A2 | B
  static constexpr uint32_t kOffBar = kStages * kStageBytes;
  static constexpr uint32_t kOffTheta = kOffBar + 256;               // float [kMaxFusedLayers][4]
  static constexpr uint32_t kSmemBytes = kOffTheta + kMaxFusedLayers * 16 + 1024;
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
                  float* __restrict__ part, int nq, int H, int B, int nt, int units_per_cta, int* status,
                  const uint32_t* __restrict__ signbits, float* __restrict__ thpart, int T) {
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
    // a stage is released by the MMA commit and, where dtheta rides along, by the four epilogue warps
    for (int s = 0; s < C::kStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], signbits ? 5 : 1); }
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
    if (signbits != nullptr) {
      // ---- dtheta: sum over this thread's row of sign(x_t) o dx_t, per layer ----
      float* th_s = reinterpret_cast<float*>(smem + C::kOffTheta);           // [nt][4]
      for (int i = threadIdx.x; i < nt * 4; i += 128) th_s[i] = 0.f;
      asm volatile("bar.sync 1, 128;" ::: "memory");
      for (int i = 0; i < steps; ++i) {
        const int s = i % C::kStages;
        const int u = u0 + i / nt, tl = i % nt, t = (int)blockIdx.z + tl, b = u / ntiles, tile = u % ntiles;
        const int grow = tile * kRows + row;
        // the row's sign words (column c: word c / 32, bit 31 - c % 32), requested before the stage is waited for
        uint32_t sg[D / 32];
        const uint32_t* sp = signbits + ((((int64_t)(b * H + h)) * T + t) * nq + (grow < nq ? grow : 0)) * (D / 32);
#pragma unroll
        for (int q = 0; q < D / 32; ++q) sg[q] = grow < nq ? sp[q] : 0u;
        if (ok) ok = mbar_wait(&bars->full[s], (i / C::kStages) & 1, status, 704, &bars->abort);
        float acc = 0.f;
        if (ok) {
          const uint8_t* xt = smem + (uint32_t)s * C::kStageBytes + 2 * C::kTileBytes;   // the dx_t tile
#pragma unroll
          for (int gx = 0; gx < C::kDBoxes; ++gx) {
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {            // 16-byte pieces of the row's 128 bytes, swizzled by the row
              const uint4 v = *reinterpret_cast<const uint4*>(xt + gx * C::kBoxBytes + row * 128 + ((ch ^ (row & 7)) << 4));
              const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
              const int c0 = gx * 64 + ch * 8;          // first column of the piece
              const uint32_t bits = sg[c0 >> 5] << (c0 & 31);            // the piece's 8 sign bits at the top
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const uint32_t lo = (w4[q] << 16) ^ ((bits << (2 * q)) & 0x80000000u);
                const uint32_t hi = (w4[q] & 0xffff0000u) ^ ((bits << (2 * q + 1)) & 0x80000000u);
                acc += __uint_as_float(lo) + __uint_as_float(hi);
              }
            }
          }
        }
        // fixed-order sum over the warp's rows, then into the layer's slot of this warp
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) {
          th_s[tl * 4 + warp] += acc;
          mbar_arrive(&bars->empty[s]);               // this warp has read the stage
        }
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      for (int tl = threadIdx.x; tl < nt; tl += 128)
        thpart[((int64_t)split * H + h) * T + (int)blockIdx.z + tl] =
            th_s[tl * 4] + th_s[tl * 4 + 1] + th_s[tl * 4 + 2] + th_s[tl * 4 + 3];
    }
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

// out[t][h] = sum over the chunks, in order.  from_contraction: partial [chunk][H][T] holds + sum sign(x) o dx (the
// gradient is its negative); else partial [chunk][T][H] already holds the negative
__global__ void dtheta_reduce_kernel(float* __restrict__ out, const float* __restrict__ partial, int chunks, int T, int H,
                                     int from_contraction) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= T * H) return;
  const int t = i / H, h = i % H;
  float acc = 0.f;
  if (from_contraction) {
    for (int c = 0; c < chunks; ++c) acc += partial[((int64_t)c * H + h) * T + t];
    acc = -acc;
  } else {
    for (int c = 0; c < chunks; ++c) acc += partial[(int64_t)c * T * H + i];
  }
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
                        SlabIndex ia2, SlabIndex ib, int nt, int splits, int units_per_cta, cudaStream_t s, int layers_z = 1,
                        const uint32_t* signbits = nullptr) {
  using C = GCfg<D>;
  static DeviceFlags smem_opt_in;
  cudaError_t e = ensure_dynamic_smem(wgrad_gram_kernel<D>, (int)C::kSmemBytes, c->device, smem_opt_in);
  if (e != cudaSuccess) return e;
  const Params& p = c->p;
  wgrad_gram_kernel<D><<<dim3((unsigned)splits, (unsigned)p.H, (unsigned)layers_z), kThreads, C::kSmemBytes, s>>>(
      a1, a2, b, ia1, ia2, ib, c->bw_wpart, (int)p.nq, (int)p.H, (int)p.B, nt, units_per_cta, c->status, signbits,
      c->bw_thpart, p.T);
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
  // dtheta rides along where the per-layer sums fit the kernel's shared memory
  const bool fused_theta = c->bw_signbits != nullptr && nt <= kMaxFusedLayers;
  const uint32_t* sgn = fused_theta ? c->bw_signbits : nullptr;
  e = p.d == 64 ? launch_gram<64>(c, ta, tz, tx, ia, iz, ix, nt, splits, upc, s, Z, sgn)
                : launch_gram<128>(c, ta, tz, tx, ia, iz, ix, nt, splits, upc, s, Z, sgn);
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
  // dtheta [T,H]: the contraction kernel's partial sums [split][H][T], or the streaming kernel's [chunk][T][H]
  if (fused_theta) {
    dtheta_reduce_kernel<<<(unsigned)((p.T * p.H + 255) / 256), 256, 0, s>>>(dTh, c->bw_thpart, splits, (int)p.T, (int)p.H, 1);
    *launches += 1;
  } else {
    const int chunks = 64;
    dtheta_partial_kernel<<<dim3(chunks, (unsigned)p.H, (unsigned)p.T), kThThreads, 0, s>>>(
        c->bw_thpart, c->bw_alpha16, c->bw_dx16, BH * p.nq * p.d, p.nq * p.d, (int)p.B, (int)p.H, p.T);
    dtheta_reduce_kernel<<<(unsigned)((p.T * p.H + 255) / 256), 256, 0, s>>>(dTh, c->bw_thpart, chunks, (int)p.T, (int)p.H, 0);
    *launches += 2;
  }
  return cudaGetLastError();
}

}  // namespace csat
