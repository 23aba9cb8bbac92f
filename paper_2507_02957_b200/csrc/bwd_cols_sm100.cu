// Backward of the compressed attention with respect to the compressed keys and values, on the sm_100a tensor cores:
//   dV~ = P^T dZ,   dK~ = scale dS^T Q,   P = exp(scale Q K~^T - L),   dS = P o (dZ V~^T - D)
// (chain rule through Z = A~ V~ and A~ = softmax(Q K~^T / sqrt(d_k)); L = log-sum-exp of a row's scores and
// D = <dZ, Z> come from the per-row kernel of the backward, like dZ itself).
//
// One CTA owns 128 measurements of one (batch, head): K~ and V~ of the block stay in shared memory, the two
// accumulators dK~ and dV~ [128 x d] in tensor memory, and the CTA walks the query tiles (128 rows):
//   warp 0   : TMA producer: Q tile and dZ tile (bf16) of the next query tile.
//   warp 1   : allocates tensor memory; one elected thread issues the MMAs:
//                S  = Q  K~^T   (A = Q tile, K-major; B = K~ block, K-major)      -> TMEM, 128 columns
//                dA = dZ V~^T   (A = dZ tile, K-major; B = V~ block, K-major)     -> TMEM, 128 columns
//              and, once the threads have written P and dS:
//                dV~ += P^T  dZ (A = P  in shared memory, MN-major: rows = queries; B = the dZ tile, MN-major)
//                dK~ += dS^T Q  (A = dS in shared memory, MN-major;                 B = the Q tile,  MN-major)
//              The Q and dZ tiles are read twice without being moved: a tile of 128 rows x d with 128-byte rows is
//              a K-major operand when its rows are the M index and an MN-major operand when they are the K index.
//   warps 2-5: one thread per query row: reads its row of S and dA, forms P and dS (zero for rows beyond n_q and
//              measurements beyond m), writes them as bf16 into the two operand tiles; at the end the same threads
//              (TMEM lane = measurement) store the accumulators as float32 and as the bf16 operand of Phi^T.
#include "csat_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace csat {
namespace {

using namespace ptx;

constexpr int kRows = 128;       // query rows per tile = measurements per block
constexpr int kThreads = 192;
constexpr uint32_t kPBytes = 2 * kRows * 128;          // P or dS: 128 queries x 128 measurements bf16, two 64-wide boxes

template <int D> struct Cfg {
  static constexpr int kDBoxes = D / 64;
  static constexpr uint32_t kBoxBytes = kRows * 128;                  // 128 rows x 64 columns
  static constexpr uint32_t kTileBytes = kDBoxes * kBoxBytes;         // 128 rows x d
  static constexpr uint32_t kOffK = 0, kOffV = kTileBytes, kOffQ = 2 * kTileBytes, kOffZ = 3 * kTileBytes;
  static constexpr uint32_t kOffP = 4 * kTileBytes, kOffS = kOffP + kPBytes, kOffBar = kOffS + kPBytes;
  static constexpr uint32_t kSmemBytes = kOffBar + 256 + 1024 /*alignment slack*/;
  static constexpr uint32_t kColS = 0, kColA = 128, kColV = 256, kColK = 256 + D, kTmemCols = 512;
  static_assert(256 + 2 * D <= 512, "TMEM budget");
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
};

struct Bars {
  uint64_t kv_full, in_full, in_free, sd_full, pm_full, acc_done;
  uint32_t tmem_slot;
  int abort;
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
bwd_cols_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_z,
                      const __grid_constant__ CUtensorMap tmap_kv, float* __restrict__ ws_dKV,
                      __nv_bfloat16* __restrict__ ws_dKV16, const float* __restrict__ ws_LD, int nq, int m, float scale,
                      int* status) {
  using C = Cfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  Bars* bars = reinterpret_cast<Bars*>(smem + C::kOffBar);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int mb = blockIdx.x, bh = blockIdx.y;
  const int ntiles = (nq + kRows - 1) / kRows;

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_q);
    prefetch_tmap(&tmap_z);
    prefetch_tmap(&tmap_kv);
    mbar_init(&bars->kv_full, 1);
    mbar_init(&bars->in_full, 1);
    mbar_init(&bars->in_free, 1);
    mbar_init(&bars->sd_full, 1);
    mbar_init(&bars->pm_full, 4 * 32);
    mbar_init(&bars->acc_done, 1);
    bars->abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_slot, C::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_slot;

  if (warp == 0) {
    if (elect_one()) {
      // K~ and V~ of the block: the workspace rows are K~_r | V~_r; boxes of 64 columns x 64 rows
      mbar_arrive_expect_tx(&bars->kv_full, 2 * C::kTileBytes);
      for (int gx = 0; gx < C::kDBoxes; ++gx)
        for (int half = 0; half < 2; ++half) {
          tma_load_3d(smem + C::kOffK + gx * C::kBoxBytes + half * 64 * 128, &tmap_kv, &bars->kv_full, gx * 64,
                      mb * kRows + half * 64, bh);
          tma_load_3d(smem + C::kOffV + gx * C::kBoxBytes + half * 64 * 128, &tmap_kv, &bars->kv_full, D + gx * 64,
                      mb * kRows + half * 64, bh);
        }
      bool ok = true;
      int issued = 0;
      for (int i = 0; i < ntiles && ok; ++i) {
        ok = mbar_wait(&bars->in_free, (i & 1) ^ 1, status, 501, &bars->abort);   // the MMAs of tile i-1 have read Q, dZ
        if (!ok) break;
        mbar_arrive_expect_tx(&bars->in_full, 2 * C::kTileBytes);
        for (int gx = 0; gx < C::kDBoxes; ++gx) {
          tma_load_3d(smem + C::kOffQ + gx * C::kBoxBytes, &tmap_q, &bars->in_full, gx * 64, i * kRows, bh);
          tma_load_3d(smem + C::kOffZ + gx * C::kBoxBytes, &tmap_z, &bars->in_full, gx * 64, i * kRows, bh);
        }
        ++issued;
      }
      if (!ok) {
        mbar_wait_drain(&bars->kv_full, 0);
        if (issued > 0) mbar_wait_drain(&bars->in_full, (issued - 1) & 1);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      constexpr uint32_t idesc_s = make_idesc_bf16(kRows, kRows, false, false);   // S, dA: both operands K-major
      constexpr uint32_t idesc_g = make_idesc_bf16(kRows, D, true, true);         // dV~, dK~: both operands MN-major
      // K-major tile of 128 rows: K step k (16 columns) lies in 64-column box k / 4, 32 (k % 4) bytes into each row
      auto kstep = [](int k) { return (uint64_t)((k / 4) * (C::kBoxBytes >> 4) + (k % 4) * 2); };
      const uint64_t kd = make_smem_desc(smem_u32(smem + C::kOffK), 16, 1024);
      const uint64_t vd = make_smem_desc(smem_u32(smem + C::kOffV), 16, 1024);
      const uint64_t qd = make_smem_desc(smem_u32(smem + C::kOffQ), 16, 1024);
      const uint64_t zd = make_smem_desc(smem_u32(smem + C::kOffZ), 16, 1024);
      // MN-major: the next 64 elements along M / N start one box (128 rows x 128 bytes) further; 16 k rows = 2048 B
      const uint64_t pm = make_smem_desc(smem_u32(smem + C::kOffP), kRows * 128, 1024);
      const uint64_t sm = make_smem_desc(smem_u32(smem + C::kOffS), kRows * 128, 1024);
      const uint64_t qn = make_smem_desc(smem_u32(smem + C::kOffQ), C::kBoxBytes, 1024);
      const uint64_t zn = make_smem_desc(smem_u32(smem + C::kOffZ), C::kBoxBytes, 1024);
      bool ok = mbar_wait(&bars->kv_full, 0, status, 502, &bars->abort);
      for (int i = 0; i < ntiles && ok; ++i) {
        ok = mbar_wait(&bars->in_full, i & 1, status, 503, &bars->abort);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < D / 16; ++k) mma_f16_ss(tmem + C::kColS, qd + kstep(k), kd + kstep(k), idesc_s, k != 0);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) mma_f16_ss(tmem + C::kColA, zd + kstep(k), vd + kstep(k), idesc_s, k != 0);
        mma_commit(&bars->sd_full);
        ok = mbar_wait(&bars->pm_full, i & 1, status, 504, &bars->abort);       // P and dS are in shared memory
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < kRows / 16; ++k) {
          mma_f16_ss(tmem + C::kColV, pm + (uint64_t)(k * 128), zn + (uint64_t)(k * 128), idesc_g, (i | k) != 0);
          mma_f16_ss(tmem + C::kColK, sm + (uint64_t)(k * 128), qn + (uint64_t)(k * 128), idesc_g, (i | k) != 0);
        }
        mma_commit(&bars->in_free);               // Q, dZ, P and dS may be overwritten
      }
      mma_commit(&bars->acc_done);
    }
  } else {
    const int q = warp & 3;                       // TMEM lanes [32q, 32q+32)
    const int row = q * 32 + lane;                // query row of the tile, later measurement of the block
    const uint32_t tbase = tmem + ((uint32_t)(q * 32) << 16);
    const float scale_log2 = scale * 1.4426950408889634f;
    uint8_t* prow = smem + C::kOffP + row * 128;
    uint8_t* srow = smem + C::kOffS + row * 128;
    bool ok = true;
    for (int i = 0; i < ntiles && ok; ++i) {
      const int gq = i * kRows + row;
      const bool live = gq < nq;
      const float L = live ? ws_LD[((int64_t)bh * nq + gq) * 2] * 1.4426950408889634f : 0.f;   // log2 domain
      const float Dr = live ? ws_LD[((int64_t)bh * nq + gq) * 2 + 1] : 0.f;
      ok = mbar_wait(&bars->sd_full, i & 1, status, 505, &bars->abort);
      if (!ok) break;
      tc_fence_after();
      // P and dS of tile i-1 have been read: sd_full of tile i follows the commit of tile i-1's last MMAs
#pragma unroll 1
      for (int c0 = 0; c0 < kRows; c0 += 16) {
        uint32_t s[16], a[16];
        tmem_ld_32x32b_x16(tbase + C::kColS + c0, s);
        tmem_ld_32x32b_x16(tbase + C::kColA + c0, a);
        tmem_wait_ld();
        uint32_t pw[8], dw[8];
#pragma unroll
        for (int e = 0; e < 16; e += 2) {
          float p0 = 0.f, p1 = 0.f;
          if (live && mb * kRows + c0 + e < m) p0 = exp2f(fmaf(__uint_as_float(s[e]), scale_log2, -L));
          if (live && mb * kRows + c0 + e + 1 < m) p1 = exp2f(fmaf(__uint_as_float(s[e + 1]), scale_log2, -L));
          const float d0 = p0 * (__uint_as_float(a[e]) - Dr) * scale, d1 = p1 * (__uint_as_float(a[e + 1]) - Dr) * scale;
          __nv_bfloat162 pp = __floats2bfloat162_rn(p0, p1), dd = __floats2bfloat162_rn(d0, d1);
          pw[e >> 1] = *reinterpret_cast<uint32_t*>(&pp);
          dw[e >> 1] = *reinterpret_cast<uint32_t*>(&dd);
        }
        // measurements c0 .. c0 + 15 of this query row: box c0 / 64, two 16-byte pieces swizzled by the row
        const uint32_t box = (uint32_t)(c0 / 64) * (kRows * 128), piece = (uint32_t)((c0 % 64) / 8);
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
          const uint32_t off = box + (((piece + h2) ^ (uint32_t)(row & 7)) << 4);
          *reinterpret_cast<uint4*>(prow + off) = make_uint4(pw[4 * h2], pw[4 * h2 + 1], pw[4 * h2 + 2], pw[4 * h2 + 3]);
          *reinterpret_cast<uint4*>(srow + off) = make_uint4(dw[4 * h2], dw[4 * h2 + 1], dw[4 * h2 + 2], dw[4 * h2 + 3]);
        }
      }
      fence_proxy_async();                        // the tensor cores read what these threads wrote
      tc_fence_before();
      mbar_arrive(&bars->pm_full);
    }
    if (ok && mbar_wait(&bars->acc_done, 0, status, 506, &bars->abort) && *(volatile int*)&bars->abort == 0) {
      tc_fence_after();
      const int r = mb * kRows + row;             // measurement
#pragma unroll 1
      for (int c0 = 0; c0 < 2 * D; c0 += 16) {
        uint32_t v[16];
        // accumulator columns: dV~ at kColV, dK~ at kColK; workspace row: dK~ | dV~
        tmem_ld_32x32b_x16(tbase + (c0 < D ? C::kColK + c0 : C::kColV + (c0 - D)), v);
        tmem_wait_ld();
        if (r < m) {
          float* o = ws_dKV + ((int64_t)bh * m + r) * 2 * D + c0;
          __nv_bfloat16* o16 = ws_dKV16 + ((int64_t)bh * m + r) * 2 * D + c0;
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            o[e] = __uint_as_float(v[e]);
            o16[e] = __float2bfloat16_rn(__uint_as_float(v[e]));
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, C::kTmemCols);
}

template <int D>
cudaError_t launch(csat_ctx* c, const void* Q, cudaStream_t s) {
  using C = Cfg<D>;
  const Params& p = c->p;
  CUtensorMap tq, tz;
  const uint64_t qd[3] = {(uint64_t)D, (uint64_t)p.nq, (uint64_t)(p.B * p.H)};
  const uint64_t qs[2] = {(uint64_t)D * 2, (uint64_t)p.nq * D * 2};
  const uint32_t qb[3] = {64, (uint32_t)kRows, 1};
  cudaError_t e;
  if ((e = make_tmap_bf16_3d(&tq, Q, qd, qs, qb)) != cudaSuccess) return e;
  if ((e = make_tmap_bf16_3d(&tz, c->bw_dZ16, qd, qs, qb)) != cudaSuccess) return e;
  static DeviceFlags smem_opt_in;
  if ((e = ensure_dynamic_smem(bwd_cols_sm100_kernel<D>, (int)C::kSmemBytes, c->device, smem_opt_in)) != cudaSuccess) return e;
  const float scale = (float)(p.scale > 0.0 ? p.scale : 1.0 / sqrt((double)D));
  const dim3 grid((unsigned)((p.m + kRows - 1) / kRows), (unsigned)(p.B * p.H));
  bwd_cols_sm100_kernel<D><<<grid, kThreads, C::kSmemBytes, s>>>(tq, tz, c->tmap_kv, c->bw_dKV, c->bw_dKV16, c->bw_LD,
                                                                (int)p.nq, (int)p.m, scale, c->status);
  return cudaGetLastError();
}

}  // namespace

// needs dZ as bf16 (bw_dZ16), L and D (bw_LD) from the per-row kernel, and K~|V~ in the workspace
cudaError_t launch_sm100_bwd_cols(csat_ctx* c, const void* Q, cudaStream_t s, int* launches) {
  *launches += 1;
  return c->p.d == 64 ? launch<64>(c, Q, s) : launch<128>(c, Q, s);
}

}  // namespace csat
