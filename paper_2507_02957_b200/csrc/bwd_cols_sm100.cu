// Backward of the compressed attention with respect to the compressed keys and values, on the sm_100a tensor cores:
//   dV~ = P^T dZ,   dK~ = scale dS^T Q,   P = exp(scale Q K~^T - L),   dS = P o (dZ V~^T - D)
// (chain rule through Z = A~ V~ and A~ = softmax(Q K~^T / sqrt(d_k)); L = log-sum-exp of a row's scores and
// D = <dZ, Z> come from the per-row stage of the backward, like dZ itself).
//
// One CTA owns 128 measurements of one (batch, head): K~ and V~ of the block stay in shared memory, the two
// accumulators dK~ and dV~ [128 x d] in tensor memory, and the CTA walks the queries in tiles of 64.  The scores are
// formed TRANSPOSED, S^T = K~ Q^T (rows = measurements), so that the thread that owns a measurement's row of S^T
// writes its row of P^T straight back into tensor memory, where it is the A operand (M = measurements, K = queries)
// of the second pair of products: neither P nor dS passes through shared memory.
//   warp 0   : TMA producer: Q and dZ tiles (bf16, 64 queries x d) and the queries' L, D (one untiled bulk copy) into
//              a ring of kStages stages.
//   warp 1   : allocates tensor memory; one elected thread issues the MMAs:
//                S^T  = K~ Q^T    (A = K~ block, K-major; B = Q tile, K-major)       -> set[i & 1], 64 columns
//                dA^T = V~ dZ^T   (A = V~ block, K-major; B = dZ tile, K-major)      -> set[i & 1], 64 columns
//              and, once the threads have written P^T and dS^T over them (bf16, two per column):
//                dV~ += P^T  dZ   (A = P^T  in tensor memory; B = the dZ tile, MN-major: rows = queries = K index)
//                dK~ += dS^T Q    (A = dS^T in tensor memory; B = the Q tile,  MN-major)
//              The Q and dZ tiles are read twice without being moved: a tile of 64 rows x d with 128-byte rows is a
//              K-major operand when its rows are the N index and an MN-major operand when they are the K index.
//              Two sets of S^T | dA^T: the products of tile i + 1 run while the threads work on tile i.  The MMAs of
//              one thread execute in issue order, so tile i + 2's scores overwrite set[i & 1] only after tile i's
//              second pair of products has read it.
//   warps 2-9: TMEM lane = measurement; warps 2-5 take the tile's queries [0, 32), warps 6-9 the queries [32, 64):
//              P = exp2(S^T scale log2 e - L log2 e), dS = scale P (dA^T - D) with the queries' L, D read from global
//              memory (the same address in every lane), zero for queries beyond n_q.  At the end the same threads
//              store the accumulators as float32 and as the bf16 operand of the product with Phi^T.
#include "csat_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace csat {
namespace {

using namespace ptx;

constexpr int kRows = 128;       // measurements per block
constexpr int kQT = 64;          // queries per tile
constexpr int kStages = 4;       // Q | dZ tiles in flight
constexpr int kSimtWarps = 8;
constexpr int kThreads = (2 + kSimtWarps) * 32;

template <int D> struct Cfg {
  static constexpr int kDBoxes = D / 64;
  static constexpr uint32_t kKvBoxBytes = kRows * 128;                // 128 rows x 64 columns
  static constexpr uint32_t kKvBytes = kDBoxes * kKvBoxBytes;         // K~ block (= V~ block)
  static constexpr uint32_t kInBoxBytes = kQT * 128;                  // 64 rows x 64 columns
  static constexpr uint32_t kInBytes = kDBoxes * kInBoxBytes;         // Q tile (= dZ tile)
  static constexpr uint32_t kOffK = 0, kOffV = kKvBytes, kOffIn = 2 * kKvBytes;   // stage s: Q at kOffIn + 2 s kInBytes, dZ after it
  // L, D of a tile's queries: 64 pairs of floats copied from the 16-byte boundary at or below the first, so 66 pairs
  static constexpr uint32_t kLdBytes = (kQT + 2) * 8, kLdStride = 544;
  static constexpr uint32_t kOffLd = kOffIn + kStages * 2 * kInBytes;
  static constexpr uint32_t kOffBar = kOffLd + kStages * kLdStride;
  static constexpr uint32_t kSmemBytes = kOffBar + 256 + 1024 /*alignment slack*/;
  // TMEM columns: set s at 128 s: S^T (64) | dA^T (64); then the accumulators
  static constexpr uint32_t kSetCols = 2 * kQT, kColA = kQT, kColV = 2 * kSetCols, kColK = kColV + D, kTmemCols = 512;
  static_assert(2 * kSetCols + 2 * D <= 512, "TMEM budget");
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
};

struct Bars {
  uint64_t kv_full, in_full[kStages], in_free[kStages], sd_full[2], pd_full[2], acc_done;
  uint32_t tmem_slot;
  int abort;
};
static_assert(sizeof(Bars) <= 256, "barrier block");

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// packed column (two bf16 per 32-bit column) of K step k (16 queries) inside S^T or dA^T: the warps of the first
// half write over the first 16 columns of their own 32 scores, the second half over columns [32, 48)
__device__ __forceinline__ constexpr uint32_t pcol(int k) { return (uint32_t)((k >> 1) * 32 + (k & 1) * 8); }

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
  const int ntiles = (nq + kQT - 1) / kQT;

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_q);
    prefetch_tmap(&tmap_z);
    prefetch_tmap(&tmap_kv);
    mbar_init(&bars->kv_full, 1);
    for (int s = 0; s < kStages; ++s) { mbar_init(&bars->in_full[s], 1); mbar_init(&bars->in_free[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&bars->sd_full[s], 1); mbar_init(&bars->pd_full[s], kSimtWarps * 32); }
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
      mbar_arrive_expect_tx(&bars->kv_full, 2 * C::kKvBytes);
      for (int gx = 0; gx < C::kDBoxes; ++gx)
        for (int half = 0; half < 2; ++half) {
          tma_load_3d(smem + C::kOffK + gx * C::kKvBoxBytes + half * 64 * 128, &tmap_kv, &bars->kv_full, gx * 64,
                      mb * kRows + half * 64, bh);
          tma_load_3d(smem + C::kOffV + gx * C::kKvBoxBytes + half * 64 * 128, &tmap_kv, &bars->kv_full, D + gx * 64,
                      mb * kRows + half * 64, bh);
        }
      bool ok = true;
      int issued = 0;
      const float2* LDg = reinterpret_cast<const float2*>(ws_LD) + (int64_t)bh * nq;
      for (int i = 0; i < ntiles && ok; ++i) {
        const int s = i % kStages;
        // the second pair of products of tile i - kStages has read the stage
        if (i >= kStages) ok = mbar_wait(&bars->in_free[s], ((i / kStages) & 1) ^ 1, status, 501, &bars->abort);
        if (!ok) break;
        uint8_t* qs = smem + C::kOffIn + (uint32_t)s * 2 * C::kInBytes;
        mbar_arrive_expect_tx(&bars->in_full[s], 2 * C::kInBytes + C::kLdBytes);
        // (the copy may run up to 65 pairs past the rows of this (batch, head), into the next one's or into the slack
        // the buffer is allocated with; those queries are masked)
        bulk_load_1d(smem + C::kOffLd + (uint32_t)s * C::kLdStride,
                     reinterpret_cast<const uint8_t*>((reinterpret_cast<uintptr_t>(LDg + i * kQT)) & ~uintptr_t(15)),
                     C::kLdBytes, &bars->in_full[s]);
        for (int gx = 0; gx < C::kDBoxes; ++gx) {
          tma_load_3d(qs + gx * C::kInBoxBytes, &tmap_q, &bars->in_full[s], gx * 64, i * kQT, bh);
          tma_load_3d(qs + C::kInBytes + gx * C::kInBoxBytes, &tmap_z, &bars->in_full[s], gx * 64, i * kQT, bh);
        }
        ++issued;
      }
      if (!ok) {                                  // gave up: let the copies in flight land before the CTA exits
        mbar_wait_drain(&bars->kv_full, 0);
        for (int i = issued > kStages ? issued - kStages : 0; i < issued; ++i)
          mbar_wait_drain(&bars->in_full[i % kStages], (i / kStages) & 1);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      constexpr uint32_t idesc_s = make_idesc_bf16(kRows, kQT, false, false);    // S^T, dA^T: both operands K-major
      constexpr uint32_t idesc_g = make_idesc_bf16(kRows, D, false, true);       // dV~, dK~: A in TMEM, B MN-major
      // K-major tile: K step k (16 columns) lies in 64-column box k / 4, 32 (k % 4) bytes into each row
      auto kstep = [](int k, uint32_t box_bytes) { return (uint64_t)((k / 4) * (box_bytes >> 4) + (k % 4) * 2); };
      const uint64_t kd = make_smem_desc(smem_u32(smem + C::kOffK), 16, 1024);
      const uint64_t vd = make_smem_desc(smem_u32(smem + C::kOffV), 16, 1024);
      // stage 0's tiles; stage s lies 2 kInBytes s further.  K-major view (rows = N index) and MN-major view
      // (rows = K index: the next 64 elements along N start one box further; 16 k rows = 2048 B) of the same bytes
      const uint64_t qk0 = make_smem_desc(smem_u32(smem + C::kOffIn), 16, 1024);
      const uint64_t zk0 = make_smem_desc(smem_u32(smem + C::kOffIn + C::kInBytes), 16, 1024);
      const uint64_t qn0 = make_smem_desc(smem_u32(smem + C::kOffIn), C::kInBoxBytes, 1024);
      const uint64_t zn0 = make_smem_desc(smem_u32(smem + C::kOffIn + C::kInBytes), C::kInBoxBytes, 1024);
      constexpr uint64_t kStageStep = (2 * C::kInBytes) >> 4;
      bool ok = mbar_wait(&bars->kv_full, 0, status, 502, &bars->abort);
      auto issue_scores = [&](int i) {            // S^T and dA^T of tile i
        const int s = i % kStages;
        ok = mbar_wait(&bars->in_full[s], (i / kStages) & 1, status, 503, &bars->abort);
        if (!ok) return;
        tc_fence_after();
        const uint32_t ts = tmem + (uint32_t)(i & 1) * C::kSetCols;
        const uint64_t st = (uint64_t)s * kStageStep;
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          mma_f16_ss(ts, kd + kstep(k, C::kKvBoxBytes), qk0 + st + kstep(k, C::kInBoxBytes), idesc_s, k != 0);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          mma_f16_ss(ts + C::kColA, vd + kstep(k, C::kKvBoxBytes), zk0 + st + kstep(k, C::kInBoxBytes), idesc_s, k != 0);
        mma_commit(&bars->sd_full[i & 1]);
      };
      if (ok) issue_scores(0);
      if (ok && ntiles > 1) issue_scores(1);
      for (int i = 0; i < ntiles && ok; ++i) {
        ok = mbar_wait(&bars->pd_full[i & 1], (i >> 1) & 1, status, 504, &bars->abort);   // P^T and dS^T are written
        if (!ok) break;
        tc_fence_after();
        const uint32_t ts = tmem + (uint32_t)(i & 1) * C::kSetCols;
        const uint64_t st = (uint64_t)(i % kStages) * kStageStep;
#pragma unroll
        for (int k = 0; k < kQT / 16; ++k) {
          mma_f16_ts(tmem + C::kColV, ts + pcol(k), zn0 + st + (uint64_t)(k * 128), idesc_g, (i | k) != 0);
          mma_f16_ts(tmem + C::kColK, ts + C::kColA + pcol(k), qn0 + st + (uint64_t)(k * 128), idesc_g, (i | k) != 0);
        }
        mma_commit(&bars->in_free[i % kStages]);  // the stage may be overwritten
        if (i + 2 < ntiles) issue_scores(i + 2);
      }
      if (ok) mma_commit(&bars->acc_done);
    }
  } else {
    const int q = warp & 3;                       // TMEM lanes [32q, 32q+32): a warp reaches only its own quarter
    const int hf = (warp - 2) >> 2;               // which 32 of the tile's 64 queries
    const uint32_t tbase = tmem + ((uint32_t)(q * 32) << 16);
    const float scale_log2 = scale * 1.4426950408889634f;
    // first pair of the tile within its staged copy: 0 or 1 (the same for every tile: 64 pairs are 512 bytes)
    const int ld_off = (int)((reinterpret_cast<uintptr_t>(reinterpret_cast<const float2*>(ws_LD) + (int64_t)bh * nq) >> 3) & 1);
    bool ok = true;
    for (int i = 0; i < ntiles && ok; ++i) {
      const uint32_t ts = tbase + (uint32_t)(i & 1) * C::kSetCols;
      // the TMEM loads and stores below are warp-wide: the whole warp gives up together
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->sd_full[i & 1], (i >> 1) & 1, status, 505, &bars->abort));
      if (!ok) break;
      // The scores' commit follows the stage's arrival in the MMA thread's program order, but this thread reads the
      // staged L, D itself, so it observes the stage's barrier too (complete by now: no waiting).
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->in_full[i % kStages], (i / kStages) & 1, status, 507, &bars->abort));
      if (!ok) break;
      const float2* ldq = reinterpret_cast<const float2*>(smem + C::kOffLd + (uint32_t)(i % kStages) * C::kLdStride) + ld_off;
      tc_fence_after();
#pragma unroll
      for (int sp = 0; sp < 2; ++sp) {            // 16 queries at a time
        const int c0 = hf * 32 + sp * 16;         // first of them within the tile = column of S^T
        uint32_t s[16], a[16];
        tmem_ld_32x32b_x16(ts + c0, s);
        tmem_ld_32x32b_x16(ts + C::kColA + c0, a);
        float2 ld[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const int gq = i * kQT + c0 + e;
          ld[e] = gq < nq ? ldq[c0 + e] : make_float2(INFINITY, 0.f);         // beyond n_q: P = exp2(-inf) = 0
        }
        tmem_wait_ld();
        uint32_t pw[8], dw[8];
#pragma unroll
        for (int e = 0; e < 16; e += 2) {
          const float p0 = ex2f(fmaf(__uint_as_float(s[e]), scale_log2, -ld[e].x * 1.4426950408889634f));
          const float p1 = ex2f(fmaf(__uint_as_float(s[e + 1]), scale_log2, -ld[e + 1].x * 1.4426950408889634f));
          const float d0 = p0 * (__uint_as_float(a[e]) - ld[e].y) * scale;
          const float d1 = p1 * (__uint_as_float(a[e + 1]) - ld[e + 1].y) * scale;
          __nv_bfloat162 pp = __floats2bfloat162_rn(p0, p1), dd = __floats2bfloat162_rn(d0, d1);
          pw[e >> 1] = *reinterpret_cast<uint32_t*>(&pp);
          dw[e >> 1] = *reinterpret_cast<uint32_t*>(&dd);
        }
        // over the scores this thread has already read (see pcol)
        tmem_st_32x32b_x8(ts + hf * 32 + sp * 8, pw);
        tmem_st_32x32b_x8(ts + C::kColA + hf * 32 + sp * 8, dw);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bars->pd_full[i & 1]);
    }
    if (__all_sync(0xffffffffu, ok && mbar_wait(&bars->acc_done, 0, status, 506, &bars->abort) &&
                                    *(volatile int*)&bars->abort == 0)) {
      tc_fence_after();
      const int r = mb * kRows + q * 32 + lane;   // measurement
      // workspace row: dK~ | dV~; the first half of the warps stores dK~, the second dV~
      const uint32_t acc = tbase + (hf == 0 ? C::kColK : C::kColV);
      float* o = ws_dKV + ((int64_t)bh * m + r) * 2 * D + hf * D;
      __nv_bfloat16* o16 = ws_dKV16 + ((int64_t)bh * m + r) * 2 * D + hf * D;
#pragma unroll 1
      for (int c0 = 0; c0 < D; c0 += 16) {
        uint32_t v[16];
        tmem_ld_32x32b_x16(acc + c0, v);          // the whole warp takes part in the load
        tmem_wait_ld();
        if (r < m) {
#pragma unroll
          for (int e = 0; e < 16; e += 4)
            *reinterpret_cast<float4*>(o + c0 + e) = make_float4(__uint_as_float(v[e]), __uint_as_float(v[e + 1]),
                                                                 __uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
          uint32_t h[8];
#pragma unroll
          for (int e = 0; e < 16; e += 2) {
            __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(v[e]), __uint_as_float(v[e + 1]));
            h[e >> 1] = *reinterpret_cast<uint32_t*>(&b2);
          }
          *reinterpret_cast<uint4*>(o16 + c0) = make_uint4(h[0], h[1], h[2], h[3]);
          *reinterpret_cast<uint4*>(o16 + c0 + 8) = make_uint4(h[4], h[5], h[6], h[7]);
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
  const uint32_t qb[3] = {64, (uint32_t)kQT, 1};
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

// needs dZ as bf16 (bw_dZ16), L and D (bw_LD) from the per-row stage, and K~|V~ in the workspace
cudaError_t launch_sm100_bwd_cols(csat_ctx* c, const void* Q, cudaStream_t s, int* launches) {
  *launches += 1;
  return c->p.d == 64 ? launch<64>(c, Q, s) : launch<128>(c, Q, s);
}

}  // namespace csat
