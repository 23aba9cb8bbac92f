// Gradient with respect to the measurement matrices (paper: Phi is "fixed or learned"; a learned Phi needs
// d Phi_K = sum_b dK~ K^T and d Phi_V = sum_b dV~ V^T, the chain rule through the compression equation
// K~ = Phi K, V~ = Phi V; the paper prints no backward pass).  The decoder's matrices are held fixed.
//
// Per head one GEMM  dPhi[m, n] = [dK~ | dV~][m, 2 d B] * [K | V]^T[2 d B, n]  whose reduction runs over the
// feature columns of keys and values and over the batch: only 2 d B long, so the kernel lives on its output
// (H m n float32).  Persistent CTAs, one per SM, walk 128 x 256 output tiles (measurement tiles fastest: the CTAs
// running together share the K, V rows of a token tile):
//   warp 0   : TMA producer: per (batch element, K or V, 64-column box) a {64 x 128} box of dK~|dV~ (bf16, as the
//              backward's dK~|dV~ stage leaves it: K-major A operand) and a {64 x 256} box of K or V (rows = tokens,
//              the caller's layout: K-major B operand, no transpose), 128-byte swizzle, 4-stage ring.
//   warp 1   : allocates tensor memory (two 256-column accumulators); one elected thread issues tcgen05.mma
//              (M = 128, N = 256, K = 16).
//   warps 2-5: epilogue of tile i (float32 stores) while the MMAs of tile i + 1 fill the other accumulator.
// With separate Phi_K / Phi_V the output has 2 H matrices and each reduces over its own half (keys or values).
#include "csat_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace csat {
namespace {

using namespace ptx;

constexpr int kTileM = 128, kTileN = 256, kChunkK = 64, kStages = 4, kThreads = 192;
constexpr uint32_t kABytes = kTileM * kChunkK * 2;       // 16 KB
constexpr uint32_t kBBytes = kTileN * kChunkK * 2;       // 32 KB: 256 tokens x 64 columns
constexpr uint32_t kStageBytes = kABytes + kBBytes;
constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;

// 32-byte store (the address is 32-byte aligned): whole sectors per lane
__device__ __forceinline__ void st_global_v8(void* p, const uint32_t* r) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]),
               "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}

struct PhiGradArgs {
  float* out;                 // [PH, m, n]
  int m, n, H, B, d;
  int PH;                     // H (one Phi per head) or 2 H (Phi_K heads, then Phi_V heads)
  int mtiles, ntiles;
};

__global__ void __launch_bounds__(kThreads, 1)
phigrad_sm100_kernel(const __grid_constant__ CUtensorMap tmap_g, const __grid_constant__ CUtensorMap tmap_k,
                     const __grid_constant__ CUtensorMap tmap_v, const PhiGradArgs a, int* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* a_buf = smem;                                  // [stages][16 KB]
  uint8_t* b_buf = smem + kStages * kABytes;              // [stages][32 KB]
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  uint64_t* empty = full + kStages;
  uint64_t* acc_full = empty + kStages;                   // [2]
  uint64_t* acc_empty = acc_full + 2;                     // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  int* cta_abort = reinterpret_cast<int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int boxes = a.d / 64;
  const bool sep = a.PH != a.H;
  // reduction steps of a tile: (batch element, half: keys / values, 64-column box); separate matrices take one half
  const int halves = sep ? 1 : 2;
  const int nk = a.B * halves * boxes;
  const int n_tiles = a.PH * a.ntiles * a.mtiles;

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_g);
    prefetch_tmap(&tmap_k);
    prefetch_tmap(&tmap_v);
    for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int u = 0; u < 2; ++u) { mbar_init(&acc_full[u], 1); mbar_init(&acc_empty[u], 4 * 32); }
    *cta_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 2 * kTileN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (elect_one()) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const int mt = tile % a.mtiles, nt = (tile / a.mtiles) % a.ntiles, hp = tile / (a.mtiles * a.ntiles);
        const int h = hp % a.H, half0 = sep ? hp / a.H : 0;
        for (int k = 0; k < nk && ok; ++k, ++it) {
          const int s = it % kStages;
          ok = mbar_wait(&empty[s], ((it / kStages) & 1) ^ 1, status, 801, cta_abort);
          if (!ok) break;
          const int gx = k % boxes, half = half0 + (k / boxes) % halves, b = k / (boxes * halves);
          const int bh = b * a.H + h;
          mbar_arrive_expect_tx(&full[s], kStageBytes);
          // dK~|dV~ rows are [dK~ (d) | dV~ (d)]
          tma_load_3d(a_buf + s * kABytes, &tmap_g, &full[s], half * a.d + gx * 64, mt * kTileM, bh);
          tma_load_3d(b_buf + s * kBBytes, half ? &tmap_v : &tmap_k, &full[s], gx * 64, nt * kTileN, bh);
        }
      }
      if (!ok)
        for (uint32_t i = it > (uint32_t)kStages ? it - kStages : 0; i < it; ++i)
          mbar_wait_drain(&full[i % kStages], (i / kStages) & 1);
    }
  } else if (warp == 1) {
    if (elect_one()) {
      constexpr uint32_t idesc = make_idesc_bf16(kTileM, kTileN, /*A MN-major*/ false, /*B MN-major*/ false);
      uint32_t it = 0, tc = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tc) {
        const uint32_t buf = tc & 1;
        ok = mbar_wait(&acc_empty[buf], ((tc >> 1) & 1) ^ 1, status, 802, cta_abort);
        if (!ok) break;
        tc_fence_after();
        const uint32_t acc = tmem_base + buf * kTileN;
        for (int k = 0; k < nk; ++k, ++it) {
          const int s = it % kStages;
          ok = mbar_wait(&full[s], (it / kStages) & 1, status, 803, cta_abort);
          if (!ok) break;
          tc_fence_after();
          const uint64_t a_desc = make_smem_desc(smem_u32(a_buf + s * kABytes), 16, 1024);
          const uint64_t b_desc = make_smem_desc(smem_u32(b_buf + s * kBBytes), 16, 1024);
#pragma unroll
          for (int kk = 0; kk < kChunkK / 16; ++kk)       // +32 B along K for both K-major operands
            mma_f16_ss(acc, a_desc + (uint64_t)(kk * 2), b_desc + (uint64_t)(kk * 2), idesc, (k | kk) != 0);
          mma_commit(&empty[s]);
        }
        mma_commit(&acc_full[buf]);
      }
    }
  } else {
    const int q = warp & 3;
    uint32_t tc = 0;
    bool ok = true;
    const bool vec = (a.n & 3) == 0;                      // rows of the output are 16-byte aligned
    const bool vec8 = (a.n & 7) == 0 && (reinterpret_cast<uintptr_t>(a.out) & 31u) == 0;   // ... 32-byte aligned
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tc) {
      const int mt = tile % a.mtiles, nt = (tile / a.mtiles) % a.ntiles, hp = tile / (a.mtiles * a.ntiles);
      const uint32_t buf = tc & 1;
      if (ok) ok = mbar_wait(&acc_full[buf], (tc >> 1) & 1, status, 804, cta_abort) && *(volatile int*)cta_abort == 0;
      ok = __all_sync(0xffffffffu, ok);                   // the TMEM loads are warp-wide
      if (!ok) break;
      tc_fence_after();
      const int row = mt * kTileM + q * 32 + lane;
      float* orow = a.out + ((int64_t)hp * a.m + row) * a.n;
#pragma unroll 1
      for (int c0 = 0; c0 < kTileN; c0 += 32) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16) + buf * kTileN + (uint32_t)c0, r);
        tmem_wait_ld();
        const int col = nt * kTileN + c0;
        if (row < a.m && col < a.n) {
          if (vec8 && col + 32 <= a.n) {
#pragma unroll
            for (int v = 0; v < 4; ++v) st_global_v8(orow + col + 8 * v, r + 8 * v);
          } else if (vec && col + 32 <= a.n) {
            float4* o = reinterpret_cast<float4*>(orow + col);
#pragma unroll
            for (int v = 0; v < 8; ++v)
              o[v] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]), __uint_as_float(r[4 * v + 2]),
                                 __uint_as_float(r[4 * v + 3]));
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e)
              if (col + e < a.n) orow[col + e] = __uint_as_float(r[e]);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(&acc_empty[buf]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, 2 * kTileN);
}

}  // namespace

// dPhi [PH, m, n] float32 from the bf16 dK~|dV~ of the most recent backward (bw_dKV16) and the caller's K, V
cudaError_t launch_sm100_phigrad(csat_ctx* c, const void* K, const void* V, float* dPhi, cudaStream_t s, int* launches) {
  const Params& p = c->p;
  *launches += 1;
  CUtensorMap tg, tk, tv;
  const uint64_t gd[3] = {(uint64_t)(2 * p.d), (uint64_t)p.m, (uint64_t)(p.B * p.H)};
  const uint64_t gs[2] = {(uint64_t)(2 * p.d) * 2, (uint64_t)p.m * 2 * p.d * 2};
  const uint32_t gb[3] = {(uint32_t)kChunkK, (uint32_t)kTileM, 1};
  const uint64_t kd[3] = {(uint64_t)p.d, (uint64_t)p.n, (uint64_t)(p.B * p.H)};
  const uint64_t ks[2] = {(uint64_t)p.d * 2, (uint64_t)p.n * p.d * 2};
  const uint32_t kb[3] = {(uint32_t)kChunkK, (uint32_t)kTileN, 1};
  cudaError_t e;
  if ((e = make_tmap_bf16_3d(&tg, c->bw_dKV16, gd, gs, gb)) != cudaSuccess) return e;
  if ((e = make_tmap_bf16_3d(&tk, K, kd, ks, kb)) != cudaSuccess) return e;
  if ((e = make_tmap_bf16_3d(&tv, V, kd, ks, kb)) != cudaSuccess) return e;
  PhiGradArgs a;
  a.out = dPhi;
  a.m = (int)p.m; a.n = (int)p.n; a.H = (int)p.H; a.B = (int)p.B; a.d = (int)p.d;
  a.PH = (int)(p.separate_phi ? 2 * p.H : p.H);
  a.mtiles = (int)((p.m + kTileM - 1) / kTileM);
  a.ntiles = (int)((p.n + kTileN - 1) / kTileN);
  const int64_t n_tiles = (int64_t)a.PH * a.mtiles * a.ntiles;
  if (n_tiles > (int64_t)1 << 30) return cudaErrorInvalidValue;
  const unsigned grid = (unsigned)(n_tiles < c->sms ? n_tiles : c->sms);
  static DeviceFlags opt_in;
  if ((e = ensure_dynamic_smem(phigrad_sm100_kernel, (int)kSmemBytes, c->device, opt_in)) != cudaSuccess) return e;
  phigrad_sm100_kernel<<<grid, kThreads, kSmemBytes, s>>>(tg, tk, tv, a, c->status);
  return cudaGetLastError();
}

}  // namespace csat
