// dK = Phi_K^T dK~,  dV = Phi_V^T dV~  (backward of the paper's compression equation K~ = Phi K, V~ = Phi V)
// on the sm_100a tensor cores.
//
// Per (batch, head) one GEMM  C[n, 2d] = Phi_h^T[n, m] * [dK~|dV~][m, 2d]  with the measurement axis m as the
// reduction.  Phi is used as it is stored ([m, n_pad], tokens contiguous): the A operand is MN-major, so no
// transposed copy of Phi exists.  One CTA owns a 128-token x 2d tile of C in tensor memory and walks the
// measurements in chunks of 64:
//   warp 0   : TMA producer.  Two {64 tokens x 64 rows} boxes of Phi (MN-major A operand, M = 128) and the
//              {64 columns x 64 rows} boxes of dK~|dV~ (MN-major B operand), 128-byte swizzle, ring of stages.
//   warp 1   : allocates tensor memory; one elected thread issues tcgen05.mma (M=128, N=2d, K=16, bf16 in, fp32
//              accumulate) and commits to the ring's "empty" barriers.
//   warps 2-5: epilogue: tcgen05.ld the accumulator, round to bf16, and write the tile's rows of dK and dV through
//              boxes of 32 tokens x 64 columns in the ring's shared memory (free once the last MMA has finished)
//              and one TMA store per box (tokens beyond n are clipped by the tensor map).
// With separate Phi_K / Phi_V a stage holds both A tiles and the K and V halves are two N = d MMAs.
// Tokens beyond n and measurements beyond m are zero-filled by TMA.
#include "csat_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace csat {
namespace {

using namespace ptx;

constexpr int kTileM = 128;      // tokens per CTA
constexpr int kChunk = 64;       // measurements per pipeline stage
constexpr int kThreads = 192;
constexpr uint32_t kABoxBytes = 64 * kChunk * 2;      // 8 KB: 64 tokens x 64 rows
constexpr uint32_t kABytes = 2 * kABoxBytes;          // 128 tokens
constexpr uint32_t kBBoxBytes = 64 * kChunk * 2;      // 8 KB: 64 columns x 64 rows

template <int D, bool SEP> struct Cfg {
  static constexpr int kN = 2 * D;
  static constexpr int kBoxes = kN / 64;
  static constexpr int kATiles = SEP ? 2 : 1;
  // two CTAs per SM (one's epilogue under the other's products): 2 x 2 stages of 48 KB at d = 128, 2 x 3 of 32 KB at d = 64
  static constexpr int kStages = SEP ? (D == 64 ? 4 : 3) : (D == 64 ? 3 : 2);
  static constexpr uint32_t kStageBytes = kATiles * kABytes + kBoxes * kBBoxBytes;
  static constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
  static constexpr uint32_t kOutBoxBytes = 32 * 128;  // epilogue staging: one warp's 32 tokens x 64 columns of bf16
  static_assert(4 * (kN / 64) * kOutBoxBytes <= kStages * kStageBytes, "the epilogue's boxes fit in the ring");
};

template <int D, bool SEP>
__global__ void __launch_bounds__(kThreads, 2)
phiT_sm100_kernel(const __grid_constant__ CUtensorMap tmap_phi, const __grid_constant__ CUtensorMap tmap_g,
                  const __grid_constant__ CUtensorMap tmap_dk, const __grid_constant__ CUtensorMap tmap_dv, int m, int n,
                  int H, int* status) {
  using C = Cfg<D, SEP>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* a_buf = smem;                                      // [stages][A tiles][2 boxes of 8 KB]
  uint8_t* b_buf = smem + C::kStages * C::kATiles * kABytes;  // [stages][boxes][8 KB]
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + C::kStages * C::kStageBytes);
  uint64_t* empty = full + C::kStages;
  uint64_t* acc_done = empty + C::kStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_done + 1);
  int* cta_abort = reinterpret_cast<int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ttile = blockIdx.x, bh = blockIdx.y, h = bh % H;
  const int nchunks = (m + kChunk - 1) / kChunk;

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_phi);
    prefetch_tmap(&tmap_g);
    prefetch_tmap(&tmap_dk);
    prefetch_tmap(&tmap_dv);
    for (int s = 0; s < C::kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_done, 1);
    *cta_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, C::kN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (elect_one()) {
      int issued = 0;
      bool ok = true;
      for (int i = 0; i < nchunks && ok; ++i) {
        const int s = i % C::kStages;
        ok = mbar_wait(&empty[s], ((i / C::kStages) & 1) ^ 1, status, 401, cta_abort);
        if (!ok) break;
        mbar_arrive_expect_tx(&full[s], C::kStageBytes);
#pragma unroll
        for (int at = 0; at < C::kATiles; ++at)
#pragma unroll
          for (int g = 0; g < 2; ++g)                         // tokens [64 g, 64 g + 64) of the tile
            tma_load_3d(a_buf + (s * C::kATiles + at) * kABytes + g * kABoxBytes, &tmap_phi, &full[s],
                        ttile * kTileM + g * 64, i * kChunk, at * H + h);
#pragma unroll
        for (int g = 0; g < C::kBoxes; ++g)
          tma_load_3d(b_buf + (s * C::kBoxes + g) * kBBoxBytes, &tmap_g, &full[s], g * 64, i * kChunk, bh);
        ++issued;
      }
      if (!ok) {
        // gave up: let copies that are still in flight land before the CTA's shared memory goes away
        for (int i = issued > C::kStages ? issued - C::kStages : 0; i < issued; ++i)
          mbar_wait_drain(&full[i % C::kStages], (i / C::kStages) & 1);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      constexpr uint32_t idesc = make_idesc_bf16(kTileM, SEP ? C::kN / 2 : C::kN, /*A MN-major*/ true, /*B MN-major*/ true);
      bool ok = true;
      for (int i = 0; i < nchunks; ++i) {
        const int s = i % C::kStages;
        ok = mbar_wait(&full[s], (i / C::kStages) & 1, status, 403, cta_abort);
        if (!ok) break;
        tc_fence_after();
        // both operands MN-major: the next 64 elements along M / N start one box further, 16 k rows are 2048 B
        const uint64_t a_desc = make_smem_desc(smem_u32(a_buf + s * C::kATiles * kABytes), kABoxBytes, 1024);
        const uint64_t b_desc = make_smem_desc(smem_u32(b_buf + s * C::kBoxes * kBBoxBytes), kBBoxBytes, 1024);
#pragma unroll
        for (int k = 0; k < kChunk / 16; ++k) {
          mma_f16_ss(tmem_base, a_desc + (uint64_t)(k * 128), b_desc + (uint64_t)(k * 128), idesc, (i | k) != 0);
          if (SEP)                                // V columns: Phi_V, the V boxes, accumulator columns [d, 2d)
            mma_f16_ss(tmem_base + C::kN / 2, a_desc + (uint64_t)((kABytes >> 4) + k * 128),
                       b_desc + (uint64_t)(((C::kBoxes / 2) * kBBoxBytes >> 4) + k * 128), idesc, (i | k) != 0);
        }
        mma_commit(&empty[s]);
      }
      mma_commit(acc_done);
    }
  } else {
    const int q = warp & 3;                       // this warp may touch TMEM lanes [32q, 32q+32)
    if (mbar_wait(acc_done, 0, status, 404, cta_abort) && *(volatile int*)cta_abort == 0) {
      tc_fence_after();
      const int tok0 = ttile * kTileM + q * 32;   // this warp's first token
#pragma unroll 1
      for (int c0 = 0; c0 < C::kN; c0 += 32) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
        tmem_wait_ld();
        // box c0 / 64 of this warp; this thread's token row of it, 16-byte pieces in the 128-byte swizzle
        uint8_t* box = smem + (q * (C::kN / 64) + c0 / 64) * C::kOutBoxBytes;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint32_t w[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            __nv_bfloat162 p = __floats2bfloat162_rn(__uint_as_float(r[v * 8 + 2 * j]),
                                                     __uint_as_float(r[v * 8 + 2 * j + 1]));
            w[j] = *reinterpret_cast<uint32_t*>(&p);
          }
          const int piece = (c0 % 64) / 8 + v;
          *reinterpret_cast<uint4*>(box + lane * 128 + ((piece ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        if (c0 % 64 == 32) {                        // the box is complete
          fence_proxy_async();
          __syncwarp();
          if (lane == 0 && tok0 < n) tma_store_3d(c0 < D ? &tmap_dk : &tmap_dv, box, (c0 % D) & ~63, tok0, bh);
        }
      }
      if (lane == 0) {
        bulk_commit_group();
        bulk_wait_group0();                         // the stores are done before the kernel ends
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, C::kN);
}

template <int D, bool SEP>
cudaError_t launch(csat_ctx* c, const void* g16, void* dK, void* dV, cudaStream_t s) {
  using C = Cfg<D, SEP>;
  const Params& p = c->p;
  CUtensorMap tphi, tg;
  const uint64_t pd[3] = {(uint64_t)p.n_pad, (uint64_t)p.m, (uint64_t)c->phi_heads()};
  const uint64_t ps[2] = {(uint64_t)p.n_pad * 2, (uint64_t)p.m * p.n_pad * 2};
  const uint32_t pb[3] = {64, (uint32_t)kChunk, 1};
  const uint64_t gd[3] = {(uint64_t)(2 * D), (uint64_t)p.m, (uint64_t)(p.B * p.H)};
  const uint64_t gs[2] = {(uint64_t)(2 * D) * 2, (uint64_t)p.m * 2 * D * 2};
  const uint32_t gb[3] = {64, (uint32_t)kChunk, 1};
  cudaError_t e;
  if ((e = make_tmap_bf16_3d(&tphi, c->phi, pd, ps, pb)) != cudaSuccess) return e;
  if ((e = make_tmap_bf16_3d(&tg, g16, gd, gs, gb)) != cudaSuccess) return e;
  CUtensorMap tdk, tdv;                           // the outputs [B H, n, d] in boxes of one warp's 32 tokens
  const uint64_t od[3] = {(uint64_t)D, (uint64_t)p.n, (uint64_t)(p.B * p.H)};
  const uint64_t os[2] = {(uint64_t)D * 2, (uint64_t)p.n * D * 2};
  const uint32_t ob[3] = {64, 32, 1};
  if ((e = make_tmap_bf16_3d(&tdk, dK, od, os, ob)) != cudaSuccess) return e;
  if ((e = make_tmap_bf16_3d(&tdv, dV, od, os, ob)) != cudaSuccess) return e;
  static DeviceFlags smem_opt_in;
  if ((e = ensure_dynamic_smem(phiT_sm100_kernel<D, SEP>, (int)C::kSmemBytes, c->device, smem_opt_in)) != cudaSuccess) return e;
  const dim3 grid((unsigned)((p.n + kTileM - 1) / kTileM), (unsigned)(p.B * p.H));
  phiT_sm100_kernel<D, SEP><<<grid, kThreads, C::kSmemBytes, s>>>(tphi, tg, tdk, tdv, (int)p.m, (int)p.n, (int)p.H, c->status);
  return cudaGetLastError();
}

}  // namespace

// g16: dK~|dV~ as bf16 [B, H, m, 2d]; bf16 contexts with d in {64, 128}
cudaError_t launch_sm100_phiT(csat_ctx* c, const void* g16, void* dK, void* dV, cudaStream_t s, int* launches) {
  *launches += 1;
  if (c->p.separate_phi) return c->p.d == 64 ? launch<64, true>(c, g16, dK, dV, s) : launch<128, true>(c, g16, dK, dV, s);
  return c->p.d == 64 ? launch<64, false>(c, g16, dK, dV, s) : launch<128, false>(c, g16, dK, dV, s);
}

}  // namespace csat
