// V~ B for the forward's recovery phase, on the sm_100a tensor cores.
//
// The LISTA recurrence of the paper starts from z B, with z = A~ V~ the compressed attention output of a query.  The
// product is associative: z B = A~ (V~ B).  Where one B serves all layers, V~ B (m rows per (batch, head)) is formed
// here once, and the attention phase accumulates P (V~ B) instead of P V~, so that the n_q products z B (and the
// round trip thread -> tensor pipe -> thread they cost every tile of queries) disappear from the recovery phase.
//
// One CTA per tile of 128 measurements of one (batch, head):
//   warp 0   : TMA: the tile's V~ rows from the K~|V~ workspace (K-major A operand) and the head's B (stored
//              [output column][k], the K-major B operand the recovery phase also uses).
//   warp 1   : allocates tensor memory; one elected thread issues the d / 16 MMAs (M = 128, N = d).
//   warps 2-5: epilogue: accumulator -> bf16 -> boxes of 32 rows x 64 columns in the V~ tile's shared memory -> TMA
//              stores into the V~ B workspace (rows beyond m are clipped by the tensor map).
// It runs as a programmatic dependent of the compression kernel and lets the attention kernel start under it.
#include "csat_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace csat {
namespace {

using namespace ptx;

constexpr int kRows = 128;       // measurements per CTA
constexpr int kMC = 64;          // rows per box of the K~|V~ tensor map
constexpr int kThreads = 192;

template <int D> struct Cfg {
  static constexpr int kDBoxes = D / 64;
  static constexpr uint32_t kTileBoxBytes = kRows * 128;            // 128 rows x 64 columns
  static constexpr uint32_t kTileBytes = kDBoxes * kTileBoxBytes;
  static constexpr uint32_t kMatBoxBytes = D * 128;                 // one 64-column box of a d x d bf16 matrix
  static constexpr uint32_t kMatBytes = kDBoxes * kMatBoxBytes;
  static constexpr uint32_t kOffA = 0, kOffB = kTileBytes, kOffBar = kTileBytes + kMatBytes;
  static constexpr uint32_t kSmemBytes = kOffBar + 64 + 1024 /*alignment slack*/;
};

struct Bars {
  uint64_t full, done;
  uint32_t tmem_slot;
  int abort;
};

template <int D>
__global__ void __launch_bounds__(kThreads, 2)
vfold_sm100_kernel(const __grid_constant__ CUtensorMap tmap_kv, const __grid_constant__ CUtensorMap tmap_mats,
                   const __grid_constant__ CUtensorMap tmap_out, int H, int bh0, int* status) {
  using C = Cfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  Bars* bars = reinterpret_cast<Bars*>(smem + C::kOffBar);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row0 = blockIdx.x * kRows, bh = bh0 + blockIdx.y, h = bh % H;

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_kv);
    prefetch_tmap(&tmap_mats);
    prefetch_tmap(&tmap_out);
    mbar_init(&bars->full, 1);
    mbar_init(&bars->done, 1);
    bars->abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_slot, D);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_slot;
  pdl_launch_dependents();        // the attention kernel's prologue may run under this kernel; it waits for this grid

  if (warp == 0) {
    if (elect_one()) {
      pdl_wait();                 // V~ comes from the compression kernel before this one in the stream
      mbar_arrive_expect_tx(&bars->full, C::kTileBytes + C::kMatBytes);
      for (int gx = 0; gx < C::kDBoxes; ++gx)
        tma_load_3d(smem + C::kOffB + gx * C::kMatBoxBytes, &tmap_mats, &bars->full, gx * 64, 0, h * 3 + 1);
      for (int gx = 0; gx < C::kDBoxes; ++gx)
        for (int half = 0; half < kRows / kMC; ++half)
          tma_load_3d(smem + C::kOffA + gx * C::kTileBoxBytes + half * (kMC * 128), &tmap_kv, &bars->full,
                      D + gx * 64, row0 + half * kMC, bh);
    }
  } else if (warp == 1) {
    if (elect_one()) {
      if (mbar_wait(&bars->full, 0, status, 801, &bars->abort)) {
        tc_fence_after();
        constexpr uint32_t idesc = make_idesc_bf16(kRows, D, false, false);     // both operands K-major
        const uint64_t ad = make_smem_desc(smem_u32(smem + C::kOffA), 16, 1024);
        const uint64_t bd = make_smem_desc(smem_u32(smem + C::kOffB), 16, 1024);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)     // K step k: 64-column box k / 4, 32 (k % 4) bytes into each row
          mma_f16_ss(tmem, ad + (uint64_t)((k / 4) * (C::kTileBoxBytes >> 4) + (k % 4) * 2),
                     bd + (uint64_t)((k / 4) * (C::kMatBoxBytes >> 4) + (k % 4) * 2), idesc, k != 0);
      }
      mma_commit(&bars->done);    // arrives when the MMAs above have finished (also after a give-up)
    }
  } else {
    const int q = warp & 3;       // this warp may touch TMEM lanes [32q, 32q+32)
    if (mbar_wait(&bars->done, 0, status, 802, &bars->abort) && *(volatile int*)&bars->abort == 0) {
      tc_fence_after();
#pragma unroll
      for (int c0 = 0; c0 < D; c0 += 32) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
        tmem_wait_ld();
        // the warp's 32 rows of box c0 / 64, in the V~ tile's shared memory (its products have finished)
        uint8_t* box = smem + C::kOffA + (c0 / 64) * C::kTileBoxBytes + q * (32 * 128);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint32_t w[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            __nv_bfloat162 p = __floats2bfloat162_rn(__uint_as_float(r[v * 8 + 2 * j]), __uint_as_float(r[v * 8 + 2 * j + 1]));
            w[j] = *reinterpret_cast<uint32_t*>(&p);
          }
          const int piece = (c0 % 64) / 8 + v;
          *reinterpret_cast<uint4*>(box + lane * 128 + ((piece ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        if (c0 % 64 == 32) {
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) tma_store_3d(&tmap_out, box, c0 & ~63, row0 + q * 32, bh);
        }
      }
      if (lane == 0) {
        bulk_commit_group();
        bulk_wait_group0();       // the stores are done before the kernel ends
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, D);
}

template <int D>
cudaError_t launch(csat_ctx* c, cudaStream_t s) {
  using C = Cfg<D>;
  const Params& p = c->p;
  static DeviceFlags smem_opt_in;
  cudaError_t e = ensure_dynamic_smem(vfold_sm100_kernel<D>, (int)C::kSmemBytes, c->device, smem_opt_in);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((p.m + kRows - 1) / kRows), (unsigned)(c->bh_cnt ? c->bh_cnt : p.B * p.H));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, vfold_sm100_kernel<D>, c->tmap_kv, c->tmap_mats, c->tmap_vb_st, (int)p.H, (int)c->bh0,
                            c->status);
}

}  // namespace

// V~ B of every (batch, head) of the launch's range into the workspace behind K~|V~ (bf16 contexts, d in {64, 128},
// one B for all layers, the decoder's operands set up)
cudaError_t launch_sm100_vfold(csat_ctx* c, cudaStream_t s, int* launches) {
  *launches += 1;
  return c->p.d == 64 ? launch<64>(c, s) : launch<128>(c, s);
}

}  // namespace csat
