// Input projections Q = X W^Q, K = X W^K, V = X W^V (paper: "Mathematical Framework", the projection equation)
// for all heads at once, written straight into the [B, H, tokens, d] layout the attention kernels read.
//
// One GEMM C[tokens, cols] = X[tokens, d_model] * W[d_model, cols] on the sm_100a tensor cores, where the columns
// of W are the projection matrices side by side ([W^Q of heads 0..H-1 | W^K ... | W^V ...], d columns per head).
// Persistent CTAs, one per SM, walk 128 x 256 output tiles (column tiles fastest, so that the CTAs running at the
// same time share the rows of X in L2; W stays L2-resident):
//   warp 0   : TMA producer.  X tile {64 k x 128 tokens} (K-major A operand) and four {64 columns x 64 k} boxes
//              of W (MN-major B operand: W is used as the caller stores it), 128-byte swizzle, 4-stage ring.
//   warp 1   : allocates tensor memory (two 256-column accumulators); one elected thread issues tcgen05.mma
//              (M = 128, N = 256, K = 16) and commits the ring's "empty" barriers and the accumulator's "full".
//   warps 2-5: epilogue of tile i while the MMAs of tile i + 1 fill the other accumulator: tcgen05.ld, round to
//              bf16, store each row's 32-column groups at their head's place in Q, K or V.
// Token tiles never straddle a batch element; tokens beyond n, columns beyond the last and k beyond d_model are
// zero-filled by TMA and skipped by the epilogue.  Every wait is bounded (see sm100_ptx.cuh).
#include "csat_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace csat {
namespace {

using namespace ptx;

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

constexpr int kTileM = 128, kTileN = 256, kChunkK = 64, kStages = 4, kThreads = 192;
constexpr uint32_t kABytes = kTileM * kChunkK * 2;       // 16 KB
constexpr uint32_t kBoxBytes = 64 * kChunkK * 2;         // 8 KB: 64 columns x 64 k
constexpr int kBoxes = kTileN / 64;
constexpr uint32_t kStageBytes = kABytes + kBoxes * kBoxBytes;
constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;

struct ProjArgs {
  __nv_bfloat16* dst[3];      // Q, K, V (any may be null if its columns are not in [col0, col0 + ncols))
  int64_t rows[3];            // tokens per (batch, head) of each destination: n_q, n, n
  int n_tok, B, H, dm;        // tokens per batch element of X; batch; heads; reduction length
  int col0, ncols;            // columns of W this launch computes
  int mtiles, ntiles;         // token tiles per batch element, column tiles
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
project_sm100_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                     const ProjArgs a, int* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* a_buf = smem;                                  // [stages][16 KB]
  uint8_t* b_buf = smem + kStages * kABytes;              // [stages][boxes][8 KB]
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  uint64_t* empty = full + kStages;
  uint64_t* acc_full = empty + kStages;                   // [2]
  uint64_t* acc_empty = acc_full + 2;                     // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  int* cta_abort = reinterpret_cast<int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nk = (a.dm + kChunkK - 1) / kChunkK;
  const int n_tiles = a.B * a.mtiles * a.ntiles;

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_x);
    prefetch_tmap(&tmap_w);
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
      uint32_t it = 0;                                    // chunks loaded so far (ring position)
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const int nt = tile % a.ntiles, mg = tile / a.ntiles, b = mg / a.mtiles, mt = mg % a.mtiles;
        for (int k = 0; k < nk && ok; ++k, ++it) {
          const int s = it % kStages;
          ok = mbar_wait(&empty[s], ((it / kStages) & 1) ^ 1, status, 301, cta_abort);
          if (!ok) break;
          mbar_arrive_expect_tx(&full[s], kStageBytes);
          tma_load_3d(a_buf + s * kABytes, &tmap_x, &full[s], k * kChunkK, mt * kTileM, b);
#pragma unroll
          for (int g = 0; g < kBoxes; ++g)
            tma_load_3d(b_buf + (s * kBoxes + g) * kBoxBytes, &tmap_w, &full[s], a.col0 + nt * kTileN + g * 64,
                        k * kChunkK, 0);
        }
      }
      if (!ok) {
        // gave up: let copies that are still in flight land before the CTA's shared memory goes away
        for (uint32_t i = it > (uint32_t)kStages ? it - kStages : 0; i < it; ++i)
          mbar_wait_drain(&full[i % kStages], (i / kStages) & 1);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      constexpr uint32_t idesc = make_idesc_bf16(kTileM, kTileN, /*A MN-major*/ false, /*B MN-major*/ true);
      uint32_t it = 0, tc = 0;                            // chunks consumed; tiles of this CTA so far
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tc) {
        const uint32_t buf = tc & 1;
        ok = mbar_wait(&acc_empty[buf], ((tc >> 1) & 1) ^ 1, status, 302, cta_abort);   // the epilogue has read it
        if (!ok) break;
        tc_fence_after();
        const uint32_t acc = tmem_base + buf * kTileN;
        for (int k = 0; k < nk; ++k, ++it) {
          const int s = it % kStages;
          ok = mbar_wait(&full[s], (it / kStages) & 1, status, 303, cta_abort);
          if (!ok) break;
          tc_fence_after();
          const uint64_t a_desc = make_smem_desc(smem_u32(a_buf + s * kABytes), 16, 1024);
          const uint64_t b_desc = make_smem_desc(smem_u32(b_buf + s * kBoxes * kBoxBytes), kBoxBytes, 1024);
#pragma unroll
          for (int kk = 0; kk < kChunkK / 16; ++kk)       // +32 B along K for A, +2048 B (16 k rows) for B
            mma_f16_ss(acc, a_desc + (uint64_t)(kk * 2), b_desc + (uint64_t)(kk * 128), idesc, (k | kk) != 0);
          mma_commit(&empty[s]);                          // stage reusable once these MMAs have read it
        }
        mma_commit(&acc_full[buf]);                       // arrives when the tile's MMAs have finished
      }
    }
  } else {
    const int q = warp & 3;                               // this warp may touch TMEM lanes [32q, 32q+32)
    const int HD = a.H * D;
    uint32_t tc = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tc) {
      const int nt = tile % a.ntiles, mg = tile / a.ntiles, b = mg / a.mtiles, mt = mg % a.mtiles;
      const uint32_t buf = tc & 1;
      ok = mbar_wait(&acc_full[buf], (tc >> 1) & 1, status, 304, cta_abort) && *(volatile int*)cta_abort == 0;
      if (!ok) break;
      tc_fence_after();
      const int tok = mt * kTileM + q * 32 + lane;
#pragma unroll 1
      for (int c0 = 0; c0 < kTileN; c0 += 32) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16) + buf * kTileN + (uint32_t)c0, r);
        tmem_wait_ld();
        const int rel = nt * kTileN + c0;                 // column within this launch's range
        if (tok < a.n_tok && rel < a.ncols) {
          // 32 consecutive columns lie inside one head (d is a multiple of 64): which matrix, head, column
          const int col = a.col0 + rel, which = col / HD, hh = (col % HD) / D, c = col % D;
          __nv_bfloat16* o = a.dst[which] + (((int64_t)b * a.H + hh) * a.rows[which] + tok) * D + c;
          uint32_t w[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            __nv_bfloat162 p = __floats2bfloat162_rn(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
            w[j] = *reinterpret_cast<uint32_t*>(&p);
          }
          uint4* o4 = reinterpret_cast<uint4*>(o);
#pragma unroll
          for (int v = 0; v < 4; ++v) o4[v] = make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
        }
      }
      tc_fence_before();
      mbar_arrive(&acc_empty[buf]);                       // 128 arrivals: the accumulator may be overwritten
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, 2 * kTileN);
}

// plain FFMA version (float32 storage, or shapes the tensor-core kernel does not take): one thread per output
template <typename T>
__global__ void project_simt_kernel(const T* __restrict__ X, const T* __restrict__ W, T* __restrict__ Qo,
                                    T* __restrict__ Ko, T* __restrict__ Vo, int64_t rows_q, int64_t rows_kv, int n_tok,
                                    int B, int H, int d, int dm, int col0, int ncols, int ldw) {
  const int64_t total = (int64_t)B * n_tok * ncols;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int rel = (int)(i % ncols);
    const int64_t bt = i / ncols;
    const int tok = (int)(bt % n_tok), b = (int)(bt / n_tok);
    const int col = col0 + rel, which = col / (H * d), hh = (col % (H * d)) / d, c = col % d;
    const T* x = X + ((int64_t)b * n_tok + tok) * dm;
    float acc = 0.f;
    for (int k = 0; k < dm; ++k) acc = fmaf(to_float(x[k]), to_float(W[(int64_t)k * ldw + col]), acc);
    T* dst = which == 0 ? Qo : (which == 1 ? Ko : Vo);
    const int64_t rows = which == 0 ? rows_q : rows_kv;
    dst[(((int64_t)b * H + hh) * rows + tok) * d + c] = from_float<T>(acc);
  }
}

}  // namespace

// One launch: columns [col0, col0 + ncols) of W applied to X [B, n_tok, dm]; the destinations those columns map to
// must be non-null.  W is [dm, 3 H d] row-major.
cudaError_t launch_project(csat_ctx* c, const void* X, const void* W, int64_t n_tok, int64_t dm, int col0, int ncols,
                           void* Q, void* K, void* V, cudaStream_t s, int* launches) {
  const Params& p = c->p;
  const int ldw = (int)(3 * p.H * p.d);
  *launches += 1;
  const bool tensor_core = p.dtype == CSAT_DTYPE_BF16 && (p.d == 64 || p.d == 128) && dm % 8 == 0 && c->force_simt == 0;
  if (!tensor_core) {
    const int64_t total = p.B * n_tok * ncols;
    int64_t g = (total + 255) / 256;
    if (g > 148 * 32) g = 148 * 32;
    if (p.dtype == CSAT_DTYPE_FP32)
      project_simt_kernel<float><<<(unsigned)g, 256, 0, s>>>((const float*)X, (const float*)W, (float*)Q, (float*)K,
                                                            (float*)V, p.nq, p.n, (int)n_tok, (int)p.B, (int)p.H,
                                                            (int)p.d, (int)dm, col0, ncols, ldw);
    else
      project_simt_kernel<__nv_bfloat16><<<(unsigned)g, 256, 0, s>>>(
          (const __nv_bfloat16*)X, (const __nv_bfloat16*)W, (__nv_bfloat16*)Q, (__nv_bfloat16*)K, (__nv_bfloat16*)V, p.nq,
          p.n, (int)n_tok, (int)p.B, (int)p.H, (int)p.d, (int)dm, col0, ncols, ldw);
    return cudaGetLastError();
  }
  CUtensorMap tx, tw;
  const uint64_t xd[3] = {(uint64_t)dm, (uint64_t)n_tok, (uint64_t)p.B};
  const uint64_t xs[2] = {(uint64_t)dm * 2, (uint64_t)n_tok * dm * 2};
  const uint32_t xb[3] = {(uint32_t)kChunkK, (uint32_t)kTileM, 1};
  const uint64_t wd[3] = {(uint64_t)ldw, (uint64_t)dm, 1};
  const uint64_t ws[2] = {(uint64_t)ldw * 2, (uint64_t)dm * ldw * 2};
  const uint32_t wb[3] = {64, (uint32_t)kChunkK, 1};
  cudaError_t e;
  if ((e = make_tmap_bf16_3d(&tx, X, xd, xs, xb)) != cudaSuccess) return e;
  if ((e = make_tmap_bf16_3d(&tw, W, wd, ws, wb)) != cudaSuccess) return e;
  ProjArgs a;
  a.dst[0] = (__nv_bfloat16*)Q; a.dst[1] = (__nv_bfloat16*)K; a.dst[2] = (__nv_bfloat16*)V;
  a.rows[0] = p.nq; a.rows[1] = p.n; a.rows[2] = p.n;
  a.n_tok = (int)n_tok; a.B = (int)p.B; a.H = (int)p.H; a.dm = (int)dm;
  a.col0 = col0; a.ncols = ncols;
  a.mtiles = (int)((n_tok + kTileM - 1) / kTileM);
  a.ntiles = (ncols + kTileN - 1) / kTileN;
  const int64_t n_tiles = (int64_t)a.B * a.mtiles * a.ntiles;
  if (n_tiles > (int64_t)1 << 30) return cudaErrorInvalidValue;
  const int sms = c->sms;
  const unsigned grid = (unsigned)(n_tiles < sms ? n_tiles : sms);
  if (p.d == 64) {
    static DeviceFlags opt_in64;
    if ((e = ensure_dynamic_smem(project_sm100_kernel<64>, (int)kSmemBytes, c->device, opt_in64)) != cudaSuccess) return e;
    project_sm100_kernel<64><<<grid, kThreads, kSmemBytes, s>>>(tx, tw, a, c->status);
  } else {
    static DeviceFlags opt_in128;
    if ((e = ensure_dynamic_smem(project_sm100_kernel<128>, (int)kSmemBytes, c->device, opt_in128)) != cudaSuccess) return e;
    project_sm100_kernel<128><<<grid, kThreads, kSmemBytes, s>>>(tx, tw, a, c->status);
  }
  return cudaGetLastError();
}

}  // namespace csat
