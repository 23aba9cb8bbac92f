// K~|V~ = Phi_h [K|V]  (paper: compression equation) on the sm_100a tensor cores.
//
// Per (batch, head) this is one GEMM  C[m, 2d] = Phi_h[m, n] * [K|V][n, 2d]  with the token axis n as the
// reduction.  One CTA owns a 128 x 2d tile of C (128 measurements, all K and V columns) in tensor memory
// and walks the tokens in chunks of 64:
//   warp 0   : TMA producer.  Phi tile {64 tokens x 128 rows} (K-major A operand) and {64 cols x 64 tokens}
//              boxes of K and V (MN-major B operand: tokens are the rows of K and V as the caller stores
//              them, so no transpose pass is needed), 128-byte swizzle, ring of kStages buffers.
//   warp 1   : allocates tensor memory; one elected thread issues tcgen05.mma (M=128, N=2d, K=16, bf16
//              in, fp32 accumulate) and commits to the ring's "empty" barriers.
//   warps 2-5: epilogue: tcgen05.ld the accumulator (each warp its 32-lane quarter), round to bf16, and write
//              row r of the tile as K~_r | V~_r into the workspace: through boxes of 32 rows x 64 columns in the
//              ring's shared memory (free once the last MMA has finished) and one TMA store per box, so that no
//              thread sits at stores of 16-byte pieces of 32 different lines.
// Rows of Phi beyond m and tokens beyond n are zero-filled by TMA (and Phi's padded columns hold zeros).
// Token-sharded use: the same kernel over a token range [phi_j0, phi_j0 + n) of Phi against a shard of K, V that
// holds only those n tokens; the epilogue then writes the float32 partial sums to `partial` instead of the
// workspace (they are summed over the shards, in a fixed order, before anything reads them).
#include "csat_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace csat {
namespace {

using namespace ptx;

constexpr int kTileM = 128;      // measurements per CTA
constexpr int kChunk = 64;       // tokens per pipeline stage (one 128-byte swizzled row of bf16)
constexpr int kThreads = 192;
constexpr uint32_t kABytes = kTileM * kChunk * 2;     // 16 KB
constexpr uint32_t kBoxBytes = 64 * kChunk * 2;       // 8 KB: 64 columns x 64 tokens

// SEP: separate measurement matrices for keys and values (a second A tile per stage, Phi_V, which multiplies the
// V columns; the K columns keep Phi_K)
// BG: batch elements per CTA.  They share the Phi tile; their K (then their V) columns sit side by side in the B
// operand and the accumulator: [K of element 0 .. K of element BG-1 | V of element 0 .. V of element BG-1].  With
// d = 64 one element gives an N = 128 MMA, which needs 32 KB of operands per 256 cycles of tensor work: right at
// what an SM can load; two elements (N = 256) halve the operand bytes per flop and the L2 reads of Phi.
// MT: measurement tiles per CTA (1 or 2; 2 only without SEP).  Two tiles of the same (batch, head) share every K, V
// chunk: a second A tile per stage and a second accumulator, so the B operand is loaded once for twice the products.
template <int D, bool SEP, int BG, int MT = 1> struct Cfg {
  static constexpr int kN = 2 * D * BG;               // accumulator columns (per measurement tile)
  static constexpr int kBoxes = kN / 64;              // B boxes per stage
  static constexpr int kATiles = SEP ? 2 : MT;
  static constexpr int kStages = (D == 64 && BG == 1) ? ((SEP || MT == 2) ? 4 : 6) : ((SEP || MT == 2) ? 3 : 4);
  static_assert(kN <= 256, "one MMA covers the accumulator");
  static_assert(!(SEP && MT == 2) && MT * kN <= 512, "tensor memory");
  static constexpr uint32_t kStageBytes = kATiles * kABytes + kBoxes * kBoxBytes;
  static constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
  static constexpr uint32_t kOutBoxBytes = 32 * 128;  // epilogue staging: one warp's 32 rows x 64 columns of bf16
  static_assert(4 * MT * (kN / 64) * kOutBoxBytes <= kStages * kStageBytes, "the epilogue's boxes fit in the ring");
};

template <int D, bool SEP, int BG, int MT>
__global__ void __launch_bounds__(kThreads, 1)
compress_sm100_kernel(const __grid_constant__ CUtensorMap tmap_phi, const __grid_constant__ CUtensorMap tmap_k,
                      const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_out,
                      __nv_bfloat16* __restrict__ kv, int m, int n, int H,
                      int B, int bh0, int* status, int phi_j0, float* __restrict__ partial) {
  using C = Cfg<D, SEP, BG, MT>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* a_buf = smem;                                      // [stages][A tiles][16 KB]
  uint8_t* b_buf = smem + C::kStages * C::kATiles * kABytes;  // [stages][boxes][8 KB]
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + C::kStages * C::kStageBytes);
  uint64_t* empty = full + C::kStages;
  uint64_t* acc_done = empty + C::kStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_done + 1);
  int* cta_abort = reinterpret_cast<int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // blockIdx.y walks the batch fastest, so that the CTAs that stream the same tile of Phi_h (one per batch
  // element) are scheduled together and all but the first find it in L2
  // (with BG > 1 blockIdx.y counts groups of BG batch elements; a group that runs past the batch repeats its
  // last element and does not store it)
  const int groups = (B + BG - 1) / BG;
  const int mtile = blockIdx.x * MT, h = blockIdx.y / groups, b0 = (blockIdx.y % groups) * BG;   // first of MT tiles
  // bh0: first (batch, head) pair of a sub-range launch (then B = 1 and blockIdx.y counts its heads); 0 otherwise
  const int hl = h;
  auto bh_of = [&](int e) { return bh0 + (b0 + e < B ? b0 + e : B - 1) * H + hl; };
  const int hphi = bh_of(0) % H;                    // head whose Phi this CTA streams
  const int nchunks = (n + kChunk - 1) / kChunk;

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_phi);
    prefetch_tmap(&tmap_k);
    prefetch_tmap(&tmap_v);
    prefetch_tmap(&tmap_out);
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    mbar_init(acc_done, 1);
    *cta_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, MT * C::kN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // the kernel after this one in the stream (attention / recovery) may be scheduled as SMs free up: its prologue
  // and its Q loads overlap this kernel's tail; it waits for this grid before it reads K~|V~
  pdl_launch_dependents();

  if (warp == 0) {
    if (elect_one()) {
      int issued = 0;
      bool ok = true;
      for (int i = 0; i < nchunks && ok; ++i) {
        const int s = i % C::kStages;
        ok = mbar_wait(&empty[s], ((i / C::kStages) & 1) ^ 1, status, 101, cta_abort);
        if (!ok) break;
        mbar_arrive_expect_tx(&full[s], C::kStageBytes);
        tma_load_3d(a_buf + s * C::kATiles * kABytes, &tmap_phi, &full[s], phi_j0 + i * kChunk, mtile * kTileM, hphi);
        if (SEP) tma_load_3d(a_buf + (s * C::kATiles + 1) * kABytes, &tmap_phi, &full[s], phi_j0 + i * kChunk, mtile * kTileM, H + hphi);
        if (MT == 2)   // the next measurement tile of the same head (rows beyond m are zero-filled)
          tma_load_3d(a_buf + (s * C::kATiles + 1) * kABytes, &tmap_phi, &full[s], phi_j0 + i * kChunk, (mtile + 1) * kTileM, hphi);
#pragma unroll
        for (int g = 0; g < C::kBoxes; ++g) {
          const bool is_v = g >= C::kBoxes / 2;
          const int gg = g % (C::kBoxes / 2);               // box within the K (or V) half: element, then 64-column box
          tma_load_3d(b_buf + (s * C::kBoxes + g) * kBoxBytes, is_v ? &tmap_v : &tmap_k, &full[s],
                      (gg % (D / 64)) * 64, i * kChunk, bh_of(gg / (D / 64)));
        }
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
      constexpr uint32_t idesc = make_idesc_bf16(kTileM, SEP ? C::kN / 2 : C::kN, /*A MN-major*/ false, /*B MN-major*/ true);
      bool ok = true;
      for (int i = 0; i < nchunks; ++i) {
        const int s = i % C::kStages;
        ok = mbar_wait(&full[s], (i / C::kStages) & 1, status, 103, cta_abort);
        if (!ok) break;
        tc_fence_after();
        const uint64_t a_desc = make_smem_desc(smem_u32(a_buf + s * C::kATiles * kABytes), 16, 1024);
        const uint64_t b_desc = make_smem_desc(smem_u32(b_buf + s * C::kBoxes * kBoxBytes), kBoxBytes, 1024);
#pragma unroll
        for (int k = 0; k < kChunk / 16; ++k) { // +32 B along K for A, +2048 B (16 token rows) for B
          mma_f16_ss(tmem_base, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)(k * 128), idesc, (i | k) != 0);
          if (SEP)                              // V columns: the second A tile, the V boxes, accumulator columns [d, 2d)
            mma_f16_ss(tmem_base + C::kN / 2, a_desc + (uint64_t)((kABytes >> 4) + k * 2),
                       b_desc + (uint64_t)(((C::kBoxes / 2) * kBoxBytes >> 4) + k * 128), idesc, (i | k) != 0);
          if (MT == 2)                          // the second measurement tile: its A tile, the same B, its own accumulator
            mma_f16_ss(tmem_base + C::kN, a_desc + (uint64_t)((kABytes >> 4) + k * 2), b_desc + (uint64_t)(k * 128), idesc,
                       (i | k) != 0);
        }
        mma_commit(&empty[s]);                  // stage reusable once these MMAs have read it
      }
      mma_commit(acc_done);                     // arrives when every MMA above has finished (also after a give-up)
    }
  } else {
    const int q = warp & 3;                     // this warp may touch TMEM lanes [32q, 32q+32)
    if (mbar_wait(acc_done, 0, status, 104, cta_abort) && *(volatile int*)cta_abort == 0) {
      tc_fence_after();
#pragma unroll 1
      for (int mt = 0; mt < MT; ++mt) {
      const int row = (mtile + mt) * kTileM + q * 32 + lane;
#pragma unroll 1
      for (int c0 = 0; c0 < C::kN; c0 += 32) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(mt * C::kN + c0), r);
        tmem_wait_ld();
        // accumulator column c0: K half or V half, batch element e of the group, feature column
        const int half = c0 / (C::kN / 2), e = (c0 % (C::kN / 2)) / D, col = c0 % D;
        if (row < m && b0 + e < B && partial != nullptr) {
          float4* o = reinterpret_cast<float4*>(partial + ((int64_t)bh_of(e) * m + row) * (2 * D) + half * D + col);
#pragma unroll
          for (int v = 0; v < 8; ++v)
            o[v] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]), __uint_as_float(r[4 * v + 2]),
                               __uint_as_float(r[4 * v + 3]));
        } else if (partial == nullptr) {
          // box (mt, c0 / 64) of this warp; this thread's row of it, 16-byte pieces in the 128-byte swizzle
          uint8_t* box = smem + ((q * MT + mt) * (C::kN / 64) + c0 / 64) * C::kOutBoxBytes;
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
          if (c0 % 64 == 32) {                      // the box is complete (rows beyond m are clipped by the tensor map)
            fence_proxy_async();
            __syncwarp();
            const int row0 = (mtile + mt) * kTileM + q * 32;
            if (lane == 0 && row0 < m && b0 + e < B)
              tma_store_3d(&tmap_out, box, half * D + (col & ~63), row0, bh_of(e));
          }
        }
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
  if (warp == 1) tmem_dealloc(tmem_base, MT * C::kN);
}

// Self-test of the bounded wait: one thread waits on a barrier that nothing arrives at.  The wait gives up after
// limit_ns, writes code 999 into the status word and the kernel returns normally (no trap, no endless loop).
__global__ void wait_timeout_selftest_kernel(int* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int cta_abort;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    cta_abort = 0;
    fence_mbar_init();
    mbar_wait(&bar, 0, status, 999, &cta_abort, limit_ns);
  }
}

// n_len tokens of K, V (a shard that starts at token phi_j0 of the sequence, or the whole sequence); partial: float32
// destination of a shard's sums, null = the workspace
template <int D, bool SEP, int BG, int MT = 1>
cudaError_t launch(csat_ctx* c, const void* K, const void* V, cudaStream_t s, int64_t phi_j0, int64_t n_len,
                   float* partial) {
  using C = Cfg<D, SEP, BG, MT>;
  const Params& p = c->p;
  CUtensorMap tk, tv;
  const uint64_t kd[3] = {(uint64_t)D, (uint64_t)n_len, (uint64_t)(p.B * p.H)};
  const uint64_t ks[2] = {(uint64_t)D * 2, (uint64_t)n_len * D * 2};
  const uint32_t kb[3] = {64, (uint32_t)kChunk, 1};
  cudaError_t e;
  if ((e = make_tmap_bf16_3d(&tk, K, kd, ks, kb)) != cudaSuccess) return e;
  if ((e = make_tmap_bf16_3d(&tv, V, kd, ks, kb)) != cudaSuccess) return e;
  static DeviceFlags smem_opt_in;
  if ((e = ensure_dynamic_smem(compress_sm100_kernel<D, SEP, BG, MT>, (int)C::kSmemBytes, c->device, smem_opt_in)) != cudaSuccess)
    return e;
  // whole batch, or a range of heads of one batch element
  const int64_t Bl = c->bh_cnt ? 1 : p.B, Hl = c->bh_cnt ? c->bh_cnt : p.H;
  const int64_t mtiles = (p.m + kTileM - 1) / kTileM;
  const dim3 grid((unsigned)((mtiles + MT - 1) / MT), (unsigned)(((Bl + BG - 1) / BG) * Hl));
  compress_sm100_kernel<D, SEP, BG, MT><<<grid, kThreads, C::kSmemBytes, s>>>(c->tmap_phi, tk, tv, c->tmap_kv_st, (__nv_bfloat16*)c->kv, (int)p.m,
                                                                 (int)n_len, (int)p.H, (int)Bl, (int)c->bh0, c->status,
                                                                 (int)phi_j0, partial);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_wait_timeout_selftest(csat_ctx* c, unsigned long long limit_ns, cudaStream_t s) {
  wait_timeout_selftest_kernel<<<1, 32, 0, s>>>(c->status, limit_ns);
  return cudaGetLastError();
}

cudaError_t make_phi_tmap(csat_ctx* c) {
  const Params& p = c->p;
  const uint64_t d[3] = {(uint64_t)p.n_pad, (uint64_t)p.m, (uint64_t)c->phi_heads()};
  const uint64_t st[2] = {(uint64_t)p.n_pad * 2, (uint64_t)p.m * p.n_pad * 2};
  const uint32_t b[3] = {(uint32_t)kChunk, (uint32_t)kTileM, 1};
  return make_tmap_bf16_3d(&c->tmap_phi, c->phi, d, st, b);
}

cudaError_t launch_sm100_compress(csat_ctx* c, const void* K, const void* V, cudaStream_t s, int* launches,
                                  int64_t phi_j0, int64_t n_len, float* partial) {
  *launches += 1;
  if (n_len <= 0) n_len = c->p.n;
  // two measurement tiles per CTA where that still leaves at least ~0.8 CTAs per SM
  const int64_t mtiles = (c->p.m + kTileM - 1) / kTileM;
  auto pairs_fill = [&](int64_t columns_of_ctas) { return mtiles >= 2 && ((mtiles + 1) / 2) * columns_of_ctas * 5 >= (int64_t)c->sms * 4; };
  // d = 64: two batch elements per CTA where the batch has them (N = 256 MMAs)
  if (c->p.d == 64 && c->p.B >= 2 && c->bh_cnt == 0) {
    if (c->p.separate_phi) return launch<64, true, 2>(c, K, V, s, phi_j0, n_len, partial);
    return pairs_fill(((c->p.B + 1) / 2) * c->p.H) ? launch<64, false, 2, 2>(c, K, V, s, phi_j0, n_len, partial)
                                                  : launch<64, false, 2>(c, K, V, s, phi_j0, n_len, partial);
  }
  if (c->p.separate_phi)
    return c->p.d == 64 ? launch<64, true, 1>(c, K, V, s, phi_j0, n_len, partial)
                        : launch<128, true, 1>(c, K, V, s, phi_j0, n_len, partial);
  if (c->p.d == 128 && pairs_fill(c->bh_cnt ? c->bh_cnt : c->p.B * c->p.H))
    return launch<128, false, 1, 2>(c, K, V, s, phi_j0, n_len, partial);
  return c->p.d == 64 ? launch<64, false, 1>(c, K, V, s, phi_j0, n_len, partial)
                      : launch<128, false, 1>(c, K, V, s, phi_j0, n_len, partial);
}

}  // namespace csat
