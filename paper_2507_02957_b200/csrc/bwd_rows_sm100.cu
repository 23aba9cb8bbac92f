// The per-query stages of the backward pass on the sm_100a tensor cores (bf16 storage, d in {64, 128}, one S, B for
// all layers).  The paper trains through its unrolled decoder but prints no backward pass: this is the chain rule
// through the LISTA recurrence alpha^{t+1} = eta_theta(alpha^t S + z B), the reconstruction C^ = Psi alpha, the
// compressed output Z = A~ V~ and the softmax over the measurements, with the derivative of eta_theta taken as 1
// where |x| > theta and 0 elsewhere.
//
// Before these kernels the forward's own kernels have left K~|V~ in the workspace, Z (bf16, as the forward rounds it
// for its first product) in bw_Z16, every row's log sum exp L in bw_LD and the layers' shrinkage decisions in
// bw_maskbits.
//
// bwd_recur_sm100_kernel, one CTA per tile of 128 queries (TMEM lane = query row, one thread per row): the recurrence
// run backwards.  The decisions |x_t| > theta_t are the forward kernel's own (it records them, one bit per column and
// layer, when it runs for the backward pass), so nothing of the forward recurrence is repeated here:
//   d alpha_T = G Psi (one MMA; G itself without a dictionary), then for t = T-1 .. 0
//        dx_t = d alpha_{t+1} o mask_t,   dZ += dx_t B^T,   d alpha_t = dx_t S^T = dx_t + dx_t (S - I)^T :
//   dx_t goes to tensor memory as the bf16 A operand of two MMAs, whose B operands are the forward's own
//   shared-memory tiles of S - I and B read as MN-major operands (a d x d tile with 128-byte rows is K-major when
//   its rows are the output columns and MN-major when they are the reduction index: the transposed product needs
//   no transposed copy); the identity part of S^T stays exact in float32 registers;
//   at the end dZ (bf16, the operand of the stages that follow) and D = <dZ, Z>.
//
// bwd_dq_sm100_kernel, one CTA per tile of 128 queries, K~|V~ streamed in chunks of 64 measurements:
//        S_j = Q K~_j^T,  dA_j = dZ V~_j^T                        (two SS MMAs into tensor memory)
//        dS_j = scale * exp(scale S_j - L) o (dA_j - D)           (one thread per row; bf16 back into tensor memory)
//        dQ  += dS_j K~_j                                         (TS MMA, K~_j read as an MN-major operand)
//   the structure of the forward's attention phase with the roles of the operands changed.
//
// Every wait is bounded (see sm100_ptx.cuh); a time-out sets the context's status word and the CTA winds down.
#include "csat_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace csat {
namespace {

using namespace ptx;

constexpr int kRows = 128;
constexpr int kMC = 64;

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

struct Waiter {
  int* status;
  int* cta_abort;
  bool dead = false;
  __device__ __forceinline__ void wait(uint64_t* bar, uint32_t parity, int code) {
    if (dead) return;
    if (!mbar_wait(bar, parity, status, code, cta_abort)) dead = true;
  }
};

// ====================================================================================================================
// recurrence backward
// ====================================================================================================================
// kUntied: one S_t, B_t per layer: the pair of the layer at work and the pair of the next one (two stages), then Psi
template <int D, bool kUntied = false> struct RCfg {
  static constexpr int kDBoxes = D / 64;
  static constexpr uint32_t kMatBoxBytes = D * 128;               // one 64-column box of a d x d bf16 matrix
  static constexpr uint32_t kMatBytes = kDBoxes * kMatBoxBytes;
  static constexpr uint32_t kOffMat = 0;                          // [3]: S - I | B | Psi, as the forward stages them
  static constexpr int kMats = kUntied ? 5 : 3;                   // untied: [stage 0: S_t - I | B_t][stage 1: ...][Psi]
  static constexpr uint32_t kOffBar = kMats * kMatBytes;
  static constexpr uint32_t kSmemBytes = kOffBar + 128 + 1024 /*alignment slack*/;
  // TMEM columns: accumulator | dZ accumulator | two bf16 operand buffers (two values per column)
  static constexpr uint32_t kColAcc = 0, kColDz = D, kColOp = 2 * D, kOpCols = D / 2;
  static constexpr uint32_t kTmemCols = (D == 64) ? 256 : 512;
  static_assert(2 * D + 2 * kOpCols <= kTmemCols, "TMEM budget");
};

struct RBars {
  uint64_t mats_full, a_full, r_full, op_free[2];
  uint64_t lm_full[2], lm_free[2];   // untied layers: a stage's pair of matrices has landed / has been read
  uint32_t tmem_slot;
  int abort;
};

constexpr int kRThreads = 160;      // warps 0-3: one thread per query row; warp 4: TMA and MMA issue

template <int D, bool kUntied>
__global__ void __launch_bounds__(kRThreads, 1)
bwd_recur_sm100_kernel(const __grid_constant__ CUtensorMap tmap_mats, const __nv_bfloat16* __restrict__ Z16,
                       const __nv_bfloat16* __restrict__ G, __nv_bfloat16* __restrict__ dZ16, float* __restrict__ ws_LD,
                       const uint32_t* __restrict__ maskbits, int nq, int H, int T, int has_psi, int* status,
                       __nv_bfloat16* __restrict__ dx_out, int64_t dx_slot) {
  using C = RCfg<D, kUntied>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  RBars* bars = reinterpret_cast<RBars*>(smem + C::kOffBar);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, h = bh % H, row0 = blockIdx.x * kRows;
  Waiter w{status, &bars->abort};

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_mats);
    mbar_init(&bars->mats_full, 1);
    mbar_init(&bars->a_full, kRows);
    mbar_init(&bars->r_full, 1);
    mbar_init(&bars->op_free[0], 1);
    mbar_init(&bars->op_free[1], 1);
    for (int s2 = 0; s2 < 2; ++s2) { mbar_init(&bars->lm_full[s2], 1); mbar_init(&bars->lm_free[s2], 1); }
    bars->abort = 0;
    fence_mbar_init();
  }
  if (warp == 4) {
    tmem_alloc(&bars->tmem_slot, C::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_slot;

  if (warp == 4) {
    if (T > 0 && elect_one()) {
      // ---- the decoder matrices of this head, then one MMA group per operand the threads publish ----
      // one S, B for all layers: tiles S - I | B | Psi of head h, loaded once.  One pair per layer (kUntied): the
      // tensor holds, per head, S_0 - I, B_0, S_1 - I, B_1, ..., then Psi; the layers are walked from the last to the
      // first through two stages, the pair of layer t - 2 loaded into the stage layer t's products have just read.
      const int mat0 = kUntied ? h * (2 * T + 1) : h * 3;
      auto load_mat = [&](int slot, int index, uint64_t* bar) {
        for (int gx = 0; gx < C::kDBoxes; ++gx)
          tma_load_3d(smem + C::kOffMat + slot * C::kMatBytes + gx * C::kMatBoxBytes, &tmap_mats, bar, gx * 64, 0, index);
      };
      auto load_layer = [&](int t) {              // into stage (T - 1 - t) & 1
        const int st = (T - 1 - t) & 1;
        mbar_arrive_expect_tx(&bars->lm_full[st], 2 * C::kMatBytes);
        load_mat(2 * st, mat0 + 2 * t, &bars->lm_full[st]);
        load_mat(2 * st + 1, mat0 + 2 * t + 1, &bars->lm_full[st]);
      };
      if (kUntied) {
        if (has_psi) {
          mbar_arrive_expect_tx(&bars->mats_full, C::kMatBytes);
          load_mat(4, mat0 + 2 * T, &bars->mats_full);
        }
        load_layer(T - 1);
        if (T > 1) load_layer(T - 2);
      } else {
        const int nmats = has_psi ? 3 : 2;
        mbar_arrive_expect_tx(&bars->mats_full, nmats * C::kMatBytes);
        for (int mat = 0; mat < nmats; ++mat) load_mat(mat, mat0 + mat, &bars->mats_full);
      }
      constexpr uint32_t idesc_t = make_idesc_bf16(kRows, D, false, true);    // transposed products: B MN-major
      const uint32_t acc = tmem + C::kColAcc, dz = tmem + C::kColDz;
      // product with the transpose of a matrix the forward stores [output column][k]: the tile's rows are now the
      // reduction index, 16 rows (2048 bytes) per K step, the next 64 output columns one box further.  The operands
      // alternate between two buffers (publication n uses buffer n & 1).
      auto mma_tr = [&](uint32_t d_t, uint32_t op, int slot, uint32_t accumulate) {
        const uint64_t bd = make_smem_desc(smem_u32(smem + C::kOffMat + slot * C::kMatBytes), C::kMatBoxBytes, 1024);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) mma_f16_ts(d_t, op + k * 8, bd + (uint64_t)(k * 128), idesc_t, k == 0 ? accumulate : 1u);
      };
      uint32_t n_ops = 0;
      auto operand_ready = [&]() {
        w.wait(&bars->a_full, n_ops & 1, 601);
        ++n_ops;
        tc_fence_after();
      };
      if (!kUntied || has_psi) w.wait(&bars->mats_full, 0, 600);
      // The threads only wait for the product they need next (r_full); the dZ product trails it and releases the
      // operand buffer (op_free) when it has read it.
      if (has_psi) {                                           // d alpha_T = G Psi
        const uint32_t op = tmem + C::kColOp + (n_ops & 1) * C::kOpCols;
        operand_ready();
        mma_tr(acc, op, kUntied ? 4 : 2, 0u);
        mma_commit(&bars->r_full);
        mma_commit(&bars->op_free[(n_ops - 1) & 1]);
      }
      for (int t = T - 1; t >= 0; --t) {
        const uint32_t op = tmem + C::kColOp + (n_ops & 1) * C::kOpCols;
        const int li = T - 1 - t, st = li & 1;                 // untied: this layer's stage
        operand_ready();
        if (kUntied) {
          w.wait(&bars->lm_full[st], (li >> 1) & 1, 602);
          tc_fence_after();
        }
        const int sS = kUntied ? 2 * st : 0, sB = kUntied ? 2 * st + 1 : 1;
        if (t > 0) {
          mma_tr(acc, op, sS, 0u);                             // dx_t (S_t - I)^T
          mma_commit(&bars->r_full);
        }
        mma_tr(dz, op, sB, t == T - 1 ? 0u : 1u);              // dZ += dx_t B_t^T
        if (t == 0) mma_commit(&bars->r_full);                 // the last result the threads wait for is dZ itself
        mma_commit(&bars->op_free[(n_ops - 1) & 1]);
        if (kUntied && t >= 2) {                               // the stage is free once these products have read it
          mma_commit(&bars->lm_free[st]);
          w.wait(&bars->lm_free[st], (li >> 1) & 1, 603);
          if (!w.dead) load_layer(t - 2);
        }
      }
      if (w.dead && kUntied) {                                 // gave up: let the copies in flight land
        mbar_wait_drain(&bars->lm_full[0], 0);                 // (whichever phase: a bounded wait either way)
        mbar_wait_drain(&bars->lm_full[1], 0);
      }
      if (w.dead && (!kUntied || has_psi)) mbar_wait_drain(&bars->mats_full, 0);
    }
  } else {
    // ---------------------------------------------- one thread per query row ----------------------------------------
    const int row = warp * 32 + lane;
    const int grow = row0 + row;
    const bool live = grow < nq;
    const uint32_t tbase = tmem + ((uint32_t)(warp * 32) << 16);
    const uint32_t acc_addr = tbase + C::kColAcc, dz_addr = tbase + C::kColDz;
    const int64_t goff = ((int64_t)bh * nq + (live ? grow : 0)) * D;
    int phase = 0;
    uint32_t n_pub = 0;                           // operands published so far (buffer n_pub & 1)
    float v[D];                                   // d alpha_{t+1}, then dx_t
    // v as the bf16 A operand; with `keep` also to global memory (dx_t, for the gradients of the decoder's weights)
    auto publish_bf16 = [&](__nv_bfloat16* keep = nullptr) {
      const uint32_t op_addr = tbase + C::kColOp + (n_pub & 1) * C::kOpCols;
      // the buffer's previous operand (two publications ago) has been read by its trailing product
      if (n_pub >= 2) w.wait(&bars->op_free[n_pub & 1], ((n_pub >> 1) - 1) & 1, 613);
      ++n_pub;
#pragma unroll
      for (int c0 = 0; c0 < D; c0 += 16) {
        uint32_t pk[8];
#pragma unroll
        for (int e = 0; e < 16; e += 2) pk[e >> 1] = pack_bf16(v[c0 + e], v[c0 + e + 1]);
        tmem_st_32x32b_x8(op_addr + c0 / 2, pk);
        if (keep != nullptr) {
          uint4* kp = reinterpret_cast<uint4*>(keep + c0);
          kp[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          kp[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
        }
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bars->a_full);
    };
    {                                             // v := the row of the output gradient (0 beyond n_q)
      const uint4* p = reinterpret_cast<const uint4*>(G + goff);
#pragma unroll
      for (int c = 0; c < D / 8; ++c) {
        const uint4 q = live ? p[c] : make_uint4(0, 0, 0, 0);
        v[8 * c + 0] = bf16_lo(q.x); v[8 * c + 1] = bf16_hi(q.x);
        v[8 * c + 2] = bf16_lo(q.y); v[8 * c + 3] = bf16_hi(q.y);
        v[8 * c + 4] = bf16_lo(q.z); v[8 * c + 5] = bf16_hi(q.z);
        v[8 * c + 6] = bf16_lo(q.w); v[8 * c + 7] = bf16_hi(q.w);
      }
    }
    if (T > 0) {
      if (has_psi) {
        publish_bf16();                                         // G is bf16 already: nothing is lost
        w.wait(&bars->r_full, phase & 1, 611); ++phase;
        tc_fence_after();
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 16) {
          uint32_t r[16];
          tmem_ld_32x32b_x16(acc_addr + c0, r);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 16; ++e) v[c0 + e] = __uint_as_float(r[e]);          // d alpha_T = G Psi
        }
      }
      // the forward's decisions of layer t: column c is bit 31 - c % 32 of word c / 32 (loaded one layer ahead)
      auto load_masks = [&](int t, uint32_t (&m)[D / 32]) {
        const uint32_t* mp = maskbits + (((int64_t)bh * T + t) * nq + (live ? grow : 0)) * (D / 32);
#pragma unroll
        for (int q = 0; q < D / 32; ++q) m[q] = live ? mp[q] : 0u;
      };
      uint32_t mwd[D / 32], mnext[D / 32];
      load_masks(T - 1, mwd);
      for (int t = T - 1; t >= 0; --t) {
        // dx_t = d alpha_{t+1} o mask_t
#pragma unroll
        for (int c = 0; c < D; ++c)
          v[c] = ((mwd[c >> 5] >> (31 - (c & 31))) & 1u) ? v[c] : 0.f;
        publish_bf16(dx_out != nullptr && live && !w.dead ? dx_out + (int64_t)t * dx_slot + goff : nullptr);
        if (t > 0) load_masks(t - 1, mnext);
        w.wait(&bars->r_full, phase & 1, 612); ++phase;
        tc_fence_after();
#pragma unroll
        for (int q = 0; q < D / 32; ++q) mwd[q] = mnext[q];
        if (t > 0) {
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 16) {
            uint32_t r[16];
            tmem_ld_32x32b_x16(acc_addr + c0, r);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; ++e) v[c0 + e] += __uint_as_float(r[e]);        // d alpha_t = dx_t + dx_t (S - I)^T
          }
        }
      }
    }
    // ---- dZ (the accumulated products; G itself without a decoder) and D = <dZ, Z> ----
    float dsum = 0.f;
    const uint4* zp = reinterpret_cast<const uint4*>(Z16 + goff);
    uint4* out = reinterpret_cast<uint4*>(dZ16 + goff);
#pragma unroll
    for (int c0 = 0; c0 < D; c0 += 16) {
      uint32_t r[16];
      if (T > 0) {                                              // uniform over the CTA: every lane takes part
        tmem_ld_32x32b_x16(dz_addr + c0, r);
        tmem_wait_ld();
      } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) r[e] = __float_as_uint(v[c0 + e]);
      }
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const uint4 z = live ? zp[c0 / 8 + half] : make_uint4(0, 0, 0, 0);
        const float* f = reinterpret_cast<const float*>(r) + 8 * half;
        dsum = fmaf(f[0], bf16_lo(z.x), dsum); dsum = fmaf(f[1], bf16_hi(z.x), dsum);
        dsum = fmaf(f[2], bf16_lo(z.y), dsum); dsum = fmaf(f[3], bf16_hi(z.y), dsum);
        dsum = fmaf(f[4], bf16_lo(z.z), dsum); dsum = fmaf(f[5], bf16_hi(z.z), dsum);
        dsum = fmaf(f[6], bf16_lo(z.w), dsum); dsum = fmaf(f[7], bf16_hi(z.w), dsum);
        if (live && !w.dead)
          out[c0 / 8 + half] = make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]),
                                          pack_bf16(f[6], f[7]));
      }
    }
    if (live && !w.dead) ws_LD[((int64_t)bh * nq + grow) * 2 + 1] = dsum;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4) tmem_dealloc(tmem, C::kTmemCols);
}

// ====================================================================================================================
// dQ
// ====================================================================================================================
template <int D> struct QCfg {
  static constexpr int kDBoxes = D / 64;
  static constexpr int kStages = 3;
  static constexpr uint32_t kTileBoxBytes = kRows * 128;            // 128 rows x 64 columns
  static constexpr uint32_t kTileBytes = kDBoxes * kTileBoxBytes;   // Q tile, dZ tile
  static constexpr uint32_t kBoxBytes = kMC * 128;                  // one 64-column box of a K~ or V~ chunk
  static constexpr uint32_t kSlotBytes = kDBoxes * kBoxBytes;
  static constexpr uint32_t kOffQ = 0, kOffZ = kTileBytes, kOffRing = 2 * kTileBytes;   // ring: [stage][K~ slot | V~ slot]
  static constexpr uint32_t kOffBar = kOffRing + kStages * 2 * kSlotBytes;
  static constexpr uint32_t kSmemBytes = kOffBar + 256 + 1024 /*alignment slack*/;
  // TMEM columns: S[2] | dA[2] | dQ accumulator; dS_j (bf16) overlays the first half of S[j & 1]
  static constexpr uint32_t kColS = 0, kColA = 2 * kMC, kColQ = 4 * kMC, kTmemCols = 512;
  static_assert(4 * kMC + D <= 512, "TMEM budget");
};

struct QBars {
  uint64_t qz_full, full[3], empty[3], s_full[2], p_full[2], acc_done;
  uint32_t tmem_slot;
  int abort;
};

constexpr int kQThreads = 192;      // warps 0-3: one thread per query row; warp 4: TMA; warp 5: MMA issue

template <int D>
__global__ void __launch_bounds__(kQThreads, 1)
bwd_dq_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_z,
                    const __grid_constant__ CUtensorMap tmap_kv, __nv_bfloat16* __restrict__ dQ,
                    const float* __restrict__ ws_LD, int nq, int m, float scale, int* status) {
  using C = QCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  QBars* bars = reinterpret_cast<QBars*>(smem + C::kOffBar);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, row0 = blockIdx.x * kRows;
  const int nchunks = (m + kMC - 1) / kMC;
  Waiter w{status, &bars->abort};
  auto k_slot = [&](int s) { return smem + C::kOffRing + (2 * s) * C::kSlotBytes; };
  auto v_slot = [&](int s) { return smem + C::kOffRing + (2 * s + 1) * C::kSlotBytes; };

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_q);
    prefetch_tmap(&tmap_z);
    prefetch_tmap(&tmap_kv);
    mbar_init(&bars->qz_full, 1);
    for (int s = 0; s < C::kStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&bars->s_full[b], 1); mbar_init(&bars->p_full[b], kRows); }
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
      mbar_arrive_expect_tx(&bars->qz_full, 2 * C::kTileBytes);
      for (int gx = 0; gx < C::kDBoxes; ++gx) {
        tma_load_3d(smem + C::kOffQ + gx * C::kTileBoxBytes, &tmap_q, &bars->qz_full, gx * 64, row0, bh);
        tma_load_3d(smem + C::kOffZ + gx * C::kTileBoxBytes, &tmap_z, &bars->qz_full, gx * 64, row0, bh);
      }
      int issued = 0;
      for (int j = 0; j < nchunks && !w.dead; ++j) {
        const int s = j % C::kStages;
        if (j >= C::kStages) w.wait(&bars->empty[s], (j / C::kStages - 1) & 1, 701);
        if (w.dead) break;
        mbar_arrive_expect_tx(&bars->full[s], 2 * C::kSlotBytes);
        for (int gx = 0; gx < C::kDBoxes; ++gx) {
          tma_load_3d(k_slot(s) + gx * C::kBoxBytes, &tmap_kv, &bars->full[s], gx * 64, j * kMC, bh);
          tma_load_3d(v_slot(s) + gx * C::kBoxBytes, &tmap_kv, &bars->full[s], D + gx * 64, j * kMC, bh);
        }
        ++issued;
      }
      if (w.dead) {
        mbar_wait_drain(&bars->qz_full, 0);
        for (int i = issued > C::kStages ? issued - C::kStages : 0; i < issued; ++i)
          mbar_wait_drain(&bars->full[i % C::kStages], (i / C::kStages) & 1);
      }
    }
  } else if (warp == 5) {
    if (elect_one()) {
      constexpr uint32_t idesc_s = make_idesc_bf16(kRows, kMC, false, false);   // S, dA: both operands K-major
      constexpr uint32_t idesc_q = make_idesc_bf16(kRows, D, false, true);      // dQ += dS K~: K~ is MN-major
      auto kstep = [](int k, uint32_t box_bytes) { return (uint64_t)((k / 4) * (box_bytes >> 4) + (k % 4) * 2); };
      const uint64_t qd = make_smem_desc(smem_u32(smem + C::kOffQ), 16, 1024);
      const uint64_t zd = make_smem_desc(smem_u32(smem + C::kOffZ), 16, 1024);
      auto issue_sd = [&](int j) {
        const int s = j % C::kStages, b = j & 1;
        w.wait(&bars->full[s], (j / C::kStages) & 1, 711);
        tc_fence_after();
        const uint64_t kd = make_smem_desc(smem_u32(k_slot(s)), 16, 1024);
        const uint64_t vd = make_smem_desc(smem_u32(v_slot(s)), 16, 1024);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          mma_f16_ss(tmem + C::kColS + b * kMC, qd + kstep(k, C::kTileBoxBytes), kd + kstep(k, C::kBoxBytes), idesc_s, k != 0);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          mma_f16_ss(tmem + C::kColA + b * kMC, zd + kstep(k, C::kTileBoxBytes), vd + kstep(k, C::kBoxBytes), idesc_s, k != 0);
        mma_commit(&bars->s_full[b]);
      };
      w.wait(&bars->qz_full, 0, 710);
      issue_sd(0);
      for (int j = 0; j < nchunks; ++j) {
        // S_{j+1}, dA_{j+1} run while the threads work on chunk j; they overwrite the buffers dS_{j-1} was read from
        // by the dQ product of chunk j-1, which was issued earlier and therefore executes first
        if (j + 1 < nchunks) issue_sd(j + 1);
        const int s = j % C::kStages, b = j & 1;
        w.wait(&bars->p_full[b], (j >> 1) & 1, 712);
        tc_fence_after();
        const uint64_t kd = make_smem_desc(smem_u32(k_slot(s)), C::kBoxBytes, 1024);      // MN-major: rows = reduction
#pragma unroll
        for (int k = 0; k < kMC / 16; ++k)
          mma_f16_ts(tmem + C::kColQ, tmem + C::kColS + b * kMC + k * 8, kd + (uint64_t)(k * 128), idesc_q, (uint32_t)((j | k) != 0));
        mma_commit(&bars->empty[s]);
      }
      mma_commit(&bars->acc_done);
    }
  } else {
    const int row = warp * 32 + lane, grow = row0 + row;
    const bool live = grow < nq;
    const uint32_t tbase = tmem + ((uint32_t)(warp * 32) << 16);
    const float l2e = 1.4426950408889634f;
    const float L2 = live ? ws_LD[((int64_t)bh * nq + grow) * 2] * l2e : 0.f;
    const float Dv = live ? ws_LD[((int64_t)bh * nq + grow) * 2 + 1] : 0.f;
    const float scale_log2 = scale * l2e;
    for (int j = 0; j < nchunks; ++j) {
      const int b = j & 1;
      w.wait(&bars->s_full[b], (j >> 1) & 1, 720);
      tc_fence_after();
#pragma unroll
      for (int hlf = 0; hlf < 2; ++hlf) {
        uint32_t sv[32], av[32];
        tmem_ld_32x32b_x32(tbase + C::kColS + b * kMC + hlf * 32, sv);
        tmem_ld_32x32b_x32(tbase + C::kColA + b * kMC + hlf * 32, av);
        tmem_wait_ld();
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          const float p0 = ex2f(fmaf(__uint_as_float(sv[e]), scale_log2, -L2));
          const float p1 = ex2f(fmaf(__uint_as_float(sv[e + 1]), scale_log2, -L2));
          const float d0 = live ? scale * p0 * (__uint_as_float(av[e]) - Dv) : 0.f;
          const float d1 = live ? scale * p1 * (__uint_as_float(av[e + 1]) - Dv) : 0.f;
          pk[e >> 1] = pack_bf16(d0, d1);
        }
        // dS over the first 32 columns of S[b]: the first half's 16 packed columns are written after both of its
        // S columns groups ... the second half's S columns (32..63) are read before columns 16..31 are overwritten
        if (hlf == 0) {
          // columns 0..15 of S[b] hold scores this thread has already read (they are in sv)
          tmem_st_32x32b_x16(tbase + C::kColS + b * kMC, pk);
        } else {
          tmem_st_32x32b_x16(tbase + C::kColS + b * kMC + 16, pk);
        }
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bars->p_full[b]);
    }
    w.wait(&bars->acc_done, 0, 721);
    tc_fence_after();
    {
      // the tensor-memory loads are warp-wide (every lane takes part); only the stores depend on the row
      const bool store = live && !w.dead && *(volatile int*)&bars->abort == 0;
      uint4* o = reinterpret_cast<uint4*>(dQ + ((int64_t)bh * nq + (live ? grow : 0)) * D);
#pragma unroll
      for (int c0 = 0; c0 < D; c0 += 16) {
        uint32_t r[16];
        tmem_ld_32x32b_x16(tbase + C::kColQ + c0, r);
        tmem_wait_ld();
        const float* f = reinterpret_cast<const float*>(r);
        if (store) {
          o[c0 / 8] = make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
          o[c0 / 8 + 1] = make_uint4(pack_bf16(f[8], f[9]), pack_bf16(f[10], f[11]), pack_bf16(f[12], f[13]), pack_bf16(f[14], f[15]));
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, C::kTmemCols);
}

template <int D, bool kUntied>
cudaError_t launch_recur(csat_ctx* c, const void* G, cudaStream_t s) {
  using C = RCfg<D, kUntied>;
  const Params& p = c->p;
  static DeviceFlags smem_opt_in;
  cudaError_t e = ensure_dynamic_smem(bwd_recur_sm100_kernel<D, kUntied>, (int)C::kSmemBytes, c->device, smem_opt_in);
  if (e != cudaSuccess) return e;
  const dim3 grid((unsigned)((p.nq + kRows - 1) / kRows), (unsigned)(p.B * p.H));
  bwd_recur_sm100_kernel<D, kUntied><<<grid, kRThreads, C::kSmemBytes, s>>>(
      kUntied ? c->tmap_lmats : c->tmap_mats, c->bw_Z16, (const __nv_bfloat16*)G, c->bw_dZ16, c->bw_LD, c->bw_maskbits, (int)p.nq, (int)p.H, p.T,
      c->psi ? 1 : 0, c->status, c->weight_grads ? c->bw_dx16 : nullptr, (int64_t)(p.B * p.H * p.nq * p.d));
  return cudaGetLastError();
}

template <int D>
cudaError_t launch_dq(csat_ctx* c, const void* Q, void* dQ, cudaStream_t s) {
  using C = QCfg<D>;
  const Params& p = c->p;
  CUtensorMap tq, tz;
  const uint64_t qd[3] = {(uint64_t)D, (uint64_t)p.nq, (uint64_t)(p.B * p.H)};
  const uint64_t qs[2] = {(uint64_t)D * 2, (uint64_t)p.nq * D * 2};
  const uint32_t qb[3] = {64, (uint32_t)kRows, 1};
  cudaError_t e;
  if ((e = make_tmap_bf16_3d(&tq, Q, qd, qs, qb)) != cudaSuccess) return e;
  if ((e = make_tmap_bf16_3d(&tz, c->bw_dZ16, qd, qs, qb)) != cudaSuccess) return e;
  static DeviceFlags smem_opt_in;
  if ((e = ensure_dynamic_smem(bwd_dq_sm100_kernel<D>, (int)C::kSmemBytes, c->device, smem_opt_in)) != cudaSuccess) return e;
  const float scale = (float)(p.scale > 0.0 ? p.scale : 1.0 / sqrt((double)D));
  const dim3 grid((unsigned)((p.nq + kRows - 1) / kRows), (unsigned)(p.B * p.H));
  bwd_dq_sm100_kernel<D><<<grid, kQThreads, C::kSmemBytes, s>>>(tq, tz, c->tmap_kv, (__nv_bfloat16*)dQ, c->bw_LD, (int)p.nq,
                                                              (int)p.m, scale, c->status);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_sm100_bwd_recur(csat_ctx* c, const void* G, cudaStream_t s, int* launches) {
  *launches += 1;
  if (c->w_S && c->w_untied && c->p.T > 0)
    return c->p.d == 64 ? launch_recur<64, true>(c, G, s) : launch_recur<128, true>(c, G, s);
  return c->p.d == 64 ? launch_recur<64, false>(c, G, s) : launch_recur<128, false>(c, G, s);
}

cudaError_t launch_sm100_bwd_dq(csat_ctx* c, const void* Q, void* dQ, cudaStream_t s, int* launches) {
  *launches += 1;
  return c->p.d == 64 ? launch_dq<64>(c, Q, dQ, s) : launch_dq<128>(c, Q, dQ, s);
}

}  // namespace csat
