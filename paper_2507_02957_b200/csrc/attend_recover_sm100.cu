// Compressed attention and sparse recovery for one tile of 128 queries, on the sm_100a tensor cores.
//
// Paper, in order: A~ = softmax(Q K~^T / sqrt(d_k)) over the m measurements; Z = A~ V~;
// alpha^{t+1} = eta_theta(S alpha^t + B Z_i) (LISTA recurrence with S = I - mu G, B = mu M); C^_i = Psi alpha^_i.
// Neither the 128 x m block of A~ nor any iterate alpha^t leaves the SM.
//
// Two CTAs are resident per SM (<= 96 registers, ~100 KB shared memory, 256 tensor-memory columns each), so
// that one tile's MMAs run while the other tile's threads do the softmax / shrinkage arithmetic.
//
// CTA = 9 warps:
//   warps 0-7 (256 threads): two threads per query row (TMEM lane = row; warps w and w+4 share the lane
//             quarter w and split the columns).  Softmax statistics, exp2, P -> bf16 -> tensor memory,
//             Z accumulation in fp32 registers, soft-threshold, output.
//   warp 8  : allocates tensor memory; one elected thread issues every TMA copy and every tcgen05.mma.
//
// Attention phase, per chunk j of 64 measurements:
//   S_j = Q K~_j^T            (SS MMA, accumulator S[j&1] in tensor memory)
//   threads read S_j, update the running row maximum, write P_j = exp2(S_j - max) as packed bf16 over the
//   first half of S[j&1]'s columns
//   Zc_j = P_j V~_j           (TS MMA: A operand from tensor memory, fresh accumulator)
//   threads fold it in: z = z * corr_j + Zc_j.
// MMAs of one CTA execute in issue order (S_0, S_1, PV_0, S_2, PV_1, ...), so S_{j+2} overwrites S[j&1] only
// after PV_j has read P_j from it.
//
// Recovery phase.  The accumulator holds r_t = c - a^_t (mu G), where c = z B and a^_t is the sum of the bf16
// increments fed to the tensor cores so far:
//   r_0 = z_bf16 B (one MMA);  alpha^{t+1} = eta_theta(alpha^t + r_t);
//   r_{t+1} = r_t + bf16(alpha^t - alpha^{t+1}) (mu G)     (one accumulating MMA per iteration).
// This is the paper's S alpha + B z with S = I - mu G: the identity part stays exact in fp32 registers, only
// the increment that multiplies mu G is rounded to bf16, and c never needs registers of its own.
#include "csat_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace csat {
namespace {

using namespace ptx;

constexpr int kRows = 128;            // queries per CTA
constexpr int kMC = 64;               // measurements per chunk
constexpr int kComputeThreads = 256;
constexpr int kThreads = 288;
constexpr int kMaxStages = 4;

template <int D> struct Cfg {
  static constexpr int kDBoxes = D / 64;                          // 64-column boxes across the head dimension
  static constexpr int kStages = (D == 64) ? 4 : 2;               // K~ / V~ chunks in flight
  static constexpr uint32_t kQBytes = kDBoxes * kRows * 128;      // Q tile; later the matrix B
  static constexpr uint32_t kBoxBytes = kMC * 128;                // one 64-column box of a K~ or V~ chunk
  static constexpr uint32_t kSlotBytes = kDBoxes * kBoxBytes;     // K~ chunk (= V~ chunk)
  static constexpr uint32_t kMatBoxBytes = D * 128;               // one 64-column box of a d x d bf16 matrix
  static constexpr uint32_t kMatBytes = kDBoxes * kMatBoxBytes;
  static constexpr uint32_t kOffQ = 0;
  static constexpr uint32_t kOffRing = kOffQ + kQBytes;           // [stage][K~ slot | V~ slot]
  static constexpr uint32_t kOffBar = kOffRing + kStages * 2 * kSlotBytes;
  static constexpr uint32_t kBarBytes = 256 + 2048;               // barriers | row-maximum exchange
  static constexpr uint32_t kSmemBytes = kOffBar + kBarBytes;     // base must be 1024-byte aligned (checked)
  // TMEM columns: S[0] | S[1] | accumulator (Zc, then r_t).  P_j overlays S[j&1]; the recovery operand S[0].
  static constexpr uint32_t kColS = 0, kColAcc = 2 * kMC, kTmemCols = 256;
  static_assert(2 * kMC + D <= 256, "TMEM budget");
  static_assert(D / 2 <= 2 * kMC, "recovery operand fits in the S columns");
  static_assert(kStages >= kDBoxes && kStages <= kMaxStages, "mu G and Psi are staged box by box in ring slots");
  static_assert(kMatBoxBytes <= kSlotBytes && kMatBytes <= kQBytes, "decoder matrices fit where they are staged");
  static_assert(2 * (kSmemBytes + 1024) <= 228 * 1024, "two CTAs per SM");
};

struct Bars {
  uint64_t q_full, mats_full, psi_full;
  uint64_t k_full[kMaxStages], k_empty[kMaxStages], v_full[kMaxStages], v_empty[kMaxStages];
  uint64_t s_full[2], p_full[2], zc_full, zc_empty;
  uint64_t a_full, r_full;
  uint32_t tmem_slot;
  int abort;
};
static_assert(sizeof(Bars) <= 256, "barrier block");

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}
// warps q and q+4 (the two halves of the same 32 rows) meet here
__device__ __forceinline__ void pair_barrier(int q) { asm volatile("bar.sync %0, 64;" ::"r"(q + 1) : "memory"); }

// A wait that never blocks for more than the time-out and turns into a no-op once anything gave up.
struct Waiter {
  int* status;
  int* cta_abort;
  bool dead = false;
  __device__ __forceinline__ void wait(uint64_t* bar, uint32_t parity, int code) {
    if (dead) return;
    if (!mbar_wait(bar, parity, status, code, cta_abort)) dead = true;
  }
};

template <int D>
__global__ void __launch_bounds__(kThreads, 2)
attend_recover_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_kv,
                            const __grid_constant__ CUtensorMap tmap_mats, __nv_bfloat16* __restrict__ out,
                            const float* __restrict__ theta, int nq, int m, int H, int T, int has_psi,
                            float scale_log2, int* status) {
  using C = Cfg<D>;
  constexpr int HC = D / 2;                    // feature columns per thread
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {          // swizzled tiles need 1024-byte alignment; never seen to fail
    if (threadIdx.x == 0) atomicCAS(status, 0, 200);
    return;
  }
  uint8_t* q_buf = smem + C::kOffQ;
  uint8_t* ring = smem + C::kOffRing;
  Bars* bars = reinterpret_cast<Bars*>(smem + C::kOffBar);
  float* xch = reinterpret_cast<float*>(smem + C::kOffBar + 256);   // [2 buffers][2 halves][128 rows] floats
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qtile = blockIdx.x, bh = blockIdx.y, h = bh % H;
  const int nchunks = (m + kMC - 1) / kMC;
  Waiter w{status, &bars->abort};
  auto k_slot = [&](int s) { return ring + (2 * s) * C::kSlotBytes; };
  auto v_slot = [&](int s) { return ring + (2 * s + 1) * C::kSlotBytes; };

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_q);
    prefetch_tmap(&tmap_kv);
    prefetch_tmap(&tmap_mats);
    mbar_init(&bars->q_full, 1);
    mbar_init(&bars->mats_full, 1);
    mbar_init(&bars->psi_full, 1);
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&bars->k_full[s], 1); mbar_init(&bars->k_empty[s], 1);
      mbar_init(&bars->v_full[s], 1); mbar_init(&bars->v_empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) { mbar_init(&bars->s_full[s], 1); mbar_init(&bars->p_full[s], kComputeThreads); }
    mbar_init(&bars->zc_full, 1);
    mbar_init(&bars->zc_empty, kComputeThreads);
    mbar_init(&bars->a_full, kComputeThreads);
    mbar_init(&bars->r_full, 1);
    bars->abort = 0;
    fence_mbar_init();
  }
  if (warp == 8) {
    tmem_alloc(&bars->tmem_slot, C::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_slot;

  if (warp == 8) {
    // ------------------------------------ TMA copies and MMA issue (one thread) -----------------------------------
    if (elect_one()) {
      constexpr uint32_t idesc_s = make_idesc_bf16(kRows, kMC, false, false);   // S  = Q  K~^T : both K-major
      constexpr uint32_t idesc_z = make_idesc_bf16(kRows, D, false, true);      // Zc = P  V~   : V~ is MN-major
      constexpr uint32_t idesc_r = make_idesc_bf16(kRows, D, false, false);     // r  = a  W^T  : both K-major
      int next_k = 0, next_v = 0;           // next chunk whose K~ / V~ copy has not been issued
      int seen_k = 0, seen_v = 0;           // chunks whose copy this thread has waited for
      bool q_issued = false, mats_issued = false, psi_issued = false, mats_seen = false, psi_seen = false;

      auto issue_k = [&](int c) {
        const int s = c % C::kStages;
        mbar_arrive_expect_tx(&bars->k_full[s], C::kSlotBytes);
        for (int g = 0; g < C::kDBoxes; ++g)
          tma_load_3d(k_slot(s) + g * C::kBoxBytes, &tmap_kv, &bars->k_full[s], g * 64, c * kMC, bh);
      };
      auto issue_v = [&](int c) {
        const int s = c % C::kStages;
        mbar_arrive_expect_tx(&bars->v_full[s], C::kSlotBytes);
        for (int g = 0; g < C::kDBoxes; ++g)
          tma_load_3d(v_slot(s) + g * C::kBoxBytes, &tmap_kv, &bars->v_full[s], D + g * 64, c * kMC, bh);
      };
      // issues every copy whose slot is free right now; never blocks
      auto service = [&]() {
        while (next_k < nchunks) {
          const int s = next_k % C::kStages, use = next_k / C::kStages;
          if (use > 0 && !mbar_try_wait(&bars->k_empty[s], (use - 1) & 1)) break;
          issue_k(next_k++);
        }
        while (next_v < nchunks) {
          const int s = next_v % C::kStages, use = next_v / C::kStages;
          if (use > 0 && !mbar_try_wait(&bars->v_empty[s], (use - 1) & 1)) break;
          issue_v(next_v++);
        }
      };
      // bounded wait that keeps the copies flowing while it spins
      auto wait_serving = [&](uint64_t* bar, uint32_t parity, int code) {
        if (w.dead) return;
        if (mbar_try_wait(bar, parity)) return;
        const unsigned long long t0 = globaltimer();
        uint32_t spins = 0;
        while (!mbar_try_wait(bar, parity)) {
          service();
          if ((++spins & 0xff) == 0) {
            if (*(volatile int*)&bars->abort != 0) { w.dead = true; return; }
            if (globaltimer() - t0 > kWaitTimeoutNs) {
              *(volatile int*)&bars->abort = 1;
              atomicCAS(status, 0, code);
              w.dead = true;
              return;
            }
          }
        }
      };
      // the copies of chunk c must have been issued before their barrier is waited for
      auto ensure_k = [&](int c) {
        while (next_k <= c && !w.dead) {
          const int s = next_k % C::kStages, use = next_k / C::kStages;
          if (use > 0) w.wait(&bars->k_empty[s], (use - 1) & 1, 201);
          if (!w.dead) issue_k(next_k++);
        }
      };
      auto ensure_v = [&](int c) {
        while (next_v <= c && !w.dead) {
          const int s = next_v % C::kStages, use = next_v / C::kStages;
          if (use > 0) w.wait(&bars->v_empty[s], (use - 1) & 1, 202);
          if (!w.dead) issue_v(next_v++);
        }
      };
      auto issue_pv = [&](int i) {
        const int s = i % C::kStages, b = i & 1;
        ensure_v(i);
        wait_serving(&bars->v_full[s], (i / C::kStages) & 1, 211);
        if (!w.dead) seen_v = i + 1;
        wait_serving(&bars->p_full[b], (i >> 1) & 1, 212);
        if (i > 0) wait_serving(&bars->zc_empty, (i - 1) & 1, 213);   // Zc_{i-1} has been folded
        tc_fence_after();
        const uint64_t b_desc = make_smem_desc(smem_u32(v_slot(s)), C::kBoxBytes, 1024);
#pragma unroll
        for (int k = 0; k < kMC / 16; ++k)     // P: 8 packed columns per 16 measurements; V~: +16 rows = 2048 B
          mma_f16_ts(tmem + C::kColAcc, tmem + C::kColS + b * kMC + k * 8, b_desc + (uint64_t)(k * 128), idesc_z, k != 0);
        mma_commit(&bars->zc_full);
        mma_commit(&bars->v_empty[s]);
      };

      mbar_arrive_expect_tx(&bars->q_full, C::kQBytes);
      for (int g = 0; g < C::kDBoxes; ++g)
        tma_load_3d(q_buf + g * kRows * 128, &tmap_q, &bars->q_full, g * 64, qtile * kRows, bh);
      q_issued = true;
      service();
      w.wait(&bars->q_full, 0, 210);
      for (int j = 0; j < nchunks; ++j) {
        const int s = j % C::kStages, b = j & 1;
        ensure_k(j);
        wait_serving(&bars->k_full[s], (j / C::kStages) & 1, 214);
        if (!w.dead) seen_k = j + 1;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t a_desc = make_smem_desc(smem_u32(q_buf + (k / 4) * kRows * 128), 16, 1024) + (uint64_t)((k % 4) * 2);
          const uint64_t b_desc = make_smem_desc(smem_u32(k_slot(s) + (k / 4) * C::kBoxBytes), 16, 1024) + (uint64_t)((k % 4) * 2);
          mma_f16_ss(tmem + C::kColS + b * kMC, a_desc, b_desc, idesc_s, k != 0);
        }
        mma_commit(&bars->s_full[b]);
        mma_commit(&bars->k_empty[s]);
        if (j > 0) issue_pv(j - 1);
        service();
      }
      if (T > 0) {
        // every S MMA has finished once the last one has: Q and the K~ slots are free for mu G and B
        const int last = nchunks - 1;
        wait_serving(&bars->k_empty[last % C::kStages], (last / C::kStages) & 1, 215);
        if (!w.dead) {
          mbar_arrive_expect_tx(&bars->mats_full, 2 * C::kMatBytes);
          for (int g = 0; g < C::kDBoxes; ++g) {
            tma_load_3d(k_slot(g), &tmap_mats, &bars->mats_full, g * 64, 0, h * 3 + 0);                          // mu G
            tma_load_3d(q_buf + g * C::kMatBoxBytes, &tmap_mats, &bars->mats_full, g * 64, 0, h * 3 + 1);       // B
          }
          mats_issued = true;
        }
      }
      issue_pv(nchunks - 1);
      if (T > 0) {
        if (has_psi) {
          // Psi goes to the V~ slots once the last P V~ product has read them
          const int last = nchunks - 1;
          w.wait(&bars->v_empty[last % C::kStages], (last / C::kStages) & 1, 216);
          if (!w.dead) {
            mbar_arrive_expect_tx(&bars->psi_full, C::kMatBytes);
            for (int g = 0; g < C::kDBoxes; ++g)
              tma_load_3d(v_slot(g), &tmap_mats, &bars->psi_full, g * 64, 0, h * 3 + 2);
            psi_issued = true;
          }
        }
        const int n_mma = T + (has_psi ? 1 : 0);            // r_0 = z B, then T-1 increments with mu G, then Psi
        for (int i = 0; i < n_mma; ++i) {
          const bool first = (i == 0), psi_step = has_psi && i == n_mma - 1;
          if (first) { w.wait(&bars->mats_full, 0, 217); if (!w.dead) mats_seen = true; }
          if (psi_step) { w.wait(&bars->psi_full, 0, 218); if (!w.dead) psi_seen = true; }
          w.wait(&bars->a_full, i & 1, 219);
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const uint8_t* box = first ? q_buf + (k / 4) * C::kMatBoxBytes : (psi_step ? v_slot(k / 4) : k_slot(k / 4));
            const uint64_t b_desc = make_smem_desc(smem_u32(box), 16, 1024) + (uint64_t)((k % 4) * 2);
            mma_f16_ts(tmem + C::kColAcc, tmem + C::kColS + k * 8, b_desc, idesc_r, (first || psi_step) ? (k != 0) : 1u);
          }
          mma_commit(&bars->r_full);
        }
      }
      if (w.dead) {
        // gave up: let the copies that are still in flight land before the CTA's shared memory goes away
        if (q_issued) mbar_wait_drain(&bars->q_full, 0);
        for (int c = seen_k; c < next_k; ++c) mbar_wait_drain(&bars->k_full[c % C::kStages], (c / C::kStages) & 1);
        for (int c = seen_v; c < next_v; ++c) mbar_wait_drain(&bars->v_full[c % C::kStages], (c / C::kStages) & 1);
        if (mats_issued && !mats_seen) mbar_wait_drain(&bars->mats_full, 0);
        if (psi_issued && !psi_seen) mbar_wait_drain(&bars->psi_full, 0);
      }
    }
  } else {
    // ------------------------------------------------ compute threads ---------------------------------------------
    const int q = warp & 3, half = warp >> 2;
    const int row = q * 32 + lane;                              // row of the tile = TMEM lane
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    float z[HC];
#pragma unroll
    for (int i = 0; i < HC; ++i) z[i] = 0.f;
    float run_max = -INFINITY, run_sum = 0.f, corr_prev = 0.f;

    auto fold_zc = [&](int i, float corr) {
      w.wait(&bars->zc_full, i & 1, 221);
      tc_fence_after();
#pragma unroll
      for (int c0 = 0; c0 < HC; c0 += 16) {
        uint32_t r[16];
        tmem_ld_32x32b_x16(tmem + lane_addr + C::kColAcc + half * HC + c0, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 16; ++e) z[c0 + e] = fmaf(z[c0 + e], corr, __uint_as_float(r[e]));
      }
      tc_fence_before();
      mbar_arrive(&bars->zc_empty);
    };

    for (int j = 0; j < nchunks; ++j) {
      const int b = j & 1;
      w.wait(&bars->s_full[b], (j >> 1) & 1, 220);
      tc_fence_after();
      uint32_t r[32];
      tmem_ld_32x32b_x32(tmem + lane_addr + C::kColS + b * kMC + half * 32, r);
      tmem_wait_ld();
      // scores in the log2 domain; measurements beyond m are masked out
      float mx = -INFINITY;
      const int col0 = j * kMC + half * 32;
      if (col0 + 32 <= m) {
#pragma unroll
        for (int e = 0; e < 32; ++e) mx = fmaxf(mx, __uint_as_float(r[e]));
      } else {
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          if (col0 + e >= m) r[e] = 0xff800000u;                // -inf
          mx = fmaxf(mx, __uint_as_float(r[e]));
        }
      }
      mx *= scale_log2;                                         // scale > 0: the maximum commutes with it
      float* slot = xch + b * 256;
      slot[half * 128 + row] = mx;
      pair_barrier(q);              // also orders this thread's S read before its partner's P write below
      mx = fmaxf(mx, slot[(half ^ 1) * 128 + row]);
      const float new_max = fmaxf(run_max, mx);                 // finite: chunk 0 has a valid measurement
      const float corr = ex2(run_max - new_max);
      run_max = new_max;
      float sum = 0.f;
      uint32_t pk[16];
#pragma unroll
      for (int e = 0; e < 32; e += 2) {
        const float p0 = ex2(fmaf(__uint_as_float(r[e]), scale_log2, -new_max));
        const float p1 = ex2(fmaf(__uint_as_float(r[e + 1]), scale_log2, -new_max));
        sum += p0 + p1;
        pk[e >> 1] = pack_bf16(p0, p1);
      }
      run_sum = fmaf(run_sum, corr, sum);
      // P_j over the first 32 columns of S[b]: this half's 32 measurements are packed columns [16 half, +16)
      tmem_st_32x32b_x16(tmem + lane_addr + C::kColS + b * kMC + half * 16, pk);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bars->p_full[b]);
      if (j > 0) fold_zc(j - 1, corr_prev);
      corr_prev = corr;
    }
    fold_zc(nchunks - 1, corr_prev);
    // the two halves of a row share max and corr; their partial sums are added once
    float* slot = xch + (nchunks & 1) * 256;   // the buffer the last chunk did not use
    slot[half * 128 + row] = run_sum;
    pair_barrier(q);
    const float inv = 1.f / (run_sum + slot[(half ^ 1) * 128 + row]);
#pragma unroll
    for (int i = 0; i < HC; ++i) z[i] *= inv;

    if (T > 0) {
      const float th = theta[h];
      const uint32_t op_addr = tmem + lane_addr + C::kColS + half * (HC / 2);   // this thread's operand columns
      // z as the bf16 A operand of r_0 = z B
#pragma unroll
      for (int c0 = 0; c0 < HC; c0 += 32) {
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 32; e += 2) pk[e >> 1] = pack_bf16(z[c0 + e], z[c0 + e + 1]);
        tmem_st_32x32b_x16(op_addr + c0 / 2, pk);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bars->a_full);
#pragma unroll
      for (int i = 0; i < HC; ++i) z[i] = 0.f;                  // z now holds alpha (alpha^0 = 0)
      int phase = 0;
      for (int it = 0; it < T; ++it) {
        w.wait(&bars->r_full, phase & 1, 230); ++phase;
        tc_fence_after();
        const bool more = it + 1 < T;
#pragma unroll
        for (int c0 = 0; c0 < HC; c0 += 16) {
          uint32_t r[16];
          tmem_ld_32x32b_x16(tmem + lane_addr + C::kColAcc + half * HC + c0, r);
          tmem_wait_ld();
          uint32_t pk[8];
#pragma unroll
          for (int e = 0; e < 16; e += 2) {
            float nd[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              const float rv = __uint_as_float(r[e + u]);
              const float x = z[c0 + e + u] + rv;               // alpha^t S + z B, identity part in fp32
              const float cl = fminf(fmaxf(x, -th), th);
              z[c0 + e + u] = x - cl;                           // eta_theta(x)
              nd[u] = cl - rv;                                  // alpha^t - alpha^{t+1}
            }
            pk[e >> 1] = pack_bf16(nd[0], nd[1]);
          }
          if (more) tmem_st_32x32b_x8(op_addr + c0 / 2, pk);
        }
        if (more) {
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(&bars->a_full);
        }
      }
      if (has_psi) {
#pragma unroll
        for (int c0 = 0; c0 < HC; c0 += 32) {
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 32; e += 2) pk[e >> 1] = pack_bf16(z[c0 + e], z[c0 + e + 1]);
          tmem_st_32x32b_x16(op_addr + c0 / 2, pk);
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bars->a_full);
        w.wait(&bars->r_full, phase & 1, 232); ++phase;
        tc_fence_after();
#pragma unroll
        for (int c0 = 0; c0 < HC; c0 += 32) {
          uint32_t r[32];
          tmem_ld_32x32b_x32(tmem + lane_addr + C::kColAcc + half * HC + c0, r);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) z[c0 + e] = __uint_as_float(r[e]);
        }
      }
    }
    const int grow = qtile * kRows + row;
    if (grow < nq && !w.dead && *(volatile int*)&bars->abort == 0) {
      uint4* o = reinterpret_cast<uint4*>(out + ((int64_t)bh * nq + grow) * D + half * HC);
#pragma unroll
      for (int c = 0; c < HC / 8; ++c)
        o[c] = make_uint4(pack_bf16(z[c * 8], z[c * 8 + 1]), pack_bf16(z[c * 8 + 2], z[c * 8 + 3]),
                          pack_bf16(z[c * 8 + 4], z[c * 8 + 5]), pack_bf16(z[c * 8 + 6], z[c * 8 + 7]));
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 8) tmem_dealloc(tmem, C::kTmemCols);
}

template <int D>
cudaError_t launch(csat_ctx* c, const void* Q, void* out, cudaStream_t s) {
  using C = Cfg<D>;
  const Params& p = c->p;
  CUtensorMap tq;
  const uint64_t qd[3] = {(uint64_t)D, (uint64_t)p.nq, (uint64_t)(p.B * p.H)};
  const uint64_t qs[2] = {(uint64_t)D * 2, (uint64_t)p.nq * D * 2};
  const uint32_t qb[3] = {64, (uint32_t)kRows, 1};
  cudaError_t e;
  if ((e = make_tmap_bf16_3d(&tq, Q, qd, qs, qb)) != cudaSuccess) return e;
  static bool attr_set = false;
  if (!attr_set) {
    e = cudaFuncSetAttribute(attend_recover_sm100_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)C::kSmemBytes);
    if (e != cudaSuccess) return e;
    // two CTAs per SM need the large shared-memory carve-out
    e = cudaFuncSetAttribute(attend_recover_sm100_kernel<D>, cudaFuncAttributePreferredSharedMemoryCarveout,
                             (int)cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const double scale = p.scale > 0.0 ? p.scale : 1.0 / sqrt((double)D);
  const float scale_log2 = (float)(scale * 1.4426950408889634);
  const dim3 grid((unsigned)((p.nq + kRows - 1) / kRows), (unsigned)(p.B * p.H));
  attend_recover_sm100_kernel<D><<<grid, kThreads, C::kSmemBytes, s>>>(
      tq, c->tmap_kv, c->tmap_mats, (__nv_bfloat16*)out, c->theta, (int)p.nq, (int)p.m, (int)p.H, p.T,
      c->psi ? 1 : 0, scale_log2, c->status);
  return cudaGetLastError();
}

}  // namespace

// tensor maps over library-owned buffers: the K~|V~ workspace and the bf16 decoder matrices
cudaError_t make_attend_tmaps(csat_ctx* c) {
  const Params& p = c->p;
  const uint64_t kd[3] = {(uint64_t)(2 * p.d), (uint64_t)p.m, (uint64_t)(p.B * p.H)};
  const uint64_t ks[2] = {(uint64_t)(2 * p.d) * 2, (uint64_t)p.m * 2 * p.d * 2};
  const uint32_t kb[3] = {64, (uint32_t)kMC, 1};
  cudaError_t e = make_tmap_bf16_3d(&c->tmap_kv, c->kv, kd, ks, kb);
  if (e != cudaSuccess) return e;
  const uint64_t md[3] = {(uint64_t)p.d, (uint64_t)p.d, (uint64_t)(p.H * 3)};
  const uint64_t ms[2] = {(uint64_t)p.d * 2, (uint64_t)p.d * p.d * 2};
  const uint32_t mb[3] = {64, (uint32_t)p.d, 1};
  return make_tmap_bf16_3d(&c->tmap_mats, c->mats_bf16, md, ms, mb);
}

cudaError_t launch_sm100_attend_recover(csat_ctx* c, const void* Q, void* out, cudaStream_t s, int* launches) {
  *launches += 1;
  return c->p.d == 64 ? launch<64>(c, Q, out, s) : launch<128>(c, Q, out, s);
}

}  // namespace csat
