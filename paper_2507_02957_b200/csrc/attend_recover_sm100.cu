// Compressed attention and sparse recovery for one tile of 128 queries, on the sm_100a tensor cores.
//
// Paper, in order: A~ = softmax(Q K~^T / sqrt(d_k)) over the m measurements; Z = A~ V~;
// alpha^{t+1} = eta_theta(S alpha^t + B Z_i) (LISTA recurrence with S = I - mu G, B = mu M); C^_i = Psi alpha^_i.
// Neither the 128 x m block of A~ nor any iterate alpha^t leaves the SM.
//
// CTA = 10 warps:
//   warps 0-7 (256 threads): two threads per query row (TMEM lane = row; warps w and w+4 share the lane
//             quarter w and split the columns).  Softmax statistics, exp2, P -> bf16 -> shared memory,
//             Z accumulation in fp32 registers, soft-threshold, output.
//   warp 8  : TMA producer (Q tile, K~|V~ chunks of kMC measurements, decoder matrices).
//   warp 9  : TMEM allocation; one elected thread issues every tcgen05.mma.
// Attention phase, per chunk j of measurements:  S_j = Q K~_j^T (TMEM, double buffered) -> threads read
// S_j, update the running row maximum, write P_j = exp2(S_j - max) as the bf16 A operand ->
// Zc_j = P_j V~_j (TMEM, fresh accumulator) -> threads fold it in: z = z * corr_j + Zc_j.
// Recovery phase: c = z B (one MMA), alpha^1 = eta(c); then T-1 times R = alpha_bf16 (mu G),
// alpha <- eta(alpha - R + c); alpha and c stay in fp32 registers, only the MMA operand copy is bf16.
#include "csat_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace csat {
namespace {

using namespace ptx;

constexpr int kRows = 128;            // queries per CTA
constexpr int kMC = 64;               // measurements per chunk
constexpr int kComputeThreads = 256;
constexpr int kThreads = 320;
constexpr int kKvStages = 3;

template <int D> struct Cfg {
  static constexpr int kDBoxes = D / 64;                          // 64-column boxes across the head dimension
  static constexpr uint32_t kABytes = kDBoxes * kRows * 128;      // Q tile / bf16 operand copy of z, alpha
  static constexpr uint32_t kKHalf = kDBoxes * kMC * 128;         // K~ chunk (= V~ chunk)
  static constexpr uint32_t kStageBytes = 2 * kKHalf;
  static constexpr uint32_t kPBytes = kRows * 128;                // P chunk: 128 x 64 bf16
  static constexpr uint32_t kMatBytes = kDBoxes * D * 128;        // one d x d bf16 matrix
  static constexpr uint32_t kOffA = 0;
  static constexpr uint32_t kOffKv = kOffA + kABytes;
  static constexpr uint32_t kOffP = kOffKv + kKvStages * kStageBytes;
  static constexpr uint32_t kOffG = kOffP + 2 * kPBytes;
  static constexpr uint32_t kOffB = kOffG + kMatBytes;
  static constexpr uint32_t kOffBar = kOffB + kMatBytes;
  static constexpr uint32_t kBarBytes = 256 + 2048;               // barriers | row statistics exchange
  static constexpr uint32_t kSmemBytes = kOffBar + kBarBytes;     // base must be 1024-byte aligned (checked)
  // TMEM columns: S[2] | Zc[2]; the recovery accumulator R reuses Zc[0]
  static constexpr uint32_t kColS = 0, kColZ = 2 * kMC, kTmemCols = (2 * kMC + 2 * D <= 256) ? 256 : 512;
  static_assert(2 * kMC + 2 * D <= 512, "TMEM budget");
  static_assert(kMatBytes <= kStageBytes, "Psi is staged in a K~|V~ buffer");
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
};

struct Bars {
  uint64_t q_full, mats_full, psi_full, attn_done;
  uint64_t kv_full[kKvStages], kv_empty[kKvStages];
  uint64_t s_full[2], s_empty[2], p_full[2], p_empty[2], zc_full[2], zc_empty[2];
  uint64_t a_full, r_full;
  uint32_t tmem_slot;
  int abort;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float soft(float x, float th) { return x - fminf(fmaxf(x, -th), th); }
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}
__device__ __forceinline__ void named_barrier_256() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

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

// writes 8 consecutive bf16 (one 16-byte chunk) of row r into a K-major 128-byte-swizzled box
__device__ __forceinline__ void st_chunk(uint8_t* box, int r, int chunk, const float* v) {
  uint4 w = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
  *reinterpret_cast<uint4*>(box + r * 128 + ((chunk ^ (r & 7)) << 4)) = w;
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
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
  uint8_t* a_buf = smem + C::kOffA;
  uint8_t* kv_buf = smem + C::kOffKv;
  uint8_t* p_buf = smem + C::kOffP;
  uint8_t* g_buf = smem + C::kOffG;
  uint8_t* b_buf = smem + C::kOffB;
  Bars* bars = reinterpret_cast<Bars*>(smem + C::kOffBar);
  float* xch = reinterpret_cast<float*>(smem + C::kOffBar + 256);   // [2 buffers][2 halves][128 rows] floats
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qtile = blockIdx.x, bh = blockIdx.y, h = bh % H;
  const int nchunks = (m + kMC - 1) / kMC;
  Waiter w{status, &bars->abort};

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_q);
    prefetch_tmap(&tmap_kv);
    prefetch_tmap(&tmap_mats);
    mbar_init(&bars->q_full, 1);
    mbar_init(&bars->mats_full, 1);
    mbar_init(&bars->psi_full, 1);
    mbar_init(&bars->attn_done, kComputeThreads);
    for (int s = 0; s < kKvStages; ++s) { mbar_init(&bars->kv_full[s], 1); mbar_init(&bars->kv_empty[s], 1); }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->s_full[s], 1);  mbar_init(&bars->s_empty[s], kComputeThreads);
      mbar_init(&bars->p_full[s], kComputeThreads);  mbar_init(&bars->p_empty[s], 1);
      mbar_init(&bars->zc_full[s], 1); mbar_init(&bars->zc_empty[s], kComputeThreads);
    }
    mbar_init(&bars->a_full, kComputeThreads);
    mbar_init(&bars->r_full, 1);
    bars->abort = 0;
    fence_mbar_init();
  }
  if (warp == 9) {
    tmem_alloc(&bars->tmem_slot, C::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_slot;

  if (warp == 8) {
    // ------------------------------------------------ TMA producer ------------------------------------------------
    if (elect_one()) {
      mbar_arrive_expect_tx(&bars->q_full, C::kABytes);
      for (int g = 0; g < C::kDBoxes; ++g)
        tma_load_3d(a_buf + g * kRows * 128, &tmap_q, &bars->q_full, g * 64, qtile * kRows, bh);
      if (T > 0) {
        mbar_arrive_expect_tx(&bars->mats_full, 2 * C::kMatBytes);
        for (int g = 0; g < C::kDBoxes; ++g) {
          tma_load_3d(g_buf + g * D * 128, &tmap_mats, &bars->mats_full, g * 64, 0, h * 3 + 0);
          tma_load_3d(b_buf + g * D * 128, &tmap_mats, &bars->mats_full, g * 64, 0, h * 3 + 1);
        }
      }
      for (int j = 0; j < nchunks; ++j) {
        const int s = j % kKvStages;
        w.wait(&bars->kv_empty[s], ((j / kKvStages) & 1) ^ 1, 201);
        if (w.dead) break;
        uint8_t* st = kv_buf + s * C::kStageBytes;
        mbar_arrive_expect_tx(&bars->kv_full[s], C::kStageBytes);
        for (int g = 0; g < C::kDBoxes; ++g) {
          tma_load_3d(st + g * kMC * 128, &tmap_kv, &bars->kv_full[s], g * 64, j * kMC, bh);                  // K~
          tma_load_3d(st + C::kKHalf + g * kMC * 128, &tmap_kv, &bars->kv_full[s], D + g * 64, j * kMC, bh);  // V~
        }
      }
      if (T > 0 && has_psi) {
        // Psi is staged in K~|V~ buffer 0 once the attention phase no longer needs it
        w.wait(&bars->attn_done, 0, 202);
        if (!w.dead) {
          mbar_arrive_expect_tx(&bars->psi_full, C::kMatBytes);
          for (int g = 0; g < C::kDBoxes; ++g)
            tma_load_3d(kv_buf + g * D * 128, &tmap_mats, &bars->psi_full, g * 64, 0, h * 3 + 2);
        }
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------ MMA issuer --------------------------------------------------
    if (elect_one()) {
      constexpr uint32_t idesc_s = make_idesc_bf16(kRows, kMC, false, false);   // S  = Q  K~^T : both K-major
      constexpr uint32_t idesc_z = make_idesc_bf16(kRows, D, false, true);      // Zc = P  V~   : V~ is MN-major
      constexpr uint32_t idesc_r = make_idesc_bf16(kRows, D, false, false);     // R  = a  W^T  : both K-major
      auto issue_pv = [&](int i) {
        const int s = i % kKvStages, b = i & 1;
        w.wait(&bars->p_full[b], (i >> 1) & 1, 211);
        w.wait(&bars->zc_empty[b], ((i >> 1) & 1) ^ 1, 212);
        tc_fence_after();
        const uint64_t a_desc = make_smem_desc(smem_u32(p_buf + b * C::kPBytes), 16, 1024);
        const uint64_t b_desc = make_smem_desc(smem_u32(kv_buf + s * C::kStageBytes + C::kKHalf), kMC * 128, 1024);
#pragma unroll
        for (int k = 0; k < kMC / 16; ++k)
          mma_f16_ss(tmem + C::kColZ + b * D, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)(k * 128), idesc_z, k != 0);
        mma_commit(&bars->zc_full[b]);
        mma_commit(&bars->kv_empty[s]);
        mma_commit(&bars->p_empty[b]);
      };
      w.wait(&bars->q_full, 0, 210);
      for (int j = 0; j < nchunks; ++j) {
        const int s = j % kKvStages, b = j & 1;
        w.wait(&bars->kv_full[s], (j / kKvStages) & 1, 213);
        w.wait(&bars->s_empty[b], ((j >> 1) & 1) ^ 1, 214);
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t a_desc = make_smem_desc(smem_u32(a_buf + (k / 4) * kRows * 128), 16, 1024) + (uint64_t)((k % 4) * 2);
          const uint64_t b_desc =
              make_smem_desc(smem_u32(kv_buf + s * C::kStageBytes + (k / 4) * kMC * 128), 16, 1024) + (uint64_t)((k % 4) * 2);
          mma_f16_ss(tmem + C::kColS + b * kMC, a_desc, b_desc, idesc_s, k != 0);
        }
        mma_commit(&bars->s_full[b]);
        if (j > 0) issue_pv(j - 1);
      }
      issue_pv(nchunks - 1);
      if (T > 0) {
        w.wait(&bars->mats_full, 0, 215);
        const int n_mma = T + (has_psi ? 1 : 0);            // c = zB, then T-1 products with mu G, then Psi
        for (int i = 0; i < n_mma; ++i) {
          const uint8_t* wsm = (i == 0) ? b_buf : g_buf;
          if (has_psi && i == n_mma - 1) {
            w.wait(&bars->psi_full, 0, 216);
            wsm = kv_buf;
          }
          w.wait(&bars->a_full, i & 1, 217);
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const uint64_t a_desc = make_smem_desc(smem_u32(a_buf + (k / 4) * kRows * 128), 16, 1024) + (uint64_t)((k % 4) * 2);
            const uint64_t b_desc = make_smem_desc(smem_u32(wsm + (k / 4) * D * 128), 16, 1024) + (uint64_t)((k % 4) * 2);
            mma_f16_ss(tmem + C::kColZ, a_desc, b_desc, idesc_r, k != 0);
          }
          mma_commit(&bars->r_full);
        }
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
      const int b = i & 1;
      w.wait(&bars->zc_full[b], (i >> 1) & 1, 221);
      tc_fence_after();
#pragma unroll
      for (int c0 = 0; c0 < HC; c0 += 32) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(tmem + lane_addr + C::kColZ + b * D + half * HC + c0, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) z[c0 + e] = fmaf(z[c0 + e], corr, __uint_as_float(r[e]));
      }
      tc_fence_before();
      mbar_arrive(&bars->zc_empty[b]);
    };

    for (int j = 0; j < nchunks; ++j) {
      const int b = j & 1;
      w.wait(&bars->s_full[b], (j >> 1) & 1, 220);
      tc_fence_after();
      uint32_t r[32];
      tmem_ld_32x32b_x32(tmem + lane_addr + C::kColS + b * kMC + half * 32, r);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(&bars->s_empty[b]);
      // scores in the log2 domain; measurements beyond m are masked out
      float t[32], mx = -INFINITY;
      const int col0 = j * kMC + half * 32;
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        t[e] = (col0 + e < m) ? __uint_as_float(r[e]) * scale_log2 : -INFINITY;
        mx = fmaxf(mx, t[e]);
      }
      float* slot = xch + b * 256;
      slot[half * 128 + row] = mx;
      named_barrier_256();
      mx = fmaxf(mx, slot[(half ^ 1) * 128 + row]);
      const float new_max = fmaxf(run_max, mx);                 // finite: chunk 0 has a valid measurement
      const float corr = ex2(run_max - new_max);
      run_max = new_max;
      float sum = 0.f;
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        t[e] = ex2(t[e] - new_max);
        sum += t[e];
      }
      run_sum = fmaf(run_sum, corr, sum);
      w.wait(&bars->p_empty[b], ((j >> 1) & 1) ^ 1, 222);       // P buffer free again
#pragma unroll
      for (int c = 0; c < 4; ++c) st_chunk(p_buf + b * C::kPBytes, row, half * 4 + c, &t[c * 8]);
      fence_proxy_async();
      mbar_arrive(&bars->p_full[b]);
      if (j > 0) fold_zc(j - 1, corr_prev);
      corr_prev = corr;
    }
    fold_zc(nchunks - 1, corr_prev);
    // the two halves of a row share max and corr; their partial sums are added once
    float* slot = xch;               // reused once every thread is past the last chunk's exchange
    named_barrier_256();
    slot[half * 128 + row] = run_sum;
    named_barrier_256();
    const float inv = 1.f / (run_sum + slot[(half ^ 1) * 128 + row]);
#pragma unroll
    for (int i = 0; i < HC; ++i) z[i] *= inv;
    mbar_arrive(&bars->attn_done);

    if (T > 0) {
      const float th = theta[h];
      // the thread's HC columns sit in box (half*HC)/64 at chunks ((half*HC)%64)/8 ...
      uint8_t* box = a_buf + ((half * HC) / 64) * kRows * 128;
      const int chunk0 = ((half * HC) % 64) / 8;
      auto publish = [&](const float* v) {                      // bf16 operand copy for the next MMA
#pragma unroll
        for (int c = 0; c < HC / 8; ++c) st_chunk(box, row, chunk0 + c, v + c * 8);
        fence_proxy_async();
        tc_fence_before();
        mbar_arrive(&bars->a_full);
      };
      float cvec[HC];
      int phase = 0;
      publish(z);
      w.wait(&bars->r_full, phase & 1, 230); ++phase;
      tc_fence_after();
#pragma unroll
      for (int c0 = 0; c0 < HC; c0 += 32) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(tmem + lane_addr + C::kColZ + half * HC + c0, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          cvec[c0 + e] = __uint_as_float(r[e]);
          z[c0 + e] = soft(cvec[c0 + e], th);                   // alpha^1 (alpha^0 = 0)
        }
      }
      for (int it = 1; it < T; ++it) {
        publish(z);
        w.wait(&bars->r_full, phase & 1, 231); ++phase;
        tc_fence_after();
#pragma unroll
        for (int c0 = 0; c0 < HC; c0 += 32) {
          uint32_t r[32];
          tmem_ld_32x32b_x32(tmem + lane_addr + C::kColZ + half * HC + c0, r);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) z[c0 + e] = soft(z[c0 + e] - __uint_as_float(r[e]) + cvec[c0 + e], th);
        }
      }
      if (has_psi) {
        publish(z);
        w.wait(&bars->r_full, phase & 1, 232); ++phase;
        tc_fence_after();
#pragma unroll
        for (int c0 = 0; c0 < HC; c0 += 32) {
          uint32_t r[32];
          tmem_ld_32x32b_x32(tmem + lane_addr + C::kColZ + half * HC + c0, r);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) z[c0 + e] = __uint_as_float(r[e]);
        }
      }
    }
    const int grow = qtile * kRows + row;
    if (grow < nq && !w.dead) {
      uint4* o = reinterpret_cast<uint4*>(out + ((int64_t)bh * nq + grow) * D + half * HC);
#pragma unroll
      for (int c = 0; c < HC / 8; ++c)
        o[c] = make_uint4(pack_bf16(z[c * 8], z[c * 8 + 1]), pack_bf16(z[c * 8 + 2], z[c * 8 + 3]),
                          pack_bf16(z[c * 8 + 4], z[c * 8 + 5]), pack_bf16(z[c * 8 + 6], z[c * 8 + 7]));
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) tmem_dealloc(tmem, C::kTmemCols);
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
