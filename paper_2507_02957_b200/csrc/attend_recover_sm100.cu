// Compressed attention and sparse recovery for two tiles of 128 queries per CTA, on the sm_100a tensor cores.
//
// Paper, in order: A~ = softmax(Q K~^T / sqrt(d_k)) over the m measurements; Z = A~ V~;
// alpha^{t+1} = eta_theta(S alpha^t + B Z_i) (LISTA recurrence with S = I - mu G, B = mu M); C^_i = Psi alpha^_i.
// Neither the n_q x m matrix A~ nor any iterate alpha^t leaves the SM.
//
// One persistent CTA per SM walks work items of 256 consecutive queries of one (batch, head), each as two
// independent tiles A and B that share the stream of K~|V~ chunks; the TMA and MMA warps run ahead into the
// next item (its Q tiles, first chunks and first S MMAs) while the compute threads finish the current one.
// While the tensor cores run one tile's MMAs the other tile's threads do their softmax / shrinkage
// arithmetic, and the other way round.
//
// CTA = 12 warps in three warpgroups (registers are re-divided between them with setmaxnreg: the two
// compute warpgroups hold a whole row of alpha per thread, the control warps need very few):
//   warps 0-3 : tile A, one thread per query row (TMEM lane = row).  Softmax reference and sum, exp2,
//               P -> bf16 -> tensor memory, soft-threshold, output.  The whole row of alpha is in registers.
//   warps 4-7 : tile B, the same.
//   warp 8    : allocates tensor memory; one elected thread issues tile A's tcgen05.mma.
//   warp 9    : one elected thread issues every TMA copy.
//   warp 10   : one elected thread issues tile B's tcgen05.mma.
//   warp 11   : idle (it only completes the control warpgroup).
// Output: each compute warp stages its 32 rows, one 64-column box at a time, in shared memory and lane 0 issues a TMA
// store of the box (the recording variants of the backward pass, which spill more and need the L1, store directly).
//
// Attention phase, per tile and per chunk j of 64 measurements:
//   S_j = Q K~_j^T            (SS MMA, accumulator S[j&1] in tensor memory)
//   the row's thread reads S_j and writes P_j = exp2(S_j - ref) as packed bf16 over the first half of
//   S[j&1]'s columns
//   Zacc += P_j V~_j          (TS MMA: A operand from tensor memory, one accumulator for all chunks)
// ref is the row's reference maximum.  It only has to keep exp2 in range, so it is raised (and the row of
// Zacc and the running sum rescaled by exp2(old - new)) only when a chunk's maximum exceeds it by more than
// 8, i.e. when some P would exceed 2^8; the final division by the row sum cancels ref exactly.
// The MMAs of one tile are issued by one thread and execute in issue order, so S_{j+2} overwrites S[j&1] only
// after P_j V~_j has read P_j.
//
// Recovery phase, per tile.  The accumulator holds r_t = theta + c - a^_t (mu G), where c = z B and a^_t is
// the sum of the bf16 increments fed to the tensor cores so far; the registers hold b_t = alpha^t - theta
// (theta = the first layer's threshold where the thresholds differ per layer; eta then uses the layer's own):
//   r_0 = theta + z_bf16 B (threads store theta, one accumulating MMA);
//   x = b_t + r_t = alpha^t S + z B;   s = sat(x / (2 theta) + 1/2);   b_{t+1} = eta_theta(x) - theta = x - 2 theta s;
//   increment b_{t+1} - b_t = r_t - 2 theta s   (from r_t, so that b_{t+1} can overwrite b_t at once);
//   r_{t+1} = r_t + bf16(b_{t+1} - b_t) (-mu G)            (one accumulating MMA per iteration; -mu G is stored).
// This is the paper's S alpha + B z with S = I - mu G: the identity part stays exact in fp32 registers, only
// the increment that multiplies mu G is rounded to bf16, and c never needs registers of its own.  The
// saturating form of the shrinkage runs on the FMA pipe (two-element packed instructions where they exist);
// it leaves O(1e-7 theta) instead of exact zeros, so the last iteration uses the exact min/max form.
//
// Untied layers (one S_t, B_t per layer, kUntied): no running accumulator is possible, so every layer is one fresh
// product r_t = [a^_t | z^] [S_t - I ; B_t] (K = 2 d, both operands bf16 in tensor memory, z^ written once) and
// x = alpha^t + r_t with alpha^t exact in registers.  The matrices of layer t take ring positions after the
// item's chunks (S_t - I in the K~ slots, B_t in the V~ slots), so layer t + 1 is loaded while layer t is computed.
// The registers hold alpha^t + theta_t, which turns the shrinkage into y - 2 theta sat(y / (2 theta)).
#include "csat_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

#include <type_traits>

namespace csat {
namespace {

using namespace ptx;

constexpr int kRows = 128;            // queries per tile
constexpr int kTiles = 2;             // tiles per CTA
constexpr int kMC = 64;               // measurements per chunk
constexpr int kTileThreads = 128;
constexpr int kThreads = 384;          // three warpgroups: tile A, tile B, control
constexpr int kMmaWarp = 8, kTmaWarp = 9, kMmaWarpB = 10;   // tile A's MMA issuer, TMA producer, tile B's MMA issuer
constexpr int kMaxStages = 6;
constexpr int kComputeRegs = 224, kControlRegs = 56;   // registers per thread after setmaxnreg (checked on the host)
constexpr int kPolyEvery = 4;          // every 4th pair of scores takes the polynomial exp2 (measured best of 1, 2, 3, 4, none)

// kStaged: the output leaves through shared-memory boxes and TMA stores (the plain forward); the recording variants
// store directly (they spill more, and the 32 KB of boxes would take the L1 those spills live in)
template <int D, bool kStaged> struct Cfg {
  static constexpr int kDBoxes = D / 64;                          // 64-column boxes across the head dimension
  static constexpr int kStages = (D == 64) ? 6 : 4;               // K~ / V~ chunks in flight
  static constexpr uint32_t kQBytes = kDBoxes * kRows * 128;      // one Q tile; tile A's buffer later holds B
  static constexpr uint32_t kBoxBytes = kMC * 128;                // one 64-column box of a K~ or V~ chunk
  static constexpr uint32_t kSlotBytes = kDBoxes * kBoxBytes;     // K~ chunk (= V~ chunk)
  static constexpr uint32_t kMatBoxBytes = D * 128;               // one 64-column box of a d x d bf16 matrix
  static constexpr uint32_t kMatBytes = kDBoxes * kMatBoxBytes;
  static constexpr uint32_t kOffQ = 0;                            // [tile]
  static constexpr uint32_t kOffRing = kOffQ + kTiles * kQBytes;  // [stage][K~ slot | V~ slot]
  static constexpr uint32_t kOffOut = kOffRing + kStages * 2 * kSlotBytes;   // [compute warp]: 32 rows of one 64-column box of the output
  static constexpr uint32_t kOutBytes = 32 * 128;
  static constexpr uint32_t kOffBar = kOffOut + (kStaged ? kTiles * 4 * kOutBytes : 0);
  static constexpr uint32_t kBarBytes = 512;
  static constexpr uint32_t kSmemBytes = kOffBar + kBarBytes;     // base must be 1024-byte aligned (checked)
  // TMEM columns per tile (tile t starts at column 256 t): S[0] | S[1] | accumulator (Zacc, then r_t).
  // P_j overlays S[j&1]; the recovery operand overlays S[0].
  static constexpr uint32_t kTileCols = 256, kColS = 0, kColAcc = 2 * kMC, kTmemCols = 512;
  static_assert(2 * kMC + D <= 256, "TMEM budget");
  static_assert(D <= 2 * kMC, "recovery operands (z and alpha, D / 2 packed columns each) fit in the S columns");
  static_assert(kStages >= kDBoxes && kStages <= kMaxStages, "mu G and Psi are staged box by box in ring slots");
  static_assert(kMatBoxBytes <= kSlotBytes && kMatBytes <= kQBytes, "decoder matrices fit where they are staged");
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
};

struct Bars {
  uint64_t q_full[kTiles], q_free[kTiles], mats_full;
  uint64_t k_full[kMaxStages], k_empty[kMaxStages], v_full[kMaxStages], v_empty[kMaxStages];
  uint64_t s_full[kTiles][2], p_full[kTiles][2], zc_full[kTiles];
  uint64_t a_full[kTiles], r_full[kTiles];
  uint32_t tmem_slot;
  int abort;
};
static_assert(sizeof(Bars) <= 512, "barrier block");

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float y;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
  return y;
}
__device__ __forceinline__ float add_sat(float a, float b) {            // clamps the result to [0, 1]
  float y;
  asm("add.sat.f32 %0, %1, %2;" : "=f"(y) : "f"(a), "f"(b));
  return y;
}
__device__ __forceinline__ float fma_sat(float a, float b, float c) {   // clamps the result to [0, 1]
  float y;
  asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
  return y;
}
// 32-byte store (the address is 32-byte aligned)
__device__ __forceinline__ void st_global_v8(void* p, const uint32_t (&r)[8]) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]),
               "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
// two-element packed fp32 arithmetic (one instruction for both halves of a register pair): the compiler's float2
// builtins, so that it sees the register pairs (inline assembly on 64-bit registers cost extra moves and spills)
using F2 = float2;
__device__ __forceinline__ F2 pack2(float lo, float hi) { return make_float2(lo, hi); }
__device__ __forceinline__ F2 pack2u(uint32_t lo, uint32_t hi) { return make_float2(__uint_as_float(lo), __uint_as_float(hi)); }
__device__ __forceinline__ void unpack2(F2 v, float& lo, float& hi) { lo = v.x; hi = v.y; }
__device__ __forceinline__ F2 fma2(F2 a, F2 b, F2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ F2 add2(F2 a, F2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ F2 sub2(F2 a, F2 b) { return __fadd2_rn(a, make_float2(-b.x, -b.y)); }
__device__ __forceinline__ F2 mul2(F2 a, F2 b) { return __fmul2_rn(a, b); }

// exp2 of both halves on the FMA pipe (the MUFU unit is the bottleneck of the softmax: 4 lanes per clock and
// sub-core).  x <= ~9; anything below -120 (masked columns are -inf) gives 2^-120.  Round-to-nearest split
// x = i + f, f in [-1/2, 1/2]; 2^f by a cubic fitted to 7.5e-5 relative error (P is rounded to bf16, 3.9e-3,
// and the row sum tolerates far more); 2^i by adding i to the exponent field.
__device__ __forceinline__ void exp2_poly2(F2 x2, float& p0, float& p1) {
  float x0, x1;
  unpack2(x2, x0, x1);
  x2 = pack2(fmaxf(x0, -120.f), fmaxf(x1, -120.f));
  const F2 magic = pack2(12582912.f, 12582912.f);          // 1.5 * 2^23: the sum's low mantissa bits hold i
  const F2 t2 = add2(x2, magic);
  const F2 f2 = sub2(x2, sub2(t2, magic));
  F2 q2 = fma2(f2, pack2(0.055171459913253784f, 0.055171459913253784f), pack2(0.2426108568906784f, 0.2426108568906784f));
  q2 = fma2(q2, f2, pack2(0.6932609677314758f, 0.6932609677314758f));
  q2 = fma2(q2, f2, pack2(0.9999281167984009f, 0.9999281167984009f));
  float t0, t1, q0, q1;
  unpack2(t2, t0, t1);
  unpack2(q2, q0, q1);
  p0 = __int_as_float(__float_as_int(q0) + (__float_as_int(t0) << 23));
  p1 = __int_as_float(__float_as_int(q1) + (__float_as_int(t1) << 23));
}

// warpgroup-wide change of the per-thread register allowance (every warp of the warpgroup executes it)
template <int N> __device__ __forceinline__ void reg_alloc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dealloc() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

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

// kMasks (backward pass only, one S, B for all layers): besides the output the kernel leaves what the backward needs:
// Z (bf16, as fed to the first product), every row's log sum exp, and the decision |x_t| > theta_t of every layer,
// one bit per column: word c / 32 of (layer, row), bit 31 - c % 32.  With alpha_out (the gradients of the decoder's
// weights need them) also the iterates alpha^1 .. alpha^T as bf16: alpha^t of (b, h, row) at slot t of alpha_slot
// elements each (slot 0, alpha^0 = 0, is the caller's to clear), and with sign_out the sign bit of every x_t in the
// layout of the decisions (the gradient of the thresholds is - sum sign(x_t) o dx_t).
// kRec: 0 = the plain forward; 1 = also Z, log sum exp and the decisions (kMasks); 2 = also the iterates and the sign
// bits of x_t (kKeep: only then are alpha_out / sign_out looked at, so that mode 1 carries none of their registers)
// kFold (plain forward, one S, B and one positive threshold for all layers, T >= 2): the V~ stream is V~ B (formed
// once per (batch, head) by vfold_sm100_kernel), so the accumulator of the attention phase already holds z B: there is
// no product with B, and the first layer's shrinkage follows the normalisation directly.
template <int D, bool kUntied, int kRec, bool kFold = false>
__global__ void __launch_bounds__(kThreads, 1)
attend_recover_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_kv,
                            const __grid_constant__ CUtensorMap tmap_mats,
                            const __grid_constant__ CUtensorMap tmap_out,
                            const __grid_constant__ CUtensorMap tmap_vb, __nv_bfloat16* __restrict__ out,
                            const float* __restrict__ theta, int theta_stride, int nq, int m, int H, int T,
                            int has_psi, float scale_log2, int items_x, int n_items, int bh0, int* status,
                            float* __restrict__ lse_out, int lse_stride, __nv_bfloat16* __restrict__ z_out,
                            uint32_t* __restrict__ mask_out, __nv_bfloat16* __restrict__ alpha_out,
                            int64_t alpha_slot, uint32_t* __restrict__ sign_out) {
  using C = Cfg<D, kRec == 0>;
  constexpr bool kMasks = kRec >= 1, kKeep = kRec >= 2, kStaged = kRec == 0;
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {          // swizzled tiles need 1024-byte alignment; never seen to fail
    if (threadIdx.x == 0) atomicCAS(status, 0, 200);
    return;
  }
  uint8_t* q_buf = smem + C::kOffQ;             // [tile]
  uint8_t* ring = smem + C::kOffRing;
  Bars* bars = reinterpret_cast<Bars*>(smem + C::kOffBar);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Work items: item = bh * items_x + x covers queries [256 x, 256 x + 256) of (batch, head) bh.  The CTA is
  // persistent: it takes items blockIdx.x, blockIdx.x + gridDim.x, ...  Every role walks the same sequence with
  // its own free-running counters (ring position, chunks and recovery MMAs per tile), from which the barrier
  // parities follow, so that the TMA and MMA warps can run ahead into the next item while the compute threads
  // finish the current one.
  const int nchunks = (m + kMC - 1) / kMC;
  // ring positions an item's decoder matrices take after its chunks: mu G | Psi once, or one set per untied layer
  const int nlayers = T > 0 ? T + (has_psi ? 1 : 0) : 0;        // recovery MMAs per tile and item
  const int nvirt = T > 0 ? (kUntied ? C::kDBoxes * nlayers : C::kDBoxes) : 0;
  Waiter w{status, &bars->abort};
  auto k_slot = [&](int s) { return ring + (2 * s) * C::kSlotBytes; };
  auto v_slot = [&](int s) { return ring + (2 * s + 1) * C::kSlotBytes; };

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_q);
    prefetch_tmap(&tmap_kv);
    prefetch_tmap(&tmap_mats);
    if (kStaged) prefetch_tmap(&tmap_out);
    if (kFold) prefetch_tmap(&tmap_vb);
    mbar_init(&bars->mats_full, 1);
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&bars->k_full[s], 1); mbar_init(&bars->k_empty[s], kTiles);     // released by both MMA issuers
      mbar_init(&bars->v_full[s], 1); mbar_init(&bars->v_empty[s], kTiles);
    }
    for (int t = 0; t < kTiles; ++t) {
      mbar_init(&bars->q_full[t], 1);
      mbar_init(&bars->q_free[t], t == 0 ? kTiles : 1);     // tile A's buffer also holds B, which both tiles read
      for (int s = 0; s < 2; ++s) { mbar_init(&bars->s_full[t][s], 1); mbar_init(&bars->p_full[t][s], kTileThreads); }
      mbar_init(&bars->zc_full[t], 1);
      mbar_init(&bars->a_full[t], kTileThreads);
      mbar_init(&bars->r_full[t], 1);
    }
    bars->abort = 0;
    fence_mbar_init();
  }
  if (warp == kMmaWarp) {
    tmem_alloc(&bars->tmem_slot, C::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_slot;

  // 2 x 128 x 224 + 128 x 56 = 64512 registers; each branch below starts with its own setmaxnreg
  if (warp >= kMmaWarp) {
  reg_dealloc<kControlRegs>();
  if (warp == kTmaWarp) {
    // ------------------------------------------------ TMA producer ------------------------------------------------
    // Ring position g counts the chunks loaded so far (stage g % kStages, use g / kStages).  After an item's
    // chunks come nvirt "virtual chunks": the boxes of mu G go to their K~ slots and those of Psi to their V~
    // slots, under the same full / empty barriers.  B goes to tile A's Q buffer once the item's S MMAs are done.
    if (elect_one()) {
      uint32_t g = 0, items_done = 0;
      uint32_t q_loads[kTiles] = {0, 0};
      uint64_t k_hist = 0, v_hist = 0;        // bit i: the copy into the K~ / V~ slot of ring position g-1-i was issued
      uint32_t mats_loads = 0;
      auto ring_wait_k = [&](uint32_t pos, int code) {
        if (pos >= (uint32_t)C::kStages) w.wait(&bars->k_empty[pos % C::kStages], (pos / C::kStages - 1) & 1, code);
      };
      auto ring_wait_v = [&](uint32_t pos, int code) {
        if (pos >= (uint32_t)C::kStages) w.wait(&bars->v_empty[pos % C::kStages], (pos / C::kStages - 1) & 1, code);
      };
      for (int item = blockIdx.x; item < n_items && !w.dead; item += gridDim.x, ++items_done) {
        const int bh = bh0 + item / items_x, row0 = (item % items_x) * (kTiles * kRows), h = bh % H;
        const int ntiles = (nq - row0 > kRows) ? 2 : 1;
#pragma unroll
        for (int t = 0; t < kTiles; ++t) {
          if (t < ntiles) {
            if (q_loads[t] > 0) w.wait(&bars->q_free[t], (q_loads[t] - 1) & 1, 205);   // released by the last user
            if (w.dead) break;
            mbar_arrive_expect_tx(&bars->q_full[t], C::kQBytes);
            for (int gx = 0; gx < C::kDBoxes; ++gx)
              tma_load_3d(q_buf + t * C::kQBytes + gx * kRows * 128, &tmap_q, &bars->q_full[t], gx * 64, row0 + t * kRows, bh);
            ++q_loads[t];
          }
        }
        // K~|V~ come from the compression kernel before this one in the stream: with a programmatic dependent launch
        // this kernel may have started (and loaded its first Q tiles) before that one finished
        if (items_done == 0) pdl_wait();
        for (int j = 0; j < nchunks && !w.dead; ++j, ++g) {
          const int s = g % C::kStages;
          ring_wait_k(g, 201);
          if (w.dead) break;
          mbar_arrive_expect_tx(&bars->k_full[s], C::kSlotBytes);
          for (int gx = 0; gx < C::kDBoxes; ++gx)
            tma_load_3d(k_slot(s) + gx * C::kBoxBytes, &tmap_kv, &bars->k_full[s], gx * 64, j * kMC, bh);
          k_hist = (k_hist << 1) | 1u;
          v_hist <<= 1;
          ring_wait_v(g, 202);
          if (w.dead) { ++g; break; }
          mbar_arrive_expect_tx(&bars->v_full[s], C::kSlotBytes);
          for (int gx = 0; gx < C::kDBoxes; ++gx)
            tma_load_3d(v_slot(s) + gx * C::kBoxBytes, kFold ? &tmap_vb : &tmap_kv, &bars->v_full[s],
                        kFold ? gx * 64 : D + gx * 64, j * kMC, bh);
          v_hist |= 1u;
        }
        if (kUntied && T > 0 && !w.dead) {
          // layer l: S_l - I to the K~ slots, B_l to the V~ slots; after the last layer Psi to V~ slots
          const int mat0 = h * (2 * T + 1);
          for (int l = 0; l < nlayers && !w.dead; ++l) {
            const bool psi_l = (l == T);
            for (int gx = 0; gx < C::kDBoxes && !w.dead; ++gx, ++g) {
              const int s = g % C::kStages;
              ring_wait_k(g, 206);
              if (w.dead) break;
              if (!psi_l) {
                mbar_arrive_expect_tx(&bars->k_full[s], C::kMatBoxBytes);
                tma_load_3d(k_slot(s), &tmap_mats, &bars->k_full[s], gx * 64, 0, mat0 + 2 * l);
                k_hist = (k_hist << 1) | 1u;
              } else {
                mbar_arrive(&bars->k_full[s]);   // nothing to load: complete the phase so that the parities stay in step
                k_hist <<= 1;
              }
              v_hist <<= 1;
              ring_wait_v(g, 207);
              if (w.dead) { ++g; break; }
              mbar_arrive_expect_tx(&bars->v_full[s], C::kMatBoxBytes);
              tma_load_3d(v_slot(s), &tmap_mats, &bars->v_full[s], gx * 64, 0, mat0 + (psi_l ? 2 * T : 2 * l + 1));
              v_hist |= 1u;
            }
          }
        }
        if (!kUntied && T > 0 && !w.dead) {
          // every S MMA of the item has finished once the last one has: tile A's Q buffer is free for B
          const uint32_t gl = g - 1;
          w.wait(&bars->k_empty[gl % C::kStages], (gl / C::kStages) & 1, 203);
          if (!w.dead && !kFold) {
            mbar_arrive_expect_tx(&bars->mats_full, C::kMatBytes);
            for (int gx = 0; gx < C::kDBoxes; ++gx)
              tma_load_3d(q_buf + gx * C::kMatBoxBytes, &tmap_mats, &bars->mats_full, gx * 64, 0, h * 3 + 1);
            ++mats_loads;
          }
          for (int gx = 0; gx < C::kDBoxes && !w.dead; ++gx, ++g) {
            const int s = g % C::kStages;
            ring_wait_k(g, 206);
            if (w.dead) break;
            mbar_arrive_expect_tx(&bars->k_full[s], C::kMatBoxBytes);
            tma_load_3d(k_slot(s), &tmap_mats, &bars->k_full[s], gx * 64, 0, h * 3 + 0);          // -mu G
            k_hist = (k_hist << 1) | 1u;
            v_hist <<= 1;
            ring_wait_v(g, 207);
            if (w.dead) { ++g; break; }
            if (has_psi) {
              mbar_arrive_expect_tx(&bars->v_full[s], C::kMatBoxBytes);
              tma_load_3d(v_slot(s), &tmap_mats, &bars->v_full[s], gx * 64, 0, h * 3 + 2);        // Psi
              v_hist |= 1u;
            } else {
              mbar_arrive(&bars->v_full[s]);     // nothing to load: complete the phase so that the parities stay in step
            }
          }
        }
      }
      if (w.dead) {
        // gave up: let the copies that are still in flight land before the CTA's shared memory goes away
#pragma unroll
        for (int t = 0; t < kTiles; ++t)
          if (q_loads[t] > 0) mbar_wait_drain(&bars->q_full[t], (q_loads[t] - 1) & 1);
        for (uint32_t i = 0; i < (uint32_t)C::kStages && i < g; ++i) {
          const uint32_t pos = g - 1 - i;
          if ((k_hist >> i) & 1u) mbar_wait_drain(&bars->k_full[pos % C::kStages], (pos / C::kStages) & 1);
          if ((v_hist >> i) & 1u) mbar_wait_drain(&bars->v_full[pos % C::kStages], (pos / C::kStages) & 1);
        }
        if (mats_loads > 0) mbar_wait_drain(&bars->mats_full, (mats_loads - 1) & 1);
      }
    }
  } else if (warp == kMmaWarp || warp == kMmaWarpB) {
    // ------------------------------------------------ MMA issuers -------------------------------------------------
    // One elected thread per tile issues that tile's MMAs (tile A: warp 8, tile B: warp 10, on different
    // sub-cores): issuing is a serial stream of a few dozen cycles per MMA, and one thread for both tiles was the
    // critical path of the attention phase.  Barriers that release something both tiles read (ring slots, tile
    // A's Q buffer when it holds B) count two arrivals, one per issuer; where an item has no second tile, tile
    // B's issuer walks the same ring positions and arrives without issuing anything.
    // Descriptors of buffers that do not move are built once, the others differ from a base by constants.
    const int t = (warp == kMmaWarp) ? 0 : 1;
    if (elect_one()) {
      constexpr uint32_t idesc_s = make_idesc_bf16(kRows, kMC, false, false);   // S  = Q  K~^T : both K-major
      constexpr uint32_t idesc_z = make_idesc_bf16(kRows, D, false, true);      // Z += P  V~   : V~ is MN-major
      constexpr uint32_t idesc_r = make_idesc_bf16(kRows, D, false, false);     // r += a (-W)^T: both K-major
      // K-major operand: K step k (16 columns) lies in 64-column box k / 4, 32 (k % 4) bytes into each row
      auto kstep = [](int k, uint32_t box_bytes) { return (uint64_t)((k / 4) * (box_bytes >> 4) + (k % 4) * 2); };
      const uint64_t q_desc0 = make_smem_desc(smem_u32(q_buf), 16, 1024);
      const uint64_t qd = q_desc0 + (uint64_t)(t * (C::kQBytes >> 4));
      const uint64_t ring_k0 = make_smem_desc(smem_u32(ring), 16, 1024);
      const uint64_t ring_v0 = make_smem_desc(smem_u32(ring + C::kSlotBytes), C::kBoxBytes, 1024);
      constexpr uint64_t kStageStep = (2 * C::kSlotBytes) >> 4;                 // descriptor distance between stages
      const uint32_t tb = tmem + t * C::kTileCols;
      uint32_t g = 0, items_done = 0;          // ring position of the item's first chunk; items of this CTA so far
      uint32_t cb = 0;                         // chunks of this tile's earlier items (S / P buffer and parities)
      uint32_t ab = 0;                         // recovery MMAs of this tile's earlier items
      uint32_t q_uses = 0;
      for (int item = blockIdx.x; item < n_items && !w.dead; item += gridDim.x, ++items_done) {
        const int row0 = (item % items_x) * (kTiles * kRows);
        const bool active = t == 0 || nq - row0 > kRows;          // the item has this tile
        // releases a buffer both issuers account for: after this thread's MMAs, or at once when it has none
        auto release = [&](uint64_t* bar) { if (active) mma_commit(bar); else mbar_arrive(bar); };
        auto issue_pv = [&](int i) {
          const uint32_t pos = g + i;
          const int s = pos % C::kStages;
          w.wait(&bars->v_full[s], (pos / C::kStages) & 1, 211);
          if (active) {
            const uint64_t b_desc = ring_v0 + (uint64_t)s * kStageStep;
            const uint32_t c = cb + i;
            const int b = c & 1;
            w.wait(&bars->p_full[t][b], (c >> 1) & 1, 212);
            tc_fence_after();
            // P: 8 packed columns per 16 measurements; V~: +16 rows = 2048 B
            mma_f16_ts(tb + C::kColAcc, tb + C::kColS + b * kMC, b_desc, idesc_z, (uint32_t)(i != 0));
#pragma unroll
            for (int k = 1; k < kMC / 16; ++k)
              mma_f16_ts(tb + C::kColAcc, tb + C::kColS + b * kMC + k * 8, b_desc + (uint64_t)(k * 128), idesc_z, 1u);
            mma_commit(&bars->zc_full[t]);
          }
          release(&bars->v_empty[s]);
        };
        if (active) { w.wait(&bars->q_full[t], q_uses & 1, 210); ++q_uses; }
        for (int j = 0; j < nchunks; ++j) {
          const uint32_t pos = g + j;
          const int s = pos % C::kStages;
          w.wait(&bars->k_full[s], (pos / C::kStages) & 1, 213);
          if (active) {
            tc_fence_after();
            const uint64_t kd = ring_k0 + (uint64_t)s * kStageStep;
            const int b = (cb + j) & 1;
            const uint32_t ds = tb + C::kColS + b * kMC;
#pragma unroll
            for (int k = 0; k < D / 16; ++k)
              mma_f16_ss(ds, qd + kstep(k, kRows * 128), kd + kstep(k, C::kBoxBytes), idesc_s, k != 0);
            mma_commit(&bars->s_full[t][b]);
          }
          release(&bars->k_empty[s]);
          if (j == nchunks - 1) {
            // the Q buffers have been read for the last time (tile A's still takes B when there is a recovery
            // with one S, B for all layers)
            if (t == 1 && active) mma_commit(&bars->q_free[1]);
            if (T == 0 || kUntied) release(&bars->q_free[0]);
          }
          if (j > 0) issue_pv(j - 1);
        }
        issue_pv(nchunks - 1);
        if (kUntied && T > 0) {
          // layer l: r = z^ B_l (+ a^_l (S_l - I) from the second layer on); then Psi on the final alpha
          for (int l = 0; l < nlayers; ++l) {
            const bool psi_l = (l == T);
            const uint32_t pl = g + nchunks + l * C::kDBoxes;     // ring position of the layer's first box
            for (int gx = 0; gx < C::kDBoxes; ++gx) {
              const uint32_t pos = pl + gx;
              w.wait(&bars->k_full[pos % C::kStages], (pos / C::kStages) & 1, 215);
              w.wait(&bars->v_full[pos % C::kStages], (pos / C::kStages) & 1, 215);
            }
            if (active) {
              w.wait(&bars->a_full[t], (ab + l) & 1, 216);
              tc_fence_after();
              const uint32_t z_cols = tb + C::kColS, a_cols = tb + C::kColS + D / 2;
#pragma unroll
              for (int k = 0; k < D / 16; ++k) {
                // the V~ slot of the layer's box k / 4: B_l (A operand z^), or Psi (A operand the final alpha)
                const uint64_t wd = ring_k0 + (uint64_t)((pl + k / 4) % C::kStages) * kStageStep +
                                    (uint64_t)(C::kSlotBytes >> 4) + (uint64_t)((k % 4) * 2);
                mma_f16_ts(tb + C::kColAcc, (psi_l ? a_cols : z_cols) + k * 8, wd, idesc_r, k == 0 ? 0u : 1u);
              }
              if (!psi_l && l > 0) {
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                  const uint64_t wd = ring_k0 + (uint64_t)((pl + k / 4) % C::kStages) * kStageStep +
                                      (uint64_t)((k % 4) * 2);                                   // S_l - I
                  mma_f16_ts(tb + C::kColAcc, a_cols + k * 8, wd, idesc_r, 1u);
                }
              }
              mma_commit(&bars->r_full[t]);
            }
            for (int gx = 0; gx < C::kDBoxes; ++gx) {     // this tile has read the layer's matrices
              release(&bars->k_empty[(pl + gx) % C::kStages]);
              release(&bars->v_empty[(pl + gx) % C::kStages]);
            }
          }
        }
        if (!kUntied && T > 0) {
          const uint32_t gv = g + nchunks;            // ring position of the first box of -mu G / Psi
          const int n_mma = nlayers;                  // r_0 = theta + z B, then T-1 increments with -mu G, then Psi
          if (kFold) release(&bars->q_free[0]);          // no B to stage: tile A's Q buffer is free
          for (int i = kFold ? 1 : 0; i < n_mma; ++i) {
            const bool first = (i == 0), psi_step = has_psi && i == n_mma - 1;
            if (first) w.wait(&bars->mats_full, items_done & 1, 214);
            if (i == 1 || psi_step)
              for (int gx = 0; gx < C::kDBoxes; ++gx) {
                const uint32_t pos = gv + gx;
                w.wait(psi_step ? &bars->v_full[pos % C::kStages] : &bars->k_full[pos % C::kStages],
                       (pos / C::kStages) & 1, 215);
              }
            if (active) {
              const uint32_t acc0 = psi_step ? 0u : 1u;
              w.wait(&bars->a_full[t], (ab + i - (kFold ? 1 : 0)) & 1, 216);
              tc_fence_after();
#pragma unroll
              for (int k = 0; k < D / 16; ++k) {
                // B: boxes of d rows in tile A's Q buffer; -mu G / Psi: box k / 4 in the K~ / V~ slot of ring
                // position gv + k / 4
                const uint64_t wd = first ? q_desc0 + (uint64_t)((k / 4) * (C::kMatBoxBytes >> 4))
                                          : ring_k0 + (uint64_t)((gv + k / 4) % C::kStages) * kStageStep +
                                                (psi_step ? (uint64_t)(C::kSlotBytes >> 4) : 0);
                mma_f16_ts(tb + C::kColAcc, tb + C::kColS + k * 8, wd + (uint64_t)((k % 4) * 2), idesc_r,
                           k == 0 ? acc0 : 1u);
              }
              mma_commit(&bars->r_full[t]);
            }
            if (first) release(&bars->q_free[0]);         // B has been read: tile A's Q buffer is free
          }
          for (int gx = 0; gx < C::kDBoxes; ++gx) {       // release the ring positions of -mu G / Psi; a position
            const uint32_t pos = gv + gx;                 // that was never read is waited for first, so that no
            if (T == 1) w.wait(&bars->k_full[pos % C::kStages], (pos / C::kStages) & 1, 215);   // phase is skipped
            if (!has_psi) w.wait(&bars->v_full[pos % C::kStages], (pos / C::kStages) & 1, 215);
            release(&bars->k_empty[pos % C::kStages]);
            release(&bars->v_empty[pos % C::kStages]);
          }
        }
        g += nchunks + nvirt;
        if (active) { cb += nchunks; ab += nlayers - ((kFold && !kUntied && T > 0) ? 1 : 0); }
      }
    }
  }
  } else {
    reg_alloc<kComputeRegs>();
    // ------------------------------------------------ compute threads ---------------------------------------------
    const int t = warp >> 2, wq = warp & 3;                     // tile, lane quarter
    const int row = wq * 32 + lane;                             // row of the tile = TMEM lane
    const uint32_t tbase = tmem + ((uint32_t)(wq * 32) << 16) + t * C::kTileCols;
    const uint32_t acc_addr = tbase + C::kColAcc;
    const F2 sc2 = pack2(scale_log2, scale_log2);
    uint32_t cb = 0;                                            // chunks of this tile's earlier items
    int phase = 0;                                              // phases of r_full[t] this thread has waited for
    uint8_t* stage = smem + C::kOffOut + warp * C::kOutBytes + lane * 128;   // this row in the warp's staging box
    // every lane of a warp leaves the loop at the same item (a lane that gave up falls through the item's waits)
    for (int item = blockIdx.x; item < n_items && !__any_sync(0xffffffffu, w.dead); item += gridDim.x) {
      const int bh = bh0 + item / items_x, row0 = (item % items_x) * (kTiles * kRows), h = bh % H;
      if (t >= ((nq - row0 > kRows) ? 2 : 1)) continue;         // this item has no second tile
      float ref = -INFINITY;                                    // reference maximum of the row (log2 domain)
      F2 sum2 = pack2(0.f, 0.f);                          // running sum of P, two partial sums
      const float kappa = T > 0 ? theta[h] : 0.f;               // loaded now, needed after the attention phase

      for (int j = 0; j < nchunks; ++j) {
        const uint32_t c = cb + j;                              // chunk count of this tile over all its items
        const int b = c & 1;
        w.wait(&bars->s_full[t][b], (c >> 1) & 1, 220);
        tc_fence_after();
        uint32_t ra[32], rb[32];                                // columns [0, 32) and [32, 64) of S_j
        tmem_ld_32x32b_x32(tbase + C::kColS + b * kMC, ra);
        tmem_ld_32x32b_x32(tbase + C::kColS + b * kMC + 32, rb);
        tmem_wait_ld();
        // scores in the log2 domain; measurements beyond m are masked out
        float mx = -INFINITY;
        if ((j + 1) * kMC <= m) {
          float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;   // independent chains
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            m0 = max3(m0, __uint_as_float(ra[e]), __uint_as_float(ra[e + 1]));
            m1 = max3(m1, __uint_as_float(ra[e + 2]), __uint_as_float(ra[e + 3]));
            m2 = max3(m2, __uint_as_float(rb[e]), __uint_as_float(rb[e + 1]));
            m3 = max3(m3, __uint_as_float(rb[e + 2]), __uint_as_float(rb[e + 3]));
          }
          mx = fmaxf(max3(m0, m1, m2), m3);
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            if (j * kMC + e >= m) ra[e] = 0xff800000u;          // -inf
            if (j * kMC + 32 + e >= m) rb[e] = 0xff800000u;
            mx = max3(mx, __uint_as_float(ra[e]), __uint_as_float(rb[e]));
          }
        }
        mx *= scale_log2;           // scale > 0: the maximum commutes with it; finite: the chunk has a valid column
        if (j == 0) {
          ref = mx;
        } else {
          const bool raise = mx > ref + 8.f;
          if (__any_sync(0xffffffffu, raise)) {
            // rare: rescale this warp's rows of the accumulator (factor 1 for rows that keep their reference)
            // A parity wait is only safe when the barrier is in the awaited phase or the one after it.  It is:
            // S_j's commit (observed above) completes after every MMA its thread issued before, P_{j-2} V~_{j-2}
            // among them, so phases up to c - 2 are over; phase c cannot end before this thread's arrival below.
            w.wait(&bars->zc_full[t], (c - 1) & 1, 221);        // P_{j-1} V~_{j-1} has been added
            tc_fence_after();
            const float f = raise ? ex2(ref - mx) : 1.f;
            if (raise) ref = mx;
            sum2 = mul2(sum2, pack2(f, f));
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 16) {
              uint32_t a[16];
              tmem_ld_32x32b_x16(acc_addr + c0, a);
              tmem_wait_ld();
#pragma unroll
              for (int e = 0; e < 16; ++e) a[e] = __float_as_uint(__uint_as_float(a[e]) * f);
              tmem_st_32x32b_x16(acc_addr + c0, a);
            }
          }
        }
        const F2 nref2 = pack2(-ref, -ref);
        // P_j over the first 32 columns of S[b] (two bf16 per column)
        auto exp_half = [&](const uint32_t (&r)[32], uint32_t col) {
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const F2 x2 = fma2(pack2u(r[e], r[e + 1]), sc2, nref2);
            float p0, p1;
            if ((e >> 1) % kPolyEvery == kPolyEvery - 1) {       // this pair on the FMA pipe, the others on the MUFU
              exp2_poly2(x2, p0, p1);
            } else {
              float t0, t1;
              unpack2(x2, t0, t1);
              p0 = ex2(t0);
              p1 = ex2(t1);
            }
            sum2 = add2(sum2, pack2(p0, p1));
            pk[e >> 1] = pack_bf16(p0, p1);
          }
          tmem_st_32x32b_x16(tbase + C::kColS + b * kMC + col, pk);
        };
        exp_half(ra, 0);
        exp_half(rb, 16);
        tmem_wait_st();                                         // also covers a rescale's stores
        tc_fence_before();
        // The item's last two phases of zc_full are observed in order, the first of them before the arrival that
        // lets the last product start (afterwards the barrier may be two phases on, which a parity wait cannot tell
        // from none).
        if (j == nchunks - 1 && j > 0) w.wait(&bars->zc_full[t], (c - 1) & 1, 223);
        mbar_arrive(&bars->p_full[t][b]);
      }
      float inv;
      {
        float s0, s1;
        unpack2(sum2, s0, s1);
        inv = 1.f / (s0 + s1);
        // the backward pass asks for the row's log sum exp of the scaled scores (natural logarithm)
        if (lse_out != nullptr && row0 + t * kRows + row < nq)
          lse_out[((int64_t)bh * nq + row0 + t * kRows + row) * lse_stride] = (ref + __log2f(s0 + s1)) * 0.69314718056f;
      }
      w.wait(&bars->zc_full[t], (cb + nchunks - 1) & 1, 222);   // every P V~ product has been added
      cb += nchunks;
      tc_fence_after();
      // v2 holds, in turn: Z, b_t = alpha^t - theta, alpha^T, Psi alpha^T  (pairs of adjacent columns)
      F2 v2[D / 2];
      {
        const F2 inv2 = pack2(inv, inv);
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 16) {
          uint32_t a[16];
          tmem_ld_32x32b_x16(acc_addr + c0, a);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 16; e += 2) v2[(c0 + e) >> 1] = mul2(pack2u(a[e], a[e + 1]), inv2);
        }
      }
      const int grow_m = row0 + t * kRows + row;                // this thread's query (may lie beyond n_q)
      // The output leaves through shared memory, one 64-column box of the warp's 32 rows at a time: each thread writes
      // its 128 bytes in the 128-byte swizzle of the tensor map and lane 0 hands the box to one TMA store, which runs
      // while the threads go on (storing 32-byte pieces of 32 different rows per instruction straight to global
      // memory kept them at the stores for ~4000 cycles per item).  Rows beyond n_q are clipped by the tensor map.
      bool staged = false;
      auto stage_box = [&](int bx) {
        if (!kStaged || out == nullptr) return;
        if (lane == 0) bulk_wait_group_read0();                 // the warp's previous store has read the buffer
        __syncwarp();
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          float x[8];
#pragma unroll
          for (int u = 0; u < 4; ++u) unpack2(v2[bx * 32 + c * 4 + u], x[2 * u], x[2 * u + 1]);
          *reinterpret_cast<uint4*>(stage + ((c ^ (lane & 7)) << 4)) =
              make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]), pack_bf16(x[6], x[7]));
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          if (grow_m < nq && !w.dead && *(volatile int*)&bars->abort == 0)
            tma_store_3d(&tmap_out, stage, bx * 64, grow_m, bh);
          bulk_commit_group();
        }
      };
      if (kMasks && z_out != nullptr && grow_m < nq) {          // Z as fed to the first product, for the backward pass
        uint4* zo = reinterpret_cast<uint4*>(z_out + ((int64_t)bh * nq + grow_m) * D);
#pragma unroll
        for (int c = 0; c < D / 8; ++c) {
          float x[8];
#pragma unroll
          for (int u = 0; u < 4; ++u) unpack2(v2[c * 4 + u], x[2 * u], x[2 * u + 1]);
          zo[c] = make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]), pack_bf16(x[6], x[7]));
        }
      }
      // kMasks: this row's place in slot 0 of the iterates (rows of 2 D bytes from a 256-byte aligned base: 32-byte stores)
      __nv_bfloat16* arow = (kKeep && alpha_out != nullptr && grow_m < nq)
                                ? alpha_out + ((int64_t)bh * nq + grow_m) * D : nullptr;
      uint32_t mw[D / 32];                                      // kMasks: the current layer's decisions
      uint32_t sw[D / 32];                                      // kMasks with sign_out: the current layer's sign bits
      const bool signs = kKeep && sign_out != nullptr;
      auto store_masks = [&](int layer) {
        if (signs && grow_m < nq) {
          uint32_t* so = sign_out + (((int64_t)bh * T + layer) * nq + grow_m) * (D / 32);
          if (D == 128) *reinterpret_cast<uint4*>(so) = make_uint4(sw[0], sw[1], sw[2], sw[D / 32 - 1]);
          else *reinterpret_cast<uint2*>(so) = make_uint2(sw[0], sw[1]);
        }
        if (kMasks && mask_out != nullptr && grow_m < nq) {
          uint32_t* mo = mask_out + (((int64_t)bh * T + layer) * nq + grow_m) * (D / 32);
          if (D == 128) *reinterpret_cast<uint4*>(mo) = make_uint4(mw[0], mw[1], mw[2], mw[D / 32 - 1]);
          else *reinterpret_cast<uint2*>(mo) = make_uint2(mw[0], mw[1]);
        }
      };
      auto publish = [&](uint32_t col) {                        // v2 as a bf16 A operand, from column col of S on
        const uint32_t op_addr = tbase + C::kColS + col;
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 16) {
          uint32_t pk[8];
#pragma unroll
          for (int e = 0; e < 16; e += 2) {
            float x0, x1;
            unpack2(v2[(c0 + e) >> 1], x0, x1);
            pk[e >> 1] = pack_bf16(x0, x1);
          }
          tmem_st_32x32b_x8(op_addr + c0 / 2, pk);
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bars->a_full[t]);
      };

      if (kUntied && T > 0) {
        // z^ in the first D / 2 packed columns (written once), a^_t in the next D / 2.  The registers hold
        // y-offset iterates b_t = alpha^t + theta_t, so that x + theta_t = b_t + r_t needs no add of its own;
        // the layer before the last adds nothing, because the last layer shrinks exactly from x = alpha + r.
        const uint32_t a_addr = tbase + C::kColS + D / 2;
        publish(0);
        {
          const float b0 = T > 1 ? theta[h] : 0.f;
#pragma unroll
          for (int i = 0; i < D / 2; ++i) v2[i] = pack2(b0, b0);      // alpha^0 = 0
        }
        for (int it = 0; it + 1 < T; ++it) {
          const float th = theta[(int64_t)it * theta_stride + h];
          const float thn = it + 2 < T ? theta[(int64_t)(it + 1) * theta_stride + h] : 0.f;
          const float inv2th = th > 0.f ? 0.5f / th : 0.f;          // theta = 0: sat(0) = 0 and eta(x) = x
          const F2 m2th2 = pack2(-2.f * th, -2.f * th);
          const F2 p2th2 = pack2(2.f * th, 2.f * th);
          const F2 nx2 = pack2(thn, thn);
          w.wait(&bars->r_full[t], phase & 1, 230); ++phase;
          tc_fence_after();
          auto shrink16 = [&](const uint32_t (&r)[16], int c0) {
            uint32_t pk[8];
#pragma unroll
            for (int e = 0; e < 16; e += 2) {
              const F2 y2 = add2(v2[(c0 + e) >> 1], pack2u(r[e], r[e + 1]));   // alpha^t S_t + z B_t + theta_t
              float y0, y1;
              unpack2(y2, y0, y1);
              if (kMasks) {
                // |x| > theta  <=>  y < 0 or y > 2 theta  <=>  y (2 theta - y) < 0: its sign bit is the decision
                float g0, g1;
                unpack2(mul2(y2, fma2(y2, pack2(-1.f, -1.f), p2th2)), g0, g1);
                mw[c0 >> 5] = __funnelshift_l(__float_as_uint(g0), mw[c0 >> 5], 1);
                mw[c0 >> 5] = __funnelshift_l(__float_as_uint(g1), mw[c0 >> 5], 1);
                if (signs) {                         // where the decision holds y and x = y - theta have the same sign
                  sw[c0 >> 5] = __funnelshift_l(__float_as_uint(y0), sw[c0 >> 5], 1);
                  sw[c0 >> 5] = __funnelshift_l(__float_as_uint(y1), sw[c0 >> 5], 1);
                }
              }
              const F2 t2 = pack2(fma_sat(y0, inv2th, 0.f), fma_sat(y1, inv2th, 0.f));
              const F2 an = fma2(t2, m2th2, y2);                               // alpha^{t+1} = eta_theta(x)
              v2[(c0 + e) >> 1] = add2(an, nx2);
              float a0, a1;
              unpack2(an, a0, a1);
              pk[e >> 1] = pack_bf16(a0, a1);
            }
            tmem_st_32x32b_x8(a_addr + c0 / 2, pk);
            if (kKeep && arow != nullptr) st_global_v8(arow + (int64_t)(it + 1) * alpha_slot + c0, pk);   // alpha^{t+1}
          };
          uint32_t r0[16], r1[16];
          tmem_ld_32x32b_x16(acc_addr, r0);
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 32) {
            tmem_wait_ld();
            tmem_ld_32x32b_x16(acc_addr + c0 + 16, r1);
            shrink16(r0, c0);
            tmem_wait_ld();
            if (c0 + 32 < D) tmem_ld_32x32b_x16(acc_addr + c0 + 32, r0);
            shrink16(r1, c0 + 16);
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(&bars->a_full[t]);
          store_masks(it);
        }
        const float th = theta[(int64_t)(T - 1) * theta_stride + h];
        w.wait(&bars->r_full[t], phase & 1, 231); ++phase;
        tc_fence_after();
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 16) {
          uint32_t r[16];
          tmem_ld_32x32b_x16(acc_addr + c0, r);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 16; e += 2) {
            float b0, b1;
            unpack2(v2[(c0 + e) >> 1], b0, b1);
            const float x0 = b0 + __uint_as_float(r[e]), x1 = b1 + __uint_as_float(r[e + 1]);
            if (kMasks) {
              mw[c0 >> 5] = __funnelshift_l(__float_as_uint(th - fabsf(x0)), mw[c0 >> 5], 1);
              mw[c0 >> 5] = __funnelshift_l(__float_as_uint(th - fabsf(x1)), mw[c0 >> 5], 1);
              if (signs) {
                sw[c0 >> 5] = __funnelshift_l(__float_as_uint(x0), sw[c0 >> 5], 1);
                sw[c0 >> 5] = __funnelshift_l(__float_as_uint(x1), sw[c0 >> 5], 1);
              }
            }
            v2[(c0 + e) >> 1] = pack2(x0 - fminf(fmaxf(x0, -th), th), x1 - fminf(fmaxf(x1, -th), th));
          }
        }
        store_masks(T - 1);
        if (kKeep && arow != nullptr) {
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 16) {
            uint32_t pa[8];
#pragma unroll
            for (int e = 0; e < 16; e += 2) {
              float a0, a1;
              unpack2(v2[(c0 + e) >> 1], a0, a1);
              pa[e >> 1] = pack_bf16(a0, a1);
            }
            st_global_v8(arow + (int64_t)T * alpha_slot + c0, pa);
          }
        }
        if (has_psi) {
          publish(D / 2);
          w.wait(&bars->r_full[t], phase & 1, 232); ++phase;
          tc_fence_after();
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 16) {
            uint32_t r[16];
            tmem_ld_32x32b_x16(acc_addr + c0, r);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; e += 2) v2[(c0 + e) >> 1] = pack2u(r[e], r[e + 1]);
          }
        }
      }
      // One positive threshold for all layers (the ISTA-derived decoder), no decisions to record: the same recurrence
      // in units of 2 theta, which saves one instruction per pair of elements.  Registers c = alpha / (2 theta),
      // accumulator r' = 1/2 + (z B - a^ mu G) / (2 theta) (the threads store 1/2, z is published divided by 2 theta):
      //   s = sat(c + r') (= sat(x / (2 theta) + 1/2), one saturating add);  increment = r' - s;  c += increment.
      const bool scaled_units = kFold || (!kUntied && !kMasks && T > 0 && theta_stride == 0 && kappa > 0.f);
      if (scaled_units) {
        const uint32_t op_addr = tbase + C::kColS;
        if (kFold) {
          // the accumulator held z B (unnormalised): r'_0 = 1/2 + z B / (2 theta) goes back into it, and the first
          // pass below reads it from there like every later one
          const float inv2th = 0.5f / kappa;
          const F2 i2 = pack2(inv2th, inv2th), hf = pack2(0.5f, 0.5f);
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 16) {
            uint32_t tb[16];
#pragma unroll
            for (int e = 0; e < 16; e += 2) {
              float r0_, r1_;
              unpack2(fma2(v2[(c0 + e) >> 1], i2, hf), r0_, r1_);
              tb[e] = __float_as_uint(r0_);
              tb[e + 1] = __float_as_uint(r1_);
            }
            tmem_st_32x32b_x16(acc_addr + c0, tb);
          }
          tmem_wait_st();
        } else {
          uint32_t tb[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) tb[e] = __float_as_uint(0.5f);
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 16) tmem_st_32x32b_x16(acc_addr + c0, tb);
          const float inv2th = 0.5f / kappa;
          const F2 i2 = pack2(inv2th, inv2th);
#pragma unroll
          for (int i = 0; i < D / 2; ++i) v2[i] = mul2(v2[i], i2);
        }
        if (!kFold) publish(0);
#pragma unroll
        for (int i = 0; i < D / 2; ++i) v2[i] = pack2(0.f, 0.f);      // alpha^0 = 0
        const F2 m1 = pack2(-1.f, -1.f);
        for (int it = 0; it + 1 < T; ++it) {
          if (!kFold || it > 0) { w.wait(&bars->r_full[t], phase & 1, 230); ++phase; }
          tc_fence_after();
          auto shrink16 = [&](const uint32_t (&r)[16], int c0) {
            uint32_t pk[8];
#pragma unroll
            for (int e = 0; e < 16; e += 2) {
              float a0, a1;
              unpack2(v2[(c0 + e) >> 1], a0, a1);
              const F2 s2 = pack2(add_sat(a0, __uint_as_float(r[e])), add_sat(a1, __uint_as_float(r[e + 1])));
              const F2 dn = fma2(s2, m1, pack2u(r[e], r[e + 1]));     // (alpha^{t+1} - alpha^t) / (2 theta)
              v2[(c0 + e) >> 1] = add2(v2[(c0 + e) >> 1], dn);
              float d0, d1;
              unpack2(dn, d0, d1);
              pk[e >> 1] = pack_bf16(d0, d1);
            }
            tmem_st_32x32b_x8(op_addr + c0 / 2, pk);
          };
          uint32_t r0[16], r1[16];
          tmem_ld_32x32b_x16(acc_addr, r0);
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 32) {
            tmem_wait_ld();
            tmem_ld_32x32b_x16(acc_addr + c0 + 16, r1);
            shrink16(r0, c0);
            tmem_wait_ld();
            if (c0 + 32 < D) tmem_ld_32x32b_x16(acc_addr + c0 + 32, r0);
            shrink16(r1, c0 + 16);
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(&bars->a_full[t]);
        }
        // last iteration, exact shrinkage, back in the data's units: alpha^T = 2 theta eta_{1/2}(c + r' - 1/2)
        w.wait(&bars->r_full[t], phase & 1, 231); ++phase;
        tc_fence_after();
        const F2 tt2 = pack2(2.f * kappa, 2.f * kappa), mh2 = pack2(-0.5f, -0.5f);
        auto last16 = [&](const uint32_t (&r)[16], int c0) {
#pragma unroll
          for (int e = 0; e < 16; e += 2) {
            float a0, a1;
            unpack2(v2[(c0 + e) >> 1], a0, a1);
            // u = c + r' = x / (2 theta) + 1/2;  eta_{1/2}(u - 1/2) = (u - 1/2) - (sat(u) - 1/2): where 0 <= u <= 1 the
            // two terms are the same float and the difference is an exact zero
            const F2 u2 = add2(pack2(a0, a1), pack2u(r[e], r[e + 1]));
            float u0, u1;
            unpack2(u2, u0, u1);
            const F2 s2 = pack2(add_sat(u0, 0.f), add_sat(u1, 0.f));
            v2[(c0 + e) >> 1] = mul2(sub2(add2(u2, mh2), add2(s2, mh2)), tt2);
          }
        };
        {
          uint32_t r0[16], r1[16];
          tmem_ld_32x32b_x16(acc_addr, r0);
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 32) {
            tmem_wait_ld();
            tmem_ld_32x32b_x16(acc_addr + c0 + 16, r1);
            last16(r0, c0);
            tmem_wait_ld();
            if (c0 + 32 < D) tmem_ld_32x32b_x16(acc_addr + c0 + 32, r0);
            last16(r1, c0 + 16);
            if (!has_psi && (c0 + 32) % 64 == 0) stage_box(c0 / 64);      // this box of the output is final
          }
          staged = !has_psi;
        }
        if (has_psi) {
          publish(0);
          w.wait(&bars->r_full[t], phase & 1, 232); ++phase;
          tc_fence_after();
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 16) {
            uint32_t r[16];
            tmem_ld_32x32b_x16(acc_addr + c0, r);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; e += 2) v2[(c0 + e) >> 1] = pack2u(r[e], r[e + 1]);
          }
        }
      }
      if (!kUntied && T > 0 && !scaled_units) {
        // layer t uses theta[t * theta_stride + h] (stride 0: one threshold for all layers).  The accumulator is
        // biased by kappa = theta of layer 0 and the registers hold b = alpha - kappa throughout.
        const uint32_t op_addr = tbase + C::kColS;
        // accumulator := kappa (r_0 = kappa + z B), and z as the bf16 A operand
        {
          uint32_t tb[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) tb[e] = __float_as_uint(kappa);
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 16) tmem_st_32x32b_x16(acc_addr + c0, tb);
        }
        publish(0);
#pragma unroll
        for (int i = 0; i < D / 2; ++i) v2[i] = pack2(-kappa, -kappa);  // alpha^0 = 0
        // per_layer is a compile-time tag: with one threshold for all layers theta_t - kappa = 0 and the add of it
        // is left out of the inner loop
        auto iterate = [&](auto per_layer) {
          for (int it = 0; it + 1 < T; ++it) {
            const float th = per_layer.value ? theta[(int64_t)it * theta_stride + h] : kappa;
            const float inv2th = th > 0.f ? 0.5f / th : 0.f;        // theta = 0: sat(1/2) = 1/2 and eta(x) = x
            const F2 m2th2 = pack2(-2.f * th, -2.f * th);
            const F2 dk2 = pack2(th - kappa, th - kappa);
            w.wait(&bars->r_full[t], phase & 1, 230); ++phase;
            tc_fence_after();
            // 16 columns at a time, the next piece's TMEM load in flight while this one is shrunk
            auto shrink16 = [&](const uint32_t (&r)[16], int c0) {
              uint32_t pk[8];
#pragma unroll
              for (int e = 0; e < 16; e += 2) {
                const F2 r2 = pack2u(r[e], r[e + 1]);
                const F2 x2 = add2(v2[(c0 + e) >> 1], r2);               // alpha^t S + z B
                float x0, x1;
                unpack2(x2, x0, x1);
                if (kMasks) {                                                  // the sign bit of theta - |x| is the decision
                  mw[c0 >> 5] = __funnelshift_l(__float_as_uint(th - fabsf(x0)), mw[c0 >> 5], 1);
                  mw[c0 >> 5] = __funnelshift_l(__float_as_uint(th - fabsf(x1)), mw[c0 >> 5], 1);
                  if (signs) {
                    sw[c0 >> 5] = __funnelshift_l(__float_as_uint(x0), sw[c0 >> 5], 1);
                    sw[c0 >> 5] = __funnelshift_l(__float_as_uint(x1), sw[c0 >> 5], 1);
                  }
                }
                const F2 t2 = pack2(fma_sat(x0, inv2th, 0.5f), fma_sat(x1, inv2th, 0.5f));
                F2 bn = fma2(t2, m2th2, x2);                             // eta_theta(x) - theta
                F2 dn = fma2(t2, m2th2, r2);                             // alpha^{t+1} - alpha^t
                if (per_layer.value) { bn = add2(bn, dk2); dn = add2(dn, dk2); }   // ... - kappa
                v2[(c0 + e) >> 1] = bn;
                float d0, d1;
                unpack2(dn, d0, d1);
                pk[e >> 1] = pack_bf16(d0, d1);
              }
              tmem_st_32x32b_x8(op_addr + c0 / 2, pk);
              if (kKeep && arow != nullptr) {                                 // alpha^{t+1} = b + kappa
                uint32_t pa[8];
#pragma unroll
                for (int e = 0; e < 16; e += 2) {
                  float a0, a1;
                  unpack2(v2[(c0 + e) >> 1], a0, a1);
                  pa[e >> 1] = pack_bf16(a0 + kappa, a1 + kappa);
                }
                st_global_v8(arow + (int64_t)(it + 1) * alpha_slot + c0, pa);
              }
            };
            uint32_t r0[16], r1[16];
            tmem_ld_32x32b_x16(acc_addr, r0);
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
              tmem_wait_ld();
              tmem_ld_32x32b_x16(acc_addr + c0 + 16, r1);
              shrink16(r0, c0);
              tmem_wait_ld();
              if (c0 + 32 < D) tmem_ld_32x32b_x16(acc_addr + c0 + 32, r0);
              shrink16(r1, c0 + 16);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&bars->a_full[t]);
            store_masks(it);
          }
        };
        if (theta_stride != 0) iterate(std::true_type{}); else iterate(std::false_type{});
        const float th = theta[(int64_t)(T - 1) * theta_stride + h];
        // last iteration, exact shrinkage: alpha^T = eta_theta(x)
        w.wait(&bars->r_full[t], phase & 1, 231); ++phase;
        tc_fence_after();
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 16) {
          uint32_t r[16];
          tmem_ld_32x32b_x16(acc_addr + c0, r);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 16; e += 2) {
            float b0, b1;
            unpack2(v2[(c0 + e) >> 1], b0, b1);
            const float x0 = b0 + __uint_as_float(r[e]), x1 = b1 + __uint_as_float(r[e + 1]);
            if (kMasks) {
              mw[c0 >> 5] = __funnelshift_l(__float_as_uint(th - fabsf(x0)), mw[c0 >> 5], 1);
              mw[c0 >> 5] = __funnelshift_l(__float_as_uint(th - fabsf(x1)), mw[c0 >> 5], 1);
              if (signs) {
                sw[c0 >> 5] = __funnelshift_l(__float_as_uint(x0), sw[c0 >> 5], 1);
                sw[c0 >> 5] = __funnelshift_l(__float_as_uint(x1), sw[c0 >> 5], 1);
              }
            }
            v2[(c0 + e) >> 1] = pack2(x0 - fminf(fmaxf(x0, -th), th), x1 - fminf(fmaxf(x1, -th), th));
          }
        }
        store_masks(T - 1);
        if (kKeep && arow != nullptr) {
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 16) {
            uint32_t pa[8];
#pragma unroll
            for (int e = 0; e < 16; e += 2) {
              float a0, a1;
              unpack2(v2[(c0 + e) >> 1], a0, a1);
              pa[e >> 1] = pack_bf16(a0, a1);
            }
            st_global_v8(arow + (int64_t)T * alpha_slot + c0, pa);
          }
        }
        if (has_psi) {
          publish(0);
          w.wait(&bars->r_full[t], phase & 1, 232); ++phase;
          tc_fence_after();
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 16) {
            uint32_t r[16];
            tmem_ld_32x32b_x16(acc_addr + c0, r);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; e += 2) v2[(c0 + e) >> 1] = pack2u(r[e], r[e + 1]);
          }
        }
      }
      if (kStaged && !staged)
#pragma unroll
        for (int bx = 0; bx < C::kDBoxes; ++bx) stage_box(bx);
      if (!kStaged && out != nullptr && grow_m < nq && !w.dead && *(volatile int*)&bars->abort == 0) {
        // a row is a multiple of 128 bytes; where the output is 32-byte aligned every store covers whole
        // 32-byte sectors (the lanes of a warp write different rows), otherwise 16-byte stores
        __nv_bfloat16* orow = out + ((int64_t)bh * nq + grow_m) * D;
        if ((reinterpret_cast<uintptr_t>(out) & 31u) == 0) {
#pragma unroll
          for (int c = 0; c < D / 16; ++c) {
            uint32_t pk[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              float x0, x1;
              unpack2(v2[c * 8 + u], x0, x1);
              pk[u] = pack_bf16(x0, x1);
            }
            st_global_v8(orow + c * 16, pk);
          }
        } else {
          uint4* o = reinterpret_cast<uint4*>(orow);
#pragma unroll
          for (int c = 0; c < D / 8; ++c) {
            float x[8];
#pragma unroll
            for (int u = 0; u < 4; ++u) unpack2(v2[c * 4 + u], x[2 * u], x[2 * u + 1]);
            o[c] = make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]), pack_bf16(x[6], x[7]));
          }
        }
      }
    }
    if (kStaged && lane == 0) bulk_wait_group0();               // the stores are done before the kernel ends
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(tmem, C::kTmemCols);
}

template <int D, bool kUntied, int kRec = 0, bool kFold = false>
cudaError_t launch(csat_ctx* c, const void* Q, void* out, cudaStream_t s, int T, float* lse_out, int lse_stride,
                   __nv_bfloat16* z_out = nullptr, uint32_t* mask_out = nullptr, __nv_bfloat16* alpha_out = nullptr) {
  using C = Cfg<D, kRec == 0>;
  const Params& p = c->p;
  CUtensorMap tq;
  const uint64_t qd[3] = {(uint64_t)D, (uint64_t)p.nq, (uint64_t)(p.B * p.H)};
  const uint64_t qs[2] = {(uint64_t)D * 2, (uint64_t)p.nq * D * 2};
  const uint32_t qb[3] = {64, (uint32_t)kRows, 1};
  cudaError_t e;
  if ((e = make_tmap_bf16_3d(&tq, Q, qd, qs, qb)) != cudaSuccess) return e;
  CUtensorMap to = tq;                                          // the output has the shape of Q; boxes of one warp's rows
  const uint32_t ob[3] = {64, 32, 1};
  if (kRec == 0 && out != nullptr && (e = make_tmap_bf16_3d(&to, out, qd, qs, ob)) != cudaSuccess) return e;
  static DeviceFlags smem_opt_in;
  if (!smem_opt_in.test(c->device)) {
    // setmaxnreg moves registers inside the pool the CTA is launched with (threads x the compiled register count); the
    // kernel asks for 2 x 128 x 224 + 128 x 56 of them, and a request the pool cannot satisfy would wait forever
    cudaFuncAttributes fa;
    if ((e = cudaFuncGetAttributes(&fa, attend_recover_sm100_kernel<D, kUntied, kRec, kFold>)) != cudaSuccess) return e;
    if ((int64_t)fa.numRegs * kThreads < (int64_t)kTiles * kTileThreads * kComputeRegs + 128 * kControlRegs)
      return cudaErrorLaunchOutOfResources;
  }
  if ((e = ensure_dynamic_smem(attend_recover_sm100_kernel<D, kUntied, kRec, kFold>, (int)C::kSmemBytes, c->device, smem_opt_in)) !=
      cudaSuccess)
    return e;
  const double scale = p.scale > 0.0 ? p.scale : 1.0 / sqrt((double)D);
  const float scale_log2 = (float)(scale * 1.4426950408889634);
  // persistent CTAs, one per SM, each walking the work items (256 queries of one (batch, head)) it owns
  const int64_t rows_per_item = kTiles * kRows;
  const int64_t items_x = (p.nq + rows_per_item - 1) / rows_per_item;
  const int64_t n_items = items_x * (c->bh_cnt ? c->bh_cnt : p.B * p.H);    // all (batch, head) pairs, or a sub-range
  if (n_items > (int64_t)1 << 30) return cudaErrorInvalidValue;
  const int sms = c->sms;
  const unsigned grid = (unsigned)(n_items < sms ? n_items : sms);
  // programmatic dependent launch: the kernel may be scheduled while the compression kernel before it still runs
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, attend_recover_sm100_kernel<D, kUntied, kRec, kFold>, tq, c->tmap_kv,
                            kUntied ? c->tmap_lmats : c->tmap_mats, to, c->tmap_vb, (__nv_bfloat16*)out, c->thr(), c->thr_stride(),
                            (int)p.nq, (int)p.m, (int)p.H, T, c->psi ? 1 : 0, scale_log2, (int)items_x, (int)n_items,
                            (int)c->bh0, c->status, lse_out, lse_stride, z_out, mask_out, alpha_out,
                            (int64_t)(p.B * p.H * p.nq * p.d), alpha_out != nullptr ? c->bw_signbits : nullptr);
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
  const uint32_t sb[3] = {64, 32, 1};                           // the compression kernel's stores: one warp's rows
  if ((e = make_tmap_bf16_3d(&c->tmap_kv_st, c->kv, kd, ks, sb)) != cudaSuccess) return e;
  // V~ B behind K~|V~: [B H, m, d]
  const __nv_bfloat16* vb = (const __nv_bfloat16*)c->kv + (size_t)(p.B * p.H * p.m * 2 * p.d);
  const uint64_t vd[3] = {(uint64_t)p.d, (uint64_t)p.m, (uint64_t)(p.B * p.H)};
  const uint64_t vs[2] = {(uint64_t)p.d * 2, (uint64_t)p.m * p.d * 2};
  const uint32_t vbx[3] = {64, (uint32_t)kMC, 1};
  if ((e = make_tmap_bf16_3d(&c->tmap_vb, vb, vd, vs, vbx)) != cudaSuccess) return e;
  if ((e = make_tmap_bf16_3d(&c->tmap_vb_st, vb, vd, vs, sb)) != cudaSuccess) return e;
  const uint64_t md[3] = {(uint64_t)p.d, (uint64_t)p.d, (uint64_t)(p.H * 3)};
  const uint64_t ms[2] = {(uint64_t)p.d * 2, (uint64_t)p.d * p.d * 2};
  const uint32_t mb[3] = {64, (uint32_t)p.d, 1};
  return make_tmap_bf16_3d(&c->tmap_mats, c->mats_bf16, md, ms, mb);
}

// tensor map over the per-layer operands [H (2 L + 1)][d][d] of untied layers
cudaError_t make_layer_weights_tmap(csat_ctx* c) {
  const Params& p = c->p;
  const uint64_t md[3] = {(uint64_t)p.d, (uint64_t)p.d, (uint64_t)(p.H * (2 * c->w_layers + 1))};
  const uint64_t ms[2] = {(uint64_t)p.d * 2, (uint64_t)p.d * p.d * 2};
  const uint32_t mb[3] = {64, (uint32_t)p.d, 1};
  return make_tmap_bf16_3d(&c->tmap_lmats, c->lmats_bf16, md, ms, mb);
}

cudaError_t launch_sm100_attend_recover(csat_ctx* c, const void* Q, void* out, cudaStream_t s, int* launches) {
  *launches += 1;
  // with untied layers and T > 0 the per-layer kernel; the set-up has then built its operands for exactly T layers
  if (c->w_S && c->w_untied && c->p.T > 0)
    return c->p.d == 64 ? launch<64, true>(c, Q, out, s, c->p.T, nullptr, 0) : launch<128, true>(c, Q, out, s, c->p.T, nullptr, 0);
  // Long jobs with the ISTA-derived decoder (one S, B and one positive threshold for all layers) fold B into the
  // values first: one more small launch, which only pays where the attention kernel walks several items per SM
  // (measured: from ~2 tiles of 128 queries per SM at d = 128, where a layer's hand-over chain is long, from ~8 at
  // d = 64).  The choice looks at the context's whole job, not at the launch's range of (batch, head) pairs, so that
  // a forward cut into sub-range launches returns the same bits as one launch.
  const int64_t tiles = ((c->p.nq + kRows - 1) / kRows) * c->p.B * c->p.H;
  if (!c->w_S && c->p.T >= 2 && c->p.lambda > 0.0 && tiles >= (c->p.d == 128 ? 2 : 8) * (int64_t)c->sms) {
    cudaError_t e = launch_sm100_vfold(c, s, launches);
    if (e != cudaSuccess) return e;
    return c->p.d == 64 ? launch<64, false, 0, true>(c, Q, out, s, c->p.T, nullptr, 0)
                        : launch<128, false, 0, true>(c, Q, out, s, c->p.T, nullptr, 0);
  }
  return c->p.d == 64 ? launch<64, false>(c, Q, out, s, c->p.T, nullptr, 0) : launch<128, false>(c, Q, out, s, c->p.T, nullptr, 0);
}

// The forward with what the backward pass needs as its only outputs: Z (bf16), the rows' log sum exp and the layers'
// shrinkage decisions (one S, B for all layers; the decoded output itself is not stored)
cudaError_t launch_sm100_attend_for_backward(csat_ctx* c, const void* Q, __nv_bfloat16* z_out, float* lse_out,
                                             int lse_stride, uint32_t* mask_out, __nv_bfloat16* alpha_out,
                                             cudaStream_t s, int* launches, void* out) {
  *launches += 1;
  const bool untied = c->w_S && c->w_untied && c->p.T > 0;      // one S_t, B_t per layer
  const bool d64 = c->p.d == 64;
#define CSAT_REC_LAUNCH(DD, UU, RR) \
  launch<DD, UU, RR>(c, Q, out, s, c->p.T, lse_out, lse_stride, z_out, mask_out, alpha_out)
  if (alpha_out != nullptr) {                   // with the iterates and the sign bits
    if (untied) return d64 ? CSAT_REC_LAUNCH(64, true, 2) : CSAT_REC_LAUNCH(128, true, 2);
    return d64 ? CSAT_REC_LAUNCH(64, false, 2) : CSAT_REC_LAUNCH(128, false, 2);
  }
  if (untied) return d64 ? CSAT_REC_LAUNCH(64, true, 1) : CSAT_REC_LAUNCH(128, true, 1);
  return d64 ? CSAT_REC_LAUNCH(64, false, 1) : CSAT_REC_LAUNCH(128, false, 1);
#undef CSAT_REC_LAUNCH
}

}  // namespace csat
