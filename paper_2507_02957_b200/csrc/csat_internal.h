// Internal declarations shared by the translation units of libcsat (not part of the ABI).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <atomic>
#include <string>
#include <vector>

#include "csat.h"

namespace csat {

// n is padded to a multiple of this in the library's Phi storage, so that every row of Phi
// starts on a 128-byte boundary for both dtypes and whole 64-token chunks can be staged.
constexpr int64_t kPhiColPad = 64;

inline int64_t round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

// The opt-in to large dynamic shared memory is a per-device attribute of a kernel: one flag per device ordinal
// (kernels keep one DeviceFlags each).  Beyond kMaxTracked ordinals the attribute is simply set on every launch.
struct DeviceFlags {
  static constexpr int kMaxTracked = 64;
  std::atomic<uint64_t> done{0};
  bool test(int dev) const { return dev >= 0 && dev < kMaxTracked && ((done.load(std::memory_order_acquire) >> dev) & 1u); }
  void set(int dev) { if (dev >= 0 && dev < kMaxTracked) done.fetch_or((uint64_t)1 << dev, std::memory_order_release); }
};

template <typename Kernel>
cudaError_t ensure_dynamic_smem(Kernel* kernel, int bytes, int device, DeviceFlags& flags) {
  if (flags.test(device)) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) flags.set(device);
  return e;
}

struct Params {            // plain values kernels need
  int64_t n, m, d, H, B, nq;
  int64_t n_pad;           // padded row length of Phi
  int dtype;               // CSAT_DTYPE_*
  int ensemble;            // CSAT_ENSEMBLE_*
  int separate_phi;        // 1: Phi holds 2H matrices, Phi_K of every head then Phi_V of every head
  int T;
  double lambda, step, scale;
  uint64_t seed;
};

}  // namespace csat

struct csat_ctx {
  csat::Params p;
  int64_t phi_heads() const { return p.H * (p.separate_phi ? 2 : 1); }   // matrices stored in phi
  int device = 0;
  int sms = 148;              // multiprocessors of `device` (grid size of the persistent kernels)
  bool broken = false;        // a setter's re-allocation failed: compute calls are refused until a setter succeeds
  int force_simt = 0;         // diagnostic: 1 = FFMA kernels for everything, 2 = for attention/recovery only

  // library-owned device memory
  void* phi = nullptr;        // [H, m, n_pad] dtype
  void* kv = nullptr;         // K~|V~ workspace [B, H, m, 2d] dtype (row r: K~_r then V~_r)
  void* psi = nullptr;        // [Hpsi, d, d] dtype (user dictionary), null = identity
  void* dmat = nullptr;       // [H, d, d] dtype (user decoder matrix), null = Phi block
  bool psi_per_head = false;
  bool phi_generated = true;  // phi holds the seeded ensemble (false once csat_set_phi replaced it)
  // structured Hadamard ensemble: what the fast-transform compression needs instead of the dense matrix.
  // had_signs: the column-sign bit stream (bit e % 32 of word e / 32, e = head * n + column); had_ab: (u0, u1) per
  // head, row r of Phi_h is row ((2 u0 + 1) r + u1) mod N of the Hadamard matrix.  Written with the ensemble.
  uint32_t* had_signs = nullptr;
  uint32_t* had_ab = nullptr;
  size_t had_bytes_signs = 0, had_bytes_ab = 0;
  int hadamard_transform = 0; // CSAT_HADAMARD_TRANSFORM
  int debug_canary = 0;       // CSAT_DEBUG_CANARY: the K~|V~ workspace is filled with NaN bit patterns before every compression
  CUtensorMap tmap_phi;       // TMA view of phi for the tensor-core compress kernel (bf16, d in {64,128})
  bool tmap_phi_valid = false;
  CUtensorMap tmap_kv;        // TMA view of the K~|V~ workspace
  CUtensorMap tmap_kv_st;     // the same workspace in boxes of 32 rows (the compression kernel's stores)
  CUtensorMap tmap_vb;        // V~ B [B H, m, d] behind K~|V~ in the same allocation (bf16 contexts), as the attention phase loads it
  CUtensorMap tmap_vb_st;     // the same in boxes of 32 rows (the stores of the kernel that forms it)
  CUtensorMap tmap_mats;      // TMA view of mats_bf16
  // bf16 operand copies of the decoder matrices for the tensor-core path: [H][3][d][d], each stored
  // [output column][k] (k contiguous): 0 = -mu G = S - I (symmetric for ISTA), 1 = B^T = (mu M)^T, 2 = Psi
  __nv_bfloat16* mats_bf16 = nullptr;
  double* Mf64 = nullptr;     // [H, d, d] scratch of the decoder set-up
  double* Gf64 = nullptr;     // [H, d, d]
  float* S_dec = nullptr;     // [H, d, d]  I - mu G
  float* B_dec = nullptr;     // [H, d, d]  mu M
  float* psi_f32 = nullptr;   // [H, d, d]  Psi as float (row-major), only when psi != null
  float* theta = nullptr;     // [H] (ISTA-derived) 
  // supplied LISTA weights (csat_set_lista_weights / csat_set_lista_layer_weights); null = ISTA-derived decoder
  void* w_S = nullptr;        // [H, d, d] dtype, or [w_layers, H, d, d] when w_untied
  void* w_B = nullptr;        // the same
  float* w_theta = nullptr;   // [w_layers, H]
  int w_layers = 0;
  bool w_untied = false;      // one S_t, B_t per layer
  // untied layers, derived by the decoder set-up: float32 copies for the FFMA kernels and the bf16 tensor-core
  // operands [H][2 w_layers + 1][d][d], each stored [output column][k]: 2t = S_t - I, 2t + 1 = B_t, last = Psi
  float* Sl_dec = nullptr;    // [w_layers, H, d, d]
  float* Bl_dec = nullptr;    // [w_layers, H, d, d]
  __nv_bfloat16* lmats_bf16 = nullptr;
  CUtensorMap tmap_lmats;     // TMA view of lmats_bf16
  size_t w_mat_count() const { return (size_t)(w_untied ? w_layers : 1) * (size_t)(p.H * p.d * p.d); }
  float* mu = nullptr;        // [H]
  int* status = nullptr;      // device status word (0 = ok)
  // float32 scratch of csat_backward, allocated by its first call: dZ [B,H,n_q,d], (L, D) [B,H,n_q,2],
  // dK~|dV~ [B,H,m,2d]
  // and the float32 transposes of the decoder matrices [2][layers or 1][H][d][d]
  float* bw_dZ = nullptr; float* bw_LD = nullptr; float* bw_dKV = nullptr; float* bw_WT = nullptr;
  __nv_bfloat16* bw_dKV16 = nullptr;     // bf16 copy of dK~|dV~ (operand of the tensor-core Phi^T product)
  __nv_bfloat16* bw_dZ16 = nullptr;      // bf16 copy of dZ (operand of the tensor-core dK~|dV~ stage)
  __nv_bfloat16* bw_Z16 = nullptr;       // Z = A~ V~ as the forward rounds it (tensor-core per-query stages)
  uint32_t* bw_maskbits = nullptr;       // the forward's decisions, one bit per (b, h, layer, query, column)
  size_t bw_bytes_Z16 = 0, bw_bytes_maskbits = 0;
  size_t bw_bytes_dZ = 0, bw_bytes_LD = 0, bw_bytes_dKV = 0, bw_bytes_WT = 0, bw_bytes_dKV16 = 0, bw_bytes_dZ16 = 0;
  // CSAT_KEEP_MASKS: the shrinkage decisions of the most recent csat_backward, one word per (b, h, query, column),
  // bit t = |x_t| > theta_t
  bool keep_masks = false;
  bool have_masks = false;
  uint32_t* bw_masks = nullptr;
  size_t bw_bytes_masks = 0;
  // CSAT_WEIGHT_GRADS: csat_backward also forms the gradients of the decoder's parameters.  The forward kernel leaves
  // the iterates alpha^0 .. alpha^T (bf16 [T+1][B,H,n_q,d]) and the recurrence kernel the dx_t (bf16 [T][B,H,n_q,d]);
  // bw_wpart = per-CTA partial sums [splits][H][2][d][d], bw_thpart = [chunks][T][H],
  // bw_wgrad = dS [H,d,d] | dB [H,d,d] | dPsi [d,d] | dtheta [T,H]
  bool weight_grads = false;
  bool have_wgrads = false;
  bool have_dkv16 = false;       // bw_dKV16 holds dK~|dV~ of the most recent csat_backward (tensor-core path)
  // CSAT_SAVE_FOR_BACKWARD: csat_forward runs the recording variant of its kernel and leaves K~|V~, Z, the softmax
  // statistics and the decisions for the next csat_backward (saved_valid until anything changes them)
  bool save_for_backward = false, saved_valid = false, saved_alpha = false;
  bool reuse_saved = false;      // set by csat_backward around launch_backward
  __nv_bfloat16* bw_alpha16 = nullptr; __nv_bfloat16* bw_dx16 = nullptr;
  float* bw_wpart = nullptr; float* bw_thpart = nullptr; float* bw_wgrad = nullptr;
  uint32_t* bw_signbits = nullptr;       // sign bit of every x_t, in the layout of bw_maskbits (for dtheta)
  size_t bw_bytes_alpha16 = 0, bw_bytes_dx16 = 0, bw_bytes_wpart = 0, bw_bytes_thpart = 0, bw_bytes_wgrad = 0;
  size_t bw_bytes_signbits = 0;
  // staging for csat_forward_host
  void* stage_q = nullptr; void* stage_k = nullptr; void* stage_v = nullptr; void* stage_o = nullptr;
  size_t stage_bytes_q = 0, stage_bytes_kv = 0;
  // streams (copy in, compute, copy out) and events of the pipelined csat_forward_host
  static constexpr int kPipeEvents = 2 + 2 * 64;
  cudaStream_t pipe_stream[3] = {};
  cudaEvent_t pipe_event[kPipeEvents] = {};
  bool pipe_ready = false;

  // per-kernel CUDA-event timing of the most recent `prof_slots` forward calls (CSAT_PROFILE)
  static constexpr int kProfMaxKernels = 8;
  int prof_slots = 0;
  int64_t prof_calls = 0;                       // forward calls since profiling was switched on
  std::vector<cudaEvent_t> prof_events;         // [slots][kProfMaxKernels + 1]
  std::vector<int> prof_ids;                    // [slots][kProfMaxKernels]
  std::vector<int> prof_count;                  // [slots]

  // thresholds the kernels read: theta_t of head h at thr()[t * thr_stride() + h]
  const float* thr() const { return w_S ? w_theta : theta; }
  int thr_stride() const { return (w_S && w_layers > 1) ? (int)p.H : 0; }

  // (batch, head) pairs [bh0, bh0 + bh_cnt) the next kernel launches cover; bh_cnt = 0 means all B*H.  A sub-range
  // may cross from one batch element into the next (csat_forward_host pipelines copies and compute run by run)
  int64_t bh0 = 0, bh_cnt = 0;

  bool decoder_dirty = true;
  bool have_forward = false;
  int last_launches = 0;
  size_t bytes = 0;
  std::string err;
};

namespace csat {

size_t elt_size(int dtype);

// phi_gen.cu
cudaError_t launch_phi_gen(void* phi, const Params& p, cudaStream_t s);
// sign stream words [ceil(heads n / 32)] and (u0, u1) per head [2 heads] of the structured Hadamard ensemble
cudaError_t launch_hadamard_tables(uint32_t* sign_words, uint32_t* ab, const Params& p, cudaStream_t s);

// fwht_compress.cu : K~|V~ of the structured Hadamard ensemble by a fast Walsh-Hadamard transform
bool fwht_compress_supported(const csat_ctx* c);
cudaError_t launch_fwht_compress(csat_ctx* c, const void* K, const void* V, cudaStream_t s, int* launches);
cudaError_t launch_phi_pack(void* phi_padded, const void* phi_dense, const Params& p, cudaStream_t s);
cudaError_t launch_phi_unpack(void* phi_dense, const void* phi_padded, const Params& p, cudaStream_t s);

// decoder_setup.cu : derives S_dec, B_dec, theta, mu (and psi_f32) on the stream; returns #launches
cudaError_t launch_decoder_setup(csat_ctx* c, cudaStream_t s, int* launches);

// simt_forward.cu : plain FFMA path (fp32 accumulate), both storage types
// (phi_j0, n_len, partial): token-sharded use, see compress_sm100.cu; defaults = the whole sequence into the workspace
cudaError_t launch_simt_compress(csat_ctx* c, const void* K, const void* V, cudaStream_t s, int* launches,
                                 int64_t phi_j0 = 0, int64_t n_len = 0, float* partial = nullptr);
// workspace := sum over r < R of partials[r] (float32 [B,H,m,2d] each), added in the order r = 0, 1, ..., rounded
// once to the context's storage type
cudaError_t launch_reduce_partials(csat_ctx* c, const float* partials, int R, cudaStream_t s, int* launches);
cudaError_t launch_simt_attend_recover(csat_ctx* c, const void* Q, void* out, cudaStream_t s, int* launches);

// compress_sm100.cu : tcgen05 / TMEM / TMA compression (bf16, d in {64, 128})
cudaError_t make_phi_tmap(csat_ctx* c);
cudaError_t launch_wait_timeout_selftest(csat_ctx* c, unsigned long long limit_ns, cudaStream_t s);
cudaError_t launch_sm100_vfold(csat_ctx* c, cudaStream_t s, int* launches);
cudaError_t launch_sm100_compress(csat_ctx* c, const void* K, const void* V, cudaStream_t s, int* launches,
                                  int64_t phi_j0 = 0, int64_t n_len = 0, float* partial = nullptr);

// attend_recover_sm100.cu : tcgen05 compressed attention + recovery (bf16, d in {64, 128})
cudaError_t make_attend_tmaps(csat_ctx* c);
cudaError_t make_layer_weights_tmap(csat_ctx* c);
cudaError_t launch_sm100_attend_recover(csat_ctx* c, const void* Q, void* out, cudaStream_t s, int* launches);
// the forward run for the backward pass: z_out [B,H,n_q,d] bf16 = Z, lse_out[row * lse_stride] = log sum exp of the
// row's scores, mask_out [B,H,T,n_q,d/32] = the layers' decisions |x_t| > theta_t (column c: word c / 32, bit 31 - c % 32)
// alpha_out (may be null): the iterates alpha^1 .. alpha^T as bf16 into slots 1 .. T of [T+1][B,H,n_q,d]
// out (may be null): the decoded output as well (a forward that saves for the backward)
cudaError_t launch_sm100_attend_for_backward(csat_ctx* c, const void* Q, __nv_bfloat16* z_out, float* lse_out,
                                             int lse_stride, uint32_t* mask_out, __nv_bfloat16* alpha_out,
                                             cudaStream_t s, int* launches, void* out = nullptr);

// wgrad_sm100.cu : gradients of the decoder's parameters from the stored iterates and dx_t (bf16, d in {64, 128}, one
// S, B for all layers) into bw_wgrad; wgrad_splits = CTAs per head of its contraction kernel
int wgrad_splits(const csat_ctx* c);
cudaError_t launch_sm100_wgrad(csat_ctx* c, const void* G, cudaStream_t s, int* launches);

// bwd_rows_sm100.cu : the per-query stages of the backward on the tensor cores (bf16, d in {64, 128}, one S, B
// for all layers).  recur: Z, G -> dZ (bf16 into bw_dZ16), D = <dZ, Z> (into bw_LD), optionally the masks;
// dq: Q, dZ, L, D, K~|V~ -> dQ
cudaError_t launch_sm100_bwd_recur(csat_ctx* c, const void* G, cudaStream_t s, int* launches);
cudaError_t launch_sm100_bwd_dq(csat_ctx* c, const void* Q, void* dQ, cudaStream_t s, int* launches);

// project_sm100.cu : input projections; one launch applies columns [col0, col0 + ncols) of W [dm, 3 H d] to
// X [B, n_tok, dm] and writes the heads of Q / K / V those columns belong to
cudaError_t launch_project(csat_ctx* c, const void* X, const void* W, int64_t n_tok, int64_t dm, int col0, int ncols,
                           void* Q, void* K, void* V, cudaStream_t s, int* launches);

// backward_simt.cu : gradients with respect to Q, K, V; K~|V~ of the same K, V must be in the workspace
cudaError_t launch_backward(csat_ctx* c, const void* Q, const void* G, void* dQ, void* dK, void* dV, cudaStream_t s,
                            int* launches);

// bwd_cols_sm100.cu : dK~ = scale dS^T Q, dV~ = P^T dZ on the tensor cores (bf16, d in {64, 128}); reads bw_dZ16,
// bw_LD and the K~|V~ workspace, writes bw_dKV and bw_dKV16
cudaError_t launch_sm100_bwd_cols(csat_ctx* c, const void* Q, cudaStream_t s, int* launches);

// phiT_sm100.cu : dK = Phi_K^T dK~, dV = Phi_V^T dV~ on the tensor cores (bf16, d in {64, 128}); g16 = dK~|dV~ as bf16
cudaError_t launch_sm100_phiT(csat_ctx* c, const void* g16, void* dK, void* dV, cudaStream_t s, int* launches);

// phigrad_sm100.cu : dPhi [H or 2H, m, n] float32 = sum over the batch of dK~ K^T (+ dV~ V^T), from bw_dKV16
cudaError_t launch_sm100_phigrad(csat_ctx* c, const void* K, const void* V, float* dPhi, cudaStream_t s, int* launches);

// copies K~ or V~ out of the interleaved workspace: dst [B,H,m,d]
cudaError_t launch_split_kv(const csat_ctx* c, void* kt, void* vt, cudaStream_t s);

}  // namespace csat
