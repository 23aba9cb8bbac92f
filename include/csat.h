/*
 * csat.h -- C-ABI of the B200 (sm_100a) compressed-sensing attention (CSAT) forward.
 *
 * What the library computes, per (batch b, head h), in the notation of the paper's
 * "Mathematical Framework" section (tokens are rows):
 *
 *   K~ = Phi_h K,  V~ = Phi_h V            compression equation, Phi_h in R^{m x n}
 *   A~ = softmax(Q K~^T / sqrt(d_k))       approximate attention matrix, softmax over the m measurements
 *   Z  = A~ V~                             compressed attention output, n_q x d_k
 *   alpha^{t+1} = eta_theta(S alpha^t + B Z_i),  t = 0..T-1, alpha^0 = 0      LISTA recurrence
 *   C^_i = Psi alpha^_i                    reconstruction equation; out = C^
 *
 * with the recurrence instantiated as ISTA for  min 1/2 ||z - alpha M^T||^2 + lambda ||alpha||_1,
 * M = D Psi, D = leading d x d block of Phi_h unless supplied, mu = 1/L^ with
 * L^ = max absolute row sum of M^T M unless supplied, S = I - mu M^T M, B = mu M, theta = mu lambda.
 * T = 0 disables recovery: out = Z.
 *
 * Conventions common to every call
 *   - All tensor pointers are DEVICE pointers unless the parameter is named *_host.
 *     They must be 16-byte aligned and contiguous in the stated layout, innermost index last.
 *   - Element type of Q, K, V, out, Phi, Psi, D is the context's CSAT_DTYPE
 *     (CSAT_DTYPE_BF16: 16-bit bfloat16; CSAT_DTYPE_FP32: IEEE binary32).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Calls enqueue work on it and return; they do not synchronise unless stated.
 *   - The caller owns every buffer it passes in and keeps it alive and unmodified until the
 *     stream has passed the call.  The library owns everything it allocates (Phi, the K~|V~
 *     workspace, decoder matrices) and frees it in csat_destroy.
 *   - Every call returns a CSAT_* status (never throws, never aborts).  A text for the most
 *     recent failure is kept per context (csat_last_error).
 *   - A context is used by one host thread at a time; different contexts are independent.
 *   - Results are deterministic: same seed, parameters and inputs give bit-identical output.
 */
#ifndef CSAT_H_
#define CSAT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct csat_ctx csat_ctx; /* opaque, library-owned */

enum {
  CSAT_OK = 0,
  CSAT_ERR_INVALID_ARG = 1, /* NULL pointer, unknown key, misaligned pointer            */
  CSAT_ERR_SHAPE = 2,       /* a size outside the supported range (see csat_create)      */
  CSAT_ERR_ALLOC = 3,       /* device or host allocation failed                          */
  CSAT_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed; text in last_error     */
  CSAT_ERR_UNSUPPORTED = 5, /* valid request this library has no kernel for              */
  CSAT_ERR_STATE = 6,       /* call not legal in the context's current state             */
  CSAT_ERR_TIMEOUT = 7      /* a bounded device-side wait gave up (reported by the next
                               host call that reads the device status word)              */
};

/* keys of csat_set_i64 / csat_get_i64 */
enum {
  CSAT_BATCH = 1,      /* B, default 1                                                   */
  CSAT_NQ = 2,         /* query tokens n_q, default n (self-attention); cross-attention
                          of text queries over compressed visual keys uses n_q != n     */
  CSAT_DTYPE = 3,      /* CSAT_DTYPE_BF16 (default) or CSAT_DTYPE_FP32                   */
  CSAT_T = 4,          /* recovery iterations (decoder depth t), default 10; 0 = out = Z */
  CSAT_FORCE_SIMT = 5, /* diagnostic: 1 routes bf16 through the plain FFMA kernels, 2 only
                          the attention/recovery stage; 0 (default) = tensor-core kernels */
  CSAT_ENSEMBLE = 7,   /* measurement ensemble: CSAT_ENSEMBLE_GAUSSIAN (default), N(0, 1/m) entries, or
                          CSAT_ENSEMBLE_RADEMACHER, +-1/sqrt(m) entries, or CSAT_ENSEMBLE_HADAMARD (the
                          three ensembles the paper lists after the compression equation):
                          m rows (a r + b mod N, a odd) of the N x N Sylvester-Hadamard matrix, N the
                          smallest power of two >= n, columns truncated to n, a random sign per
                          column, scaled by 1/sqrt(m).  Changing it regenerates Phi from the seed  */
  CSAT_SEPARATE_PHI = 8, /* 0 (default): one matrix per head, Phi_K = Phi_V.  1: separate Phi_K and Phi_V per head
                          (paper: K~ = Phi_K K, V~ = Phi_V V); Phi_V of head h is drawn as head H + h of the
                          same seeded generator, the decoder's default D is the block of Phi_V, and
                          csat_set_phi / csat_get_phi then move [2H, m, n]: the H matrices Phi_K, then the H
                          matrices Phi_V.  Changing it regenerates both from the seed                 */
  CSAT_HADAMARD_TRANSFORM = 10, /* 1: with CSAT_ENSEMBLE_HADAMARD (seeded, not replaced by csat_set_phi) and n <= 16384,
                          csat_forward compresses by a fast Walsh-Hadamard transform over the tokens followed by a
                          gather of the m selected rows (n log n additions per column instead of m n multiply-adds; the
                          same K~, V~ up to the order of the float32 sums).  0 (default): the dense product.  Other
                          ensembles, supplied matrices and longer sequences keep the dense product either way      */
  CSAT_DEBUG_CANARY = 11, /* debugging aid: 1 fills the K~|V~ workspace with NaN bit patterns (one extra memset on the
                          call's stream) before csat_forward / csat_backward compress, so that a row the compression
                          failed to write shows as NaN in the output instead of reusing an earlier call's values  */
  CSAT_SAVE_FOR_BACKWARD = 13, /* 1: csat_forward (tensor-core path: bf16, d in {64, 128}) also keeps what csat_backward
                          needs from it (K~|V~ stay in the workspace; Z, the rows' softmax statistics and one decision
                          bit per layer, query and column go to the backward's scratch, which this then allocates),
                          and the next csat_backward on the same Q, K, V skips its own compression and forward pass
                          (about a third of its time).  The saved state is dropped by any setter and by any other
                          compute call in between; it is the caller's contract that Q, K, V are unchanged.  The
                          forward then costs about a third more.  0 (default): csat_backward recomputes  */
  CSAT_WEIGHT_GRADS = 12, /* 1: csat_backward also forms the gradients with respect to the decoder's parameters (S, B,
                          the thresholds, the dictionary) for csat_get_weight_grads; tensor-core path only (bf16, d in
                          {64, 128}, CSAT_T >= 1), else csat_backward returns
                          CSAT_ERR_UNSUPPORTED.  It then keeps every layer's iterate and its gradient as bf16:
                          (2 T + 1) B H n_q d more 16-bit values of scratch.  0 (default): not formed  */
  CSAT_KEEP_MASKS = 9, /* 1: csat_backward also keeps its shrinkage decisions (one 32-bit word per (b, h, query,
                          column); needs CSAT_T <= 32) for csat_get_backward_masks.  0 (default): not kept  */
  CSAT_PROFILE = 6     /* keep per-kernel CUDA-event times of the last v forward calls
                          (0 = off, default; at most 4096).  Setting it creates/destroys
                          events, so set it outside the timed region                    */
};

/* kernel ids reported by csat_get_profile */
enum {
  CSAT_KERNEL_DECODER_SETUP = 0, /* the three small set-up launches, timed together      */
  CSAT_KERNEL_COMPRESS = 1,      /* K~|V~ = Phi [K|V]                                    */
  CSAT_KERNEL_ATTEND_RECOVER = 2 /* softmax(Q K~^T) V~, recovery iterations, Psi         */
};
enum { CSAT_DTYPE_BF16 = 0, CSAT_DTYPE_FP32 = 1 };
enum { CSAT_ENSEMBLE_GAUSSIAN = 0, CSAT_ENSEMBLE_RADEMACHER = 1, CSAT_ENSEMBLE_HADAMARD = 2 };

/* keys of csat_set_f64 / csat_get_f64 */
enum {
  CSAT_LAMBDA = 1, /* LASSO weight lambda >= 0, default 0.1; per-step threshold is mu*lambda */
  CSAT_STEP = 2,   /* step mu > 0; 0 (default) = 1 / max-abs-row-sum(M^T M), per head       */
  CSAT_SCALE = 3   /* score scale; 0 (default) = 1/sqrt(d)                                   */
};

/*
 * csat_create -- paper: compression equation (Phi in R^{m x n}) and the sentence after it
 * (Gaussian ensemble).  Builds a context for n key/value tokens, m measurements, head size d
 * and H heads on the CURRENT CUDA device, and generates one measurement matrix per head,
 * Phi[h,r,j] ~ N(0, 1/m) i.i.d. from `seed` (Philox4x32-10 keyed by seed, counter = flat element
 * index / 4, Box-Muller; Phi_K = Phi_V = Phi_h, shared over the batch).  With CSAT_ENSEMBLE_RADEMACHER the
 * entries are +-1/sqrt(m): element e takes bit e % 32 of word (e / 32) % 4 of the Philox block with counter
 * (e / 128, 0, 1, 0) as (low, high, third, fourth) words; a set bit means the negative sign.
 * Requires 1 <= m <= n, d >= 1, H >= 1, d <= 256 and d % 8 == 0.  Returns NULL on failure;
 * csat_last_error(NULL) then gives the reason (thread-local).
 * Allocates device memory and synchronises.  Changing CSAT_DTYPE, CSAT_BATCH or CSAT_NQ later
 * re-allocates (and, for CSAT_DTYPE, re-generates Phi from the seed).
 */
csat_ctx* csat_create(int64_t n, int64_t m, int64_t d, int64_t H, uint64_t seed);

/* Frees everything the context owns.  NULL is a no-op.  Synchronises the device. */
int csat_destroy(csat_ctx* ctx);

/* Tunables m, t, Phi, Psi of the paper ("Interpretation and Benefits") that are not fixed at
 * creation.  Setters validate and record; dependent decoder quantities (S, B, theta) are
 * re-derived by the next csat_forward on that call's stream.  Must not be called while a
 * forward of the same context is still running on the device.
 * CSAT_BATCH, CSAT_DTYPE and CSAT_SEPARATE_PHI re-allocate.  If that fails (CSAT_ERR_ALLOC) the context keeps
 * the new value but holds no usable buffers: csat_forward, csat_forward_host, csat_backward, csat_set_phi and the
 * getters of device data return CSAT_ERR_STATE until one of those three setters succeeds (setting the same value
 * again retries the allocation). */
int csat_set_i64(csat_ctx* ctx, int key, int64_t value);
int csat_get_i64(const csat_ctx* ctx, int key, int64_t* value_host);
int csat_set_f64(csat_ctx* ctx, int key, double value);
int csat_get_f64(const csat_ctx* ctx, int key, double* value_host);

/* csat_set_phi / csat_get_phi -- the paper allows measurement matrices that are fixed or trained.
 * phi: [H, m, n] dense, context dtype.  set overrides the seeded matrix (copied into the
 * library's padded storage); get writes the matrix in use.  Enqueued on `stream`. */
int csat_set_phi(csat_ctx* ctx, const void* phi, void* stream);
int csat_get_phi(const csat_ctx* ctx, void* phi_out, void* stream);

/* csat_set_dictionary -- paper: dictionary Psi in R^{d_k x d_k} with C_i = Psi alpha_i.
 * psi: [d, d] (per_head = 0) or [H, d, d] (per_head = 1), context dtype, row-major
 * (Psi[a][b] multiplies alpha_b).  NULL restores Psi = I.  Copied on `stream`. */
int csat_set_dictionary(csat_ctx* ctx, const void* psi, int per_head, void* stream);

/* csat_set_decoder_matrix -- the paper decodes with the values' measurement matrix;
 * the decoder's sensing matrix D is d x d (see file header).  D: [H, d, d], context
 * dtype.  NULL restores the default D_h = Phi_h[0:d, 0:d], which needs m >= d and n >= d
 * (otherwise csat_forward with T > 0 returns CSAT_ERR_SHAPE).  Copied on `stream`. */
int csat_set_decoder_matrix(csat_ctx* ctx, const void* D, void* stream);

/* csat_set_lista_weights -- paper: LISTA recurrence alpha^{t+1} = eta_theta(S alpha^t + B Z_i), whose matrices
 * S, B and shrinkage eta_theta are trained and carry no layer index.  Replaces the ISTA-derived
 * decoder by supplied weights, row-vector convention alpha <- eta(alpha S + z B):
 *   S, Bm   [H, d, d], context dtype, device (row-major: S[a][b] multiplies alpha_a into column b)
 *   theta   [layers, H] float32, device, every entry >= 0; layers = 1 uses the same threshold in every
 *           layer, otherwise layers must equal CSAT_T when csat_forward runs (else CSAT_ERR_STATE).
 * The weights are copied on `stream`.  CSAT_LAMBDA, CSAT_STEP and the decoder matrix D are ignored while supplied
 * weights are in force; the dictionary Psi still applies to the reconstruction.  S = NULL restores the
 * ISTA-derived decoder.  On the bf16 tensor-core path S enters as I - W with W = I - S rounded to bf16. */
int csat_set_lista_weights(csat_ctx* ctx, const void* S, const void* Bm, const float* theta, int layers, void* stream);

/* csat_set_lista_layer_weights -- the same LISTA recurrence with untied layers: layer t has its own matrices,
 * alpha^{t+1} = eta_{theta_t}(alpha^t S_t + z B_t), t = 0 .. layers-1 (the paper's recurrence writes S, B
 * without a layer index; one matrix per layer is the usual generalisation of the unrolled decoder).
 *   S, Bm   [layers, H, d, d], context dtype, device (row-major as in csat_set_lista_weights)
 *   theta   [layers, H] float32, device, every entry >= 0
 * 1 <= layers <= 4096, and layers must equal CSAT_T when csat_forward runs (else CSAT_ERR_STATE).  Copied on `stream`; replaces weights
 * set by csat_set_lista_weights and is cleared by csat_set_lista_weights(ctx, NULL, ...).  csat_get_decoder
 * then returns layer 0's S, B and theta.  On the bf16 tensor-core path every layer is one product
 * [alpha^t | z] [S_t - I ; B_t] with bf16 operands, added to alpha^t kept in float32; the matrices
 * of layer t stream through shared memory while layer t-1 is computed. */
int csat_set_lista_layer_weights(csat_ctx* ctx, const void* S, const void* Bm, const float* theta, int layers,
                                 void* stream);

/* csat_backward -- gradients of csat_forward with respect to its inputs.  The paper's decoder is an
 * unrolled network meant to be trained by backpropagation (its section on the sparse decoder), but the paper
 * prints no backward pass; this is the chain rule through the forward's equations in reverse order, with the
 * derivative of eta_theta taken as 1 where |x| > theta and 0 elsewhere.  Phi, Psi and the decoder weights are
 * constants.
 *   Q [B,H,n_q,d], K, V [B,H,n,d]   the forward's inputs          (context dtype, device)
 *   dOut [B,H,n_q,d]                gradient of the loss with respect to csat_forward's output
 *   dQ [B,H,n_q,d], dK, dV [B,H,n,d]  outputs (context dtype)
 * Unless the last csat_forward ran with CSAT_SAVE_FOR_BACKWARD, nothing of an earlier csat_forward is reused: the
 * call compresses K, V again and recomputes what it needs.  Its
 * first call allocates scratch (B H (n_q (d + 2) + 2 m d) floats and transposed copies of the decoder matrices;
 * bf16 copies of Z, dZ and dK~|dV~ and B H T n_q d / 32 decision words on the tensor-core path; B H n_q d words
 * more with CSAT_KEEP_MASKS; all counted by csat_workspace_bytes).
 * Two paths.  bf16 contexts with d in {64, 128} run every stage on the tensor cores (one S, B for all layers, or one
 * pair per layer streamed through shared memory from the last layer to the first): the forward
 * kernel once more (it keeps Z, the softmax statistics and one decision bit per layer, query and column), the
 * backward recurrence, dQ, the gradients of K~|V~ (P^T dZ, dS^T Q) and the product with Phi^T, all with bf16
 * operands and float32 accumulation; any CSAT_T.  Everything else (float32 contexts, other d) runs
 * float32 FFMA kernels that recompute each query row and keep the decisions of one (query, column) in one word:
 * CSAT_T <= 32 there and with CSAT_KEEP_MASKS.  d <= 256 and B H <= 32767.  Otherwise CSAT_ERR_UNSUPPORTED. */
int csat_backward(csat_ctx* ctx, const void* Q, const void* K, const void* V, const void* dOut, void* dQ, void* dK,
                  void* dV, void* stream);

/* csat_get_backward_masks -- the decisions |x_t| > theta_t the most recent csat_backward took in the layers of the
 * LISTA recurrence (the derivative of eta_theta is 1 or 0 by that decision; the paper prints no backward pass).
 *   masks_out [B, H, n_q, d] uint32, device: bit t of a word = the decision of layer t for that query and column.
 * The derivative of eta_theta is discontinuous, so two implementations in different precisions may decide an entry
 * within rounding distance of its threshold differently; a reference that is given these decisions can be compared
 * with csat_backward's gradients element by element.  Needs CSAT_KEEP_MASKS = 1 before that csat_backward and
 * CSAT_T >= 1, else CSAT_ERR_STATE.  Copied on `stream`. */
int csat_get_backward_masks(const csat_ctx* ctx, uint32_t* masks_out, void* stream);

/* csat_get_weight_grads -- gradients of the loss with respect to the decoder's parameters, formed by the most recent
 * csat_backward with CSAT_WEIGHT_GRADS = 1.  The paper trains S, B, theta (its LISTA recurrence
 * alpha^{t+1} = eta_theta(S alpha^t + B Z_i)) and the dictionary Psi (C^_i = Psi alpha^_i) by backpropagation and
 * prints no backward pass; this is the chain rule with x_t = alpha^t S + Z B in the row-vector form the library
 * computes in (csat_set_lista_weights takes S, B in the same form):
 *   dS     [H, d, d] float32  = sum over layers, queries, batch of (alpha^t)^T dx_t
 *   dB     [H, d, d] float32  = ... of Z^T dx_t
 *          (with one S_t, B_t per layer, csat_set_lista_layer_weights: dS, dB [T, H, d, d], layer by layer, no sum)
 *   dtheta [T, H]    float32  = per layer: - sum of sign(x_t) o dx_t   (one threshold for all layers: add the rows)
 *   dPsi   [d, d]    float32  = sum over heads too of G^T alpha^T (C^ = alpha^T Psi^T); zeros without a dictionary;
 *                               may be NULL
 * with dx_t = d alpha^{t+1} where |x_t| > theta_t, 0 elsewhere.  All device pointers, copied on `stream`.  The
 * products take the iterates and the dx_t rounded to bf16 and accumulate in float32, in a fixed order (the same bits
 * on every run).  CSAT_ERR_STATE if no such csat_backward has run. */
int csat_get_weight_grads(const csat_ctx* ctx, float* dS, float* dB, float* dtheta, float* dPsi, void* stream);

/* csat_backward_phi -- gradient of the loss with respect to the measurement matrices, for a Phi that is learned (the
 * paper allows fixed or learned sensing matrices and prints no backward pass): the chain rule through the
 * compression K~ = Phi K, V~ = Phi V with the decoder's matrices held fixed,
 *   dPhi [H, m, n] float32 = sum over the batch of dK~ K^T + dV~ V^T      (one Phi per head), or
 *   dPhi [2H, m, n]: the H matrices dPhi_K = sum dK~ K^T, then the H matrices dPhi_V = sum dV~ V^T (CSAT_SEPARATE_PHI).
 * dK~, dV~ are the ones the most recent csat_backward of this context formed (kept as bf16); K, V [B,H,n,d] (device,
 * context dtype) must be the tensors that call was given.  One tensor-core product per head with float32
 * accumulation, written once (H m n floats: size the call for it).  Only after a csat_backward on the tensor-core path
 * (bf16, d in {64, 128}), else CSAT_ERR_STATE. */
int csat_backward_phi(csat_ctx* ctx, const void* K, const void* V, float* dPhi, void* stream);

/* csat_project_qkv -- paper: the projection equation Q = X W^Q, K = X W^K, V = X W^V ("Mathematical Framework"),
 * for all heads at once, written in the layout csat_forward reads.
 *   Xq   [B, n_q, d_model]  tokens the queries come from           (context dtype, device)
 *   Xkv  [B, n,   d_model]  tokens the keys and values come from; the same pointer as Xq for self-attention
 *   W    [d_model, 3 H d]   row-major; columns [0, H d) = W^Q of heads 0..H-1 (d columns each), then W^K, then W^V
 *   Q    [B, H, n_q, d]   K, V  [B, H, n, d]                        (outputs, context dtype)
 * Float32 accumulation, outputs rounded to the context dtype.  With Xq == Xkv and n_q == n this is one launch over
 * all 3 H d columns, otherwise one for Q and one for K and V.  Enqueued on `stream`, no allocation.  bf16 with
 * d in {64, 128} and d_model a multiple of 8 runs on the tensor cores; everything else on a plain FFMA kernel.
 * All pointers 16-byte aligned, else CSAT_ERR_INVALID_ARG. */
int csat_project_qkv(csat_ctx* ctx, const void* Xq, const void* Xkv, const void* W, int64_t d_model, void* Q, void* K,
                     void* V, void* stream);

/*
 * csat_forward -- paper: compression, approximate attention matrix, compressed output,
 * LISTA recurrence and reconstruction equations (all of the hot path).
 *   Q   [B, H, n_q, d]   K, V [B, H, n, d]   out [B, H, n_q, d]   device, context dtype.
 * out must not overlap Q, K or V (checked on the byte ranges: CSAT_ERR_INVALID_ARG).  Launch-only: no allocation, no synchronisation, no host
 * access to the tensors.  The n_q x m attention matrix and the recovery iterates never reach
 * global memory; K~|V~ (m x 2d per (b,h)) live in the context's workspace (bf16 contexts keep m x d more per (b,h)
 * for V~ B: long jobs with one S, B and one positive threshold for all layers use z B = A~ (V~ B), LISTA recurrence).
 * Errors: CSAT_ERR_INVALID_ARG (NULL/misaligned), CSAT_ERR_SHAPE (default D with m < d or
 * n < d), CSAT_ERR_CUDA (launch failure), CSAT_ERR_TIMEOUT (a previous launch's bounded wait
 * gave up; its output is invalid).
 */
int csat_forward(csat_ctx* ctx, const void* Q, const void* K, const void* V, void* out, void* stream);

/*
 * Token-sharded forward -- paper: "Efficiency and Scaling" (sequences beyond one device) and the compression
 * equation, whose sum over the n tokens splits over shards: Phi K = sum over shards s of Phi[:, shard s] K[shard s].
 * When the keys and values of one (batch, head) pair are spread over several GPUs, every GPU
 *   1. csat_compress_partial: multiplies its token shard by the matching columns of Phi (every GPU generates the
 *      same Phi from the seed) and gets the float32 partial sums for K~|V~;
 *   2. exchanges the partials with the other GPUs (the caller's collective, e.g. an all-gather: the library takes no
 *      communicator) and
 *   3. csat_reduce_partials: adds them in the order given -- the same order on every GPU, so all hold bit-identical
 *      K~|V~ -- into the context's workspace, rounded once to the context dtype;
 *   4. csat_attend: attention and recovery for its own queries (the context's CSAT_NQ = the number of local
 *      queries); no further exchange.
 *
 *   K_shard, V_shard [B, H, n_len, d]   tokens n0 .. n0 + n_len - 1 of the sequence (context dtype, device)
 *   partial_out      [B, H, m, 2d]      float32, device: row r = K~_r | V~_r partial sums
 *   partials         [count][B, H, m, 2d] float32, device, contiguous: the shards' partials in the agreed order
 *   Q, out           [B, H, n_q, d]     as for csat_forward
 * n0 must be a multiple of 8 (shard boundaries at multiples of 64 keep every load aligned to a 128-byte line) and
 * [n0, n0 + n_len) inside [0, n): else CSAT_ERR_SHAPE.  Launch-only, no allocation.  csat_attend needs a workspace
 * filled by csat_reduce_partials or csat_forward (CSAT_ERR_STATE otherwise).  One shard covering all n tokens
 * followed by csat_reduce_partials(count = 1) and csat_attend equals csat_forward up to the rounding of the sums.
 */
int csat_compress_partial(csat_ctx* ctx, const void* K_shard, const void* V_shard, int64_t n0, int64_t n_len,
                          float* partial_out, void* stream);
int csat_reduce_partials(csat_ctx* ctx, const float* partials, int count, void* stream);
int csat_attend(csat_ctx* ctx, const void* Q, void* out, void* stream);

/*
 * csat_forward_host -- same computation with HOST buffers (same layouts and dtype; pinned memory gives
 * asynchronous copies).  Copies Q, K, V to staging buffers the context owns (allocated by the first call, so
 * that call also allocates), computes, copies out back and returns once `stream` has reached the end of all of
 * it.  On the tensor-core path (and with CSAT_PROFILE off) the job is pipelined in runs of consecutive
 * (batch, head) pairs (about four runs per batch element, at most 64 in all) over three internal streams (copy in, compute, copy out) ordered after `stream`, so that the
 * copies overlap the compute and each other; otherwise everything runs in order on `stream`.
 */
int csat_forward_host(csat_ctx* ctx, const void* Q_host, const void* K_host, const void* V_host,
                      void* out_host, void* stream);

/* csat_get_compressed -- paper: K~, V~ of the compression equation, as left in the workspace
 * by the most recent csat_forward.  kt_out, vt_out: [B, H, m, d] each, context dtype (either may
 * be NULL).  Enqueued on `stream`.  CSAT_ERR_STATE before the first forward. */
int csat_get_compressed(const csat_ctx* ctx, void* kt_out, void* vt_out, void* stream);

/* csat_get_decoder -- paper: S, B, theta of the LISTA recurrence as derived for the current
 * parameters: S_out, B_out [H, d, d] float32 (row-vector convention: alpha <- eta(alpha S + z B)),
 * theta_out [H] float32, mu_out [H] float32 (any may be NULL).  Derives them on `stream` first if
 * parameters changed. */
int csat_get_decoder(csat_ctx* ctx, float* S_out, float* B_out, float* theta_out, float* mu_out, void* stream);

/* csat_get_profile -- measurement aid, no counterpart in the paper.  With CSAT_PROFILE = v > 0
 * every csat_forward records CUDA events on its stream before the first and after each of its
 * kernels.  call_index counts forward calls since CSAT_PROFILE was set (0-based; only the most
 * recent v are kept).  Writes up to `cap` kernel ids and their durations in milliseconds to the
 * HOST arrays and the number of kernels to *count_host.  Synchronises on the call's last event.
 * CSAT_ERR_STATE if profiling is off or the call is no longer / not yet recorded. */
int csat_get_profile(const csat_ctx* ctx, int64_t call_index, int cap, int* kernel_ids_host, float* ms_host,
                     int* count_host);

/*
 * csat_attend_noalloc -- the paper has no counterpart; this is a deployment aid.
 *
 * Some callers may not allocate device memory at the point where they need attention: code that
 * runs inside another framework's memory plan or after its arena has been sealed, real-time loops
 * where cudaMalloc's implicit device synchronisation is not acceptable, and processes whose memory
 * budget is fixed up front.  csat_create/csat_forward are closed to them because the K~|V~
 * workspace comes from cudaMalloc.  This entry point computes the compressed attention with
 * recovery disabled,
 *     out = softmax(Q (Phi K)^T * scale) (Phi V)        (same result as csat_forward with CSAT_T = 0),
 * and keeps K~|V~ in a fixed CSAT_NOALLOC_SCRATCH_BYTES array that is part of the library image.
 * It calls no cudaMalloc/cudaFree and no allocating library routine, and needs no context.
 *
 *   Q [B,H,n_q,d], K,V [B,H,n,d], phi [H,m,n] dense (e.g. from csat_get_phi), out [B,H,n_q,d]:
 *   device pointers, 16-byte aligned, element type `dtype` (CSAT_DTYPE_*).  scale 0 = 1/sqrt(d).
 *   err_host/err_cap: optional host buffer that receives a message when the call fails.
 *
 * Limits and rules
 *   - B*H*m*2*d*sizeof(element) must not exceed CSAT_NOALLOC_SCRATCH_BYTES; larger problems are
 *     refused with CSAT_ERR_SHAPE and a message stating both numbers.
 *   - Every GPU that loads the library holds the array (8 MiB) until the process exits.
 *   - The first call on each device looks the array's device address up (cudaGetSymbolAddress,
 *     with that device current); make that first call before starting any stream capture.
 *   - All calls on a device share the one array.  Each call overwrites the part it reads, so
 *     nothing needs clearing, but two calls that overlap on the GPU (different streams, or
 *     different host threads without ordering) race on it: serialise them on one stream.
 */
#define CSAT_NOALLOC_SCRATCH_BYTES (8u << 20)
int csat_attend_noalloc(const void* Q, const void* K, const void* V, const void* phi, void* out, int64_t B,
                        int64_t H, int64_t n, int64_t n_q, int64_t m, int64_t d, int dtype, double scale,
                        void* stream, char* err_host, size_t err_cap);

/* csat_selftest_wait_timeout / csat_clear_status -- failure-detection aids, no counterpart in the paper.
 * Every device-side wait of this library is bounded; when one gives up, the kernel records a code in the
 * context's status word and returns, and host calls report CSAT_ERR_TIMEOUT from then on.
 * csat_selftest_wait_timeout launches a one-thread kernel that waits `limit_us` microseconds (1 .. 1000000) on a
 * barrier nothing arrives at, synchronises `stream` and returns CSAT_ERR_TIMEOUT if (as it must) the wait gave
 * up and the status word was set, CSAT_ERR_STATE if it was not.  The context stays usable for queries; its
 * csat_forward calls return CSAT_ERR_TIMEOUT until csat_clear_status, which synchronises the device, resets the
 * status word and returns the code it held (0 = none). */
int csat_selftest_wait_timeout(csat_ctx* ctx, int64_t limit_us, void* stream);
int csat_clear_status(csat_ctx* ctx, int* code_host);

/* csat_debug_fail_alloc -- test aid, no counterpart in the paper.  Makes the countdown-th device allocation any
 * context of this process attempts from now on fail as if the device were out of memory (0 switches the aid off;
 * it also switches itself off after firing).  Lets a test drive the CSAT_ERR_ALLOC paths without exhausting a
 * GPU.  Process-wide; not for production use. */
int csat_debug_fail_alloc(int countdown);

/* Bytes of device memory the context currently owns (Phi, workspace, decoder matrices, staging). */
size_t csat_workspace_bytes(const csat_ctx* ctx);

/* Number of kernels the most recent csat_forward enqueued (0 before the first). */
int csat_last_launch_count(const csat_ctx* ctx);

/* Text of the most recent failure of this context; with NULL, of the calling thread's most
 * recent failed csat_create.  Also looks at the status word kernels write when a bounded wait
 * gives up (host-mapped memory, read without synchronising), so a CSAT_ERR_TIMEOUT raised by a
 * finished launch becomes visible.  The pointer stays valid until the next call on the same
 * context / thread. */
const char* csat_last_error(const csat_ctx* ctx);

/* Library version: major*10000 + minor*100 + patch. */
int csat_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CSAT_H_ */
