// Host side of libcsat: context, parameter handling, dispatch.  See include/csat.h for the contract.
#include <cstdio>
#include <cstring>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "csat_internal.h"

namespace {

thread_local std::string g_create_error;

int fail(csat_ctx* c, int code, const std::string& msg) {
  if (c) c->err = msg;
  else g_create_error = msg;
  return code;
}

int fail_cuda(csat_ctx* c, cudaError_t e, const char* what) {
  return fail(c, CSAT_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// byte ranges [a, a + na) and [b, b + nb) share at least one byte
bool ranges_overlap(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
  return a0 < b0 + nb && b0 < a0 + na;
}

// An NVTX range around a host call (visible in a timeline tool; a no-op when none is attached).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
};

// csat_debug_fail_alloc: the k-th device allocation from now on fails (0 = off)
std::atomic<int> g_fail_alloc_countdown{0};

template <typename T>
cudaError_t dev_alloc(csat_ctx* c, T** p, size_t bytes) {
  *p = nullptr;
  if (bytes == 0) return cudaSuccess;
  if (g_fail_alloc_countdown.load() > 0 && g_fail_alloc_countdown.fetch_sub(1) == 1) return cudaErrorMemoryAllocation;
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), bytes);
  if (e == cudaSuccess) c->bytes += bytes;
  return e;
}

template <typename T>
void dev_free(csat_ctx* c, T** p, size_t bytes) {
  if (*p) {
    cudaFree(*p);
    c->bytes -= bytes;
    *p = nullptr;
  }
}

size_t phi_bytes(const csat::Params& p) {
  return (size_t)(p.H * (p.separate_phi ? 2 : 1) * p.m * p.n_pad) * csat::elt_size(p.dtype);
}
// the generators see Phi_V of head h as head H + h
csat::Params gen_params(const csat::Params& p) {
  csat::Params g = p;
  g.H = p.H * (p.separate_phi ? 2 : 1);
  return g;
}
// K~|V~ [B H, m, 2 d]; bf16 contexts keep V~ B [B H, m, d] (the recovery phase's first product, folded into the
// values) behind it in the same allocation
size_t kv_bytes(const csat::Params& p) {
  const int64_t cols = 2 * p.d + (p.dtype == CSAT_DTYPE_BF16 ? p.d : 0);
  return (size_t)(p.B * p.H * p.m * cols) * csat::elt_size(p.dtype);
}
size_t dd_bytes(const csat::Params& p, size_t elt) { return (size_t)(p.H * p.d * p.d) * elt; }

void prof_destroy(csat_ctx* c);

void free_lista(csat_ctx* c) {
  const csat::Params& p = c->p;
  const size_t mats = c->w_mat_count();
  dev_free(c, &c->w_S, mats * csat::elt_size(p.dtype));
  dev_free(c, &c->w_B, mats * csat::elt_size(p.dtype));
  dev_free(c, &c->w_theta, (size_t)c->w_layers * p.H * 4);
  dev_free(c, &c->Sl_dec, mats * 4);
  dev_free(c, &c->Bl_dec, mats * 4);
  dev_free(c, &c->lmats_bf16, (size_t)(2 * c->w_layers + 1) * dd_bytes(p, 2));
  c->w_layers = 0;
  c->w_untied = false;
}

void free_hadamard_tables(csat_ctx* c) {
  dev_free(c, &c->had_signs, c->had_bytes_signs);
  dev_free(c, &c->had_ab, c->had_bytes_ab);
  c->had_bytes_signs = c->had_bytes_ab = 0;
}

// the fast-transform compression's tables, (re)written whenever the structured Hadamard ensemble is generated
int make_hadamard_tables(csat_ctx* c) {
  free_hadamard_tables(c);
  if (c->p.ensemble != CSAT_ENSEMBLE_HADAMARD) return CSAT_OK;
  const csat::Params g = gen_params(c->p);
  const size_t bs = (size_t)((g.H * g.n + 31) / 32) * 4, ba = (size_t)g.H * 8;
  if (dev_alloc(c, &c->had_signs, bs) != cudaSuccess || dev_alloc(c, &c->had_ab, ba) != cudaSuccess) {
    free_hadamard_tables(c);
    return fail(c, CSAT_ERR_ALLOC, "cudaMalloc(Hadamard tables) failed");
  }
  c->had_bytes_signs = bs;
  c->had_bytes_ab = ba;
  cudaError_t e = csat::launch_hadamard_tables(c->had_signs, c->had_ab, g, 0);
  if (e == cudaSuccess) e = cudaStreamSynchronize(0);
  if (e != cudaSuccess) return fail_cuda(c, e, "Hadamard tables");
  return CSAT_OK;
}

void free_backward(csat_ctx* c) {
  dev_free(c, &c->bw_dZ, c->bw_bytes_dZ);
  dev_free(c, &c->bw_LD, c->bw_bytes_LD);
  dev_free(c, &c->bw_dKV, c->bw_bytes_dKV);
  dev_free(c, &c->bw_WT, c->bw_bytes_WT);
  dev_free(c, &c->bw_dKV16, c->bw_bytes_dKV16);
  dev_free(c, &c->bw_dZ16, c->bw_bytes_dZ16);
  dev_free(c, &c->bw_masks, c->bw_bytes_masks);
  dev_free(c, &c->bw_Z16, c->bw_bytes_Z16);
  dev_free(c, &c->bw_maskbits, c->bw_bytes_maskbits);
  dev_free(c, &c->bw_alpha16, c->bw_bytes_alpha16);
  dev_free(c, &c->bw_dx16, c->bw_bytes_dx16);
  dev_free(c, &c->bw_wpart, c->bw_bytes_wpart);
  dev_free(c, &c->bw_thpart, c->bw_bytes_thpart);
  dev_free(c, &c->bw_wgrad, c->bw_bytes_wgrad);
  dev_free(c, &c->bw_signbits, c->bw_bytes_signbits);
  c->bw_bytes_signbits = 0;
  c->bw_bytes_alpha16 = c->bw_bytes_dx16 = c->bw_bytes_wpart = c->bw_bytes_thpart = c->bw_bytes_wgrad = 0;
  c->have_wgrads = false;
  c->have_dkv16 = false;
  c->saved_valid = false;
  c->bw_bytes_Z16 = c->bw_bytes_maskbits = 0;
  c->bw_bytes_masks = 0;
  c->have_masks = false;
  c->bw_bytes_dZ = c->bw_bytes_LD = c->bw_bytes_dKV = c->bw_bytes_WT = c->bw_bytes_dKV16 = c->bw_bytes_dZ16 = 0;
}

void free_staging(csat_ctx* c) {
  dev_free(c, &c->stage_q, c->stage_bytes_q);
  dev_free(c, &c->stage_o, c->stage_bytes_q);
  dev_free(c, &c->stage_k, c->stage_bytes_kv);
  dev_free(c, &c->stage_v, c->stage_bytes_kv);
  c->stage_bytes_q = c->stage_bytes_kv = 0;
}

void free_all(csat_ctx* c) {
  const csat::Params& p = c->p;
  dev_free(c, &c->phi, phi_bytes(p));
  dev_free(c, &c->kv, kv_bytes(p));
  dev_free(c, &c->psi, (size_t)((c->psi_per_head ? p.H : 1) * p.d * p.d) * csat::elt_size(p.dtype));
  dev_free(c, &c->dmat, dd_bytes(p, csat::elt_size(p.dtype)));
  dev_free(c, &c->Mf64, dd_bytes(p, 8));
  dev_free(c, &c->Gf64, dd_bytes(p, 8));
  dev_free(c, &c->S_dec, dd_bytes(p, 4));
  dev_free(c, &c->B_dec, dd_bytes(p, 4));
  dev_free(c, &c->psi_f32, dd_bytes(p, 4));
  dev_free(c, &c->theta, (size_t)p.H * 4);
  dev_free(c, &c->mu, (size_t)p.H * 4);
  dev_free(c, &c->mats_bf16, 3 * dd_bytes(p, 2));
  free_hadamard_tables(c);
  free_lista(c);
  free_staging(c);
  free_backward(c);
  prof_destroy(c);
  if (c->pipe_ready) {
    for (int i = 0; i < 3; ++i) cudaStreamDestroy(c->pipe_stream[i]);
    for (int i = 0; i < csat_ctx::kPipeEvents; ++i) cudaEventDestroy(c->pipe_event[i]);
    c->pipe_ready = false;
  }
  if (c->status) {
    cudaFreeHost(c->status);
    c->status = nullptr;
  }
}

// (re)allocates everything whose size depends on dtype / B and regenerates Phi from the seed
int allocate_and_generate(csat_ctx* c) {
  const csat::Params& p = c->p;
  cudaError_t e;
  // Until everything below has succeeded the context holds no usable Phi / workspace: compute calls are refused.
  c->broken = true;
  c->tmap_phi_valid = false;
  if ((e = dev_alloc(c, &c->phi, phi_bytes(p))) != cudaSuccess) return fail(c, CSAT_ERR_ALLOC, "cudaMalloc(Phi) failed");
  if ((e = dev_alloc(c, &c->kv, kv_bytes(p))) != cudaSuccess) {
    dev_free(c, &c->phi, phi_bytes(p));
    return fail(c, CSAT_ERR_ALLOC, "cudaMalloc(K~|V~) failed");
  }
  if ((e = csat::launch_phi_gen(c->phi, gen_params(p), 0)) != cudaSuccess) return fail_cuda(c, e, "phi_gen launch");
  if ((e = cudaStreamSynchronize(0)) != cudaSuccess) return fail_cuda(c, e, "phi_gen");
  c->phi_generated = true;
  if (int rc = make_hadamard_tables(c)) return rc;
  c->tmap_phi_valid = false;
  if (p.dtype == CSAT_DTYPE_BF16 && (p.d == 64 || p.d == 128)) {
    if ((e = csat::make_phi_tmap(c)) != cudaSuccess) return fail_cuda(c, e, "tensor map for Phi");
    if ((e = csat::make_attend_tmaps(c)) != cudaSuccess) return fail_cuda(c, e, "tensor maps for K~|V~");
    c->tmap_phi_valid = true;
  }
  c->decoder_dirty = true;
  c->have_forward = false;
  c->broken = false;
  return CSAT_OK;
}

// refusal of compute calls and getters after a failed re-allocation
const char* kBrokenMsg =
    "an earlier setter failed to re-allocate the context's buffers; set CSAT_BATCH, CSAT_DTYPE or CSAT_SEPARATE_PHI "
    "again (successfully) before using the context";

int allocate_and_generate_with_batch(csat_ctx* c, int64_t B) {
  dev_free(c, &c->phi, phi_bytes(c->p));
  dev_free(c, &c->kv, kv_bytes(c->p));
  c->p.B = B;
  return allocate_and_generate(c);
}

void prof_destroy(csat_ctx* c) {
  for (cudaEvent_t e : c->prof_events) cudaEventDestroy(e);
  c->prof_events.clear();
  c->prof_ids.clear();
  c->prof_count.clear();
  c->prof_slots = 0;
  c->prof_calls = 0;
}

// records the event that closes kernel `id` of the current call (id < 0: the opening event)
void prof_mark(csat_ctx* c, cudaStream_t s, int id) {
  if (c->prof_slots == 0) return;
  const int K = csat_ctx::kProfMaxKernels;
  const int slot = (int)(c->prof_calls % c->prof_slots);
  if (id < 0) {
    c->prof_count[slot] = 0;
    cudaEventRecord(c->prof_events[(size_t)slot * (K + 1)], s);
    return;
  }
  int& n = c->prof_count[slot];
  if (n >= K) return;
  c->prof_ids[(size_t)slot * K + n] = id;
  cudaEventRecord(c->prof_events[(size_t)slot * (K + 1) + n + 1], s);
  ++n;
}

bool on_device(const csat_ctx* c, std::string* why) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev != c->device) {
    *why = "context was created on another CUDA device than the current one";
    return false;
  }
  return true;
}

}  // namespace

extern "C" {

int csat_version(void) { return 100; }

csat_ctx* csat_create(int64_t n, int64_t m, int64_t d, int64_t H, uint64_t seed) {
  NvtxRange range("csat_create");
  if (n < 1 || m < 1 || m > n || d < 1 || H < 1) {
    fail(nullptr, CSAT_ERR_SHAPE, "csat_create: need 1 <= m <= n, d >= 1, H >= 1");
    return nullptr;
  }
  if (d > 256 || d % 8 != 0) {
    fail(nullptr, CSAT_ERR_SHAPE, "csat_create: need d <= 256 and d % 8 == 0");
    return nullptr;
  }
  if (n > (int64_t)1 << 31 || H * m * csat::round_up(n, csat::kPhiColPad) > (int64_t)1 << 38) {
    fail(nullptr, CSAT_ERR_SHAPE, "csat_create: problem too large");
    return nullptr;
  }
  int ndev = 0;
  cudaError_t e = cudaGetDeviceCount(&ndev);
  if (e != cudaSuccess || ndev == 0) {
    fail(nullptr, CSAT_ERR_CUDA, std::string("csat_create: no CUDA device: ") + cudaGetErrorString(e));
    return nullptr;
  }
  csat_ctx* c = new (std::nothrow) csat_ctx();
  if (!c) {
    fail(nullptr, CSAT_ERR_ALLOC, "csat_create: host allocation failed");
    return nullptr;
  }
  cudaGetDevice(&c->device);
  if (cudaDeviceGetAttribute(&c->sms, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess || c->sms <= 0) c->sms = 148;
  csat::Params& p = c->p;
  p.n = n; p.m = m; p.d = d; p.H = H; p.B = 1; p.nq = n;
  p.n_pad = csat::round_up(n, csat::kPhiColPad);
  p.dtype = CSAT_DTYPE_BF16;
  p.ensemble = CSAT_ENSEMBLE_GAUSSIAN;
  p.separate_phi = 0;
  p.T = 10; p.lambda = 0.1; p.step = 0.0; p.scale = 0.0; p.seed = seed;

  int rc = CSAT_OK;
  e = cudaHostAlloc(reinterpret_cast<void**>(&c->status), sizeof(int), cudaHostAllocMapped);
  if (e != cudaSuccess) rc = fail(c, CSAT_ERR_ALLOC, "cudaHostAlloc(status) failed");
  else *c->status = 0;
  if (rc == CSAT_OK && (dev_alloc(c, &c->Mf64, dd_bytes(p, 8)) != cudaSuccess ||
                        dev_alloc(c, &c->Gf64, dd_bytes(p, 8)) != cudaSuccess ||
                        dev_alloc(c, &c->S_dec, dd_bytes(p, 4)) != cudaSuccess ||
                        dev_alloc(c, &c->B_dec, dd_bytes(p, 4)) != cudaSuccess ||
                        dev_alloc(c, &c->psi_f32, dd_bytes(p, 4)) != cudaSuccess ||
                        dev_alloc(c, &c->theta, (size_t)H * 4) != cudaSuccess ||
                        dev_alloc(c, &c->mu, (size_t)H * 4) != cudaSuccess ||
                        dev_alloc(c, &c->mats_bf16, 3 * dd_bytes(p, 2)) != cudaSuccess))
    rc = fail(c, CSAT_ERR_ALLOC, "cudaMalloc(decoder matrices) failed");
  if (rc == CSAT_OK) rc = allocate_and_generate(c);
  if (rc != CSAT_OK) {
    g_create_error = "csat_create: " + c->err;
    cudaGetLastError();
    free_all(c);
    delete c;
    return nullptr;
  }
  return c;
}

int csat_destroy(csat_ctx* c) {
  if (!c) return CSAT_OK;
  cudaDeviceSynchronize();
  free_all(c);
  delete c;
  return CSAT_OK;
}

int csat_set_i64(csat_ctx* c, int key, int64_t v) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  c->saved_valid = false;
  csat::Params& p = c->p;
  switch (key) {
    case CSAT_BATCH: {
      if (v < 1 || v > (1 << 20)) return fail(c, CSAT_ERR_SHAPE, "CSAT_BATCH must be >= 1");
      if (v == p.B && !c->broken) return CSAT_OK;
      cudaDeviceSynchronize();
      if (!c->phi) return allocate_and_generate_with_batch(c, v);   // after a failed re-allocation: start over
      dev_free(c, &c->kv, kv_bytes(p));
      free_staging(c);
      p.B = v;
      c->have_forward = false;
      c->broken = true;
      if (dev_alloc(c, &c->kv, kv_bytes(p)) != cudaSuccess) return fail(c, CSAT_ERR_ALLOC, "cudaMalloc(K~|V~) failed");
      if (c->tmap_phi_valid && csat::make_attend_tmaps(c) != cudaSuccess)
        return fail(c, CSAT_ERR_CUDA, "tensor maps for K~|V~");
      c->broken = false;
      return CSAT_OK;
    }
    case CSAT_NQ:
      if (v < 1 || v > ((int64_t)1 << 31)) return fail(c, CSAT_ERR_SHAPE, "CSAT_NQ must be >= 1");
      if (v != p.nq) { cudaDeviceSynchronize(); free_staging(c); }
      p.nq = v;
      return CSAT_OK;
    case CSAT_DTYPE: {
      if (v != CSAT_DTYPE_BF16 && v != CSAT_DTYPE_FP32) return fail(c, CSAT_ERR_INVALID_ARG, "unknown CSAT_DTYPE");
      if ((int)v == p.dtype && !c->broken) return CSAT_OK;
      cudaDeviceSynchronize();
      dev_free(c, &c->phi, phi_bytes(p));
      dev_free(c, &c->kv, kv_bytes(p));
      dev_free(c, &c->psi, (size_t)((c->psi_per_head ? p.H : 1) * p.d * p.d) * csat::elt_size(p.dtype));
      dev_free(c, &c->dmat, dd_bytes(p, csat::elt_size(p.dtype)));
      free_lista(c);
      free_staging(c);
      p.dtype = (int)v;
      return allocate_and_generate(c);   // user-set Phi, Psi, D are dropped with the old dtype
    }
    case CSAT_ENSEMBLE: {
      if (v != CSAT_ENSEMBLE_GAUSSIAN && v != CSAT_ENSEMBLE_RADEMACHER && v != CSAT_ENSEMBLE_HADAMARD)
        return fail(c, CSAT_ERR_INVALID_ARG, "unknown CSAT_ENSEMBLE");
      if ((int)v == p.ensemble) return CSAT_OK;
      if (c->broken) return fail(c, CSAT_ERR_STATE, kBrokenMsg);
      cudaDeviceSynchronize();
      p.ensemble = (int)v;
      cudaError_t e = csat::launch_phi_gen(c->phi, gen_params(p), 0);   // a Phi set by csat_set_phi is replaced as well
      if (e == cudaSuccess) e = cudaStreamSynchronize(0);
      if (e != cudaSuccess) return fail_cuda(c, e, "phi_gen");
      c->phi_generated = true;
      c->decoder_dirty = true;
      return make_hadamard_tables(c);
    }
    case CSAT_DEBUG_CANARY:
      if (v != 0 && v != 1) return fail(c, CSAT_ERR_INVALID_ARG, "CSAT_DEBUG_CANARY must be 0 or 1");
      c->debug_canary = (int)v;
      return CSAT_OK;
    case CSAT_HADAMARD_TRANSFORM:
      if (v != 0 && v != 1) return fail(c, CSAT_ERR_INVALID_ARG, "CSAT_HADAMARD_TRANSFORM must be 0 or 1");
      c->hadamard_transform = (int)v;
      return CSAT_OK;
    case CSAT_SEPARATE_PHI: {
      if (v != 0 && v != 1) return fail(c, CSAT_ERR_INVALID_ARG, "CSAT_SEPARATE_PHI must be 0 or 1");
      if ((int)v == p.separate_phi && !c->broken) return CSAT_OK;
      cudaDeviceSynchronize();
      dev_free(c, &c->phi, phi_bytes(p));
      dev_free(c, &c->kv, kv_bytes(p));
      p.separate_phi = (int)v;
      return allocate_and_generate(c);
    }
    case CSAT_T:
      if (v < 0 || v > 100000) return fail(c, CSAT_ERR_INVALID_ARG, "CSAT_T must be in [0, 100000]");
      p.T = (int)v;
      return CSAT_OK;
    case CSAT_FORCE_SIMT:
      if (v < 0 || v > 2) return fail(c, CSAT_ERR_INVALID_ARG, "CSAT_FORCE_SIMT must be 0, 1 or 2");
      c->force_simt = (int)v;
      return CSAT_OK;
    case CSAT_KEEP_MASKS:
      if (v != 0 && v != 1) return fail(c, CSAT_ERR_INVALID_ARG, "CSAT_KEEP_MASKS must be 0 or 1");
      if ((v != 0) != c->keep_masks) { cudaDeviceSynchronize(); free_backward(c); }
      c->keep_masks = v != 0;
      return CSAT_OK;
    case CSAT_SAVE_FOR_BACKWARD:
      if (v != 0 && v != 1) return fail(c, CSAT_ERR_INVALID_ARG, "CSAT_SAVE_FOR_BACKWARD must be 0 or 1");
      c->save_for_backward = v != 0;
      return CSAT_OK;
    case CSAT_WEIGHT_GRADS:
      if (v != 0 && v != 1) return fail(c, CSAT_ERR_INVALID_ARG, "CSAT_WEIGHT_GRADS must be 0 or 1");
      if ((v != 0) != c->weight_grads) { cudaDeviceSynchronize(); free_backward(c); }
      c->weight_grads = v != 0;
      return CSAT_OK;
    case CSAT_PROFILE: {
      if (v < 0 || v > 4096) return fail(c, CSAT_ERR_INVALID_ARG, "CSAT_PROFILE must be in [0, 4096]");
      cudaDeviceSynchronize();
      prof_destroy(c);
      const int K = csat_ctx::kProfMaxKernels;
      c->prof_events.reserve((size_t)v * (K + 1));
      for (int64_t i = 0; i < v * (K + 1); ++i) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) {
          prof_destroy(c);
          return fail(c, CSAT_ERR_ALLOC, "cudaEventCreate failed");
        }
        c->prof_events.push_back(e);
      }
      c->prof_ids.assign((size_t)v * K, 0);
      c->prof_count.assign((size_t)v, 0);
      c->prof_slots = (int)v;
      return CSAT_OK;
    }
    default:
      return fail(c, CSAT_ERR_INVALID_ARG, "csat_set_i64: unknown key");
  }
}

int csat_get_i64(const csat_ctx* c, int key, int64_t* out) {
  if (!c || !out) return CSAT_ERR_INVALID_ARG;
  switch (key) {
    case CSAT_BATCH: *out = c->p.B; return CSAT_OK;
    case CSAT_NQ: *out = c->p.nq; return CSAT_OK;
    case CSAT_DTYPE: *out = c->p.dtype; return CSAT_OK;
    case CSAT_T: *out = c->p.T; return CSAT_OK;
    case CSAT_ENSEMBLE: *out = c->p.ensemble; return CSAT_OK;
    case CSAT_SEPARATE_PHI: *out = c->p.separate_phi; return CSAT_OK;
    case CSAT_FORCE_SIMT: *out = c->force_simt; return CSAT_OK;
    case CSAT_PROFILE: *out = c->prof_slots; return CSAT_OK;
    case CSAT_KEEP_MASKS: *out = c->keep_masks ? 1 : 0; return CSAT_OK;
    case CSAT_WEIGHT_GRADS: *out = c->weight_grads ? 1 : 0; return CSAT_OK;
    case CSAT_SAVE_FOR_BACKWARD: *out = c->save_for_backward ? 1 : 0; return CSAT_OK;
    case CSAT_HADAMARD_TRANSFORM: *out = c->hadamard_transform; return CSAT_OK;
    case CSAT_DEBUG_CANARY: *out = c->debug_canary; return CSAT_OK;
    default: return CSAT_ERR_INVALID_ARG;
  }
}

int csat_set_f64(csat_ctx* c, int key, double v) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  c->saved_valid = false;
  if (!(v == v)) return fail(c, CSAT_ERR_INVALID_ARG, "csat_set_f64: NaN");
  switch (key) {
    case CSAT_LAMBDA:
      if (v < 0) return fail(c, CSAT_ERR_INVALID_ARG, "CSAT_LAMBDA must be >= 0");
      c->p.lambda = v; c->decoder_dirty = true; return CSAT_OK;
    case CSAT_STEP:
      if (v < 0) return fail(c, CSAT_ERR_INVALID_ARG, "CSAT_STEP must be >= 0 (0 = automatic)");
      c->p.step = v; c->decoder_dirty = true; return CSAT_OK;
    case CSAT_SCALE:
      if (v < 0) return fail(c, CSAT_ERR_INVALID_ARG, "CSAT_SCALE must be >= 0 (0 = 1/sqrt(d))");
      c->p.scale = v; return CSAT_OK;
    default:
      return fail(c, CSAT_ERR_INVALID_ARG, "csat_set_f64: unknown key");
  }
}

int csat_get_f64(const csat_ctx* c, int key, double* out) {
  if (!c || !out) return CSAT_ERR_INVALID_ARG;
  switch (key) {
    case CSAT_LAMBDA: *out = c->p.lambda; return CSAT_OK;
    case CSAT_STEP: *out = c->p.step; return CSAT_OK;
    case CSAT_SCALE: *out = c->p.scale; return CSAT_OK;
    default: return CSAT_ERR_INVALID_ARG;
  }
}

int csat_set_phi(csat_ctx* c, const void* phi, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  c->saved_valid = false;
  if (!phi || !aligned16(phi)) return fail(c, CSAT_ERR_INVALID_ARG, "csat_set_phi: NULL or misaligned pointer");
  if (c->broken) return fail(c, CSAT_ERR_STATE, kBrokenMsg);
  std::string why;
  if (!on_device(c, &why)) return fail(c, CSAT_ERR_STATE, why);
  cudaError_t e = csat::launch_phi_pack(c->phi, phi, gen_params(c->p), (cudaStream_t)stream);
  if (e != cudaSuccess) return fail_cuda(c, e, "csat_set_phi");
  c->phi_generated = false;                // a supplied matrix has no structure the fast transform could use
  c->decoder_dirty = true;
  return CSAT_OK;
}

int csat_get_phi(const csat_ctx* c, void* phi_out, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  csat_ctx* mc = const_cast<csat_ctx*>(c);
  if (!phi_out || !aligned16(phi_out)) return fail(mc, CSAT_ERR_INVALID_ARG, "csat_get_phi: NULL or misaligned pointer");
  if (c->broken) return fail(mc, CSAT_ERR_STATE, kBrokenMsg);
  std::string why;
  if (!on_device(c, &why)) return fail(mc, CSAT_ERR_STATE, why);
  cudaError_t e = csat::launch_phi_unpack(phi_out, c->phi, gen_params(c->p), (cudaStream_t)stream);
  if (e != cudaSuccess) return fail_cuda(mc, e, "csat_get_phi");
  return CSAT_OK;
}

int csat_set_dictionary(csat_ctx* c, const void* psi, int per_head, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  c->saved_valid = false;
  csat::Params& p = c->p;
  const size_t es = csat::elt_size(p.dtype);
  if (psi && !aligned16(psi)) return fail(c, CSAT_ERR_INVALID_ARG, "csat_set_dictionary: misaligned pointer");
  const size_t old_bytes = (size_t)((c->psi_per_head ? p.H : 1) * p.d * p.d) * es;
  const size_t new_bytes = (size_t)((per_head ? p.H : 1) * p.d * p.d) * es;
  if (c->psi && (!psi || old_bytes != new_bytes)) {
    cudaDeviceSynchronize();
    dev_free(c, &c->psi, old_bytes);
  }
  c->decoder_dirty = true;
  if (!psi) { c->psi_per_head = false; return CSAT_OK; }
  c->psi_per_head = per_head != 0;
  if (!c->psi && dev_alloc(c, &c->psi, new_bytes) != cudaSuccess)
    return fail(c, CSAT_ERR_ALLOC, "cudaMalloc(Psi) failed");
  cudaError_t e = cudaMemcpyAsync(c->psi, psi, new_bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream);
  if (e != cudaSuccess) return fail_cuda(c, e, "csat_set_dictionary");
  return CSAT_OK;
}

int csat_set_decoder_matrix(csat_ctx* c, const void* D, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  c->saved_valid = false;
  csat::Params& p = c->p;
  const size_t bytes = dd_bytes(p, csat::elt_size(p.dtype));
  if (D && !aligned16(D)) return fail(c, CSAT_ERR_INVALID_ARG, "csat_set_decoder_matrix: misaligned pointer");
  c->decoder_dirty = true;
  if (!D) {
    if (c->dmat) { cudaDeviceSynchronize(); dev_free(c, &c->dmat, bytes); }
    return CSAT_OK;
  }
  if (!c->dmat && dev_alloc(c, &c->dmat, bytes) != cudaSuccess)
    return fail(c, CSAT_ERR_ALLOC, "cudaMalloc(D) failed");
  cudaError_t e = cudaMemcpyAsync(c->dmat, D, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream);
  if (e != cudaSuccess) return fail_cuda(c, e, "csat_set_decoder_matrix");
  return CSAT_OK;
}

static int set_weights(csat_ctx* c, const void* S, const void* Bm, const float* theta, int layers, bool untied,
                       void* stream, const char* who) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  csat::Params& p = c->p;
  c->decoder_dirty = true;
  if (!S) {
    if (c->w_S) { cudaDeviceSynchronize(); free_lista(c); }
    return CSAT_OK;
  }
  const std::string name(who);
  if (!Bm || !theta) return fail(c, CSAT_ERR_INVALID_ARG, name + ": NULL pointer");
  if (!aligned16(S) || !aligned16(Bm)) return fail(c, CSAT_ERR_INVALID_ARG, name + ": misaligned pointer");
  if (layers < 1 || layers > 100000) return fail(c, CSAT_ERR_INVALID_ARG, name + ": layers must be >= 1");
  if (c->w_S && (c->w_layers != layers || c->w_untied != untied)) { cudaDeviceSynchronize(); free_lista(c); }
  c->saved_valid = false;
  const size_t elt = csat::elt_size(p.dtype);
  if (!c->w_S) {
    c->w_layers = layers;
    c->w_untied = untied;
    const size_t mats = c->w_mat_count();
    bool ok = dev_alloc(c, &c->w_S, mats * elt) == cudaSuccess && dev_alloc(c, &c->w_B, mats * elt) == cudaSuccess &&
              dev_alloc(c, &c->w_theta, (size_t)layers * p.H * 4) == cudaSuccess;
    if (ok && untied) {
      ok = dev_alloc(c, &c->Sl_dec, mats * 4) == cudaSuccess && dev_alloc(c, &c->Bl_dec, mats * 4) == cudaSuccess;
      if (ok && p.dtype == CSAT_DTYPE_BF16 && (p.d == 64 || p.d == 128))
        ok = dev_alloc(c, &c->lmats_bf16, (size_t)(2 * layers + 1) * dd_bytes(p, 2)) == cudaSuccess &&
             csat::make_layer_weights_tmap(c) == cudaSuccess;
    }
    if (!ok) {
      cudaGetLastError();
      free_lista(c);
      return fail(c, CSAT_ERR_ALLOC, "cudaMalloc(LISTA weights) failed");
    }
  }
  cudaStream_t s = (cudaStream_t)stream;
  const size_t mat_bytes = c->w_mat_count() * elt;
  cudaError_t e;
  if ((e = cudaMemcpyAsync(c->w_S, S, mat_bytes, cudaMemcpyDeviceToDevice, s)) != cudaSuccess ||
      (e = cudaMemcpyAsync(c->w_B, Bm, mat_bytes, cudaMemcpyDeviceToDevice, s)) != cudaSuccess ||
      (e = cudaMemcpyAsync(c->w_theta, theta, (size_t)layers * p.H * 4, cudaMemcpyDeviceToDevice, s)) != cudaSuccess)
    return fail_cuda(c, e, who);
  return CSAT_OK;
}

int csat_set_lista_weights(csat_ctx* c, const void* S, const void* Bm, const float* theta, int layers, void* stream) {
  return set_weights(c, S, Bm, theta, layers, false, stream, "csat_set_lista_weights");
}

int csat_set_lista_layer_weights(csat_ctx* c, const void* S, const void* Bm, const float* theta, int layers,
                                 void* stream) {
  if (c && !S) return fail(c, CSAT_ERR_INVALID_ARG, "csat_set_lista_layer_weights: NULL pointer");
  if (c && layers > 4096) return fail(c, CSAT_ERR_INVALID_ARG, "csat_set_lista_layer_weights: at most 4096 layers");
  return set_weights(c, S, Bm, theta, layers, true, stream, "csat_set_lista_layer_weights");
}

static int ensure_decoder(csat_ctx* c, cudaStream_t s, int* launches) {
  const csat::Params& p = c->p;
  if (!c->w_S && !c->dmat && (p.m < p.d || p.n < p.d))
    return fail(c, CSAT_ERR_SHAPE, "default decoder matrix D = Phi[0:d,0:d] needs m >= d and n >= d");
  if (!c->decoder_dirty) return CSAT_OK;
  cudaError_t e = csat::launch_decoder_setup(c, s, launches);
  if (e != cudaSuccess) return fail_cuda(c, e, "decoder set-up launch");
  c->decoder_dirty = false;
  return CSAT_OK;
}

static int ensure_backward_scratch(csat_ctx* c);

int csat_forward(csat_ctx* c, const void* Q, const void* K, const void* V, void* out, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  if (!Q || !K || !V || !out) return fail(c, CSAT_ERR_INVALID_ARG, "csat_forward: NULL tensor pointer");
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(out))
    return fail(c, CSAT_ERR_INVALID_ARG, "csat_forward: tensor pointers must be 16-byte aligned");
  if (c->broken) return fail(c, CSAT_ERR_STATE, kBrokenMsg);
  NvtxRange range("csat_forward");
  {
    const csat::Params& p = c->p;
    const size_t es = csat::elt_size(p.dtype);
    const size_t bq = (size_t)(p.B * p.H * p.nq * p.d) * es, bkv = (size_t)(p.B * p.H * p.n * p.d) * es;
    if (ranges_overlap(out, bq, Q, bq) || ranges_overlap(out, bq, K, bkv) || ranges_overlap(out, bq, V, bkv))
      return fail(c, CSAT_ERR_INVALID_ARG, "csat_forward: out overlaps an input");
  }
  std::string why;
  if (!on_device(c, &why)) return fail(c, CSAT_ERR_STATE, why);
  if (*(volatile int*)c->status != 0)
    return fail(c, CSAT_ERR_TIMEOUT, "a bounded device-side wait of an earlier launch gave up; its output is invalid");
  cudaStream_t s = (cudaStream_t)stream;
  int launches = 0;
  prof_mark(c, s, -1);
  if (c->p.T > 0 && c->w_S && (c->w_layers != 1 || c->w_untied) && c->w_layers != c->p.T)
    return fail(c, CSAT_ERR_STATE, "the supplied LISTA weights are for a number of layers other than CSAT_T");
  if (c->p.T > 0) {
    const bool was_dirty = c->decoder_dirty;
    int rc = ensure_decoder(c, s, &launches);
    if (rc != CSAT_OK) return rc;
    if (was_dirty) prof_mark(c, s, CSAT_KERNEL_DECODER_SETUP);
  }
  cudaError_t e;
  // float32 contexts, and head sizes without a tensor-core kernel, take the FFMA kernels
  const bool tc_compress = c->tmap_phi_valid && c->force_simt != 1;
  const bool tc_attend = c->tmap_phi_valid && c->force_simt == 0;
  if (c->debug_canary && (e = cudaMemsetAsync(c->kv, 0xFF, kv_bytes(c->p), s)) != cudaSuccess)
    return fail_cuda(c, e, "canary fill");
  if (c->hadamard_transform && csat::fwht_compress_supported(c))
    e = csat::launch_fwht_compress(c, K, V, s, &launches);   // structured ensemble: transform instead of the dense product
  else
    e = tc_compress ? csat::launch_sm100_compress(c, K, V, s, &launches) : csat::launch_simt_compress(c, K, V, s, &launches);
  if (e != cudaSuccess) return fail_cuda(c, e, "compress launch");
  prof_mark(c, s, CSAT_KERNEL_COMPRESS);
  c->saved_valid = false;
  if (c->save_for_backward && tc_attend && c->p.B * c->p.H <= 32767) {
    // the recording variant of the same kernel: the output, and Z, the rows' log sum exp, the layers' decisions (and
    // the iterates with CSAT_WEIGHT_GRADS) where csat_backward will look for them
    if (int rc = ensure_backward_scratch(c)) return rc;
    const bool wg = c->weight_grads && c->p.T > 0 && c->bw_alpha16 != nullptr;
    if (wg && (e = cudaMemsetAsync(c->bw_alpha16, 0, (size_t)(c->p.B * c->p.H * c->p.nq * c->p.d) * 2, s)) != cudaSuccess)
      return fail_cuda(c, e, "memset");
    e = csat::launch_sm100_attend_for_backward(c, Q, c->bw_Z16, c->bw_LD, 2, c->bw_maskbits, wg ? c->bw_alpha16 : nullptr, s,
                                               &launches, out);
    if (e == cudaSuccess) { c->saved_valid = true; c->saved_alpha = wg; }
  } else {
    e = tc_attend ? csat::launch_sm100_attend_recover(c, Q, out, s, &launches)
                  : csat::launch_simt_attend_recover(c, Q, out, s, &launches);
  }
  if (e != cudaSuccess) return fail_cuda(c, e, "attend/recover launch");
  prof_mark(c, s, CSAT_KERNEL_ATTEND_RECOVER);
  if (c->prof_slots) ++c->prof_calls;
  c->have_forward = true;
  c->last_launches = launches;
  return CSAT_OK;
}

// ---- token-sharded use: one (batch, head) pair's keys and values spread over several GPUs ----------------------
int csat_compress_partial(csat_ctx* c, const void* K_shard, const void* V_shard, int64_t n0, int64_t n_len,
                          float* partial_out, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  c->saved_valid = false;
  if (!K_shard || !V_shard || !partial_out) return fail(c, CSAT_ERR_INVALID_ARG, "csat_compress_partial: NULL pointer");
  if (!aligned16(K_shard) || !aligned16(V_shard) || !aligned16(partial_out))
    return fail(c, CSAT_ERR_INVALID_ARG, "csat_compress_partial: pointers must be 16-byte aligned");
  const csat::Params& p = c->p;
  if (n0 < 0 || n_len < 1 || n0 + n_len > p.n)
    return fail(c, CSAT_ERR_SHAPE, "csat_compress_partial: the shard [n0, n0 + n_len) must lie inside [0, n)");
  if (n0 % 8 != 0) return fail(c, CSAT_ERR_SHAPE, "csat_compress_partial: n0 must be a multiple of 8");
  if (c->broken) return fail(c, CSAT_ERR_STATE, kBrokenMsg);
  std::string why;
  if (!on_device(c, &why)) return fail(c, CSAT_ERR_STATE, why);
  if (*(volatile int*)c->status != 0)
    return fail(c, CSAT_ERR_TIMEOUT, "a bounded device-side wait of an earlier launch gave up; its output is invalid");
  NvtxRange range("csat_compress_partial");
  cudaStream_t s = (cudaStream_t)stream;
  int launches = 0;
  const bool tc = c->tmap_phi_valid && c->force_simt != 1;
  cudaError_t e = tc ? csat::launch_sm100_compress(c, K_shard, V_shard, s, &launches, n0, n_len, partial_out)
                     : csat::launch_simt_compress(c, K_shard, V_shard, s, &launches, n0, n_len, partial_out);
  if (e != cudaSuccess) return fail_cuda(c, e, "csat_compress_partial launch");
  c->last_launches = launches;
  return CSAT_OK;
}

int csat_reduce_partials(csat_ctx* c, const float* partials, int count, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  c->saved_valid = false;
  if (!partials || !aligned16(partials)) return fail(c, CSAT_ERR_INVALID_ARG, "csat_reduce_partials: NULL or misaligned pointer");
  if (count < 1 || count > 4096) return fail(c, CSAT_ERR_INVALID_ARG, "csat_reduce_partials: count must be in [1, 4096]");
  if (c->broken) return fail(c, CSAT_ERR_STATE, kBrokenMsg);
  std::string why;
  if (!on_device(c, &why)) return fail(c, CSAT_ERR_STATE, why);
  int launches = 0;
  cudaError_t e = csat::launch_reduce_partials(c, partials, count, (cudaStream_t)stream, &launches);
  if (e != cudaSuccess) return fail_cuda(c, e, "csat_reduce_partials launch");
  c->have_forward = true;                 // the workspace now holds K~|V~
  c->last_launches = launches;
  return CSAT_OK;
}

int csat_attend(csat_ctx* c, const void* Q, void* out, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  c->saved_valid = false;
  if (!Q || !out) return fail(c, CSAT_ERR_INVALID_ARG, "csat_attend: NULL tensor pointer");
  if (!aligned16(Q) || !aligned16(out)) return fail(c, CSAT_ERR_INVALID_ARG, "csat_attend: tensor pointers must be 16-byte aligned");
  if (c->broken) return fail(c, CSAT_ERR_STATE, kBrokenMsg);
  if (!c->have_forward)
    return fail(c, CSAT_ERR_STATE, "csat_attend: the workspace holds no K~|V~ yet (csat_reduce_partials or csat_forward first)");
  {
    const csat::Params& p = c->p;
    const size_t bq = (size_t)(p.B * p.H * p.nq * p.d) * csat::elt_size(p.dtype);
    if (ranges_overlap(out, bq, Q, bq)) return fail(c, CSAT_ERR_INVALID_ARG, "csat_attend: out overlaps Q");
  }
  std::string why;
  if (!on_device(c, &why)) return fail(c, CSAT_ERR_STATE, why);
  if (*(volatile int*)c->status != 0)
    return fail(c, CSAT_ERR_TIMEOUT, "a bounded device-side wait of an earlier launch gave up; its output is invalid");
  if (c->p.T > 0 && c->w_S && (c->w_layers != 1 || c->w_untied) && c->w_layers != c->p.T)
    return fail(c, CSAT_ERR_STATE, "the supplied LISTA weights are for a number of layers other than CSAT_T");
  NvtxRange range("csat_attend");
  cudaStream_t s = (cudaStream_t)stream;
  int launches = 0;
  if (c->p.T > 0) {
    int rc = ensure_decoder(c, s, &launches);
    if (rc != CSAT_OK) return rc;
  }
  const bool tc_attend = c->tmap_phi_valid && c->force_simt == 0;
  cudaError_t e = tc_attend ? csat::launch_sm100_attend_recover(c, Q, out, s, &launches)
                            : csat::launch_simt_attend_recover(c, Q, out, s, &launches);
  if (e != cudaSuccess) return fail_cuda(c, e, "csat_attend launch");
  c->last_launches = launches;
  return CSAT_OK;
}

// scratch of csat_backward (and of a csat_forward that saves for it), (re)allocated when a size has changed
static int ensure_backward_scratch(csat_ctx* c) {
  const csat::Params& p = c->p;
  const size_t bz = (size_t)(p.B * p.H * p.nq * p.d) * 4, bl = (size_t)(p.B * p.H * p.nq * 2) * 4 + 1024 /* read past the end by whole-tile copies */,
               bk = (size_t)(p.B * p.H * p.m * 2 * p.d) * 4,
               bw = (size_t)(2 * (c->w_untied ? c->w_layers : 1) * p.H * p.d * p.d) * 4,
               b16 = c->tmap_phi_valid ? bk / 2 : 0, z16 = c->tmap_phi_valid ? bz / 2 : 0,
               bm = c->keep_masks && p.T > 0 ? bz : 0,
               bmb = c->tmap_phi_valid ? (size_t)(p.B * p.H * p.T * p.nq * (p.d / 32)) * 4 : 0,
               bal = c->weight_grads ? (size_t)((p.T + 1) * p.B * p.H * p.nq * p.d) * 2 : 0,
               bdx = c->weight_grads ? (size_t)(p.T * p.B * p.H * p.nq * p.d) * 2 : 0,
               wz = (size_t)(c->w_untied && p.T > 0 ? p.T : 1),      // one dS, dB per layer with per-layer weights
               bwp = c->weight_grads ? (size_t)(csat::wgrad_splits(c) * p.H * 2 * p.d * p.d) * wz * 4 : 0,
               bsg = c->weight_grads ? bmb : 0,
               bth = c->weight_grads ? (size_t)((csat::wgrad_splits(c) > 64 ? csat::wgrad_splits(c) : 64) * p.T * p.H) * 4 : 0,
               bwg = c->weight_grads ? ((size_t)(2 * p.H * p.d * p.d) * wz + (size_t)(p.d * p.d + p.T * p.H)) * 4 : 0;
  if (c->bw_bytes_signbits != bsg || c->bw_bytes_alpha16 != bal || c->bw_bytes_dx16 != bdx || c->bw_bytes_wpart != bwp || c->bw_bytes_thpart != bth ||
      c->bw_bytes_wgrad != bwg || c->bw_bytes_maskbits != bmb || c->bw_bytes_Z16 != z16 || c->bw_bytes_masks != bm || c->bw_bytes_dZ != bz || c->bw_bytes_LD != bl || c->bw_bytes_dKV != bk || c->bw_bytes_WT != bw ||
      c->bw_bytes_dKV16 != b16 || c->bw_bytes_dZ16 != z16) {
    cudaDeviceSynchronize();
    free_backward(c);
    c->bw_bytes_dZ = bz; c->bw_bytes_LD = bl; c->bw_bytes_dKV = bk; c->bw_bytes_WT = bw; c->bw_bytes_dKV16 = b16;
    c->bw_bytes_dZ16 = z16;
    c->bw_bytes_masks = bm;
    c->bw_bytes_Z16 = z16;
    c->bw_bytes_maskbits = bmb;
    c->bw_bytes_alpha16 = bal; c->bw_bytes_dx16 = bdx; c->bw_bytes_wpart = bwp; c->bw_bytes_thpart = bth; c->bw_bytes_wgrad = bwg;
    c->bw_bytes_signbits = bsg;
    if (dev_alloc(c, &c->bw_signbits, bsg) != cudaSuccess || dev_alloc(c, &c->bw_alpha16, bal) != cudaSuccess || dev_alloc(c, &c->bw_dx16, bdx) != cudaSuccess ||
        dev_alloc(c, &c->bw_wpart, bwp) != cudaSuccess || dev_alloc(c, &c->bw_thpart, bth) != cudaSuccess ||
        dev_alloc(c, &c->bw_wgrad, bwg) != cudaSuccess || dev_alloc(c, &c->bw_maskbits, bmb) != cudaSuccess || dev_alloc(c, &c->bw_Z16, z16) != cudaSuccess || dev_alloc(c, &c->bw_masks, bm) != cudaSuccess || dev_alloc(c, &c->bw_dZ, bz) != cudaSuccess || dev_alloc(c, &c->bw_LD, bl) != cudaSuccess ||
        dev_alloc(c, &c->bw_dKV, bk) != cudaSuccess || dev_alloc(c, &c->bw_WT, bw) != cudaSuccess ||
        dev_alloc(c, &c->bw_dKV16, b16) != cudaSuccess || dev_alloc(c, &c->bw_dZ16, z16) != cudaSuccess) {
      free_backward(c);
      return fail(c, CSAT_ERR_ALLOC, "cudaMalloc(backward scratch) failed");
    }
  }
  return CSAT_OK;
}

int csat_backward(csat_ctx* c, const void* Q, const void* K, const void* V, const void* dOut, void* dQ, void* dK,
                  void* dV, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  if (!Q || !K || !V || !dOut || !dQ || !dK || !dV) return fail(c, CSAT_ERR_INVALID_ARG, "csat_backward: NULL pointer");
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(dOut) || !aligned16(dQ) || !aligned16(dK) ||
      !aligned16(dV))
    return fail(c, CSAT_ERR_INVALID_ARG, "csat_backward: pointers must be 16-byte aligned");
  if (c->broken) return fail(c, CSAT_ERR_STATE, kBrokenMsg);
  NvtxRange range("csat_backward");
  std::string why;
  if (!on_device(c, &why)) return fail(c, CSAT_ERR_STATE, why);
  if (*(volatile int*)c->status != 0)
    return fail(c, CSAT_ERR_TIMEOUT, "a bounded device-side wait of an earlier launch gave up; its output is invalid");
  const csat::Params& p = c->p;
  const bool tc_all_stages = c->tmap_phi_valid && c->force_simt == 0 && !c->keep_masks;
  if (p.T > 32 && !tc_all_stages)
    return fail(c, CSAT_ERR_UNSUPPORTED,
                "csat_backward: the float32 kernels and CSAT_KEEP_MASKS keep one decision bit per layer in a 32-bit "
                "word: CSAT_T <= 32");
  if (p.d > 256) return fail(c, CSAT_ERR_UNSUPPORTED, "csat_backward: d <= 256");
  if (c->weight_grads && !(c->tmap_phi_valid && c->force_simt == 0 && p.T > 0))
    return fail(c, CSAT_ERR_UNSUPPORTED,
                "CSAT_WEIGHT_GRADS: the gradients of the decoder's parameters are formed on the tensor-core path only "
                "(bf16, d in {64, 128}, CSAT_T > 0)");
  if (p.B * p.H > 32767) return fail(c, CSAT_ERR_UNSUPPORTED, "csat_backward: B * H <= 32767");
  if (p.T > 0 && c->w_S && (c->w_layers != 1 || c->w_untied) && c->w_layers != p.T)
    return fail(c, CSAT_ERR_STATE, "the supplied LISTA weights are for a number of layers other than CSAT_T");
  cudaStream_t s = (cudaStream_t)stream;
  int launches = 0;
  if (p.T > 0) {
    int rc = ensure_decoder(c, s, &launches);
    if (rc != CSAT_OK) return rc;
  }
  if (int rc = ensure_backward_scratch(c)) return rc;
  const bool tc_compress = c->tmap_phi_valid && c->force_simt != 1;
  // what a csat_forward with CSAT_SAVE_FOR_BACKWARD left (K~|V~, Z, the softmax statistics, the decisions, the iterates
  // if asked for) replaces the compression and the forward pass of this call
  c->reuse_saved = c->save_for_backward && c->saved_valid && c->tmap_phi_valid && c->force_simt == 0 &&
                   (!c->weight_grads || c->saved_alpha);
  cudaError_t e = cudaSuccess;
  if (!c->reuse_saved) {
    e = c->debug_canary ? cudaMemsetAsync(c->kv, 0xFF, kv_bytes(p), s) : cudaSuccess;
    if (e != cudaSuccess) return fail_cuda(c, e, "canary fill");
    e = tc_compress ? csat::launch_sm100_compress(c, K, V, s, &launches) : csat::launch_simt_compress(c, K, V, s, &launches);
    if (e != cudaSuccess) return fail_cuda(c, e, "csat_backward: compress launch");
  }
  e = csat::launch_backward(c, Q, dOut, dQ, dK, dV, s, &launches);
  c->reuse_saved = false;
  if (e != cudaSuccess) return fail_cuda(c, e, "csat_backward launch");
  c->have_masks = c->bw_masks != nullptr;
  c->have_wgrads = c->weight_grads && c->bw_wgrad != nullptr;
  c->have_dkv16 = c->bw_dKV16 != nullptr && c->tmap_phi_valid && c->force_simt == 0;
  c->have_forward = true;
  c->last_launches = launches;
  return CSAT_OK;
}

// streams and events of the pipelined host-buffer forward (created by its first call)
static int ensure_pipeline(csat_ctx* c) {
  if (c->pipe_ready) return CSAT_OK;
  cudaError_t e = cudaSuccess;
  for (int i = 0; i < 3 && e == cudaSuccess; ++i) e = cudaStreamCreateWithFlags(&c->pipe_stream[i], cudaStreamNonBlocking);
  for (int i = 0; i < csat_ctx::kPipeEvents && e == cudaSuccess; ++i)
    e = cudaEventCreateWithFlags(&c->pipe_event[i], cudaEventDisableTiming);
  if (e != cudaSuccess) return fail_cuda(c, e, "csat_forward_host: stream/event creation");
  c->pipe_ready = true;
  return CSAT_OK;
}

int csat_forward_host(csat_ctx* c, const void* Qh, const void* Kh, const void* Vh, void* outh, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  c->saved_valid = false;
  if (!Qh || !Kh || !Vh || !outh) return fail(c, CSAT_ERR_INVALID_ARG, "csat_forward_host: NULL pointer");
  if (c->broken) return fail(c, CSAT_ERR_STATE, kBrokenMsg);
  NvtxRange range("csat_forward_host");
  const csat::Params& p = c->p;
  const size_t es = csat::elt_size(p.dtype);
  const size_t bq = (size_t)(p.B * p.H * p.nq * p.d) * es, bkv = (size_t)(p.B * p.H * p.n * p.d) * es;
  if (c->stage_bytes_q != bq || c->stage_bytes_kv != bkv) {
    cudaDeviceSynchronize();
    free_staging(c);
    c->stage_bytes_q = bq; c->stage_bytes_kv = bkv;
    if (dev_alloc(c, &c->stage_q, bq) != cudaSuccess || dev_alloc(c, &c->stage_o, bq) != cudaSuccess ||
        dev_alloc(c, &c->stage_k, bkv) != cudaSuccess || dev_alloc(c, &c->stage_v, bkv) != cudaSuccess) {
      free_staging(c);
      return fail(c, CSAT_ERR_ALLOC, "cudaMalloc(staging) failed");
    }
  }
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e;
  const bool tensor_core_path = c->tmap_phi_valid && c->force_simt == 0;
  if (!tensor_core_path || c->prof_slots != 0) {
    // plain order: copy everything in, compute, copy out
    if ((e = cudaMemcpyAsync(c->stage_q, Qh, bq, cudaMemcpyHostToDevice, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(c->stage_k, Kh, bkv, cudaMemcpyHostToDevice, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(c->stage_v, Vh, bkv, cudaMemcpyHostToDevice, s)) != cudaSuccess)
      return fail_cuda(c, e, "host->device copy");
    int rc = csat_forward(c, c->stage_q, c->stage_k, c->stage_v, c->stage_o, stream);
    if (rc != CSAT_OK) return rc;
    if ((e = cudaMemcpyAsync(outh, c->stage_o, bq, cudaMemcpyDeviceToHost, s)) != cudaSuccess)
      return fail_cuda(c, e, "device->host copy");
    if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return fail_cuda(c, e, "csat_forward_host");
    if (*(volatile int*)c->status != 0) return fail(c, CSAT_ERR_TIMEOUT, "a bounded device-side wait gave up");
    return CSAT_OK;
  }

  // Pipelined: the job is cut into chunks of a few heads of one batch element (contiguous in every tensor); chunk
  // i's host->device copies, its two kernels and its device->host copy run on three streams, so that the copies
  // of neighbouring chunks overlap the compute and each other (the two directions of the bus are independent).
  std::string why;
  if (!on_device(c, &why)) return fail(c, CSAT_ERR_STATE, why);
  if (*(volatile int*)c->status != 0)
    return fail(c, CSAT_ERR_TIMEOUT, "a bounded device-side wait of an earlier launch gave up; its output is invalid");
  int rc = ensure_pipeline(c);
  if (rc != CSAT_OK) return rc;
  cudaStream_t s_in = c->pipe_stream[0], s_run = c->pipe_stream[1], s_out = c->pipe_stream[2];
  cudaEvent_t ev_start = c->pipe_event[0], ev_done = c->pipe_event[1];
  // order after the caller's stream
  if ((e = cudaEventRecord(ev_start, s)) != cudaSuccess || (e = cudaStreamWaitEvent(s_in, ev_start, 0)) != cudaSuccess ||
      (e = cudaStreamWaitEvent(s_run, ev_start, 0)) != cudaSuccess || (e = cudaStreamWaitEvent(s_out, ev_start, 0)) != cudaSuccess)
    return fail_cuda(c, e, "csat_forward_host: stream ordering");
  int launches = 0;
  if (p.T > 0) {
    rc = ensure_decoder(c, s_run, &launches);
    if (rc != CSAT_OK) return rc;
  }
  // Chunks are runs of consecutive (batch, head) pairs (contiguous in every tensor; a run may cross from one batch
  // element into the next): about four per batch element, fewer when that would need more events than there are.
  const int64_t pairs = p.B * p.H;
  const int64_t max_chunks = (csat_ctx::kPipeEvents - 2) / 2;
  int64_t per_chunk = (p.H + 3) / 4;
  if ((pairs + per_chunk - 1) / per_chunk > max_chunks) per_chunk = (pairs + max_chunks - 1) / max_chunks;
  int chunk = 0;
  for (int64_t bh0 = 0; bh0 < pairs; bh0 += per_chunk, ++chunk) {
    const int64_t cnt = pairs - bh0 < per_chunk ? pairs - bh0 : per_chunk;
    const size_t oq = (size_t)(bh0 * p.nq * p.d) * es, okv = (size_t)(bh0 * p.n * p.d) * es;
    const size_t nq_b = (size_t)(cnt * p.nq * p.d) * es, nkv_b = (size_t)(cnt * p.n * p.d) * es;
    cudaEvent_t ev_in = c->pipe_event[2 + 2 * chunk], ev_run = c->pipe_event[3 + 2 * chunk];
    if ((e = cudaMemcpyAsync((char*)c->stage_k + okv, (const char*)Kh + okv, nkv_b, cudaMemcpyHostToDevice, s_in)) != cudaSuccess ||
        (e = cudaMemcpyAsync((char*)c->stage_v + okv, (const char*)Vh + okv, nkv_b, cudaMemcpyHostToDevice, s_in)) != cudaSuccess ||
        (e = cudaMemcpyAsync((char*)c->stage_q + oq, (const char*)Qh + oq, nq_b, cudaMemcpyHostToDevice, s_in)) != cudaSuccess ||
        (e = cudaEventRecord(ev_in, s_in)) != cudaSuccess || (e = cudaStreamWaitEvent(s_run, ev_in, 0)) != cudaSuccess)
      return fail_cuda(c, e, "csat_forward_host: host->device copy");
    c->bh0 = bh0;
    c->bh_cnt = cnt;
    e = csat::launch_sm100_compress(c, c->stage_k, c->stage_v, s_run, &launches);
    if (e == cudaSuccess) e = csat::launch_sm100_attend_recover(c, c->stage_q, c->stage_o, s_run, &launches);
    c->bh0 = 0;
    c->bh_cnt = 0;
    if (e != cudaSuccess) return fail_cuda(c, e, "csat_forward_host: launch");
    if ((e = cudaEventRecord(ev_run, s_run)) != cudaSuccess || (e = cudaStreamWaitEvent(s_out, ev_run, 0)) != cudaSuccess ||
        (e = cudaMemcpyAsync((char*)outh + oq, (const char*)c->stage_o + oq, nq_b, cudaMemcpyDeviceToHost, s_out)) != cudaSuccess)
      return fail_cuda(c, e, "csat_forward_host: device->host copy");
  }
  // the caller's stream continues after the last copy; this call returns once everything has landed
  if ((e = cudaEventRecord(ev_done, s_out)) != cudaSuccess || (e = cudaStreamWaitEvent(s, ev_done, 0)) != cudaSuccess ||
      (e = cudaStreamSynchronize(s)) != cudaSuccess)
    return fail_cuda(c, e, "csat_forward_host");
  c->have_forward = true;
  c->last_launches = launches;
  if (*(volatile int*)c->status != 0) return fail(c, CSAT_ERR_TIMEOUT, "a bounded device-side wait gave up");
  return CSAT_OK;
}

int csat_project_qkv(csat_ctx* c, const void* Xq, const void* Xkv, const void* W, int64_t d_model, void* Q, void* K,
                     void* V, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  if (!Xq || !Xkv || !W || !Q || !K || !V) return fail(c, CSAT_ERR_INVALID_ARG, "csat_project_qkv: NULL pointer");
  if (!aligned16(Xq) || !aligned16(Xkv) || !aligned16(W) || !aligned16(Q) || !aligned16(K) || !aligned16(V))
    return fail(c, CSAT_ERR_INVALID_ARG, "csat_project_qkv: pointers must be 16-byte aligned");
  if (d_model < 1 || d_model > (1 << 20)) return fail(c, CSAT_ERR_INVALID_ARG, "csat_project_qkv: d_model out of range");
  NvtxRange range("csat_project_qkv");
  std::string why;
  if (!on_device(c, &why)) return fail(c, CSAT_ERR_STATE, why);
  if (*(volatile int*)c->status != 0)
    return fail(c, CSAT_ERR_TIMEOUT, "a bounded device-side wait of an earlier launch gave up; its output is invalid");
  const csat::Params& p = c->p;
  if (3 * p.H * p.d > (1 << 24)) return fail(c, CSAT_ERR_SHAPE, "csat_project_qkv: 3 H d too large");
  cudaStream_t s = (cudaStream_t)stream;
  const int hd = (int)(p.H * p.d);
  int launches = 0;
  cudaError_t e;
  if (Xq == Xkv && p.nq == p.n) {
    e = csat::launch_project(c, Xq, W, p.n, d_model, 0, 3 * hd, Q, K, V, s, &launches);
  } else {
    e = csat::launch_project(c, Xq, W, p.nq, d_model, 0, hd, Q, K, V, s, &launches);
    if (e == cudaSuccess) e = csat::launch_project(c, Xkv, W, p.n, d_model, hd, 2 * hd, Q, K, V, s, &launches);
  }
  if (e != cudaSuccess) return fail_cuda(c, e, "csat_project_qkv launch");
  c->last_launches = launches;
  return CSAT_OK;
}

int csat_get_compressed(const csat_ctx* c, void* kt, void* vt, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  csat_ctx* mc = const_cast<csat_ctx*>(c);
  if (c->broken) return fail(mc, CSAT_ERR_STATE, kBrokenMsg);
  if (!c->have_forward) return fail(mc, CSAT_ERR_STATE, "csat_get_compressed: no forward has run yet");
  if ((kt && !aligned16(kt)) || (vt && !aligned16(vt)))
    return fail(mc, CSAT_ERR_INVALID_ARG, "csat_get_compressed: misaligned pointer");
  cudaError_t e = csat::launch_split_kv(c, kt, vt, (cudaStream_t)stream);
  if (e != cudaSuccess) return fail_cuda(mc, e, "csat_get_compressed");
  return CSAT_OK;
}

int csat_get_decoder(csat_ctx* c, float* S_out, float* B_out, float* theta_out, float* mu_out, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  if (c->broken) return fail(c, CSAT_ERR_STATE, kBrokenMsg);
  cudaStream_t s = (cudaStream_t)stream;
  int launches = 0;
  int rc = ensure_decoder(c, s, &launches);
  if (rc != CSAT_OK) return rc;
  const csat::Params& p = c->p;
  cudaError_t e = cudaSuccess;
  if (S_out && e == cudaSuccess) e = cudaMemcpyAsync(S_out, c->S_dec, dd_bytes(p, 4), cudaMemcpyDeviceToDevice, s);
  if (B_out && e == cudaSuccess) e = cudaMemcpyAsync(B_out, c->B_dec, dd_bytes(p, 4), cudaMemcpyDeviceToDevice, s);
  if (theta_out && e == cudaSuccess) e = cudaMemcpyAsync(theta_out, c->thr(), (size_t)p.H * 4, cudaMemcpyDeviceToDevice, s);
  if (mu_out && e == cudaSuccess) e = cudaMemcpyAsync(mu_out, c->mu, (size_t)p.H * 4, cudaMemcpyDeviceToDevice, s);
  if (e != cudaSuccess) return fail_cuda(c, e, "csat_get_decoder");
  return CSAT_OK;
}

int csat_get_backward_masks(const csat_ctx* c, uint32_t* masks_out, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  csat_ctx* mc = const_cast<csat_ctx*>(c);
  if (!masks_out || !aligned16(masks_out)) return fail(mc, CSAT_ERR_INVALID_ARG, "csat_get_backward_masks: NULL or misaligned pointer");
  if (!c->have_masks)
    return fail(mc, CSAT_ERR_STATE, "csat_get_backward_masks: no csat_backward with CSAT_KEEP_MASKS = 1 and CSAT_T > 0 has run");
  cudaError_t e = cudaMemcpyAsync(masks_out, c->bw_masks, c->bw_bytes_masks, cudaMemcpyDeviceToDevice, (cudaStream_t)stream);
  if (e != cudaSuccess) return fail_cuda(mc, e, "csat_get_backward_masks");
  return CSAT_OK;
}

int csat_backward_phi(csat_ctx* c, const void* K, const void* V, float* dPhi, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  if (!K || !V || !dPhi) return fail(c, CSAT_ERR_INVALID_ARG, "csat_backward_phi: NULL pointer");
  if (!aligned16(K) || !aligned16(V) || !aligned16(dPhi))
    return fail(c, CSAT_ERR_INVALID_ARG, "csat_backward_phi: pointers must be 16-byte aligned");
  if (c->broken) return fail(c, CSAT_ERR_STATE, kBrokenMsg);
  if (!c->have_dkv16)
    return fail(c, CSAT_ERR_STATE,
                "csat_backward_phi: no csat_backward on the tensor-core path (bf16, d in {64, 128}) has run on this context");
  if (*(volatile int*)c->status != 0)
    return fail(c, CSAT_ERR_TIMEOUT, "a bounded device-side wait of an earlier launch gave up; its output is invalid");
  NvtxRange range("csat_backward_phi");
  int launches = 0;
  cudaError_t e = csat::launch_sm100_phigrad(c, K, V, dPhi, (cudaStream_t)stream, &launches);
  if (e != cudaSuccess) return fail_cuda(c, e, "csat_backward_phi launch");
  c->last_launches = launches;
  return CSAT_OK;
}

int csat_get_weight_grads(const csat_ctx* c, float* dS, float* dB, float* dtheta, float* dPsi, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  csat_ctx* mc = const_cast<csat_ctx*>(c);
  if (!dS || !dB || !dtheta) return fail(mc, CSAT_ERR_INVALID_ARG, "csat_get_weight_grads: NULL pointer");
  if (!c->have_wgrads)
    return fail(mc, CSAT_ERR_STATE, "csat_get_weight_grads: no csat_backward with CSAT_WEIGHT_GRADS = 1 has run");
  const csat::Params& p = c->p;
  const size_t dd = (size_t)(p.d * p.d), hdd = (size_t)p.H * dd * (size_t)(c->w_untied && p.T > 0 ? p.T : 1);
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e = cudaMemcpyAsync(dS, c->bw_wgrad, hdd * 4, cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(dB, c->bw_wgrad + hdd, hdd * 4, cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess && dPsi) e = cudaMemcpyAsync(dPsi, c->bw_wgrad + 2 * hdd, dd * 4, cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(dtheta, c->bw_wgrad + 2 * hdd + dd, (size_t)(p.T * p.H) * 4, cudaMemcpyDeviceToDevice, s);
  if (e != cudaSuccess) return fail_cuda(mc, e, "csat_get_weight_grads");
  return CSAT_OK;
}

int csat_get_profile(const csat_ctx* c, int64_t call_index, int cap, int* ids, float* ms, int* count) {
  if (!c || !count || cap < 0 || (cap > 0 && (!ids || !ms))) return CSAT_ERR_INVALID_ARG;
  csat_ctx* mc = const_cast<csat_ctx*>(c);
  if (c->prof_slots == 0) return fail(mc, CSAT_ERR_STATE, "csat_get_profile: CSAT_PROFILE is off");
  if (call_index < 0 || call_index >= c->prof_calls || call_index < c->prof_calls - c->prof_slots)
    return fail(mc, CSAT_ERR_STATE, "csat_get_profile: that call is not recorded");
  const int K = csat_ctx::kProfMaxKernels;
  const int slot = (int)(call_index % c->prof_slots);
  const int n = c->prof_count[slot];
  const cudaEvent_t* ev = &c->prof_events[(size_t)slot * (K + 1)];
  cudaError_t e = cudaEventSynchronize(ev[n]);
  if (e != cudaSuccess) return fail_cuda(mc, e, "csat_get_profile");
  *count = n;
  for (int i = 0; i < n && i < cap; ++i) {
    ids[i] = c->prof_ids[(size_t)slot * K + i];
    if ((e = cudaEventElapsedTime(&ms[i], ev[i], ev[i + 1])) != cudaSuccess) return fail_cuda(mc, e, "csat_get_profile");
  }
  return CSAT_OK;
}

int csat_selftest_wait_timeout(csat_ctx* c, int64_t limit_us, void* stream) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  if (limit_us < 1 || limit_us > 1000000) return fail(c, CSAT_ERR_INVALID_ARG, "csat_selftest_wait_timeout: limit_us must be in [1, 1000000]");
  std::string why;
  if (!on_device(c, &why)) return fail(c, CSAT_ERR_STATE, why);
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e = csat::launch_wait_timeout_selftest(c, (unsigned long long)limit_us * 1000ull, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return fail_cuda(c, e, "csat_selftest_wait_timeout");
  if (*(volatile int*)c->status == 0) return fail(c, CSAT_ERR_STATE, "the bounded wait did not report its time-out");
  return fail(c, CSAT_ERR_TIMEOUT, "a bounded device-side wait gave up (self-test)");
}

int csat_clear_status(csat_ctx* c, int* code_host) {
  if (!c) return CSAT_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  if (code_host) *code_host = *(volatile int*)c->status;
  *(volatile int*)c->status = 0;
  c->err.clear();
  return CSAT_OK;
}

int csat_debug_fail_alloc(int countdown) {
  if (countdown < 0) return CSAT_ERR_INVALID_ARG;
  g_fail_alloc_countdown.store(countdown);
  return CSAT_OK;
}

size_t csat_workspace_bytes(const csat_ctx* c) { return c ? c->bytes : 0; }

int csat_last_launch_count(const csat_ctx* c) { return c ? c->last_launches : 0; }

const char* csat_last_error(const csat_ctx* c) {
  if (!c) return g_create_error.c_str();
  if (c->status && *(volatile int*)c->status != 0 && c->err.empty())
    const_cast<csat_ctx*>(c)->err = "a bounded device-side wait gave up (CSAT_ERR_TIMEOUT)";
  return c->err.c_str();
}

}  // extern "C"
