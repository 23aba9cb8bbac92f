#include "tma_host.h"

#include <mutex>

namespace csat {
namespace {

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
  static EncodeFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeFn>(p);
  });
  return fn;
}

}  // namespace

// The encoding is a pure function of its arguments, and callers ask for the same few maps (the caller's Q, K, V and
// output, the library's own buffers) on every launch: a small per-thread memo keeps the driver call off the launch path.
namespace {
struct TmapKey {
  const void* base;
  uint64_t dims[3], strides[2];
  uint32_t box[3];
  bool operator==(const TmapKey& o) const {
    return base == o.base && dims[0] == o.dims[0] && dims[1] == o.dims[1] && dims[2] == o.dims[2] &&
           strides[0] == o.strides[0] && strides[1] == o.strides[1] && box[0] == o.box[0] && box[1] == o.box[1] &&
           box[2] == o.box[2];
  }
};
struct TmapSlot {
  bool used = false;
  TmapKey key;
  CUtensorMap map;
};
constexpr int kTmapSlots = 64;
}  // namespace

cudaError_t make_tmap_bf16_3d(CUtensorMap* out, const void* base, const uint64_t dims[3],
                              const uint64_t strides_bytes[2], const uint32_t box[3]) {
  static thread_local TmapSlot memo[kTmapSlots];
  const TmapKey key{base, {dims[0], dims[1], dims[2]}, {strides_bytes[0], strides_bytes[1]}, {box[0], box[1], box[2]}};
  const uint64_t hsh = (reinterpret_cast<uintptr_t>(base) >> 8) * 0x9E3779B97F4A7C15ull + box[1] * 31u + dims[1];
  TmapSlot& slot = memo[(hsh >> 32) % kTmapSlots];
  if (slot.used && slot.key == key) {
    *out = slot.map;
    return cudaSuccess;
  }
  EncodeFn fn = encode_fn();
  if (!fn) return cudaErrorUnknown;
  cuuint64_t gdim[3] = {dims[0], dims[1], dims[2]};
  cuuint64_t gstr[2] = {strides_bytes[0], strides_bytes[1]};
  cuuint32_t bx[3] = {box[0], box[1], box[2]};
  cuuint32_t es[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), gdim, gstr, bx, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return cudaErrorUnknown;
  slot.used = true;
  slot.key = key;
  slot.map = *out;
  return cudaSuccess;
}

}  // namespace csat
