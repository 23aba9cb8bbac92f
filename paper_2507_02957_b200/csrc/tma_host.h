// Host-side creation of TMA tensor maps (cuTensorMapEncodeTiled reached through the runtime's driver
// entry-point lookup, so the library does not link against libcuda and loads on machines without a GPU).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace csat {

// bf16 tensor of rank 3, innermost dimension contiguous; 128-byte swizzle; out-of-range elements read 0.
//   dims[0..2] = extents (inner first), strides_bytes[0..1] = byte strides of dims 1 and 2 (multiples of 16),
//   box[0..2] = tile extents (box[0] * 2 bytes must be 128).
// Returns cudaSuccess or cudaErrorUnknown (encode failed / entry point missing).
cudaError_t make_tmap_bf16_3d(CUtensorMap* out, const void* base, const uint64_t dims[3],
                              const uint64_t strides_bytes[2], const uint32_t box[3]);

}  // namespace csat
