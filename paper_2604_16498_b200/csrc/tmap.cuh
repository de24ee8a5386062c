// Host-side construction of TMA tensor maps.  The driver entry point is looked up through
// the runtime, so the library does not link against libcuda and still loads on a machine
// without a driver.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace forge {

// Encodes a tiled tensor map over 16-bit elements with 128-byte swizzle.
//   rank      : 2 or 3
//   dims[i]   : extent of dimension i in elements, innermost first
//   strides[i]: byte stride of dimension i+1 (rank-1 entries), multiples of 16
//   box[i]    : tile extent of dimension i; box[0] * 2 bytes must be 128 (one swizzle span)
// Returns false (and records the CUDA error, if any) on failure.
bool encode_tmap_bf16_sw128(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                            const uint64_t* strides_bytes, const uint32_t* box);

// Encodes a tiled tensor map over 16-bit elements without swizzle (the tile lies row by row in shared memory);
// box[0] * 2 bytes must be a multiple of 16.  Same conventions and return value as above.
bool encode_tmap_bf16_plain(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                            const uint64_t* strides_bytes, const uint32_t* box);

// Encodes a tiled tensor map over bytes without swizzle (the tile lands row by row).  box[0] must be a
// multiple of 16 bytes.  Same conventions and return value as above.
bool encode_tmap_u8_plain(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                          const uint64_t* strides_bytes, const uint32_t* box);

}  // namespace forge
