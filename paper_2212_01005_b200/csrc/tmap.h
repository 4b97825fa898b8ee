// Host-side encoding of TMA tensor maps (bf16 tiles) through the driver entry
// point, fetched at run time so the library links against the runtime only.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <string>

namespace ago {

// rank <= 5; dims / box innermost first (elements); strides in bytes for dims 1..rank-1
// (multiples of 16). swizzle_bytes in {0, 32, 64, 128}; the inner box extent in
// bytes must not exceed it when it is non-zero. Out-of-bounds elements read 0.
bool encode_tmap_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                      const uint32_t* box, int swizzle_bytes, std::string* err);

}  // namespace ago
