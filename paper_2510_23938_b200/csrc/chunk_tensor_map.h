// The tensor map that describes a blob's whole chunks to the TMA unit (tiled bulk copies).
#pragma once
#include <cuda.h>          // CUtensorMap (types only; the encoder is fetched through the runtime)

#include <cstdint>

namespace ivk {

// The blob's whole chunks as a 2-D byte tensor [rows][chunk_bytes] (row pitch = chunk size, a multiple of 16;
// d_data 16-byte aligned), box = 32 rows x 128 bytes, 128-byte swizzle.  False if the driver has no encoder
// or the extents do not fit.
bool make_chunk_tensor_map(CUtensorMap *map, const uint8_t *d_data, uint64_t chunk_bytes, uint64_t rows);

}  // namespace ivk
