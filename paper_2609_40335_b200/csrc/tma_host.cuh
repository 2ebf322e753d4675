// Host-side construction of TMA tensor maps (driver entry point fetched through the
// runtime, so the library does not link against libcuda).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dp_common.cuh"

namespace dpg {

// bf16 tensor seen as (batch, rows, cols) with row pitch `ld` elements and batch pitch
// rows*ld; tiles of box_rows x box_cols elements, 128-byte swizzle (box_cols*2 == 128).
// Reads outside [0,cols) x [0,rows) x [0,batch) return zeros.
// Encoded maps are cached per (address, pitch, extents, box).
dp_status make_tmap_bf16_3d(CUtensorMap* out, const void* base, int64_t ld, int cols, int rows,
                            int batch, int box_cols, int box_rows);
// driver encodes made so far (cache misses)
long long tmap_encode_count();

}  // namespace dpg
