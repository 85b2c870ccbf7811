// Host helpers for TMA tensor maps (cuTensorMapEncodeTiled, reached through the runtime's
// driver entry point so that the library links against the CUDA runtime only).
#pragma once

#include <cuda.h>

#include "fa_common.cuh"

namespace fa {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// nullptr if the driver does not export the encoder.
EncodeTiledFn encode_tiled_fn();

// 3-D view (dim, row, batch * KV head) of a bf16 window buffer [B][Hkv][rows][d]; box = 64 dims x
// 64 rows, 128-byte swizzle, rows past the end read as zero.  Maps are cached by (base, rows, d,
// heads).  False if rows == 0 (the map is zeroed and must not be used) or on an encoder error.
bool window_map(CUtensorMap* tm, const void* base, int rows, int d, int n_bh);

}  // namespace fa
