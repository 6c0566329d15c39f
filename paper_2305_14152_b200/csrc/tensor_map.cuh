// Host-side lookup of the driver's tensor-map encoder (cuTensorMapEncodeTiled), shared by
// every translation unit that builds TMA descriptors.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace peqa {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Resolved once per process through the runtime (no link against libcuda).
int tensor_map_encoder(EncodeTiledFn* out);

}  // namespace peqa
