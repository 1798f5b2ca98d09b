// Host-side helpers shared by the translation units of libunitscale.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/unitscale.h"

namespace us {
namespace host {
// Number of SMs of the current device (cached per device), or -1 on error.
int sm_count();
// cuTensorMapEncodeTiled, looked up through the runtime (the library does not link against libcuda); nullptr if unavailable.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn();
}  // namespace host
}  // namespace us
