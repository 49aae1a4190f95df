// Host access to the driver's tensor-map encoder (cuTensorMapEncodeTiled), looked up once through
// the runtime so that the library does not link against libcuda.
#pragma once
#include <cuda.h>

namespace rmsmp {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// nullptr when the driver entry point cannot be had.
EncodeTiledFn tensor_map_encoder();

}  // namespace rmsmp
