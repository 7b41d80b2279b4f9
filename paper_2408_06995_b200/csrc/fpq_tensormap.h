// Tensor maps for the TMA loads and stores of all kernels: one place that finds the driver's encoder and
// remembers the maps it has made.
#pragma once
#include <cuda.h>

namespace fpq {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// A function with the signature of cuTensorMapEncodeTiled that returns the map made earlier for the same
// arguments (address, extents, strides, box, element type and modes all compared) and calls the driver otherwise;
// nullptr if the driver's entry point cannot be found.  A layer called again on the same buffers (every step of
// a network) then costs no encoding.  Each host thread keeps its own small table: no lock, and a map is 128 bytes
// of plain data that depends on nothing but the arguments.
EncodeTiledFn tensor_map_encoder();

}  // namespace fpq
