// Host-side helpers shared by the tensor-core kernels' launchers.
#pragma once

#include <cuda.h>

namespace sqn {

// cuTensorMapEncodeTiled for a tensor of 16-bit elements (bf16, or fp16 when f16 is set): `rank` dimensions (innermost
// first), strides of dimensions 1.. in bytes, box extents, swizzle chosen by the box's inner extent in bytes
// (32/64/128, else none).  False on failure.
bool tmap_encode_16(CUtensorMap* m, int rank, const void* ptr, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
                    const cuuint32_t* box, unsigned inner_bytes, int f16);

int sm_count();     // SMs of the current device

}  // namespace sqn
