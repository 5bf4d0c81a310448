// Host-side construction of TMA tensor maps for [tokens, heads, head_dim] bf16 tensors.
// The driver entry point is resolved at run time so that the library carries no link-time dependency
// on libcuda (it must load on a machine without a GPU driver).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mpipe {

// View a [T, H, D] tensor (element strides tok_stride / head_stride, D contiguous) as the 3-D tensor
// (D, H, T) and describe boxes of box_d x 1 x box_rows elements.  elem_bytes is 2 (bf16) or 4 (fp32);
// swizzle_bytes is 128, 64 or 32 and must equal box_d * elem_bytes.  Out-of-range elements read as
// zero and are not written.  Returns false on failure.
bool make_tensor_map_thd(CUtensorMap* out, const void* base, int64_t T, int64_t H, int64_t D, int64_t tok_stride,
                         int64_t head_stride, uint32_t box_d, uint32_t box_rows, int swizzle_bytes,
                         int elem_bytes = 2);

}  // namespace mpipe
