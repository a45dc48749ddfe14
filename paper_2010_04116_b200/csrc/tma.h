// Tensor-map construction shared by the kernels that stage operands with TMA.
#pragma once
#include <cuda.h>

namespace il {

// Tiled bf16 tensor map with 128-byte swizzle and zero fill outside the tensor.  dims/box have `rank`
// entries (innermost first); strides_bytes has rank-1 entries (stride of dimensions 1..rank-1, multiples
// of 16).  Returns false if the driver rejects the description.
bool tma_encode_bf16(CUtensorMap* tm, const void* ptr, int rank, const unsigned long long* dims,
                     const unsigned long long* strides_bytes, const unsigned* box);

// The same for fp32 tensors (inner box extent at most 32 elements = 128 bytes).
bool tma_encode_f32(CUtensorMap* tm, const void* ptr, int rank, const unsigned long long* dims,
                    const unsigned long long* strides_bytes, const unsigned* box);

}  // namespace il
