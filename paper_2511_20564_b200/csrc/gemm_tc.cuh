// Tensor-core (tcgen05) dense transform for bf16 operands.
#pragma once

#include "common.cuh"

namespace e2egrec {

// h' = act(cat W^T + b) for `rows` (a multiple of 128) rows of cat [rows x k] and W [n x k], both
// bf16 row-major; rows at and beyond *m_dev are written as zeros.  Returns false when the shape is
// outside what the kernel takes, in which case nothing was enqueued.
bool tc_update_forward(const __nv_bfloat16 *cat, int64_t rows, int k, const __nv_bfloat16 *W, int n, const float *bias,
                       int relu, __nv_bfloat16 *out, const int32_t *m_dev, cudaStream_t st);

}  // namespace e2egrec
