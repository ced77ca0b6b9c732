#include "gemm_tc.cuh"

namespace e2egrec {

bool tc_update_forward(const __nv_bfloat16 *, int64_t, int, const __nv_bfloat16 *, int, const float *, int,
                       __nv_bfloat16 *, const int32_t *, cudaStream_t)
{
    return false;
}

}  // namespace e2egrec
