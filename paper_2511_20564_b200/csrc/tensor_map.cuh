// Tensor maps and the TMA row gather (cp.async.bulk.tensor, tile::gather4) shared by the kernels that stream gathered
// rows through shared memory.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <stdint.h>

namespace e2egrec {

typedef CUresult (*TensorMapEncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                      const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline TensorMapEncodeFn tensor_map_encode_fn()
{
    static TensorMapEncodeFn fn = []() -> TensorMapEncodeFn {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<TensorMapEncodeFn>(p);
    }();
    return fn;
}

// A bf16 table [rows x d] with leading dimension ld (elements) as a 2-D tensor whose box is one row: the map of a row
// gather.  base 16-byte aligned, ld * 2 a multiple of 16, d <= 256, rows < 2^31.
inline bool make_row_gather_map(CUtensorMap *map, const void *base, int64_t rows, int d, int64_t ld)
{
    TensorMapEncodeFn fn = tensor_map_encode_fn();
    if (!fn || rows <= 0 || rows > 0x7fffffffll || d <= 0 || d > 256) return false;
    if (reinterpret_cast<uintptr_t>(base) % 16 || (ld * 2) % 16) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)d, 1};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

#ifdef __CUDACC__
__device__ inline uint32_t tm_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Bounded wait for the phase with the given parity of an mbarrier that only the calling warp uses.  Each try may
// suspend the thread for up to kTmWaitHintNs inside the hardware, so a warp that waits for its rows leaves the issue
// slots to the others instead of polling.
constexpr uint32_t kTmWaitHintNs = 2000;
__device__ inline bool tm_mbar_wait(uint64_t *bar, uint32_t parity)
{
    const uint32_t addr = tm_smem_u32(bar);
    for (uint32_t it = 0; it < 4u * 1000u * 1000u; ++it) {
        uint32_t done;
        asm volatile(
            "{\n"
            ".reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
            "selp.u32 %0, 1, 0, p;\n"
            "}\n"
            : "=r"(done)
            : "r"(addr), "r"(parity), "r"(kTmWaitHintNs)
            : "memory");
        if (done) return true;
    }
    return false;
}

__device__ inline void tm_mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(tm_smem_u32(bar)), "r"(count));
}

// One thread: the slot was read through the generic proxy; order those reads before the copy that overwrites it, tell
// the barrier how many bytes to expect (four rows of row_bytes) and start the copy of rows r0 .. r3 of the map's table.
// A row index outside the table reads zeros.
__device__ inline void tm_gather4(void *smem_dst, const CUtensorMap *map, int r0, int r1, int r2, int r3, uint64_t *bar,
                                  uint32_t row_bytes)
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(tm_smem_u32(bar)), "r"(4 * row_bytes) : "memory");
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(tm_smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(r0), "r"(r1), "r"(r2), "r"(r3),
        "r"(tm_smem_u32(bar))
        : "memory");
}
#endif

}  // namespace e2egrec
