// e2egrec_aggregate_forward_static: whole-graph mean aggregation for callers that cannot allocate.
//
// The same launches as e2egrec_aggregate_forward (same kernels, same run lengths, same summation order, hence the
// same bits), but the partial-sum scratch is a fixed array that is part of the library image, so the call needs no
// workspace argument and never touches an allocator.
#include <mutex>
#include <stdio.h>

#include "internal.cuh"

namespace e2egrec {

// Scratch of the segment reduction (one fp32 row per window for a segment that continues from earlier windows, one
// for a segment that continues into later ones, one record per window).  8 MiB; every device that loads the library
// carries it until the process exits.
constexpr size_t kStaticScratchBytes = size_t(8) << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;

// Device address of g_static_scratch per device ordinal.  In host code the array's name is only a
// handle for the runtime; the address a kernel can use comes from cudaGetSymbolAddress, asked once
// per device while that device is current.
static std::mutex g_static_mutex;
static void *g_static_addr[kMaxDevices] = {};

static int32_t static_scratch_address(void **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        set_last_error("aggregate_forward_static: cannot identify the current device");
        return E2EGREC_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_addr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) {
            char buf[200];
            snprintf(buf, sizeof(buf), "aggregate_forward_static: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
            set_last_error(buf);
            return E2EGREC_ERR_CUDA;
        }
        g_static_addr[dev] = p;
    }
    *out = g_static_addr[dev];
    return E2EGREC_OK;
}

}  // namespace e2egrec

using namespace e2egrec;

extern "C" size_t e2egrec_aggregate_forward_static_limit(void) { return kStaticScratchBytes; }

extern "C" int32_t e2egrec_aggregate_forward_static(int64_t n_dst, int64_t n_entries, const int64_t *indptr,
                                                    const int32_t *indices, const e2egrec_mat *X,
                                                    const e2egrec_mat *out, uint32_t flags, void *stream)
{
    if (n_dst < 0 || n_entries < 0) return E2EGREC_ERR_ARG;
    if (n_dst >= (1ll << 31)) return E2EGREC_ERR_UNSUPPORTED;
    int32_t rc = check_mats(X, out, n_dst);
    if (rc != E2EGREC_OK) return rc;
    if (!indptr || (n_entries > 0 && !indices)) return E2EGREC_ERR_NULL;
    const size_t need = full_ws_bytes(n_entries, X->dim, X->dtype);
    if (need > kStaticScratchBytes) {
        char buf[200];
        snprintf(buf, sizeof(buf),
                 "aggregate_forward_static: %lld entries x dim %d need %zu bytes of scratch, the built-in buffer holds %zu",
                 (long long)n_entries, X->dim, need, kStaticScratchBytes);
        set_last_error(buf);
        return E2EGREC_ERR_WORKSPACE;
    }
    void *base = nullptr;
    rc = static_scratch_address(&base);
    if (rc != E2EGREC_OK) return rc;
    return full_aggregate(n_dst, n_entries, indptr, indices, nullptr, X, out, (flags & E2EGREC_AGG_SUM) ? 0 : 1, base,
                          static_cast<cudaStream_t>(stream));
}
