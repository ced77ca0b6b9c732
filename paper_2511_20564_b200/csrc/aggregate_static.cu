// e2egrec_aggregate_forward_static: whole-graph mean aggregation for callers that cannot allocate.
//
// Same kernels as e2egrec_aggregate_forward, but the partial-sum scratch is a fixed array that is part of
// the library image, so the call needs no workspace argument and never touches an allocator.
#include <mutex>
#include <stdio.h>

#include "aggregate.cuh"

namespace e2egrec {

// Two halves: partial sums of segments that continue from an earlier chunk ("head") and of segments
// that continue into a later chunk ("tail").  8 MiB in total; every device that loads the library
// carries it until the process exits.
constexpr size_t kStaticScratchBytes = size_t(8) << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kStaticChunk = 128;
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

template <typename T, int LPR, int CPL>
static void launch_static(const T *in, int64_t ld_in, const int64_t *ptr, const int32_t *idx, int64_t n_seg,
                          int64_t n_chunks, int d, float *head, float *tail, const SegOut<T> &o, cudaStream_t st)
{
    note_launch();
    seg_chunk_kernel<T, int64_t, LPR, CPL, false><<<(unsigned)ceil_div(n_chunks * 32, kAggThreads), kAggThreads, 0, st>>>(
        in, ld_in, ptr, idx, nullptr, n_seg, nullptr, kStaticChunk, d, head, tail, o);
    const int64_t empty_blocks = ceil_div((n_seg > 0 ? n_seg : 1) * 8, kAggThreads);
    note_launch();
    seg_finish_kernel<T, int64_t><<<(unsigned)(n_chunks + empty_blocks), kAggThreads, 0, st>>>(
        ptr, nullptr, n_seg, kStaticChunk, d, head, tail, n_chunks, o);
}

template <typename T>
static void dispatch_static(const e2egrec_mat *X, const e2egrec_mat *out, const int64_t *ptr, const int32_t *idx,
                            int64_t n_seg, int64_t n_chunks, int mean, float *head, float *tail, cudaStream_t st)
{
    SegOut<T> o{};
    o.out = static_cast<T *>(out->data);
    o.ld_out = out->ld;
    o.mean = mean;
    const T *in = static_cast<const T *>(X->data);
    const RowShape rs = row_shape(X->dim, X->dtype);
#define E2E_CASE(L, C) \
    if (rs.lpr == L && rs.cpl == C) return launch_static<T, L, C>(in, X->ld, ptr, idx, n_seg, n_chunks, X->dim, head, tail, o, st);
    E2E_CASE(4, 1) E2E_CASE(8, 1) E2E_CASE(16, 1) E2E_CASE(32, 1) E2E_CASE(32, 2) E2E_CASE(32, 4)
#undef E2E_CASE
}

}  // namespace e2egrec

using namespace e2egrec;

extern "C" size_t e2egrec_aggregate_forward_static_limit(void) { return kStaticScratchBytes; }

extern "C" int32_t e2egrec_aggregate_forward_static(int64_t n_dst, int64_t n_entries, const int64_t *indptr,
                                                    const int32_t *indices, const e2egrec_mat *X,
                                                    const e2egrec_mat *out, uint32_t flags, void *stream)
{
    if (!X || !out || !X->data || !out->data || !indptr || (n_entries > 0 && !indices)) return E2EGREC_ERR_NULL;
    if (n_dst < 0 || n_entries < 0) return E2EGREC_ERR_ARG;
    if (n_dst >= (1ll << 31)) return E2EGREC_ERR_UNSUPPORTED;
    if (X->dtype != E2EGREC_F32 && X->dtype != E2EGREC_BF16) return E2EGREC_ERR_DTYPE;
    if (out->dtype != X->dtype) return E2EGREC_ERR_DTYPE;
    if (X->dim < 1 || X->dim > kMaxDim) return E2EGREC_ERR_UNSUPPORTED;
    if (out->dim != X->dim || out->rows < n_dst || X->ld < X->dim || out->ld < out->dim) return E2EGREC_ERR_ARG;
    const size_t es = dtype_size(X->dtype);
    if ((X->dim * es) % 16 || (X->ld * es) % 16 || (out->ld * es) % 16 || reinterpret_cast<uintptr_t>(X->data) % 16 ||
        reinterpret_cast<uintptr_t>(out->data) % 16)
        return E2EGREC_ERR_ALIGN;
    const int64_t n_chunks = ceil_div(n_entries > 0 ? n_entries : 1, kStaticChunk);
    const size_t half = align_up((size_t)n_chunks * X->dim * sizeof(float), 256);
    if (2 * half > kStaticScratchBytes) {
        char buf[200];
        snprintf(buf, sizeof(buf),
                 "aggregate_forward_static: %lld entries x dim %d need %zu bytes of scratch, the built-in buffer holds %zu",
                 (long long)n_entries, X->dim, 2 * half, kStaticScratchBytes);
        set_last_error(buf);
        return E2EGREC_ERR_WORKSPACE;
    }
    void *base = nullptr;
    int32_t rc = static_scratch_address(&base);
    if (rc != E2EGREC_OK) return rc;
    float *head = static_cast<float *>(base);
    float *tail = reinterpret_cast<float *>(static_cast<char *>(base) + half);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int mean = (flags & E2EGREC_AGG_SUM) ? 0 : 1;
    if (X->dtype == E2EGREC_BF16) dispatch_static<__nv_bfloat16>(X, out, indptr, indices, n_dst, n_chunks, mean, head, tail, st);
    else dispatch_static<float>(X, out, indptr, indices, n_dst, n_chunks, mean, head, tail, st);
    return check_launch("aggregate_forward_static");
}
