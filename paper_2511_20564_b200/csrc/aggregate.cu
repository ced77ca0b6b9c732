// Whole-graph mean aggregation and its transpose (no sampling): the same chunked segment
// reduction as the sampled backward pass, with 64-bit offsets so that rows of any degree are
// shared by many warps.
#include <algorithm>

#include "internal.cuh"
#include "segreduce.cuh"

namespace e2egrec {

// Entries per run of the segment reduction: long runs on large inputs (fewer window records, fewer cut segments),
// short ones where the input would not fill the machine otherwise.
static inline int full_run_len(int64_t n_entries)
{
    return n_entries >= (1ll << 24) ? 256 : n_entries >= (1ll << 22) ? 128 : n_entries >= (1ll << 20) ? 64 : 32;
}

size_t full_ws_bytes(int64_t n_entries, int d, int32_t dtype)
{
    return seg_scratch_carve(n_entries, full_run_len(n_entries), d, dtype_size(dtype), nullptr).bytes;
}

template <typename T, bool kWeight>
static bool dispatch_seg64(const T *in, int64_t ld_in, const int64_t *ptr, const int32_t *idx, int64_t n_seg,
                           int64_t n_entries, const float *w, int d, void *ws, const SegOut<T> &o, int32_t dtype,
                           cudaStream_t st)
{
    const int run_len = full_run_len(n_entries);
    const SegScratch sc = seg_scratch_carve(n_entries, run_len, d, dtype_size(dtype), ws);
    return dispatch_seg_reduce<T, int64_t, kWeight, 2>(in, ld_in, ptr, idx, nullptr, n_seg, n_seg, w, run_len, d, dtype, nullptr, sc, o, st);
}

static int32_t unsupported_width(const char *what)
{
    set_last_error(what);
    return E2EGREC_ERR_UNSUPPORTED;
}

int32_t check_mats(const e2egrec_mat *in, const e2egrec_mat *out, int64_t out_rows)
{
    if (!in || !out || !in->data || !out->data) return E2EGREC_ERR_NULL;
    if (in->dtype != E2EGREC_F32 && in->dtype != E2EGREC_BF16) return E2EGREC_ERR_DTYPE;
    if (out->dtype != in->dtype) return E2EGREC_ERR_DTYPE;
    if (in->dim < 1 || in->dim > kMaxDim) return E2EGREC_ERR_UNSUPPORTED;
    if (out->dim != in->dim || out->rows < out_rows || in->ld < in->dim || out->ld < out->dim) return E2EGREC_ERR_ARG;
    const size_t es = dtype_size(in->dtype);
    if ((in->dim * es) % 16 || (in->ld * es) % 16 || (out->ld * es) % 16 ||
        reinterpret_cast<uintptr_t>(in->data) % 16 || reinterpret_cast<uintptr_t>(out->data) % 16)
        return E2EGREC_ERR_ALIGN;
    return E2EGREC_OK;
}

// Shared body of the entry points (e2egrec_aggregate_forward_static calls it with the library's built-in scratch).
int32_t full_aggregate(int64_t n_seg, int64_t n_entries, const int64_t *ptr, const int32_t *idx, const float *w,
                       const e2egrec_mat *in, const e2egrec_mat *out, int mean, void *ws, cudaStream_t st)
{
    bool ok;
    if (in->dtype == E2EGREC_BF16) {
        using T = __nv_bfloat16;
        SegOut<T> o{};
        o.out = static_cast<T *>(out->data);
        o.ld_out = out->ld;
        o.mean = mean;
        ok = w ? dispatch_seg64<T, true>(static_cast<const T *>(in->data), in->ld, ptr, idx, n_seg, n_entries, w, in->dim, ws, o,
                                         in->dtype, st)
               : dispatch_seg64<T, false>(static_cast<const T *>(in->data), in->ld, ptr, idx, n_seg, n_entries, w, in->dim, ws, o,
                                          in->dtype, st);
    } else {
        using T = float;
        SegOut<T> o{};
        o.out = static_cast<T *>(out->data);
        o.ld_out = out->ld;
        o.mean = mean;
        ok = w ? dispatch_seg64<T, true>(static_cast<const T *>(in->data), in->ld, ptr, idx, n_seg, n_entries, w, in->dim, ws, o,
                                         in->dtype, st)
               : dispatch_seg64<T, false>(static_cast<const T *>(in->data), in->ld, ptr, idx, n_seg, n_entries, w, in->dim, ws, o,
                                          in->dtype, st);
    }
    if (!ok) return unsupported_width("aggregate: no kernel for this row width");
    return check_launch("aggregate");
}


}  // namespace e2egrec

using namespace e2egrec;

static int32_t aggregate_entry(int64_t n_seg, int64_t n_entries, const int64_t *ptr, const int32_t *idx, const float *w,
                               const e2egrec_mat *in, const e2egrec_mat *out, int mean, void *ws, size_t *ws_bytes,
                               void *stream)
{
    if (!ws_bytes) return E2EGREC_ERR_NULL;
    if (n_seg < 0 || n_entries < 0) return E2EGREC_ERR_ARG;
    if (n_seg >= (1ll << 31)) return E2EGREC_ERR_UNSUPPORTED;
    int32_t rc = check_mats(in, out, n_seg);
    if (rc != E2EGREC_OK) return rc;
    const size_t need = full_ws_bytes(n_entries, in->dim, in->dtype);
    if (!ws) { *ws_bytes = need; return E2EGREC_OK; }
    if (*ws_bytes < need) { *ws_bytes = need; return E2EGREC_ERR_WORKSPACE; }
    if (reinterpret_cast<uintptr_t>(ws) % 256) return E2EGREC_ERR_ALIGN;
    if (!ptr || (n_entries > 0 && !idx)) return E2EGREC_ERR_NULL;
    return full_aggregate(n_seg, n_entries, ptr, idx, w, in, out, mean, ws, static_cast<cudaStream_t>(stream));
}

extern "C" int32_t e2egrec_aggregate_forward(int64_t n_dst, int64_t n_entries, const int64_t *indptr,
                                             const int32_t *indices, const e2egrec_mat *X, const e2egrec_mat *out,
                                             uint32_t flags, void *ws, size_t *ws_bytes, void *stream)
{
    return aggregate_entry(n_dst, n_entries, indptr, indices, nullptr, X, out, (flags & E2EGREC_AGG_SUM) ? 0 : 1, ws,
                           ws_bytes, stream);
}

extern "C" int32_t e2egrec_aggregate_backward(int64_t n_src, int64_t n_entries, const int64_t *csc_ptr,
                                              const int32_t *csc_row, const float *inv_deg, const e2egrec_mat *G,
                                              const e2egrec_mat *dX, void *ws, size_t *ws_bytes, void *stream)
{
    return aggregate_entry(n_src, n_entries, csc_ptr, csc_row, inv_deg, G, dX, 0, ws, ws_bytes, stream);
}

// ------------------------------------------------------------------------------------------ LightGCN
namespace e2egrec {

struct LayerList { const void *p[9]; };

// Y = (sum of n_in matrices) * scale, summed in fp32 and rounded once
template <typename T>
__global__ void layer_mean_kernel(LayerList list, int n_in, int64_t cells, float scale, T *__restrict__ out)
{
    const T *const *in = reinterpret_cast<const T *const *>(list.p);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < cells; i += (int64_t)gridDim.x * blockDim.x) {
        float s = 0.f;
        for (int l = 0; l < n_in; ++l) s += to_float<T>(in[l][i]);
        out[i] = from_float<T>(s * scale);
    }
}

// out = A_hat in:  out[u] = s[u] * sum_{i in row u} s[i] * in[i]
static int32_t lightgcn_propagate(int64_t n, int64_t m, const int64_t *ptr, const int32_t *idx, const float *s,
                                  const e2egrec_mat *in, void *out_data, void *ws, cudaStream_t st)
{
    bool ok;
    if (in->dtype == E2EGREC_BF16) {
        using T = __nv_bfloat16;
        SegOut<T> o{};
        o.out = static_cast<T *>(out_data);
        o.ld_out = in->dim;
        o.seg_scale = s;
        ok = dispatch_seg64<T, true>(static_cast<const T *>(in->data), in->ld, ptr, idx, n, m, s, in->dim, ws, o, in->dtype, st);
    } else {
        using T = float;
        SegOut<T> o{};
        o.out = static_cast<T *>(out_data);
        o.ld_out = in->dim;
        o.seg_scale = s;
        ok = dispatch_seg64<T, true>(static_cast<const T *>(in->data), in->ld, ptr, idx, n, m, s, in->dim, ws, o, in->dtype, st);
    }
    if (!ok) return unsupported_width("lightgcn: no kernel for this row width");
    return check_launch("lightgcn_propagate");
}

}  // namespace e2egrec

// Shared body of e2egrec_lightgcn_forward / _backward: Y = (1/(L+1)) sum_{l=0..L} A^l H0 with A given by (ptr, idx, s).
static int32_t lightgcn_entry(int64_t n, int64_t m, const int64_t *ptr, const int32_t *idx, const float *s, int32_t n_layers,
                              const e2egrec_mat *H0, const e2egrec_mat *Y, void *ws, size_t *ws_bytes, void *stream)
{
    if (!ws_bytes) return E2EGREC_ERR_NULL;
    if (n < 0 || m < 0 || n_layers < 0 || n_layers > 8) return E2EGREC_ERR_ARG;
    if (n >= (1ll << 31)) return E2EGREC_ERR_UNSUPPORTED;
    int32_t rc = check_mats(H0, Y, n);
    if (rc != E2EGREC_OK) return rc;
    if (H0->ld != H0->dim || Y->ld != Y->dim) return E2EGREC_ERR_ARG;
    const size_t es = dtype_size(H0->dtype);
    const size_t layer_bytes = align_up((size_t)(n > 0 ? n : 1) * H0->dim * es, 256);
    const size_t seg_bytes = align_up(full_ws_bytes(m, H0->dim, H0->dtype), 256);
    const size_t need = seg_bytes + (size_t)n_layers * layer_bytes;
    if (!ws) { *ws_bytes = need; return E2EGREC_OK; }
    if (*ws_bytes < need) { *ws_bytes = need; return E2EGREC_ERR_WORKSPACE; }
    if (reinterpret_cast<uintptr_t>(ws) % 256) return E2EGREC_ERR_ALIGN;
    if (!ptr || !s || (m > 0 && !idx)) return E2EGREC_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *base = static_cast<char *>(ws);
    LayerList layers{};
    layers.p[0] = H0->data;
    e2egrec_mat cur = *H0;
    for (int l = 0; l < n_layers; ++l) {
        void *next = base + seg_bytes + (size_t)l * layer_bytes;
        rc = lightgcn_propagate(n, m, ptr, idx, s, &cur, next, base, st);
        if (rc != E2EGREC_OK) return rc;
        layers.p[l + 1] = next;
        cur.data = next;
    }
    const int64_t cells = n * H0->dim;
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(cells > 0 ? cells : 1, 256), 148 * 16);
    note_launch();
    if (H0->dtype == E2EGREC_BF16)
        layer_mean_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(layers, n_layers + 1, cells, 1.0f / (float)(n_layers + 1),
                                                             static_cast<__nv_bfloat16 *>(Y->data));
    else
        layer_mean_kernel<float><<<grid, 256, 0, st>>>(layers, n_layers + 1, cells,
                                                       1.0f / (float)(n_layers + 1), static_cast<float *>(Y->data));
    return check_launch("lightgcn");
}

extern "C" int32_t e2egrec_lightgcn_forward(int64_t n_nodes, int64_t n_entries, const int64_t *indptr,
                                            const int32_t *indices, const float *inv_sqrt_deg, int32_t n_layers,
                                            const e2egrec_mat *H0, const e2egrec_mat *Y, void *ws, size_t *ws_bytes,
                                            void *stream)
{
    return lightgcn_entry(n_nodes, n_entries, indptr, indices, inv_sqrt_deg, n_layers, H0, Y, ws, ws_bytes, stream);
}

extern "C" int32_t e2egrec_lightgcn_backward(int64_t n_nodes, int64_t n_entries, const int64_t *csc_ptr,
                                             const int32_t *csc_row, const float *inv_sqrt_deg, int32_t n_layers,
                                             const e2egrec_mat *dY, const e2egrec_mat *dH0, void *ws, size_t *ws_bytes,
                                             void *stream)
{
    return lightgcn_entry(n_nodes, n_entries, csc_ptr, csc_row, inv_sqrt_deg, n_layers, dY, dH0, ws, ws_bytes, stream);
}
