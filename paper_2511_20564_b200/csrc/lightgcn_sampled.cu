// LightGCN (Sec. 3.1, Eqs. 4-7) on sampled blocks: no weights, no activation.  One propagation over a block is the
// weighted segment reduction of segreduce.cuh,
//     out_i = t_i * sum_{e in S(i)} s_{col e} * H[col e],     s_v = 1/sqrt|N(v)|,  t_i = sqrt|N(i)| / |S(i)|,
// (the sum over N(i) of Eqs. 4-5 estimated from the sampled multiset; exact when S(i) = N(i)), and the adjoint is the
// same reduction over the block's CSC with the two scales exchanged.
#include <algorithm>

#include "segreduce.cuh"

namespace e2egrec {
namespace {

constexpr int kLgRun = 32;            // entries per lane group of the segment reduction

struct LgPlan {
    int n_hops, d;
    size_t es;
    size_t s_off[kMaxHops], t_off[kMaxHops];     // per block: source scales [cap_src], destination scales [cap_dst]
    size_t h_off[kMaxHops];                      // H^(l+1), l = 0 .. L-1: [cap_dst of block L-1-l x d]
    size_t seg_off, seg_bytes, bytes;
};

int32_t plan_lightgcn(const e2egrec_block *blocks, int32_t n_hops, int d, int32_t dtype, bool backward, LgPlan *p)
{
    if (!blocks) return E2EGREC_ERR_NULL;
    if (n_hops < 1 || n_hops > kMaxHops) return E2EGREC_ERR_UNSUPPORTED;
    if (dtype != E2EGREC_F32 && dtype != E2EGREC_BF16) return E2EGREC_ERR_DTYPE;
    if (d < 1 || d > kMaxDim) return E2EGREC_ERR_UNSUPPORTED;
    p->n_hops = n_hops;
    p->d = d;
    p->es = dtype_size(dtype);
    if ((d * p->es) % 16) return E2EGREC_ERR_ALIGN;
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += align_up(b, 256); return o; };
    size_t seg = 0;
    for (int h = 0; h < n_hops; ++h) {
        const e2egrec_block &b = blocks[h];
        if (b.cap_dst < 0 || b.cap_src < b.cap_dst || b.cap_edges < 0) return E2EGREC_ERR_ARG;
        if (h + 1 < n_hops && blocks[h + 1].cap_dst < b.cap_src) return E2EGREC_ERR_ARG;    // F_h = D_(h+1)
        if (!backward) {
            p->s_off[h] = take((size_t)std::max(b.cap_src, 1) * sizeof(float));
            p->t_off[h] = take((size_t)std::max(b.cap_dst, 1) * sizeof(float));
        }
        seg = std::max(seg, seg_scratch_carve(b.cap_edges, kLgRun, d, p->es, nullptr).bytes);
    }
    if (backward) {                               // two gradient buffers of the largest inner frontier, and the scaled dY
        size_t rows = 1;
        for (int h = 0; h + 1 < n_hops; ++h) rows = std::max<size_t>(rows, (size_t)blocks[h].cap_src);
        p->h_off[0] = take(rows * d * p->es);
        p->h_off[1] = take(rows * d * p->es);
        p->h_off[2] = take((size_t)std::max(blocks[0].cap_dst, 1) * d * p->es);
    } else {
        for (int l = 0; l < n_hops; ++l) p->h_off[l] = take((size_t)std::max(blocks[n_hops - 1 - l].cap_dst, 1) * d * p->es);
    }
    p->seg_bytes = seg;
    p->seg_off = take(seg);
    p->bytes = off;
    return E2EGREC_OK;
}

// s_src[j] = s[F[j]] for the block's sources, t_dst[i] = (1/|S(i)|) / s[D[i]] for its destinations (0 without neighbours)
__global__ void lightgcn_scales_kernel(const int32_t *__restrict__ src_nodes, const int32_t *__restrict__ counts,
                                       const float *__restrict__ inv_cnt, const float *__restrict__ inv_sqrt_deg,
                                       float *__restrict__ s_src, float *__restrict__ t_dst)
{
    const int32_t n_src = counts[CNT_SRC], n_dst = counts[CNT_DST];
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n_src; j += (int64_t)gridDim.x * blockDim.x) {
        const float s = inv_sqrt_deg[src_nodes[j]];
        s_src[j] = s;
        if (j < n_dst) t_dst[j] = s > 0.f ? inv_cnt[j] / s : 0.f;
    }
}

struct LgLayers { const void *h[kMaxHops]; };

// Y[i] = (X[seed_i] + sum_l H^(l)[i]) / (L + 1) on the seed rows, summed in fp32 and rounded once
template <typename T>
__global__ void lightgcn_mean_kernel(const T *__restrict__ X, int64_t ldx, const int32_t *__restrict__ seed_ids,
                                     const int32_t *__restrict__ counts0, LgLayers layers, int n_layers, int d, float scale,
                                     T *__restrict__ Y, int64_t ldy)
{
    const int64_t cells = (int64_t)counts0[CNT_DST] * d;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < cells; c += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = c / d;
        const int k = (int)(c % d);
        float v = to_float<T>(X[(int64_t)seed_ids[i] * ldx + k]);
        for (int l = 0; l < n_layers; ++l) v += to_float<T>(static_cast<const T *>(layers.h[l])[i * d + k]);
        Y[i * ldy + k] = from_float<T>(v * scale);
    }
}

// out[i] = in[i] * scale (the seed rows of dY, stored in the feature type)
template <typename T>
__global__ void lightgcn_scale_rows_kernel(const T *__restrict__ in, int64_t ld_in, const int32_t *__restrict__ counts0, int d,
                                           float scale, T *__restrict__ out)
{
    const int64_t cells = (int64_t)counts0[CNT_DST] * d;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < cells; c += (int64_t)gridDim.x * blockDim.x)
        out[c] = from_float<T>(to_float<T>(in[(c / d) * ld_in + c % d]) * scale);
}

// G[i] += add[i] on the seed rows (stored again in the feature type)
template <typename T>
__global__ void lightgcn_add_rows_kernel(T *__restrict__ G, int64_t ld_g, const T *__restrict__ add,
                                         const int32_t *__restrict__ counts0, int d)
{
    const int64_t cells = (int64_t)counts0[CNT_DST] * d;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < cells; c += (int64_t)gridDim.x * blockDim.x) {
        T *g = G + (c / d) * ld_g + c % d;
        *g = from_float<T>(to_float<T>(*g) + to_float<T>(add[c]));
    }
}

unsigned lg_grid(int64_t n) { return (unsigned)std::min<int64_t>(std::max<int64_t>(1, ceil_div(n, 256)), 148 * 8); }

template <typename T>
int32_t forward_impl(const e2egrec_block *blocks, const LgPlan &p, const e2egrec_mat *X, const float *inv_sqrt_deg, char *ctx,
                     const e2egrec_mat *Y, cudaStream_t st)
{
    const int L = p.n_hops;
    for (int h = 0; h < L; ++h) {
        const e2egrec_block &b = blocks[h];
        note_launch();
        lightgcn_scales_kernel<<<lg_grid(b.cap_src), 256, 0, st>>>(b.src_nodes, b.counts, b.inv_cnt, inv_sqrt_deg,
                                                                   reinterpret_cast<float *>(ctx + p.s_off[h]),
                                                                   reinterpret_cast<float *>(ctx + p.t_off[h]));
    }
    LgLayers layers{};
    for (int l = 0; l < L; ++l) {
        const e2egrec_block &b = blocks[L - 1 - l];
        T *out = reinterpret_cast<T *>(ctx + p.h_off[l]);
        SegOut<T> o{};
        o.out = out;
        o.ld_out = p.d;
        o.seg_scale = reinterpret_cast<const float *>(ctx + p.t_off[L - 1 - l]);
        const SegScratch sc = seg_scratch_carve(b.cap_edges, kLgRun, p.d, p.es, ctx + p.seg_off);
        bool ok;
        if (l == 0)     // H^(0) rows are read straight from the feature table through the global ids
            ok = dispatch_seg_reduce<T, int32_t, true>(static_cast<const T *>(X->data), X->ld, b.indptr, b.nbr_global,
                                                  &b.counts[CNT_DST], 0, b.cap_dst, inv_sqrt_deg, kLgRun, p.d, X->dtype, nullptr,
                                                  sc, o, st);
        else
            ok = dispatch_seg_reduce<T, int32_t, true>(reinterpret_cast<const T *>(ctx + p.h_off[l - 1]), p.d, b.indptr, b.col,
                                                  &b.counts[CNT_DST], 0, b.cap_dst,
                                                  reinterpret_cast<const float *>(ctx + p.s_off[L - 1 - l]), kLgRun, p.d,
                                                  X->dtype, nullptr, sc, o, st);
        if (!ok) {
            set_last_error("lightgcn_sampled_forward: no kernel for this row width");
            return E2EGREC_ERR_UNSUPPORTED;
        }
        layers.h[l] = out;
    }
    note_launch();
    lightgcn_mean_kernel<T><<<lg_grid((int64_t)blocks[0].cap_dst * p.d), 256, 0, st>>>(
        static_cast<const T *>(X->data), X->ld, blocks[0].src_nodes, blocks[0].counts, layers, L, p.d, 1.0f / (float)(L + 1),
        static_cast<T *>(Y->data), Y->ld);
    return check_launch("lightgcn_sampled_forward");
}

template <typename T>
int32_t backward_impl(const e2egrec_block *blocks, const LgPlan &fp, const LgPlan &bp, int32_t dtype, const char *ctx,
                      const e2egrec_mat *dY, const e2egrec_mat *dX_rows, char *scratch, cudaStream_t st)
{
    const int L = fp.n_hops, d = fp.d;
    T *buf[2] = {reinterpret_cast<T *>(scratch + bp.h_off[0]), reinterpret_cast<T *>(scratch + bp.h_off[1])};
    T *dys = reinterpret_cast<T *>(scratch + bp.h_off[2]);
    const int32_t *counts0 = blocks[0].counts;
    note_launch();
    lightgcn_scale_rows_kernel<T><<<lg_grid((int64_t)blocks[0].cap_dst * d), 256, 0, st>>>(
        static_cast<const T *>(dY->data), dY->ld, counts0, d, 1.0f / (float)(L + 1), dys);
    const T *g_in = dys;
    for (int l = L - 1; l >= 0; --l) {
        const e2egrec_block &b = blocks[L - 1 - l];
        T *out = l == 0 ? static_cast<T *>(dX_rows->data) : buf[l & 1];
        const int64_t ld_out = l == 0 ? dX_rows->ld : d;
        SegOut<T> o{};
        o.out = out;
        o.ld_out = ld_out;
        o.seg_scale = reinterpret_cast<const float *>(ctx + fp.s_off[L - 1 - l]);
        const SegScratch sc = seg_scratch_carve(b.cap_edges, kLgRun, d, fp.es, scratch + bp.seg_off);
        if (!dispatch_seg_reduce<T, int32_t, true>(g_in, d, b.csc_ptr, b.csc_row, &b.counts[CNT_SRC], 0, b.cap_src,
                                                   reinterpret_cast<const float *>(ctx + fp.t_off[L - 1 - l]), kLgRun, d, dtype,
                                                   b.csc_col, sc, o, st)) {
            set_last_error("lightgcn_sampled_backward: no kernel for this row width");
            return E2EGREC_ERR_UNSUPPORTED;
        }
        note_launch();
        lightgcn_add_rows_kernel<T><<<lg_grid((int64_t)blocks[0].cap_dst * d), 256, 0, st>>>(out, ld_out, dys, counts0, d);
        g_in = out;
    }
    return check_launch("lightgcn_sampled_backward");
}

}  // namespace
}  // namespace e2egrec

using namespace e2egrec;

extern "C" int32_t e2egrec_lightgcn_sampled_forward(const e2egrec_block *blocks, int32_t n_hops, const e2egrec_mat *X,
                                                    const float *inv_sqrt_deg, void *ctx, size_t *ctx_bytes,
                                                    const e2egrec_mat *Y, void *stream)
{
    if (!ctx_bytes || !X) return E2EGREC_ERR_NULL;
    LgPlan p;
    int32_t rc = plan_lightgcn(blocks, n_hops, X->dim, X->dtype, false, &p);
    if (rc != E2EGREC_OK) return rc;
    if (!ctx) { *ctx_bytes = p.bytes; return E2EGREC_OK; }
    if (*ctx_bytes < p.bytes) { *ctx_bytes = p.bytes; return E2EGREC_ERR_WORKSPACE; }
    if (reinterpret_cast<uintptr_t>(ctx) % 256) return E2EGREC_ERR_ALIGN;
    if (!X->data || !inv_sqrt_deg || !Y || !Y->data) return E2EGREC_ERR_NULL;
    if (Y->dtype != X->dtype) return E2EGREC_ERR_DTYPE;
    if (Y->dim != X->dim || Y->rows < blocks[0].cap_dst || X->ld < X->dim || Y->ld < Y->dim) return E2EGREC_ERR_ARG;
    if ((X->ld * p.es) % 16 || reinterpret_cast<uintptr_t>(X->data) % 16) return E2EGREC_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (X->dtype == E2EGREC_BF16) return forward_impl<__nv_bfloat16>(blocks, p, X, inv_sqrt_deg, static_cast<char *>(ctx), Y, st);
    return forward_impl<float>(blocks, p, X, inv_sqrt_deg, static_cast<char *>(ctx), Y, st);
}

extern "C" int32_t e2egrec_lightgcn_sampled_backward(const e2egrec_block *blocks, int32_t n_hops, const void *ctx,
                                                     const e2egrec_mat *dY, const e2egrec_mat *dX_rows, void *scratch,
                                                     size_t *scratch_bytes, void *stream)
{
    if (!scratch_bytes || !dY) return E2EGREC_ERR_NULL;
    LgPlan fp, bp;
    int32_t rc = plan_lightgcn(blocks, n_hops, dY->dim, dY->dtype, false, &fp);
    if (rc == E2EGREC_OK) rc = plan_lightgcn(blocks, n_hops, dY->dim, dY->dtype, true, &bp);
    if (rc != E2EGREC_OK) return rc;
    if (!scratch) { *scratch_bytes = bp.bytes; return E2EGREC_OK; }
    if (*scratch_bytes < bp.bytes) { *scratch_bytes = bp.bytes; return E2EGREC_ERR_WORKSPACE; }
    if (reinterpret_cast<uintptr_t>(scratch) % 256 || reinterpret_cast<uintptr_t>(ctx) % 256) return E2EGREC_ERR_ALIGN;
    if (!ctx || !dY->data || !dX_rows || !dX_rows->data) return E2EGREC_ERR_NULL;
    if (dX_rows->dtype != dY->dtype) return E2EGREC_ERR_DTYPE;
    if (dX_rows->dim != dY->dim || dX_rows->rows < blocks[n_hops - 1].cap_src || dY->rows < blocks[0].cap_dst ||
        dY->ld < dY->dim || dX_rows->ld < dX_rows->dim)
        return E2EGREC_ERR_ARG;
    if ((dX_rows->ld * fp.es) % 16 || reinterpret_cast<uintptr_t>(dX_rows->data) % 16) return E2EGREC_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (SideStream *side = SideStream::get(st)) side->join_pending(st);     // a deferred block transposition
    if (dY->dtype == E2EGREC_BF16)
        return backward_impl<__nv_bfloat16>(blocks, fp, bp, dY->dtype, static_cast<const char *>(ctx), dY, dX_rows,
                                            static_cast<char *>(scratch), st);
    return backward_impl<float>(blocks, fp, bp, dY->dtype, static_cast<const char *>(ctx), dY, dX_rows,
                                static_cast<char *>(scratch), st);
}
