// GraphSAGE forward / backward over sampled blocks: host orchestration and kernel dispatch.
#include <algorithm>
#include <stdlib.h>

#include "aggregate.cuh"
#include "common.cuh"
#include "gemm_simt.cuh"
#include "gather_stream.cuh"
#include "gemm_tc.cuh"
#include "segreduce.cuh"

namespace e2egrec {

static inline int64_t pad128(int64_t rows) { return (rows + 127) / 128 * 128; }

struct LayerPlan {
    int block;          // index into blocks[]: layer l runs on block n_layers-1-l
    int d_in, d_out;
    int64_t rows;       // destination rows allocated (cap_dst rounded up to 128)
    size_t cat_off, h_off;    // offsets into ctx: [rows x 2 d_in], [rows x d_out]
};

// Layout of the saved activations; forward and backward derive it from the same arguments.
static int32_t plan_layers(const e2egrec_block *blocks, int32_t n_layers, const e2egrec_mat *X, const e2egrec_mat *W,
                           LayerPlan *plan, size_t *ctx_bytes)
{
    if (!blocks || !X || !W) return E2EGREC_ERR_NULL;
    if (n_layers < 1 || n_layers > kMaxHops) return E2EGREC_ERR_UNSUPPORTED;
    if (X->dtype != E2EGREC_F32 && X->dtype != E2EGREC_BF16) return E2EGREC_ERR_DTYPE;
    const size_t es = dtype_size(X->dtype);
    if (X->dim < 1 || X->dim > kMaxDim) return E2EGREC_ERR_UNSUPPORTED;
    if ((X->dim * es) % 16 || (X->ld * es) % 16 || reinterpret_cast<uintptr_t>(X->data) % 16) return E2EGREC_ERR_ALIGN;
    if (!X->data || X->ld < X->dim) return X->data ? E2EGREC_ERR_ARG : E2EGREC_ERR_NULL;
    size_t off = 0;
    int d_in = X->dim;
    for (int l = 0; l < n_layers; ++l) {
        const e2egrec_mat &w = W[l];
        if (!w.data) return E2EGREC_ERR_NULL;
        if (w.dtype != X->dtype) return E2EGREC_ERR_DTYPE;
        if (w.dim != 2 * d_in || w.ld != w.dim || w.rows < 1 || w.rows > kMaxDim) return E2EGREC_ERR_ARG;
        if ((w.rows * es) % 16 || reinterpret_cast<uintptr_t>(w.data) % 16) return E2EGREC_ERR_ALIGN;
        LayerPlan &p = plan[l];
        p.block = n_layers - 1 - l;
        p.d_in = d_in;
        p.d_out = (int)w.rows;
        p.rows = pad128(blocks[p.block].cap_dst);
        p.cat_off = off;
        off += align_up((size_t)p.rows * 2 * d_in * es, 256);
        p.h_off = off;
        off += align_up((size_t)p.rows * p.d_out * es, 256);
        d_in = p.d_out;
    }
    for (int l = 0; l + 1 < n_layers; ++l)      // the sources of a block are the destinations of the next one out
        if (blocks[plan[l + 1].block].cap_src > blocks[plan[l].block].cap_dst) return E2EGREC_ERR_ARG;
    *ctx_bytes = off;
    return E2EGREC_OK;
}

// ------------------------------------------------------------------------------ launch helpers
template <typename T, int LPR, int CPL>
static void launch_sage_aggregate(const T *Hsrc, int64_t ld, const int32_t *nbr, const int32_t *self_ids,
                                  const e2egrec_block &b, T *cat, int d, int64_t rows, cudaStream_t st)
{
    // one warp per destination at a time, the warps stride over the destinations: at most eight blocks per SM for the
    // capacities of small batches (most of such a grid finds no destination), 32 where a block can hold a million rows
    const int64_t per_sm = rows >= (1ll << 20) ? 32 : 8;
    const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>(ceil_div(rows * 32, kAggThreads), 148 * per_sm));
    note_launch();
    launch_pdl(sage_aggregate_kernel<T, LPR, CPL>, dim3(grid), dim3(kAggThreads), 0, st, Hsrc, ld, nbr, self_ids, b.indptr,
               b.counts, cat, d, (int32_t)rows);
}

template <typename T>
static bool dispatch_sage_aggregate(const T *Hsrc, int64_t ld, const int32_t *nbr, const int32_t *self_ids,
                                    const e2egrec_block &b, T *cat, int d, int64_t rows, int32_t dtype, cudaStream_t st)
{
    const RowShape rs = row_shape(d, dtype);
#define E2E_CASE(L, C)                                                                           \
    if (rs.lpr == L && rs.cpl == C) {                                                            \
        launch_sage_aggregate<T, L, C>(Hsrc, ld, nbr, self_ids, b, cat, d, rows, st);            \
        return true;                                                                             \
    }
    E2E_CASE(4, 1) E2E_CASE(8, 1) E2E_CASE(16, 1) E2E_CASE(32, 1) E2E_CASE(32, 2) E2E_CASE(32, 4)
    if constexpr (sizeof(T) == 4) {      // rows of 2049 .. 4096 bytes exist only for fp32 (dim <= kMaxDim)
        E2E_CASE(32, 8)
    }
#undef E2E_CASE
    return false;
}

// transposed-block entries per lane group: 16, or 128 where the block can hold a million entries or more (the longer run's
// lower overhead per entry wins there; measured on the 2 * 10^9-entry workload: 0.69 -> 0.63 ms)
// (longer runs were measured with the streamed rows as well: 256 entries 0.422 ms, 512 0.461, 1024 0.777 against 0.421)
// A block that can hold two million entries gets runs of 128 entries.  Where the rows can be streamed through shared
// memory (512-byte bf16 rows) the long runs and the streaming start at a million (2 * 10^9-entry workload: the outer
// block alone 2.207 ms per step, the middle block as well 2.168; with 2^17 the top block joins and its 0.065 ms become
// 0.127).  Capacities, not sizes, are what the host knows: a small batch in large buffers pays for the long runs (a
// 71 k-entry block in a 1.2 M-entry buffer: 0.327 -> 0.362 ms per joint step), hence no lower than this.
static inline bool streamable_rows(int d, size_t es) { return es == 2 && d == 256; }
static inline int64_t big_block_edges(int d, size_t es) { return streamable_rows(d, es) ? (1ll << 20) : (1ll << 21); }
static inline int block_run_len(int64_t cap_edges, int d, size_t es) { return cap_edges >= big_block_edges(d, es) ? 128 : 16; }
constexpr int kDwSplits = 148;        // split-K factor of the weight-gradient product

// A layer whose weight-gradient product may move this many bytes or more (by the capacity of its block) keeps that
// product on the caller's stream.  Beside the input-gradient product and the transposed aggregation of such a layer it
// only competes with them for the same HBM bandwidth and SM slots (measured on the 2 * 10^9-entry workload: the three
// kernels take 0.18 + 0.25 + 0.47 ms one after the other and 1.0 ms overlapped); small layers, whose kernels are
// bound by latency, gain from the overlap.  E2EGREC_DW_SERIAL_MB overrides the threshold (in MB).
static size_t dw_serial_bytes()
{
    static const size_t v = []() {
        const char *e = getenv("E2EGREC_DW_SERIAL_MB");
        const long mb = (e && *e) ? atol(e) : 256;
        return (size_t)(mb < 0 ? 0 : mb) << 20;
    }();
    return v;
}

// E2EGREC_FUSED_FORWARD=1: bf16 layers whose shapes allow it run Eq. 2 and Eq. 3 as one kernel (the aggregated rows are
// built in shared memory as the A operand of the dense transform).  Off by default: measured slower than the two
// kernels on every workload of the benchmark.
static bool fused_forward_enabled()
{
    static const bool on = []() { const char *e = getenv("E2EGREC_FUSED_FORWARD"); return e && *e && e[0] != '0'; }();
    return on;
}

// bf16 layers with 256-value rows whose block can hold a million entries or more aggregate with the rows streamed
// through shared memory by the TMA unit (gather_stream.cu) instead of register-staged loads: 0.347 -> 0.240 ms on the
// outer block of the 2 * 10^9-entry workload, same bits.  Smaller blocks are bound by launch and latency, where the
// one-warp-per-destination kernel is faster.  E2EGREC_NO_STREAM_GATHER=1 switches it off.
static bool stream_gather_enabled()
{
    static const bool off = []() { const char *e = getenv("E2EGREC_NO_STREAM_GATHER"); return e && *e && e[0] != '0'; }();
    return !off;
}

// ------------------------------------------------------------------------------ forward
template <typename T>
static int32_t forward_impl(const e2egrec_block *blocks, int32_t n_layers, const e2egrec_mat *X, const e2egrec_mat *W,
                            const float *const *bias, const int32_t *act, const LayerPlan *plan, char *ctx,
                            const e2egrec_mat *H_out, cudaStream_t st)
{
    const size_t es = sizeof(T);
    const int64_t out_rows = blocks[0].cap_dst < H_out->rows ? blocks[0].cap_dst : H_out->rows;
    bool top_stored = false;
    for (int l = 0; l < n_layers; ++l) {
        const LayerPlan &p = plan[l];
        const e2egrec_block &b = blocks[p.block];
        T *cat = reinterpret_cast<T *>(ctx + p.cat_off);
        T *hn = reinterpret_cast<T *>(ctx + p.h_off);
        if (X->dtype == E2EGREC_BF16 && fused_forward_enabled()) {
            const bool top = l == n_layers - 1;
            const __nv_bfloat16 *src = l == 0 ? static_cast<const __nv_bfloat16 *>(X->data)
                                              : reinterpret_cast<const __nv_bfloat16 *>(ctx + plan[l - 1].h_off);
            if (l == 0) tap_begin(TAP_AGG_FWD_OUTER, st);
            const bool fused = tc_sage_fused_forward(
                src, l == 0 ? X->ld : p.d_in, l == 0 ? b.nbr_global : b.col, l == 0 ? b.src_nodes : nullptr, b.indptr, p.d_in,
                reinterpret_cast<__nv_bfloat16 *>(cat), p.rows, static_cast<const __nv_bfloat16 *>(W[l].data), p.d_out,
                bias ? bias[l] : nullptr, act ? act[l] : 1, reinterpret_cast<__nv_bfloat16 *>(hn), &b.counts[CNT_DST],
                &b.counts[CNT_STATUS], st, top ? static_cast<__nv_bfloat16 *>(H_out->data) : nullptr, H_out->ld, out_rows);
            if (l == 0) tap_end(TAP_AGG_FWD_OUTER, st);
            if (fused) {
                if (l == 0) { tap_begin(TAP_UPDATE_FWD_OUTER, st); tap_end(TAP_UPDATE_FWD_OUTER, st); }
                top_stored = top_stored || top;
                continue;
            }
        }
        bool agg_ok = false;
        if (l == 0) tap_begin(TAP_AGG_FWD_OUTER, st);
        if (X->dtype == E2EGREC_BF16 && streamable_rows(p.d_in, sizeof(T)) && b.cap_edges >= big_block_edges(p.d_in, sizeof(T)) && stream_gather_enabled())
            agg_ok = stream_sage_aggregate(l == 0 ? static_cast<const __nv_bfloat16 *>(X->data)
                                                  : reinterpret_cast<const __nv_bfloat16 *>(ctx + plan[l - 1].h_off),
                                           l == 0 ? X->rows : plan[l - 1].rows, l == 0 ? X->ld : p.d_in,
                                           l == 0 ? b.nbr_global : b.col, l == 0 ? b.src_nodes : nullptr, b.indptr, b.counts,
                                           reinterpret_cast<__nv_bfloat16 *>(cat), p.d_in, p.rows, st);
        if (agg_ok) {
            if (l == 0) tap_end(TAP_AGG_FWD_OUTER, st);
        } else if (l == 0) {  // h^(0) rows are read straight from the feature table through the global ids
            agg_ok = dispatch_sage_aggregate<T>(static_cast<const T *>(X->data), X->ld, b.nbr_global, b.src_nodes, b, cat,
                                                p.d_in, p.rows, X->dtype, st);
            tap_end(TAP_AGG_FWD_OUTER, st);
        } else
            agg_ok = dispatch_sage_aggregate<T>(reinterpret_cast<const T *>(ctx + plan[l - 1].h_off), p.d_in, b.col, nullptr, b,
                                                cat, p.d_in, p.rows, X->dtype, st);
        if (!agg_ok) {
            set_last_error("sage_forward: no aggregation kernel for this row width");
            return E2EGREC_ERR_UNSUPPORTED;
        }
        const float *bl = bias ? bias[l] : nullptr;
        const int relu = act ? act[l] : 1;
        bool done = false;
        if (l == 0) tap_begin(TAP_UPDATE_FWD_OUTER, st);
        if (X->dtype == E2EGREC_BF16) {
            // the last layer's product stores its rows into H_out as well as into the context
            const bool top = l == n_layers - 1;
            done = tc_update_forward(reinterpret_cast<const __nv_bfloat16 *>(cat), p.rows, 2 * p.d_in,
                                     static_cast<const __nv_bfloat16 *>(W[l].data), p.d_out, bl, relu,
                                     reinterpret_cast<__nv_bfloat16 *>(hn), &b.counts[CNT_DST], &b.counts[CNT_STATUS], st,
                                     top ? static_cast<__nv_bfloat16 *>(H_out->data) : nullptr, H_out->ld, out_rows);
            top_stored = done && top;
        }
        if (!done) {
            EpiUpdate<T> epi{hn, p.d_out, bl, relu};
            dim3 grid((unsigned)std::max<int64_t>(1, ceil_div(p.rows, kGemmBM)), (unsigned)ceil_div(p.d_out, kGemmBN), 1);
            note_launch();
            gemm_simt_kernel<T, false, false, EpiUpdate<T>><<<grid, kGemmThreads, 0, st>>>(
                cat, 2 * p.d_in, static_cast<const T *>(W[l].data), 2 * p.d_in, p.rows, p.d_out, 2 * p.d_in,
                &b.counts[CNT_DST], nullptr, epi);
        }
        if (l == 0) tap_end(TAP_UPDATE_FWD_OUTER, st);
    }
    const LayerPlan &top = plan[n_layers - 1];
    const int64_t rows = out_rows;
    if (rows > 0 && !top_stored)
        cudaMemcpy2DAsync(H_out->data, (size_t)H_out->ld * es, ctx + top.h_off, (size_t)top.d_out * es,
                      (size_t)top.d_out * es, (size_t)rows, cudaMemcpyDeviceToDevice, st);
    return check_launch("sage_forward");
}

// ------------------------------------------------------------------------------ backward
struct BackwardScratch {
    size_t dz_off[2], dcat_off, seg_off, seg_bytes, chain_off, chain_bytes, part_off, wt_off, bytes;
};

static BackwardScratch plan_backward(const e2egrec_block *blocks, int32_t n_layers, const LayerPlan *plan, size_t es, int n_rhs)
{
    BackwardScratch s{};
    size_t dz = 0, dcat = 0, part = 0, ht = 0, wt = 0, chain = 0;
    for (int l = 0; l < n_layers; ++l) {
        const LayerPlan &p = plan[l];
        dz = std::max(dz, (size_t)n_rhs * p.rows * p.d_out * es);
        dcat = std::max(dcat, (size_t)n_rhs * p.rows * 2 * p.d_in * es);
        part = std::max(part, (size_t)kDwSplits * p.d_out * 2 * p.d_in * sizeof(float));
        wt = std::max(wt, (size_t)p.d_out * 2 * p.d_in * es);
        ht = std::max(ht, seg_scratch_carve(blocks[p.block].cap_edges, block_run_len(blocks[p.block].cap_edges, p.d_in, es), p.d_in, es, nullptr, n_rhs).bytes);
        chain = std::max(chain, seg_chain_bytes(blocks[p.block].cap_edges, block_run_len(blocks[p.block].cap_edges, p.d_in, es), p.d_in, es, n_rhs));
    }
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += align_up(b, 256); return o; };
    s.dz_off[0] = take(dz);
    s.dz_off[1] = take(dz);
    s.dcat_off = take(dcat);
    s.seg_off = take(ht);
    s.seg_bytes = ht;
    s.chain_off = take(chain);
    s.chain_bytes = chain;
    s.part_off = take(part);
    s.wt_off = take(wt);
    s.bytes = off;
    return s;
}

template <typename T>
// n_rhs gradients (dH_out[r] -> dX_rows[r]) go through the layers together: their rows are stacked in blocks of p.rows rows
// in dZ and dCat, every kernel of a layer is launched once for all of them, and dW / dbias receive the sum over them.
static int32_t backward_impl(const e2egrec_block *blocks, int32_t n_layers, const e2egrec_mat *X, const e2egrec_mat *W,
                             const int32_t *act, const LayerPlan *plan, const char *ctx, const e2egrec_mat *dH_out, int n_rhs,
                             float *const *dW, float *const *dbias, const e2egrec_mat *dX_rows, char *scratch,
                             const BackwardScratch &bs, uint32_t flags, cudaStream_t st)
{
    const int accumulate = (flags & E2EGREC_ACCUMULATE_DW) ? 1 : 0;
    T *dz_buf[2] = {reinterpret_cast<T *>(scratch + bs.dz_off[0]), reinterpret_cast<T *>(scratch + bs.dz_off[1])};
    T *dcat = reinterpret_cast<T *>(scratch + bs.dcat_off);
    float *part = reinterpret_cast<float *>(scratch + bs.part_off);

    // counters of the transposed aggregation (one per window of a block's entry stream); every launch leaves them zero
    cudaMemsetAsync(scratch + bs.chain_off, 0, bs.chain_bytes, st);
    // gradient entering the top layer, masked by its activation
    {
        const LayerPlan &p = plan[n_layers - 1];
        const e2egrec_block &b = blocks[p.block];
        const int64_t total = p.rows * p.d_out;
        note_launch();
        launch_pdl(relu_mask_kernel<T>, dim3((unsigned)std::max<int64_t>(1, ceil_div(total, 256)), (unsigned)n_rhs), dim3(256), 0, st,
                   static_cast<const T *>(dH_out[0].data), dH_out[0].ld, reinterpret_cast<const T *>(ctx + p.h_off), (int64_t)p.d_out,
                   &b.counts[CNT_DST], p.rows, p.d_out, act ? act[n_layers - 1] : 1, dz_buf[(n_layers - 1) & 1],
                   static_cast<const T *>(dH_out[n_rhs - 1].data), dH_out[n_rhs - 1].ld);
    }
    SideStream *side = SideStream::get(st);
    cudaEvent_t dz_free[2] = {nullptr, nullptr};
    for (int l = n_layers - 1; l >= 0; --l) {
        const LayerPlan &p = plan[l];
        const e2egrec_block &b = blocks[p.block];
        const T *dz = dz_buf[l & 1];
        const T *cat = reinterpret_cast<const T *>(ctx + p.cat_off);
        const int32_t *n_dst = &b.counts[CNT_DST];
        const int two_d = 2 * p.d_in;
        // dW_l = dZ^T [h | agg]   (split over the rows, partial sums added in a fixed order).  Nothing later in
        // this call reads dW, so it runs on the helper stream beside the dCat product and the transposed
        // aggregation; `dz_free` holds the event after which the helper stream no longer reads a dZ buffer.
        cudaStream_t ws = st;
        const bool dw_beside = side && (size_t)p.rows * (n_rhs * p.d_out + two_d) * sizeof(T) < dw_serial_bytes();
        if (dw_beside) {
            side->fork(st);
            ws = side->stream;
        }
        if (l == 0) tap_begin(TAP_DW_OUTER, ws);
        bool dw_done = false;
        // Splits of the tensor-core product: as many as there are SMs for a small layer (its few k-blocks spread over the
        // whole machine), one wave of CTAs over all output tiles for a large one, where every further wave pays the set-up
        // of a CTA and another set of fp32 partials (2 * 10^9-entry workload, 256 x 512 weights: 0.191 ms with 148
        // splits in four waves, 0.153 ms with 37 in one).
        const int tc_splits = dw_beside ? kDwSplits : std::max(1, kDwSplits / tc_weight_grad_tiles(p.d_out, two_d));
        if (X->dtype == E2EGREC_BF16)
            dw_done = tc_weight_grad(reinterpret_cast<const __nv_bfloat16 *>(dz), p.rows, p.d_out,
                                     reinterpret_cast<const __nv_bfloat16 *>(cat), two_d, n_dst, part, tc_splits,
                                     &b.counts[CNT_STATUS], ws, n_rhs);
        const int64_t n_w = (int64_t)p.d_out * two_d;
        if (dw_done) {
            note_launch();
            launch_pdl(splitk_reduce_kernel, dim3((unsigned)ceil_div(n_w, 256)), dim3(256), 0, ws, part, n_w, tc_splits, accumulate,
                       dW[l], n_dst, n_rhs);
        } else {
            for (int r = 0; r < n_rhs; ++r) {             // fp32-FMA product: one right-hand side per pass, added up
                EpiPartial epi{part, two_d, n_w};
                dim3 grid((unsigned)ceil_div(p.d_out, kGemmBM), (unsigned)ceil_div(two_d, kGemmBN), kDwSplits);
                note_launch();
                gemm_simt_kernel<T, true, true, EpiPartial><<<grid, kGemmThreads, 0, ws>>>(
                    dz + (int64_t)r * p.rows * p.d_out, p.d_out, cat, two_d, p.d_out, two_d, p.rows, nullptr, n_dst, epi);
                note_launch();
                launch_pdl(splitk_reduce_kernel, dim3((unsigned)ceil_div(n_w, 256)), dim3(256), 0, ws, part, n_w, kDwSplits,
                           (accumulate || r > 0) ? 1 : 0, dW[l], (const int32_t *)nullptr, 1);
            }
        }
        if (l == 0) tap_end(TAP_DW_OUTER, ws);
        if (dbias && dbias[l]) {
            for (int r = 0; r < n_rhs; ++r) {
                note_launch();
                colsum_kernel<T><<<(unsigned)ceil_div(p.d_out, 32), 256, 0, ws>>>(dz + (int64_t)r * p.rows * p.d_out, p.d_out, n_dst,
                                                                                 p.d_out, (accumulate || r > 0) ? 1 : 0, dbias[l]);
            }
        }
        if (dw_beside) {
            dz_free[l & 1] = side->event();
            cudaEventRecord(dz_free[l & 1], side->stream);
        }
        // dCat = dZ W_l, the agg half scaled by 1/|S|
        if (l == 0) tap_begin(TAP_DCAT_OUTER, st);
        bool dcat_done = false;
        if (X->dtype == E2EGREC_BF16) {
            if (W[l].ld == two_d)               // W as stored: the product reads it with its N index contiguous
                dcat_done = tc_dcat_backward(reinterpret_cast<const __nv_bfloat16 *>(dz), p.rows, p.d_out,
                                             static_cast<const __nv_bfloat16 *>(W[l].data), two_d, b.inv_cnt,
                                             reinterpret_cast<__nv_bfloat16 *>(dcat), n_dst, &b.counts[CNT_STATUS], st, n_rhs);
        }
        if (!dcat_done) {
            for (int r = 0; r < n_rhs; ++r) {
                EpiDCat<T> epi{dcat + (int64_t)r * p.rows * two_d, two_d, p.d_in, b.inv_cnt};
                dim3 grid((unsigned)std::max<int64_t>(1, ceil_div(p.rows, kGemmBM)), (unsigned)ceil_div(two_d, kGemmBN), 1);
                note_launch();
                gemm_simt_kernel<T, false, true, EpiDCat<T>><<<grid, kGemmThreads, 0, st>>>(
                    dz + (int64_t)r * p.rows * p.d_out, p.d_out, static_cast<const T *>(W[l].data), two_d, p.rows, two_d, p.d_out,
                    n_dst, nullptr, epi);
            }
        }
        if (l == 0) tap_end(TAP_DCAT_OUTER, st);
        // transposed aggregation: gather over the block's CSC, plus the self rows, masked by the
        // activation of the layer below
        SegOut<T> o{};
        o.self = dcat;
        o.ld_self = two_d;
        o.n_self = n_dst;
        o.mean = 0;
        o.n_rhs = n_rhs;
        o.rhs_in = o.rhs_self = (int64_t)p.rows * two_d;
        o.in_rows = (int64_t)p.rows * n_rhs;
        o.status = &b.counts[CNT_STATUS];
        if (l > 0) {
            // the buffer that receives dZ of the layer below may still be read by the helper stream (layer l+1)
            if (side && dz_free[(l - 1) & 1]) {
                cudaStreamWaitEvent(st, dz_free[(l - 1) & 1], 0);
                dz_free[(l - 1) & 1] = nullptr;
            }
            o.out = dz_buf[(l - 1) & 1];
            o.ld_out = p.d_in;
            o.pad_rows = plan[l - 1].rows;
            o.rhs_out = plan[l - 1].rows * p.d_in;
            const int relu_below = act ? act[l - 1] : 1;
            o.mask = relu_below ? reinterpret_cast<const T *>(ctx + plan[l - 1].h_off) : nullptr;
            o.ld_mask = p.d_in;
        } else {
            o.out = static_cast<T *>(dX_rows[0].data);
            o.ld_out = dX_rows[0].ld;
            o.mask = nullptr;
            o.rhs_out = static_cast<T *>(dX_rows[n_rhs - 1].data) - static_cast<T *>(dX_rows[0].data);
        }
        if (l == 0) tap_begin(TAP_AGG_BWD_OUTER, st);
        SegScratch sc = seg_scratch_carve(b.cap_edges, block_run_len(b.cap_edges, p.d_in, dtype_size(X->dtype)), p.d_in, dtype_size(X->dtype), scratch + bs.seg_off, n_rhs);
        sc.chain_cnt = reinterpret_cast<int32_t *>(scratch + bs.chain_off);
        const bool seg_ok = dispatch_seg_reduce<T, int32_t, false>(dcat + p.d_in, two_d, b.csc_ptr, b.csc_row, &b.counts[CNT_SRC], 0,
                                                                   b.cap_src, nullptr, block_run_len(b.cap_edges, p.d_in, dtype_size(X->dtype)), p.d_in, X->dtype,
                                                                   b.csc_col, sc, o, st);
        if (l == 0) tap_end(TAP_AGG_BWD_OUTER, st);
        if (!seg_ok) {
            if (side) side->join(st);
            set_last_error("sage_backward: no aggregation kernel for this row width");
            return E2EGREC_ERR_UNSUPPORTED;
        }
    }
    if (side) side->join(st);
    return check_launch("sage_backward");
}

}  // namespace e2egrec

using namespace e2egrec;

extern "C" int32_t e2egrec_sage_forward(const e2egrec_block *blocks, int32_t n_layers, const e2egrec_mat *X,
                                        const e2egrec_mat *W, const float *const *bias, const int32_t *act,
                                        void *ctx, size_t *ctx_bytes, const e2egrec_mat *H_out, void *stream)
{
    if (!ctx_bytes) return E2EGREC_ERR_NULL;
    LayerPlan plan[kMaxHops];
    size_t need = 0;
    int32_t rc = plan_layers(blocks, n_layers, X, W, plan, &need);
    if (rc != E2EGREC_OK) return rc;
    if (!ctx) { *ctx_bytes = need; return E2EGREC_OK; }
    if (*ctx_bytes < need) { *ctx_bytes = need; return E2EGREC_ERR_WORKSPACE; }
    if (reinterpret_cast<uintptr_t>(ctx) % 256) return E2EGREC_ERR_ALIGN;
    if (!H_out || !H_out->data) return E2EGREC_ERR_NULL;
    if (H_out->dtype != X->dtype) return E2EGREC_ERR_DTYPE;
    if (H_out->dim != plan[n_layers - 1].d_out || H_out->ld < H_out->dim) return E2EGREC_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (X->dtype == E2EGREC_BF16)
        return forward_impl<__nv_bfloat16>(blocks, n_layers, X, W, bias, act, plan, static_cast<char *>(ctx), H_out, st);
    return forward_impl<float>(blocks, n_layers, X, W, bias, act, plan, static_cast<char *>(ctx), H_out, st);
}

extern "C" int32_t e2egrec_sage_ctx_layout(const e2egrec_block *blocks, int32_t n_layers, const e2egrec_mat *X,
                                           const e2egrec_mat *W, size_t *cat_offset, size_t *h_offset, int64_t *rows)
{
    if (!cat_offset || !h_offset || !rows) return E2EGREC_ERR_NULL;
    LayerPlan plan[kMaxHops];
    size_t need = 0;
    int32_t rc = plan_layers(blocks, n_layers, X, W, plan, &need);
    if (rc != E2EGREC_OK) return rc;
    for (int l = 0; l < n_layers; ++l) {
        cat_offset[l] = plan[l].cat_off;
        h_offset[l] = plan[l].h_off;
        rows[l] = plan[l].rows;
    }
    return E2EGREC_OK;
}

static int32_t sage_backward_entry(const e2egrec_block *blocks, int32_t n_layers, const e2egrec_mat *X, const e2egrec_mat *W,
                                   const int32_t *act, const void *ctx, const e2egrec_mat *dH_out, int32_t n_rhs,
                                   float *const *dW, float *const *dbias, const e2egrec_mat *dX_rows, void *scratch,
                                   size_t *scratch_bytes, uint32_t flags, void *stream)
{
    if (!scratch_bytes) return E2EGREC_ERR_NULL;
    if (n_rhs < 1 || n_rhs > 2) return E2EGREC_ERR_ARG;
    LayerPlan plan[kMaxHops];
    size_t ctx_need = 0;
    int32_t rc = plan_layers(blocks, n_layers, X, W, plan, &ctx_need);
    if (rc != E2EGREC_OK) return rc;
    const BackwardScratch bs = plan_backward(blocks, n_layers, plan, dtype_size(X->dtype), n_rhs);
    if (!scratch) { *scratch_bytes = bs.bytes; return E2EGREC_OK; }
    if (*scratch_bytes < bs.bytes) { *scratch_bytes = bs.bytes; return E2EGREC_ERR_WORKSPACE; }
    if (reinterpret_cast<uintptr_t>(scratch) % 256 || reinterpret_cast<uintptr_t>(ctx) % 256) return E2EGREC_ERR_ALIGN;
    if (!ctx || !dH_out || !dW || !dX_rows) return E2EGREC_ERR_NULL;
    for (int l = 0; l < n_layers; ++l)
        if (!dW[l]) return E2EGREC_ERR_NULL;
    const size_t es = dtype_size(X->dtype);
    for (int r = 0; r < n_rhs; ++r) {
        if (!dH_out[r].data || !dX_rows[r].data) return E2EGREC_ERR_NULL;
        if (dH_out[r].dtype != X->dtype || dX_rows[r].dtype != X->dtype) return E2EGREC_ERR_DTYPE;
        if (dH_out[r].dim != plan[n_layers - 1].d_out || dX_rows[r].dim != X->dim) return E2EGREC_ERR_ARG;
        if (dX_rows[r].rows < blocks[n_layers - 1].cap_src || dH_out[r].rows < blocks[0].cap_dst) return E2EGREC_ERR_ARG;
        if ((dX_rows[r].ld * es) % 16 || reinterpret_cast<uintptr_t>(dX_rows[r].data) % 16) return E2EGREC_ERR_ALIGN;
        if (dX_rows[r].ld != dX_rows[0].ld) return E2EGREC_ERR_ARG;       // the results share one leading dimension
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (SideStream *side = SideStream::get(st)) side->join_pending(st);     // a deferred block transposition
    if (X->dtype == E2EGREC_BF16)
        return backward_impl<__nv_bfloat16>(blocks, n_layers, X, W, act, plan, static_cast<const char *>(ctx), dH_out, n_rhs, dW,
                                            dbias, dX_rows, static_cast<char *>(scratch), bs, flags, st);
    return backward_impl<float>(blocks, n_layers, X, W, act, plan, static_cast<const char *>(ctx), dH_out, n_rhs, dW, dbias,
                                dX_rows, static_cast<char *>(scratch), bs, flags, st);
}

extern "C" int32_t e2egrec_sage_backward(const e2egrec_block *blocks, int32_t n_layers, const e2egrec_mat *X,
                                         const e2egrec_mat *W, const int32_t *act, const void *ctx,
                                         const e2egrec_mat *dH_out, float *const *dW, float *const *dbias,
                                         const e2egrec_mat *dX_rows, void *scratch, size_t *scratch_bytes,
                                         uint32_t flags, void *stream)
{
    return sage_backward_entry(blocks, n_layers, X, W, act, ctx, dH_out, 1, dW, dbias, dX_rows, scratch, scratch_bytes, flags, stream);
}

extern "C" int32_t e2egrec_sage_backward_multi(const e2egrec_block *blocks, int32_t n_layers, const e2egrec_mat *X,
                                               const e2egrec_mat *W, const int32_t *act, const void *ctx,
                                               const e2egrec_mat *dH_out, int32_t n_rhs, float *const *dW, float *const *dbias,
                                               const e2egrec_mat *dX_rows, void *scratch, size_t *scratch_bytes,
                                               uint32_t flags, void *stream)
{
    return sage_backward_entry(blocks, n_layers, X, W, act, ctx, dH_out, n_rhs, dW, dbias, dX_rows, scratch, scratch_bytes, flags,
                               stream);
}
