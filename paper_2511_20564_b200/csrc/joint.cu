// Joint training step: sampled GraphSAGE encoder + MLP ranking tower + BCE loss, forward and backward
// in one call (Theorem 1: z_i = [h_theta || b_i] feeds the scorer, so the ranking loss reaches the GNN
// weights and the node features; Sec. 4.2: the chain loss -> tower -> embeddings -> GNN).
#include <algorithm>

#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "internal.cuh"
#include "segreduce.cuh"

namespace e2egrec {
namespace {

inline int64_t pad128(int64_t r) { return (r + 127) / 128 * 128; }
constexpr int kSplits = 148;
constexpr int kPairRun = 32;

struct JointPlan {
    int n_hops, d0, dL, dense_dim, zdim, h1, h2, unit;        // unit = elements per 16 bytes
    size_t es;
    int32_t P, P2;
    int64_t rowsP;
    int32_t cd[kMaxHops], cs[kMaxHops], ce[kMaxHops];
    size_t sampler_bytes, ctx_bytes, bwd_bytes, seg_bytes;
    size_t blk_off[kMaxHops][10];
    size_t ctx_off, bwd_off, seg_off;
    size_t seeds_off, pair_local_off, entry_unit_off, pcounts_off, pcsc_ptr_off, pcsc_idx_off, pcsc_eid_off, pcsc_col_off,
        pmeta_off;
    size_t hseed_off, dhseed_off, z_off, a1_off, a2_off, dt_off, dz2_off, dz1_off, dz_off, wt_off, part_off;
    size_t zf_off, gate_off, dzf_off, gpre_off;               // gated step only: fused input, gate, its gradient, scratch
    int gated;
    size_t bytes;
};

void fill_blocks(const JointPlan &jp, char *ws, e2egrec_block *blocks)
{
    for (int h = 0; h < jp.n_hops; ++h) {
        e2egrec_block &b = blocks[h];
        b.cap_dst = jp.cd[h];
        b.cap_src = jp.cs[h];
        b.cap_edges = jp.ce[h];
        int32_t **slots[9] = {&b.counts, &b.indptr, &b.col, &b.nbr_global, &b.src_nodes, &b.csc_ptr, &b.csc_row, &b.csc_eid,
                              &b.csc_col};
        for (int k = 0; k < 9; ++k) *slots[k] = reinterpret_cast<int32_t *>(ws + jp.blk_off[h][k]);
        b.inv_cnt = reinterpret_cast<float *>(ws + jp.blk_off[h][9]);
    }
}

// ------------------------------------------------------------------------------------------ kernels
__global__ void joint_meta_kernel(int32_t *pmeta, int32_t n_pairs) { pmeta[0] = n_pairs; }

// z[p] = [ h[user seed] | h[item seed] | dense[p] ] in the feature dtype; rows P .. rows_alloc-1 are zero.
template <typename T>
__global__ void build_z_kernel(const T *__restrict__ H, int dL, const int32_t *__restrict__ pair_local,
                               const float *__restrict__ dense, int dense_dim, int32_t P, int64_t rows_alloc,
                               T *__restrict__ z)
{
    const int zdim = 2 * dL + dense_dim;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t p = t / zdim;
    const int k = (int)(t - p * zdim);
    if (p >= rows_alloc) return;
    T v = from_float<T>(0.f);
    if (p < P) {
        if (k < dL) v = H[(int64_t)pair_local[p] * dL + k];
        else if (k < 2 * dL) v = H[(int64_t)pair_local[P + p] * dL + (k - dL)];
        else v = from_float<T>(dense[p * (int64_t)dense_dim + (k - 2 * dL)]);
    }
    z[t] = v;
}

// logits t[p] = b + <a[p], w>, fp32, one warp per pair
template <typename T>
__global__ void __launch_bounds__(256)
logit_kernel(const T *__restrict__ a, int d, const T *__restrict__ w, const float *__restrict__ b, int32_t P,
             float *__restrict__ logits)
{
    const int lane = threadIdx.x & 31;
    const int64_t p = ((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5;
    if (p >= P) return;
    float s = 0.f;
    for (int k = lane; k < d; k += 32) s = fmaf(to_float<T>(a[p * d + k]), to_float<T>(w[k]), s);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) logits[p] = s + (b ? b[0] : 0.f);
}

// loss = mean_p [ max(t,0) - y t + log(1 + exp(-|t|)) ],  dt = (sigmoid(t) - y) / P,  db3 = sum dt.
// One block; sums run in a fixed order.
__global__ void __launch_bounds__(1024)
bce_kernel(const float *__restrict__ logits, const float *__restrict__ labels, int32_t P, float *__restrict__ loss,
           float *__restrict__ dt, float *__restrict__ db3, int accumulate)
{
    __shared__ float red[2][1024];
    float ls = 0.f, ds = 0.f;
    const float invP = 1.0f / (float)P;
    for (int p = threadIdx.x; p < P; p += 1024) {
        const float t = logits[p], y = labels[p];
        ls += fmaxf(t, 0.f) - y * t + log1pf(expf(-fabsf(t)));
        const float sg = t >= 0.f ? 1.0f / (1.0f + expf(-t)) : expf(t) / (1.0f + expf(t));
        const float g = (sg - y) * invP;
        dt[p] = g;
        ds += g;
    }
    red[0][threadIdx.x] = ls;
    red[1][threadIdx.x] = ds;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if (threadIdx.x < o) {
            red[0][threadIdx.x] += red[0][threadIdx.x + o];
            red[1][threadIdx.x] += red[1][threadIdx.x + o];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        loss[0] = red[0][0] * invP;
        if (db3) db3[0] = (accumulate ? db3[0] : 0.f) + red[1][0];
    }
}

// dW3[j] = sum_p dt[p] a2[p, j]   (one block per 32 columns, rows in a fixed order)
template <typename T>
__global__ void __launch_bounds__(256)
weighted_colsum_kernel(const T *__restrict__ a, int d, const float *__restrict__ wgt, int32_t P, int accumulate,
                       float *__restrict__ out)
{
    __shared__ float red[8][32];
    const int col = blockIdx.x * 32 + (threadIdx.x & 31);
    const int rl = threadIdx.x >> 5;
    float s = 0.f;
    if (col < d)
        for (int64_t r = rl; r < P; r += 8) s = fmaf(wgt[r], to_float<T>(a[r * d + col]), s);
    red[rl][threadIdx.x & 31] = s;
    __syncthreads();
    if (rl == 0 && col < d) {
        float t = accumulate ? out[col] : 0.f;
        for (int w = 0; w < 8; ++w) t += red[w][threadIdx.x & 31];
        out[col] = t;
    }
}

// dZ2[p, j] = dt[p] * W3[j] where a2[p, j] > 0 (everywhere with the identity activation), stored in the feature dtype;
// padding rows are zero.
template <typename T>
__global__ void dz_top_kernel(const float *__restrict__ dt, const T *__restrict__ w3, const T *__restrict__ a2, int d,
                              int32_t P, int64_t rows_alloc, int relu, T *__restrict__ dz2)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t p = t / d;
    const int j = (int)(t - p * d);
    if (p >= rows_alloc) return;
    float v = 0.f;
    if (p < P && (!relu || to_float<T>(a2[t]) > 0.f)) v = dt[p] * to_float<T>(w3[j]);
    dz2[t] = from_float<T>(v);
}

// ------------------------------------------------------------------------------------------ dense helpers
template <typename T> bool use_tc() { return false; }
template <> bool use_tc<__nv_bfloat16>() { return true; }

// out = mask * act(A W^T + b), A [rows x k], W [n x k]
template <typename T>
void linear_forward(const T *A, int64_t rows, int k, const T *W, int n, const float *bias, int relu, T *out,
                    const int32_t *m_dev, int32_t *status, cudaStream_t st)
{
    if (use_tc<T>() &&
        tc_linear(reinterpret_cast<const __nv_bfloat16 *>(A), rows, k, reinterpret_cast<const __nv_bfloat16 *>(W), n, bias,
                  relu, nullptr, 0, reinterpret_cast<__nv_bfloat16 *>(out), n, m_dev, status, st))
        return;
    EpiUpdate<T> epi{out, n, bias, relu};
    dim3 grid((unsigned)ceil_div(rows, kGemmBM), (unsigned)ceil_div(n, kGemmBN), 1);
    note_launch();
    gemm_simt_kernel<T, false, false, EpiUpdate<T>><<<grid, kGemmThreads, 0, st>>>(A, k, W, k, rows, n, k, m_dev, nullptr, epi);
}

// dX = mask * (dY W), dY [rows x n_out], W [n_out x n_in] -> dX [rows x n_in]; wt is scratch for W^T
template <typename T>
void linear_backward_input(const T *dY, int64_t rows, int n_out, const T *W, int n_in, const T *mask, T *dX, T *wt,
                           const int32_t *m_dev, int32_t *status, cudaStream_t st)
{
    if (use_tc<T>()) {
        // W [n_out x n_in] as stored is the [k x n] operand of dY W
        if (tc_linear(reinterpret_cast<const __nv_bfloat16 *>(dY), rows, n_out, reinterpret_cast<const __nv_bfloat16 *>(W),
                      n_in, nullptr, 0, reinterpret_cast<const __nv_bfloat16 *>(mask), n_in,
                      reinterpret_cast<__nv_bfloat16 *>(dX), n_in, m_dev, status, st, true))
            return;
        // shapes the tensor-core kernel does not take in that form: through a transposed copy
        note_launch();
        transpose_kernel<T><<<dim3((unsigned)ceil_div(n_in, 32), (unsigned)ceil_div(n_out, 32)), dim3(32, 8), 0, st>>>(
            W, n_out, n_in, wt);
        if (tc_linear(reinterpret_cast<const __nv_bfloat16 *>(dY), rows, n_out, reinterpret_cast<const __nv_bfloat16 *>(wt),
                      n_in, nullptr, 0, reinterpret_cast<const __nv_bfloat16 *>(mask), n_in,
                      reinterpret_cast<__nv_bfloat16 *>(dX), n_in, m_dev, status, st))
            return;
    }
    EpiMasked<T> epi{dX, n_in, mask, n_in};
    dim3 grid((unsigned)ceil_div(rows, kGemmBM), (unsigned)ceil_div(n_in, kGemmBN), 1);
    note_launch();
    gemm_simt_kernel<T, false, true, EpiMasked<T>><<<grid, kGemmThreads, 0, st>>>(dY, n_out, W, n_in, rows, n_in, n_out, m_dev,
                                                                                 nullptr, epi);
}

// dW = dY^T X (fp32, rows split kSplits ways and added in order), db = column sums of dY
template <typename T>
void linear_backward_weight(const T *dY, int64_t rows, int n_out, const T *Xin, int n_in, const int32_t *m_dev,
                            float *part, float *dW, float *db, int32_t *status, cudaStream_t st)
{
    const bool on_tc = use_tc<T>() && tc_weight_grad(reinterpret_cast<const __nv_bfloat16 *>(dY), rows, n_out,
                                                     reinterpret_cast<const __nv_bfloat16 *>(Xin), n_in, m_dev, part, kSplits,
                                                     status, st);
    if (!on_tc) {
        EpiPartial epi{part, n_in, (int64_t)n_out * n_in};
        dim3 grid((unsigned)ceil_div(n_out, kGemmBM), (unsigned)ceil_div(n_in, kGemmBN), kSplits);
        note_launch();
        gemm_simt_kernel<T, true, true, EpiPartial><<<grid, kGemmThreads, 0, st>>>(dY, n_out, Xin, n_in, n_out, n_in, rows,
                                                                                  nullptr, m_dev, epi);
    }
    const int64_t n = (int64_t)n_out * n_in;
    note_launch();
    splitk_reduce_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, st>>>(part, n, kSplits, 0, dW, on_tc ? m_dev : nullptr);
    if (db) {
        note_launch();
        colsum_kernel<T><<<(unsigned)ceil_div(n_out, 32), 256, 0, st>>>(dY, n_out, m_dev, n_out, 0, db);
    }
}

// ------------------------------------------------------------------------------------------ gated fusion (Sec. 4.3.2)
//   g = sigmoid(F Wg^T + bg),  F_fused = g * F.  bf16 shapes the tensor-core kernel takes: one launch, sigmoid and the
//   product with F in the epilogue of the F Wg^T product; otherwise the product runs on the fp32-FMA kernel and the gate
//   is applied element-wise.  Backward: d pre = dFused * F * g (1 - g) element-wise, dWg = d pre^T F, and
//   dF = d pre Wg + dFused * g with the second term added in the product's epilogue on the tensor-core path.
__global__ void gate_meta_kernel(int32_t *meta, int32_t n_rows) { meta[0] = n_rows; }

// gate = sigmoid(pre), fused = gate * F for rows < n_rows; zero rows up to rows_alloc
template <typename T>
__global__ void gate_apply_kernel(const T *__restrict__ pre, const T *__restrict__ F, int64_t ldf, int d, int32_t n_rows,
                                  int64_t rows_alloc, T *__restrict__ gate, int64_t ldg, T *__restrict__ fused, int64_t ldo)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = t / d;
    const int k = (int)(t - i * d);
    if (i >= rows_alloc) return;
    float g = 0.f, o = 0.f;
    if (i < n_rows) {
        const float p = to_float<T>(pre[i * d + k]);
        const float e = expf(-fabsf(p));
        g = to_float<T>(from_float<T>(p >= 0.f ? 1.0f / (1.0f + e) : e / (1.0f + e)));      // the stored gate
        o = g * to_float<T>(F[i * ldf + k]);
    }
    gate[i * ldg + k] = from_float<T>(g);
    fused[i * ldo + k] = from_float<T>(o);
}

// dpre = dFused * F * g (1 - g) for rows < n_rows, zero rows up to rows_alloc
template <typename T>
__global__ void gate_dpre_kernel(const T *__restrict__ dFused, int64_t ldd, const T *__restrict__ F, int64_t ldf,
                                 const T *__restrict__ gate, int64_t ldg, int d, int32_t n_rows, int64_t rows_alloc,
                                 T *__restrict__ dpre)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = t / d;
    const int k = (int)(t - i * d);
    if (i >= rows_alloc) return;
    float v = 0.f;
    if (i < n_rows) {
        const float g = to_float<T>(gate[i * ldg + k]);
        v = to_float<T>(dFused[i * ldd + k]) * to_float<T>(F[i * ldf + k]) * g * (1.0f - g);
    }
    dpre[i * d + k] = from_float<T>(v);
}

// dF = t + dFused * g for rows < n_rows
template <typename T>
__global__ void gate_dF_kernel(const T *__restrict__ tprod, const T *__restrict__ dFused, int64_t ldd,
                               const T *__restrict__ gate, int64_t ldg, int d, int32_t n_rows, T *__restrict__ dF, int64_t ldo)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = t / d;
    const int k = (int)(t - i * d);
    if (i >= n_rows) return;
    dF[i * ldo + k] = from_float<T>(to_float<T>(tprod[i * d + k]) + to_float<T>(dFused[i * ldd + k]) * to_float<T>(gate[i * ldg + k]));
}

unsigned cells_grid(int64_t rows, int d) { return (unsigned)std::max<int64_t>(1, ceil_div(rows * d, 256)); }

// Matrix as the gate cores see it: data, leading dimension, rows allocated.
template <typename T> struct GMat { T *p; int64_t ld, rows; };

// F [rows x d] (rows a multiple of 128, all allocated); meta = {n_rows}; pre: scratch [rows x d] (only used off the
// tensor cores).  gate / fused receive n_rows rows (and zero rows up to the next multiple of 128 when they have room).
template <typename T>
void gate_forward_core(GMat<const T> F, int64_t rows, int32_t n_rows, int d, const T *Wg, const float *bg, T *pre,
                       GMat<T> gate, GMat<T> fused, const int32_t *meta, int32_t *status, cudaStream_t st)
{
    if (use_tc<T>() && F.ld == d && gate.rows >= rows && fused.rows >= rows) {
        TcFuse fz{};
        fz.gate_in = reinterpret_cast<const __nv_bfloat16 *>(F.p);
        fz.ld_gate_in = F.ld;
        fz.gate_out = reinterpret_cast<__nv_bfloat16 *>(gate.p);
        fz.ld_gate_out = gate.ld;
        if (tc_linear(reinterpret_cast<const __nv_bfloat16 *>(F.p), rows, d, reinterpret_cast<const __nv_bfloat16 *>(Wg), d, bg, 0,
                      nullptr, 0, reinterpret_cast<__nv_bfloat16 *>(fused.p), fused.ld, meta, status, st, false, &fz))
            return;
    }
    if (F.ld == d) {
        linear_forward<T>(F.p, rows, d, Wg, d, bg, 0, pre, meta, status, st);
    } else {
        EpiUpdate<T> epi{pre, d, bg, 0};
        dim3 grid((unsigned)ceil_div(rows, kGemmBM), (unsigned)ceil_div(d, kGemmBN), 1);
        note_launch();
        gemm_simt_kernel<T, false, false, EpiUpdate<T>><<<grid, kGemmThreads, 0, st>>>(F.p, F.ld, Wg, d, rows, d, d, meta, nullptr, epi);
    }
    note_launch();
    gate_apply_kernel<T><<<cells_grid(rows, d), 256, 0, st>>>(pre, F.p, F.ld, d, n_rows,
                                                             std::min<int64_t>(rows, std::min(gate.rows, fused.rows)), gate.p, gate.ld,
                                                             fused.p, fused.ld);
}

// dpre, tprod: scratch [rows x d]; wt: scratch [d x d]; part: scratch [kSplits x d x d] fp32.
template <typename T>
void gate_backward_core(GMat<const T> dFused, GMat<const T> F, GMat<const T> gate, int64_t rows, int32_t n_rows, int d, const T *Wg,
                        T *dpre, T *tprod, T *wt, float *part, GMat<T> dF, float *dWg, float *dbg, const int32_t *meta,
                        int32_t *status, cudaStream_t st)
{
    note_launch();
    gate_dpre_kernel<T><<<cells_grid(rows, d), 256, 0, st>>>(dFused.p, dFused.ld, F.p, F.ld, gate.p, gate.ld, d, n_rows, rows, dpre);
    if (F.ld == d) {
        linear_backward_weight<T>(dpre, rows, d, F.p, d, meta, part, dWg, dbg, status, st);
    } else {                                                             // strided F: fp32-FMA product
        EpiPartial epi{part, d, (int64_t)d * d};
        dim3 grid((unsigned)ceil_div(d, kGemmBM), (unsigned)ceil_div(d, kGemmBN), kSplits);
        note_launch();
        gemm_simt_kernel<T, true, true, EpiPartial><<<grid, kGemmThreads, 0, st>>>(dpre, d, F.p, F.ld, d, d, rows, nullptr, meta, epi);
        note_launch();
        splitk_reduce_kernel<<<(unsigned)ceil_div((int64_t)d * d, 256), 256, 0, st>>>(part, (int64_t)d * d, kSplits, 0, dWg, nullptr);
        if (dbg) {
            note_launch();
            colsum_kernel<T><<<(unsigned)ceil_div(d, 32), 256, 0, st>>>(dpre, d, meta, d, 0, dbg);
        }
    }
    if (use_tc<T>() && dF.rows >= rows && dFused.rows >= rows && gate.rows >= rows) {
        TcFuse fz{};
        fz.add_a = reinterpret_cast<const __nv_bfloat16 *>(dFused.p);
        fz.ld_add_a = dFused.ld;
        fz.add_b = reinterpret_cast<const __nv_bfloat16 *>(gate.p);
        fz.ld_add_b = gate.ld;
        if (tc_linear(reinterpret_cast<const __nv_bfloat16 *>(dpre), rows, d, reinterpret_cast<const __nv_bfloat16 *>(Wg), d, nullptr, 0,
                      nullptr, 0, reinterpret_cast<__nv_bfloat16 *>(dF.p), dF.ld, meta, status, st, true, &fz))
            return;
    }
    linear_backward_input<T>(dpre, rows, d, Wg, d, nullptr, tprod, wt, meta, status, st);
    note_launch();
    gate_dF_kernel<T><<<cells_grid(n_rows > 0 ? n_rows : 1, d), 256, 0, st>>>(tprod, dFused.p, dFused.ld, gate.p, gate.ld, d, n_rows,
                                                                            dF.p, dF.ld);
}

// ------------------------------------------------------------------------------------------ plan
int32_t make_plan(const e2egrec_csr *graph, const e2egrec_mat *X, int32_t n_pairs, int32_t dense_dim, int32_t n_hops,
                  const int32_t *fanouts, const e2egrec_mat *W_gnn, const e2egrec_mat *W_tower, uint32_t flags, JointPlan &jp)
{
    if (!graph || !X || !fanouts || !W_gnn || !W_tower) return E2EGREC_ERR_NULL;
    if (n_pairs < 1 || n_pairs > (1 << 28) || dense_dim < 0) return E2EGREC_ERR_ARG;
    if (X->dtype != E2EGREC_F32 && X->dtype != E2EGREC_BF16) return E2EGREC_ERR_DTYPE;
    jp.n_hops = n_hops;
    jp.es = dtype_size(X->dtype);
    jp.unit = (int)(16 / jp.es);
    jp.P = n_pairs;
    jp.P2 = 2 * n_pairs;
    jp.rowsP = pad128(n_pairs);
    int32_t rc = khop_caps(graph->n_nodes, jp.P2, n_hops, fanouts, jp.cd, jp.cs, jp.ce);
    if (rc != E2EGREC_OK) return rc;
    jp.d0 = X->dim;
    for (int l = 0; l < n_hops; ++l)
        if (!W_gnn[l].data || W_gnn[l].dtype != X->dtype) return W_gnn[l].data ? E2EGREC_ERR_DTYPE : E2EGREC_ERR_NULL;
    jp.dL = (int)W_gnn[n_hops - 1].rows;
    jp.dense_dim = dense_dim;
    jp.zdim = 2 * jp.dL + dense_dim;
    for (int k = 0; k < 3; ++k)
        if (!W_tower[k].data || W_tower[k].dtype != X->dtype) return W_tower[k].data ? E2EGREC_ERR_DTYPE : E2EGREC_ERR_NULL;
    jp.h1 = (int)W_tower[0].rows;
    jp.h2 = (int)W_tower[1].rows;
    if (W_tower[0].dim != jp.zdim || W_tower[1].dim != jp.h1 || W_tower[2].dim != jp.h2 || W_tower[2].rows != 1)
        return E2EGREC_ERR_ARG;
    for (int k = 0; k < 3; ++k)
        if (W_tower[k].ld != W_tower[k].dim) return E2EGREC_ERR_ARG;
    jp.gated = (flags & E2EGREC_JOINT_GATE) ? 1 : 0;
    if (jp.gated) {
        const e2egrec_mat &wg = W_tower[3];
        if (!wg.data) return E2EGREC_ERR_NULL;
        if (wg.dtype != X->dtype) return E2EGREC_ERR_DTYPE;
        if (wg.rows != jp.zdim || wg.dim != jp.zdim || wg.ld != jp.zdim) return E2EGREC_ERR_ARG;
    }
    if (jp.zdim % jp.unit || jp.dL % jp.unit || jp.h1 % jp.unit || jp.h2 % jp.unit) return E2EGREC_ERR_ALIGN;

    int64_t md = 0, ms = 0, me = 0;
    for (int h = 0; h < n_hops; ++h) {
        md = std::max<int64_t>(md, jp.cd[h]);
        ms = std::max<int64_t>(ms, jp.cs[h]);
        me = std::max<int64_t>(me, jp.ce[h]);
    }
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += align_up(b, 256); return o; };
    jp.sampler_bytes = sampler_scratch_bytes(graph->n_nodes, md, ms, me);
    take(jp.sampler_bytes);                                    // the sampler scratch is the head of the workspace
    for (int h = 0; h < n_hops; ++h) {
        const size_t d = jp.cd[h], s = jp.cs[h], e = std::max(jp.ce[h], 1);
        const size_t n[10] = {4, d + 1, e, e, std::max<size_t>(s, 1), s + 1, e, e, e, std::max<size_t>(d, 1)};
        for (int k = 0; k < 10; ++k) jp.blk_off[h][k] = take(n[k] * 4);
    }
    // sizes of the encoder's own buffers come from its size queries
    e2egrec_block blocks[kMaxHops];
    fill_blocks(jp, nullptr, blocks);
    size_t need = 0;
    rc = e2egrec_sage_forward(blocks, n_hops, X, W_gnn, nullptr, nullptr, nullptr, &need, nullptr, nullptr);
    if (rc != E2EGREC_OK) return rc;
    jp.ctx_bytes = need;
    jp.ctx_off = take(need);
    rc = e2egrec_sage_backward(blocks, n_hops, X, W_gnn, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, &need, 0,
                               nullptr);
    if (rc != E2EGREC_OK) return rc;
    jp.bwd_bytes = need;
    jp.bwd_off = take(need);
    jp.seg_bytes = seg_scratch_carve(jp.P2, kPairRun, jp.dL, dtype_size(X->dtype), nullptr).bytes;
    jp.seg_off = take(jp.seg_bytes);
    const size_t p2 = (size_t)jp.P2;
    jp.seeds_off = take(p2 * 4);
    jp.pair_local_off = take(p2 * 4);
    jp.entry_unit_off = take(p2 * 4);
    jp.pcounts_off = take(16);
    jp.pcsc_ptr_off = take((p2 + 1) * 4);
    jp.pcsc_idx_off = take(p2 * 4);
    jp.pcsc_eid_off = take(p2 * 4);
    jp.pcsc_col_off = take(p2 * 4);
    jp.pmeta_off = take(16);
    const size_t rs = (size_t)pad128(jp.cd[0]);
    jp.hseed_off = take(rs * jp.dL * jp.es);
    jp.dhseed_off = take(rs * jp.dL * jp.es);
    const size_t rp = (size_t)jp.rowsP;
    jp.z_off = take(rp * jp.zdim * jp.es);
    jp.a1_off = take(rp * jp.h1 * jp.es);
    jp.a2_off = take(rp * jp.h2 * jp.es);
    jp.dt_off = take(rp * sizeof(float));
    jp.dz2_off = take(rp * jp.h2 * jp.es);
    jp.dz1_off = take(rp * jp.h1 * jp.es);
    jp.dz_off = take(rp * jp.zdim * jp.es);
    const size_t w_max = (size_t)std::max(std::max(jp.h1 * jp.zdim, jp.h2 * jp.h1), jp.gated ? jp.zdim * jp.zdim : 0);
    jp.wt_off = take(w_max * jp.es);
    jp.part_off = take((size_t)kSplits * w_max * sizeof(float));
    if (jp.gated) {
        jp.zf_off = take(rp * jp.zdim * jp.es);
        jp.gate_off = take(rp * jp.zdim * jp.es);
        jp.dzf_off = take(rp * jp.zdim * jp.es);
        jp.gpre_off = take(rp * jp.zdim * jp.es);
    }
    jp.bytes = off;
    return E2EGREC_OK;
}

template <typename T>
int32_t run_joint(const JointPlan &jp, const e2egrec_csr *graph, const e2egrec_mat *X, const int32_t *pair_user,
                  const int32_t *pair_item, const float *dense, const float *labels, const int32_t *fanouts,
                  const e2egrec_mat *W_gnn, const e2egrec_mat *W_tower, const float *const *b_tower, uint64_t seed,
                  uint32_t step, float *loss, float *logits, float *const *dW_gnn, float *const *dW_tower,
                  float *const *db_tower, const e2egrec_mat *dX_rows, int32_t *dX_ids, int32_t *n_dX_rows, char *ws,
                  uint32_t phase, uint32_t flags, cudaStream_t st)
{
    const int relu = (flags & E2EGREC_JOINT_LINEAR) ? 0 : 1;
    int32_t acts[kMaxHops];
    for (int l = 0; l < kMaxHops; ++l) acts[l] = relu;
    e2egrec_block blocks[kMaxHops];
    fill_blocks(jp, ws, blocks);
    auto i32 = [&](size_t off) { return reinterpret_cast<int32_t *>(ws + off); };
    auto tp = [&](size_t off) { return reinterpret_cast<T *>(ws + off); };
    int32_t *pcounts = i32(jp.pcounts_off), *pmeta = i32(jp.pmeta_off);
    int32_t *status = &blocks[0].counts[CNT_STATUS];

    // 1. seeds from the pairs, k-hop sample
    PairInput pi{};
    pi.user = pair_user;
    pi.item = pair_item;
    pi.n_pairs = jp.P;
    pi.seeds_out = i32(jp.seeds_off);
    pi.pair_local = i32(jp.pair_local_off);
    pi.entry_unit = i32(jp.entry_unit_off);
    pi.pcounts = pcounts;
    pi.pcsc_ptr = i32(jp.pcsc_ptr_off);
    pi.pcsc_idx = i32(jp.pcsc_idx_off);
    pi.pcsc_eid = i32(jp.pcsc_eid_off);
    pi.pcsc_col = i32(jp.pcsc_col_off);
    pi.units_per_row = jp.zdim / jp.unit;
    pi.item_unit_off = jp.dL / jp.unit;
    int32_t rc = E2EGREC_OK;
    if (phase != E2EGREC_JOINT_COMPUTE) {
        // alone, the sampling phase completes the block transposition before it returns (the other phase may run
        // on another stream); inside a whole step the transposition is joined by the encoder backward
        rc = sample_khop_impl(graph, nullptr, jp.P2, &pi, jp.n_hops, fanouts, seed, step,
                              phase == E2EGREC_JOINT_SAMPLE ? 0u : E2EGREC_SAMPLE_DEFER_TRANSPOSE, blocks, ws, jp.sampler_bytes, st);
        if (rc != E2EGREC_OK) return rc;
        note_launch();
        joint_meta_kernel<<<1, 1, 0, st>>>(pmeta, jp.P);
        if (phase == E2EGREC_JOINT_SAMPLE) return check_launch("joint_step(sample)");
    }

    // 2. encoder forward: embeddings of the seeds
    e2egrec_mat Hs{tp(jp.hseed_off), pad128(jp.cd[0]), jp.dL, jp.dL, X->dtype};
    size_t ctx_bytes = jp.ctx_bytes;
    rc = e2egrec_sage_forward(blocks, jp.n_hops, X, W_gnn, nullptr, acts, ws + jp.ctx_off, &ctx_bytes, &Hs, st);
    if (rc != E2EGREC_OK) return rc;

    // 3. tower forward and loss
    T *z = tp(jp.z_off), *a1 = tp(jp.a1_off), *a2 = tp(jp.a2_off);
    const T *W1 = static_cast<const T *>(W_tower[0].data), *W2 = static_cast<const T *>(W_tower[1].data),
            *W3 = static_cast<const T *>(W_tower[2].data);
    const float *b1 = b_tower ? b_tower[0] : nullptr, *b2 = b_tower ? b_tower[1] : nullptr,
                *b3 = b_tower ? b_tower[2] : nullptr;
    float *dt = reinterpret_cast<float *>(ws + jp.dt_off);
    {
        const int64_t n = jp.rowsP * jp.zdim;
        note_launch();
        build_z_kernel<T><<<(unsigned)ceil_div(n, 256), 256, 0, st>>>(tp(jp.hseed_off), jp.dL, pi.pair_local, dense, jp.dense_dim,
                                                                     jp.P, jp.rowsP, z);
    }
    // gating fusion (Sec. 4.3.2): the tower reads z_fused = sigmoid(W_g z + b_g) * z instead of z
    const T *tin = z;
    T *gate = nullptr;
    if (jp.gated) {
        T *zf = tp(jp.zf_off);
        gate = tp(jp.gate_off);
        gate_forward_core<T>(GMat<const T>{z, jp.zdim, jp.rowsP}, jp.rowsP, jp.P, jp.zdim, static_cast<const T *>(W_tower[3].data),
                             b_tower ? b_tower[3] : nullptr, tp(jp.gpre_off), GMat<T>{gate, jp.zdim, jp.rowsP},
                             GMat<T>{zf, jp.zdim, jp.rowsP}, pmeta, status, st);
        tin = zf;
    }
    linear_forward<T>(tin, jp.rowsP, jp.zdim, W1, jp.h1, b1, relu, a1, pmeta, status, st);
    linear_forward<T>(a1, jp.rowsP, jp.h1, W2, jp.h2, b2, relu, a2, pmeta, status, st);
    note_launch();
    logit_kernel<T><<<(unsigned)ceil_div((int64_t)jp.P * 32, 256), 256, 0, st>>>(a2, jp.h2, W3, b3, jp.P, logits);
    note_launch();
    bce_kernel<<<1, 1024, 0, st>>>(logits, labels, jp.P, loss, dt, db_tower ? db_tower[2] : nullptr, 0);

    // 4. tower backward
    T *dz2 = tp(jp.dz2_off), *dz1 = tp(jp.dz1_off), *dz = tp(jp.dz_off), *wt = tp(jp.wt_off);
    float *part = reinterpret_cast<float *>(ws + jp.part_off);
    note_launch();
    weighted_colsum_kernel<T><<<(unsigned)ceil_div(jp.h2, 32), 256, 0, st>>>(a2, jp.h2, dt, jp.P, 0, dW_tower[2]);
    {
        const int64_t n = jp.rowsP * jp.h2;
        note_launch();
        dz_top_kernel<T><<<(unsigned)ceil_div(n, 256), 256, 0, st>>>(dt, W3, a2, jp.h2, jp.P, jp.rowsP, relu, dz2);
    }
    // the weight gradients feed nothing later in the step: they go to the helper stream (behind the block
    // transposition that the sampler left there); the encoder backward waits for that stream before its first launch
    SideStream *side = SideStream::get(st);
    cudaStream_t ws_st = st;
    if (side) {
        side->fork(st);
        ws_st = side->stream;
    }
    linear_backward_weight<T>(dz2, jp.rowsP, jp.h2, a1, jp.h1, pmeta, part, dW_tower[1], db_tower ? db_tower[1] : nullptr, status, ws_st);
    linear_backward_input<T>(dz2, jp.rowsP, jp.h2, W2, jp.h1, relu ? a1 : nullptr, dz1, wt, pmeta, status, st);
    if (side) side->fork(st);
    linear_backward_weight<T>(dz1, jp.rowsP, jp.h1, tin, jp.zdim, pmeta, part, dW_tower[0], db_tower ? db_tower[0] : nullptr, status, ws_st);
    if (side) side->defer();
    if (!jp.gated) {
        linear_backward_input<T>(dz1, jp.rowsP, jp.h1, W1, jp.zdim, nullptr, dz, wt, pmeta, status, st);
    } else {
        // through the gate: dz = dz_fused * g + (dz_fused * z * g (1 - g)) W_g, and the gate's own gradients.  The weight
        // gradient above still uses `part` on the helper stream, so the caller's stream waits for it first.
        T *dzf = tp(jp.dzf_off);
        linear_backward_input<T>(dz1, jp.rowsP, jp.h1, W1, jp.zdim, nullptr, dzf, wt, pmeta, status, st);
        if (side) side->join(st);
        gate_backward_core<T>(GMat<const T>{dzf, jp.zdim, jp.rowsP}, GMat<const T>{z, jp.zdim, jp.rowsP},
                              GMat<const T>{gate, jp.zdim, jp.rowsP}, jp.rowsP, jp.P, jp.zdim, static_cast<const T *>(W_tower[3].data),
                              tp(jp.gpre_off), tp(jp.zf_off), wt, part, GMat<T>{dz, jp.zdim, jp.rowsP}, dW_tower[3],
                              db_tower ? db_tower[3] : nullptr, pmeta, status, st);
    }

    // 5. gradient of every seed embedding: the rows of dz that belong to it, added in pair order
    {
        SegOut<T> o{};
        o.out = tp(jp.dhseed_off);
        o.ld_out = jp.dL;
        const SegScratch sc = seg_scratch_carve(jp.P2, kPairRun, jp.dL, dtype_size(X->dtype), ws + jp.seg_off);
        if (!dispatch_seg_reduce<T, int32_t, false>(dz, jp.unit, pi.pcsc_ptr, pi.pcsc_idx, &pcounts[CNT_SRC], 0, jp.P2, nullptr,
                                                    kPairRun, jp.dL, X->dtype, pi.pcsc_col, sc, o, st)) {
            set_last_error("joint_step: no reduction kernel for this embedding width");
            return E2EGREC_ERR_UNSUPPORTED;
        }
    }

    // 6. encoder backward
    e2egrec_mat dHs{tp(jp.dhseed_off), pad128(jp.cd[0]), jp.dL, jp.dL, X->dtype};
    size_t bwd_bytes = jp.bwd_bytes;
    rc = e2egrec_sage_backward(blocks, jp.n_hops, X, W_gnn, acts, ws + jp.ctx_off, &dHs, dW_gnn, nullptr, dX_rows,
                               ws + jp.bwd_off, &bwd_bytes, 0, st);
    if (rc != E2EGREC_OK) return rc;
    const e2egrec_block &outer = blocks[jp.n_hops - 1];
    cudaMemcpyAsync(dX_ids, outer.src_nodes, sizeof(int32_t) * (size_t)outer.cap_src, cudaMemcpyDeviceToDevice, st);
    cudaMemcpyAsync(n_dX_rows, &outer.counts[CNT_SRC], sizeof(int32_t), cudaMemcpyDeviceToDevice, st);
    cudaMemcpyAsync(n_dX_rows + 1, status, sizeof(int32_t), cudaMemcpyDeviceToDevice, st);
    return check_launch("joint_step");
}

}  // namespace
}  // namespace e2egrec

using namespace e2egrec;

extern "C" int32_t e2egrec_joint_step(const e2egrec_csr *graph, const e2egrec_mat *X, const int32_t *pair_user,
                                      const int32_t *pair_item, int32_t n_pairs, const float *dense, int32_t dense_dim,
                                      const float *labels, int32_t n_hops, const int32_t *fanouts,
                                      const e2egrec_mat *W_gnn, const e2egrec_mat *W_tower, const float *const *b_tower,
                                      uint64_t seed, uint32_t step, float *loss, float *logits, float *const *dW_gnn,
                                      float *const *dW_tower, float *const *db_tower, const e2egrec_mat *dX_rows,
                                      int32_t *dX_ids, int32_t *n_dX_rows, void *ws, size_t *ws_bytes, void *stream)
{
    return e2egrec_joint_step_phase(graph, X, pair_user, pair_item, n_pairs, dense, dense_dim, labels, n_hops, fanouts, W_gnn,
                                    W_tower, b_tower, seed, step, loss, logits, dW_gnn, dW_tower, db_tower, dX_rows, dX_ids,
                                    n_dX_rows, ws, ws_bytes, E2EGREC_JOINT_WHOLE, stream);
}

extern "C" int32_t e2egrec_joint_step_phase(const e2egrec_csr *graph, const e2egrec_mat *X, const int32_t *pair_user,
                                            const int32_t *pair_item, int32_t n_pairs, const float *dense,
                                            int32_t dense_dim, const float *labels, int32_t n_hops,
                                            const int32_t *fanouts, const e2egrec_mat *W_gnn, const e2egrec_mat *W_tower,
                                            const float *const *b_tower, uint64_t seed, uint32_t step, float *loss,
                                            float *logits, float *const *dW_gnn, float *const *dW_tower,
                                            float *const *db_tower, const e2egrec_mat *dX_rows, int32_t *dX_ids,
                                            int32_t *n_dX_rows, void *ws, size_t *ws_bytes, uint32_t phase, void *stream)
{
    if (!ws_bytes) return E2EGREC_ERR_NULL;
    const uint32_t flags = phase & ~0xFFu;
    phase &= 0xFFu;
    if (phase > E2EGREC_JOINT_COMPUTE || (flags & ~(E2EGREC_JOINT_LINEAR | E2EGREC_JOINT_GATE))) return E2EGREC_ERR_ARG;
    JointPlan jp{};
    int32_t rc = make_plan(graph, X, n_pairs, dense_dim, n_hops, fanouts, W_gnn, W_tower, flags, jp);
    if (rc != E2EGREC_OK) return rc;
    if (!ws) { *ws_bytes = jp.bytes; return E2EGREC_OK; }
    if (*ws_bytes < jp.bytes) { *ws_bytes = jp.bytes; return E2EGREC_ERR_WORKSPACE; }
    if (reinterpret_cast<uintptr_t>(ws) % 256) return E2EGREC_ERR_ALIGN;
    if (!pair_user || !pair_item || !labels || !loss || !logits || !dW_gnn || !dW_tower || !dX_rows || !dX_rows->data ||
        !dX_ids || !n_dX_rows || (dense_dim > 0 && !dense))
        return E2EGREC_ERR_NULL;
    for (int l = 0; l < n_hops; ++l)
        if (!dW_gnn[l]) return E2EGREC_ERR_NULL;
    for (int k = 0; k < 3 + jp.gated; ++k)
        if (!dW_tower[k]) return E2EGREC_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (X->dtype == E2EGREC_BF16)
        return run_joint<__nv_bfloat16>(jp, graph, X, pair_user, pair_item, dense, labels, fanouts, W_gnn, W_tower, b_tower, seed,
                                        step, loss, logits, dW_gnn, dW_tower, db_tower, dX_rows, dX_ids, n_dX_rows,
                                        static_cast<char *>(ws), phase, flags, st);
    return run_joint<float>(jp, graph, X, pair_user, pair_item, dense, labels, fanouts, W_gnn, W_tower, b_tower, seed, step, loss,
                            logits, dW_gnn, dW_tower, db_tower, dX_rows, dX_ids, n_dX_rows, static_cast<char *>(ws), phase, flags,
                            st);
}

extern "C" int32_t e2egrec_joint_step_layout(const e2egrec_csr *graph, const e2egrec_mat *X, int32_t n_pairs, int32_t dense_dim,
                                             int32_t n_hops, const int32_t *fanouts, const e2egrec_mat *W_gnn,
                                             const e2egrec_mat *W_tower, uint32_t flags, size_t *tower_offset,
                                             size_t *enc_h_offset, int64_t *enc_rows, int64_t *pair_rows,
                                             size_t *counts_offset)
{
    if (!tower_offset || !enc_h_offset || !enc_rows || !pair_rows || !counts_offset) return E2EGREC_ERR_NULL;
    if (flags & ~(E2EGREC_JOINT_LINEAR | E2EGREC_JOINT_GATE)) return E2EGREC_ERR_ARG;
    JointPlan jp{};
    int32_t rc = make_plan(graph, X, n_pairs, dense_dim, n_hops, fanouts, W_gnn, W_tower, flags, jp);
    if (rc != E2EGREC_OK) return rc;
    e2egrec_block blocks[kMaxHops];
    fill_blocks(jp, nullptr, blocks);
    size_t cat_off[kMaxHops], h_off[kMaxHops];
    rc = e2egrec_sage_ctx_layout(blocks, n_hops, X, W_gnn, cat_off, h_off, enc_rows);
    if (rc != E2EGREC_OK) return rc;
    for (int l = 0; l < n_hops; ++l) enc_h_offset[l] = jp.ctx_off + h_off[l];
    for (int h = 0; h < n_hops; ++h) counts_offset[h] = jp.blk_off[h][0];
    tower_offset[0] = jp.z_off;
    tower_offset[1] = jp.a1_off;
    tower_offset[2] = jp.a2_off;
    tower_offset[3] = jp.gated ? jp.gate_off : jp.z_off;
    tower_offset[4] = jp.gated ? jp.zf_off : jp.z_off;
    *pair_rows = jp.rowsP;
    return E2EGREC_OK;
}

namespace e2egrec {
namespace {

struct GatePlan {
    int d;
    int64_t rows;          // rows of the scratch matrices: n_rows rounded up to 128
    size_t es, meta_off, a_off, b_off, wt_off, part_off, bytes;
};

int32_t gate_plan(const e2egrec_mat *F, int32_t n_rows, const e2egrec_mat *Wg, GatePlan &gp)
{
    if (!F || !Wg || !F->data || !Wg->data) return E2EGREC_ERR_NULL;
    if (F->dtype != E2EGREC_F32 && F->dtype != E2EGREC_BF16) return E2EGREC_ERR_DTYPE;
    if (Wg->dtype != F->dtype) return E2EGREC_ERR_DTYPE;
    if (n_rows < 0 || F->dim < 1 || F->dim > kMaxDim || F->ld < F->dim) return E2EGREC_ERR_ARG;
    if (Wg->rows != F->dim || Wg->dim != F->dim || Wg->ld != Wg->dim) return E2EGREC_ERR_ARG;
    gp.d = F->dim;
    gp.es = dtype_size(F->dtype);
    gp.rows = pad128(n_rows > 0 ? n_rows : 1);
    if (F->rows < gp.rows) return E2EGREC_ERR_ARG;       // the dense products read whole 128-row tiles of F
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += align_up(b, 256); return o; };
    gp.meta_off = take(256);
    gp.a_off = take((size_t)gp.rows * gp.d * gp.es);     // pre-activation / d pre
    gp.b_off = take((size_t)gp.rows * gp.d * gp.es);     // d pre Wg
    gp.wt_off = take((size_t)gp.d * gp.d * gp.es);
    gp.part_off = take((size_t)kSplits * gp.d * gp.d * sizeof(float));
    gp.bytes = off;
    return E2EGREC_OK;
}

template <typename T> GMat<const T> cmat(const e2egrec_mat *m) { return GMat<const T>{static_cast<const T *>(m->data), m->ld, m->rows}; }
template <typename T> GMat<T> wmat(const e2egrec_mat *m) { return GMat<T>{static_cast<T *>(m->data), m->ld, m->rows}; }

template <typename T>
int32_t gate_forward_impl(const GatePlan &gp, const e2egrec_mat *F, int32_t n_rows, const e2egrec_mat *Wg, const float *bg,
                          const e2egrec_mat *gate, const e2egrec_mat *fused, char *ws, cudaStream_t st)
{
    int32_t *meta = reinterpret_cast<int32_t *>(ws + gp.meta_off);      // {rows, status}
    note_launch();
    gate_meta_kernel<<<1, 1, 0, st>>>(meta, n_rows);
    cudaMemsetAsync(meta + 1, 0, sizeof(int32_t), st);
    gate_forward_core<T>(cmat<T>(F), gp.rows, n_rows, gp.d, static_cast<const T *>(Wg->data), bg,
                         reinterpret_cast<T *>(ws + gp.a_off), wmat<T>(gate), wmat<T>(fused), meta, meta + 1, st);
    return check_launch("gate_fusion_forward");
}

template <typename T>
int32_t gate_backward_impl(const GatePlan &gp, const e2egrec_mat *dFused, const e2egrec_mat *F, int32_t n_rows,
                           const e2egrec_mat *gate, const e2egrec_mat *Wg, const e2egrec_mat *dF, float *dWg, float *dbg,
                           char *ws, cudaStream_t st)
{
    int32_t *meta = reinterpret_cast<int32_t *>(ws + gp.meta_off);
    note_launch();
    gate_meta_kernel<<<1, 1, 0, st>>>(meta, n_rows);
    cudaMemsetAsync(meta + 1, 0, sizeof(int32_t), st);
    gate_backward_core<T>(cmat<T>(dFused), cmat<T>(F), cmat<T>(gate), gp.rows, n_rows, gp.d, static_cast<const T *>(Wg->data),
                          reinterpret_cast<T *>(ws + gp.a_off), reinterpret_cast<T *>(ws + gp.b_off),
                          reinterpret_cast<T *>(ws + gp.wt_off), reinterpret_cast<float *>(ws + gp.part_off), wmat<T>(dF), dWg, dbg,
                          meta, meta + 1, st);
    return check_launch("gate_fusion_backward");
}

int32_t gate_check_out(const e2egrec_mat *m, const e2egrec_mat *F, int32_t n_rows)
{
    if (!m || !m->data) return E2EGREC_ERR_NULL;
    if (m->dtype != F->dtype) return E2EGREC_ERR_DTYPE;
    if (m->dim != F->dim || m->ld < m->dim || m->rows < n_rows) return E2EGREC_ERR_ARG;
    return E2EGREC_OK;
}

}  // namespace
}  // namespace e2egrec

extern "C" int32_t e2egrec_gate_fusion_forward(const e2egrec_mat *F, int32_t n_rows, const e2egrec_mat *Wg, const float *bg,
                                               const e2egrec_mat *gate, const e2egrec_mat *fused, void *ws, size_t *ws_bytes,
                                               void *stream)
{
    if (!ws_bytes) return E2EGREC_ERR_NULL;
    GatePlan gp{};
    int32_t rc = gate_plan(F, n_rows, Wg, gp);
    if (rc != E2EGREC_OK) return rc;
    if (!ws) { *ws_bytes = gp.bytes; return E2EGREC_OK; }
    if (*ws_bytes < gp.bytes) { *ws_bytes = gp.bytes; return E2EGREC_ERR_WORKSPACE; }
    if (reinterpret_cast<uintptr_t>(ws) % 256) return E2EGREC_ERR_ALIGN;
    if ((rc = gate_check_out(gate, F, n_rows)) != E2EGREC_OK || (rc = gate_check_out(fused, F, n_rows)) != E2EGREC_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (F->dtype == E2EGREC_BF16)
        return gate_forward_impl<__nv_bfloat16>(gp, F, n_rows, Wg, bg, gate, fused, static_cast<char *>(ws), st);
    return gate_forward_impl<float>(gp, F, n_rows, Wg, bg, gate, fused, static_cast<char *>(ws), st);
}

extern "C" int32_t e2egrec_gate_fusion_backward(const e2egrec_mat *dFused, const e2egrec_mat *F, int32_t n_rows,
                                                const e2egrec_mat *gate, const e2egrec_mat *Wg, const e2egrec_mat *dF,
                                                float *dWg, float *dbg, void *ws, size_t *ws_bytes, void *stream)
{
    if (!ws_bytes) return E2EGREC_ERR_NULL;
    GatePlan gp{};
    int32_t rc = gate_plan(F, n_rows, Wg, gp);
    if (rc != E2EGREC_OK) return rc;
    if (!ws) { *ws_bytes = gp.bytes; return E2EGREC_OK; }
    if (*ws_bytes < gp.bytes) { *ws_bytes = gp.bytes; return E2EGREC_ERR_WORKSPACE; }
    if (reinterpret_cast<uintptr_t>(ws) % 256) return E2EGREC_ERR_ALIGN;
    if (!dWg) return E2EGREC_ERR_NULL;
    if ((rc = gate_check_out(dFused, F, n_rows)) != E2EGREC_OK || (rc = gate_check_out(gate, F, n_rows)) != E2EGREC_OK ||
        (rc = gate_check_out(dF, F, n_rows)) != E2EGREC_OK)
        return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (F->dtype == E2EGREC_BF16)
        return gate_backward_impl<__nv_bfloat16>(gp, dFused, F, n_rows, gate, Wg, dF, dWg, dbg, static_cast<char *>(ws), st);
    return gate_backward_impl<float>(gp, dFused, F, n_rows, gate, Wg, dF, dWg, dbg, static_cast<char *>(ws), st);
}
