// The self-supervised task of the GNN and the balancing of the two task weights (SSL task: Sec. 4.2; GradNorm: Sec. 4.3.1):
//   L_ssl = || X_seeds - H ||_F^2   (graph feature auto-encoder with the identity decoder),
//   G_i   = || grad of (w_i L_i) with respect to the shared input rows ||_2,
//   GradNorm step for the weights w_i.
// Sums run in a fixed order (slices per block, then one block over the slice sums), so results are
// bit-identical from run to run.
#include <algorithm>

#include "common.cuh"

namespace e2egrec {
namespace {

constexpr int kSumBlocks = 148 * 8;   // slices of the first stage (fixed, so that the order of the additions is)
constexpr int kSumThreads = 256;
constexpr int kMaxTasks = 8;
constexpr int kMaxNorms = 4;          // matrices of one e2egrec_gradient_norms call

__device__ inline float block_sum_256(float v, float *red)
{
    red[threadIdx.x] = v;
    __syncthreads();
    for (int o = kSumThreads / 2; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    return red[0];
}

struct NormArgs {
    const void *A[kMaxNorms];
    int64_t lda[kMaxNorms];
};

// Stage 1.  kSsl: v = h - x (x read through the seed ids), dH = 2 w v is written; else v = a (matrix blockIdx.y).
// part[matrix][block] = sum of v^2 over the block's slice of the n_rows x d cells, walked in 16-byte chunks where the
// rows allow it.
template <typename T, bool kSsl>
__global__ void __launch_bounds__(kSumThreads)
sumsq_slices_kernel(NormArgs a, const T *__restrict__ X, int64_t ldx, const int32_t *__restrict__ ids,
                    const int32_t *__restrict__ n_rows_dev, int64_t n_rows_cap, int d, int vec,
                    const float *__restrict__ weight, T *__restrict__ dH, int64_t ldh, float *__restrict__ part)
{
    __shared__ float red[kSumThreads];
    constexpr int E = Chunk<T>::kElems;
    const T *__restrict__ A = static_cast<const T *>(a.A[blockIdx.y]);
    const int64_t lda = a.lda[blockIdx.y];
    int64_t rows = n_rows_dev ? (int64_t)*n_rows_dev : n_rows_cap;
    if (rows > n_rows_cap) rows = n_rows_cap;
    const float w2 = kSsl ? 2.0f * weight[0] : 0.f;
    float s = 0.f;
    if (vec) {
        const int cpr = d / E;                                 // chunks per row
        const int64_t chunks = rows * cpr;
        const int64_t per = (chunks + kSumBlocks - 1) / kSumBlocks;
        const int64_t c0 = (int64_t)blockIdx.x * per, c1 = min(c0 + per, chunks);
        for (int64_t c = c0 + threadIdx.x; c < c1; c += kSumThreads) {
            const int64_t i = c / cpr;
            const int k = (int)(c - i * cpr) * E;
            float v[E];
            Chunk<T>::load(A + i * lda + k, v);
            if (kSsl) {
                float x[E];
                Chunk<T>::load(X + (int64_t)ids[i] * ldx + k, x);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    v[e] -= x[e];
                    x[e] = w2 * v[e];
                }
                Chunk<T>::store(dH + i * ldh + k, x);
            }
#pragma unroll
            for (int e = 0; e < E; ++e) s += v[e] * v[e];
        }
    } else {
        const int64_t cells = rows * d;
        const int64_t per = (cells + kSumBlocks - 1) / kSumBlocks;
        const int64_t c0 = (int64_t)blockIdx.x * per, c1 = min(c0 + per, cells);
        for (int64_t c = c0 + threadIdx.x; c < c1; c += kSumThreads) {
            const int64_t i = c / d;
            const int k = (int)(c % d);
            float v = to_float<T>(A[i * lda + k]);
            if (kSsl) {
                v -= to_float<T>(X[(int64_t)ids[i] * ldx + k]);
                dH[i * ldh + k] = from_float<T>(w2 * v);
            }
            s += v * v;
        }
    }
    const float tot = block_sum_256(s, red);
    if (threadIdx.x == 0) part[(int64_t)blockIdx.y * kSumBlocks + blockIdx.x] = tot;
}

// Stage 2: out[matrix] = sum of the slice sums in slice order (its square root with take_sqrt); one block per matrix
__global__ void __launch_bounds__(kSumThreads)
sumsq_final_kernel(const float *__restrict__ part, int take_sqrt, float *__restrict__ out)
{
    __shared__ float red[kSumThreads];
    const float *p = part + (int64_t)blockIdx.x * kSumBlocks;
    float s = 0.f;
    for (int j = threadIdx.x; j < kSumBlocks; j += kSumThreads) s += p[j];
    const float tot = block_sum_256(s, red);
    if (threadIdx.x == 0) out[blockIdx.x] = take_sqrt ? sqrtf(tot) : tot;
}

// rows of 16-byte chunks: width, leading dimension and base address all allow vector loads
template <typename T>
int vec_ok(const void *p, int64_t ld, int d)
{
    constexpr int E = Chunk<T>::kElems;
    return d % E == 0 && ld % E == 0 && reinterpret_cast<uintptr_t>(p) % 16 == 0;
}

// One GradNorm step, one thread (a handful of scalars)
__global__ void gradnorm_kernel(float *__restrict__ w, const float *__restrict__ L, const float *__restrict__ L0,
                                const float *__restrict__ g, int T, float gamma, float lr, float w_min,
                                float *__restrict__ L_gn)
{
    float G[kMaxTasks], ratio[kMaxTasks];
    float g_mean = 0.f, r_mean = 0.f;
    for (int i = 0; i < T; ++i) {
        G[i] = w[i] * g[i];
        ratio[i] = L[i] / L0[i];
        g_mean += G[i];
        r_mean += ratio[i];
    }
    g_mean /= (float)T;
    r_mean /= (float)T;
    float obj = 0.f, sum = 0.f, wn[kMaxTasks];
    for (int i = 0; i < T; ++i) {
        const float c = g_mean * powf(ratio[i] / r_mean, gamma);
        const float diff = G[i] - c;
        obj += fabsf(diff);
        const float sgn = diff > 0.f ? 1.f : (diff < 0.f ? -1.f : 0.f);
        wn[i] = fmaxf(w[i] - lr * sgn * g[i], w_min);
        sum += wn[i];
    }
    for (int i = 0; i < T; ++i) w[i] = wn[i] * ((float)T / sum);
    if (L_gn) L_gn[0] = obj;
}

int32_t check_mat(const e2egrec_mat *m)
{
    if (!m || !m->data) return E2EGREC_ERR_NULL;
    if (m->dtype != E2EGREC_F32 && m->dtype != E2EGREC_BF16) return E2EGREC_ERR_DTYPE;
    if (m->dim < 1 || m->rows < 0 || m->ld < m->dim) return E2EGREC_ERR_ARG;
    return E2EGREC_OK;
}

}  // namespace
}  // namespace e2egrec

using namespace e2egrec;

extern "C" int32_t e2egrec_ssl_loss(const e2egrec_mat *H, const e2egrec_mat *X, const int32_t *seed_ids,
                                    const int32_t *n_rows_dev, const float *weight, float *loss, const e2egrec_mat *dH,
                                    void *ws, size_t *ws_bytes, void *stream)
{
    if (!ws_bytes) return E2EGREC_ERR_NULL;
    const size_t need = (size_t)kMaxNorms * kSumBlocks * sizeof(float);
    if (!ws) { *ws_bytes = need; return E2EGREC_OK; }
    if (*ws_bytes < need) { *ws_bytes = need; return E2EGREC_ERR_WORKSPACE; }
    int32_t rc = check_mat(H);
    if (rc == E2EGREC_OK) rc = check_mat(X);
    if (rc == E2EGREC_OK) rc = check_mat(dH);
    if (rc != E2EGREC_OK) return rc;
    if (!seed_ids || !weight || !loss) return E2EGREC_ERR_NULL;
    if (X->dtype != H->dtype || dH->dtype != H->dtype) return E2EGREC_ERR_DTYPE;
    if (X->dim != H->dim || dH->dim != H->dim || dH->rows < H->rows) return E2EGREC_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float *part = static_cast<float *>(ws);
    NormArgs na{};
    na.A[0] = H->data;
    na.lda[0] = H->ld;
    note_launch();
    if (H->dtype == E2EGREC_BF16) {
        using T = __nv_bfloat16;
        const int vec = vec_ok<T>(H->data, H->ld, H->dim) && vec_ok<T>(X->data, X->ld, X->dim) && vec_ok<T>(dH->data, dH->ld, dH->dim);
        sumsq_slices_kernel<T, true><<<kSumBlocks, kSumThreads, 0, st>>>(na, static_cast<const T *>(X->data), X->ld, seed_ids, n_rows_dev,
                                                                        H->rows, H->dim, vec, weight, static_cast<T *>(dH->data),
                                                                        dH->ld, part);
    } else {
        using T = float;
        const int vec = vec_ok<T>(H->data, H->ld, H->dim) && vec_ok<T>(X->data, X->ld, X->dim) && vec_ok<T>(dH->data, dH->ld, dH->dim);
        sumsq_slices_kernel<T, true><<<kSumBlocks, kSumThreads, 0, st>>>(na, static_cast<const T *>(X->data), X->ld, seed_ids, n_rows_dev,
                                                                        H->rows, H->dim, vec, weight, static_cast<T *>(dH->data),
                                                                        dH->ld, part);
    }
    note_launch();
    sumsq_final_kernel<<<1, kSumThreads, 0, st>>>(part, 0, loss);
    return check_launch("ssl_loss");
}

static int32_t gradient_norms_impl(const e2egrec_mat *A, int32_t n, const int32_t *n_rows_dev, float *norms, void *ws,
                                   size_t *ws_bytes, void *stream)
{
    if (!ws_bytes) return E2EGREC_ERR_NULL;
    if (n < 1 || n > kMaxNorms) return E2EGREC_ERR_ARG;
    const size_t need = (size_t)kMaxNorms * kSumBlocks * sizeof(float);
    if (!ws) { *ws_bytes = need; return E2EGREC_OK; }
    if (*ws_bytes < need) { *ws_bytes = need; return E2EGREC_ERR_WORKSPACE; }
    NormArgs na{};
    int vec = 1;
    for (int i = 0; i < n; ++i) {
        const int32_t rc = check_mat(&A[i]);
        if (rc != E2EGREC_OK) return rc;
        if (A[i].dtype != A[0].dtype) return E2EGREC_ERR_DTYPE;
        if (A[i].dim != A[0].dim || A[i].rows != A[0].rows) return E2EGREC_ERR_ARG;
        na.A[i] = A[i].data;
        na.lda[i] = A[i].ld;
        vec = vec && (A[0].dtype == E2EGREC_BF16 ? vec_ok<__nv_bfloat16>(A[i].data, A[i].ld, A[i].dim)
                                                 : vec_ok<float>(A[i].data, A[i].ld, A[i].dim));
    }
    if (!norms) return E2EGREC_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float *part = static_cast<float *>(ws);
    note_launch();
    if (A[0].dtype == E2EGREC_BF16)
        sumsq_slices_kernel<__nv_bfloat16, false><<<dim3(kSumBlocks, n), kSumThreads, 0, st>>>(na, nullptr, 0, nullptr, n_rows_dev,
                                                                                              A[0].rows, A[0].dim, vec, nullptr,
                                                                                              nullptr, 0, part);
    else
        sumsq_slices_kernel<float, false><<<dim3(kSumBlocks, n), kSumThreads, 0, st>>>(na, nullptr, 0, nullptr, n_rows_dev, A[0].rows,
                                                                                      A[0].dim, vec, nullptr, nullptr, 0, part);
    note_launch();
    sumsq_final_kernel<<<n, kSumThreads, 0, st>>>(part, 1, norms);
    return check_launch("gradient_norm");
}

extern "C" int32_t e2egrec_gradient_norm(const e2egrec_mat *A, const int32_t *n_rows_dev, float *norm, void *ws,
                                         size_t *ws_bytes, void *stream)
{
    if (!A && ws) return E2EGREC_ERR_NULL;
    return gradient_norms_impl(A, 1, n_rows_dev, norm, ws, ws_bytes, stream);
}

extern "C" int32_t e2egrec_gradient_norms(const e2egrec_mat *A, int32_t n, const int32_t *n_rows_dev, float *norms, void *ws,
                                          size_t *ws_bytes, void *stream)
{
    if (!A && ws) return E2EGREC_ERR_NULL;
    return gradient_norms_impl(A, n, n_rows_dev, norms, ws, ws_bytes, stream);
}

extern "C" int32_t e2egrec_gradnorm_update(float *w, const float *L, const float *L0, const float *g, int32_t n_tasks,
                                           float gamma, float lr, float *L_gn, void *stream)
{
    if (!w || !L || !L0 || !g) return E2EGREC_ERR_NULL;
    if (n_tasks < 1 || n_tasks > kMaxTasks || !(lr >= 0.f)) return E2EGREC_ERR_ARG;
    note_launch();
    gradnorm_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(w, L, L0, g, n_tasks, gamma, lr, 1e-6f, L_gn);
    return check_launch("gradnorm_update");
}
