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

constexpr int kSumBlocks = 256;       // slices of the first stage
constexpr int kSumThreads = 256;
constexpr int kMaxTasks = 8;

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

// Stage 1.  kSsl: v = h - x (x read through the seed ids), dH = 2 w v is written; else v = a.
// part[block] = sum of v^2 over the block's slice of the n_rows x d cells.
template <typename T, bool kSsl>
__global__ void __launch_bounds__(kSumThreads)
sumsq_slices_kernel(const T *__restrict__ A, int64_t lda, const T *__restrict__ X, int64_t ldx,
                    const int32_t *__restrict__ ids, const int32_t *__restrict__ n_rows_dev, int64_t n_rows_cap, int d,
                    const float *__restrict__ weight, T *__restrict__ dH, int64_t ldh, float *__restrict__ part)
{
    __shared__ float red[kSumThreads];
    int64_t rows = n_rows_dev ? (int64_t)*n_rows_dev : n_rows_cap;
    if (rows > n_rows_cap) rows = n_rows_cap;
    const int64_t cells = rows * d;
    const int64_t per = (cells + kSumBlocks - 1) / kSumBlocks;
    const int64_t c0 = (int64_t)blockIdx.x * per, c1 = min(c0 + per, cells);
    const float w2 = kSsl ? 2.0f * weight[0] : 0.f;
    float s = 0.f;
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
    const float tot = block_sum_256(s, red);
    if (threadIdx.x == 0) part[blockIdx.x] = tot;
}

// Stage 2: out = sum of the slice sums (its square root with take_sqrt)
__global__ void __launch_bounds__(kSumThreads)
sumsq_final_kernel(const float *__restrict__ part, int take_sqrt, float *__restrict__ out)
{
    __shared__ float red[kSumThreads];
    const float tot = block_sum_256(threadIdx.x < kSumBlocks ? part[threadIdx.x] : 0.f, red);
    if (threadIdx.x == 0) out[0] = take_sqrt ? sqrtf(tot) : tot;
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
    const size_t need = kSumBlocks * sizeof(float);
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
    note_launch();
    if (H->dtype == E2EGREC_BF16)
        sumsq_slices_kernel<__nv_bfloat16, true><<<kSumBlocks, kSumThreads, 0, st>>>(
            static_cast<const __nv_bfloat16 *>(H->data), H->ld, static_cast<const __nv_bfloat16 *>(X->data), X->ld, seed_ids,
            n_rows_dev, H->rows, H->dim, weight, static_cast<__nv_bfloat16 *>(dH->data), dH->ld, part);
    else
        sumsq_slices_kernel<float, true><<<kSumBlocks, kSumThreads, 0, st>>>(
            static_cast<const float *>(H->data), H->ld, static_cast<const float *>(X->data), X->ld, seed_ids, n_rows_dev,
            H->rows, H->dim, weight, static_cast<float *>(dH->data), dH->ld, part);
    note_launch();
    sumsq_final_kernel<<<1, kSumThreads, 0, st>>>(part, 0, loss);
    return check_launch("ssl_loss");
}

extern "C" int32_t e2egrec_gradient_norm(const e2egrec_mat *A, const int32_t *n_rows_dev, float *norm, void *ws,
                                         size_t *ws_bytes, void *stream)
{
    if (!ws_bytes) return E2EGREC_ERR_NULL;
    const size_t need = kSumBlocks * sizeof(float);
    if (!ws) { *ws_bytes = need; return E2EGREC_OK; }
    if (*ws_bytes < need) { *ws_bytes = need; return E2EGREC_ERR_WORKSPACE; }
    const int32_t rc = check_mat(A);
    if (rc != E2EGREC_OK) return rc;
    if (!norm) return E2EGREC_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float *part = static_cast<float *>(ws);
    note_launch();
    if (A->dtype == E2EGREC_BF16)
        sumsq_slices_kernel<__nv_bfloat16, false><<<kSumBlocks, kSumThreads, 0, st>>>(
            static_cast<const __nv_bfloat16 *>(A->data), A->ld, nullptr, 0, nullptr, n_rows_dev, A->rows, A->dim, nullptr,
            nullptr, 0, part);
    else
        sumsq_slices_kernel<float, false><<<kSumBlocks, kSumThreads, 0, st>>>(static_cast<const float *>(A->data), A->ld, nullptr,
                                                                             0, nullptr, n_rows_dev, A->rows, A->dim, nullptr,
                                                                             nullptr, 0, part);
    note_launch();
    sumsq_final_kernel<<<1, kSumThreads, 0, st>>>(part, 1, norm);
    return check_launch("gradient_norm");
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
