// fp32-FMA tiled GEMM for the true-fp32 path (rel 1e-5 against float64 rules out TF32) and as
// the reference path for shapes the tensor-core kernels do not take.
//   C(m, n) = sum_k A(m, k) * B(n, k)
// A_KM: A is stored k-major (element (m,k) at A[k*lda + m]) instead of m-major (A[m*lda + k]).
// B_KN: B is stored k-major (element (n,k) at B[k*ldb + n]) instead of n-major (B[n*ldb + k]).
// M and/or K may live on the device (m_dev / k_dev); the grid is sized for the caps.
// gridDim.z splits K; the epilogue receives the split index.
#pragma once

#include "common.cuh"

namespace e2egrec {

constexpr int kGemmBM = 64, kGemmBN = 64, kGemmBK = 16, kGemmThreads = 256;

template <typename T, bool A_KM, bool B_KN, class Epi>
__global__ void __launch_bounds__(kGemmThreads)
gemm_simt_kernel(const T *__restrict__ A, int64_t lda, const T *__restrict__ B, int64_t ldb, int64_t M_host,
                 int N, int64_t K_host, const int32_t *m_dev, const int32_t *k_dev, Epi epi)
{
    __shared__ float As[kGemmBK][kGemmBM + 4];
    __shared__ float Bs[kGemmBK][kGemmBN + 4];
    const int64_t M = m_dev ? min((int64_t)*m_dev, M_host) : M_host;
    const int64_t K = k_dev ? min((int64_t)*k_dev, K_host) : K_host;
    const int64_t m0 = (int64_t)blockIdx.x * kGemmBM;
    const int n0 = blockIdx.y * kGemmBN;
    if (m0 >= M) return;
    // K range of this split, a multiple of the k tile
    const int64_t k_per = ceil_div(ceil_div(K, (int64_t)gridDim.z), kGemmBK) * kGemmBK;
    const int64_t kb = (int64_t)blockIdx.z * k_per;
    const int64_t ke = min(K, kb + k_per);
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int64_t k0 = kb; k0 < ke; k0 += kGemmBK) {
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int id = threadIdx.x + t * kGemmThreads;
            int r, kk;
            if (A_KM) { r = id & 63; kk = id >> 6; } else { r = id >> 4; kk = id & 15; }
            const int64_t m = m0 + r, k = k0 + kk;
            float v = 0.f;
            if (m < M && k < ke) v = to_float<T>(A_KM ? A[k * lda + m] : A[m * lda + k]);
            As[kk][r] = v;
            if (B_KN) { r = id & 63; kk = id >> 6; } else { r = id >> 4; kk = id & 15; }
            const int64_t n = n0 + r;
            v = 0.f;
            if (n < N && k0 + kk < ke) v = to_float<T>(B_KN ? B[(k0 + kk) * ldb + n] : B[n * ldb + k0 + kk]);
            Bs[kk][r] = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kGemmBK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t m = m0 + ty * 4 + i;
            const int n = n0 + tx * 4 + j;
            if (m < M && n < N) epi(m, n, acc[i][j], blockIdx.z);
        }
}

// h' = act(z + b), stored in the feature dtype
template <typename T>
struct EpiUpdate {
    T *out; int64_t ldo; const float *bias; int relu;
    __device__ void operator()(int64_t m, int n, float z, int) const {
        if (bias) z += bias[n];
        if (relu && z < 0.f) z = 0.f;
        out[m * ldo + n] = from_float<T>(z);
    }
};

// dCat = [dSelf | dAgg * (1/|S|)], stored in the feature dtype
template <typename T>
struct EpiDCat {
    T *out; int64_t ldo; int d_in; const float *inv_cnt;
    __device__ void operator()(int64_t m, int n, float v, int) const {
        if (n >= d_in) v *= inv_cnt[m];
        out[m * ldo + n] = from_float<T>(v);
    }
};

// split-K partial sums, fp32
struct EpiPartial {
    float *out; int64_t ldo; int64_t split_stride;
    __device__ void operator()(int64_t m, int n, float v, int z) const { out[z * split_stride + m * ldo + n] = v; }
};

// out = (accumulate ? out : 0) + sum_z partial[z], z ascending.  With rows_dev the partials come from the
// tensor-core weight-gradient kernel, which only fills the first ceil(total / per) splits
// (total = ceil(rows / 64) k-blocks, per = max(8, ceil(total / splits))); without it all splits are added.
static __global__ void splitk_reduce_kernel(const float *__restrict__ partial, int64_t n, int splits, int accumulate,
                                            float *__restrict__ out, const int32_t *rows_dev, int n_rhs = 1)
{
    pdl_launch_dependents();
    pdl_wait();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    int active = splits;
    if (rows_dev) {
        const int64_t total = (((int64_t)*rows_dev + 63) / 64) * n_rhs;
        const int64_t per = max((int64_t)8, (total + splits - 1) / splits);
        active = (int)max((int64_t)1, (total + per - 1) / per);
    }
    float s = accumulate ? out[i] : 0.f;
    for (int z = 0; z < active; ++z) s += partial[(int64_t)z * n + i];
    out[i] = s;
}

// dZ = dH where the stored output is positive (or everywhere for the identity activation);
// rows in [n, rows_alloc) are set to zero.  gridDim.y = 2: a second gradient dH1 goes to the block of rows_alloc
// rows behind the first in dZ (two right-hand sides sent through the backward pass together).
template <typename T>
__global__ void relu_mask_kernel(const T *__restrict__ dH, int64_t ld_dh, const T *__restrict__ H, int64_t ld_h,
                                 const int32_t *n_dev, int64_t rows_alloc, int d, int relu, T *__restrict__ dZ,
                                 const T *__restrict__ dH1 = nullptr, int64_t ld_dh1 = 0)
{
    pdl_launch_dependents();
    pdl_wait();
    if (blockIdx.y == 1) {
        dH = dH1;
        ld_dh = ld_dh1;
        dZ += rows_alloc * d;
    }
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t r = i / d;
    const int k = (int)(i - r * d);
    if (r >= rows_alloc) return;
    T v = from_float<T>(0.f);
    if (r < *n_dev) {
        v = dH[r * ld_dh + k];
        if (relu && !(to_float<T>(H[r * ld_h + k]) > 0.f)) v = from_float<T>(0.f);
    }
    dZ[r * d + k] = v;
}

// db[o] = (accumulate ? db[o] : 0) + sum over rows of dZ[:, o]; one block per 32 columns, rows in a fixed order.
template <typename T>
__global__ void __launch_bounds__(256)
colsum_kernel(const T *__restrict__ dZ, int64_t ld, const int32_t *n_dev, int d, int accumulate, float *__restrict__ db)
{
    __shared__ float red[8][32];
    const int col = blockIdx.x * 32 + (threadIdx.x & 31);
    const int rl = threadIdx.x >> 5;
    const int64_t n = *n_dev;
    float s = 0.f;
    if (col < d)
        for (int64_t r = rl; r < n; r += 8) s += to_float<T>(dZ[r * ld + col]);
    red[rl][threadIdx.x & 31] = s;
    __syncthreads();
    if (rl == 0 && col < d) {
        float t = accumulate ? db[col] : 0.f;
        for (int w = 0; w < 8; ++w) t += red[w][threadIdx.x & 31];
        db[col] = t;
    }
}

// Wt[j][o] = W[o][j]: the dCat product reads the layer weight with d_out as the contraction index.
template <typename T>
__global__ void transpose_kernel(const T *__restrict__ W, int rows, int cols, T *__restrict__ Wt)
{
    __shared__ T tile[32][33];
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    for (int i = threadIdx.y; i < 32; i += blockDim.y)
        if (r0 + i < rows && c0 + threadIdx.x < cols) tile[i][threadIdx.x] = W[(int64_t)(r0 + i) * cols + c0 + threadIdx.x];
    __syncthreads();
    for (int i = threadIdx.y; i < 32; i += blockDim.y)
        if (c0 + i < cols && r0 + threadIdx.x < rows) Wt[(int64_t)(c0 + i) * rows + r0 + threadIdx.x] = tile[threadIdx.x][i];
}

// masked copy of the gradient of a dense layer input: out = acc where mask > 0 (no mask: plain store)
template <typename T>
struct EpiMasked {
    T *out; int64_t ldo; const T *mask; int64_t ld_mask;
    __device__ void operator()(int64_t m, int n, float v, int) const {
        if (mask && !(to_float<T>(mask[m * ld_mask + n]) > 0.f)) v = 0.f;
        out[m * ldo + n] = from_float<T>(v);
    }
};

}  // namespace e2egrec
