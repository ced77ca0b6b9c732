// Exclusive prefix sums of int32 counts whose length lives on the device.
// out[i] = sum of in[0..i), for i = 0..n (n+1 values; out[n] is the total).
#pragma once

#include "common.cuh"

namespace e2egrec {

constexpr int kScanThreads = 256;
constexpr int kScanItems = 8;
constexpr int kScanTile = kScanThreads * kScanItems;

// Scratch ints needed to scan up to `cap` values.
inline size_t scan_scratch_ints(int64_t cap) { return (size_t)ceil_div(cap > 0 ? cap : 1, kScanTile) + 2; }

template <typename AccT>
__device__ inline AccT warp_inclusive_scan(AccT v)
{
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        AccT t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Exclusive scan across the block of one value per thread; returns the exclusive prefix,
// `total` receives the block sum.  smem must hold THREADS/32 values.
template <int THREADS, typename AccT>
__device__ inline AccT block_exclusive_scan(AccT v, AccT &total, AccT *smem)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    AccT inc = warp_inclusive_scan(v);
    if (lane == 31) smem[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        AccT w = lane < THREADS / 32 ? smem[lane] : AccT(0);
        AccT wi = warp_inclusive_scan(w);
        if (lane < THREADS / 32) smem[lane] = wi - w;
        if (lane == THREADS / 32 - 1) smem[THREADS / 32] = wi;
    }
    __syncthreads();
    AccT res = smem[warp] + inc - v;
    total = smem[THREADS / 32];
    __syncthreads();
    return res;
}

__device__ inline int64_t scan_len(const int32_t *n_dev, int64_t n_host, int64_t cap)
{
    int64_t n = n_dev ? (int64_t)*n_dev : n_host;
    if (n < 0) n = 0;
    return n > cap ? cap : n;
}

template <typename OutT>
__global__ void __launch_bounds__(kScanThreads)
scan_reduce_kernel(const int32_t *__restrict__ in, const int32_t *n_dev, int64_t n_host, int64_t cap,
                   OutT *__restrict__ partials)
{
    __shared__ OutT sm[kScanThreads / 32 + 1];
    const int64_t n = scan_len(n_dev, n_host, cap);
    const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
    OutT s = 0;
#pragma unroll
    for (int k = 0; k < kScanItems; ++k)
        if (base + k < n) s += in[base + k];
    OutT total;
    block_exclusive_scan<kScanThreads, OutT>(s, total, sm);
    if (threadIdx.x == 0) partials[blockIdx.x] = total;
}

// Single block: in-place exclusive scan of partials[0..nb), total to partials[nb].
template <typename OutT>
__global__ void __launch_bounds__(1024)
scan_partials_kernel(OutT *partials, int nb)
{
    __shared__ OutT sm[1024 / 32 + 1];
    OutT carry = 0;
    for (int base = 0; base < nb; base += 1024) {
        int i = base + threadIdx.x;
        OutT v = i < nb ? partials[i] : OutT(0);
        OutT total;
        OutT ex = block_exclusive_scan<1024, OutT>(v, total, sm);
        if (i < nb) partials[i] = carry + ex;
        carry += total;
    }
    if (threadIdx.x == 0) partials[nb] = carry;
}

template <typename OutT>
__global__ void __launch_bounds__(kScanThreads)
scan_final_kernel(const int32_t *__restrict__ in, OutT *__restrict__ out, const int32_t *n_dev, int64_t n_host,
                  int64_t cap, const OutT *__restrict__ partials, int nb)
{
    __shared__ OutT sm[kScanThreads / 32 + 1];
    const int64_t n = scan_len(n_dev, n_host, cap);
    const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
    int32_t v[kScanItems];
    OutT s = 0;
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
        v[k] = base + k < n ? in[base + k] : 0;
        s += v[k];
    }
    OutT total;
    OutT ex = block_exclusive_scan<kScanThreads, OutT>(s, total, sm) + partials[blockIdx.x];
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
        if (base + k < n) out[base + k] = ex;
        ex += v[k];
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) out[n] = partials[nb];
}

// Host launcher.  `scratch` holds scan_scratch_ints(cap) values of OutT.
template <typename OutT>
inline void exclusive_scan(const int32_t *in, OutT *out, const int32_t *n_dev, int64_t n_host, int64_t cap,
                           OutT *scratch, cudaStream_t st)
{
    const int nb = (int)ceil_div(cap > 0 ? cap : 1, kScanTile);
    note_launch(); note_launch(); note_launch();
    scan_reduce_kernel<OutT><<<nb, kScanThreads, 0, st>>>(in, n_dev, n_host, cap, scratch);
    scan_partials_kernel<OutT><<<1, 1024, 0, st>>>(scratch, nb);
    scan_final_kernel<OutT><<<nb, kScanThreads, 0, st>>>(in, out, n_dev, n_host, cap, scratch, nb);
}

}  // namespace e2egrec
