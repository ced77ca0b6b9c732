// Row-gather reductions: the neighbourhood mean (Eq. 2) over a sampled block, and the types
// shared with the general "segment s = sum of gathered rows" kernels (segreduce.cuh) used by the
// transposed aggregation (gather over the block's CSC) and by whole-graph aggregation with hub rows.
//
// A row of d values is d*sizeof(T)/16 chunks of 16 bytes.  LPR lanes (a power of two) own
// one row at a time, lane c of the group holding chunks c, c+LPR, ... (CPL of them), so a
// warp works on 32/LPR gathered rows at once and every lane issues several independent
// 16-byte loads before it adds anything.  Sums are fp32; nothing uses floating-point atomics.
#pragma once

#include "common.cuh"

namespace e2egrec {

constexpr int kAggThreads = 256;

// ---------------------------------------------------------------------------------------
// Sampled-block mean aggregation, one warp per destination (|S(i)| <= 128).
// Writes cat[i] = [ self row | mean row ] (2d values) for i < n_dst and zero rows up to
// the next multiple of 128 (the dense transform reads whole 128-row tiles).
// ---------------------------------------------------------------------------------------
template <typename T, int LPR, int CPL>
__global__ void __launch_bounds__(kAggThreads, CPL == 1 ? 4 : 1)
sage_aggregate_kernel(const T *__restrict__ Hsrc, int64_t ld, const int32_t *__restrict__ nbr,
                      const int32_t *__restrict__ self_ids, const int32_t *__restrict__ indptr,
                      const int32_t *__restrict__ counts, T *__restrict__ cat, int d, int32_t cap_dst)
{
    constexpr int E = Chunk<T>::kElems;
    constexpr int G = 32 / LPR;
    constexpr int U = CPL >= 4 ? 1 : 4 / CPL;
    const int lane = threadIdx.x & 31;
    const int g = lane / LPR, c = lane % LPR;
    const int n_chunks = d / E;
    pdl_launch_dependents();
    pdl_wait();                                    // the kernel before this one in the stream has completed
    const int32_t n_dst = counts[CNT_DST];
    int64_t pad_end = ((int64_t)n_dst + 127) / 128 * 128;
    if (pad_end > cap_dst) pad_end = cap_dst;
    // The grid is sized for the machine, not for the capacity: every warp walks over destinations
    // i, i + warps, ... and fetches the offsets, the first 32 neighbour ids and the self id of its next
    // destination before it sums the current one.
    const int64_t warps = (int64_t)gridDim.x * (kAggThreads / 32);
    int64_t i = ((int64_t)blockIdx.x * kAggThreads + threadIdx.x) >> 5;
    int32_t beg = 0, end = 0, mine = 0;
    int64_t self_row = 0;
    auto fetch = [&](int64_t ii, int32_t &b, int32_t &e, int32_t &m, int64_t &sr) {
        b = e = m = 0;
        sr = ii;
        if (ii < n_dst) {
            b = indptr[ii];
            e = indptr[ii + 1];
            if (lane < e - b) m = nbr[b + lane];
            if (self_ids) sr = (int64_t)self_ids[ii];
        }
    };
    fetch(i, beg, end, mine, self_row);
    while (i < pad_end) {
        const int64_t i_next = i + warps;
        int32_t beg_n, end_n, mine_n;
        int64_t self_n;
        fetch(i_next, beg_n, end_n, mine_n, self_n);
        T *out = cat + i * 2 * d;
        if (i >= n_dst) {
            float z[E];
#pragma unroll
            for (int k = 0; k < E; ++k) z[k] = 0.f;
            for (int q = lane; q < 2 * n_chunks; q += 32) Chunk<T>::store(out + q * E, z);
        } else {
            // self half: plain 16-byte copies
            for (int q = lane; q < n_chunks; q += 32)
                *reinterpret_cast<uint4 *>(out + q * E) = __ldg(reinterpret_cast<const uint4 *>(Hsrc + self_row * ld + q * E));

            float acc[CPL][E];
#pragma unroll
            for (int q = 0; q < CPL; ++q)
#pragma unroll
                for (int k = 0; k < E; ++k) acc[q][k] = 0.f;

            for (int32_t base = beg; base < end; base += 32) {
                const int m = min(32, end - base);
                if (base != beg) mine = lane < m ? nbr[base + lane] : 0;
                for (int t = 0; t * G < m; t += U) {
                    uint4 v[U][CPL];                      // raw 16-byte chunks; unpacked when they are added
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int j = (t + u) * G + g;
                        const int32_t id = __shfl_sync(0xffffffffu, mine, j & 31);
                        const T *row = Hsrc + (int64_t)id * ld;
#pragma unroll
                        for (int q = 0; q < CPL; ++q) {
                            const int ch = c + q * LPR;
                            v[u][q] = make_uint4(0, 0, 0, 0);     // zero bits are 0.0 in both types
                            if (j < m && ch < n_chunks) v[u][q] = Chunk<T>::load_raw(row + ch * E);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u)
#pragma unroll
                        for (int q = 0; q < CPL; ++q) {
                            float x[E];
                            Chunk<T>::unpack(v[u][q], x);
#pragma unroll
                            for (int k = 0; k < E; k += 2) add2(acc[q][k], acc[q][k + 1], x[k], x[k + 1]);
                        }
                }
            }
#pragma unroll
            for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
                for (int q = 0; q < CPL; ++q)
#pragma unroll
                    for (int k = 0; k < E; ++k) acc[q][k] += __shfl_xor_sync(0xffffffffu, acc[q][k], off);
            if (g == 0) {
                const int32_t cnt = end - beg;
                const float inv = cnt > 0 ? 1.0f / (float)cnt : 0.0f;
#pragma unroll
                for (int q = 0; q < CPL; ++q) {
                    const int ch = c + q * LPR;
                    if (ch < n_chunks) {
#pragma unroll
                        for (int k = 0; k < E; ++k) acc[q][k] *= inv;
                        Chunk<T>::store(out + d + ch * E, acc[q]);
                    }
                }
            }
        }
        i = i_next;
        beg = beg_n;
        end = end_n;
        mine = mine_n;
        self_row = self_n;
    }
}

// ---------------------------------------------------------------------------------------
// General segment reduction   out[s] = fin( sum_{k in [ptr[s], ptr[s+1])} w[idx[k]] * in[idx[k]] )
// with  fin(x) = mask_s * ( x * (mean ? 1/len : 1) + self[s] ); the kernels are in segreduce.cuh.
// ---------------------------------------------------------------------------------------
template <typename T>
struct SegOut {
    T *out;                 // [n_seg x d], leading dimension ld_out
    int64_t ld_out;
    const T *self;          // optional rows added for s < *n_self
    int64_t ld_self;
    const int32_t *n_self;
    const T *mask;          // optional: result is zeroed where mask[s][k] <= 0 (ReLU derivative)
    int64_t ld_mask;
    int mean;               // divide the sum by the segment length
    const float *seg_scale; // optional: multiply the sum of segment s by seg_scale[s] (not together with mean)
    int64_t pad_rows;       // if > 0: rows n_seg .. min(next multiple of 128, pad_rows) - 1 of out are zeroed
    // Several right-hand sides in one call (same segments and indices, different rows): right-hand side r reads
    // in + r * rhs_in and self + r * rhs_self and writes out + r * rhs_out (element strides); the mask is shared.
    int n_rhs;              // 0 or 1: one
    int64_t rhs_in, rhs_self, rhs_out;
    // For the form that streams the gathered rows through shared memory (seg_run_block_kernel<..., kStream>): the rows
    // that `in` holds over all right-hand sides (0: unknown, the form is not used) and the device status word that
    // receives E2EGREC_DEV_TIMEOUT when a bounded wait for the rows runs out.
    int64_t in_rows;
    int32_t *status;
};

template <typename T>
__device__ inline float seg_finish_value(const SegOut<T> &o, int64_t s, int64_t len, int k, float sum, bool has_self)
{
    float v = o.mean ? (len > 0 ? sum * (1.0f / (float)len) : 0.f) : (o.seg_scale ? sum * o.seg_scale[s] : sum);
    if (has_self) v += to_float<T>(o.self[s * o.ld_self + k]);
    v = to_float<T>(from_float<T>(v));                      // storage rounding before the mask
    if (o.mask && !(to_float<T>(o.mask[s * o.ld_mask + k]) > 0.f)) v = 0.f;
    return v;
}

template <typename PtrT>
__device__ inline int64_t seg_containing(const PtrT *__restrict__ ptr, int64_t n_seg, int64_t k)
{
    // largest s in [0, n_seg) with ptr[s] <= k   (k < ptr[n_seg])
    int64_t lo = 0, hi = n_seg;
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if ((int64_t)ptr[mid] <= k) lo = mid; else hi = mid;
    }
    return lo;
}

// Host side --------------------------------------------------------------------------------

struct RowShape { int lpr, cpl; };

inline RowShape row_shape_bytes(int64_t row_bytes)
{
    const int chunks = (int)(row_bytes / 16);
    int lpr = 4;
    while (lpr < 32 && lpr < chunks) lpr <<= 1;
    int cpl = 1;
    while (lpr * cpl < chunks) cpl <<= 1;
    return {lpr, cpl};
}

inline RowShape row_shape(int d, int32_t dtype) { return row_shape_bytes((int64_t)d * (int64_t)dtype_size(dtype)); }

}  // namespace e2egrec
