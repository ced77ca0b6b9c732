// Segment reduction by gathered rows, two kernels, no atomics, fixed summation order:
//
//     out[s] = fin( sum_{k in [ptr[s], ptr[s+1])} w[idx[k]] * in[idx[k]] ),   fin as in SegOut.
//
// This is the transposed aggregation of the backward pass (segments = columns of the block CSC)
// and the whole-graph aggregation in either direction (segments = CSR rows or CSC columns).
//
// seg_run_kernel.  The entry stream is cut into runs of `run_len` consecutive entries and every group of
//   LPR lanes owns one run.  The group streams through its run with several row loads in flight and closes
//   a segment whenever the running entry index reaches the segment's end, so thousands of one-entry
//   segments and one segment of millions of entries cost the same per entry.  A segment that lies inside
//   the run is finished there.  Otherwise its part stays in shared memory: head[run] (segment began in an
//   earlier run) or tail[run] (segment began here and continues).  The optional self row of a segment is
//   added where the segment begins, so partial sums already contain it.
//   After a block barrier the runs of the block (its "window") are joined: the group whose run holds the
//   end of a cut segment adds tail[first] + head[first+1] + ... + head[last] in run order and writes the
//   result; a segment that also leaves the window leaves one row in head2[window] or tail2[window].
// seg_final_kernel.  Adds tail2[first] + head2[first+1..last] for every segment cut by window boundaries
//   (all threads of a block share one such sum), and extra blocks write fin(0) for segments without entries.
#pragma once

#include <stdlib.h>

#include <algorithm>

#include <type_traits>

#include "aggregate.cuh"
#include "tensor_map.cuh"

namespace e2egrec {


// runs per window = lane groups per block of seg_run_kernel
inline int seg_runs_per_window(int d, size_t elem_size) { return kAggThreads / row_shape_bytes((int64_t)d * elem_size).lpr; }

struct SegScratch {
    float *head2, *tail2;          // [n_windows x d]
    int4 *win_info;                // {segment whose sum continues from an earlier window or -1, it ends here, segment
                                   //  that continues into the next window or -1, 0}
    int64_t cap_runs, n_windows;
    int runs_per_window;
    size_t bytes;
    // One counter per window, for callers of the sampled-block form: nullptr (the default) keeps the two-kernel form.
    // The caller sets it to n_windows zeroed int32 (seg_chain_bytes) before the first launch that uses them; every
    // launch leaves them zero again.
    int32_t *chain_cnt;
};

inline size_t seg_chain_bytes(int64_t cap_entries, int run_len, int d, size_t elem_size, int n_rhs = 1)
{
    const int64_t runs = ceil_div(cap_entries > 0 ? cap_entries : 1, run_len);
    return align_up((size_t)n_rhs * ceil_div(runs, seg_runs_per_window(d, elem_size)) * sizeof(int32_t), 256);
}

// n_rhs right-hand sides (SegOut::n_rhs) keep their partial rows side by side: every array holds n_rhs blocks of
// n_windows entries.
inline SegScratch seg_scratch_carve(int64_t cap_entries, int run_len, int d, size_t elem_size, void *base, int n_rhs = 1)
{
    SegScratch s{};
    s.runs_per_window = seg_runs_per_window(d, elem_size);
    s.cap_runs = ceil_div(cap_entries > 0 ? cap_entries : 1, run_len);
    s.n_windows = ceil_div(s.cap_runs, s.runs_per_window);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        char *p = base ? static_cast<char *>(base) + off : nullptr;
        off += align_up(bytes, 256);
        return p;
    };
    s.head2 = (float *)take((size_t)n_rhs * s.n_windows * d * sizeof(float));
    s.tail2 = (float *)take((size_t)n_rhs * s.n_windows * d * sizeof(float));
    s.win_info = (int4 *)take((size_t)n_rhs * s.n_windows * sizeof(int4));
    s.bytes = off;
    return s;
}

// ------------------------------------------------------------------------------------ helpers
// (sum [* 1/len]) rounded to the storage type; the self row is already part of `sum` (level 1 adds it
// where the segment begins), the mask is applied by the caller.
template <typename T>
__device__ inline float seg_round(const SegOut<T> &o, float inv_len, float sum)
{
    const float v = (o.mean || o.seg_scale) ? sum * inv_len : sum;
    return to_float<T>(from_float<T>(v));
}

template <typename T> __device__ inline float4 load4(const T *p);
template <> __device__ inline float4 load4<float>(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }
template <> __device__ inline float4 load4<__nv_bfloat16>(const __nv_bfloat16 *p)
{
    const uint2 r = __ldg(reinterpret_cast<const uint2 *>(p));
    return make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xFFFF0000u), __uint_as_float(r.y << 16),
                       __uint_as_float(r.y & 0xFFFF0000u));
}

template <typename T> __device__ inline void store4(T *p, const float (&v)[4]);
template <> __device__ inline void store4<float>(float *p, const float (&v)[4])
{
    *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
template <> __device__ inline void store4<__nv_bfloat16>(__nv_bfloat16 *p, const float (&v)[4])
{
    __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
    *reinterpret_cast<uint2 *>(p) = make_uint2(*reinterpret_cast<uint32_t *>(&a), *reinterpret_cast<uint32_t *>(&b));
}

// ------------------------------------------------------------------------------------ runs and windows
// Advances the walk from segment s to the segment that holds entry k (k >= end of segment s): a few steps one
// by one, then by bisection if a long stretch of empty segments is in the way.  Returns {segment, its end}; kept
// out of line (the streaming loop stays short) and by value (nothing of the caller is forced into memory).
struct SegStep { int64_t seg, end; };
template <typename PtrT>
__device__ __noinline__ SegStep seg_advance(const PtrT *__restrict__ ptr, int64_t n_seg, int64_t k, int64_t s)
{
    int64_t end;
    int step = 0;
    do { ++s; end = (int64_t)ptr[s + 1]; } while (end <= k && ++step < 4);
    if (end <= k) {
        s = seg_containing(ptr, n_seg, k);
        end = (int64_t)ptr[s + 1];
    }
    return SegStep{s, end};
}

// Finishes segment `seg` whose entries (and self row) sum to acc: scale, round to the storage type, mask, store.
template <typename T, int LPR, int CPL, int kExtra>
__device__ __forceinline__ void seg_store_row(const SegOut<T> &o, int32_t seg, float inv, const float (&acc)[CPL][Chunk<T>::kElems],
                                              const uint4 (&mrow)[CPL], int c, int n_chunks)
{
    constexpr int E = Chunk<T>::kElems;
#pragma unroll
    for (int q = 0; q < CPL; ++q) {
        const int ch = c + q * LPR;
        if (ch < n_chunks) {
            // the store rounds to the storage type, once; a masked element is zero before and after that rounding alike
            float r[E];
#pragma unroll
            for (int e = 0; e < E; ++e) r[e] = acc[q][e] * inv;                                 // inv = 1 without mean / scale
            if (kExtra == 2 && o.mask) {
                float m[E];
                Chunk<T>::unpack(mrow[q], m);
#pragma unroll
                for (int e = 0; e < E; ++e)
                    if (!(m[e] > 0.f)) r[e] = 0.f;
            }
            Chunk<T>::store(o.out + (int64_t)seg * o.ld_out + ch * E, r);
        }
    }
}

// A lane group has just written its window's part (a row of head2 or tail2) of segment sg, which is cut by window
// boundaries.  The parts of a segment are counted in chain_cnt[its first window]; the group that brings the count to
// the number of windows the segment spans adds the parts in window order -- tail2[first], head2[first + 1], ... -- and
// stores the finished row, so the sum does not depend on which group closes it.  No group waits for another.
template <typename T, int LPR, int kExtra>
__device__ __forceinline__ void seg_chain_arrive(int32_t sg, const int32_t *__restrict__ ptr, int run_len, int d, int c, int n_chunks,
                                                 const float *head2, const float *tail2, int32_t *chain_cnt, const SegOut<T> &o)
{
    constexpr int E = Chunk<T>::kElems;
    constexpr int RB = kAggThreads / LPR;
    const int32_t beg = ptr[sg], end = ptr[sg + 1];
    const int32_t first = (beg / run_len) / RB, last = ((end - 1) / run_len) / RB;
    const int group_lane0 = (threadIdx.x & 31) / LPR * LPR;
    const unsigned gmask = LPR >= 32 ? 0xffffffffu : (((1u << (LPR & 31)) - 1u) << group_lane0);
    __threadfence();                               // this lane's share of the part is visible before the count moves
    __syncwarp(gmask);
    int32_t old = 0;
    if (c == 0) old = atomicAdd(&chain_cnt[first], 1);
    old = __shfl_sync(gmask, old, group_lane0);
    if (old != last - first) return;               // other windows' parts are still to come: their group will close it
    if (c == 0) chain_cnt[first] = 0;              // idle again for the next launch
    __threadfence();
    float acc[1][E];
    uint4 mrow[1] = {make_uint4(0, 0, 0, 0)};
#pragma unroll
    for (int e = 0; e < E; ++e) acc[0][e] = 0.f;
    if (c < n_chunks) {
        const float *t = tail2 + (int64_t)first * d + c * E;
#pragma unroll
        for (int e = 0; e < E; e += 4) {
            const float4 x = __ldcg(reinterpret_cast<const float4 *>(t + e));
            acc[0][e] = x.x; acc[0][e + 1] = x.y; acc[0][e + 2] = x.z; acc[0][e + 3] = x.w;
        }
        for (int32_t p0 = first + 1; p0 <= last; p0 += 4) {
            float4 x[4][E / 4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int e = 0; e < E / 4; ++e)
                    x[u][e] = p0 + u <= last ? __ldcg(reinterpret_cast<const float4 *>(head2 + (int64_t)(p0 + u) * d + c * E + 4 * e))
                                             : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int e = 0; e < E / 4; ++e) {
                    acc[0][4 * e] += x[u][e].x; acc[0][4 * e + 1] += x[u][e].y;
                    acc[0][4 * e + 2] += x[u][e].z; acc[0][4 * e + 3] += x[u][e].w;
                }
        }
        if (kExtra == 2 && o.mask) mrow[0] = Chunk<T>::load_raw(o.mask + (int64_t)sg * o.ld_mask + c * E);
    }
    seg_store_row<T, LPR, 1, kExtra>(o, sg, 1.0f, acc, mrow, c, n_chunks);
}

// Second half of a run kernel: every lane group has left the parts of the segments that its run cuts in sh_head /
// sh_tail (head_seg / head_ends / tail_seg say which); after a block barrier the runs of the block (its window) are
// joined.  The group of run rl acts where a chain of parts of one cut segment ends: at the run that holds the
// segment's end, or at the window's last run.  It walks back to the run in which the segment began (if that run is in
// the window) and adds the parts forward, in run order.  A segment that also leaves the window leaves one row in
// head2[window] or tail2[window] and a record in win_info[window].  Called by all threads of the block.
// With chain_cnt (sampled-block form, CPL = 1, no mean / scale) nothing is left for a second kernel: a group that has
// written a window's part of a cut segment counts it in chain_cnt[first window of the segment]; the group whose part
// completes the count adds all parts of the segment in window order and stores the row (seg_chain_arrive).
template <typename T, typename PtrT, int LPR, int CPL, int kExtra>
__device__ __forceinline__ void seg_join_window(float *sh_head, float *sh_tail, int4 *sh_info, int32_t *sh_win, int rl, int c,
                                                int n_chunks, int d, int32_t head_seg, int32_t head_ends, int32_t tail_seg,
                                                const PtrT *__restrict__ ptr, float *__restrict__ head2, float *__restrict__ tail2,
                                                int4 *__restrict__ win_info, const SegOut<T> &o, int32_t *chain_cnt = nullptr,
                                                int run_len = 0)
{
    constexpr int E = Chunk<T>::kElems;
    constexpr int RB = kAggThreads / LPR;
    constexpr int ROW = LPR * CPL * E;
    if (c == 0) sh_info[rl] = make_int4(head_seg, head_ends, tail_seg, 0);
    if (threadIdx.x < 4) sh_win[threadIdx.x] = threadIdx.x == 1 || threadIdx.x == 3 ? 0 : -1;
    __syncthreads();

    // ---- join the runs of the window.  The group of run rl acts where a chain of parts of one cut segment
    // ends: at the run that holds the segment's end, or at the window's last run.  It walks back to the run in
    // which the segment began (if that run is in the window) and adds the parts forward, in run order.
    {
        const bool last_run = rl == RB - 1;
        if (head_seg >= 0 && (head_ends || last_run)) {
            int first = rl - 1;                    // the run whose tail begins the chain, or -1: began before the window
            while (first >= 0 && sh_info[first].z != head_seg) --first;
            float acc[CPL][E];
            uint4 mrow[CPL];
#pragma unroll
            for (int q = 0; q < CPL; ++q) {
                const int ch = c + q * LPR;
                mrow[q] = make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int e = 0; e < E; ++e) acc[q][e] = 0.f;
                if (first >= 0) {
#pragma unroll
                    for (int e = 0; e < E; ++e) acc[q][e] = sh_tail[first * ROW + ch * E + e];
                }
                for (int j = first + 1; j <= rl; ++j) {
#pragma unroll
                    for (int e = 0; e < E; ++e) acc[q][e] += sh_head[j * ROW + ch * E + e];
                }
            }
            if (first >= 0 && head_ends) {
                const int64_t sg = head_seg;
                float inv = 1.0f;
                if (o.mean) inv = 1.0f / (float)((int64_t)ptr[sg + 1] - (int64_t)ptr[sg]);
                else if (o.seg_scale) inv = o.seg_scale[sg];
                if (kExtra == 2 && o.mask) {
#pragma unroll
                    for (int q = 0; q < CPL; ++q) {
                        const int ch = c + q * LPR;
                        if (ch < n_chunks) mrow[q] = Chunk<T>::load_raw(o.mask + sg * o.ld_mask + ch * E);
                    }
                }
                seg_store_row<T, LPR, CPL, kExtra>(o, head_seg, inv, acc, mrow, c, n_chunks);
            } else {
                // leaves the window: towards earlier windows (head2) or, begun here and still open, later ones (tail2)
                float *dst = (first >= 0 ? tail2 : head2) + (int64_t)blockIdx.x * d;
#pragma unroll
                for (int q = 0; q < CPL; ++q) {
                    const int ch = c + q * LPR;
                    if (ch < n_chunks) {
#pragma unroll
                        for (int e = 0; e < E; e += 4)
                            *reinterpret_cast<float4 *>(dst + ch * E + e) = make_float4(acc[q][e], acc[q][e + 1], acc[q][e + 2], acc[q][e + 3]);
                    }
                }
                if (c == 0) {
                    if (first >= 0) sh_win[2] = head_seg;
                    else { sh_win[0] = head_seg; sh_win[1] = head_ends; }
                }
                if constexpr (CPL == 1 && sizeof(PtrT) == 4)
                    if (chain_cnt) seg_chain_arrive<T, LPR, kExtra>(head_seg, ptr, run_len, d, c, n_chunks, head2, tail2, chain_cnt, o);
            }
        }
        if (last_run && tail_seg >= 0) {           // a segment that begins in the window's last run and continues
            float *dst = tail2 + (int64_t)blockIdx.x * d;
#pragma unroll
            for (int q = 0; q < CPL; ++q) {
                const int ch = c + q * LPR;
                if (ch < n_chunks) {
#pragma unroll
                    for (int e = 0; e < E; e += 4)
                        *reinterpret_cast<float4 *>(dst + ch * E + e) = *reinterpret_cast<const float4 *>(sh_tail + rl * ROW + ch * E + e);
                }
            }
            if (c == 0) sh_win[2] = tail_seg;
            if constexpr (CPL == 1 && sizeof(PtrT) == 4)
                if (chain_cnt) seg_chain_arrive<T, LPR, kExtra>(tail_seg, ptr, run_len, d, c, n_chunks, head2, tail2, chain_cnt, o);
        }
    }
    if (chain_cnt) return;                        // no record: nobody reads it
    __syncthreads();
    if (threadIdx.x == 0) win_info[blockIdx.x] = make_int4(sh_win[0], sh_win[1], sh_win[2], 0);
}

// Shared memory of seg_run_kernel (dynamic): head and tail rows of the block's runs, fp32, one row of
// LPR*CPL*E floats per run, then one record per run.
template <int LPR, int CPL, int E>
constexpr size_t seg_run_smem_bytes()
{
    return (size_t)2 * (kAggThreads / LPR) * (LPR * CPL * E) * sizeof(float) + (size_t)(kAggThreads / LPR) * sizeof(int4);
}

// kExtra: 1 = the output has a self row per segment, 2 = a self row and / or a mask row (they are fetched together
// with the segment's first gathered row); 0 = neither, and those registers and branches disappear.
// kInFlight: gathered rows a lane group requests before it adds any.  Four suit the short streams of a sampled
// block (few resident warps, latency hidden inside the thread); on streams that fill the machine two are faster,
// because the smaller register footprint keeps five blocks resident per SM instead of three.
template <typename T, typename PtrT, int LPR, int CPL, bool kWeight, int kExtra, int kInFlight>
__global__ void __launch_bounds__(kAggThreads, (kInFlight <= 2 && !kExtra) ? 5 : 1)
seg_run_kernel(const T *__restrict__ in, int64_t ld_in, const PtrT *__restrict__ ptr, const int32_t *__restrict__ idx,
               const int32_t *n_seg_dev, int64_t n_seg_host, const float *__restrict__ w, int run_len, int d,
               float *__restrict__ head2, float *__restrict__ tail2, int4 *__restrict__ win_info, int64_t cap_runs,
               const int32_t *__restrict__ seg_of, SegOut<T> o)
{
    constexpr int E = Chunk<T>::kElems;
    constexpr int U = CPL >= kInFlight ? 1 : kInFlight / CPL;
    constexpr int RB = kAggThreads / LPR;          // runs of this block = one window
    constexpr int ROW = LPR * CPL * E;             // floats per shared row (>= d)
    constexpr int kFar = 1 << 30;
    extern __shared__ float4 seg_smem[];
    float *sh_head = reinterpret_cast<float *>(seg_smem);
    float *sh_tail = sh_head + RB * ROW;
    int4 *sh_info = reinterpret_cast<int4 *>(sh_tail + RB * ROW);
    __shared__ int32_t sh_win[4];

    const int c = threadIdx.x % LPR;
    const int rl = threadIdx.x / LPR;              // run within the block
    const int n_chunks = d / E;
    const int64_t run = (int64_t)blockIdx.x * RB + rl;
    pdl_launch_dependents();
    pdl_wait();                                    // the kernel before this one in the stream has completed
    const int64_t n_seg = n_seg_dev ? (int64_t)*n_seg_dev : n_seg_host;
    const int64_t total = n_seg > 0 ? (int64_t)ptr[n_seg] : 0;
    const int64_t k0 = run * run_len;
    // a window that lies wholly beyond the stream (grids are sized for capacities) has nothing to do, not even a
    // record: seg_final_kernel only looks at the windows that hold entries
    if ((int64_t)blockIdx.x * RB * run_len >= total) return;
    int32_t head_seg = -1, head_ends = 0, tail_seg = -1;

    // finishes segment `seg` whose entries sum to acc: scale, round to the storage type, mask, store
    auto finish = [&](int32_t seg, float inv, const float (&acc)[CPL][E], const uint4 (&mrow)[CPL]) {
#pragma unroll
        for (int q = 0; q < CPL; ++q) {
            const int ch = c + q * LPR;
            if (ch < n_chunks) {
                float r[E];
#pragma unroll
                for (int e = 0; e < E; ++e) r[e] = to_float<T>(from_float<T>(acc[q][e] * inv));   // inv = 1 without mean / scale
                if (kExtra == 2 && o.mask) {
                    float m[E];
                    Chunk<T>::unpack(mrow[q], m);
#pragma unroll
                    for (int e = 0; e < E; ++e)
                        if (!(m[e] > 0.f)) r[e] = 0.f;
                }
                Chunk<T>::store(o.out + (int64_t)seg * o.ld_out + ch * E, r);
            }
        }
    };

    if (run < cap_runs && k0 < total) {
        const int len = (int)min((int64_t)run_len, total - k0);   // entries of this run; positions below are relative to k0
        const int32_t *__restrict__ idx0 = idx + k0;
        const int32_t *__restrict__ seg0 = seg_of ? seg_of + k0 : nullptr;
        const int64_t n_self = (kExtra && o.self) ? (o.n_self ? (int64_t)*o.n_self : n_seg) : 0;

        // Segment boundaries are found one iteration ahead of the sums.  With an entry -> segment array a
        // boundary is a change of that value; without it the offsets are walked.
        int64_t ws;                    // segment of the entry classified last
        int rel_end = kFar;            // its end (walk mode)
        int first_beg_rel = 0;         // where the run's first segment begins (<= 0)
        bool first_begins, last_ends = false;
        if (seg0) {
            ws = seg0[0];
            first_begins = k0 == 0 || seg0[-1] != (int32_t)ws;
            last_ends = k0 + len == total || seg0[len] != seg0[len - 1];
            if (o.mean) first_beg_rel = (int)max((int64_t)ptr[ws] - k0, (int64_t)-kFar);
        } else {
            ws = seg_containing(ptr, n_seg, k0);
            const int64_t wb = (int64_t)ptr[ws] - k0;
            first_begins = wb >= 0;
            first_beg_rel = (int)max(wb, (int64_t)-kFar);
            rel_end = (int)min((int64_t)ptr[ws + 1] - k0, (int64_t)kFar);
        }

        int32_t seg_n[U], id_n[U];
        bool start_n[U];
        auto classify = [&](int r0) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int r = r0 + u;
                start_n[u] = false;
                seg_n[u] = 0;
                id_n[u] = 0;
                if (r < len) {
                    if (seg0) {
                        const int32_t sg = seg0[r];
                        start_n[u] = r == 0 || sg != (int32_t)ws;
                        ws = sg;
                    } else if (r == 0) {
                        start_n[u] = true;
                    } else if (r >= rel_end) {
                        const SegStep nx = seg_advance(ptr, n_seg, k0 + r, ws);
                        ws = nx.seg;
                        rel_end = (int)min(nx.end - k0, (int64_t)kFar);
                        start_n[u] = true;
                    }
                    seg_n[u] = (int32_t)ws;
                    id_n[u] = idx0[r];
                }
            }
        };

        int32_t cur_seg = -1;
        int cur_beg_rel = 0;
        bool cur_begins = false;
        uint4 cur_mask[CPL];
        float acc[CPL][E];
#pragma unroll
        for (int q = 0; q < CPL; ++q) {
            cur_mask[q] = make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int e = 0; e < E; ++e) acc[q][e] = 0.f;
        }

        // closes the current segment, which ends at relative position end_rel, with the sum in acc
        auto emit = [&](bool ended, int end_rel) {
            if (cur_begins && ended) {
                const float inv = o.mean ? 1.0f / (float)(end_rel - cur_beg_rel) : (o.seg_scale ? o.seg_scale[cur_seg] : 1.0f);
                finish(cur_seg, inv, acc, cur_mask);
            } else {
                float *dst = (cur_begins ? sh_tail : sh_head) + rl * ROW;
#pragma unroll
                for (int q = 0; q < CPL; ++q) {
                    const int ch = c + q * LPR;
#pragma unroll
                    for (int e = 0; e < E; e += 4)
                        *reinterpret_cast<float4 *>(dst + ch * E + e) = make_float4(acc[q][e], acc[q][e + 1], acc[q][e + 2], acc[q][e + 3]);
                }
                if (cur_begins) tail_seg = cur_seg;
                else { head_seg = cur_seg; head_ends = ended ? 1 : 0; }
            }
        };

        classify(0);
        for (int r0 = 0; r0 < len; r0 += U) {
            int32_t seg_c[U];
            bool start_c[U];
            float wt[U];
            uint4 v[U][CPL], sv[kExtra ? U : 1][CPL], mv[kExtra == 2 ? U : 1][CPL];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                seg_c[u] = seg_n[u];
                start_c[u] = start_n[u];
                wt[u] = 1.f;
                const bool live = r0 + u < len;
                const int32_t id = id_n[u];
                if (kWeight && live) wt[u] = w[id];
#pragma unroll
                for (int q = 0; q < CPL; ++q) {
                    const int ch = c + q * LPR;
                    v[u][q] = make_uint4(0, 0, 0, 0);
                    if (live && ch < n_chunks) v[u][q] = Chunk<T>::load_raw(in + (int64_t)id * ld_in + ch * E);
                    if (kExtra) {
                        sv[u][q] = make_uint4(0, 0, 0, 0);
                        if (kExtra == 2) mv[u][q] = make_uint4(0, 0, 0, 0);
                        if (live && start_c[u] && ch < n_chunks) {
                            const bool begins = r0 + u != 0 || first_begins;
                            if (begins && seg_c[u] < n_self)
                                sv[u][q] = Chunk<T>::load_raw(o.self + (int64_t)seg_c[u] * o.ld_self + ch * E);
                            if (kExtra == 2 && o.mask)
                                mv[u][q] = Chunk<T>::load_raw(o.mask + (int64_t)seg_c[u] * o.ld_mask + ch * E);
                        }
                    }
                }
            }
            if (r0 + U < len) classify(r0 + U);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (r0 + u < len) {
                    if (start_c[u]) {
                        if (cur_seg >= 0) emit(true, r0 + u);
                        cur_seg = seg_c[u];
                        cur_begins = r0 + u != 0 || first_begins;
                        cur_beg_rel = r0 + u != 0 ? r0 + u : first_beg_rel;
#pragma unroll
                        for (int q = 0; q < CPL; ++q) {
                            if (kExtra) {
                                Chunk<T>::unpack(sv[u][q], acc[q]);          // the self row (zeros if there is none)
                                if (kExtra == 2) cur_mask[q] = mv[u][q];
                            } else {
#pragma unroll
                                for (int e = 0; e < E; ++e) acc[q][e] = 0.f;
                            }
                        }
                    }
#pragma unroll
                    for (int q = 0; q < CPL; ++q) {
                        float x[E];
                        Chunk<T>::unpack(v[u][q], x);
#pragma unroll
                        for (int e = 0; e < E; e += 2) {
                            if (kWeight) {
                                acc[q][e] = fmaf(wt[u], x[e], acc[q][e]);
                                acc[q][e + 1] = fmaf(wt[u], x[e + 1], acc[q][e + 1]);
                            } else {
                                add2(acc[q][e], acc[q][e + 1], x[e], x[e + 1]);
                            }
                        }
                    }
                }
            }
        }
        emit(seg0 ? last_ends : rel_end <= len, len);
    }
    seg_join_window<T, PtrT, LPR, CPL, kExtra>(sh_head, sh_tail, sh_info, sh_win, rl, c, n_chunks, d, head_seg, head_ends, tail_seg, ptr,
                                               head2, tail2, win_info, o);
}

// ------------------------------------------------------------------------------------ the sampled-block form
// seg_run_kernel for the transposed aggregation of a sampled block, where the entry -> segment array exists, offsets
// are 32-bit, a row is one 16-byte chunk per lane, entries carry no weight and the output is the plain sum plus the
// self row (kMask: zeroed where the mask row is not positive).  Same runs, same order of additions, same records for
// the join and for seg_final_kernel, hence the same bits as the general kernel; but the walk over the run is written
// for this case alone (entry ids and segment ids fetched four at a time, 32-bit arithmetic, no scale, no walk of the
// offsets), which takes the instructions per entry from ~110 to ~35: with two entries per segment on average the
// general kernel was bound by instruction issue, not by memory.
//
// kStream (bf16 rows of 512 bytes, one warp per run): the gathered rows do not pass through registers on their way in.
// Every warp hands the entry ids of its run, four at a time, to the TMA unit (tile::gather4 on `in_map`, the table `in`
// as a 2-D tensor), which lands the rows in the warp's own ring of kStreamSlots slots in shared memory; the warp adds
// them up from there in the same order.  Twice the rows in flight per warp at the same register count; the self and
// mask rows of beginning segments are still loaded directly.
constexpr int kStreamSlots = 2;
constexpr uint32_t kStreamRowBytes = 512;

template <typename T, int LPR, bool kMask, int U = 4, int kMinBlocks = (kMask ? 3 : 4), bool kStream = false>
__global__ void __launch_bounds__(kAggThreads, kMinBlocks)
seg_run_block_kernel(const __grid_constant__ CUtensorMap in_map, const T *__restrict__ in, int64_t ld_in, const int32_t *__restrict__ ptr, const int32_t *__restrict__ idx,
                     const int32_t *__restrict__ seg_of, const int32_t *__restrict__ n_seg_dev, int run_len, int d,
                     float *__restrict__ head2, float *__restrict__ tail2, int4 *__restrict__ win_info, int64_t cap_runs,
                     int32_t *__restrict__ chain_cnt, SegOut<T> o)
{
    constexpr int E = Chunk<T>::kElems;
    constexpr int RB = kAggThreads / LPR;
    constexpr int ROW = LPR * E;
    constexpr int kExtra = kMask ? 2 : 1;
    extern __shared__ float4 seg_smem[];
    float *sh_head = reinterpret_cast<float *>(seg_smem);
    float *sh_tail = sh_head + RB * ROW;
    int4 *sh_info = reinterpret_cast<int4 *>(sh_tail + RB * ROW);
    __shared__ int32_t sh_win[4];
    __shared__ uint64_t sh_bar[kStream ? RB : 1][kStreamSlots];

    const int c = threadIdx.x % LPR;
    const int rl = threadIdx.x / LPR;
    const int n_chunks = d / E;
    const int64_t run = (int64_t)blockIdx.x * RB + rl;
    // kStream: the warp's ring behind the join's rows and records, its barriers, the row offset of its right-hand side
    uint8_t *ring_w = nullptr;
    int32_t row_off = 0;
    if constexpr (kStream) {
        ring_w = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(sh_info + RB) + 127) & ~uintptr_t(127)) +
                 (size_t)rl * kStreamSlots * 4 * kStreamRowBytes;
        if (c == 0) {
            for (int s = 0; s < kStreamSlots; ++s) tm_mbar_init(&sh_bar[rl][s], 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        __syncwarp();
    }
    pdl_launch_dependents();
    pdl_wait();                                    // the kernel before this one in the stream has completed
    if (blockIdx.y) {                              // the second right-hand side: other rows, same segments
        const int64_t r = blockIdx.y, nw = gridDim.x;
        if constexpr (kStream) row_off = (int32_t)(r * (o.rhs_in / ld_in));
        in += r * o.rhs_in;
        o.self += r * o.rhs_self;
        o.out += r * o.rhs_out;
        head2 += r * nw * d;
        tail2 += r * nw * d;
        if (chain_cnt) chain_cnt += r * nw;
    }
    const int32_t n_seg = *n_seg_dev;
    const int32_t total = n_seg > 0 ? ptr[n_seg] : 0;
    const int64_t k0 = run * run_len;
    int32_t head_seg = -1, head_ends = 0, tail_seg = -1;
    // a window that lies wholly beyond the stream (grids are sized for capacities) has no run work and no join, but
    // still takes its share of the segments without entries below
    const bool live_window = (int64_t)blockIdx.x * RB * run_len < total;

    if (run < cap_runs && k0 < total) {
        const int len = (int)min((int64_t)run_len, (int64_t)total - k0);
        const int32_t *__restrict__ idx0 = idx + k0;
        const int32_t *__restrict__ seg0 = seg_of + k0;
        const int32_t n_self = o.n_self ? *o.n_self : n_seg;
        const bool lane_on = c < n_chunks;
        const T *__restrict__ in_c = in + c * E;
        const T *__restrict__ self_c = o.self + c * E;
        const T *__restrict__ mask_c = kMask ? o.mask + c * E : nullptr;
        const bool vec_ok = ((reinterpret_cast<uintptr_t>(idx0) | reinterpret_cast<uintptr_t>(seg0)) & 15u) == 0;
        const bool first_begins = k0 == 0 || seg0[-1] != seg0[0];
        const bool last_ends = k0 + len == total || seg0[len] != seg0[len - 1];

        int32_t cur_seg = -1, last_sg = -1;
        bool cur_begins = false;
        float acc[1][E];
        uint4 cur_mask[1] = {make_uint4(0, 0, 0, 0)};
#pragma unroll
        for (int e = 0; e < E; ++e) acc[0][e] = 0.f;

        // closes the current segment: a whole segment goes to the output, a part of one to the block's shared rows
        auto emit = [&](bool ended) {
            if (cur_begins && ended) {
                seg_store_row<T, LPR, 1, kExtra>(o, cur_seg, 1.0f, acc, cur_mask, c, n_chunks);
            } else {
                float *dst = (cur_begins ? sh_tail : sh_head) + rl * ROW + c * E;
#pragma unroll
                for (int e = 0; e < E; e += 4) *reinterpret_cast<float4 *>(dst + e) = make_float4(acc[0][e], acc[0][e + 1], acc[0][e + 2], acc[0][e + 3]);
                if (cur_begins) tail_seg = cur_seg;
                else { head_seg = cur_seg; head_ends = ended ? 1 : 0; }
            }
        };

        // kStream: the ids of group g (entries 4g .. 4g + 3 of the run; beyond the run's end the first id again), and the
        // hand-over of a group to the TMA unit by the warp's first lane
        bool stream_ok = true;
        auto group_ids = [&](int g) -> int4 {
            const int r = 4 * g;
            if (vec_ok && r + 4 <= len) return __ldg(reinterpret_cast<const int4 *>(idx0 + r));
            const int32_t first = __ldg(idx0 + (r < len ? r : 0));
            return make_int4(first, r + 1 < len ? __ldg(idx0 + r + 1) : first, r + 2 < len ? __ldg(idx0 + r + 2) : first,
                             r + 3 < len ? __ldg(idx0 + r + 3) : first);
        };
        auto issue_group = [&](int g, const int4 &ids) {
            if (c == 0)
                tm_gather4(ring_w + (size_t)(g % kStreamSlots) * 4 * kStreamRowBytes, &in_map, ids.x + row_off, ids.y + row_off,
                           ids.z + row_off, ids.w + row_off, &sh_bar[rl][g % kStreamSlots], kStreamRowBytes);
        };
        int n_issued = 0;
        if constexpr (kStream) {
            // Three things are in flight per warp: the rows of the next kStreamSlots groups (ring), the self / mask rows of
            // the next group's beginning segments (registers, fetched one group ahead), the segment ids two groups ahead.
            static_assert(!kStream || U == 4, "a group of the ring is four entries");
            const int n_g = (len + 3) >> 2;
            auto load_sg = [&](int g) -> int4 {
                const int r = 4 * g;
                if (vec_ok && r + 4 <= len) return __ldg(reinterpret_cast<const int4 *>(seg0 + r));
                return make_int4(r < len ? __ldg(seg0 + r) : -1, r + 1 < len ? __ldg(seg0 + r + 1) : -1,
                                 r + 2 < len ? __ldg(seg0 + r + 2) : -1, r + 3 < len ? __ldg(seg0 + r + 3) : -1);
            };
            // the entries of group g that begin a segment (bit u) and the self / mask rows of those segments
            auto load_starts = [&](int g, const int4 &sgv, int32_t prev_last, uint4 (&svv)[4], uint4 (&mvv)[kMask ? 4 : 1]) -> unsigned {
                const int32_t sgs[4] = {sgv.x, sgv.y, sgv.z, sgv.w};
                unsigned starts = 0;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int r = 4 * g + u;
                    const bool st = r < len && sgs[u] != (u == 0 ? prev_last : sgs[u - 1]);
                    svv[u] = make_uint4(0, 0, 0, 0);
                    if (kMask) mvv[u] = make_uint4(0, 0, 0, 0);
                    if (st) {
                        starts |= 1u << u;
                        if (lane_on) {
                            if ((r != 0 || first_begins) && sgs[u] < n_self) svv[u] = Chunk<T>::load_raw(self_c + (int64_t)sgs[u] * o.ld_self);
                            if (kMask) mvv[u] = Chunk<T>::load_raw(mask_c + (int64_t)sgs[u] * o.ld_mask);
                        }
                    }
                }
                return starts;
            };
            for (int g = 0; g < kStreamSlots && g < n_g; ++g, ++n_issued) issue_group(g, group_ids(g));
            int4 ids_ahead = kStreamSlots < n_g ? group_ids(kStreamSlots) : make_int4(0, 0, 0, 0);
            int4 sg_cur = load_sg(0);
            int4 sg_next = n_g > 1 ? load_sg(1) : make_int4(-1, -1, -1, -1);
            uint4 sv_cur[4], sv_next[4], mv_cur[kMask ? 4 : 1], mv_next[kMask ? 4 : 1];
            unsigned starts_cur = load_starts(0, sg_cur, -1, sv_cur, mv_cur), starts_next = 0;
            for (int g = 0; g < n_g; ++g) {
                if (g + 1 < n_g) starts_next = load_starts(g + 1, sg_next, sg_cur.w, sv_next, mv_next);
                const int4 sg_after = g + 2 < n_g ? load_sg(g + 2) : make_int4(-1, -1, -1, -1);
                const int slot = g % kStreamSlots;
                stream_ok = stream_ok && __all_sync(0xffffffffu, tm_mbar_wait(&sh_bar[rl][slot], (uint32_t)(g / kStreamSlots) & 1u));
                const uint8_t *rows = ring_w + (size_t)slot * 4 * kStreamRowBytes + c * 16;
                const int32_t sgs[4] = {sg_cur.x, sg_cur.y, sg_cur.z, sg_cur.w};
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int r = 4 * g + u;
                    if (r < len) {
                        if ((starts_cur >> u) & 1u) {
                            if (cur_seg >= 0) emit(true);
                            cur_seg = sgs[u];
                            cur_begins = r != 0 || first_begins;
                            Chunk<T>::unpack(sv_cur[u], acc[0]);             // the self row (zeros if there is none)
                            if (kMask) cur_mask[0] = mv_cur[u];
                        }
                        float x[E];
                        // (after a wait that ran out the slot holds stale rows: the launch is reported as failed)
                        Chunk<T>::unpack(*reinterpret_cast<const uint4 *>(rows + u * kStreamRowBytes), x);
#pragma unroll
                        for (int e = 0; e < E; e += 2) add2(acc[0][e], acc[0][e + 1], x[e], x[e + 1]);
                    }
                }
                __syncwarp();                                   // every lane has read the slot
                if (stream_ok && g + kStreamSlots < n_g) {
                    issue_group(g + kStreamSlots, ids_ahead);
                    n_issued = g + kStreamSlots + 1;
                    if (g + kStreamSlots + 1 < n_g) ids_ahead = group_ids(g + kStreamSlots + 1);
                }
                sg_cur = sg_next;
                sg_next = sg_after;
                starts_cur = starts_next;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    sv_cur[u] = sv_next[u];
                    if (kMask) mv_cur[u] = mv_next[u];
                }
            }
        } else
        for (int r0 = 0; r0 < len; r0 += U) {
            int32_t id[U], sg[U];
            if (vec_ok && r0 + U <= len) {
#pragma unroll
                for (int q = 0; q < U / 4; ++q) {
                    const int4 a = __ldg(reinterpret_cast<const int4 *>(idx0 + r0) + q);
                    const int4 b = __ldg(reinterpret_cast<const int4 *>(seg0 + r0) + q);
                    id[4 * q] = a.x; id[4 * q + 1] = a.y; id[4 * q + 2] = a.z; id[4 * q + 3] = a.w;
                    sg[4 * q] = b.x; sg[4 * q + 1] = b.y; sg[4 * q + 2] = b.z; sg[4 * q + 3] = b.w;
                }
            } else {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const bool live = r0 + u < len;
                    id[u] = live ? __ldg(idx0 + r0 + u) : 0;
                    sg[u] = live ? __ldg(seg0 + r0 + u) : -1;
                }
            }
            uint4 v[U], sv[U], mv[kMask ? U : 1];
            bool start[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const bool live = r0 + u < len;
                start[u] = live && sg[u] != (u == 0 ? last_sg : sg[u - 1]);      // entry 0 always starts (last_sg = -1)
                v[u] = make_uint4(0, 0, 0, 0);
                sv[u] = make_uint4(0, 0, 0, 0);
                if (kMask) mv[u] = make_uint4(0, 0, 0, 0);
                if (live && lane_on) {
                    v[u] = Chunk<T>::load_raw(in_c + (int64_t)id[u] * ld_in);
                    if (start[u]) {
                        if ((r0 + u != 0 || first_begins) && sg[u] < n_self) sv[u] = Chunk<T>::load_raw(self_c + (int64_t)sg[u] * o.ld_self);
                        if (kMask) mv[u] = Chunk<T>::load_raw(mask_c + (int64_t)sg[u] * o.ld_mask);
                    }
                }
            }
            last_sg = sg[U - 1];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (r0 + u < len) {
                    if (start[u]) {
                        if (cur_seg >= 0) emit(true);
                        cur_seg = sg[u];
                        cur_begins = r0 + u != 0 || first_begins;
                        Chunk<T>::unpack(sv[u], acc[0]);                 // the self row (zeros if there is none)
                        if (kMask) cur_mask[0] = mv[u];
                    }
                    float x[E];
                    Chunk<T>::unpack(v[u], x);
#pragma unroll
                    for (int e = 0; e < E; e += 2) add2(acc[0][e], acc[0][e + 1], x[e], x[e + 1]);
                }
            }
        }
        emit(last_ends);
        if constexpr (kStream) {
            if (!stream_ok) {
                // a wait for rows ran out: report it and let the copies that were started land before the block leaves
                if (c == 0 && o.status) atomicOr(reinterpret_cast<unsigned *>(o.status), E2EGREC_DEV_TIMEOUT);
                for (int g = max(0, n_issued - kStreamSlots); g < n_issued; ++g)
                    tm_mbar_wait(&sh_bar[rl][g % kStreamSlots], (uint32_t)(g / kStreamSlots) & 1u);
            }
        }
    }
    if (live_window)
        seg_join_window<T, int32_t, LPR, 1, kExtra>(sh_head, sh_tail, sh_info, sh_win, rl, c, n_chunks, d, head_seg, head_ends,
                                                    tail_seg, ptr, head2, tail2, win_info, o, chain_cnt, run_len);
    if (!chain_cnt) return;                        // the two-kernel form: seg_final_kernel writes the rest

    // ---- segments without entries (their row is the self row, masked, or zero) and the zero rows up to the next
    // multiple of 128: every block of the grid takes a slice, one lane group per segment
    {
        const int32_t n_self = o.n_self ? *o.n_self : n_seg;
        const int32_t per = (n_seg + (int32_t)gridDim.x - 1) / (int32_t)gridDim.x;
        const int32_t s1 = min(n_seg, ((int32_t)blockIdx.x + 1) * per);
        for (int32_t sg = (int32_t)blockIdx.x * per + rl; sg < s1; sg += RB) {
            if (ptr[sg + 1] != ptr[sg]) continue;
            float acc[1][E];
            uint4 mrow[1] = {make_uint4(0, 0, 0, 0)};
            uint4 raw = make_uint4(0, 0, 0, 0);
            if (c < n_chunks) {
                if (sg < n_self) raw = Chunk<T>::load_raw(o.self + (int64_t)sg * o.ld_self + c * E);
                if (kMask) mrow[0] = Chunk<T>::load_raw(o.mask + (int64_t)sg * o.ld_mask + c * E);
            }
            Chunk<T>::unpack(raw, acc[0]);
            seg_store_row<T, LPR, 1, kExtra>(o, sg, 1.0f, acc, mrow, c, n_chunks);
        }
        if (o.pad_rows > 0) {
            const int64_t pad_end = min(((int64_t)n_seg + 127) / 128 * 128, o.pad_rows);
            const int64_t cells = (pad_end - n_seg) * d;
            for (int64_t t = (int64_t)blockIdx.x * kAggThreads + threadIdx.x; t < cells; t += (int64_t)gridDim.x * kAggThreads)
                o.out[(n_seg + t / d) * o.ld_out + t % d] = from_float<T>(0.f);
        }
    }
}

// ------------------------------------------------------------------------------------ across windows
constexpr int kFinalWindows = 8;        // windows per block and round of seg_final_kernel: one per warp
constexpr int kFinalWarpParts = 64;     // longest chain of window parts that one warp adds by itself
template <typename T, typename PtrT>
__global__ void __launch_bounds__(kAggThreads)
seg_final_kernel(const PtrT *__restrict__ ptr, const int32_t *n_seg_dev, int64_t n_seg_host, int run_len, int runs_per_window,
                 int d, const float *__restrict__ head2, const float *__restrict__ tail2, const int4 *__restrict__ win_info,
                 int64_t n_windows, int64_t n_window_blocks, SegOut<T> o)
{
    __shared__ float4 red[kAggThreads];
    __shared__ int32_t sh_seg[kFinalWindows];
    __shared__ int sh_long[kFinalWindows];
    __shared__ int sh_n_long;
    pdl_launch_dependents();
    pdl_wait();
    const int64_t n_seg = n_seg_dev ? (int64_t)*n_seg_dev : n_seg_host;
    if (n_seg < 0) return;
    const int64_t n_self = o.self ? (o.n_self ? (int64_t)*o.n_self : n_seg) : 0;

    if ((int64_t)blockIdx.x >= n_window_blocks) {
        // segments without entries, the extra blocks stride over all segments
        const int64_t n_extra = (int64_t)gridDim.x - n_window_blocks;
        const int64_t b = (int64_t)blockIdx.x - n_window_blocks;
        if (!o.self && (d * (int)sizeof(T)) % 16 == 0 && o.ld_out * (int64_t)sizeof(T) % 16 == 0 &&
            reinterpret_cast<uintptr_t>(o.out) % 16 == 0) {
            // fin(0) = 0: one thread per segment, whole row in 16-byte stores
            const int n16 = d * (int)sizeof(T) / 16;
            for (int64_t s = b * kAggThreads + threadIdx.x; s < n_seg; s += n_extra * kAggThreads) {
                if (ptr[s + 1] != ptr[s]) continue;
                uint4 *row = reinterpret_cast<uint4 *>(o.out + s * o.ld_out);
                for (int q = 0; q < n16; ++q) row[q] = make_uint4(0, 0, 0, 0);
            }
        } else if ((d * (int)sizeof(T)) % 16 == 0 && o.ld_out * (int64_t)sizeof(T) % 16 == 0 &&
                   reinterpret_cast<uintptr_t>(o.out) % 16 == 0 && o.ld_self * (int64_t)sizeof(T) % 16 == 0 &&
                   reinterpret_cast<uintptr_t>(o.self) % 16 == 0 &&
                   (!o.mask || (o.ld_mask * (int64_t)sizeof(T) % 16 == 0 && reinterpret_cast<uintptr_t>(o.mask) % 16 == 0))) {
            // fin(0) = mask * self: eight lanes per segment, 16-byte chunks
            constexpr int E = Chunk<T>::kElems;
            const int n16 = d / E;
            for (int64_t s = (b * kAggThreads + threadIdx.x) >> 3; s < n_seg; s += n_extra * (kAggThreads / 8)) {
                if (ptr[s + 1] != ptr[s]) continue;
                for (int q = threadIdx.x & 7; q < n16; q += 8) {
                    float v[E];
#pragma unroll
                    for (int e = 0; e < E; ++e) v[e] = 0.f;
                    if (s < n_self) Chunk<T>::load(o.self + s * o.ld_self + q * E, v);
                    if (o.mask) {
                        float m[E];
                        Chunk<T>::load(o.mask + s * o.ld_mask + q * E, m);
#pragma unroll
                        for (int e = 0; e < E; ++e)
                            if (!(m[e] > 0.f)) v[e] = 0.f;
                    }
                    Chunk<T>::store(o.out + s * o.ld_out + q * E, v);
                }
            }
        } else {
            for (int64_t s = (b * kAggThreads + threadIdx.x) >> 3; s < n_seg; s += n_extra * (kAggThreads / 8)) {
                if (ptr[s + 1] != ptr[s]) continue;
                for (int k = threadIdx.x & 7; k < d; k += 8)
                    o.out[s * o.ld_out + k] = from_float<T>(seg_finish_value(o, s, 0, k, 0.f, s < n_self));
            }
        }
        if (o.pad_rows > 0) {                           // zero rows up to the next multiple of 128
            const int64_t pad_end = min((n_seg + 127) / 128 * 128, o.pad_rows);
            const int64_t cells = (pad_end - n_seg) * d;
            for (int64_t t = b * kAggThreads + threadIdx.x; t < cells; t += n_extra * kAggThreads)
                o.out[(n_seg + t / d) * o.ld_out + t % d] = from_float<T>(0.f);
        }
        return;
    }
    if (n_seg == 0) return;
    {   // only the windows that hold entries carry a record
        const int64_t total = (int64_t)ptr[n_seg];
        const int64_t live = ceil_div(ceil_div(total, (int64_t)run_len), (int64_t)runs_per_window);
        if (live < n_windows) n_windows = live;
    }

    // kFinalWindows windows per block and round; the window blocks stride over the windows.  A chain of up to kFinalWarpParts parts is added by one warp (the warps of
    // the block work on different windows at the same time); a longer one is left to the whole block.
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int64_t win0 = (int64_t)blockIdx.x * kFinalWindows; win0 < n_windows; win0 += n_window_blocks * kFinalWindows) {
    if (threadIdx.x < kFinalWindows) {
        int32_t sg = -1;
        const int64_t wi = win0 + threadIdx.x;
        if (wi < n_windows) {
            const int4 info = win_info[wi];
            if (info.x >= 0 && info.y) sg = info.x;         // a segment that began in an earlier window ends here
        }
        sh_seg[threadIdx.x] = sg;
    }
    if (threadIdx.x == 0) sh_n_long = 0;
    __syncthreads();
    const int n_vec = d / 4;                                // float4 columns (<= kAggThreads since d <= 1024)
    for (int j = warp; j < kFinalWindows; j += kAggThreads / 32) {
        const int32_t sg = sh_seg[j];
        if (sg < 0) continue;                               // uniform over the warp
        const int64_t win = win0 + j;
        const int64_t seg_beg = (int64_t)ptr[sg], seg_end = (int64_t)ptr[sg + 1];
        const int64_t first = (seg_beg / run_len) / runs_per_window;     // its first part is tail2[first]
        const int64_t n_parts = win - first + 1;
        if (n_parts > kFinalWarpParts) {
            if (lane == 0) sh_long[atomicAdd(&sh_n_long, 1)] = j;
            continue;
        }
        for (int vb = 0; vb < n_vec; vb += 32) {
            const int q = vb + lane;
            if (q >= n_vec) continue;
            float4 a = *reinterpret_cast<const float4 *>(tail2 + first * d + q * 4);
            for (int64_t p0 = 1; p0 < n_parts; p0 += 4) {
                float4 x[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    x[t] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (p0 + t < n_parts) x[t] = *reinterpret_cast<const float4 *>(head2 + (first + p0 + t) * d + q * 4);
                }
#pragma unroll
                for (int t = 0; t < 4; ++t) { a.x += x[t].x; a.y += x[t].y; a.z += x[t].z; a.w += x[t].w; }
            }
            const float r[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                o.out[(int64_t)sg * o.ld_out + q * 4 + kk] =
                    from_float<T>(seg_finish_value(o, sg, seg_end - seg_beg, q * 4 + kk, r[kk], false));
        }
    }
    __syncthreads();
    const int n_long = sh_n_long;
    const int q = threadIdx.x % n_vec, pl = threadIdx.x / n_vec;
    const int n_pl = kAggThreads / n_vec;                   // part lanes; threads with pl >= n_pl idle
    for (int i = 0; i < n_long; ++i) {
        const int j = sh_long[i];
        const int32_t sg = sh_seg[j];
        const int64_t win = win0 + j;
        const int64_t seg_beg = (int64_t)ptr[sg], seg_end = (int64_t)ptr[sg + 1];
        const int64_t first = (seg_beg / run_len) / runs_per_window;
        const int64_t n_parts = win - first + 1;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        if (pl < n_pl) {
            for (int64_t p0 = pl; p0 < n_parts; p0 += (int64_t)n_pl * 8) {
                float4 x[8];
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    const int64_t p = p0 + (int64_t)t * n_pl;
                    x[t] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (p < n_parts)
                        x[t] = *reinterpret_cast<const float4 *>((p == 0 ? tail2 + first * d : head2 + (first + p) * d) + q * 4);
                }
#pragma unroll
                for (int t = 0; t < 8; ++t) { a.x += x[t].x; a.y += x[t].y; a.z += x[t].z; a.w += x[t].w; }
            }
        }
        red[threadIdx.x] = a;
        __syncthreads();
        if (pl == 0) {
            float4 t = red[q];
            for (int w2 = 1; w2 < n_pl; ++w2) {
                const float4 x = red[w2 * n_vec + q];
                t.x += x.x; t.y += x.y; t.z += x.z; t.w += x.w;
            }
            const float r[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                o.out[(int64_t)sg * o.ld_out + q * 4 + kk] =
                    from_float<T>(seg_finish_value(o, sg, seg_end - seg_beg, q * 4 + kk, r[kk], false));
        }
        __syncthreads();
    }
    __syncthreads();                               // sh_seg / sh_long are rewritten by the next round
    }
}

// ------------------------------------------------------------------------------------ host
// E2EGREC_SEG_GENERAL=1 keeps sampled blocks on the general kernel (to compare the two forms; same results).
inline bool seg_general_only()
{
    static const bool v = []() {
        const char *e = getenv("E2EGREC_SEG_GENERAL");
        return e && *e && e[0] != '0';
    }();
    return v;
}

// E2EGREC_NO_STREAM_GATHER=1: no kernel streams its gathered rows through shared memory.
inline bool seg_stream_off()
{
    static const bool v = []() {
        const char *e = getenv("E2EGREC_NO_STREAM_GATHER"), *t = getenv("E2EGREC_NO_STREAM_TRANSPOSED");
        return (e && *e && e[0] != '0') || (t && *t && t[0] != '0');
    }();
    return v;
}

template <typename T, typename PtrT, int LPR, int CPL, bool kWeight, int kInFlight>
inline void launch_seg_reduce(const T *in, int64_t ld_in, const PtrT *ptr, const int32_t *idx, const int32_t *n_seg_dev,
                              int64_t n_seg_host, int64_t cap_seg, const float *w, int run_len, int d,
                              const int32_t *seg_of, const SegScratch &sc, const SegOut<T> &o, cudaStream_t st)
{
    constexpr size_t smem = seg_run_smem_bytes<LPR, CPL, Chunk<T>::kElems>();
    bool block_form = false;
    if constexpr (CPL == 1 && !kWeight && sizeof(PtrT) == 4)
        block_form = seg_of && n_seg_dev && o.self && !o.mean && !o.seg_scale && !seg_general_only();
    if (o.n_rhs > 1 && !(block_form && sc.chain_cnt)) {
        // the general kernels take one right-hand side per pass
        for (int r = 0; r < o.n_rhs; ++r) {
            SegOut<T> o1 = o;
            o1.n_rhs = 1;
            o1.out = o.out + r * o.rhs_out;
            if (o.self) o1.self = o.self + r * o.rhs_self;
            SegScratch s1 = sc;
            s1.head2 = sc.head2 + (size_t)r * sc.n_windows * d;
            s1.tail2 = sc.tail2 + (size_t)r * sc.n_windows * d;
            s1.win_info = sc.win_info + (size_t)r * sc.n_windows;
            s1.chain_cnt = nullptr;
            launch_seg_reduce<T, PtrT, LPR, CPL, kWeight, kInFlight>(in + r * o.rhs_in, ld_in, ptr, idx, n_seg_dev, n_seg_host, cap_seg, w,
                                                                     run_len, d, seg_of, s1, o1, st);
        }
        return;
    }
    tap_begin(TAP_SEG_L1, st);
    note_launch();
    const unsigned grid1 = (unsigned)sc.n_windows;
    if constexpr (CPL == 1 && !kWeight && sizeof(PtrT) == 4) {
        // the transposed aggregation of a sampled block: the kernel written for that case
        if (block_form) {
            block_form = true;
            const dim3 grid_b(grid1, (unsigned)(o.n_rhs > 1 && sc.chain_cnt ? o.n_rhs : 1));
            CUtensorMap in_map{};
            bool streamed = false;
            if constexpr (std::is_same<T, __nv_bfloat16>::value && LPR == 32) {
                // 512-byte rows in long runs: the rows come in through the TMA unit and a ring in shared memory
                if (d == 256 && run_len >= 64 && o.in_rows > 0 && !seg_stream_off() && make_row_gather_map(&in_map, in, o.in_rows, d, ld_in)) {
                    constexpr size_t smem_s = smem + 128 + (size_t)(kAggThreads / LPR) * kStreamSlots * 4 * kStreamRowBytes;
                    static bool attr_set[2][64] = {};
                    int dev = 0;
                    cudaGetDevice(&dev);
                    const int mk = o.mask ? 1 : 0;
                    if (dev >= 0 && dev < 64 && !attr_set[mk][dev]) {
                        const cudaError_t e =
                            mk ? cudaFuncSetAttribute(seg_run_block_kernel<T, LPR, true, 4, 3, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_s)
                               : cudaFuncSetAttribute(seg_run_block_kernel<T, LPR, false, 4, 4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_s);
                        attr_set[mk][dev] = e == cudaSuccess;
                    }
                    if (dev >= 0 && dev < 64 && attr_set[mk][dev]) {
                        streamed = true;
                        if (o.mask)
                            launch_pdl(seg_run_block_kernel<T, LPR, true, 4, 3, true>, grid_b, dim3(kAggThreads), smem_s, st, in_map, in, ld_in, ptr,
                                       idx, seg_of, n_seg_dev, run_len, d, sc.head2, sc.tail2, sc.win_info, sc.cap_runs, sc.chain_cnt, o);
                        else
                            launch_pdl(seg_run_block_kernel<T, LPR, false, 4, 4, true>, grid_b, dim3(kAggThreads), smem_s, st, in_map, in, ld_in, ptr,
                                       idx, seg_of, n_seg_dev, run_len, d, sc.head2, sc.tail2, sc.win_info, sc.cap_runs, sc.chain_cnt, o);
                    }
                }
            }
            if (streamed) {
            } else if (o.mask)
                launch_pdl(seg_run_block_kernel<T, LPR, true>, grid_b, dim3(kAggThreads), smem, st, in_map, in, ld_in, ptr, idx, seg_of,
                           n_seg_dev, run_len, d, sc.head2, sc.tail2, sc.win_info, sc.cap_runs, sc.chain_cnt, o);
            else
                launch_pdl(seg_run_block_kernel<T, LPR, false>, grid_b, dim3(kAggThreads), smem, st, in_map, in, ld_in, ptr, idx, seg_of,
                           n_seg_dev, run_len, d, sc.head2, sc.tail2, sc.win_info, sc.cap_runs, sc.chain_cnt, o);
            if (sc.chain_cnt) {                   // chains, empty segments and padding were all done in that launch
                tap_end(TAP_SEG_L1, st);
                tap_begin(TAP_SEG_L3, st);        // (an armed tap of the second kernel reads zero)
                tap_end(TAP_SEG_L3, st);
                return;
            }
        }
    }
    if (block_form) {
    } else if (o.mask) {
        auto kern = seg_run_kernel<T, PtrT, LPR, CPL, kWeight, 2, kInFlight>;
        if (smem > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        launch_pdl(kern, dim3(grid1), dim3(kAggThreads), smem, st, in, ld_in, ptr, idx, n_seg_dev, n_seg_host, w, run_len, d, sc.head2,
                   sc.tail2, sc.win_info, sc.cap_runs, seg_of, o);
    } else if (o.self) {
        auto kern = seg_run_kernel<T, PtrT, LPR, CPL, kWeight, 1, kInFlight>;
        if (smem > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        launch_pdl(kern, dim3(grid1), dim3(kAggThreads), smem, st, in, ld_in, ptr, idx, n_seg_dev, n_seg_host, w, run_len, d, sc.head2,
                   sc.tail2, sc.win_info, sc.cap_runs, seg_of, o);
    } else {
        auto kern = seg_run_kernel<T, PtrT, LPR, CPL, kWeight, 0, kInFlight>;
        if (smem > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        launch_pdl(kern, dim3(grid1), dim3(kAggThreads), smem, st, in, ld_in, ptr, idx, n_seg_dev, n_seg_host, w, run_len, d, sc.head2,
                   sc.tail2, sc.win_info, sc.cap_runs, seg_of, o);
    }
    tap_end(TAP_SEG_L1, st);
    const int64_t window_blocks = std::min<int64_t>(ceil_div(sc.n_windows, kFinalWindows), 148 * 16);
    const int64_t empty_blocks = std::min<int64_t>(ceil_div(cap_seg > 0 ? cap_seg : 1, kAggThreads), 148 * 8);
    tap_begin(TAP_SEG_L3, st);
    note_launch();
    launch_pdl(seg_final_kernel<T, PtrT>, dim3((unsigned)(window_blocks + empty_blocks)), dim3(kAggThreads), 0, st, ptr, n_seg_dev,
               n_seg_host, run_len, sc.runs_per_window, d, (const float *)sc.head2, (const float *)sc.tail2, (const int4 *)sc.win_info,
               sc.n_windows, window_blocks, o);
    tap_end(TAP_SEG_L3, st);
}

// Returns false (nothing enqueued) when no kernel is built for the row width; rows of up to 4096 bytes (kMaxDim fp32
// values) are covered, so callers that checked dim <= kMaxDim never see it.
template <typename T, typename PtrT, bool kWeight, int kInFlight = 4>
inline bool dispatch_seg_reduce(const T *in, int64_t ld_in, const PtrT *ptr, const int32_t *idx, const int32_t *n_seg_dev,
                                int64_t n_seg_host, int64_t cap_seg, const float *w, int run_len, int d, int32_t dtype,
                                const int32_t *seg_of, const SegScratch &sc, const SegOut<T> &o, cudaStream_t st)
{
    const RowShape rs = row_shape(d, dtype);
#define E2E_CASE(L, C)                                                                                                \
    if (rs.lpr == L && rs.cpl == C) {                                                                                 \
        launch_seg_reduce<T, PtrT, L, C, kWeight, kInFlight>(in, ld_in, ptr, idx, n_seg_dev, n_seg_host, cap_seg, w, run_len, \
                                                         d, seg_of, sc, o, st);                                       \
        return true;                                                                                                  \
    }
    E2E_CASE(4, 1) E2E_CASE(8, 1) E2E_CASE(16, 1) E2E_CASE(32, 1) E2E_CASE(32, 2) E2E_CASE(32, 4)
    if constexpr (sizeof(T) == 4) {      // rows of 2049 .. 4096 bytes exist only for fp32 (dim <= kMaxDim)
        E2E_CASE(32, 8)
    }
#undef E2E_CASE
    return false;
}

}  // namespace e2egrec
