// Segment reduction by gathered rows, three levels, no atomics, fixed summation order:
//
//     out[s] = fin( sum_{k in [ptr[s], ptr[s+1])} w[idx[k]] * in[idx[k]] ),   fin as in SegOut.
//
// This is the transposed aggregation of the backward pass (segments = columns of the block CSC)
// and the whole-graph aggregation in either direction (segments = CSR rows or CSC columns).
//
// Level 1 (seg_run_kernel): the entry stream is cut into runs of `run_len` consecutive entries and
//   every group of LPR lanes owns one run.  The group streams through its run with several row loads
//   in flight and closes a segment whenever the running entry index reaches the segment's end, so
//   thousands of one-entry segments and one segment of millions of entries cost the same per entry.
//   A segment that lies inside the run is finished there; otherwise its part goes to head[run]
//   (segment began in an earlier run) or tail[run] (segment began here and continues), and run_info
//   records which segments those are.
// Level 2 (seg_window_kernel): one warp per window of 32 runs adds the parts of segments that span
//   runs of the window, in run order; segments that also leave the window go to head2/tail2.
// Level 3 (seg_final_kernel): one block per window adds tail2[first] + head2[first+1..last] for the
//   segment that ends in its window, and extra blocks write fin(0) for segments without entries.
#pragma once

#include "aggregate.cuh"

namespace e2egrec {

constexpr int kSegWindow = 32;     // runs per level-2 window

struct SegScratch {
    float *head, *tail;            // [cap_runs x d]
    int4 *run_info;                // {head segment or -1, head ends in this run, tail segment or -1, 0}
    float *head2, *tail2;          // [n_windows x d]
    int4 *win_info;
    int64_t cap_runs, n_windows;
    size_t bytes;
};

inline SegScratch seg_scratch_carve(int64_t cap_entries, int run_len, int d, void *base)
{
    SegScratch s{};
    s.cap_runs = ceil_div(cap_entries > 0 ? cap_entries : 1, run_len);
    s.n_windows = ceil_div(s.cap_runs, kSegWindow);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        char *p = base ? static_cast<char *>(base) + off : nullptr;
        off += align_up(bytes, 256);
        return p;
    };
    s.head = (float *)take((size_t)s.cap_runs * d * sizeof(float));
    s.tail = (float *)take((size_t)s.cap_runs * d * sizeof(float));
    s.run_info = (int4 *)take((size_t)s.n_windows * kSegWindow * sizeof(int4));
    s.head2 = (float *)take((size_t)s.n_windows * d * sizeof(float));
    s.tail2 = (float *)take((size_t)s.n_windows * d * sizeof(float));
    s.win_info = (int4 *)take((size_t)s.n_windows * sizeof(int4));
    s.bytes = off;
    return s;
}

// ------------------------------------------------------------------------------------ level 1
template <typename T, typename PtrT, int LPR, int CPL, bool kWeight>
__global__ void __launch_bounds__(kAggThreads)
seg_run_kernel(const T *__restrict__ in, int64_t ld_in, const PtrT *__restrict__ ptr, const int32_t *__restrict__ idx,
               const int32_t *n_seg_dev, int64_t n_seg_host, const float *__restrict__ w, int run_len, int d,
               float *__restrict__ head, float *__restrict__ tail, int4 *__restrict__ run_info, int64_t cap_runs,
               SegOut<T> o)
{
    constexpr int E = Chunk<T>::kElems;
    constexpr int U = CPL >= 4 ? 1 : 4 / CPL;
    const int c = threadIdx.x % LPR;
    const int n_chunks = d / E;
    const int64_t run = ((int64_t)blockIdx.x * kAggThreads + threadIdx.x) / LPR;
    if (run >= cap_runs) return;
    const int64_t n_seg = n_seg_dev ? (int64_t)*n_seg_dev : n_seg_host;
    const int64_t total = n_seg > 0 ? (int64_t)ptr[n_seg] : 0;
    const int64_t k0 = run * run_len;
    if (k0 >= total) {
        if (c == 0) run_info[run] = make_int4(-1, 0, -1, 0);
        return;
    }
    const int64_t k1 = min(k0 + (int64_t)run_len, total);
    const int64_t n_self = o.self ? (o.n_self ? (int64_t)*o.n_self : n_seg) : 0;

    int64_t s = seg_containing(ptr, n_seg, k0);
    int64_t cur_beg = (int64_t)ptr[s], cur_end = (int64_t)ptr[s + 1];
    int32_t head_seg = -1, head_ends = 0, tail_seg = -1;

    float acc[CPL][E];
#pragma unroll
    for (int q = 0; q < CPL; ++q)
#pragma unroll
        for (int kk = 0; kk < E; ++kk) acc[q][kk] = 0.f;

    // closes the current segment [cur_beg, cur_end) with the sum in acc
    auto emit = [&](bool ended) {
        const bool begins = cur_beg >= k0;
#pragma unroll
        for (int q = 0; q < CPL; ++q) {
            const int ch = c + q * LPR;
            if (ch < n_chunks) {
                if (begins && ended) {
                    float r[E];
#pragma unroll
                    for (int kk = 0; kk < E; ++kk)
                        r[kk] = seg_finish_value(o, s, cur_end - cur_beg, ch * E + kk, acc[q][kk], s < n_self);
                    Chunk<T>::store(o.out + s * o.ld_out + ch * E, r);
                } else {
                    float *dst = (begins ? tail : head) + run * d + ch * E;
#pragma unroll
                    for (int kk = 0; kk < E; kk += 4)
                        *reinterpret_cast<float4 *>(dst + kk) =
                            make_float4(acc[q][kk], acc[q][kk + 1], acc[q][kk + 2], acc[q][kk + 3]);
                }
            }
#pragma unroll
            for (int kk = 0; kk < E; ++kk) acc[q][kk] = 0.f;
        }
        if (!(begins && ended)) {
            if (begins) tail_seg = (int32_t)s;
            else { head_seg = (int32_t)s; head_ends = ended ? 1 : 0; }
        }
    };

    int32_t id_next[U];
#pragma unroll
    for (int u = 0; u < U; ++u) id_next[u] = k0 + u < k1 ? idx[k0 + u] : 0;

    for (int64_t k = k0; k < k1; k += U) {
        float v[U][CPL][E];
        float wt[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int32_t id = id_next[u];
            wt[u] = 1.f;
            if (k + u < k1) {
                if (kWeight) wt[u] = w[id];
                const T *row = in + (int64_t)id * ld_in;
#pragma unroll
                for (int q = 0; q < CPL; ++q) {
                    const int ch = c + q * LPR;
                    if (ch < n_chunks) Chunk<T>::load(row + ch * E, v[u][q]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) id_next[u] = k + U + u < k1 ? idx[k + U + u] : 0;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t kk2 = k + u;
            if (kk2 < k1) {
                if (kk2 >= cur_end) {
                    emit(true);
                    do { ++s; cur_end = (int64_t)ptr[s + 1]; } while (cur_end <= kk2);   // skips empty segments
                    cur_beg = (int64_t)ptr[s];
                }
#pragma unroll
                for (int q = 0; q < CPL; ++q)
                    if (c + q * LPR < n_chunks)
#pragma unroll
                        for (int e = 0; e < E; ++e) {
                            if (kWeight) acc[q][e] = fmaf(wt[u], v[u][q][e], acc[q][e]);
                            else acc[q][e] += v[u][q][e];
                        }
            }
        }
    }
    emit(cur_end <= k1);
    if (c == 0) run_info[run] = make_int4(head_seg, head_ends, tail_seg, 0);
}

// ------------------------------------------------------------------------------------ level 2
template <typename T, typename PtrT>
__global__ void __launch_bounds__(kAggThreads)
seg_window_kernel(const PtrT *__restrict__ ptr, const int32_t *n_seg_dev, int64_t n_seg_host, int d,
                  const float *__restrict__ head, const float *__restrict__ tail, const int4 *__restrict__ run_info,
                  float *__restrict__ head2, float *__restrict__ tail2, int4 *__restrict__ win_info,
                  int64_t cap_runs, int64_t n_windows, SegOut<T> o)
{
    const int lane = threadIdx.x & 31;
    const int64_t win = ((int64_t)blockIdx.x * kAggThreads + threadIdx.x) >> 5;
    if (win >= n_windows) return;
    const int64_t n_seg = n_seg_dev ? (int64_t)*n_seg_dev : n_seg_host;
    const int64_t n_self = o.self ? (o.n_self ? (int64_t)*o.n_self : n_seg) : 0;
    const int64_t r0 = win * kSegWindow;
    int4 info = make_int4(-1, 0, -1, 0);
    if (r0 + lane < cap_runs) info = run_info[r0 + lane];
    const unsigned any = __ballot_sync(0xffffffffu, info.x >= 0 || info.z >= 0);
    int32_t w_head = -1, w_head_ends = 0, w_tail = -1;
    if (any) {
        const int n_vec = d / 4;
        for (int vb = 0; vb < n_vec; vb += 32) {
            const int q = vb + lane;
            const bool act = q < n_vec;
            int32_t cur = -1;
            bool from_tail = false;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            w_head = -1; w_head_ends = 0; w_tail = -1;
            for (int rb = 0; rb < kSegWindow; rb += 4) {
                // fetch the records of four runs, then walk them in order
                float4 hv[4], tv[4];
                int32_t hs[4], he[4], ts[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    hs[j] = __shfl_sync(0xffffffffu, info.x, rb + j);
                    he[j] = __shfl_sync(0xffffffffu, info.y, rb + j);
                    ts[j] = __shfl_sync(0xffffffffu, info.z, rb + j);
                    hv[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                    tv[j] = hv[j];
                    if (act && hs[j] >= 0) hv[j] = *reinterpret_cast<const float4 *>(head + (r0 + rb + j) * d + q * 4);
                    if (act && ts[j] >= 0) tv[j] = *reinterpret_cast<const float4 *>(tail + (r0 + rb + j) * d + q * 4);
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (hs[j] >= 0) {
                        if (cur != hs[j]) { cur = hs[j]; from_tail = false; acc = make_float4(0.f, 0.f, 0.f, 0.f); }
                        acc.x += hv[j].x; acc.y += hv[j].y; acc.z += hv[j].z; acc.w += hv[j].w;
                        if (he[j]) {
                            if (from_tail) {
                                if (act) {
                                    const int64_t s = cur;
                                    const int64_t len = (int64_t)ptr[s + 1] - (int64_t)ptr[s];
                                    const float r[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
                                    for (int e = 0; e < 4; ++e)
                                        o.out[s * o.ld_out + q * 4 + e] =
                                            from_float<T>(seg_finish_value(o, s, len, q * 4 + e, r[e], s < n_self));
                                }
                            } else {
                                if (act) *reinterpret_cast<float4 *>(head2 + win * d + q * 4) = acc;
                                w_head = cur; w_head_ends = 1;
                            }
                            cur = -1;
                        }
                    }
                    if (ts[j] >= 0) { cur = ts[j]; from_tail = true; acc = tv[j]; }
                }
            }
            if (cur >= 0) {
                if (from_tail) {
                    if (act) *reinterpret_cast<float4 *>(tail2 + win * d + q * 4) = acc;
                    w_tail = cur;
                } else {
                    if (act) *reinterpret_cast<float4 *>(head2 + win * d + q * 4) = acc;
                    w_head = cur; w_head_ends = 0;
                }
            }
        }
    }
    if (lane == 0) win_info[win] = make_int4(w_head, w_head_ends, w_tail, 0);
}

// ------------------------------------------------------------------------------------ level 3
template <typename T, typename PtrT>
__global__ void __launch_bounds__(kAggThreads)
seg_final_kernel(const PtrT *__restrict__ ptr, const int32_t *n_seg_dev, int64_t n_seg_host, int run_len, int d,
                 const float *__restrict__ head2, const float *__restrict__ tail2, const int4 *__restrict__ win_info,
                 int64_t n_windows, SegOut<T> o)
{
    constexpr int W = kAggThreads / 32;
    __shared__ float4 red[W][32];
    const int64_t n_seg = n_seg_dev ? (int64_t)*n_seg_dev : n_seg_host;
    if (n_seg <= 0) return;
    const int64_t n_self = o.self ? (o.n_self ? (int64_t)*o.n_self : n_seg) : 0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    if ((int64_t)blockIdx.x >= n_windows) {
        // segments without entries: 8 lanes per segment
        const int64_t s = ((int64_t)(blockIdx.x - n_windows) * kAggThreads + threadIdx.x) >> 3;
        if (s >= n_seg || ptr[s + 1] != ptr[s]) return;
        for (int k = threadIdx.x & 7; k < d; k += 8)
            o.out[s * o.ld_out + k] = from_float<T>(seg_finish_value(o, s, 0, k, 0.f, s < n_self));
        return;
    }
    const int64_t win = blockIdx.x;
    const int4 info = win_info[win];
    if (info.x < 0 || !info.y) return;                   // no segment that began earlier ends in this window
    const int64_t s = info.x;
    const int64_t seg_beg = (int64_t)ptr[s], seg_end = (int64_t)ptr[s + 1];
    const int64_t first = (seg_beg / run_len) / kSegWindow;      // its first part is tail2[first]
    const int64_t n_parts = win - first + 1;
    const int n_vec = d / 4;
    for (int vb = 0; vb < n_vec; vb += 32) {
        const int q = vb + lane;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        if (q < n_vec) {
            for (int64_t p0 = warp * 4; p0 < n_parts; p0 += W * 4) {
                float4 x[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int64_t p = p0 + j;
                    x[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (p < n_parts)
                        x[j] = *reinterpret_cast<const float4 *>((p == 0 ? tail2 + first * d : head2 + (first + p) * d) + q * 4);
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) { a.x += x[j].x; a.y += x[j].y; a.z += x[j].z; a.w += x[j].w; }
            }
        }
        red[warp][lane] = a;
        __syncthreads();
        if (warp == 0 && q < n_vec) {
            float4 t = red[0][lane];
#pragma unroll
            for (int w2 = 1; w2 < W; ++w2) {
                const float4 x = red[w2][lane];
                t.x += x.x; t.y += x.y; t.z += x.z; t.w += x.w;
            }
            const float r[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                o.out[s * o.ld_out + q * 4 + kk] =
                    from_float<T>(seg_finish_value(o, s, seg_end - seg_beg, q * 4 + kk, r[kk], s < n_self));
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------ host
template <typename T, typename PtrT, int LPR, int CPL, bool kWeight>
inline void launch_seg_reduce(const T *in, int64_t ld_in, const PtrT *ptr, const int32_t *idx, const int32_t *n_seg_dev,
                              int64_t n_seg_host, int64_t cap_seg, const float *w, int run_len, int d,
                              const SegScratch &sc, const SegOut<T> &o, cudaStream_t st)
{
    note_launch();
    seg_run_kernel<T, PtrT, LPR, CPL, kWeight><<<(unsigned)ceil_div(sc.cap_runs * LPR, kAggThreads), kAggThreads, 0, st>>>(
        in, ld_in, ptr, idx, n_seg_dev, n_seg_host, w, run_len, d, sc.head, sc.tail, sc.run_info, sc.cap_runs, o);
    note_launch();
    seg_window_kernel<T, PtrT><<<(unsigned)ceil_div(sc.n_windows * 32, kAggThreads), kAggThreads, 0, st>>>(
        ptr, n_seg_dev, n_seg_host, d, sc.head, sc.tail, sc.run_info, sc.head2, sc.tail2, sc.win_info, sc.cap_runs,
        sc.n_windows, o);
    const int64_t empty_blocks = ceil_div((cap_seg > 0 ? cap_seg : 1) * 8, kAggThreads);
    note_launch();
    seg_final_kernel<T, PtrT><<<(unsigned)(sc.n_windows + empty_blocks), kAggThreads, 0, st>>>(
        ptr, n_seg_dev, n_seg_host, run_len, d, sc.head2, sc.tail2, sc.win_info, sc.n_windows, o);
}

template <typename T, typename PtrT, bool kWeight>
inline void dispatch_seg_reduce(const T *in, int64_t ld_in, const PtrT *ptr, const int32_t *idx, const int32_t *n_seg_dev,
                                int64_t n_seg_host, int64_t cap_seg, const float *w, int run_len, int d, int32_t dtype,
                                const SegScratch &sc, const SegOut<T> &o, cudaStream_t st)
{
    const RowShape rs = row_shape(d, dtype);
#define E2E_CASE(L, C)                                                                                                \
    if (rs.lpr == L && rs.cpl == C)                                                                                   \
        return launch_seg_reduce<T, PtrT, L, C, kWeight>(in, ld_in, ptr, idx, n_seg_dev, n_seg_host, cap_seg, w, run_len, \
                                                         d, sc, o, st);
    E2E_CASE(4, 1) E2E_CASE(8, 1) E2E_CASE(16, 1) E2E_CASE(32, 1) E2E_CASE(32, 2) E2E_CASE(32, 4)
#undef E2E_CASE
}

}  // namespace e2egrec
