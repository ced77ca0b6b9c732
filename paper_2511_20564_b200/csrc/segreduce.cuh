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
//   records which segments those are.  The optional self row of a segment is added where the segment
//   begins, so partial sums already contain it.
// Level 2 (seg_window_kernel): one warp per window of 32 runs adds the parts of segments that span
//   runs of the window, in run order; segments that also leave the window go to head2/tail2.
// Level 3 (seg_final_kernel): one block per window adds tail2[first] + head2[first+1..last] for the
//   segment that ends in its window, and extra blocks write fin(0) for segments without entries.
#pragma once

#include <algorithm>

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

// ------------------------------------------------------------------------------------ level 1
// Partial sums of a run go out as float4 stores.  Inlined on purpose: a call that receives the accumulators by
// reference would pin them in local memory, and every add of the streaming loop would then store to it.
template <int CPL, int E>
__device__ __forceinline__ void seg_store_partial(float *dst, const float (&acc)[CPL][E], int c, int lpr, int n_chunks)
{
#pragma unroll
    for (int q = 0; q < CPL; ++q) {
        const int ch = c + q * lpr;
        if (ch < n_chunks) {
#pragma unroll
            for (int e = 0; e < E; e += 4)
                *reinterpret_cast<float4 *>(dst + ch * E + e) = make_float4(acc[q][e], acc[q][e + 1], acc[q][e + 2], acc[q][e + 3]);
        }
    }
}

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

// kExtra: the output has a self row and/or a mask row per segment (they are fetched together with the
// segment's first gathered row); without it those registers and branches disappear.
template <typename T, typename PtrT, int LPR, int CPL, bool kWeight, bool kExtra>
__global__ void __launch_bounds__(kAggThreads)
seg_run_kernel(const T *__restrict__ in, int64_t ld_in, const PtrT *__restrict__ ptr, const int32_t *__restrict__ idx,
               const int32_t *n_seg_dev, int64_t n_seg_host, const float *__restrict__ w, int run_len, int d,
               float *__restrict__ head, float *__restrict__ tail, int4 *__restrict__ run_info, int64_t cap_runs,
               const int32_t *__restrict__ seg_of, SegOut<T> o)
{
    constexpr int E = Chunk<T>::kElems;
    constexpr int U = CPL >= 4 ? 1 : 4 / CPL;
    constexpr int kFar = 1 << 30;
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
    const int len = (int)min((int64_t)run_len, total - k0);       // entries of this run; positions below are relative to k0
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
    int32_t head_seg = -1, head_ends = 0, tail_seg = -1;

    // closes the current segment, which ends at relative position end_rel, with the sum in acc
    auto emit = [&](bool ended, int end_rel) {
        if (cur_begins && ended) {
            const float inv = o.mean ? 1.0f / (float)(end_rel - cur_beg_rel) : (o.seg_scale ? o.seg_scale[cur_seg] : 1.0f);
#pragma unroll
            for (int q = 0; q < CPL; ++q) {
                const int ch = c + q * LPR;
                if (ch < n_chunks) {
                    float r[E];
#pragma unroll
                    for (int e = 0; e < E; ++e) r[e] = to_float<T>(from_float<T>(acc[q][e] * inv));   // inv = 1 without mean / scale
                    if (kExtra && o.mask) {
                        float m[E];
                        Chunk<T>::unpack(cur_mask[q], m);
#pragma unroll
                        for (int e = 0; e < E; ++e)
                            if (!(m[e] > 0.f)) r[e] = 0.f;
                    }
                    Chunk<T>::store(o.out + (int64_t)cur_seg * o.ld_out + ch * E, r);
                }
            }
        } else {
            seg_store_partial<CPL, E>((cur_begins ? tail : head) + run * d, acc, c, LPR, n_chunks);
            if (cur_begins) tail_seg = cur_seg;
            else { head_seg = cur_seg; head_ends = ended ? 1 : 0; }
        }
    };

    classify(0);
    for (int r0 = 0; r0 < len; r0 += U) {
        int32_t seg_c[U];
        bool start_c[U];
        float wt[U];
        uint4 v[U][CPL], sv[kExtra ? U : 1][CPL], mv[kExtra ? U : 1][CPL];
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
                    mv[u][q] = make_uint4(0, 0, 0, 0);
                    if (live && start_c[u] && ch < n_chunks) {
                        const bool begins = r0 + u != 0 || first_begins;
                        if (begins && seg_c[u] < n_self)
                            sv[u][q] = Chunk<T>::load_raw(o.self + (int64_t)seg_c[u] * o.ld_self + ch * E);
                        if (o.mask) mv[u][q] = Chunk<T>::load_raw(o.mask + (int64_t)seg_c[u] * o.ld_mask + ch * E);
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
                            cur_mask[q] = mv[u][q];
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
                    for (int e = 0; e < E; ++e) {
                        if (kWeight) acc[q][e] = fmaf(wt[u], x[e], acc[q][e]);
                        else acc[q][e] += x[e];
                    }
                }
            }
        }
    }
    emit(seg0 ? last_ends : rel_end <= len, len);
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
    constexpr int kB = 8;                         // runs fetched together
    const int lane = threadIdx.x & 31;
    const int64_t win = ((int64_t)blockIdx.x * kAggThreads + threadIdx.x) >> 5;
    if (win >= n_windows) return;
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
            for (int rb = 0; rb < kSegWindow; rb += kB) {
                // fetch the records of kB runs (and the mask rows of segments that end in them), then walk them in order
                float4 hv[kB], tv[kB], mk[kB];
                int32_t hs[kB], he[kB], ts[kB];
#pragma unroll
                for (int j = 0; j < kB; ++j) {
                    hs[j] = __shfl_sync(0xffffffffu, info.x, rb + j);
                    he[j] = __shfl_sync(0xffffffffu, info.y, rb + j);
                    ts[j] = __shfl_sync(0xffffffffu, info.z, rb + j);
                    hv[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                    tv[j] = hv[j];
                    mk[j] = make_float4(1.f, 1.f, 1.f, 1.f);
                    if (act && hs[j] >= 0) hv[j] = *reinterpret_cast<const float4 *>(head + (r0 + rb + j) * d + q * 4);
                    if (act && ts[j] >= 0) tv[j] = *reinterpret_cast<const float4 *>(tail + (r0 + rb + j) * d + q * 4);
                    if (act && hs[j] >= 0 && he[j] && o.mask) mk[j] = load4<T>(o.mask + (int64_t)hs[j] * o.ld_mask + q * 4);
                }
#pragma unroll
                for (int j = 0; j < kB; ++j) {
                    if (hs[j] >= 0) {
                        if (cur != hs[j]) { cur = hs[j]; from_tail = false; acc = make_float4(0.f, 0.f, 0.f, 0.f); }
                        acc.x += hv[j].x; acc.y += hv[j].y; acc.z += hv[j].z; acc.w += hv[j].w;
                        if (he[j]) {
                            if (from_tail) {
                                if (act) {
                                    const int64_t s = cur;
                                    float inv = 0.f;
                                    if (o.mean) inv = 1.0f / (float)((int64_t)ptr[s + 1] - (int64_t)ptr[s]);
                                    else if (o.seg_scale) inv = o.seg_scale[s];
                                    const float m[4] = {mk[j].x, mk[j].y, mk[j].z, mk[j].w};
                                    float r[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
                                    for (int e = 0; e < 4; ++e) {
                                        r[e] = seg_round(o, inv, r[e]);
                                        if (!(m[e] > 0.f)) r[e] = 0.f;
                                    }
                                    store4<T>(o.out + s * o.ld_out + q * 4, r);
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
    if (n_seg < 0) return;
    const int64_t n_self = o.self ? (o.n_self ? (int64_t)*o.n_self : n_seg) : 0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    if ((int64_t)blockIdx.x >= n_windows) {
        // segments without entries: 8 lanes per segment, the extra blocks stride over all segments
        const int64_t n_extra = (int64_t)gridDim.x - n_windows;
        for (int64_t s = ((int64_t)(blockIdx.x - n_windows) * kAggThreads + threadIdx.x) >> 3; s < n_seg;
             s += n_extra * (kAggThreads / 8)) {
            if (ptr[s + 1] != ptr[s]) continue;
            for (int k = threadIdx.x & 7; k < d; k += 8)
                o.out[s * o.ld_out + k] = from_float<T>(seg_finish_value(o, s, 0, k, 0.f, s < n_self));
        }
        if (o.pad_rows > 0) {                           // zero rows up to the next multiple of 128
            const int64_t pad_end = min((n_seg + 127) / 128 * 128, o.pad_rows);
            const int64_t cells = (pad_end - n_seg) * d;
            for (int64_t t = (int64_t)(blockIdx.x - n_windows) * kAggThreads + threadIdx.x; t < cells;
                 t += n_extra * kAggThreads)
                o.out[(n_seg + t / d) * o.ld_out + t % d] = from_float<T>(0.f);
        }
        return;
    }
    if (n_seg == 0) return;
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
                    from_float<T>(seg_finish_value(o, s, seg_end - seg_beg, q * 4 + kk, r[kk], false));
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------ host
template <typename T, typename PtrT, int LPR, int CPL, bool kWeight>
inline void launch_seg_reduce(const T *in, int64_t ld_in, const PtrT *ptr, const int32_t *idx, const int32_t *n_seg_dev,
                              int64_t n_seg_host, int64_t cap_seg, const float *w, int run_len, int d,
                              const int32_t *seg_of, const SegScratch &sc, const SegOut<T> &o, cudaStream_t st)
{
    tap_begin(TAP_SEG_L1, st);
    note_launch();
    const unsigned grid1 = (unsigned)ceil_div(sc.cap_runs * LPR, kAggThreads);
    if (o.self || o.mask)
        seg_run_kernel<T, PtrT, LPR, CPL, kWeight, true><<<grid1, kAggThreads, 0, st>>>(
            in, ld_in, ptr, idx, n_seg_dev, n_seg_host, w, run_len, d, sc.head, sc.tail, sc.run_info, sc.cap_runs, seg_of, o);
    else
        seg_run_kernel<T, PtrT, LPR, CPL, kWeight, false><<<grid1, kAggThreads, 0, st>>>(
            in, ld_in, ptr, idx, n_seg_dev, n_seg_host, w, run_len, d, sc.head, sc.tail, sc.run_info, sc.cap_runs, seg_of, o);
    tap_end(TAP_SEG_L1, st);
    tap_begin(TAP_SEG_L2, st);
    note_launch();
    seg_window_kernel<T, PtrT><<<(unsigned)ceil_div(sc.n_windows * 32, kAggThreads), kAggThreads, 0, st>>>(
        ptr, n_seg_dev, n_seg_host, d, sc.head, sc.tail, sc.run_info, sc.head2, sc.tail2, sc.win_info, sc.cap_runs,
        sc.n_windows, o);
    tap_end(TAP_SEG_L2, st);
    const int64_t empty_blocks = std::min<int64_t>(ceil_div((cap_seg > 0 ? cap_seg : 1) * 8, kAggThreads), 148 * 8);
    tap_begin(TAP_SEG_L3, st);
    note_launch();
    seg_final_kernel<T, PtrT><<<(unsigned)(sc.n_windows + empty_blocks), kAggThreads, 0, st>>>(
        ptr, n_seg_dev, n_seg_host, run_len, d, sc.head2, sc.tail2, sc.win_info, sc.n_windows, o);
    tap_end(TAP_SEG_L3, st);
}

template <typename T, typename PtrT, bool kWeight>
inline void dispatch_seg_reduce(const T *in, int64_t ld_in, const PtrT *ptr, const int32_t *idx, const int32_t *n_seg_dev,
                                int64_t n_seg_host, int64_t cap_seg, const float *w, int run_len, int d, int32_t dtype,
                                const int32_t *seg_of, const SegScratch &sc, const SegOut<T> &o, cudaStream_t st)
{
    const RowShape rs = row_shape(d, dtype);
#define E2E_CASE(L, C)                                                                                                \
    if (rs.lpr == L && rs.cpl == C)                                                                                   \
        return launch_seg_reduce<T, PtrT, L, C, kWeight>(in, ld_in, ptr, idx, n_seg_dev, n_seg_host, cap_seg, w, run_len, \
                                                         d, seg_of, sc, o, st);
    E2E_CASE(4, 1) E2E_CASE(8, 1) E2E_CASE(16, 1) E2E_CASE(32, 1) E2E_CASE(32, 2) E2E_CASE(32, 4)
#undef E2E_CASE
}

}  // namespace e2egrec
