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

#include <algorithm>

#include "aggregate.cuh"

namespace e2egrec {

constexpr int kSegRing = 8;        // entries requested ahead in the ring form of seg_run_kernel

// runs per window = lane groups per block of seg_run_kernel
inline int seg_runs_per_window(int d, size_t elem_size) { return kAggThreads / row_shape_bytes((int64_t)d * elem_size).lpr; }

struct SegScratch {
    float *head2, *tail2;          // [n_windows x d]
    int4 *win_info;                // {segment whose sum continues from an earlier window or -1, it ends here, segment
                                   //  that continues into the next window or -1, 0}
    int64_t cap_runs, n_windows;
    int runs_per_window;
    size_t bytes;
};

inline SegScratch seg_scratch_carve(int64_t cap_entries, int run_len, int d, size_t elem_size, void *base)
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

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

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
// kRing > 0 (sampled blocks with a self row, 16-byte chunk per lane): the gathered chunk of every entry, and the self
// chunk where a segment begins, are requested kRing entries ahead with cp.async into a ring in shared memory (each
// thread reads back only what it requested itself, so the ring needs no barrier); the bytes in flight then no longer
// occupy registers and do not stop at the four rows of a batch.
template <typename T, typename PtrT, int LPR, int CPL, bool kWeight, int kExtra, int kInFlight, int kRing = 0>
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

        static_assert(kRing == 0 || (CPL == 1 && !kWeight && kExtra == 1 && kRing >= U), "ring form: one chunk per lane, self rows only");
        constexpr int kSlot = kAggThreads * 16;               // bytes of one ring slot (one 16-byte chunk per thread)
        uint8_t *ring_g = reinterpret_cast<uint8_t *>(sh_info + RB) + threadIdx.x * 16;     // gathered chunks
        uint8_t *ring_s = ring_g + (kRing > 0 ? kRing : 1) * kSlot;                            // self chunks
        // requests entry r (same tests as the sums below make when they read the slot back)
        auto issue = [&](int r) {
            if (kRing > 0) {
                if (r < len && c < n_chunks) {
                    const int slot = r % (kRing > 0 ? kRing : 1);
                    cp_async16(ring_g + slot * kSlot, in + (int64_t)idx0[r] * ld_in + c * E);
                    const int32_t sg = seg0[r];
                    const bool st = r == 0 || sg != seg0[r - 1];
                    if (st && (r != 0 || first_begins) && sg < n_self)
                        cp_async16(ring_s + slot * kSlot, o.self + (int64_t)sg * o.ld_self + c * E);
                }
                cp_async_commit();
            }
        };
        if (kRing > 0) {
#pragma unroll
            for (int r = 0; r < (kRing > 0 ? kRing : 1); ++r) issue(r);
        }

        classify(0);
        for (int r0 = 0; r0 < len; r0 += U) {
            int32_t seg_c[U];
            bool start_c[U];
            float wt[U];
            uint4 v[U][CPL], sv[kExtra ? U : 1][CPL], mv[kExtra == 2 ? U : 1][CPL];
            if (kRing > 0) cp_async_wait<(kRing > U ? kRing - U : 0)>();       // the entries of this batch have landed
#pragma unroll
            for (int u = 0; u < U; ++u) {
                seg_c[u] = seg_n[u];
                start_c[u] = start_n[u];
                wt[u] = 1.f;
                const bool live = r0 + u < len;
                const int32_t id = id_n[u];
                if (kWeight && live) wt[u] = w[id];
                if (kRing > 0) {
                    const int slot = (r0 + u) % (kRing > 0 ? kRing : 1);
                    v[u][0] = make_uint4(0, 0, 0, 0);
                    sv[u][0] = make_uint4(0, 0, 0, 0);
                    if (live && c < n_chunks) {
                        v[u][0] = *reinterpret_cast<const uint4 *>(ring_g + slot * kSlot);
                        if (start_c[u] && (r0 + u != 0 || first_begins) && seg_c[u] < n_self)
                            sv[u][0] = *reinterpret_cast<const uint4 *>(ring_s + slot * kSlot);
                    }
                }
                if (kRing == 0) {
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
            if (kRing > 0) {                                  // the slots just read take the entries kRing further on
#pragma unroll
                for (int u = 0; u < U; ++u) issue(r0 + (kRing > 0 ? kRing : 1) + u);
            }
        }
        if (kRing > 0) cp_async_wait<0>();
        emit(seg0 ? last_ends : rel_end <= len, len);
    }
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
                finish(head_seg, inv, acc, mrow);
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
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) win_info[blockIdx.x] = make_int4(sh_win[0], sh_win[1], sh_win[2], 0);
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
template <typename T, typename PtrT, int LPR, int CPL, bool kWeight, int kInFlight>
inline void launch_seg_reduce(const T *in, int64_t ld_in, const PtrT *ptr, const int32_t *idx, const int32_t *n_seg_dev,
                              int64_t n_seg_host, int64_t cap_seg, const float *w, int run_len, int d,
                              const int32_t *seg_of, const SegScratch &sc, const SegOut<T> &o, cudaStream_t st)
{
    constexpr size_t smem = seg_run_smem_bytes<LPR, CPL, Chunk<T>::kElems>();
    tap_begin(TAP_SEG_L1, st);
    note_launch();
    const unsigned grid1 = (unsigned)sc.n_windows;
    if (o.mask) {
        auto kern = seg_run_kernel<T, PtrT, LPR, CPL, kWeight, 2, kInFlight>;
        if (smem > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        kern<<<grid1, kAggThreads, smem, st>>>(in, ld_in, ptr, idx, n_seg_dev, n_seg_host, w, run_len, d, sc.head2, sc.tail2,
                                               sc.win_info, sc.cap_runs, seg_of, o);
    } else if (o.self && run_len >= 128 && kSegRing > 0 && CPL == 1 && !kWeight && sizeof(PtrT) == 4 && LPR >= 16 && kInFlight == 4 &&
               seg_of) {
        // rows of 256 bytes and more on a sampled block that can hold millions of entries (long runs: the rows it gathers do
        // not fit in L2): the ring form.  On smaller blocks, whose rows come from L2, registers in flight are faster.
        if constexpr (CPL == 1 && !kWeight && sizeof(PtrT) == 4 && LPR >= 16 && kInFlight == 4) {
            constexpr size_t smem_ring = smem + (size_t)2 * kSegRing * kAggThreads * 16;
            auto kern = seg_run_kernel<T, PtrT, LPR, CPL, kWeight, 1, kInFlight, kSegRing>;
            cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_ring);
            kern<<<grid1, kAggThreads, smem_ring, st>>>(in, ld_in, ptr, idx, n_seg_dev, n_seg_host, w, run_len, d, sc.head2,
                                                        sc.tail2, sc.win_info, sc.cap_runs, seg_of, o);
        }
    } else if (o.self) {
        auto kern = seg_run_kernel<T, PtrT, LPR, CPL, kWeight, 1, kInFlight>;
        if (smem > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        kern<<<grid1, kAggThreads, smem, st>>>(in, ld_in, ptr, idx, n_seg_dev, n_seg_host, w, run_len, d, sc.head2, sc.tail2,
                                               sc.win_info, sc.cap_runs, seg_of, o);
    } else {
        auto kern = seg_run_kernel<T, PtrT, LPR, CPL, kWeight, 0, kInFlight>;
        if (smem > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        kern<<<grid1, kAggThreads, smem, st>>>(in, ld_in, ptr, idx, n_seg_dev, n_seg_host, w, run_len, d, sc.head2, sc.tail2,
                                               sc.win_info, sc.cap_runs, seg_of, o);
    }
    tap_end(TAP_SEG_L1, st);
    const int64_t window_blocks = std::min<int64_t>(ceil_div(sc.n_windows, kFinalWindows), 148 * 16);
    const int64_t empty_blocks = std::min<int64_t>(ceil_div(cap_seg > 0 ? cap_seg : 1, kAggThreads), 148 * 8);
    tap_begin(TAP_SEG_L3, st);
    note_launch();
    seg_final_kernel<T, PtrT><<<(unsigned)(window_blocks + empty_blocks), kAggThreads, 0, st>>>(
        ptr, n_seg_dev, n_seg_host, run_len, sc.runs_per_window, d, sc.head2, sc.tail2, sc.win_info, sc.n_windows,
        window_blocks, o);
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
