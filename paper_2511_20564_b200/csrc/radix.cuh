// Building blocks shared by the sampler and the graph ingest: single-pass prefix sums across thread
// blocks, and a stable least-significant-digit radix sort of (int32 key, int32 value) pairs with one
// launch per digit.
#pragma once

#include "common.cuh"
#include "scan.cuh"

namespace e2egrec {

constexpr int kSortThreads = 256;
constexpr int kSortItems = 16;
constexpr int kSortTile = kSortThreads * kSortItems;
constexpr int kMaxRadix = 1024;
constexpr int kMaxPasses = 4;

// ---------------------------------------------------------------------------------------
// Single-pass prefix sums across thread blocks ("chained scan"): every tile publishes its own sum,
// then looks back over the tiles before it until it meets one whose full prefix is known.  Tiles
// are handed out by an atomic ticket, so a tile only ever waits for tiles that already run.  Every
// wait is bounded; when the bound is hit the status word gets E2EGREC_DEV_TIMEOUT and the tile goes
// on with what it has.
// ---------------------------------------------------------------------------------------
constexpr unsigned long long kChainAgg = 1ull << 62, kChainPrefix = 2ull << 62, kChainMask = (1ull << 62) - 1;
constexpr int kChainSpinLimit = 1 << 22;

__device__ inline unsigned long long chain_read(const unsigned long long *slot)
{
    return *reinterpret_cast<const volatile unsigned long long *>(slot);
}

// Called by all threads of the block.  Returns the sum of the aggregates of tiles 0 .. tile-1.
__device__ inline long long chain_lookback(unsigned long long *state, int tile, long long aggregate, int32_t *status,
                                           long long *bcast)
{
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        long long excl = 0;
        if (lane == 0) atomicExch(&state[tile], (tile == 0 ? kChainPrefix : kChainAgg) | (unsigned long long)aggregate);
        if (tile > 0) {
            int p = tile - 1;
            bool done = false;
            while (!done) {
                const int idx = p - lane;
                unsigned long long v = kChainPrefix;                 // before tile 0: an empty prefix
                bool timed_out = false;
                for (int spin = 0;; ++spin) {
                    if (idx >= 0) v = chain_read(&state[idx]);
                    if (__all_sync(0xffffffffu, (v >> 62) != 0)) break;
                    if (spin >= kChainSpinLimit) { timed_out = true; break; }
                }
                timed_out = __any_sync(0xffffffffu, timed_out);
                const unsigned pref = __ballot_sync(0xffffffffu, (v >> 62) == 2);
                const int first = pref ? __ffs(pref) - 1 : 31;
                long long c = lane <= first ? (long long)(v & kChainMask) : 0;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
                excl += c;
                if (timed_out) {
                    if (lane == 0) atomicOr(reinterpret_cast<unsigned *>(status), E2EGREC_DEV_TIMEOUT);
                    done = true;
                } else if (pref) {
                    done = true;
                } else {
                    p -= 32;
                }
            }
            if (lane == 0) atomicExch(&state[tile], kChainPrefix | (unsigned long long)(excl + aggregate));
        }
        if (lane == 0) *bcast = excl;
    }
    __syncthreads();
    return *bcast;
}

__device__ inline int chain_ticket(unsigned *ticket, int *bcast)
{
    if (threadIdx.x == 0) *bcast = (int)atomicAdd(ticket, 1u);
    __syncthreads();
    return *bcast;
}


// ---------------------------------------------------------------------------------------
// Stable LSD radix sort of (key = col, value = block position), one launch per digit.  A block owns
// a tile of kSortTile consecutive elements, ranks equal digits in element order (per warp by
// match_any, then across warps), and finds where its elements of each digit start from the digit's
// global start (digit counts of the whole array, known beforehand) plus a per-digit chained scan
// over the tiles before it.
// ---------------------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(kSortThreads)
sort_pass_kernel(const int32_t *__restrict__ keys_in, const int32_t *__restrict__ vals_in,
                 int32_t *__restrict__ counts, int shift, const unsigned *__restrict__ ghist, int n_tiles,
                 unsigned long long *__restrict__ state, unsigned *ticket, int32_t *__restrict__ keys_out,
                 int32_t *__restrict__ vals_out)
{
    constexpr int R = 1 << BITS;
    constexpr int W = kSortThreads / 32;
    __shared__ int32_t wc[W][R];                 // per-warp digit counts, then start offsets
    __shared__ int32_t bin_base[R];
    __shared__ int32_t scan_sm[kSortThreads / 32 + 1];
    __shared__ int tile_s;
    const int tile = chain_ticket(ticket, &tile_s);
    const int32_t n = counts[CNT_EDGES];
    if ((int64_t)tile * kSortTile >= n) return;
    for (int d = threadIdx.x; d < W * R; d += kSortThreads) (&wc[0][0])[d] = 0;
    // start of every digit's bin: exclusive scan of the global digit counts
    {
        int32_t carry = 0;
        for (int d0 = 0; d0 < R; d0 += kSortThreads) {
            const int d = d0 + threadIdx.x;
            const int32_t v = d < R ? (int32_t)ghist[d] : 0;
            int32_t tot;
            const int32_t ex = block_exclusive_scan<kSortThreads, int32_t>(v, tot, scan_sm);
            if (d < R) bin_base[d] = carry + ex;
            carry += tot;
        }
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t wbase = (int64_t)tile * kSortTile + (int64_t)warp * (32 * kSortItems);
    int32_t key[kSortItems], val[kSortItems], rank[kSortItems];
#pragma unroll
    for (int k = 0; k < kSortItems; ++k) {
        const int64_t idx = wbase + k * 32 + lane;
        const bool ok = idx < n;
        key[k] = ok ? keys_in[idx] : 0;
        val[k] = ok ? (vals_in ? vals_in[idx] : (int32_t)idx) : 0;
        const uint32_t digit = ok ? (uint32_t)((key[k] >> shift) & (R - 1)) : 0xFFFFFFFFu;
        const uint32_t peers = __match_any_sync(0xffffffffu, digit);
        const int leader = __ffs(peers) - 1;
        int32_t base = 0;
        if (ok && lane == leader) {
            base = wc[warp][digit];
            wc[warp][digit] = base + __popc(peers);
        }
        base = __shfl_sync(0xffffffffu, base, leader);
        rank[k] = base + __popc(peers & ((1u << lane) - 1u));
        __syncwarp();
    }
    __syncthreads();
    // per digit: publish this tile's count, then a chained look-back over earlier tiles, then warp start offsets
    constexpr int DPT = (R + kSortThreads - 1) / kSortThreads;
    int32_t cnt[DPT];
#pragma unroll
    for (int q = 0; q < DPT; ++q) {
        const int d = threadIdx.x + q * kSortThreads;
        cnt[q] = 0;
        if (d < R) {
#pragma unroll
            for (int w = 0; w < W; ++w) cnt[q] += wc[w][d];
            atomicExch(&state[(size_t)d * n_tiles + tile], (tile == 0 ? kChainPrefix : kChainAgg) | (unsigned long long)cnt[q]);
        }
    }
    // look-back for all of this thread's digits together: a batch of earlier tiles per digit is read at
    // once, then taken in order; an entry that is not published yet is polled (bounded) before going on
    long long excl[DPT];
    int next_p[DPT];
    bool timed_out = false;
#pragma unroll
    for (int q = 0; q < DPT; ++q) {
        excl[q] = 0;
        next_p[q] = (threadIdx.x + q * kSortThreads < R && tile > 0) ? tile - 1 : -1;
    }
    for (;;) {
        bool any = false;
#pragma unroll
        for (int q = 0; q < DPT; ++q) any = any || next_p[q] >= 0;
        if (!any || timed_out) break;
        constexpr int kBatch = 8;
        unsigned long long v[DPT][kBatch];
#pragma unroll
        for (int q = 0; q < DPT; ++q) {
            const unsigned long long *st = state + (size_t)(threadIdx.x + q * kSortThreads) * n_tiles;
#pragma unroll
            for (int j = 0; j < kBatch; ++j) v[q][j] = next_p[q] - j >= 0 ? chain_read(&st[next_p[q] - j]) : kChainPrefix;
        }
#pragma unroll
        for (int q = 0; q < DPT; ++q) {
            if (next_p[q] < 0) continue;
            const unsigned long long *st = state + (size_t)(threadIdx.x + q * kSortThreads) * n_tiles;
            bool found = false;
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                if (found || timed_out) continue;
                unsigned long long x = v[q][j];
                for (int spin = 0; (x >> 62) == 0; ++spin) {
                    if (spin >= kChainSpinLimit) { timed_out = true; break; }
                    x = chain_read(&st[next_p[q] - j]);
                }
                if (timed_out) continue;
                excl[q] += (long long)(x & kChainMask);
                if ((x >> 62) == 2) found = true;
            }
            next_p[q] = found ? -1 : next_p[q] - kBatch;
        }
    }
    if (timed_out) atomicOr(reinterpret_cast<unsigned *>(&counts[CNT_STATUS]), E2EGREC_DEV_TIMEOUT);
#pragma unroll
    for (int q = 0; q < DPT; ++q) {
        const int d = threadIdx.x + q * kSortThreads;
        if (d >= R) continue;
        if (tile > 0) atomicExch(&state[(size_t)d * n_tiles + tile], kChainPrefix | (unsigned long long)(excl[q] + cnt[q]));
        int32_t run = bin_base[d] + (int32_t)excl[q];
#pragma unroll
        for (int w = 0; w < W; ++w) {
            const int32_t c2 = wc[w][d];
            wc[w][d] = run;
            run += c2;
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kSortItems; ++k) {
        const int64_t idx = wbase + k * 32 + lane;
        if (idx < n) {
            const int32_t pos = wc[warp][(key[k] >> shift) & (R - 1)] + rank[k];
            keys_out[pos] = key[k];
            vals_out[pos] = val[k];
        }
    }
}


struct SortPlan { int bits, passes; };

static inline SortPlan sort_plan(int32_t cap_src)
{
    int key_bits = 1;
    while (key_bits < 31 && (1ll << key_bits) < (int64_t)cap_src) ++key_bits;
    if (key_bits <= 8) return {8, 1};
    if (key_bits <= 10) return {10, 1};
    if (key_bits <= 16) return {8, 2};
    if (key_bits <= 20) return {10, 2};
    if (key_bits <= 24) return {8, 3};
    if (key_bits <= 30) return {10, 3};
    return {8, 4};
}

// csc_col / csc_eid = columns and positions of the block entries ordered by (col, position).

// Digit counts of a key array for every pass of the sort (what sort_pass_kernel needs beforehand).
static __global__ void __launch_bounds__(256)
key_hist_kernel(const int32_t *__restrict__ keys, const int32_t *__restrict__ counts, int bits, int passes,
                unsigned *__restrict__ ghist)
{
    __shared__ unsigned h[kMaxPasses * kMaxRadix];
    const int R = 1 << bits;
    for (int d = threadIdx.x; d < passes * R; d += 256) h[d] = 0;
    __syncthreads();
    const int32_t n = counts[CNT_EDGES];
    for (int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x; e < n; e += (int64_t)gridDim.x * 256) {
        const int32_t c = keys[e];
        for (int p = 0; p < passes; ++p) atomicAdd(&h[p * R + ((c >> (p * bits)) & (R - 1))], 1u);
    }
    __syncthreads();
    for (int d = threadIdx.x; d < passes * R; d += 256)
        if (h[d]) atomicAdd(&ghist[(d / R) * kMaxRadix + (d % R)], h[d]);
}

// Buffers of one sort: two ping-pong pairs and the zeroed arena (tickets, digit counts, tile states).
struct RadixScratch {
    int32_t *keys[2], *vals[2];        // [n] each
    unsigned *tickets;                 // [kMaxPasses]
    unsigned *ghist;                   // [kMaxPasses x kMaxRadix]
    unsigned long long *state;         // [kMaxPasses x kMaxRadix x tiles]
    int64_t tiles;
};

// Sorts (keys, vals) by key, stable; vals == nullptr means "value = position".  counts[CNT_EDGES] holds the
// number of elements (device).  ghist must already hold the digit counts; tickets / state must be zero.
static inline void radix_sort_pairs(const int32_t *keys, const int32_t *vals, int32_t *counts, int64_t cap,
                                    int32_t *keys_out, int32_t *vals_out, const SortPlan &sp, const RadixScratch &rs,
                                    cudaStream_t st)
{
    const int n_tiles = (int)ceil_div(cap > 0 ? cap : 1, kSortTile);
    const int32_t *kin = keys;
    const int32_t *vin = vals;
    for (int p = 0; p < sp.passes; ++p) {
        const bool last = p == sp.passes - 1;
        int32_t *kout = last ? keys_out : rs.keys[p & 1];
        int32_t *vout = last ? vals_out : rs.vals[p & 1];
        unsigned long long *state = rs.state + (size_t)p * kMaxRadix * (size_t)rs.tiles;
        note_launch();
        if (sp.bits == 8)
            sort_pass_kernel<8><<<n_tiles, kSortThreads, 0, st>>>(kin, vin, counts, p * sp.bits, rs.ghist + p * kMaxRadix, n_tiles,
                                                                 state, rs.tickets + p, kout, vout);
        else
            sort_pass_kernel<10><<<n_tiles, kSortThreads, 0, st>>>(kin, vin, counts, p * sp.bits, rs.ghist + p * kMaxRadix, n_tiles,
                                                                  state, rs.tickets + p, kout, vout);
        kin = kout;
        vin = vout;
    }
}

}  // namespace e2egrec
