// Building blocks shared by the sampler and the graph ingest: single-pass prefix sums across thread
// blocks, and a stable least-significant-digit radix sort of (int32 key, int32 value) pairs (counts per
// tile, scan over tiles, scatter: three launches per digit).
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
// Stable LSD radix sort of (key = col, value = block position), three launches per digit and no
// waiting between thread blocks: (1) digit counts of every tile of kSortTile consecutive elements,
// (2) per digit an exclusive scan of those counts over the tiles, (3) the scatter: a block ranks
// the equal digits of its tile in element order (per warp by match_any, then across warps) and
// places them at  start of the digit's bin (digit counts of the whole array, known beforehand)
// + count of that digit in the tiles before it + rank.
// ---------------------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(kSortThreads)
tile_hist_kernel(const int32_t *__restrict__ keys, const int32_t *__restrict__ counts, int shift,
                 int32_t *__restrict__ thist)
{
    constexpr int R = 1 << BITS;
    constexpr int W = kSortThreads / 32;
    __shared__ int32_t h[W][R];                  // one histogram per warp: fewer colliding atomics
    const int32_t n = counts[CNT_EDGES];
    const int64_t n_live = ((int64_t)n + kSortTile - 1) / kSortTile;
    const int warp = threadIdx.x >> 5;
    for (int64_t tile = blockIdx.x; tile < n_live; tile += gridDim.x) {
        for (int d = threadIdx.x; d < W * R; d += kSortThreads) (&h[0][0])[d] = 0;
        __syncthreads();
        const int64_t base = tile * kSortTile;
#pragma unroll
        for (int k = 0; k < kSortItems; ++k) {
            const int64_t idx = base + k * kSortThreads + threadIdx.x;
            if (idx < n) atomicAdd(&h[warp][(keys[idx] >> shift) & (R - 1)], 1);
        }
        __syncthreads();
        for (int d = threadIdx.x; d < R; d += kSortThreads) {
            int32_t c = 0;
#pragma unroll
            for (int w = 0; w < W; ++w) c += h[w][d];
            thist[tile * R + d] = c;
        }
        __syncthreads();
    }
}

// thist[tile][d] <- sum of thist[tile'][d] over tile' < tile; one block per digit d
template <int BITS>
__global__ void __launch_bounds__(kSortThreads)
tile_scan_kernel(const int32_t *__restrict__ counts, int32_t *__restrict__ thist)
{
    constexpr int R = 1 << BITS;
    __shared__ int32_t scan_sm[kSortThreads / 32 + 1];
    const int32_t n = counts[CNT_EDGES];
    const int64_t n_live = ((int64_t)n + kSortTile - 1) / kSortTile;
    const int d = blockIdx.x;
    int32_t carry = 0;
    for (int64_t t0 = 0; t0 < n_live; t0 += kSortThreads) {
        const int64_t t = t0 + threadIdx.x;
        const int32_t v = t < n_live ? thist[t * R + d] : 0;
        int32_t tot;
        const int32_t ex = block_exclusive_scan<kSortThreads, int32_t>(v, tot, scan_sm);
        if (t < n_live) thist[t * R + d] = carry + ex;
        carry += tot;
    }
}

template <int BITS>
__global__ void __launch_bounds__(kSortThreads)
sort_pass_kernel(const int32_t *__restrict__ keys_in, const int32_t *__restrict__ vals_in,
                 const int32_t *__restrict__ counts, int shift, const unsigned *__restrict__ ghist,
                 const int32_t *__restrict__ thist, int32_t *__restrict__ keys_out, int32_t *__restrict__ vals_out)
{
    constexpr int R = 1 << BITS;
    constexpr int W = kSortThreads / 32;
    __shared__ int32_t wc[W][R];                 // per-warp digit counts, then start offsets
    __shared__ int32_t bin_base[R];
    __shared__ int32_t scan_sm[kSortThreads / 32 + 1];
    const int64_t tile = blockIdx.x;
    const int32_t n = counts[CNT_EDGES];
    if (tile * kSortTile >= n) return;
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
    const int64_t wbase = tile * kSortTile + (int64_t)warp * (32 * kSortItems);
    int32_t key[kSortItems], val[kSortItems], rank[kSortItems];
    // all loads first: the warp barrier inside the ranking loop would otherwise keep every round's load behind it
#pragma unroll
    for (int k = 0; k < kSortItems; ++k) {
        const int64_t idx = wbase + k * 32 + lane;
        const bool ok = idx < n;
        key[k] = ok ? keys_in[idx] : 0;
        val[k] = ok ? (vals_in ? vals_in[idx] : (int32_t)idx) : 0;
    }
#pragma unroll
    for (int k = 0; k < kSortItems; ++k) {
        const int64_t idx = wbase + k * 32 + lane;
        const bool ok = idx < n;
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
    // per digit: where the elements of each warp start
    for (int d = threadIdx.x; d < R; d += kSortThreads) {
        int32_t run = bin_base[d] + thist[tile * R + d];
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

// Buffers of one sort: two ping-pong pairs, the digit counts of the whole array (filled before the sort) and
// the per-tile digit counts (written before they are read: no zeroing needed).
struct RadixScratch {
    int32_t *keys[2], *vals[2];        // [n] each
    unsigned *ghist;                   // [kMaxPasses x kMaxRadix]
    int32_t *thist;                    // [tiles x radix], reused by every pass
    int64_t tiles;
};

constexpr size_t radix_thist_bytes(int64_t tiles) { return sizeof(int32_t) * (size_t)kMaxRadix * (size_t)tiles; }

template <int BITS>
static inline void radix_pass(const int32_t *kin, const int32_t *vin, int32_t *counts, int n_tiles, int shift,
                              const unsigned *ghist, int32_t *thist, int32_t *kout, int32_t *vout, cudaStream_t st)
{
    const int hist_grid = n_tiles < 8 * 148 ? n_tiles : 8 * 148;
    note_launch();
    tile_hist_kernel<BITS><<<hist_grid, kSortThreads, 0, st>>>(kin, counts, shift, thist);
    note_launch();
    tile_scan_kernel<BITS><<<1 << BITS, kSortThreads, 0, st>>>(counts, thist);
    note_launch();
    sort_pass_kernel<BITS><<<n_tiles, kSortThreads, 0, st>>>(kin, vin, counts, shift, ghist, thist, kout, vout);
}

// Sorts (keys, vals) by key, stable; vals == nullptr means "value = position".  counts[CNT_EDGES] holds the
// number of elements (device).  ghist must already hold the digit counts.
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
        if (sp.bits == 8)
            radix_pass<8>(kin, vin, counts, n_tiles, p * sp.bits, rs.ghist + p * kMaxRadix, rs.thist, kout, vout, st);
        else
            radix_pass<10>(kin, vin, counts, n_tiles, p * sp.bits, rs.ghist + p * kMaxRadix, rs.thist, kout, vout, st);
        kin = kout;
        vin = vout;
    }
}

}  // namespace e2egrec
