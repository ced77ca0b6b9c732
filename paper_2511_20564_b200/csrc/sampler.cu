// k-hop neighbour sampling, frontier relabelling and block transposition.
//
// Everything here is integer work whose result is fixed by (graph, seeds, fanouts,
// seed, step): Philox4x32-10 draws keyed by the global node id, a bitmap + rank scan
// that yields the new frontier nodes in ascending id order, and a stable least-
// significant-digit radix sort that orders the transposed block by (source, position).
// All element counts stay on the device; grids are sized for the worst case and the
// surplus threads leave at once.
#include "common.cuh"
#include "scan.cuh"
#include "internal.cuh"
#include "radix.cuh"

#include <algorithm>

namespace e2egrec {

// ---------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies with a
// Weyl key schedule.
// ---------------------------------------------------------------------------------------
__device__ inline uint4 philox4x32_10(uint4 c, uint2 k)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
        k.x += 0x9E3779B9u;
        k.y += 0xBB67AE85u;
    }
    return c;
}

// ---------------------------------------------------------------------------------------
// Scratch layout (host and device agree through this struct).
// ---------------------------------------------------------------------------------------
constexpr int kDstTile = 64;           // destinations per block of the sampling kernel
constexpr int kDstThreads = 256;       // its threads: one per destination for the counts, then all of them draw
constexpr int kWordTile = 2048;        // bitmap words per block of the frontier kernel

// Everything one block transposition (radix sort by column + offsets) needs; one lane per hop, so that the
// transposition of hop h can run beside the sampling of hop h+1.
struct SortLane {
    int32_t  *edge_row;    // [max cap_edges]   destination of each block entry
    int32_t  *keys[2];     // [max cap_edges]   radix sort ping-pong
    int32_t  *vals[2];
    unsigned *ghist;                   // [kMaxPasses x kMaxRadix] digit counts of the whole key array (zeroed before relabel)
    int32_t  *thist;                   // [sort tiles x kMaxRadix] digit counts per tile of the pass that runs
};

struct SamplerScratch {
    uint32_t *step_offset; // [1]         added to the `step` argument of every call (see e2egrec_sampler_set_step)
    int32_t  *local_id;    // [n_nodes]   -1 when idle, else position in the current frontier
    uint32_t *bitmap;      // [n_words]   newly reached nodes of the hop in progress; 0 when idle
    // chain arena of the sampling / frontier kernels, zeroed at the start of every hop
    char     *arena;
    size_t    arena_bytes;
    unsigned *tickets;                 // [2]
    unsigned long long *state_dst;     // [dst tiles]
    unsigned long long *state_words;   // [word tiles]
    SortLane  lane[kMaxHops];
    int64_t   sort_tiles;
    size_t    bytes;
    int64_t   n_words;
};

static SamplerScratch carve(int64_t n_nodes, int64_t max_dst, int64_t max_src, int64_t max_edges, void *base)
{
    (void)max_src;
    SamplerScratch s;
    s.n_words = ceil_div(n_nodes, 32);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        char *p = base ? static_cast<char *>(base) + off : nullptr;
        off += align_up(bytes, 256);
        return p;
    };
    s.sort_tiles = ceil_div(max_edges > 0 ? max_edges : 1, kSortTile);
    s.step_offset = (uint32_t *)take(256);
    s.local_id = (int32_t *)take(sizeof(int32_t) * (size_t)n_nodes);
    s.bitmap = (uint32_t *)take(sizeof(uint32_t) * (size_t)s.n_words);
    size_t begin = off;
    s.arena = base ? static_cast<char *>(base) + off : nullptr;
    s.tickets = (unsigned *)take(256);
    s.state_dst = (unsigned long long *)take(8 * (size_t)(ceil_div(max_dst > 0 ? max_dst : 1, kDstTile) + 1));
    s.state_words = (unsigned long long *)take(8 * (size_t)(ceil_div(s.n_words > 0 ? s.n_words : 1, kWordTile) + 1));
    s.arena_bytes = off - begin;
    for (int h = 0; h < kMaxHops; ++h) {
        SortLane &l = s.lane[h];
        l.edge_row = (int32_t *)take(sizeof(int32_t) * (size_t)(max_edges + 1));
        for (int i = 0; i < 2; ++i) l.keys[i] = (int32_t *)take(sizeof(int32_t) * (size_t)(max_edges + 1));
        for (int i = 0; i < 2; ++i) l.vals[i] = (int32_t *)take(sizeof(int32_t) * (size_t)(max_edges + 1));
        l.ghist = (unsigned *)take(sizeof(unsigned) * kMaxPasses * kMaxRadix);
        l.thist = (int32_t *)take(radix_thist_bytes(s.sort_tiles));
    }
    s.bytes = off;
    return s;
}

// ---------------------------------------------------------------------------------------
// Kernels
// ---------------------------------------------------------------------------------------
__global__ void fill_i32_kernel(int32_t *p, int64_t n, int32_t v)
{
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        p[i] = v;
}

// Seeds become the first frontier: local id = position in the batch.
__global__ void seed_init_kernel(const int32_t *__restrict__ seeds, int32_t n_seeds, int64_t n_nodes,
                                 int32_t *__restrict__ local_id, int32_t *counts0)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        counts0[CNT_DST] = n_seeds;
        counts0[CNT_STATUS] = 0;
    }
    if (i >= n_seeds) return;
    const int32_t u = seeds[i];
    if ((uint32_t)u < (uint64_t)n_nodes) local_id[u] = i;
}

// One hop of sampling in one launch.  A block owns kDstTile destinations: |S(u)| = min(deg, fanout) per
// destination, a chained scan for the block's offset into the entry arrays, then one thread per
// (destination, slot).  Slot j of node u at hop h draws with the counter (j/2, u, (1<<8)|h, step) and
// key (seed lo, seed hi); words 2(j%2), 2(j%2)+1 form r and the picked row position is
// floor(r * deg / 2^64); with running sums of integer edge weights (g_cum) it is the first entry of the row
// whose running sum exceeds floor(r * total / 2^64).  deg <= fanout copies the row instead.  Sampled nodes
// that are not yet in the frontier are marked in the bitmap.
__global__ void __launch_bounds__(kDstThreads)
hop_sample_kernel(const int64_t *__restrict__ g_indptr, const int32_t *__restrict__ g_indices,
                  const uint64_t *__restrict__ g_cum, int64_t n_nodes,
                  const int32_t *__restrict__ dst_nodes, const int32_t *n_dst_ptr, int32_t cap_dst, int32_t cap_edges,
                  int32_t fanout, int32_t hop, uint32_t seed_lo, uint32_t seed_hi, uint32_t step_arg,
                  const uint32_t *__restrict__ step_offset, int first_hop, int32_t *__restrict__ counts,
                  int32_t *__restrict__ blk_indptr, float *__restrict__ inv_cnt, int32_t *__restrict__ src_nodes,
                  int32_t *__restrict__ nbr_global, int32_t *__restrict__ edge_row,
                  const int32_t *__restrict__ local_id, uint32_t *__restrict__ bitmap, unsigned *ticket,
                  unsigned long long *state)
{
    __shared__ int32_t off[kDstTile + 1];
    __shared__ int32_t node[kDstTile];
    __shared__ int64_t gbeg_s[kDstTile];
    __shared__ int64_t deg_s[kDstTile];
    __shared__ int32_t scan_sm[kDstThreads / 32 + 1];
    __shared__ long long bcast;
    __shared__ int tile_s;
    const int tile = chain_ticket(ticket, &tile_s);
    int32_t n_dst = *n_dst_ptr;
    const bool over = n_dst > cap_dst;
    if (over) n_dst = cap_dst;
    if (tile == 0 && threadIdx.x == 0) {
        counts[CNT_DST] = n_dst;
        if (!first_hop) counts[CNT_STATUS] = 0;
        if (over) atomicOr((unsigned *)&counts[CNT_STATUS], E2EGREC_DEV_CAPACITY);
    }
    const int64_t i0 = (int64_t)tile * kDstTile;
    if (i0 >= n_dst) {
        if (n_dst == 0 && tile == 0 && threadIdx.x == 0) { blk_indptr[0] = 0; counts[CNT_EDGES] = 0; }
        return;
    }
    const int64_t i = i0 + threadIdx.x;
    int32_t c = 0;
    if (threadIdx.x < kDstTile && i < n_dst) {
        int32_t u = dst_nodes[i];
        int64_t gb = 0, deg = 0;
        if ((uint32_t)u < (uint64_t)n_nodes) {
            gb = g_indptr[u];
            deg = g_indptr[u + 1] - gb;
        } else {
            atomicOr((unsigned *)&counts[CNT_STATUS], E2EGREC_DEV_RANGE);
            u = 0;
        }
        c = deg < fanout ? (int32_t)deg : fanout;
        node[threadIdx.x] = u;
        gbeg_s[threadIdx.x] = gb;
        deg_s[threadIdx.x] = deg;
        inv_cnt[i] = c > 0 ? 1.0f / (float)c : 0.0f;
        src_nodes[i] = u;
    }
    int32_t tile_total;
    const int32_t ex = block_exclusive_scan<kDstThreads, int32_t>(c, tile_total, scan_sm);
    if (threadIdx.x < kDstTile) off[threadIdx.x] = ex;
    if (threadIdx.x == 0) off[kDstTile] = tile_total;
    const long long base = chain_lookback(state, tile, tile_total, &counts[CNT_STATUS], &bcast);   // syncs the block
    if (threadIdx.x < kDstTile && i < n_dst) blk_indptr[i] = (int32_t)(base + ex);
    const bool last_tile = i0 + kDstTile >= n_dst;
    if (last_tile && threadIdx.x == 0) {
        const long long total = base + tile_total;
        blk_indptr[n_dst] = (int32_t)total;
        counts[CNT_EDGES] = total > cap_edges ? cap_edges : (int32_t)total;
        if (total > cap_edges) atomicOr((unsigned *)&counts[CNT_STATUS], E2EGREC_DEV_CAPACITY);
    }
    const uint32_t step = step_arg + *step_offset;
    // four slots per thread and round, so that the loads of the graph entry, of the frontier position and of
    // the bitmap word are in flight for all four before any of them is needed
    constexpr int S = 4;
    for (int32_t sl0 = threadIdx.x; sl0 < tile_total; sl0 += kDstThreads * S) {
        int rr[S];
        long long e[S];
        int64_t src[S];
        bool ok[S];
#pragma unroll
        for (int q = 0; q < S; ++q) {
            const int32_t sl = sl0 + q * kDstThreads;
            ok[q] = sl < tile_total;
            rr[q] = 0;
            e[q] = 0;
            src[q] = 0;
            if (!ok[q]) continue;
            int lo = 0, hi = kDstTile;               // largest r with off[r] <= sl
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (off[mid] <= sl) lo = mid; else hi = mid;
            }
            rr[q] = lo;
            const int32_t j = sl - off[lo];
            e[q] = base + sl;
            if (e[q] >= cap_edges) { ok[q] = false; continue; }
            const int64_t deg = deg_s[lo];
            int64_t pos = j;
            if (deg > fanout) {
                const uint4 r4 = philox4x32_10(make_uint4((uint32_t)(j >> 1), (uint32_t)node[lo], (1u << 8) | (uint32_t)hop, step),
                                               make_uint2(seed_lo, seed_hi));
                const uint64_t rnd = (j & 1) ? (((uint64_t)r4.w << 32) | r4.z) : (((uint64_t)r4.y << 32) | r4.x);
                const uint64_t *cum = g_cum ? g_cum + gbeg_s[lo] : nullptr;
                const uint64_t total = cum ? cum[deg - 1] : 0;
                if (total > 0) {
                    // weighted draw: the first entry of the row whose running sum exceeds t
                    const uint64_t t = __umul64hi(rnd, total);
                    int64_t a = 0, b = deg - 1;                 // cum[b] > t always
                    while (a < b) {
                        const int64_t mid = (a + b) >> 1;
                        if (cum[mid] > t) b = mid; else a = mid + 1;
                    }
                    pos = a;
                } else {
                    pos = (int64_t)__umul64hi(rnd, (uint64_t)deg);
                }
            }
            src[q] = gbeg_s[lo] + pos;
        }
        int32_t v[S];
#pragma unroll
        for (int q = 0; q < S; ++q) v[q] = ok[q] ? __ldg(&g_indices[src[q]]) : 0;
        int32_t lid[S];
#pragma unroll
        for (int q = 0; q < S; ++q) {
            if (ok[q] && (uint32_t)v[q] >= (uint64_t)n_nodes) {
                atomicOr((unsigned *)&counts[CNT_STATUS], E2EGREC_DEV_RANGE);
                v[q] = node[rr[q]];
            }
            lid[q] = ok[q] ? local_id[v[q]] : 0;
        }
        uint32_t word[S];
#pragma unroll
        for (int q = 0; q < S; ++q)   // hubs are sampled thousands of times per hop: look before the atomic
            word[q] = (ok[q] && lid[q] < 0) ? *reinterpret_cast<volatile uint32_t *>(&bitmap[v[q] >> 5]) : 0xFFFFFFFFu;
#pragma unroll
        for (int q = 0; q < S; ++q) {
            if (!ok[q]) continue;
            nbr_global[e[q]] = v[q];
            edge_row[e[q]] = (int32_t)(i0 + rr[q]);
            if (lid[q] < 0 && !(word[q] & (1u << (v[q] & 31)))) atomicOr(&bitmap[v[q] >> 5], 1u << (v[q] & 31));
        }
    }
}

// New frontier nodes in one launch: a block owns kWordTile bitmap words, counts their set bits, takes
// its rank offset from a chained scan and hands out local ids n_dst, n_dst+1, ... in ascending id order.
// The bitmap returns to 0.
__global__ void __launch_bounds__(256)
frontier_kernel(uint32_t *__restrict__ bitmap, int64_t n_words, int32_t *__restrict__ counts, int32_t cap_src,
                int32_t *__restrict__ local_id, int32_t *__restrict__ src_nodes, unsigned *ticket,
                unsigned long long *state)
{
    constexpr int WPT = kWordTile / 256;
    __shared__ int32_t scan_sm[256 / 32 + 1];
    __shared__ long long bcast;
    __shared__ int tile_s;
    const int tile = chain_ticket(ticket, &tile_s);
    const int64_t w0 = (int64_t)tile * kWordTile + (int64_t)threadIdx.x * WPT;
    uint32_t bits[WPT];
    int32_t c = 0;
#pragma unroll
    for (int k = 0; k < WPT; ++k) {
        bits[k] = w0 + k < n_words ? bitmap[w0 + k] : 0u;
        c += __popc(bits[k]);
    }
    int32_t tile_total;
    const int32_t ex = block_exclusive_scan<256, int32_t>(c, tile_total, scan_sm);
    const long long base = chain_lookback(state, tile, tile_total, &counts[CNT_STATUS], &bcast);
    const int32_t n_dst = counts[CNT_DST];
    const bool last_tile = (int64_t)(tile + 1) * kWordTile >= n_words;
    if (last_tile && threadIdx.x == 0) {
        long long n_src = (long long)n_dst + base + tile_total;
        if (n_src > cap_src) { n_src = cap_src; atomicOr((unsigned *)&counts[CNT_STATUS], E2EGREC_DEV_CAPACITY); }
        counts[CNT_SRC] = (int32_t)n_src;
    }
    long long r = (long long)n_dst + base + ex;
#pragma unroll
    for (int k = 0; k < WPT; ++k) {
        uint32_t b = bits[k];
        if (!b) continue;
        bitmap[w0 + k] = 0;
        while (b) {
            const int bit = __ffs(b) - 1;
            b &= b - 1;
            const int32_t id = (int32_t)((w0 + k) * 32 + bit);
            if (r < cap_src) {
                local_id[id] = (int32_t)r;
                src_nodes[r] = id;
            }
            ++r;
        }
    }
}

// col[e] = position of the sampled node in the frontier, and the digit counts of the whole col array
// for every pass of the radix sort that follows.
__global__ void __launch_bounds__(256)
relabel_kernel(const int32_t *__restrict__ nbr_global, const int32_t *__restrict__ local_id,
               const int32_t *__restrict__ counts, int32_t *__restrict__ col, int bits, int passes,
               unsigned *__restrict__ ghist)
{
    __shared__ unsigned h[kMaxPasses * kMaxRadix];
    const int R = 1 << bits;
    for (int d = threadIdx.x; d < passes * R; d += 256) h[d] = 0;
    __syncthreads();
    const int32_t n = counts[CNT_EDGES];
    const int32_t n_src = counts[CNT_SRC];
    for (int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x; e < n; e += (int64_t)gridDim.x * 256) {
        int32_t c = local_id[nbr_global[e]];
        if (c < 0 || c >= n_src) c = 0;              // only after a capacity overrun, which is flagged
        col[e] = c;
        for (int p = 0; p < passes; ++p) atomicAdd(&h[p * R + ((c >> (p * bits)) & (R - 1))], 1u);
    }
    __syncthreads();
    for (int d = threadIdx.x; d < passes * R; d += 256)
        if (h[d]) atomicAdd(&ghist[(d / R) * kMaxRadix + (d % R)], h[d]);
}

__global__ void frontier_release_kernel(const int32_t *__restrict__ src_nodes, const int32_t *__restrict__ counts,
                                        int32_t *__restrict__ local_id)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < counts[CNT_SRC]) local_id[src_nodes[i]] = -1;
}

// csc_ptr[s] = first position whose column is >= s (the columns are sorted), and the destination of
// every transposed entry.
__global__ void csc_finalize_kernel(const int32_t *__restrict__ csc_col, const int32_t *__restrict__ csc_eid,
                                    const int32_t *__restrict__ edge_row, const int32_t *__restrict__ counts,
                                    int32_t *__restrict__ csc_ptr, int32_t *__restrict__ csc_row)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int32_t n = counts[CNT_EDGES], n_src = counts[CNT_SRC];
    if (t < n) csc_row[t] = edge_row[csc_eid[t]];
    if (t <= n_src) {
        int32_t lo = 0, hi = n;                      // lower bound of t in csc_col[0..n)
        while (lo < hi) {
            const int32_t mid = (lo + hi) >> 1;
            if (csc_col[mid] < (int32_t)t) lo = mid + 1; else hi = mid;
        }
        csc_ptr[t] = lo;
    }
}

// Joint step: the endpoints of the training pairs become the seed set.  Every endpoint is marked in the
// bitmap (frontier_kernel then lists the marked ids in ascending order and gives them local ids).
__global__ void pair_mark_kernel(const int32_t *__restrict__ user, const int32_t *__restrict__ item, int32_t n_pairs,
                                 int64_t n_nodes, uint32_t *__restrict__ bitmap, int32_t *__restrict__ counts)
{
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= n_pairs) return;
    const int32_t ids[2] = {user[p], item[p]};
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        if ((uint32_t)ids[k] < (uint64_t)n_nodes) atomicOr(&bitmap[ids[k] >> 5], 1u << (ids[k] & 31));
        else atomicOr((unsigned *)&counts[CNT_STATUS], E2EGREC_DEV_RANGE);
    }
}

// pair_local[e] = seed position of entry e (e < P: the user of pair e, else the item of pair e - P),
// entry_unit[e] = where that entry's gradient row starts inside the tower's input-gradient matrix, in
// 16-byte units, and the digit counts of pair_local for the sort that groups the entries by seed.
__global__ void __launch_bounds__(256)
pair_local_kernel(const int32_t *__restrict__ user, const int32_t *__restrict__ item, int32_t n_pairs, int64_t n_nodes,
                  const int32_t *__restrict__ local_id, int32_t *__restrict__ pair_local,
                  int32_t *__restrict__ entry_unit, int units_per_row, int item_unit_off, int32_t *__restrict__ pcounts,
                  int bits, int passes, unsigned *__restrict__ ghist)
{
    __shared__ unsigned h[kMaxPasses * kMaxRadix];
    const int R = 1 << bits;
    for (int d = threadIdx.x; d < passes * R; d += 256) h[d] = 0;
    __syncthreads();
    if (blockIdx.x == 0 && threadIdx.x == 0) pcounts[CNT_EDGES] = 2 * n_pairs;
    for (int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x; e < 2 * (int64_t)n_pairs; e += (int64_t)gridDim.x * 256) {
        const bool is_item = e >= n_pairs;
        const int32_t pr = (int32_t)(is_item ? e - n_pairs : e);
        const int32_t id = is_item ? item[pr] : user[pr];
        int32_t c = (uint32_t)id < (uint64_t)n_nodes ? local_id[id] : 0;
        if (c < 0) c = 0;
        pair_local[e] = c;
        entry_unit[e] = pr * units_per_row + (is_item ? item_unit_off : 0);
        for (int p = 0; p < passes; ++p) atomicAdd(&h[p * R + ((c >> (p * bits)) & (R - 1))], 1u);
    }
    __syncthreads();
    for (int d = threadIdx.x; d < passes * R; d += 256)
        if (h[d]) atomicAdd(&ghist[(d / R) * kMaxRadix + (d % R)], h[d]);
}

static void sort_by_col(const int32_t *col, int32_t *counts, int32_t cap_edges, int32_t *csc_col, int32_t *csc_eid,
                        const SortPlan &sp, const SortLane &l, int64_t sort_tiles, cudaStream_t st)
{
    RadixScratch rs{};
    rs.keys[0] = l.keys[0]; rs.keys[1] = l.keys[1];
    rs.vals[0] = l.vals[0]; rs.vals[1] = l.vals[1];
    rs.ghist = l.ghist;
    rs.thist = l.thist;
    rs.tiles = sort_tiles;
    radix_sort_pairs(col, nullptr, counts, cap_edges, csc_col, csc_eid, sp, rs, st);
}

static inline unsigned grid_for(int64_t n, int threads) { return (unsigned)ceil_div(n > 0 ? n : 1, threads); }

size_t sampler_scratch_bytes(int64_t n_nodes, int64_t max_dst, int64_t max_src, int64_t max_edges)
{
    return carve(n_nodes, max_dst, max_src, max_edges, nullptr).bytes;
}

}  // namespace e2egrec

using namespace e2egrec;

// ---------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------
int32_t e2egrec::khop_caps(int64_t n_nodes, int32_t n_seeds, int32_t n_hops, const int32_t *fanouts,
                         int32_t *cap_dst, int32_t *cap_src, int32_t *cap_edges)
{
    if (!fanouts || !cap_dst || !cap_src || !cap_edges) return E2EGREC_ERR_NULL;
    if (n_nodes < 0 || n_seeds < 0) return E2EGREC_ERR_ARG;
    if (n_nodes >= (1ll << 31) || n_hops > kMaxHops) return E2EGREC_ERR_UNSUPPORTED;
    if (n_hops < 1) return E2EGREC_ERR_ARG;
    int64_t dst = n_seeds;
    for (int h = 0; h < n_hops; ++h) {
        if (fanouts[h] < 1) return E2EGREC_ERR_ARG;
        if (fanouts[h] > kMaxFanout) return E2EGREC_ERR_UNSUPPORTED;
        int64_t edges = dst * fanouts[h];
        int64_t src = dst + edges;
        if (src > n_nodes) src = n_nodes;
        if (src < dst) src = dst;
        if (edges >= (1ll << 31) - 1) return E2EGREC_ERR_UNSUPPORTED;
        cap_dst[h] = (int32_t)dst;
        cap_edges[h] = (int32_t)edges;
        cap_src[h] = (int32_t)src;
        dst = src;
    }
    return E2EGREC_OK;
}

extern "C" int32_t e2egrec_sample_khop_workspace(int64_t n_nodes, int32_t n_seeds, int32_t n_hops,
                                                 const int32_t *fanouts, int32_t *cap_dst, int32_t *cap_src,
                                                 int32_t *cap_edges, size_t *scratch_bytes)
{
    if (!scratch_bytes) return E2EGREC_ERR_NULL;
    int32_t rc = khop_caps(n_nodes, n_seeds, n_hops, fanouts, cap_dst, cap_src, cap_edges);
    if (rc != E2EGREC_OK) return rc;
    int64_t md = 0, ms = 0, me = 0;
    for (int h = 0; h < n_hops; ++h) {
        if (cap_dst[h] > md) md = cap_dst[h];
        if (cap_src[h] > ms) ms = cap_src[h];
        if (cap_edges[h] > me) me = cap_edges[h];
    }
    *scratch_bytes = carve(n_nodes, md, ms, me, nullptr).bytes;
    return E2EGREC_OK;
}

extern "C" int32_t e2egrec_sampler_scratch_init(int64_t n_nodes, void *scratch, size_t scratch_bytes, void *stream)
{
    if (!scratch) return E2EGREC_ERR_NULL;
    if (n_nodes < 0) return E2EGREC_ERR_ARG;
    if (n_nodes >= (1ll << 31)) return E2EGREC_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(scratch) % 256) return E2EGREC_ERR_ALIGN;
    SamplerScratch s = carve(n_nodes, 0, 0, 0, scratch);
    if (scratch_bytes < s.bytes) return E2EGREC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    note_launch();
    fill_i32_kernel<<<(unsigned)std::min<int64_t>(ceil_div(n_nodes > 0 ? n_nodes : 1, 256), 148 * 16), 256, 0, st>>>(
        s.local_id, n_nodes, -1);
    cudaMemsetAsync(s.step_offset, 0, 256, st);
    cudaMemsetAsync(s.bitmap, 0, sizeof(uint32_t) * (size_t)s.n_words, st);
    return check_launch("sampler_scratch_init");
}

__global__ void set_u32_kernel(uint32_t *p, uint32_t v) { *p = v; }

extern "C" int32_t e2egrec_sampler_set_step(void *scratch, uint32_t step_offset, void *stream)
{
    if (!scratch) return E2EGREC_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(scratch) % 256) return E2EGREC_ERR_ALIGN;
    SamplerScratch s = carve(0, 0, 0, 0, scratch);
    note_launch();
    set_u32_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(s.step_offset, step_offset);
    return check_launch("sampler_set_step");
}

// Running sums of the integer edge weights of every row, one warp per row at a time: 32 entries per round, a
// 64-bit warp scan, the carry kept in a register.
__global__ void __launch_bounds__(256)
edge_cumulate_kernel(int64_t n_nodes, const int64_t *__restrict__ indptr, const uint32_t *__restrict__ q,
                     uint64_t *__restrict__ cum)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t u = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; u < n_nodes; u += warps) {
        const int64_t beg = indptr[u], end = indptr[u + 1];
        uint64_t carry = 0;
        for (int64_t e0 = beg; e0 < end; e0 += 32) {
            const int64_t e = e0 + lane;
            uint64_t v = e < end ? (uint64_t)q[e] : 0;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint64_t up = __shfl_up_sync(0xffffffffu, v, off);
                if (lane >= off) v += up;
            }
            if (e < end) cum[e] = carry + v;
            carry += __shfl_sync(0xffffffffu, v, 31);
        }
    }
}

extern "C" int32_t e2egrec_edge_cumulate(int64_t n_nodes, int64_t n_edges, const int64_t *indptr, const uint32_t *q,
                                         uint64_t *cum, void *stream)
{
    if (n_nodes < 0 || n_edges < 0) return E2EGREC_ERR_ARG;
    if (!indptr || (n_edges > 0 && (!q || !cum))) return E2EGREC_ERR_NULL;
    if (n_nodes == 0 || n_edges == 0) return E2EGREC_OK;
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(n_nodes * 32, 256), 148 * 16);
    note_launch();
    edge_cumulate_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(n_nodes, indptr, q, cum);
    return check_launch("edge_cumulate");
}

extern "C" int32_t e2egrec_sample_khop(const e2egrec_csr *graph, const int32_t *seeds, int32_t n_seeds,
                                       int32_t n_hops, const int32_t *fanouts, uint64_t seed, uint32_t step,
                                       uint32_t flags, const e2egrec_block *blocks,
                                       void *scratch, size_t scratch_bytes, void *stream)
{
    if (n_seeds > 0 && !seeds) return E2EGREC_ERR_NULL;
    return sample_khop_impl(graph, seeds, n_seeds, nullptr, n_hops, fanouts, seed, step, flags, blocks, scratch, scratch_bytes,
                            static_cast<cudaStream_t>(stream));
}

int32_t e2egrec::sample_khop_impl(const e2egrec_csr *graph, const int32_t *seeds, int32_t n_seeds, const PairInput *pairs,
                                  int32_t n_hops, const int32_t *fanouts, uint64_t seed, uint32_t step, uint32_t flags,
                                  const e2egrec_block *blocks, void *scratch, size_t scratch_bytes, cudaStream_t st)
{
    if (!graph || !fanouts || !blocks || !scratch || !graph->indptr) return E2EGREC_ERR_NULL;
    if (graph->n_edges > 0 && !graph->indices) return E2EGREC_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(scratch) % 256) return E2EGREC_ERR_ALIGN;
    int32_t cd[kMaxHops], cs[kMaxHops], ce[kMaxHops];
    int32_t rc = khop_caps(graph->n_nodes, n_seeds, n_hops, fanouts, cd, cs, ce);
    if (rc != E2EGREC_OK) return rc;
    int64_t md = 0, ms = 0, me = 0;
    for (int h = 0; h < n_hops; ++h) {
        const e2egrec_block &b = blocks[h];
        if (!b.counts || !b.indptr || !b.col || !b.nbr_global || !b.src_nodes || !b.csc_ptr || !b.csc_row ||
            !b.csc_eid || !b.csc_col || !b.inv_cnt)
            return E2EGREC_ERR_NULL;
        if (b.cap_dst < cd[h] || b.cap_src < cs[h] || b.cap_edges < ce[h]) return E2EGREC_ERR_WORKSPACE;
        if (b.cap_dst > md) md = b.cap_dst;
        if (b.cap_src > ms) ms = b.cap_src;
        if (b.cap_edges > me) me = b.cap_edges;
    }
    SamplerScratch s = carve(graph->n_nodes, md, ms, me, scratch);
    if (scratch_bytes < s.bytes) return E2EGREC_ERR_WORKSPACE;

    const int T = 256;
    const int64_t n = graph->n_nodes;
    tap_begin(TAP_SAMPLE, st);
    const int32_t *dst_nodes = seeds;
    const int32_t *n_dst_ptr = &blocks[0].counts[CNT_DST];
    if (!pairs) {
        note_launch();
        seed_init_kernel<<<grid_for(n_seeds, T), T, 0, st>>>(seeds, n_seeds, n, s.local_id, blocks[0].counts);
    } else {
        // seeds = ascending distinct endpoints of the pairs; entries (pair, side) grouped by seed
        const PairInput &pi = *pairs;
        const int32_t P2 = 2 * pi.n_pairs;
        cudaMemsetAsync(s.arena, 0, s.arena_bytes, st);
        cudaMemsetAsync(pi.pcounts, 0, 4 * sizeof(int32_t), st);
        cudaMemsetAsync(blocks[0].counts, 0, 4 * sizeof(int32_t), st);
        note_launch();
        pair_mark_kernel<<<grid_for(pi.n_pairs, T), T, 0, st>>>(pi.user, pi.item, pi.n_pairs, n, s.bitmap, blocks[0].counts);
        note_launch();
        frontier_kernel<<<grid_for(s.n_words, kWordTile), 256, 0, st>>>(s.bitmap, s.n_words, pi.pcounts, P2, s.local_id,
                                                                        pi.seeds_out, s.tickets + 1, s.state_words);
        const SortPlan sp = sort_plan(P2 > 1 ? P2 : 2);
        const SortLane &l = s.lane[0];
        cudaMemsetAsync(l.ghist, 0, sizeof(unsigned) * kMaxPasses * kMaxRadix, st);
        note_launch();
        pair_local_kernel<<<(unsigned)std::min<int64_t>(grid_for(P2, T), 148 * 4), T, 0, st>>>(
            pi.user, pi.item, pi.n_pairs, n, s.local_id, pi.pair_local, pi.entry_unit, pi.units_per_row, pi.item_unit_off,
            pi.pcounts, sp.bits, sp.passes, l.ghist);
        sort_by_col(pi.pair_local, pi.pcounts, P2, pi.pcsc_col, pi.pcsc_eid, sp, l, s.sort_tiles, st);
        note_launch();
        csc_finalize_kernel<<<grid_for((int64_t)P2 + 1, T), T, 0, st>>>(pi.pcsc_col, pi.pcsc_eid, pi.entry_unit, pi.pcounts,
                                                                       pi.pcsc_ptr, pi.pcsc_idx);
        dst_nodes = pi.seeds_out;
        n_dst_ptr = &pi.pcounts[CNT_SRC];
    }
    // The transposition of a hop (sort + offsets) is only needed by the backward pass, so it runs on the
    // helper stream beside the sampling of the next hop; everything is joined before this call returns.
    SideStream *side = SideStream::get(st);
    if (side) side->join_pending(st);               // a transposition deferred by an earlier call still uses the lanes
    for (int h = 0; h < n_hops; ++h) {
        const e2egrec_block &b = blocks[h];
        const int32_t f = fanouts[h];
        const SortPlan sp = sort_plan(b.cap_src);
        const SortLane &l = s.lane[h];
        cudaMemsetAsync(s.arena, 0, s.arena_bytes, st);
        note_launch();
        hop_sample_kernel<<<grid_for(b.cap_dst, kDstTile), kDstThreads, 0, st>>>(
            graph->indptr, graph->indices, graph->edge_cum, n, dst_nodes, n_dst_ptr, b.cap_dst, b.cap_edges, f, h + 1,
            (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32), step, s.step_offset, h == 0, b.counts, b.indptr,
            b.inv_cnt, b.src_nodes, b.nbr_global, l.edge_row, s.local_id, s.bitmap, s.tickets + 0, s.state_dst);
        note_launch();
        frontier_kernel<<<grid_for(s.n_words, kWordTile), 256, 0, st>>>(s.bitmap, s.n_words, b.counts, b.cap_src,
                                                                        s.local_id, b.src_nodes, s.tickets + 1,
                                                                        s.state_words);
        cudaMemsetAsync(l.ghist, 0, sizeof(unsigned) * kMaxPasses * kMaxRadix, st);
        note_launch();
        relabel_kernel<<<(unsigned)std::min<int64_t>(grid_for(b.cap_edges, T), 148 * 4), T, 0, st>>>(
            b.nbr_global, s.local_id, b.counts, b.col, sp.bits, sp.passes, l.ghist);
        if (!(flags & E2EGREC_SAMPLE_NO_TRANSPOSE)) {
            cudaStream_t ts = st;                    // stream of the transposition
            if (side) {
                side->fork(st);
                ts = side->stream;
            }
            sort_by_col(b.col, b.counts, b.cap_edges, b.csc_col, b.csc_eid, sp, l, s.sort_tiles, ts);
            note_launch();
            csc_finalize_kernel<<<grid_for(std::max<int64_t>(b.cap_edges, (int64_t)b.cap_src + 1), T), T, 0, ts>>>(
                b.csc_col, b.csc_eid, l.edge_row, b.counts, b.csc_ptr, b.csc_row);
        }
        dst_nodes = b.src_nodes;
        n_dst_ptr = &b.counts[CNT_SRC];
    }
    if (side && !(flags & E2EGREC_SAMPLE_NO_TRANSPOSE)) {
        if (flags & E2EGREC_SAMPLE_DEFER_TRANSPOSE) side->defer();
        else side->join(st);
    }
    const e2egrec_block &last = blocks[n_hops - 1];
    note_launch();
    frontier_release_kernel<<<grid_for(last.cap_src, T), T, 0, st>>>(last.src_nodes, last.counts, s.local_id);
    tap_end(TAP_SAMPLE, st);
    return check_launch("sample_khop");
}

// The transposed form of blocks sampled with E2EGREC_SAMPLE_NO_TRANSPOSE: the sort of every block by source and
// its offsets, from what the sampling left in the blocks and in the scratch (entry rows, digit counts of the
// columns).  Blocks are independent, so every other one runs on the helper stream.
extern "C" int32_t e2egrec_blocks_transpose(int64_t n_nodes, int32_t n_hops, const e2egrec_block *blocks, void *scratch,
                                            size_t scratch_bytes, void *stream)
{
    using namespace e2egrec;
    if (!blocks || !scratch) return E2EGREC_ERR_NULL;
    if (n_hops < 1 || n_hops > kMaxHops || n_nodes < 1) return E2EGREC_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(scratch) % 256) return E2EGREC_ERR_ALIGN;
    int64_t md = 0, ms = 0, me = 0;
    for (int h = 0; h < n_hops; ++h) {
        const e2egrec_block &b = blocks[h];
        if (!b.counts || !b.col || !b.csc_ptr || !b.csc_row || !b.csc_eid || !b.csc_col) return E2EGREC_ERR_NULL;
        if (b.cap_dst > md) md = b.cap_dst;
        if (b.cap_src > ms) ms = b.cap_src;
        if (b.cap_edges > me) me = b.cap_edges;
    }
    SamplerScratch s = carve(n_nodes, md, ms, me, scratch);
    if (scratch_bytes < s.bytes) return E2EGREC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SideStream *side = SideStream::get(st);
    if (side) side->join_pending(st);
    const int T = 256;
    const bool forked = side && n_hops > 1;
    if (forked) side->fork(st);
    for (int h = n_hops - 1; h >= 0; --h) {          // the largest block first, on the caller's stream
        const e2egrec_block &b = blocks[h];
        const SortPlan sp = sort_plan(b.cap_src);
        const SortLane &l = s.lane[h];
        cudaStream_t ts = st;
        if (forked && ((n_hops - 1 - h) & 1)) ts = side->stream;
        sort_by_col(b.col, b.counts, b.cap_edges, b.csc_col, b.csc_eid, sp, l, s.sort_tiles, ts);
        note_launch();
        csc_finalize_kernel<<<grid_for(std::max<int64_t>(b.cap_edges, (int64_t)b.cap_src + 1), T), T, 0, ts>>>(
            b.csc_col, b.csc_eid, l.edge_row, b.counts, b.csc_ptr, b.csc_row);
    }
    if (forked) side->join(st);
    return check_launch("blocks_transpose");
}

