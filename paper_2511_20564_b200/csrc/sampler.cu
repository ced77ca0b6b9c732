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
struct SamplerScratch {
    uint32_t *step_offset; // [1]         added to the `step` argument of every call (see e2egrec_sampler_set_step)
    int32_t  *local_id;    // [n_nodes]   -1 when idle, else position in the current frontier
    uint32_t *bitmap;      // [n_words]   newly reached nodes of the hop in progress; 0 when idle
    int32_t  *word_cnt;    // [n_words]
    int32_t  *word_rank;   // [n_words+1]
    int32_t  *cnt;         // [max cap_dst]     |S(u)| per destination
    int32_t  *csc_cnt;     // [max cap_src]
    int32_t  *edge_row;    // [max cap_edges]   destination of each block entry
    int32_t  *keys[2];     // [max cap_edges]   radix sort ping-pong
    int32_t  *vals[2];
    int32_t  *hist;        // [radix * sort blocks]
    int32_t  *hist_off;    // [radix * sort blocks + 1]
    int32_t  *scan_tmp;    // scan partials
    size_t    bytes;
    int64_t   n_words;
};

constexpr int kSortThreads = 256;
constexpr int kSortItems = 16;
constexpr int kSortTile = kSortThreads * kSortItems;
constexpr int kMaxRadix = 1024;

static SamplerScratch carve(int64_t n_nodes, int64_t max_dst, int64_t max_src, int64_t max_edges, void *base)
{
    SamplerScratch s;
    s.n_words = ceil_div(n_nodes, 32);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        char *p = base ? static_cast<char *>(base) + off : nullptr;
        off += align_up(bytes, 256);
        return p;
    };
    const int64_t sort_blocks = ceil_div(max_edges > 0 ? max_edges : 1, kSortTile);
    const int64_t hist_len = (int64_t)kMaxRadix * sort_blocks;
    int64_t longest = hist_len + 1;
    if (s.n_words > longest) longest = s.n_words;
    if (max_src + 1 > longest) longest = max_src + 1;
    s.step_offset = (uint32_t *)take(256);
    s.local_id = (int32_t *)take(sizeof(int32_t) * (size_t)n_nodes);
    s.bitmap = (uint32_t *)take(sizeof(uint32_t) * (size_t)s.n_words);
    s.word_cnt = (int32_t *)take(sizeof(int32_t) * (size_t)s.n_words);
    s.word_rank = (int32_t *)take(sizeof(int32_t) * (size_t)(s.n_words + 1));
    s.cnt = (int32_t *)take(sizeof(int32_t) * (size_t)(max_dst + 1));
    s.csc_cnt = (int32_t *)take(sizeof(int32_t) * (size_t)(max_src + 1));
    s.edge_row = (int32_t *)take(sizeof(int32_t) * (size_t)(max_edges + 1));
    for (int i = 0; i < 2; ++i) s.keys[i] = (int32_t *)take(sizeof(int32_t) * (size_t)(max_edges + 1));
    for (int i = 0; i < 2; ++i) s.vals[i] = (int32_t *)take(sizeof(int32_t) * (size_t)(max_edges + 1));
    s.hist = (int32_t *)take(sizeof(int32_t) * (size_t)hist_len);
    s.hist_off = (int32_t *)take(sizeof(int32_t) * (size_t)(hist_len + 1));
    s.scan_tmp = (int32_t *)take(sizeof(int32_t) * scan_scratch_ints(longest));
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

// |S(u)| = min(deg(u), fanout), 1/|S(u)|, and the destination prefix of the frontier.
__global__ void hop_count_kernel(const int64_t *__restrict__ g_indptr, int64_t n_nodes,
                                 const int32_t *__restrict__ dst_nodes, const int32_t *n_dst_ptr, int32_t cap_dst,
                                 int32_t fanout, int32_t *__restrict__ counts, int32_t *__restrict__ cnt,
                                 float *__restrict__ inv_cnt, int32_t *__restrict__ src_nodes, int first_hop)
{
    int32_t n_dst = *n_dst_ptr;
    uint32_t status = 0;
    if (n_dst > cap_dst) { n_dst = cap_dst; status |= E2EGREC_DEV_CAPACITY; }
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        counts[CNT_DST] = n_dst;
        if (!first_hop) counts[CNT_STATUS] = 0;
        if (status) atomicOr((unsigned *)&counts[CNT_STATUS], status);
    }
    if (i >= n_dst) return;
    int32_t u = dst_nodes[i];
    int32_t c = 0;
    if ((uint32_t)u < (uint64_t)n_nodes) {
        const int64_t deg = g_indptr[u + 1] - g_indptr[u];
        c = deg < fanout ? (int32_t)deg : fanout;
    } else {
        atomicOr((unsigned *)&counts[CNT_STATUS], E2EGREC_DEV_RANGE);
        u = 0;
        c = 0;
    }
    cnt[i] = c;
    inv_cnt[i] = c > 0 ? 1.0f / (float)c : 0.0f;
    src_nodes[i] = u;
}

// One thread per (destination, slot).  Slot j of node u at hop h draws with the counter
// (j/2, u, (1<<8)|h, step) and key (seed lo, seed hi); words 2(j%2), 2(j%2)+1 form r and the
// picked row position is floor(r * deg / 2^64).  deg <= fanout copies the row instead.
__global__ void hop_draw_kernel(const int64_t *__restrict__ g_indptr, const int32_t *__restrict__ g_indices,
                                int64_t n_nodes, const int32_t *__restrict__ src_nodes,
                                const int32_t *__restrict__ blk_indptr, int32_t *__restrict__ counts,
                                int32_t fanout, int32_t hop, uint32_t seed_lo, uint32_t seed_hi, uint32_t step_arg,
                                const uint32_t *__restrict__ step_offset,
                                int32_t cap_edges, int32_t *__restrict__ nbr_global, int32_t *__restrict__ edge_row,
                                const int32_t *__restrict__ local_id, uint32_t *__restrict__ bitmap)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int32_t n_dst = counts[CNT_DST];
    const uint32_t step = step_arg + *step_offset;
    if (t == 0) counts[CNT_EDGES] = min(blk_indptr[n_dst], cap_edges);
    const int64_t i = t / fanout;
    const int32_t j = (int32_t)(t - i * fanout);
    if (i >= n_dst) return;
    const int32_t beg = blk_indptr[i];
    const int32_t c = blk_indptr[i + 1] - beg;
    if (j >= c) return;
    const int32_t e = beg + j;
    if (e >= cap_edges) { atomicOr((unsigned *)&counts[CNT_STATUS], E2EGREC_DEV_CAPACITY); return; }
    const int32_t u = src_nodes[i];
    const int64_t gbeg = g_indptr[u];
    const int64_t deg = g_indptr[u + 1] - gbeg;
    int64_t pos = j;
    if (deg > fanout) {
        const uint4 r4 = philox4x32_10(make_uint4((uint32_t)(j >> 1), (uint32_t)u, (1u << 8) | (uint32_t)hop, step),
                                       make_uint2(seed_lo, seed_hi));
        const uint64_t r = (j & 1) ? (((uint64_t)r4.w << 32) | r4.z) : (((uint64_t)r4.y << 32) | r4.x);
        pos = (int64_t)__umul64hi(r, (uint64_t)deg);
    }
    int32_t v = g_indices[gbeg + pos];
    if ((uint32_t)v >= (uint64_t)n_nodes) {
        atomicOr((unsigned *)&counts[CNT_STATUS], E2EGREC_DEV_RANGE);
        v = u;
    }
    nbr_global[e] = v;
    edge_row[e] = (int32_t)i;
    if (local_id[v] < 0) atomicOr(&bitmap[v >> 5], 1u << (v & 31));
}

__global__ void bitmap_popc_kernel(const uint32_t *__restrict__ bitmap, int64_t n_words, int32_t *__restrict__ word_cnt)
{
    const int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (w < n_words) word_cnt[w] = __popc(bitmap[w]);
}

// New nodes, in ascending id order, take local ids n_dst, n_dst+1, ...; the bitmap returns to 0.
__global__ void frontier_assign_kernel(uint32_t *__restrict__ bitmap, const int32_t *__restrict__ word_rank,
                                       int64_t n_words, int32_t *__restrict__ counts, int32_t cap_src,
                                       int32_t *__restrict__ local_id, int32_t *__restrict__ src_nodes)
{
    const int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int32_t n_dst = counts[CNT_DST];
    if (w == 0) {
        int64_t n_src = (int64_t)n_dst + word_rank[n_words];
        if (n_src > cap_src) { n_src = cap_src; atomicOr((unsigned *)&counts[CNT_STATUS], E2EGREC_DEV_CAPACITY); }
        counts[CNT_SRC] = (int32_t)n_src;
    }
    if (w >= n_words) return;
    uint32_t bits = bitmap[w];
    if (!bits) return;
    bitmap[w] = 0;
    int32_t r = n_dst + word_rank[w];
    while (bits) {
        const int b = __ffs(bits) - 1;
        bits &= bits - 1;
        const int32_t id = (int32_t)(w * 32 + b);
        if (r < cap_src) {
            local_id[id] = r;
            src_nodes[r] = id;
        }
        ++r;
    }
}

// col[e] = position of the sampled node in the frontier; column histogram for the transpose.
__global__ void relabel_kernel(const int32_t *__restrict__ nbr_global, const int32_t *__restrict__ local_id,
                               const int32_t *__restrict__ counts, int32_t *__restrict__ col,
                               int32_t *__restrict__ csc_cnt)
{
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= counts[CNT_EDGES]) return;
    int32_t c = local_id[nbr_global[e]];
    if (c < 0 || c >= counts[CNT_SRC]) c = 0;        // only after a capacity overrun, which is flagged
    col[e] = c;
    atomicAdd(&csc_cnt[c], 1);
}

__global__ void frontier_release_kernel(const int32_t *__restrict__ src_nodes, const int32_t *__restrict__ counts,
                                        int32_t *__restrict__ local_id)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < counts[CNT_SRC]) local_id[src_nodes[i]] = -1;
}

// ---------------------------------------------------------------------------------------
// Stable LSD radix sort of (key = col, value = block position).  Tiles of kSortTile
// consecutive elements; per pass: tile histograms, one scan over the digit-major
// (digit, tile) table, then a scatter that ranks equal digits in element order.
// ---------------------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(kSortThreads)
sort_hist_kernel(const int32_t *__restrict__ keys, const int32_t *__restrict__ counts, int shift, int n_tiles,
                 int32_t *__restrict__ hist)
{
    constexpr int R = 1 << BITS;
    __shared__ int32_t h[R];
    for (int d = threadIdx.x; d < R; d += kSortThreads) h[d] = 0;
    __syncthreads();
    const int32_t n = counts[CNT_EDGES];
    const int64_t base = (int64_t)blockIdx.x * kSortTile;
#pragma unroll 4
    for (int k = 0; k < kSortItems; ++k) {
        const int64_t idx = base + k * kSortThreads + threadIdx.x;
        if (idx < n) atomicAdd(&h[(keys[idx] >> shift) & (R - 1)], 1);
    }
    __syncthreads();
    for (int d = threadIdx.x; d < R; d += kSortThreads) hist[(int64_t)d * n_tiles + blockIdx.x] = h[d];
}

template <int BITS>
__global__ void __launch_bounds__(kSortThreads)
sort_scatter_kernel(const int32_t *__restrict__ keys_in, const int32_t *__restrict__ vals_in,
                    const int32_t *__restrict__ counts, int shift, int n_tiles,
                    const int32_t *__restrict__ hist_off, int32_t *__restrict__ keys_out,
                    int32_t *__restrict__ vals_out)
{
    constexpr int R = 1 << BITS;
    constexpr int W = kSortThreads / 32;
    __shared__ int32_t wc[W][R];                 // per-warp digit counts, then start offsets
    for (int d = threadIdx.x; d < W * R; d += kSortThreads) (&wc[0][0])[d] = 0;
    __syncthreads();
    const int32_t n = counts[CNT_EDGES];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t wbase = (int64_t)blockIdx.x * kSortTile + (int64_t)warp * (32 * kSortItems);
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
    for (int d = threadIdx.x; d < R; d += kSortThreads) {
        int32_t run = hist_off[(int64_t)d * n_tiles + blockIdx.x];
#pragma unroll
        for (int w = 0; w < W; ++w) {
            const int32_t c = wc[w][d];
            wc[w][d] = run;
            run += c;
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kSortItems; ++k) {
        const int64_t idx = wbase + k * 32 + lane;
        if (idx < n) {
            const int32_t pos = wc[warp][(key[k] >> shift) & (R - 1)] + rank[k];
            if (keys_out) keys_out[pos] = key[k];
            vals_out[pos] = val[k];
        }
    }
}

__global__ void csc_rows_kernel(const int32_t *__restrict__ csc_eid, const int32_t *__restrict__ edge_row,
                                const int32_t *__restrict__ counts, int32_t *__restrict__ csc_row)
{
    const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (k < counts[CNT_EDGES]) csc_row[k] = edge_row[csc_eid[k]];
}

template <int BITS>
static void sort_pass(const int32_t *kin, const int32_t *vin, int32_t *kout, int32_t *vout, const int32_t *counts,
                      int shift, int n_tiles, SamplerScratch &s, cudaStream_t st)
{
    constexpr int R = 1 << BITS;
    note_launch();
    sort_hist_kernel<BITS><<<n_tiles, kSortThreads, 0, st>>>(kin, counts, shift, n_tiles, s.hist);
    exclusive_scan<int32_t>(s.hist, s.hist_off, nullptr, (int64_t)R * n_tiles, (int64_t)R * n_tiles, s.scan_tmp, st);
    note_launch();
    sort_scatter_kernel<BITS><<<n_tiles, kSortThreads, 0, st>>>(kin, vin, counts, shift, n_tiles, s.hist_off, kout, vout);
}

// csc_eid = positions of the block entries ordered by (col, position).
static void sort_by_col(const e2egrec_block &b, SamplerScratch &s, cudaStream_t st)
{
    int key_bits = 1;
    while (key_bits < 31 && (1ll << key_bits) < (int64_t)b.cap_src) ++key_bits;
    int bits, passes;
    if (key_bits <= 8) { bits = 8; passes = 1; }
    else if (key_bits <= 10) { bits = 10; passes = 1; }
    else if (key_bits <= 16) { bits = 8; passes = 2; }
    else if (key_bits <= 20) { bits = 10; passes = 2; }
    else if (key_bits <= 24) { bits = 8; passes = 3; }
    else if (key_bits <= 30) { bits = 10; passes = 3; }
    else { bits = 8; passes = 4; }
    const int n_tiles = (int)ceil_div(b.cap_edges > 0 ? b.cap_edges : 1, kSortTile);
    const int32_t *kin = b.col;
    const int32_t *vin = nullptr;                 // first pass: value = own position
    for (int p = 0; p < passes; ++p) {
        const bool last = p == passes - 1;
        int32_t *kout = last ? b.csc_col : s.keys[p & 1];
        int32_t *vout = last ? b.csc_eid : s.vals[p & 1];
        if (bits == 8) sort_pass<8>(kin, vin, kout, vout, b.counts, p * bits, n_tiles, s, st);
        else sort_pass<10>(kin, vin, kout, vout, b.counts, p * bits, n_tiles, s, st);
        kin = kout;
        vin = vout;
    }
}

static inline unsigned grid_for(int64_t n, int threads) { return (unsigned)ceil_div(n > 0 ? n : 1, threads); }

}  // namespace e2egrec

using namespace e2egrec;

// ---------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------
static int32_t khop_caps(int64_t n_nodes, int32_t n_seeds, int32_t n_hops, const int32_t *fanouts,
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

extern "C" int32_t e2egrec_sample_khop(const e2egrec_csr *graph, const int32_t *seeds, int32_t n_seeds,
                                       int32_t n_hops, const int32_t *fanouts, uint64_t seed, uint32_t step,
                                       uint32_t flags, const e2egrec_block *blocks,
                                       void *scratch, size_t scratch_bytes, void *stream)
{
    (void)flags;
    if (!graph || !fanouts || !blocks || !scratch || !graph->indptr) return E2EGREC_ERR_NULL;
    if (n_seeds > 0 && !seeds) return E2EGREC_ERR_NULL;
    if (graph->n_edges > 0 && !graph->indices) return E2EGREC_ERR_NULL;
    if (graph->edge_weight) return E2EGREC_ERR_UNSUPPORTED;
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

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int T = 256;
    const int64_t n = graph->n_nodes;
    tap_begin(TAP_SAMPLE, st);
    note_launch();
    seed_init_kernel<<<grid_for(n_seeds, T), T, 0, st>>>(seeds, n_seeds, n, s.local_id, blocks[0].counts);
    const int32_t *dst_nodes = seeds;
    const int32_t *n_dst_ptr = &blocks[0].counts[CNT_DST];
    for (int h = 0; h < n_hops; ++h) {
        const e2egrec_block &b = blocks[h];
        const int32_t f = fanouts[h];
        note_launch();
        hop_count_kernel<<<grid_for(b.cap_dst, T), T, 0, st>>>(graph->indptr, n, dst_nodes, n_dst_ptr, b.cap_dst, f,
                                                              b.counts, s.cnt, b.inv_cnt, b.src_nodes, h == 0);
        exclusive_scan<int32_t>(s.cnt, b.indptr, &b.counts[CNT_DST], 0, b.cap_dst, s.scan_tmp, st);
        note_launch();
        hop_draw_kernel<<<grid_for((int64_t)b.cap_dst * f, T), T, 0, st>>>(
            graph->indptr, graph->indices, n, b.src_nodes, b.indptr, b.counts, f, h + 1,
            (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32), step, s.step_offset, b.cap_edges, b.nbr_global, s.edge_row,
            s.local_id, s.bitmap);
        note_launch();
        bitmap_popc_kernel<<<grid_for(s.n_words, T), T, 0, st>>>(s.bitmap, s.n_words, s.word_cnt);
        exclusive_scan<int32_t>(s.word_cnt, s.word_rank, nullptr, s.n_words, s.n_words, s.scan_tmp, st);
        note_launch();
        frontier_assign_kernel<<<grid_for(s.n_words, T), T, 0, st>>>(s.bitmap, s.word_rank, s.n_words, b.counts,
                                                                    b.cap_src, s.local_id, b.src_nodes);
        cudaMemsetAsync(s.csc_cnt, 0, sizeof(int32_t) * (size_t)(b.cap_src + 1), st);
        note_launch();
        relabel_kernel<<<grid_for(b.cap_edges, T), T, 0, st>>>(b.nbr_global, s.local_id, b.counts, b.col, s.csc_cnt);
        exclusive_scan<int32_t>(s.csc_cnt, b.csc_ptr, &b.counts[CNT_SRC], 0, b.cap_src, s.scan_tmp, st);
        sort_by_col(b, s, st);
        note_launch();
        csc_rows_kernel<<<grid_for(b.cap_edges, T), T, 0, st>>>(b.csc_eid, s.edge_row, b.counts, b.csc_row);
        dst_nodes = b.src_nodes;
        n_dst_ptr = &b.counts[CNT_SRC];
    }
    const e2egrec_block &last = blocks[n_hops - 1];
    note_launch();
    frontier_release_kernel<<<grid_for(last.cap_src, T), T, 0, st>>>(last.src_nodes, last.counts, s.local_id);
    tap_end(TAP_SAMPLE, st);
    return check_launch("sample_khop");
}
