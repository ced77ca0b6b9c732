// Graph ingest on the device: canonical CSR from an edge list, and the CSC (transpose) of a CSR.
// Both are two or three stable radix sorts plus offset look-ups, so the result depends only on the
// multiset of edges: rows ordered by (row, col), columns by (col, CSR position), parallel edges kept.
#include <algorithm>

#include "radix.cuh"

namespace e2egrec {
namespace {

struct IngestScratch {
    int32_t *counts;                 // int32[4], counts[CNT_EDGES] = m
    int32_t *a, *b, *c;              // three arrays of m
    RadixScratch rs;
    char *arena;
    size_t arena_bytes, bytes;
};

IngestScratch carve_ingest(int64_t m, void *base)
{
    IngestScratch s{};
    size_t off = 0;
    auto take = [&](size_t bytes) {
        char *p = base ? static_cast<char *>(base) + off : nullptr;
        off += align_up(bytes, 256);
        return p;
    };
    const size_t mm = (size_t)(m > 0 ? m : 1);
    s.counts = (int32_t *)take(256);
    s.a = (int32_t *)take(mm * 4);
    s.b = (int32_t *)take(mm * 4);
    s.c = (int32_t *)take(mm * 4);
    for (int i = 0; i < 2; ++i) s.rs.keys[i] = (int32_t *)take(mm * 4);
    for (int i = 0; i < 2; ++i) s.rs.vals[i] = (int32_t *)take(mm * 4);
    s.rs.tiles = ceil_div((int64_t)mm, kSortTile);
    const size_t arena_begin = off;
    s.arena = base ? static_cast<char *>(base) + off : nullptr;
    s.rs.ghist = (unsigned *)take(sizeof(unsigned) * kMaxPasses * kMaxRadix);
    s.arena_bytes = off - arena_begin;
    s.rs.thist = (int32_t *)take(radix_thist_bytes(s.rs.tiles));
    s.bytes = off;
    return s;
}

__global__ void ingest_begin_kernel(int32_t *counts, int32_t m)
{
    counts[CNT_DST] = 0;
    counts[CNT_SRC] = 0;
    counts[CNT_EDGES] = m;
    counts[CNT_STATUS] = 0;
}

// ids outside [0, n) are flagged and clamped so that the sorts stay in range
__global__ void clamp_ids_kernel(const int32_t *__restrict__ in, int64_t m, int64_t n, int32_t *__restrict__ out,
                                 int32_t *counts)
{
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < m; i += (int64_t)gridDim.x * blockDim.x) {
        int32_t v = in[i];
        if ((uint32_t)v >= (uint64_t)n) {
            atomicOr((unsigned *)&counts[CNT_STATUS], E2EGREC_DEV_RANGE);
            v = 0;
        }
        out[i] = v;
    }
}

// out[i] = src[pos[i]], flagged and clamped like clamp_ids_kernel
__global__ void gather_ids_kernel(const int32_t *__restrict__ src, const int32_t *__restrict__ pos, int64_t m, int64_t n,
                                  int32_t *__restrict__ out, int32_t *counts)
{
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < m; i += (int64_t)gridDim.x * blockDim.x) {
        int32_t v = src[pos[i]];
        if ((uint32_t)v >= (uint64_t)n) {
            atomicOr((unsigned *)&counts[CNT_STATUS], E2EGREC_DEV_RANGE);
            v = 0;
        }
        out[i] = v;
    }
}

// ptr[s] = first position of the sorted key array whose key is >= s, for s = 0 .. n
__global__ void offsets_kernel(const int32_t *__restrict__ sorted, int64_t m, int64_t n, int64_t *__restrict__ ptr)
{
    for (int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; s <= n; s += (int64_t)gridDim.x * blockDim.x) {
        int64_t lo = 0, hi = m;
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            if ((int64_t)sorted[mid] < s) lo = mid + 1; else hi = mid;
        }
        ptr[s] = lo;
    }
}

// row and CSR position of every transposed entry
__global__ void transpose_rows_kernel(const int32_t *__restrict__ eid32, int64_t m, const int64_t *__restrict__ indptr,
                                      int64_t n_rows, int32_t *__restrict__ csc_row, int64_t *__restrict__ csc_eid)
{
    for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < m; k += (int64_t)gridDim.x * blockDim.x) {
        const int64_t e = eid32[k];
        int64_t lo = 0, hi = n_rows;                 // largest r with indptr[r] <= e
        while (hi - lo > 1) {
            const int64_t mid = (lo + hi) >> 1;
            if (indptr[mid] <= e) lo = mid; else hi = mid;
        }
        csc_row[k] = (int32_t)lo;
        csc_eid[k] = e;
    }
}

unsigned wide_grid(int64_t n) { return (unsigned)std::min<int64_t>(ceil_div(n > 0 ? n : 1, 256), 148 * 16); }

// stable sort of (keys, vals) by key; vals == nullptr: value = position
void sort_stage(const int32_t *keys, const int32_t *vals, int32_t *keys_out, int32_t *vals_out, int64_t m, int64_t key_range,
                IngestScratch &s, cudaStream_t st)
{
    const SortPlan sp = sort_plan((int32_t)std::min<int64_t>(std::max<int64_t>(key_range, 2), 0x7fffffff));
    cudaMemsetAsync(s.arena, 0, s.arena_bytes, st);
    note_launch();
    key_hist_kernel<<<wide_grid(m), 256, 0, st>>>(keys, s.counts, sp.bits, sp.passes, s.rs.ghist);
    radix_sort_pairs(keys, vals, s.counts, m, keys_out, vals_out, sp, s.rs, st);
}

}  // namespace
}  // namespace e2egrec

using namespace e2egrec;

extern "C" int32_t e2egrec_graph_from_coo(int64_t n_nodes, int64_t n_edges, const int32_t *row, const int32_t *col,
                                          int64_t *indptr, int32_t *indices, int32_t *status, void *ws,
                                          size_t *ws_bytes, void *stream)
{
    if (!ws_bytes) return E2EGREC_ERR_NULL;
    if (n_nodes < 0 || n_edges < 0) return E2EGREC_ERR_ARG;
    if (n_nodes >= (1ll << 31) || n_edges >= (1ll << 31) - 1) return E2EGREC_ERR_UNSUPPORTED;
    IngestScratch s = carve_ingest(n_edges, ws);
    if (!ws) { *ws_bytes = s.bytes; return E2EGREC_OK; }
    if (*ws_bytes < s.bytes) { *ws_bytes = s.bytes; return E2EGREC_ERR_WORKSPACE; }
    if (reinterpret_cast<uintptr_t>(ws) % 256) return E2EGREC_ERR_ALIGN;
    if (!indptr || (n_edges > 0 && (!row || !col || !indices))) return E2EGREC_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t m = n_edges;
    note_launch();
    ingest_begin_kernel<<<1, 1, 0, st>>>(s.counts, (int32_t)m);
    if (m > 0) {
        // 1. by column (value = position), 2. by row with the sorted columns as values: (row, col) order
        note_launch();
        clamp_ids_kernel<<<wide_grid(m), 256, 0, st>>>(col, m, n_nodes, s.a, s.counts);
        sort_stage(s.a, nullptr, s.b, s.c, m, n_nodes, s, st);            // s.b = columns sorted, s.c = their positions
        note_launch();
        gather_ids_kernel<<<wide_grid(m), 256, 0, st>>>(row, s.c, m, n_nodes, s.a, s.counts);
        sort_stage(s.a, s.b, s.c, indices, m, n_nodes, s, st);            // s.c = rows sorted
    }
    note_launch();
    offsets_kernel<<<wide_grid(n_nodes + 1), 256, 0, st>>>(s.c, m, n_nodes, indptr);
    if (status) cudaMemcpyAsync(status, &s.counts[CNT_STATUS], sizeof(int32_t), cudaMemcpyDeviceToDevice, st);
    return check_launch("graph_from_coo");
}

extern "C" int32_t e2egrec_csr_transpose(const e2egrec_csr *csr, int64_t n_cols, int64_t *csc_ptr, int32_t *csc_row,
                                         int64_t *csc_eid, int32_t *status, void *ws, size_t *ws_bytes, void *stream)
{
    if (!ws_bytes || !csr) return E2EGREC_ERR_NULL;
    if (csr->n_nodes < 0 || csr->n_edges < 0 || n_cols < 0) return E2EGREC_ERR_ARG;
    if (csr->n_nodes >= (1ll << 31) || n_cols >= (1ll << 31) || csr->n_edges >= (1ll << 31) - 1) return E2EGREC_ERR_UNSUPPORTED;
    IngestScratch s = carve_ingest(csr->n_edges, ws);
    if (!ws) { *ws_bytes = s.bytes; return E2EGREC_OK; }
    if (*ws_bytes < s.bytes) { *ws_bytes = s.bytes; return E2EGREC_ERR_WORKSPACE; }
    if (reinterpret_cast<uintptr_t>(ws) % 256) return E2EGREC_ERR_ALIGN;
    if (!csr->indptr || !csc_ptr || (csr->n_edges > 0 && (!csr->indices || !csc_row || !csc_eid))) return E2EGREC_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t m = csr->n_edges;
    note_launch();
    ingest_begin_kernel<<<1, 1, 0, st>>>(s.counts, (int32_t)m);
    if (m > 0) {
        note_launch();
        clamp_ids_kernel<<<wide_grid(m), 256, 0, st>>>(csr->indices, m, n_cols, s.a, s.counts);
        sort_stage(s.a, nullptr, s.b, s.c, m, n_cols, s, st);             // s.b = columns sorted, s.c = CSR positions
        note_launch();
        transpose_rows_kernel<<<wide_grid(m), 256, 0, st>>>(s.c, m, csr->indptr, csr->n_nodes, csc_row, csc_eid);
    }
    note_launch();
    offsets_kernel<<<wide_grid(n_cols + 1), 256, 0, st>>>(s.b, m, n_cols, csc_ptr);
    if (status) cudaMemcpyAsync(status, &s.counts[CNT_STATUS], sizeof(int32_t), cudaMemcpyDeviceToDevice, st);
    return check_launch("csr_transpose");
}
