// Functions shared between the translation units of the library (not part of the C ABI).
#pragma once

#include "common.cuh"

namespace e2egrec {

// sampler.cu ------------------------------------------------------------------------------
// Seeds derived from training pairs (joint step).  All arrays are device memory of 2 * n_pairs
// entries unless noted.
struct PairInput {
    const int32_t *user, *item;   // [n_pairs] global node ids
    int32_t n_pairs;
    int32_t *seeds_out;           // ascending distinct endpoints
    int32_t *pair_local;          // seed position of entry e (e < P: user of pair e; else item of pair e - P)
    int32_t *entry_unit;          // start of the entry's gradient row, in 16-byte units
    int32_t *pcounts;             // int32[4]: {0, n_seeds, 2 n_pairs, status}
    int32_t *pcsc_ptr;            // [2P + 1] entries grouped by seed: offsets,
    int32_t *pcsc_idx;            //          gradient-row unit of each grouped entry,
    int32_t *pcsc_eid, *pcsc_col; //          its entry number and its seed
    int units_per_row, item_unit_off;
};

int32_t khop_caps(int64_t n_nodes, int32_t n_seeds, int32_t n_hops, const int32_t *fanouts, int32_t *cap_dst,
                  int32_t *cap_src, int32_t *cap_edges);
size_t sampler_scratch_bytes(int64_t n_nodes, int64_t max_dst, int64_t max_src, int64_t max_edges);
int32_t sample_khop_impl(const e2egrec_csr *graph, const int32_t *seeds, int32_t n_seeds, const PairInput *pairs,
                         int32_t n_hops, const int32_t *fanouts, uint64_t seed, uint32_t step, uint32_t flags,
                         const e2egrec_block *blocks, void *scratch, size_t scratch_bytes, cudaStream_t st);

// aggregate.cu ----------------------------------------------------------------------------
// Whole-graph segment reduction shared by e2egrec_aggregate_forward / _backward and the workspace-free entry point:
// argument checks, the scratch size for n_entries entries of d values, and the launch itself on scratch `ws`.
int32_t check_mats(const e2egrec_mat *in, const e2egrec_mat *out, int64_t out_rows);
size_t full_ws_bytes(int64_t n_entries, int d, int32_t dtype);
int32_t full_aggregate(int64_t n_seg, int64_t n_entries, const int64_t *ptr, const int32_t *idx, const float *w,
                       const e2egrec_mat *in, const e2egrec_mat *out, int mean, void *ws, cudaStream_t st);

}  // namespace e2egrec
