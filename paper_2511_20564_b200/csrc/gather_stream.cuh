// Mean aggregation of a sampled block (Eq. 2) for 512-byte rows, the gathered rows streamed through shared memory by
// the TMA unit.
#pragma once

#include "common.cuh"

namespace e2egrec {

// cat[i] = [ Hsrc[self_ids ? self_ids[i] : i] | mean over k in [indptr[i], indptr[i+1]) of Hsrc[nbr[k]] ] for i < counts[CNT_DST],
// zero rows up to the next multiple of 128 (at most cap_dst rows): the result of sage_aggregate_kernel, bit for bit, for
// bf16 rows of 256 values.  Every warp owns a contiguous range of destinations, hence a contiguous stretch of the
// neighbour list, and keeps a private ring of rows in flight: it hands four row ids at a time to the TMA unit
// (cp.async.bulk.tensor, tile::gather4), which lands the rows in the warp's ring, and adds them up from there.  Rows in
// flight cost shared memory instead of registers: sixteen per warp against four.
// src_rows: rows of Hsrc that the ids may address.  Returns false (nothing enqueued) when the shape is not covered.
bool stream_sage_aggregate(const __nv_bfloat16 *Hsrc, int64_t src_rows, int64_t ld, const int32_t *nbr, const int32_t *self_ids,
                           const int32_t *indptr, const int32_t *counts, __nv_bfloat16 *cat, int d, int64_t cap_dst,
                           cudaStream_t st);

}  // namespace e2egrec
