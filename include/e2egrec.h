/*
 * e2egrec.h -- C ABI of the sampled-GNN training pass of E2E-GRec (arXiv 2511.20564)
 * for one NVIDIA B200 (sm_100a).
 *
 * The library runs, per training step, what the paper's Figure 1 pipeline does for
 * the GNN branch: build the sampled multi-hop subgraph of the batch (Sec. 4.1), run
 * the GraphSAGE encoder on it (Sec. 3.1, Eqs. 2-3), and send the gradient that the
 * recommendation model returns back through the encoder to its weights and to the
 * input node features (Sec. 4.3.2, gradient of L_total w.r.t. the GNN parameters).
 *
 * Conventions shared by every entry point
 * ---------------------------------------
 *  - Every pointer marked "device" is memory of the current CUDA device, allocated
 *    and owned by the caller; the library allocates no device memory and frees none.
 *    Pointers marked "host" are ordinary host memory read during the call only.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All work
 *    is enqueued on it; no entry point synchronises with the device, so results are
 *    valid once the stream reaches the end of the enqueued work.
 *  - Sizes that depend on the data (how many distinct nodes a hop reaches) stay on the
 *    device: each block carries `counts` = {n_dst, n_src, n_edges, status}; buffers are
 *    sized for the worst case reported by the *_workspace / size-query calls.
 *  - Return value: E2EGREC_OK (0) or a negative E2EGREC_ERR_* code for errors detected
 *    on the host before anything is enqueued.  Errors that only the device can see (a
 *    seed id out of range, a capacity overrun) set bits of counts[3] of the block (or of
 *    the status word named by the call) and the offending element is skipped; nothing
 *    traps, asserts or spins without a bound.
 *  - Node ids are int32 (n_nodes < 2^31), graph offsets int64, block offsets int32.
 *  - Feature matrices are row-major; dtype E2EGREC_F32 or E2EGREC_BF16; every row must
 *    start on a 16-byte boundary (dim * element size and ld * element size multiples of 16).
 *  - Size queries: where a call takes `void* buf, size_t* bytes`, calling it with
 *    buf == NULL writes the required size to *bytes and returns E2EGREC_OK without
 *    enqueuing anything; otherwise *bytes is the size provided and must be >= required.
 */
#ifndef E2EGREC_H
#define E2EGREC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define E2EGREC_OK               0
#define E2EGREC_ERR_NULL        -1   /* a required pointer is NULL */
#define E2EGREC_ERR_ARG         -2   /* a size or count is out of its documented range */
#define E2EGREC_ERR_DTYPE       -3   /* unknown dtype, or operands of one call disagree */
#define E2EGREC_ERR_ALIGN       -4   /* a row does not start on a 16-byte boundary */
#define E2EGREC_ERR_WORKSPACE   -5   /* buffer smaller than the size query reports */
#define E2EGREC_ERR_UNSUPPORTED -6   /* n_nodes >= 2^31, more than 4 hops, fanout > 128, dim > 1024 */
#define E2EGREC_ERR_CUDA        -7   /* a launch failed; e2egrec_last_error() holds the CUDA text */

/* bits of the device status word (counts[3]) */
#define E2EGREC_DEV_RANGE     1u     /* a seed / node id was outside [0, n_nodes) and was skipped */
#define E2EGREC_DEV_CAPACITY  2u     /* a buffer capacity would have been exceeded; output truncated */
#define E2EGREC_DEV_TIMEOUT   4u     /* a bounded wait inside a kernel ran out */

#define E2EGREC_F32  0
#define E2EGREC_BF16 1

/* flags of e2egrec_aggregate_forward */
#define E2EGREC_AGG_SUM 1u           /* plain sum instead of the mean */

/* flags of e2egrec_sample_khop */
#define E2EGREC_SAMPLE_DEFER_TRANSPOSE 1u   /* csc_* arrays become valid only after e2egrec_sage_backward / e2egrec_sample_join */
#define E2EGREC_SAMPLE_NO_TRANSPOSE 2u      /* csc_* arrays are not built; e2egrec_blocks_transpose builds them later */

/* flags of e2egrec_sage_backward */
#define E2EGREC_ACCUMULATE_DW 1u     /* add to dW / dbias instead of overwriting them */

/* Graph G=(V,E) in compressed sparse row form (Sec. 3, Notation): row u lists N(u),
 * parallel edges kept.  indptr: device int64[n_nodes+1]; indices: device int32[n_edges].
 * edge_cum: NULL (uniform sampling) or device uint64[n_edges], the running sums of integer edge
 * weights inside every row as e2egrec_edge_cumulate writes them; the sampler then draws a neighbour
 * with probability q_uv / sum_k q_uk (the importance sampling of Sec. 4.1 with q for omega^beta). */
typedef struct e2egrec_csr {
    int64_t         n_nodes;
    int64_t         n_edges;
    const int64_t  *indptr;
    const int32_t  *indices;
    const uint64_t *edge_cum;
} e2egrec_csr;

/* Row-major matrix on the device: `rows` x `dim`, leading dimension `ld` elements. */
typedef struct e2egrec_mat {
    void   *data;
    int64_t rows;
    int32_t dim;
    int64_t ld;
    int32_t dtype;
} e2egrec_mat;

/* One sampled hop ("block"): the bipartite graph from the frontier F_h (sources) to the
 * nodes D_h = F_{h-1} that were sampled for (destinations).  All arrays are device
 * memory of the stated capacity, provided by the caller:
 *   counts     int32[4]            {n_dst, n_src, n_edges, status bits}
 *   indptr     int32[cap_dst+1]    block CSR offsets, destination i owns [indptr[i], indptr[i+1])
 *   col        int32[cap_edges]    local source id (position in src_nodes) of each entry
 *   nbr_global int32[cap_edges]    global node id of each entry
 *   src_nodes  int32[cap_src]      F_h: the destinations first (same order), then the newly
 *                                  reached nodes in ascending id order
 *   csc_ptr    int32[cap_src+1]    transposed block: source s owns [csc_ptr[s], csc_ptr[s+1])
 *   csc_row    int32[cap_edges]    destination of each transposed entry
 *   csc_eid    int32[cap_edges]    its position in the block CSR; ascending inside a column
 *   csc_col    int32[cap_edges]    its source (the column it belongs to): csc_col[k] = s for k in column s
 *   inv_cnt    float[cap_dst]      1/|S(u)| per destination, 0 for an isolated node */
typedef struct e2egrec_block {
    int32_t  cap_dst, cap_src, cap_edges;
    int32_t *counts;
    int32_t *indptr, *col, *nbr_global, *src_nodes;
    int32_t *csc_ptr, *csc_row, *csc_eid, *csc_col;
    float   *inv_cnt;
} e2egrec_block;

/* Static text for a status code / the CUDA error text of the last E2EGREC_ERR_CUDA
 * returned on this thread ("" if none). */
const char *e2egrec_status_string(int32_t code);
const char *e2egrec_last_error(void);

/* Benchmark instrumentation (no counterpart in the paper).
 * e2egrec_launch_count: number of kernels this library has launched in this process so far.
 * e2egrec_profile_tap: arms a timing tap on the calling thread.  The next entry point that reaches
 * kernel group `which` records start_event (a cudaEvent_t) on its stream just before the group and
 * stop_event just after it, then disarms the tap.  Groups: 1 = mean aggregation of the outermost
 * block (layer 0, gathers from X), 2 = transposed aggregation of the outermost block (writes dX_rows),
 * 3 = dense transform of layer 0, 4 = weight gradient of layer 0, 5 = input gradient (dCat) of layer 0,
 * 6 = the whole of e2egrec_sample_khop, 7 / 9 = the two kernels (runs and their join; chains across windows) of
 * the first segment reduction that follows (the innermost layer's transposed aggregation in
 * e2egrec_sage_backward); 8 is unused.  which = 0 disarms. */
uint64_t e2egrec_launch_count(void);
int32_t e2egrec_profile_tap(int32_t which, void *start_event, void *stop_event);

/* Graph ingest (Sec. 3, Notation: G = (V, E), N(u)); set-up work, not part of a training step.
 * e2egrec_graph_from_coo: canonical CSR of an edge list.  row, col: device int32[n_edges]; outputs indptr
 * device int64[n_nodes+1] and indices device int32[n_edges]: row u lists its neighbours in ascending id
 * order, parallel edges kept.  The result depends only on the multiset of edges.
 * e2egrec_csr_transpose: the CSC of a CSR with n_cols columns: csc_ptr device int64[n_cols+1]; for every
 * transposed entry csc_row int32 (its row) and csc_eid int64 (its CSR position), entries of a column in
 * CSR order.  status: optional device int32, receives E2EGREC_DEV_RANGE if an id was out of range (such
 * ids are treated as 0).  ws: scratch (size query with ws == NULL).  Limits: n_edges < 2^31 - 1. */
int32_t e2egrec_graph_from_coo(int64_t n_nodes, int64_t n_edges, const int32_t *row, const int32_t *col,
                               int64_t *indptr, int32_t *indices, int32_t *status, void *ws, size_t *ws_bytes,
                               void *stream);
int32_t e2egrec_csr_transpose(const e2egrec_csr *csr, int64_t n_cols, int64_t *csc_ptr, int32_t *csc_row,
                              int64_t *csc_eid, int32_t *status, void *ws, size_t *ws_bytes, void *stream);

/* Worst-case capacities of the blocks of a k-hop sample and the scratch size
 * (Sec. 4.1: depth L, at most k neighbours per node).  fanouts: host int32[n_hops],
 * fanouts[0] is the hop taken from the seeds.  cap_dst / cap_src / cap_edges: host
 * int32[n_hops] outputs.  Limits: 1 <= n_hops <= 4, 1 <= fanout <= 128, n_nodes < 2^31. */
int32_t e2egrec_sample_khop_workspace(int64_t n_nodes, int32_t n_seeds, int32_t n_hops,
                                      const int32_t *fanouts, int32_t *cap_dst, int32_t *cap_src,
                                      int32_t *cap_edges, size_t *scratch_bytes);

/* Puts a sampler scratch buffer (device, scratch_bytes from the query above, 256-byte
 * aligned) into its idle state.  Call once after allocating it; e2egrec_sample_khop
 * leaves the buffer idle again when it finishes, so one buffer serves every step. */
int32_t e2egrec_sampler_scratch_init(int64_t n_nodes, void *scratch, size_t scratch_bytes, void *stream);

/* Table of the weighted sampler (Sec. 4.1, sampling probability p(u->v) = omega_uv^beta / sum_k omega_uk^beta).
 * q: device uint32[n_edges], the caller's integer quantisation of omega^beta per CSR entry (integers make the
 * draw exact and the sampled lists identical on every machine); cum: device uint64[n_edges], receives
 * cum[e] = q[first entry of e's row] + ... + q[e].  Set-up work, once per graph (and per beta). */
int32_t e2egrec_edge_cumulate(int64_t n_nodes, int64_t n_edges, const int64_t *indptr, const uint32_t *q,
                              uint64_t *cum, void *stream);

/* Sets the step offset kept in the sampler scratch: every later e2egrec_sample_khop that uses this
 * scratch draws with step = its `step` argument + step_offset (mod 2^32).  init sets it to 0.  This is
 * for callers that record the kernels of one training step once (a CUDA graph) and replay them: the
 * recorded `step` argument is fixed, the offset, which lives in device memory, is what moves on. */
int32_t e2egrec_sampler_set_step(void *scratch, uint32_t step_offset, void *stream);

/* k-hop neighbour sampling (Sec. 3.1: multiset S_l(u) of N(u); Sec. 4.1: sampling
 * probability with beta = 0, i.e. uniform over the stored entries of the row, at most
 * fanout neighbours per node, depth n_hops).
 *   seeds  device int32[n_seeds], distinct node ids (the batch's source nodes).
 *   Hop h = 1..n_hops samples for every node of D_h = F_{h-1} (F_0 = seeds):
 *     deg <= fanout: all stored neighbours once, in CSR order;
 *     deg  > fanout: fanout independent uniform draws with replacement.  Draw j of node u
 *       uses Philox4x32-10 with key = (seed low, seed high) and counter
 *       (j/2, u, (1<<8)|h, step); output words 2(j%2), 2(j%2)+1 form a 64-bit r and the
 *       entry picked is floor(r * deg / 2^64).  The lists are therefore a function of
 *       (seed, step, h, u) only and reproducible bit for bit.
 *       With graph->edge_cum the draw is weighted (beta > 0): t = floor(r * total / 2^64) with total
 *       the row's last running sum, and the first entry of the row whose running sum exceeds t is
 *       picked; a row whose weights sum to zero is drawn uniformly as above.
 *   blocks host array[n_hops] of structs holding device pointers; blocks[h-1] receives hop h
 *       including its transposed form.  F_h = D_h followed by the new nodes in ascending order.
 *   scratch device buffer initialised by e2egrec_sampler_scratch_init for the same n_nodes.
 *   flags 0, E2EGREC_SAMPLE_DEFER_TRANSPOSE or E2EGREC_SAMPLE_NO_TRANSPOSE.
 * The transposed form of a hop is built on a helper stream of the library (one per device and caller stream,
 * created on the first call, at the caller stream's priority, kept until the process ends) beside the sampling of
 * the next hop.  By default the call joins that work back into `stream` before it returns.  With
 * E2EGREC_SAMPLE_DEFER_TRANSPOSE it does not: indptr / col / nbr_global / src_nodes / inv_cnt / counts are valid in
 * stream order as always, but the csc_* arrays are only complete after the next e2egrec_sage_backward,
 * e2egrec_lightgcn_sampled_backward, e2egrec_sample_khop or e2egrec_sample_join that the host issues on any stream
 * of the same device: that call makes its stream wait for every transposition deferred on the device so far
 * (e2egrec_sage_forward does not need the csc_* arrays, so the forward pass overlaps the transposition).  Inside a
 * stream capture the deferring call and the joining call must belong to the same capture.  Calls that share a
 * caller stream must not be issued from two host threads at once. */
int32_t e2egrec_sample_khop(const e2egrec_csr *graph, const int32_t *seeds, int32_t n_seeds,
                            int32_t n_hops, const int32_t *fanouts, uint64_t seed, uint32_t step,
                            uint32_t flags, const e2egrec_block *blocks,
                            void *scratch, size_t scratch_bytes, void *stream);

/* Makes `stream` wait for every block transposition that e2egrec_sample_khop calls have deferred on the current device
 * (on whichever stream; no-op if there is none). */
int32_t e2egrec_sample_join(void *stream);

/* The transposed form (csc_ptr / csc_row / csc_eid / csc_col: the block's entries ordered by source, then by
 * position; what the backward aggregation of Sec. 4.1's sampled sub-graph walks) of blocks that
 * e2egrec_sample_khop filled with E2EGREC_SAMPLE_NO_TRANSPOSE.  A training loop can so build the transposed
 * form of one batch beside the sampling of the next and the forward/backward of the previous one.
 *   n_nodes, n_hops, blocks, scratch, scratch_bytes: as given to that e2egrec_sample_khop call; the scratch
 *       must not have been used by another call in between (it still holds the entries' rows and the digit
 *       counts of the columns).
 * Independent blocks run partly on the library's helper stream; all work is joined into `stream` before the
 * call returns.  Host errors: E2EGREC_ERR_NULL / _ARG / _ALIGN / _WORKSPACE, nothing is enqueued then. */
int32_t e2egrec_blocks_transpose(int64_t n_nodes, int32_t n_hops, const e2egrec_block *blocks, void *scratch,
                                 size_t scratch_bytes, void *stream);

/* GraphSAGE forward over sampled blocks (Sec. 3.1): for layer l = 0..n_layers-1, on block
 * h = n_layers - l,
 *     agg_i = (1/|S(i)|) sum_{v in S(i)} h_v                         (Eq. 2; 0 if S(i) is empty)
 *     h'_i  = act( W_l [h_i || agg_i] + b_l )                        (Eq. 3; act = ReLU or identity)
 * Layer 0 reads h = X[src_nodes] of the outermost block directly (the h^(0) lookup).
 *   X      features of all nodes, rows >= n_nodes.
 *   W      host array[n_layers]; W[l] is device [d_out x 2*d_in] row-major, same dtype as X;
 *          its first d_in columns multiply h_i, the rest multiply agg_i.
 *   bias   host array[n_layers] of device float[d_out] pointers, or NULL, or NULL entries.
 *   act    host int32[n_layers]: 1 = ReLU, 0 = identity.
 *   ctx    device buffer that keeps [h_i || agg_i] and h' of every layer for the backward pass
 *          (size query: ctx == NULL).  ctx_bytes in/out as described above.
 *   H_out  device [cap_dst(block 0) x d_L]: rows [0, n_seeds) receive the final embeddings.
 * bf16 operands are multiplied on the tensor cores with fp32 accumulation; fp32 operands use
 * fp32 FMA.  The mean is accumulated in fp32 and stored in the feature dtype. */
int32_t e2egrec_sage_forward(const e2egrec_block *blocks, int32_t n_layers, const e2egrec_mat *X,
                             const e2egrec_mat *W, const float *const *bias, const int32_t *act,
                             void *ctx, size_t *ctx_bytes, const e2egrec_mat *H_out, void *stream);

/* Where e2egrec_sage_forward keeps its activations inside ctx (for callers that want the
 * intermediate embeddings, Sec. 3.1 H^(l)): for layer l, cat_offset[l] is the byte offset of
 * [h_i || agg_i], a row-major [rows[l] x 2*d_in] matrix, and h_offset[l] that of the layer output
 * h', [rows[l] x d_out]; rows[l] is the destination capacity of the layer's block rounded up to a
 * multiple of 128; only the first n_dst rows are meaningful.  All three are host arrays[n_layers]. */
int32_t e2egrec_sage_ctx_layout(const e2egrec_block *blocks, int32_t n_layers, const e2egrec_mat *X,
                                const e2egrec_mat *W, size_t *cat_offset, size_t *h_offset, int64_t *rows);

/* Backward of e2egrec_sage_forward (Sec. 4.3.2: the GNN receives J^T times the gradient at
 * its output; chain of Sec. 4.2).  dH_out: gradient w.r.t. H_out, same shape and dtype.
 *   dW     host array[n_layers] of device float[d_out x 2*d_in]   (always fp32)
 *   dbias  host array[n_layers] of device float[d_out], or NULL / NULL entries to skip
 *   dX_rows device [cap_src(outermost block) x d_0], feature dtype: gradient w.r.t. the rows
 *          X[src_nodes[i]]; row i belongs to node blocks[n_layers-1].src_nodes[i] (distinct ids).
 *   scratch device buffer (size query: scratch == NULL).
 * The transposed aggregation runs as a gather over the block's csc arrays: no floating-point
 * atomics, results are bit-identical from run to run. */
int32_t e2egrec_sage_backward(const e2egrec_block *blocks, int32_t n_layers, const e2egrec_mat *X,
                              const e2egrec_mat *W, const int32_t *act, const void *ctx,
                              const e2egrec_mat *dH_out, float *const *dW, float *const *dbias,
                              const e2egrec_mat *dX_rows, void *scratch, size_t *scratch_bytes,
                              uint32_t flags, void *stream);

/* e2egrec_sage_backward for several gradients in one pass (Sec. 4.3.1, gradient-based task weighting: G_i(t), the norm
 * of each task's gradient with respect to the shared input h^(0), needs the input gradient of every task at every step;
 * Sec. 4.3.2, the GNN receives w_SSL grad L_SSL + w_r J^T dL_reward/dF_gnn + ...).  dH_out and dX_rows are host arrays of
 * n_rhs (1 or 2) matrices: gradient r arrives as dH_out[r] and its input-feature gradient leaves as dX_rows[r] (all of one
 * shape, dtype and leading dimension; see e2egrec_sage_backward).  dW and dbias receive the sum over the gradients, so a
 * caller folds the task weights into dH_out.  Every layer runs each of its kernels once for all gradients: their rows are
 * stacked in the dense products (the weight gradient contracts over both stacks at once), and the transposed aggregation
 * walks the block's csc arrays for both in one launch.  Each dX_rows[r] equals what e2egrec_sage_backward returns for
 * dH_out[r] alone, bit for bit; dW equals the sum of the separate calls up to the order of the fp32 additions.
 * scratch: size query with scratch == NULL (it depends on n_rhs). */
int32_t e2egrec_sage_backward_multi(const e2egrec_block *blocks, int32_t n_layers, const e2egrec_mat *X,
                                    const e2egrec_mat *W, const int32_t *act, const void *ctx,
                                    const e2egrec_mat *dH_out, int32_t n_rhs, float *const *dW, float *const *dbias,
                                    const e2egrec_mat *dX_rows, void *scratch, size_t *scratch_bytes,
                                    uint32_t flags, void *stream);

/* One joint training step of the GNN and the ranking model (Theorem 1: z_i = [h_theta(x_i) || b_i] is the
 * scorer's input, so the ranking loss reaches the GNN; Sec. 4.2 chain rule; binary cross-entropy as
 * in Sec. 5.1).  For n_pairs training pairs (user u_p, item i_p, dense features b_p, label y_p):
 *   seeds  = the distinct endpoints of the pairs in ascending id order;
 *   blocks = k-hop sample of the seeds (as e2egrec_sample_khop);  h = GraphSAGE(X) on the seeds
 *            (as e2egrec_sage_forward, ReLU on every layer, no bias);
 *   z_p    = [h(u_p) || h(i_p) || b_p];  a1 = ReLU(W_t0 z + b_t0);  a2 = ReLU(W_t1 a1 + b_t1);
 *   t_p    = W_t2 a2 + b_t2;  loss = mean_p [max(t,0) - y t + log(1 + exp(-|t|))];
 *   then the full backward: tower weights and biases, the encoder weights, and the feature rows.
 * Arguments (device memory unless "host"):
 *   pair_user, pair_item int32[n_pairs] global node ids; dense float[n_pairs x dense_dim]; labels float[n_pairs];
 *   W_gnn host array[n_hops] (as in e2egrec_sage_forward); W_tower host array[3] of matrices
 *   [h1 x (2 d_L + dense_dim)], [h2 x h1], [1 x h2] in the dtype of X; b_tower host array[3] of device
 *   float vectors, or NULL (entries may be NULL);
 *   loss float[1]; logits float[n_pairs]; dW_gnn / dW_tower host arrays of device float matrices of the
 *   weights' shapes; db_tower host array[3] of device float vectors or NULL;
 *   dX_rows [cap_src of the outermost block x d_0] and dX_ids int32[same capacity]: gradient rows and the
 *   node id of each row; n_dX_rows int32[2] = {number of valid rows, device status bits of the step}.
 *   ws: workspace (size query with ws == NULL).  Its head is a sampler scratch: initialise it once with
 *   e2egrec_sampler_scratch_init(n_nodes, ws, ws_bytes, stream).  n_pairs a multiple of 128 and all
 *   widths multiples of 64 take the tensor-core kernels for bf16; other shapes use fp32-FMA kernels.
 * With bf16 storage z, a1, a2 and the gradients flowing between the layers are stored as bf16; logits,
 * loss and all weight gradients are fp32. */
int32_t e2egrec_joint_step(const e2egrec_csr *graph, const e2egrec_mat *X, const int32_t *pair_user,
                           const int32_t *pair_item, int32_t n_pairs, const float *dense, int32_t dense_dim,
                           const float *labels, int32_t n_hops, const int32_t *fanouts,
                           const e2egrec_mat *W_gnn, const e2egrec_mat *W_tower, const float *const *b_tower,
                           uint64_t seed, uint32_t step, float *loss, float *logits, float *const *dW_gnn,
                           float *const *dW_tower, float *const *db_tower, const e2egrec_mat *dX_rows,
                           int32_t *dX_ids, int32_t *n_dX_rows, void *ws, size_t *ws_bytes, void *stream);

/* The joint step in two phases, for callers that prepare the sub-graph of the next batch (Sec. 4.1: "constructed in
 * real time") while the current batch trains: phase E2EGREC_JOINT_SAMPLE derives the seeds from the pairs and samples
 * the blocks into ws (only graph, the pairs, fanouts, seed, step and ws are read; the other arguments fix the layout
 * of ws and must be the ones of the later call); phase E2EGREC_JOINT_COMPUTE runs everything else of
 * e2egrec_joint_step on the blocks that a SAMPLE call with the same shapes left in ws (the two calls may be issued
 * on different streams; the caller orders them).  E2EGREC_JOINT_WHOLE is e2egrec_joint_step. */
#define E2EGREC_JOINT_WHOLE   0u
#define E2EGREC_JOINT_SAMPLE  1u
#define E2EGREC_JOINT_COMPUTE 2u
/* Options, or-ed into `phase` (they fix the layout of ws, so every call on one workspace passes the same ones):
 * E2EGREC_JOINT_LINEAR  identity activations in every encoder layer and in both hidden tower layers (a linear ranking
 *     model; also what lets a test hold every gradient element to the plain tolerance, since no sign is decided).
 * E2EGREC_JOINT_GATE    concatenation with gating (Sec. 4.3.2): the tower reads z_fused = g * z with
 *     g = sigmoid(W_g z + b_g) instead of z.  W_tower, b_tower, dW_tower and db_tower then have a fourth entry each:
 *     W_tower[3] = W_g [zdim x zdim] (zdim = 2 d_L + dense_dim), b_tower[3] = b_g (device float[zdim] or NULL),
 *     dW_tower[3] (device float[zdim x zdim]) and db_tower[3] (device float[zdim] or NULL) receive their gradients.
 *     For bf16 shapes the tensor-core kernel takes, sigmoid and the product with z run in the epilogue of the W_g
 *     product; the pre-activation, g and z_fused are stored as bf16, as are the gradients between the steps. */
#define E2EGREC_JOINT_LINEAR  0x100u
#define E2EGREC_JOINT_GATE    0x200u
int32_t e2egrec_joint_step_phase(const e2egrec_csr *graph, const e2egrec_mat *X, const int32_t *pair_user,
                                 const int32_t *pair_item, int32_t n_pairs, const float *dense, int32_t dense_dim,
                                 const float *labels, int32_t n_hops, const int32_t *fanouts,
                                 const e2egrec_mat *W_gnn, const e2egrec_mat *W_tower, const float *const *b_tower,
                                 uint64_t seed, uint32_t step, float *loss, float *logits, float *const *dW_gnn,
                                 float *const *dW_tower, float *const *db_tower, const e2egrec_mat *dX_rows,
                                 int32_t *dX_ids, int32_t *n_dX_rows, void *ws, size_t *ws_bytes, uint32_t phase,
                                 void *stream);

/* Where a joint step keeps its activations inside ws (for callers that want the intermediate embeddings of Sec. 3.1
 * or the tower's hidden layers; the arguments are those of the step, flags = the options or-ed into its `phase`).
 *   tower_offset  host size_t[5]: byte offsets of z, a1, a2, the gate g and z_fused (the last two equal z's offset
 *                 without E2EGREC_JOINT_GATE); row-major [*pair_rows x width] in X's dtype, widths zdim, h1, h2, zdim,
 *                 zdim; *pair_rows = n_pairs rounded up to 128, rows >= n_pairs are zero.
 *   enc_h_offset  host size_t[n_hops], enc_rows host int64[n_hops]: the output of encoder layer l, row-major
 *                 [enc_rows[l] x d_out(l)]; only the first n_dst rows of the layer's block are meaningful.
 *   counts_offset host size_t[n_hops]: the int32[4] counts {n_dst, n_src, n_edges, status} of the block of hop h+1. */
int32_t e2egrec_joint_step_layout(const e2egrec_csr *graph, const e2egrec_mat *X, int32_t n_pairs, int32_t dense_dim,
                                  int32_t n_hops, const int32_t *fanouts, const e2egrec_mat *W_gnn,
                                  const e2egrec_mat *W_tower, uint32_t flags, size_t *tower_offset, size_t *enc_h_offset,
                                  int64_t *enc_rows, int64_t *pair_rows, size_t *counts_offset);

/* Whole-graph neighbourhood aggregation without sampling (Sec. 3.1 Eq. 2 with S(u) = N(u); the
 * "complete graph" case of Sec. 4.1):  out[i] = (1/deg i) sum_{e in row i} X[indices[e]]  (0 for an
 * empty row; the plain sum with E2EGREC_AGG_SUM).  indptr: device int64[n_dst+1], indices: device
 * int32[n_entries]; X has a row for every id in indices; out has n_dst rows, same dtype and dim.
 * Rows of any degree are split over many warps; partial sums are added in a fixed order (no atomics).
 * ws: device scratch, 256-byte aligned (size query: ws == NULL). */
int32_t e2egrec_aggregate_forward(int64_t n_dst, int64_t n_entries, const int64_t *indptr,
                                  const int32_t *indices, const e2egrec_mat *X, const e2egrec_mat *out,
                                  uint32_t flags, void *ws, size_t *ws_bytes, void *stream);

/* Its transpose, run as a gather over the CSC form of the same matrix (Sec. 4.3.2: J^T applied to the
 * incoming gradient):  dX[s] = sum_{k in column s} inv_deg[csc_row[k]] * G[csc_row[k]].
 * csc_ptr: device int64[n_src+1], csc_row: device int32[n_entries] (the destination of each entry),
 * inv_deg: device float[n_dst] = 1/deg (pass 1.0 everywhere for the transposed sum), G: gradient
 * w.r.t. out, dX: n_src rows. */
int32_t e2egrec_aggregate_backward(int64_t n_src, int64_t n_entries, const int64_t *csc_ptr,
                                   const int32_t *csc_row, const float *inv_deg, const e2egrec_mat *G,
                                   const e2egrec_mat *dX, void *ws, size_t *ws_bytes, void *stream);

/* LightGCN propagation over the whole graph (Sec. 3.1, Eqs. 4-7): H^(l+1) = A_hat H^(l) with
 * A_hat[u][i] = (number of stored entries (u, i)) * s[u] * s[i], s = inv_sqrt_deg (1/sqrt(|N(u)|), 0 for an
 * isolated node; device float[n_nodes], supplied by the caller), and Y = (1/(L+1)) sum_{l=0..L} H^(l).
 * H0 and Y are [n_nodes x dim] dense (ld = dim) matrices of one dtype; every H^(l) is stored in that dtype,
 * Y is rounded once from the fp32 sum of the layers.  e2egrec_lightgcn_backward is the adjoint,
 * dH0 = (1/(L+1)) sum_l (A_hat^T)^l dY, and takes the CSC arrays of the same graph (for a graph stored in
 * both directions they equal the CSR arrays).  The products run on the segment-reduction kernels of the
 * mean aggregation with a per-entry and a per-row weight.  ws: scratch (size query with ws == NULL);
 * 0 <= n_layers <= 8. */
int32_t e2egrec_lightgcn_forward(int64_t n_nodes, int64_t n_entries, const int64_t *indptr,
                                 const int32_t *indices, const float *inv_sqrt_deg, int32_t n_layers,
                                 const e2egrec_mat *H0, const e2egrec_mat *Y, void *ws, size_t *ws_bytes,
                                 void *stream);
int32_t e2egrec_lightgcn_backward(int64_t n_nodes, int64_t n_entries, const int64_t *csc_ptr,
                                  const int32_t *csc_row, const float *inv_sqrt_deg, int32_t n_layers,
                                  const e2egrec_mat *dY, const e2egrec_mat *dH0, void *ws, size_t *ws_bytes,
                                  void *stream);

/* LightGCN on sampled blocks (Sec. 3.1, Eqs. 4-7, on the sub-graph of Sec. 4.1; the paper's default backbone).
 * Layer l = 0 .. L-1 runs on block L-1-l:  H^(l+1)_i = t_i * sum_{e in S(i)} s_{v(e)} H^(l)_{v(e)}  with
 * s_v = inv_sqrt_deg[v] = 1/sqrt|N(v)| (device float[n_nodes], supplied by the caller, 0 for an isolated node) and
 * t_i = sqrt|N(i)| / |S(i)|: the sum over N(i) of Eqs. 4-5 estimated from the sampled multiset, equal to the entry of
 * A_hat when S(i) = N(i).  H^(0) = X rows of the outermost frontier; Y_i = (1/(L+1)) sum_{l=0..L} H^(l)_i on the seed
 * rows i < n_seeds (Eq. 7), Y: [>= blocks[0].cap_dst x dim].  Every H^(l) is stored in X's dtype, Y is rounded once
 * from the fp32 sum.  ctx: device buffer (size query with ctx == NULL) that keeps the scales for the backward call.
 * e2egrec_lightgcn_sampled_backward is the adjoint with respect to those X rows: dX_rows [>= blocks[L-1].cap_src x dim],
 * aligned with blocks[L-1].src_nodes; dY: [>= blocks[0].cap_dst x dim], rows >= n_seeds ignored.  Storage points:
 * dY/(L+1), every propagated gradient, and the seed rows after dY/(L+1) has been added to them.  It needs the csc_*
 * arrays of the blocks (a deferred transposition is joined first).  scratch: size query with scratch == NULL. */
int32_t e2egrec_lightgcn_sampled_forward(const e2egrec_block *blocks, int32_t n_hops, const e2egrec_mat *X,
                                         const float *inv_sqrt_deg, void *ctx, size_t *ctx_bytes,
                                         const e2egrec_mat *Y, void *stream);
int32_t e2egrec_lightgcn_sampled_backward(const e2egrec_block *blocks, int32_t n_hops, const void *ctx,
                                          const e2egrec_mat *dY, const e2egrec_mat *dX_rows, void *scratch,
                                          size_t *scratch_bytes, void *stream);

/* The self-supervised task of the GNN and the balancing of the two losses (the SSL task: Sec. 4.2; the
 * gradient-based task weighting: Sec. 4.3.1).
 * e2egrec_ssl_loss: graph feature auto-encoder with the identity decoder, L_ssl = || X_seeds - H ||_F^2 over the rows
 *   i < *n_rows_dev (NULL: all H->rows rows) with X_seeds[i] = X[seed_ids[i]]; loss: device float[1] (unweighted);
 *   dH [>= H->rows x dim] receives the gradient of weight[0] * L_ssl with respect to H, 2 weight (H - X), in H's
 *   dtype (weight: device float[1], so that a weight updated on the device feeds the next step without a host round
 *   trip).  H is the encoder output (e2egrec_sage_forward's H_out), whose width must equal X's.
 * e2egrec_gradient_norm: || A[:n_rows] ||_2 into norm (device float[1]): GradNorm's gradient norm of one task with
 *   respect to the shared input rows (the dX_rows of a backward pass run with that task's gradient alone).
 *   e2egrec_gradient_norms does the same for n <= 4 matrices of one shape and dtype in one pass (A: host array[n],
 *   norms: device float[n]): the norms of all tasks of a step, e.g. of the results of e2egrec_sage_backward_multi.
 * e2egrec_gradnorm_update: one GradNorm step for n_tasks <= 8 weights w (device, updated in place) from the current
 *   and initial losses L, L0 and the norms g of the unweighted task gradients (G_i = w_i g_i): with r_i =
 *   (L_i/L0_i) / mean_j (L_j/L0_j) and the targets c_i = mean(G) r_i^gamma held constant, w_i takes one step of size
 *   lr down the gradient sign(G_i - c_i) g_i of sum_i |G_i - c_i|, stays >= 1e-6 and the weights are rescaled to sum
 *   to n_tasks; L_gn (optional, device float[1]) receives the objective.  The paper fixes gamma = 1 and leaves lr open.
 * ws: scratch (size query with ws == NULL).  All sums run in a fixed order. */
int32_t e2egrec_ssl_loss(const e2egrec_mat *H, const e2egrec_mat *X, const int32_t *seed_ids, const int32_t *n_rows_dev,
                         const float *weight, float *loss, const e2egrec_mat *dH, void *ws, size_t *ws_bytes,
                         void *stream);
int32_t e2egrec_gradient_norm(const e2egrec_mat *A, const int32_t *n_rows_dev, float *norm, void *ws, size_t *ws_bytes,
                              void *stream);
int32_t e2egrec_gradient_norms(const e2egrec_mat *A, int32_t n, const int32_t *n_rows_dev, float *norms, void *ws,
                               size_t *ws_bytes, void *stream);
int32_t e2egrec_gradnorm_update(float *w, const float *L, const float *L0, const float *g, int32_t n_tasks, float gamma,
                                float lr, float *L_gn, void *stream);

/* Feature fusion by concatenation with gating (Sec. 4.3.2):  g = sigmoid(F Wg^T + bg),  F_fused = g * F, for the
 * n_rows rows of F [rows x d] (the concatenated feature groups, GNN output among them); Wg [d x d] row-major in F's
 * dtype, bg device float[d] or NULL.  gate and fused: [>= n_rows x d] outputs (the gate is kept for the backward call).
 * e2egrec_gate_fusion_backward: dF = dFused * g + (dFused * F * g (1 - g)) Wg, dWg = (dFused * F * g (1 - g))^T F
 * (device float[d x d]), dbg its column sums (device float[d] or NULL).  F must have at least n_rows rounded up to 128
 * rows allocated, holding finite values (the dense products read whole 128-row tiles); bf16 shapes with d a multiple
 * of 64 and ld = d run on the tensor cores, others on fp32 FMA.  With bf16 the pre-activation, the gate, the fused
 * features and the intermediate gradients are stored as bf16.  ws: scratch (size query with ws == NULL). */
int32_t e2egrec_gate_fusion_forward(const e2egrec_mat *F, int32_t n_rows, const e2egrec_mat *Wg, const float *bg,
                                    const e2egrec_mat *gate, const e2egrec_mat *fused, void *ws, size_t *ws_bytes,
                                    void *stream);
int32_t e2egrec_gate_fusion_backward(const e2egrec_mat *dFused, const e2egrec_mat *F, int32_t n_rows,
                                     const e2egrec_mat *gate, const e2egrec_mat *Wg, const e2egrec_mat *dF, float *dWg,
                                     float *dbg, void *ws, size_t *ws_bytes, void *stream);

/* e2egrec_aggregate_forward without a workspace argument (the paper has no counterpart; this is a
 * packaging variant of the call above: it enqueues the same kernels with the same launch shapes, so its
 * output equals that call's bit for bit).
 *
 * Who needs it: code that is not allowed to obtain device memory at the point where it aggregates --
 * a plug-in running inside a host application that owns the whole memory pool, a step executed while
 * an allocator lock is held or inside a region where cudaMalloc would synchronise the device, or a
 * process started with all memory already handed out.  Such callers can still pass their inputs and
 * the output matrix, but have no way to size and provide `ws`.
 *
 * Here the partial-sum scratch is an 8 MiB array built into the library (every GPU that loads the
 * library holds it until the process ends; e2egrec_aggregate_forward_static_limit() returns the size).
 * The call allocates and frees nothing.  A problem fits if the scratch size that
 * e2egrec_aggregate_forward's size query reports for the same n_entries, dim and dtype is at most
 * 8 MiB: e.g. about 260 thousand entries of 1024 fp32 values, or about 130 million entries of 64 bf16 values.
 * Larger inputs are rejected with E2EGREC_ERR_WORKSPACE and e2egrec_last_error() then says how many
 * bytes were needed; nothing is enqueued in that case.
 *
 * The first call on each device looks up the device address of the built-in array (with that device
 * current).  Make that first call outside any stream capture.  All calls on a device share the one
 * array, and it keeps whatever the previous call left in it: nothing in it has to start at zero,
 * because each call writes every partial sum before it reads it, but two calls whose kernels can run
 * at the same time on one GPU (different streams, different host threads) would overwrite each
 * other's partial sums -- keep calls on one device in stream order.
 * Arguments, layout, flags and error codes otherwise as for e2egrec_aggregate_forward. */
int32_t e2egrec_aggregate_forward_static(int64_t n_dst, int64_t n_entries, const int64_t *indptr,
                                         const int32_t *indices, const e2egrec_mat *X, const e2egrec_mat *out,
                                         uint32_t flags, void *stream);
size_t e2egrec_aggregate_forward_static_limit(void);

#ifdef __cplusplus
}
#endif
#endif /* E2EGREC_H */
