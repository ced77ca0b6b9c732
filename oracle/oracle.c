/*
 * CPU oracle for the sampled-GNN training pass of E2E-GRec (arXiv 2511.20564).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * GPU library must compute.  It shares no code, header, table or helper with the
 * CUDA sources; only tests, the smoke check and the benchmark's CPU-baseline leg
 * may build or call it.  Everything is scalar C with double accumulation; there
 * is no blocking, fusion or reordering beyond what each definition states.
 *
 * Every function carries the passage of the paper it follows.  Where the paper
 * leaves a choice open (sampling with replacement, degree <= fanout, isolated
 * nodes, frontier order, random-number contract, bf16 storage points) the
 * reading taken is stated at the function.
 *
 * Pins (tests that tie each function to something other than itself):
 *   philox4x32_10        published known-answer vectors; independent big-int restatement
 *   csr_from_coo         dense adjacency by brute force; numpy lexsort
 *   csr_transpose        dense transpose; round trip
 *   sample_hop           subset / count / take-all invariants; chi-square uniformity;
 *                        fanout >= max degree reproduces the full neighbourhood
 *   relabel, block_csc   src_nodes[col[e]] == nbr[e]; dense block transpose
 *   mean_aggregate       dense D^-1 A X; mean of a constant; scipy sparse product
 *   sage_update          numpy matmul; ReLU special cases
 *   *_backward           adjoint identity; central finite differences in double
 *   tower / bce          closed form at logit 0; finite differences; numpy restatement
 *   round_bf16           torch float32 -> bfloat16 conversion
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Threads.  The loops over destination rows (or over feature columns, where rows collide) carry an OpenMP
 * pragma so that the oracle can be timed on one core and on all of them.  Every output element is still
 * produced by one thread that adds its terms in the order written here, so the results do not depend on
 * the number of threads. */
int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int n)
{
#ifdef _OPENMP
    omp_set_num_threads(n > 0 ? n : 1);
#else
    (void)n;
#endif
}

/* ------------------------------------------------------------------------- */
/* Storage rounding                                                           */
/* ------------------------------------------------------------------------- */

/* Nearest bfloat16 value (8 significant bits, ties to even) of a double.
 * Used only at the storage points of the bf16 contract: features and weights
 * on input, the mean after division, each layer output after activation, and
 * the gradient rows written between backward steps. */
double oracle_round_bf16(double x)
{
    if (x == 0.0 || isnan(x) || isinf(x)) return x;
    int e;
    double m = frexp(x, &e);            /* x = m * 2^e, 0.5 <= |m| < 1 */
    double r = nearbyint(m * 256.0);     /* default rounding mode: ties to even */
    return ldexp(r, e - 8);
}

void oracle_round_bf16_array(double *a, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) a[i] = oracle_round_bf16(a[i]);
}

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as   */
/* easy as 1, 2, 3", SC'11).  The paper names no generator; the sampler's     */
/* draws are defined through this one so that index lists are reproducible.   */
/* ------------------------------------------------------------------------- */

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;               /* key schedule: golden-ratio / sqrt(3)-1 Weyl steps */
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* ------------------------------------------------------------------------- */
/* Graph ingest (Sec. 3, Notation: G=(V,E), A, N(u))                          */
/* ------------------------------------------------------------------------- */

static int cmp_i32(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/* Canonical CSR of an edge list: row u holds N(u) as a multiset (parallel edges
 * kept), entries of a row in ascending column order.  Returns 0, or -1 on an id
 * out of range. */
int oracle_csr_from_coo(int64_t n, int64_t m, const int32_t *row, const int32_t *col,
                        int64_t *indptr, int32_t *indices)
{
    for (int64_t u = 0; u <= n; ++u) indptr[u] = 0;
    for (int64_t e = 0; e < m; ++e) {
        if (row[e] < 0 || row[e] >= n || col[e] < 0 || col[e] >= n) return -1;
        indptr[row[e] + 1] += 1;
    }
    for (int64_t u = 0; u < n; ++u) indptr[u + 1] += indptr[u];
    int64_t *fill = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n > 0 ? n : 1));
    for (int64_t u = 0; u < n; ++u) fill[u] = indptr[u];
    for (int64_t e = 0; e < m; ++e) indices[fill[row[e]]++] = col[e];
    free(fill);
    for (int64_t u = 0; u < n; ++u)
        qsort(indices + indptr[u], (size_t)(indptr[u + 1] - indptr[u]), sizeof(int32_t), cmp_i32);
    return 0;
}

/* Transpose of a CSR matrix with n_rows rows and n_cols columns: column s lists
 * the rows that hold s, ordered by CSR position (hence by row, then by position
 * in the row); eid is that CSR position. */
void oracle_csr_transpose(int64_t n_rows, int64_t n_cols, const int64_t *indptr, const int32_t *indices,
                          int64_t *csc_ptr, int32_t *csc_row, int64_t *csc_eid)
{
    for (int64_t s = 0; s <= n_cols; ++s) csc_ptr[s] = 0;
    for (int64_t e = 0; e < indptr[n_rows]; ++e) csc_ptr[indices[e] + 1] += 1;
    for (int64_t s = 0; s < n_cols; ++s) csc_ptr[s + 1] += csc_ptr[s];
    int64_t *fill = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n_cols > 0 ? n_cols : 1));
    for (int64_t s = 0; s < n_cols; ++s) fill[s] = csc_ptr[s];
    for (int64_t u = 0; u < n_rows; ++u)
        for (int64_t e = indptr[u]; e < indptr[u + 1]; ++e) {
            int64_t k = fill[indices[e]]++;
            csc_row[k] = (int32_t)u;
            csc_eid[k] = e;
        }
    free(fill);
}

/* ------------------------------------------------------------------------- */
/* Neighbour sampling (Sec. 3.1 GraphSAGE: "sample a multiset S_l(u) of       */
/* N(u) of size m_l"; Sec. 4.1: per-draw probability p_{u->v} ~ w_uv^beta,    */
/* number of sampled neighbours bounded by k)                                 */
/* ------------------------------------------------------------------------- */

/* Running sums of the integer edge weights inside every row: cum[e] = q[row begin] + ... + q[e].
 * q_e is the caller's quantisation of omega_e^beta (Sec. 4.1); the integers make the weighted draw
 * exact and identical on every machine. */
void oracle_edge_cumulate(int64_t n_nodes, const int64_t *indptr, const uint32_t *q, uint64_t *cum)
{
    for (int64_t u = 0; u < n_nodes; ++u) {
        uint64_t run = 0;
        for (int64_t e = indptr[u]; e < indptr[u + 1]; ++e) {
            run += q[e];
            cum[e] = run;
        }
    }
}

/* One hop.  For every destination u = dst_nodes[i]:
 *   deg <= fanout : S(u) = N(u), every stored entry once, in CSR order
 *                   (k is an upper bound; the mean is then exact);
 *   deg  > fanout : fanout independent draws with replacement (a multiset),
 *                   each uniform over the stored entries of the row, i.e.
 *                   beta = 0, or w = edge multiplicity with beta = 1.
 * Draw j of node u at hop h of step t uses Philox with
 *   key = (seed low word, seed high word),
 *   counter = (j / 2, u, (1 << 8) | h, t),
 * takes output words (2*(j%2), 2*(j%2)+1) as the low and high half of a 64-bit
 * number r and picks entry floor(r * deg / 2^64) of the row.  The counter holds
 * the global node id, so S(u) does not depend on which other nodes share the
 * batch or on their order.
 * With g_cum (the per-row running sums of integer edge weights q_e, see
 * oracle_edge_cumulate) a draw is weighted instead: p(u -> v) = q_uv / sum_k q_uk,
 * the sampling probability of Sec. 4.1 with q standing for omega^beta; t =
 * floor(r * total / 2^64) and the first entry whose running sum exceeds t is
 * picked.  A row whose weights sum to zero is drawn uniformly.
 * Outputs: blk_indptr[n_dst+1] (prefix sums of |S(u)|), nbr_global[...] (global
 * ids, row after row).  Returns the number of entries written. */
int64_t oracle_sample_hop(const int64_t *g_indptr, const int32_t *g_indices, const uint64_t *g_cum,
                          const int32_t *dst_nodes, int32_t n_dst, int32_t fanout,
                          uint64_t seed, uint32_t step, int32_t hop,
                          int32_t *blk_indptr, int32_t *nbr_global)
{
    int64_t w = 0;
    blk_indptr[0] = 0;
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    for (int32_t i = 0; i < n_dst; ++i) {
        int64_t u = dst_nodes[i];
        int64_t beg = g_indptr[u], deg = g_indptr[u + 1] - beg;
        if (deg <= fanout) {
            for (int64_t p = 0; p < deg; ++p) nbr_global[w++] = g_indices[beg + p];
        } else {
            for (int32_t j = 0; j < fanout; ++j) {
                uint32_t ctr[4] = { (uint32_t)(j >> 1), (uint32_t)u, (1u << 8) | (uint32_t)hop, step };
                uint32_t out[4];
                oracle_philox4x32_10(ctr, key, out);
                int half = j & 1;
                uint64_t r = ((uint64_t)out[2 * half + 1] << 32) | out[2 * half];
                uint64_t pos;
                uint64_t total = g_cum ? g_cum[beg + deg - 1] : 0;
                if (total > 0) {
                    /* importance sampling (Sec. 4.1): t is uniform over [0, total), the entry whose interval
                     * [cum[e-1], cum[e]) holds t is drawn, i.e. entry e with probability q_e / total */
                    uint64_t t = (uint64_t)(((unsigned __int128)r * (unsigned __int128)total) >> 64);
                    pos = 0;
                    while (g_cum[beg + (int64_t)pos] <= t) ++pos;
                } else {
                    pos = (uint64_t)(((unsigned __int128)r * (unsigned __int128)(uint64_t)deg) >> 64);
                }
                nbr_global[w++] = g_indices[beg + (int64_t)pos];
            }
        }
        blk_indptr[i + 1] = (int32_t)w;
    }
    return w;
}

/* Frontier of the hop: F = D ++ (ascending distinct sampled ids not in D), and
 * the block's column ids col[e] = position of nbr_global[e] in F.  The paper
 * speaks only of "the subgraph"; this order is the canonical one chosen here.
 * dst_nodes must be distinct.  Returns |F| (or -1 on an id out of range). */
int32_t oracle_relabel(int64_t n_nodes, const int32_t *dst_nodes, int32_t n_dst,
                       const int32_t *nbr_global, int64_t n_edges,
                       int32_t *src_nodes, int32_t *col)
{
    int32_t *local = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_nodes > 0 ? n_nodes : 1));
    for (int64_t v = 0; v < n_nodes; ++v) local[v] = -1;
    for (int32_t i = 0; i < n_dst; ++i) {
        if (dst_nodes[i] < 0 || dst_nodes[i] >= n_nodes) { free(local); return -1; }
        local[dst_nodes[i]] = i;
        src_nodes[i] = dst_nodes[i];
    }
    int32_t n_new = 0;
    for (int64_t e = 0; e < n_edges; ++e) {
        int32_t v = nbr_global[e];
        if (local[v] == -1) { local[v] = -2; src_nodes[n_dst + n_new++] = v; }
    }
    qsort(src_nodes + n_dst, (size_t)n_new, sizeof(int32_t), cmp_i32);
    for (int32_t r = 0; r < n_new; ++r) local[src_nodes[n_dst + r]] = n_dst + r;
    for (int64_t e = 0; e < n_edges; ++e) col[e] = local[nbr_global[e]];
    free(local);
    return n_dst + n_new;
}

/* Transposed block (needed by the backward pass, Sec. 4.3.2: the GNN receives
 * J^T times the upstream gradient): for every source s the destinations that
 * sampled it, ordered by block-CSR position; plus 1/|S(u)| per destination in
 * single precision (0 for an isolated destination). */
void oracle_block_csc(int32_t n_dst, int32_t n_src, const int32_t *blk_indptr, const int32_t *col,
                      int32_t *csc_ptr, int32_t *csc_row, int32_t *csc_eid, float *inv_cnt)
{
    for (int32_t s = 0; s <= n_src; ++s) csc_ptr[s] = 0;
    for (int32_t e = 0; e < blk_indptr[n_dst]; ++e) csc_ptr[col[e] + 1] += 1;
    for (int32_t s = 0; s < n_src; ++s) csc_ptr[s + 1] += csc_ptr[s];
    int32_t *fill = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_src > 0 ? n_src : 1));
    for (int32_t s = 0; s < n_src; ++s) fill[s] = csc_ptr[s];
    for (int32_t i = 0; i < n_dst; ++i) {
        int32_t cnt = blk_indptr[i + 1] - blk_indptr[i];
        inv_cnt[i] = cnt > 0 ? 1.0f / (float)cnt : 0.0f;
        for (int32_t e = blk_indptr[i]; e < blk_indptr[i + 1]; ++e) {
            int32_t k = fill[col[e]]++;
            csc_row[k] = i;
            csc_eid[k] = e;
        }
    }
    free(fill);
}

/* ------------------------------------------------------------------------- */
/* Forward pass (Sec. 3.1, GraphSAGE)                                         */
/* ------------------------------------------------------------------------- */

/* h^(0) = X: rows of the feature matrix for the given node ids ("embedding lookup"). */
void oracle_gather_rows(const double *X, int64_t ld, const int32_t *ids, int64_t n, int32_t d, double *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        for (int32_t k = 0; k < d; ++k) out[i * d + k] = X[(int64_t)ids[i] * ld + k];
}

/* Mean aggregation (Eq. 2): agg_i = (1/|S(i)|) * sum over the row's entries of
 * H[col[e]].  An empty row gives 0.  With round_bf16 the mean is stored as bf16. */
void oracle_mean_aggregate(const int64_t *indptr, const int32_t *col, int64_t n_dst,
                           const double *H, int32_t d, double *agg, int round_bf16)
{
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t i = 0; i < n_dst; ++i) {
        int64_t cnt = indptr[i + 1] - indptr[i];
        for (int32_t k = 0; k < d; ++k) {
            double s = 0.0;
            for (int64_t e = indptr[i]; e < indptr[i + 1]; ++e) s += H[(int64_t)col[e] * d + k];
            double a = cnt > 0 ? s / (double)cnt : 0.0;
            agg[i * d + k] = round_bf16 ? oracle_round_bf16(a) : a;
        }
    }
}

/* Update (Eq. 3): z_i = W * CONCAT(h_i, agg_i) (+ b), h'_i = sigma(z_i) with
 * sigma = ReLU when act != 0 and the identity otherwise.  W is [d_out x 2*d_in]
 * row-major; its first d_in columns meet h_i, the rest meet agg_i.  Z keeps the
 * pre-activation (unrounded); with round_bf16 the output is stored as bf16. */
void oracle_sage_update(const double *Hself, const double *agg, int64_t n_dst, int32_t d_in,
                        const double *W, const double *bias, int32_t d_out, int act,
                        double *Z, double *Hout, int round_bf16)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n_dst; ++i)
        for (int32_t o = 0; o < d_out; ++o) {
            const double *w = W + (int64_t)o * 2 * d_in;
            double z = bias ? bias[o] : 0.0;
            for (int32_t k = 0; k < d_in; ++k) z += w[k] * Hself[i * d_in + k];
            for (int32_t k = 0; k < d_in; ++k) z += w[d_in + k] * agg[i * d_in + k];
            Z[i * d_out + o] = z;
            double h = (act && z < 0.0) ? 0.0 : z;
            Hout[i * d_out + o] = round_bf16 ? oracle_round_bf16(h) : h;
        }
}

/* ------------------------------------------------------------------------- */
/* Backward pass (Sec. 4.3.2, gradient of the total loss w.r.t. the GNN:      */
/* J^T applied to the gradient arriving at the GNN output; chain rule of      */
/* Sec. 4.2's cascaded-gradient expression)                                   */
/* ------------------------------------------------------------------------- */

/* Adjoint of the update.  dZ = dHout where the stored output is positive (ReLU)
 * or everywhere (identity); dW += dZ^T [Hself | agg]; db += column sums of dZ;
 * dSelf = dZ W[:, :d_in]; dAgg = dZ W[:, d_in:].  dW [d_out x 2 d_in] and db
 * [d_out] are accumulated into (caller zeroes them). */
void oracle_sage_update_backward(const double *dHout, const double *Hout, const double *Hself,
                                 const double *agg, const double *W, int64_t n_dst, int32_t d_in,
                                 int32_t d_out, int act, double *dW, double *db,
                                 double *dSelf, double *dAgg)
{
    /* dZ for all rows first; then every row of dSelf / dAgg and every row of dW / entry of db is the work of
     * one thread, which adds its terms in ascending order of o (dSelf, dAgg) or of i (dW, db) */
    double *dz = (double *)malloc(sizeof(double) * (size_t)(n_dst > 0 ? n_dst : 1) * (size_t)d_out);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n_dst; ++i) {
        for (int32_t o = 0; o < d_out; ++o)
            dz[i * d_out + o] = (act && !(Hout[i * d_out + o] > 0.0)) ? 0.0 : dHout[i * d_out + o];
        for (int32_t k = 0; k < d_in; ++k) { dSelf[i * d_in + k] = 0.0; dAgg[i * d_in + k] = 0.0; }
        for (int32_t o = 0; o < d_out; ++o) {
            const double *w = W + (int64_t)o * 2 * d_in;
            for (int32_t k = 0; k < d_in; ++k) {
                dSelf[i * d_in + k] += dz[i * d_out + o] * w[k];
                dAgg[i * d_in + k] += dz[i * d_out + o] * w[d_in + k];
            }
        }
    }
#pragma omp parallel for schedule(static)
    for (int32_t o = 0; o < d_out; ++o) {
        double *gw = dW + (int64_t)o * 2 * d_in;
        for (int64_t i = 0; i < n_dst; ++i) {
            const double g = dz[i * d_out + o];
            if (db) db[o] += g;
            for (int32_t k = 0; k < d_in; ++k) {
                gw[k] += g * Hself[i * d_in + k];
                gw[d_in + k] += g * agg[i * d_in + k];
            }
        }
    }
    free(dz);
}

/* Adjoint of the mean aggregation plus the self path:
 *   dH[s] = [s < n_dst] dSelf[s] + sum over entries e with col[e] = s of dAgg[row(e)] / |S(row(e))|.
 * With round_bf16, dSelf and dAgg/|S| are stored as bf16 before the sum and dH after it
 * (the points at which the GPU path writes them to memory). */
void oracle_mean_aggregate_backward(const int64_t *indptr, const int32_t *col, int64_t n_dst, int64_t n_src,
                                    const double *dSelf, const double *dAgg, int32_t d,
                                    double *dH, int round_bf16)
{
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < n_src; ++s)
        for (int32_t k = 0; k < d; ++k) {
            double v = (dSelf && s < n_dst) ? dSelf[s * d + k] : 0.0;
            dH[s * d + k] = round_bf16 ? oracle_round_bf16(v) : v;
        }
    /* rows of dH collide between destinations, feature columns do not: every thread owns a range of columns and
     * walks all entries in order, so an element receives its terms in the same order whatever the thread count */
#pragma omp parallel
    {
        int nt = 1, tid = 0;
#ifdef _OPENMP
        nt = omp_get_num_threads();
        tid = omp_get_thread_num();
#endif
        const int32_t k0 = (int32_t)((int64_t)d * tid / nt), k1 = (int32_t)((int64_t)d * (tid + 1) / nt);
        double *g = (double *)malloc(sizeof(double) * (size_t)(d > 0 ? d : 1));
        for (int64_t i = 0; i < n_dst && k0 < k1; ++i) {
            int64_t cnt = indptr[i + 1] - indptr[i];
            if (cnt == 0) continue;
            for (int32_t k = k0; k < k1; ++k) {
                double v = dAgg[i * d + k] / (double)cnt;
                g[k] = round_bf16 ? oracle_round_bf16(v) : v;
            }
            for (int64_t e = indptr[i]; e < indptr[i + 1]; ++e)
                for (int32_t k = k0; k < k1; ++k) dH[(int64_t)col[e] * d + k] += g[k];
        }
        free(g);
    }
    if (round_bf16) oracle_round_bf16_array(dH, n_src * d);
}

/* ------------------------------------------------------------------------- */
/* Ranking tower and loss (Theorem 1: z_i = [h_theta || b_i], scorer s_psi;   */
/* Sec. 5.1: binary cross-entropy on the towers)                              */
/* ------------------------------------------------------------------------- */

/* One dense layer y = act(W x + b) over n rows; W [d_out x d_in] row-major. */
void oracle_dense_forward(const double *Xin, int64_t n, int32_t d_in, const double *W, const double *b,
                          int32_t d_out, int act, double *Y, int round_bf16)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        for (int32_t o = 0; o < d_out; ++o) {
            double z = b ? b[o] : 0.0;
            for (int32_t k = 0; k < d_in; ++k) z += W[(int64_t)o * d_in + k] * Xin[i * d_in + k];
            if (act && z < 0.0) z = 0.0;
            Y[i * d_out + o] = round_bf16 ? oracle_round_bf16(z) : z;
        }
}

/* Adjoint of one dense layer; dW, db accumulated into. */
void oracle_dense_backward(const double *dY, const double *Y, const double *Xin, const double *W,
                           int64_t n, int32_t d_in, int32_t d_out, int act,
                           double *dW, double *db, double *dX, int round_bf16)
{
    /* as in oracle_sage_update_backward: rows of dX, then rows of dW, each summed by one thread in ascending order */
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        for (int32_t k = 0; k < d_in; ++k) dX[i * d_in + k] = 0.0;
        for (int32_t o = 0; o < d_out; ++o) {
            double dz = (act && !(Y[i * d_out + o] > 0.0)) ? 0.0 : dY[i * d_out + o];
            for (int32_t k = 0; k < d_in; ++k) dX[i * d_in + k] += dz * W[(int64_t)o * d_in + k];
        }
        if (round_bf16)
            for (int32_t k = 0; k < d_in; ++k) dX[i * d_in + k] = oracle_round_bf16(dX[i * d_in + k]);
    }
#pragma omp parallel for schedule(static)
    for (int32_t o = 0; o < d_out; ++o)
        for (int64_t i = 0; i < n; ++i) {
            double dz = (act && !(Y[i * d_out + o] > 0.0)) ? 0.0 : dY[i * d_out + o];
            db[o] += dz;
            for (int32_t k = 0; k < d_in; ++k) dW[(int64_t)o * d_in + k] += dz * Xin[i * d_in + k];
        }
}

/* Binary cross-entropy on logits t with labels y, mean over the n pairs:
 *   loss = (1/n) sum [ max(t,0) - y t + log(1 + exp(-|t|)) ],  dt = (sigmoid(t) - y) / n. */
double oracle_bce_with_logits(const double *t, const double *y, int64_t n, double *dt)
{
    double loss = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        double a = fabs(t[i]);
        loss += (t[i] > 0.0 ? t[i] : 0.0) - y[i] * t[i] + log1p(exp(-a));
        double sg = t[i] >= 0.0 ? 1.0 / (1.0 + exp(-t[i])) : exp(t[i]) / (1.0 + exp(t[i]));
        if (dt) dt[i] = (sg - y[i]) / (double)n;
    }
    return loss / (double)n;
}

/* ------------------------------------------------------------------------- */
/* Full-graph mean aggregation (Sec. 3.1 Eq. 2 with S(u) = N(u)) and adjoint  */
/* ------------------------------------------------------------------------- */

/* dX[s] = sum over rows i and entries e of row i with indices[e] = s of G[i] / deg(i).
 * deg(i) = |N(i)| is the length of row i, unless row_len is given: then the CSR holds only part of the
 * entries (those whose column is wanted) and row_len[i] is the size of the whole neighbourhood. */
void oracle_full_aggregate_backward(const int64_t *indptr, const int32_t *indices, int64_t n_dst, int64_t n_src,
                                    const double *G, int32_t d, double *dX, int round_bf16, const int64_t *row_len)
{
    for (int64_t s = 0; s < n_src * d; ++s) dX[s] = 0.0;
    for (int64_t i = 0; i < n_dst; ++i) {
        int64_t deg = row_len ? row_len[i] : indptr[i + 1] - indptr[i];
        for (int64_t e = indptr[i]; e < indptr[i + 1]; ++e)
            for (int32_t k = 0; k < d; ++k) dX[(int64_t)indices[e] * d + k] += G[i * d + k] / (double)deg;
    }
    if (round_bf16) oracle_round_bf16_array(dX, n_src * d);
}

/* ------------------------------------------------------------------------- */
/* LightGCN (Sec. 3.1, Eqs. 4-7)                                              */
/* ------------------------------------------------------------------------- */

/* One propagation: out_u = sum_{i in N(u)} h_i / (sqrt|N(u)| sqrt|N(i)|)  (Eqs. 4-5; H' = A_hat H, Eq. 6).
 * N(.) are the rows of the (square) CSR; a node without neighbours gives and receives 0.
 * With round_bf16 the result is stored as bf16. */
void oracle_lightgcn_propagate(const int64_t *indptr, const int32_t *indices, int64_t n, const double *H, int32_t d,
                               double *out, int round_bf16)
{
    for (int64_t u = 0; u < n; ++u) {
        const int64_t du = indptr[u + 1] - indptr[u];
        for (int32_t k = 0; k < d; ++k) {
            double s = 0.0;
            for (int64_t e = indptr[u]; e < indptr[u + 1]; ++e) {
                const int64_t i = indices[e];
                const int64_t di = indptr[i + 1] - indptr[i];
                if (di > 0) s += H[i * d + k] / (sqrt((double)du) * sqrt((double)di));
            }
            out[u * d + k] = round_bf16 ? oracle_round_bf16(s) : s;
        }
    }
}

/* LightGCN on sampled blocks.  One propagation over a block with destinations D and sources F:
 *   out_i = t_i * sum_{e in S(i)} s_{col e} * H[col e],   s_v = 1/sqrt|N(v)|,   t_i = sqrt|N(i)| / |S(i)|.
 * This is Eqs. 4-5 with the sum over N(i) estimated from the sampled multiset S(i): the factor |N(i)|/|S(i)|
 * makes the estimate of the sum unbiased, and with S(i) = N(i) (fanout >= degree) it is A_hat exactly.
 * s [n_src] and t [n_dst] are passed in.  With round_bf16 the result is stored as bf16. */
void oracle_lightgcn_block_forward(const int64_t *blk_indptr, const int32_t *col, int64_t n_dst, const double *H,
                                   const double *s, const double *t, int32_t d, double *out, int round_bf16)
{
    for (int64_t i = 0; i < n_dst; ++i)
        for (int32_t k = 0; k < d; ++k) {
            double sum = 0.0;
            for (int64_t e = blk_indptr[i]; e < blk_indptr[i + 1]; ++e) sum += s[col[e]] * H[(int64_t)col[e] * d + k];
            sum *= t[i];
            out[i * d + k] = round_bf16 ? oracle_round_bf16(sum) : sum;
        }
}

/* Its adjoint: dH_j = s_j * sum over entries (i, j) of t_i * G_i. */
void oracle_lightgcn_block_backward(const int64_t *blk_indptr, const int32_t *col, int64_t n_dst, int64_t n_src,
                                    const double *G, const double *s, const double *t, int32_t d, double *dH,
                                    int round_bf16)
{
    for (int64_t j = 0; j < n_src * d; ++j) dH[j] = 0.0;
    for (int64_t i = 0; i < n_dst; ++i)
        for (int64_t e = blk_indptr[i]; e < blk_indptr[i + 1]; ++e)
            for (int32_t k = 0; k < d; ++k) dH[(int64_t)col[e] * d + k] += t[i] * G[i * d + k];
    for (int64_t j = 0; j < n_src; ++j)
        for (int32_t k = 0; k < d; ++k) {
            double v = s[j] * dH[j * d + k];
            dH[j * d + k] = round_bf16 ? oracle_round_bf16(v) : v;
        }
}
