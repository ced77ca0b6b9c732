"""Python face of the CPU oracle (test infrastructure, never a product path).

Loads ``liboracle.so`` (plain C, built from ``oracle.c`` with gcc) and strings
its per-step functions together in the order the paper gives them: sample a hop,
build the frontier, transpose the block; then per layer the mean aggregation
(Sec. 3.1, Eq. 2) and the update (Eq. 3); then the adjoints in reverse order.
All floating-point arrays are float64.  Nothing here imports the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "liboracle.so")
_SRC = os.path.join(_HERE, "oracle.c")


def build(force: bool = False) -> str:
    """Compile oracle.c into liboracle.so (gcc -O2, strict IEEE arithmetic)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-fopenmp",
                               "-o", _SO, _SRC, "-lm"])
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_round_bf16.restype = C.c_double
        _lib.oracle_round_bf16.argtypes = [C.c_double]
        _lib.oracle_sample_hop.restype = C.c_int64
        _lib.oracle_relabel.restype = C.c_int32
        _lib.oracle_csr_from_coo.restype = C.c_int
        _lib.oracle_bce_with_logits.restype = C.c_double
        _lib.oracle_max_threads.restype = C.c_int
    return _lib


def max_threads() -> int:
    """Threads the row loops of the C functions use (OpenMP's current maximum)."""
    return int(lib().oracle_max_threads())


def set_threads(n: int) -> None:
    """Sets that number (1 = the single-core program).  Results do not depend on it: every output element is
    still summed by one thread in the written order."""
    lib().oracle_set_threads(C.c_int(int(n)))


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


# ----------------------------------------------------------------------------- basics

def round_bf16(a):
    a = _f64(a).copy()
    lib().oracle_round_bf16_array(_p(a), C.c_int64(a.size))
    return a


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, np.uint32)
    lib().oracle_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def csr_from_coo(n, row, col):
    row, col = _i32(row), _i32(col)
    m = row.size
    indptr = np.zeros(n + 1, np.int64)
    indices = np.zeros(m, np.int32)
    rc = lib().oracle_csr_from_coo(C.c_int64(n), C.c_int64(m), _p(row), _p(col), _p(indptr), _p(indices))
    if rc != 0:
        raise ValueError("node id out of range")
    return indptr, indices


def csr_transpose(n_rows, n_cols, indptr, indices):
    indptr, indices = _i64(indptr), _i32(indices)
    m = int(indptr[n_rows])
    csc_ptr = np.zeros(n_cols + 1, np.int64)
    csc_row = np.zeros(m, np.int32)
    csc_eid = np.zeros(m, np.int64)
    lib().oracle_csr_transpose(C.c_int64(n_rows), C.c_int64(n_cols), _p(indptr), _p(indices),
                               _p(csc_ptr), _p(csc_row), _p(csc_eid))
    return csc_ptr, csc_row, csc_eid


# ----------------------------------------------------------------------------- sampling

def edge_cumulate(indptr, q):
    """Per-row running sums (uint64) of integer edge weights q (uint32), the table of the weighted sampler."""
    indptr = _i64(indptr)
    q = np.ascontiguousarray(q, dtype=np.uint32)
    cum = np.zeros(q.size, np.uint64)
    lib().oracle_edge_cumulate(C.c_int64(indptr.size - 1), _p(indptr), _p(q), _p(cum))
    return cum


def sample_khop(indptr, indices, seeds, fanouts, seed, step, edge_cum=None):
    """k-hop sampled blocks (Sec. 4.1 subgraph construction; Sec. 3.1 multiset S_l(u)).

    Hop h (1-based) samples for every node of D_h = F_{h-1} (F_0 = the seeds) with
    fanouts[h-1]; returns one dict per hop with the block CSR (indptr, col,
    nbr_global), the frontier src_nodes = F_h, the transposed block and 1/|S|.
    edge_cum (from edge_cumulate) switches the draws to the weighted form p ~ q of Sec. 4.1.
    """
    indptr, indices = _i64(indptr), _i32(indices)
    if edge_cum is not None:
        edge_cum = np.ascontiguousarray(edge_cum, dtype=np.uint64)
    n = indptr.size - 1
    dst = _i32(seeds)
    blocks = []
    for h, f in enumerate(fanouts, start=1):
        n_dst = dst.size
        cap = max(1, n_dst * int(f))
        blk_indptr = np.zeros(n_dst + 1, np.int32)
        nbr = np.zeros(cap, np.int32)
        ne = lib().oracle_sample_hop(_p(indptr), _p(indices), _p(edge_cum), _p(dst), C.c_int32(n_dst), C.c_int32(int(f)),
                                     C.c_uint64(int(seed)), C.c_uint32(int(step)), C.c_int32(h),
                                     _p(blk_indptr), _p(nbr))
        nbr = nbr[:ne].copy()
        src = np.zeros(n_dst + ne, np.int32)
        col = np.zeros(max(ne, 1), np.int32)
        n_src = lib().oracle_relabel(C.c_int64(n), _p(dst), C.c_int32(n_dst), _p(nbr), C.c_int64(ne),
                                     _p(src), _p(col))
        if n_src < 0:
            raise ValueError("seed id out of range")
        src = src[:n_src].copy()
        col = col[:ne].copy()
        csc_ptr = np.zeros(n_src + 1, np.int32)
        csc_row = np.zeros(max(ne, 1), np.int32)
        csc_eid = np.zeros(max(ne, 1), np.int32)
        inv_cnt = np.zeros(max(n_dst, 1), np.float32)
        lib().oracle_block_csc(C.c_int32(n_dst), C.c_int32(n_src), _p(blk_indptr), _p(col),
                               _p(csc_ptr), _p(csc_row), _p(csc_eid), _p(inv_cnt))
        blocks.append(dict(n_dst=n_dst, n_src=n_src, n_edges=int(ne), indptr=blk_indptr, col=col,
                           nbr_global=nbr, src_nodes=src, csc_ptr=csc_ptr, csc_row=csc_row[:ne].copy(),
                           csc_eid=csc_eid[:ne].copy(), csc_col=col[csc_eid[:ne]].copy(),
                           inv_cnt=inv_cnt[:n_dst].copy()))
        dst = src
    return blocks


# ----------------------------------------------------------------------------- GraphSAGE

def mean_aggregate(indptr, col, H, bf16=False):
    """Eq. 2 over a block (or a whole CSR): one mean row per destination."""
    indptr, col, H = _i64(indptr), _i32(col), _f64(H)
    n_dst, d = indptr.size - 1, H.shape[1]
    agg = np.zeros((n_dst, d), np.float64)
    lib().oracle_mean_aggregate(_p(indptr), _p(col), C.c_int64(n_dst), _p(H), C.c_int32(d), _p(agg),
                                C.c_int(int(bf16)))
    return agg


def sage_update(Hself, agg, W, bias, act, bf16=False):
    """Eq. 3: sigma(W [h || agg] (+ b)).  Returns (Z pre-activation, H)."""
    Hself, agg, W = _f64(Hself), _f64(agg), _f64(W)
    n_dst, d_in = Hself.shape
    d_out = W.shape[0]
    assert W.shape[1] == 2 * d_in
    b = None if bias is None else _f64(bias)
    Z = np.zeros((n_dst, d_out), np.float64)
    Hout = np.zeros((n_dst, d_out), np.float64)
    lib().oracle_sage_update(_p(Hself), _p(agg), C.c_int64(n_dst), C.c_int32(d_in), _p(W), _p(b),
                             C.c_int32(d_out), C.c_int(int(act)), _p(Z), _p(Hout), C.c_int(int(bf16)))
    return Z, Hout


def sage_forward(blocks, X, Ws, biases=None, acts=None, bf16=False, gathered=False):
    """L-layer forward on sampled blocks.  Layer l runs on block L-l; layer 0 reads X rows of F_L.

    With gathered=True, X already holds those rows (X[i] = features of node F_L[i]); for feature tables
    whose float64 copy would not fit the host."""
    L = len(Ws)
    acts = [1] * L if acts is None else list(acts)
    biases = [None] * L if biases is None else list(biases)
    X = _f64(X)
    ids = _i32(blocks[L - 1]["src_nodes"])
    if gathered:
        if X.shape[0] != ids.size:
            raise ValueError("gathered X must have one row per node of the outermost frontier")
        H = X.copy()
    else:
        H = np.zeros((ids.size, X.shape[1]), np.float64)
        lib().oracle_gather_rows(_p(X), C.c_int64(X.shape[1]), _p(ids), C.c_int64(ids.size),
                                 C.c_int32(X.shape[1]), _p(H))
    ctx = dict(H=[H], agg=[], Z=[])
    for l in range(L):
        blk = blocks[L - 1 - l]
        H = ctx["H"][l]
        agg = mean_aggregate(blk["indptr"], blk["col"], H, bf16)
        Z, Hn = sage_update(H[: blk["n_dst"]], agg, Ws[l], biases[l], acts[l], bf16)
        ctx["agg"].append(agg)
        ctx["Z"].append(Z)
        ctx["H"].append(Hn)
    return ctx["H"][L], ctx


def sage_backward(blocks, ctx, Ws, dH_out, acts=None, bf16=False, with_bias=False, trace=None):
    """Adjoint of sage_forward: returns (dWs, dbs, dX_rows) with dX_rows aligned to F_L.

    If `trace` is a list it receives, per layer l, the gradient that arrived at that layer's output."""
    L = len(Ws)
    acts = [1] * L if acts is None else list(acts)
    dH = _f64(dH_out)
    dWs, dbs = [None] * L, [None] * L
    for l in range(L - 1, -1, -1):
        blk = blocks[L - 1 - l]
        W = _f64(Ws[l])
        d_out, d_in = W.shape[0], W.shape[1] // 2
        n_dst, n_src = blk["n_dst"], blk["n_src"]
        Hl = _f64(ctx["H"][l])
        Hself = np.ascontiguousarray(Hl[:n_dst])
        agg, Hout = _f64(ctx["agg"][l]), _f64(ctx["H"][l + 1])
        dW = np.zeros_like(W)
        db = np.zeros(d_out, np.float64)
        dSelf = np.zeros((n_dst, d_in), np.float64)
        dAgg = np.zeros((n_dst, d_in), np.float64)
        dH = _f64(dH)
        if trace is not None:
            trace.insert(0, dH.copy())
        lib().oracle_sage_update_backward(_p(dH), _p(Hout), _p(Hself), _p(agg), _p(W), C.c_int64(n_dst),
                                          C.c_int32(d_in), C.c_int32(d_out), C.c_int(int(acts[l])),
                                          _p(dW), _p(db) if with_bias else None, _p(dSelf), _p(dAgg))
        dHl = np.zeros((n_src, d_in), np.float64)
        ip = _i64(blk["indptr"])
        cl = _i32(blk["col"])
        lib().oracle_mean_aggregate_backward(_p(ip), _p(cl), C.c_int64(n_dst), C.c_int64(n_src),
                                             _p(dSelf), _p(dAgg), C.c_int32(d_in), _p(dHl), C.c_int(int(bf16)))
        dWs[l], dbs[l] = dW, db
        dH = dHl
    return dWs, dbs, dH


# ----------------------------------------------------------------------------- tower + loss

def dense_forward(Xin, W, b, act, bf16=False):
    Xin, W = _f64(Xin), _f64(W)
    n, d_in = Xin.shape
    d_out = W.shape[0]
    bb = None if b is None else _f64(b)
    Y = np.zeros((n, d_out), np.float64)
    lib().oracle_dense_forward(_p(Xin), C.c_int64(n), C.c_int32(d_in), _p(W), _p(bb), C.c_int32(d_out),
                               C.c_int(int(act)), _p(Y), C.c_int(int(bf16)))
    return Y


def dense_backward(dY, Y, Xin, W, act, bf16=False):
    dY, Y, Xin, W = _f64(dY), _f64(Y), _f64(Xin), _f64(W)
    n, d_in = Xin.shape
    d_out = W.shape[0]
    dW = np.zeros_like(W)
    db = np.zeros(d_out, np.float64)
    dX = np.zeros((n, d_in), np.float64)
    lib().oracle_dense_backward(_p(dY), _p(Y), _p(Xin), _p(W), C.c_int64(n), C.c_int32(d_in), C.c_int32(d_out),
                                C.c_int(int(act)), _p(dW), _p(db), _p(dX), C.c_int(int(bf16)))
    return dW, db, dX


def bce_with_logits(t, y):
    t, y = _f64(t).ravel(), _f64(y).ravel()
    dt = np.zeros_like(t)
    loss = lib().oracle_bce_with_logits(_p(t), _p(y), C.c_int64(t.size), _p(dt))
    return float(loss), dt


# ----------------------------------------------------------------------------- full graph

def full_aggregate_backward(indptr, indices, n_src, G, bf16=False, row_len=None):
    """Adjoint of the whole-graph mean aggregation (Eq. 2 with S(u) = N(u)): dX = A^T D^-1 G.

    row_len: sizes |N(i)| of the whole neighbourhoods when the CSR passed holds only the entries of some
    columns (to check a few columns of a graph too large to run whole); default: the row lengths."""
    indptr, indices, G = _i64(indptr), _i32(indices), _f64(G)
    n_dst, d = indptr.size - 1, G.shape[1]
    dX = np.zeros((n_src, d), np.float64)
    rl = None if row_len is None else _i64(row_len)
    lib().oracle_full_aggregate_backward(_p(indptr), _p(indices), C.c_int64(n_dst), C.c_int64(n_src),
                                         _p(G), C.c_int32(d), _p(dX), C.c_int(int(bf16)), _p(rl))
    return dX


# ----------------------------------------------------------------------------- joint step

def joint_step(indptr, indices, X, pair_user, pair_item, dense, labels, fanouts, W_gnn, W_tower, b_tower,
               seed, step, bf16=False, acts_gnn=None, acts_tower=(1, 1), gate=None):
    """Joint GNN + ranking-tower step (Theorem 1: z = [h_theta || b]; BCE on the tower output, Sec. 5.1).

    seeds = ascending distinct endpoints of the pairs; z_p = [h(u_p) || h(i_p) || b_p]; three dense layers
    (ReLU, ReLU, none); loss = mean BCE-with-logits; then the adjoints back to the tower parameters, the GNN
    weights and the sampled feature rows.  Returns a dict of everything the GPU call returns.

    acts_gnn / acts_tower: 1 = ReLU (default), 0 = identity, per encoder layer / for the two hidden tower layers.
    gate = (W_g [zdim x zdim], b_g [zdim] or None): the concatenated features pass through the gating fusion of
    Sec. 4.3.2, z_fused = sigmoid(W_g z + b_g) * z, before the tower; the result then carries dW_gate, db_gate.
    The entry "trace" keeps the intermediate activations and gradients in the order they were formed.
    """
    pair_user, pair_item = _i32(pair_user), _i32(pair_item)
    seeds = np.unique(np.concatenate([pair_user, pair_item])).astype(np.int32)
    blocks = sample_khop(indptr, indices, seeds, fanouts, seed, step)
    H, ctx = sage_forward(blocks, X, W_gnn, acts=acts_gnn, bf16=bf16)
    pos_u, pos_i = np.searchsorted(seeds, pair_user), np.searchsorted(seeds, pair_item)
    dL = H.shape[1]
    dense = _f64(dense)
    if bf16:
        dense = round_bf16(dense)
    z = np.concatenate([H[pos_u], H[pos_i], dense], axis=1)
    b = [None, None, None] if b_tower is None else list(b_tower)
    zf, g = (z, None) if gate is None else gate_fusion_forward(z, gate[0], gate[1], bf16)
    a1 = dense_forward(zf, W_tower[0], b[0], acts_tower[0], bf16)
    a2 = dense_forward(a1, W_tower[1], b[1], acts_tower[1], bf16)
    t = dense_forward(a2, W_tower[2], b[2], 0, False)
    loss, dt = bce_with_logits(t[:, 0], labels)
    dW3, db3, da2 = dense_backward(dt[:, None], t, a2, W_tower[2], 0, bf16)
    dW2, db2, da1 = dense_backward(da2, a2, a1, W_tower[1], acts_tower[1], bf16)
    dW1, db1, dzf = dense_backward(da1, a1, zf, W_tower[0], acts_tower[0], bf16)
    out = {}
    if gate is None:
        dz = dzf
    else:
        dz, out["dW_gate"], out["db_gate"] = gate_fusion_backward(dzf, z, g, gate[0], bf16)
    dH = np.zeros_like(H)
    np.add.at(dH, pos_u, dz[:, :dL])
    np.add.at(dH, pos_i, dz[:, dL:2 * dL])
    if bf16:
        dH = round_bf16(dH)
    enc_trace = []
    dW_gnn, _, dX = sage_backward(blocks, ctx, W_gnn, dH, acts=acts_gnn, bf16=bf16, trace=enc_trace)
    out.update(seeds=seeds, blocks=blocks, loss=loss, logits=t[:, 0], dW_tower=[dW1, dW2, dW3],
               db_tower=[db1, db2, db3], dW_gnn=dW_gnn, dX=dX, dX_ids=blocks[-1]["src_nodes"], H=H, dH=dH,
               trace=dict(ctx=ctx, enc=enc_trace, pos_u=pos_u, pos_i=pos_i, z=z, gate=g, zf=zf, a1=a1, a2=a2, dt=dt,
                          da2=da2, da1=da1, dzf=dzf, dz=dz))
    return out


# ----------------------------------------------------------------------------- LightGCN

def lightgcn_propagate(indptr, indices, H, bf16=False):
    """Eqs. 4-6: one application of the symmetrically normalised adjacency (degrees = row lengths)."""
    indptr, indices, H = _i64(indptr), _i32(indices), _f64(H)
    n, d = indptr.size - 1, H.shape[1]
    out = np.zeros((n, d), np.float64)
    lib().oracle_lightgcn_propagate(_p(indptr), _p(indices), C.c_int64(n), _p(H), C.c_int32(d), _p(out),
                                    C.c_int(int(bf16)))
    return out


def lightgcn_forward(indptr, indices, H0, n_layers, bf16=False):
    """Eq. 7: Y = (1/(L+1)) sum_l H^(l), H^(l+1) = A_hat H^(l).  On a symmetric graph the adjoint w.r.t. H0 is
    the same map applied to dY."""
    H = _f64(H0)
    acc = H.copy()
    for _ in range(n_layers):
        H = lightgcn_propagate(indptr, indices, H, bf16)
        acc += H
    Y = acc / (n_layers + 1)
    return round_bf16(Y) if bf16 else Y


def _lightgcn_block_scales(blk, inv_sqrt_deg):
    """s_v = 1/sqrt|N(v)| for the sources, t_i = sqrt|N(i)| / |S(i)| = (1/|S(i)|) / s_i for the destinations
    (0 for a node without neighbours).  inv_sqrt_deg is the caller's float32 table over all nodes."""
    s = np.asarray(inv_sqrt_deg, np.float32)[blk["src_nodes"]].astype(np.float64)
    cnt = np.diff(blk["indptr"]).astype(np.float64)
    sd = s[: blk["n_dst"]]
    t = np.where((cnt > 0) & (sd > 0), (1.0 / np.maximum(cnt, 1)) / np.where(sd > 0, sd, 1.0), 0.0)
    return s, t


def lightgcn_sampled_forward(blocks, X, inv_sqrt_deg, bf16=False, gathered=False):
    """LightGCN (Eqs. 4-7) on sampled blocks: layer l runs on block L-l, H^0 = X rows of the outermost frontier, and
    Y = (1/(L+1)) sum_l H^l on the seed rows (the seeds open every frontier).  Returns (Y [n_seeds x d], ctx)."""
    L = len(blocks)
    X = _f64(X)
    ids = _i32(blocks[L - 1]["src_nodes"])
    H = X.copy() if gathered else X[ids]
    n_seeds = blocks[0]["n_dst"]
    acc = H[:n_seeds].copy()
    scales = []
    for l in range(L):
        blk = blocks[L - 1 - l]
        s, t = _lightgcn_block_scales(blk, inv_sqrt_deg)
        scales.append((s, t))
        out = np.zeros((blk["n_dst"], H.shape[1]), np.float64)
        lib().oracle_lightgcn_block_forward(_p(_i64(blk["indptr"])), _p(_i32(blk["col"])), C.c_int64(blk["n_dst"]),
                                            _p(np.ascontiguousarray(H)), _p(s), _p(t), C.c_int32(H.shape[1]), _p(out),
                                            C.c_int(int(bf16)))
        H = out
        acc += H[:n_seeds]
    Y = acc / (L + 1)
    return (round_bf16(Y) if bf16 else Y), dict(scales=scales)


def lightgcn_sampled_backward(blocks, ctx, dY, bf16=False):
    """Adjoint of lightgcn_sampled_forward with respect to the rows of the outermost frontier: dX_rows [n_src_L x d].
    Storage points with bf16: dY/(L+1); every propagated gradient; the seed rows after dY/(L+1) is added to them."""
    L = len(blocks)
    dYs = _f64(dY) / (L + 1)
    if bf16:
        dYs = round_bf16(dYs)
    n_seeds = blocks[0]["n_dst"]
    G = dYs.copy()
    for l in range(L - 1, -1, -1):
        blk = blocks[L - 1 - l]
        s, t = ctx["scales"][l]
        dH = np.zeros((blk["n_src"], G.shape[1]), np.float64)
        lib().oracle_lightgcn_block_backward(_p(_i64(blk["indptr"])), _p(_i32(blk["col"])), C.c_int64(blk["n_dst"]),
                                             C.c_int64(blk["n_src"]), _p(np.ascontiguousarray(G)), _p(s), _p(t),
                                             C.c_int32(G.shape[1]), _p(dH), C.c_int(int(bf16)))
        dH[:n_seeds] += dYs
        if bf16:
            dH[:n_seeds] = round_bf16(dH[:n_seeds])
        G = dH
    return G


# ----------------------------------------------------------------------------- SSL task (Sec. 4.2) and GradNorm (Sec. 4.3.1)

def ssl_loss(H, X_rows, weight=1.0, bf16=False):
    """Graph feature auto-encoder loss with the identity decoder (Sec. 4.2): L_ssl = ||X - H||_F^2 over the seed
    rows, and the gradient of weight * L_ssl with respect to H, 2 * weight * (H - X) (stored as bf16 with bf16)."""
    H, X_rows = _f64(H), _f64(X_rows)
    diff = H - X_rows
    dH = 2.0 * float(weight) * diff
    return float((diff * diff).sum()), (round_bf16(dH) if bf16 else dH)


def frobenius_norm(a):
    """||a||_2 over all elements: the norm of GradNorm's G_i for the gradient rows of the shared input h^(0)."""
    a = _f64(a)
    return float(np.sqrt((a * a).sum()))


def gradnorm_update(w, L, L0, g, gamma=1.0, lr=0.025, w_min=1e-6):
    """One GradNorm step for the task weights (Sec. 4.3.1, "Gradient-Based Task Weighting").

    w: current weights; L, L0: current and initial task losses; g: norms of the *unweighted* task gradients with
    respect to the shared input, so that G_i = w_i g_i.  With r_i = (L_i/L0_i) / mean_j(L_j/L0_j) and the targets
    c_i = mean(G) r_i^gamma held constant, L_gn = sum_i |G_i - c_i| has dL_gn/dw_i = sign(G_i - c_i) g_i; the
    weights take one gradient step of size lr, stay >= w_min and are rescaled to sum to the number of tasks.
    Returns (w_new, L_gn)."""
    w, L, L0, g = (_f64(np.atleast_1d(v)) for v in (w, L, L0, g))
    T = w.size
    G = w * g
    ratio = L / L0
    r = ratio / ratio.mean()
    c = G.mean() * r ** gamma
    L_gn = float(np.abs(G - c).sum())
    w_new = np.maximum(w - lr * np.sign(G - c) * g, w_min)
    return w_new * (T / w_new.sum()), L_gn


# ----------------------------------------------------------------------------- gated fusion (Sec. 4.3.2)

def gate_fusion_forward(F, Wg, bg, bf16=False):
    """Concatenation with gating: g = sigmoid(F Wg^T + bg), F_fused = g * F (element-wise), F = the concatenated
    feature groups [N x d].  Storage points with bf16: the pre-activation, the gate, the fused features.
    Returns (fused, gate)."""
    F, Wg = _f64(F), _f64(Wg)
    pre = F @ Wg.T + (0.0 if bg is None else _f64(bg))
    if bf16:
        pre = round_bf16(pre)
    g = np.where(pre >= 0, 1.0 / (1.0 + np.exp(-np.abs(pre))), np.exp(-np.abs(pre)) / (1.0 + np.exp(-np.abs(pre))))
    if bf16:
        g = round_bf16(g)
    fused = g * F
    return (round_bf16(fused) if bf16 else fused), g


def gate_fusion_backward(dFused, F, gate, Wg, bf16=False):
    """Adjoint of gate_fusion_forward: returns (dF, dWg, dbg).  d pre = dFused * F * g (1 - g);
    dF = dFused * g + d pre Wg; dWg = d pre^T F; dbg = column sums of d pre.  Storage points with bf16: d pre, the
    product d pre Wg, dF."""
    dFused, F, g, Wg = _f64(dFused), _f64(F), _f64(gate), _f64(Wg)
    dpre = dFused * F * g * (1.0 - g)
    if bf16:
        dpre = round_bf16(dpre)
    t = dpre @ Wg
    if bf16:
        t = round_bf16(t)
    dF = t + dFused * g
    return (round_bf16(dF) if bf16 else dF), dpre.T @ F, dpre.sum(0)
