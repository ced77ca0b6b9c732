"""Pins for the oracle's GraphSAGE forward/backward, tower and loss (CPU only, float64)."""
import numpy as np
import scipy.sparse as sp

import oracle


def _graph(rng, n, m):
    row = rng.integers(0, n, m).astype(np.int32)
    col = rng.integers(0, n, m).astype(np.int32)
    return oracle.csr_from_coo(n, row, col)


def _dense_block(blk):
    A = np.zeros((blk["n_dst"], blk["n_src"]))
    for i in range(blk["n_dst"]):
        for e in range(blk["indptr"][i], blk["indptr"][i + 1]):
            A[i, blk["col"][e]] += 1.0
    return A


def _setup(seed=0, n=60, m=500, d=6, hidden=(5, 4), fan=(4, 3), n_seeds=12):
    rng = np.random.default_rng(seed)
    indptr, indices = _graph(rng, n, m)
    seeds = rng.choice(n, n_seeds, replace=False).astype(np.int32)
    blocks = oracle.sample_khop(indptr, indices, seeds, fan, seed=3, step=1)
    X = rng.standard_normal((n, d))
    Ws, d_in = [], d
    for h in hidden:
        Ws.append(rng.standard_normal((h, 2 * d_in)) / np.sqrt(2 * d_in))
        d_in = h
    return rng, indptr, indices, seeds, blocks, X, Ws


def test_mean_aggregate_equals_dense_normalised_product():
    rng, _, _, _, blocks, X, _ = _setup()
    blk = blocks[1]
    H = rng.standard_normal((blk["n_src"], 7))
    A = _dense_block(blk)
    cnt = A.sum(1, keepdims=True)
    want = np.where(cnt > 0, A @ H / np.maximum(cnt, 1), 0.0)       # D_S^-1 A_S H
    got = oracle.mean_aggregate(blk["indptr"], blk["col"], H)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-13)
    # library sparse product
    S = sp.csr_matrix((np.ones(blk["n_edges"]), blk["col"], blk["indptr"]), shape=(blk["n_dst"], blk["n_src"]))
    assert np.allclose(got * np.maximum(cnt, 1), S @ H, rtol=1e-13, atol=1e-13)


def test_mean_of_constant_is_constant_and_empty_rows_are_zero():
    indptr = np.array([0, 3, 3, 5], np.int64)
    col = np.array([0, 1, 1, 2, 0], np.int32)
    H = np.full((3, 4), 2.5)
    got = oracle.mean_aggregate(indptr, col, H)
    assert np.array_equal(got[0], np.full(4, 2.5)) and np.array_equal(got[2], np.full(4, 2.5))
    assert np.array_equal(got[1], np.zeros(4))


def test_update_equals_numpy_restatement():
    rng = np.random.default_rng(1)
    h, a = rng.standard_normal((9, 5)), rng.standard_normal((9, 5))
    W, b = rng.standard_normal((4, 10)), rng.standard_normal(4)
    Z, H = oracle.sage_update(h, a, W, b, act=1)
    want = np.concatenate([h, a], 1) @ W.T + b
    assert np.allclose(Z, want, rtol=1e-13, atol=1e-13)
    assert np.array_equal(H, np.maximum(Z, 0.0))
    Z2, H2 = oracle.sage_update(h, a, W, None, act=0)
    assert np.allclose(H2, want - b, rtol=1e-13, atol=1e-13) and np.array_equal(Z2, H2)
    # the first d_in columns of W meet the self row, the rest the neighbourhood mean
    W0 = W.copy(); W0[:, 5:] = 0
    assert np.allclose(oracle.sage_update(h, a, W0, None, 0)[0], h @ W[:, :5].T)


def test_full_fanout_equals_dense_full_neighbourhood_gnn():
    """With every fanout >= max degree the sampled GNN on the seeds is the exact 2-layer GNN."""
    rng, indptr, indices, seeds, _, X, Ws = _setup(seed=5, n=40, m=160)
    maxdeg = int(np.diff(indptr).max())
    blocks = oracle.sample_khop(indptr, indices, seeds, (maxdeg, maxdeg), seed=0, step=0)
    out, _ = oracle.sage_forward(blocks, X, Ws)
    n = indptr.size - 1
    A = np.zeros((n, n))
    for u in range(n):
        for e in range(indptr[u], indptr[u + 1]):
            A[u, indices[e]] += 1
    deg = A.sum(1, keepdims=True)
    P = np.where(deg > 0, A / np.maximum(deg, 1), 0.0)
    H = X
    for W in Ws:
        H = np.maximum(np.concatenate([H, P @ H], 1) @ W.T, 0.0)
    assert np.allclose(out, H[seeds], rtol=1e-12, atol=1e-12)


def test_aggregation_adjoint_identity():
    rng, _, _, _, blocks, _, _ = _setup(seed=6)
    blk = blocks[1]
    d = 5
    Xs = rng.standard_normal((blk["n_src"], d))
    G = rng.standard_normal((blk["n_dst"], d))
    AX = oracle.mean_aggregate(blk["indptr"], blk["col"], Xs)
    dH = np.zeros((blk["n_src"], d))
    ip = blk["indptr"].astype(np.int64)
    oracle.lib().oracle_mean_aggregate_backward(oracle._p(ip), oracle._p(blk["col"]),
                                                oracle.C.c_int64(blk["n_dst"]), oracle.C.c_int64(blk["n_src"]),
                                                None, oracle._p(G), oracle.C.c_int32(d), oracle._p(dH),
                                                oracle.C.c_int(0))
    assert np.isclose((AX * G).sum(), (Xs * dH).sum(), rtol=1e-12)       # <A X, G> = <X, A^T G>
    # and it is the dense transpose
    A = _dense_block(blk)
    cnt = A.sum(1, keepdims=True)
    P = np.where(cnt > 0, A / np.maximum(cnt, 1), 0.0)
    assert np.allclose(dH, P.T @ G, rtol=1e-12, atol=1e-12)


def _loss(blocks, X, Ws, R, bs=None, acts=None):
    out, ctx = oracle.sage_forward(blocks, X, Ws, bs, acts)
    return float((out * R).sum()), ctx


def test_backward_matches_central_finite_differences():
    rng, _, _, _, blocks, X, Ws = _setup(seed=7)
    R = rng.standard_normal((blocks[0]["n_dst"], Ws[-1].shape[0]))
    _, ctx = _loss(blocks, X, Ws, R)
    # stay off the ReLU kinks
    assert min(np.abs(z).min() for z in ctx["Z"]) > 1e-5
    dWs, _, dXr = oracle.sage_backward(blocks, ctx, Ws, R)
    eps = 1e-6
    for l, W in enumerate(Ws):
        for _ in range(12):
            i, j = rng.integers(0, W.shape[0]), rng.integers(0, W.shape[1])
            Wp = [w.copy() for w in Ws]; Wm = [w.copy() for w in Ws]
            Wp[l][i, j] += eps; Wm[l][i, j] -= eps
            fd = (_loss(blocks, X, Wp, R)[0] - _loss(blocks, X, Wm, R)[0]) / (2 * eps)
            assert np.isclose(dWs[l][i, j], fd, rtol=1e-6, atol=1e-8)
    ids = blocks[-1]["src_nodes"]
    for _ in range(20):
        r, k = rng.integers(0, ids.size), rng.integers(0, X.shape[1])
        Xp, Xm = X.copy(), X.copy()
        Xp[ids[r], k] += eps; Xm[ids[r], k] -= eps
        fd = (_loss(blocks, Xp, Ws, R)[0] - _loss(blocks, Xm, Ws, R)[0]) / (2 * eps)
        assert np.isclose(dXr[r, k], fd, rtol=1e-6, atol=1e-8)
    # rows of X outside the sampled frontier get no gradient: dX_rows covers exactly F_L
    assert dXr.shape == (ids.size, X.shape[1])


def test_backward_bias_and_identity_activation():
    rng, _, _, _, blocks, X, Ws = _setup(seed=8)
    bs = [rng.standard_normal(W.shape[0]) for W in Ws]
    acts = [1, 0]
    R = rng.standard_normal((blocks[0]["n_dst"], Ws[-1].shape[0]))
    _, ctx = _loss(blocks, X, Ws, R, bs, acts)
    _, dbs, _ = oracle.sage_backward(blocks, ctx, Ws, R, acts, with_bias=True)
    eps = 1e-6
    for l in range(2):
        for o in range(bs[l].size):
            bp = [b.copy() for b in bs]; bm = [b.copy() for b in bs]
            bp[l][o] += eps; bm[l][o] -= eps
            fd = (_loss(blocks, X, Ws, R, bp, acts)[0] - _loss(blocks, X, Ws, R, bm, acts)[0]) / (2 * eps)
            assert np.isclose(dbs[l][o], fd, rtol=1e-6, atol=1e-8)


def test_bf16_contract_only_rounds_at_storage_points():
    rng, _, _, _, blocks, X, Ws = _setup(seed=9)
    Xb = oracle.round_bf16(X)
    Wb = [oracle.round_bf16(W) for W in Ws]
    out_b, ctx_b = oracle.sage_forward(blocks, Xb, Wb, bf16=True)
    out_d, _ = oracle.sage_forward(blocks, Xb, Wb, bf16=False)
    for a in ctx_b["agg"] + ctx_b["H"]:
        assert np.array_equal(a, oracle.round_bf16(a))            # stored tensors are bf16 values
    assert np.allclose(out_b, out_d, rtol=3e-2, atol=3e-2) and not np.array_equal(out_b, out_d)
    # first layer: rounding the double result of the unrounded path gives the stored value
    agg0 = oracle.mean_aggregate(blocks[1]["indptr"], blocks[1]["col"], ctx_b["H"][0])
    assert np.array_equal(ctx_b["agg"][0], oracle.round_bf16(agg0))


def test_full_graph_backward_is_transpose_of_forward():
    rng = np.random.default_rng(10)
    n = 50
    indptr, indices = _graph(rng, n, 400)
    d = 4
    X, G = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    AX = oracle.mean_aggregate(indptr, indices, X)
    dX = oracle.full_aggregate_backward(indptr, indices, n, G)
    assert np.isclose((AX * G).sum(), (X * dX).sum(), rtol=1e-12)
    A = np.zeros((n, n))
    for u in range(n):
        for e in range(indptr[u], indptr[u + 1]):
            A[u, indices[e]] += 1
    deg = A.sum(1, keepdims=True)
    P = np.where(deg > 0, A / np.maximum(deg, 1), 0.0)
    assert np.allclose(AX, P @ X, atol=1e-12) and np.allclose(dX, P.T @ G, atol=1e-12)
    # a few columns only: the CSR keeps just their entries (renumbered), the neighbourhood sizes are passed
    cols = np.array([3, 17, 41])
    keep = np.isin(indices, cols)
    rows = np.repeat(np.arange(n), np.diff(indptr))[keep]
    sub_ptr = np.zeros(n + 1, np.int64)
    np.cumsum(np.bincount(rows, minlength=n), out=sub_ptr[1:])
    sub_idx = np.searchsorted(cols, indices[keep]).astype(np.int32)
    part = oracle.full_aggregate_backward(sub_ptr, sub_idx, cols.size, G, row_len=np.diff(indptr))
    assert np.allclose(part, (P.T @ G)[cols], atol=1e-12)


# ----------------------------------------------------------------------------- tower + loss

def test_bce_closed_forms():
    n = 8
    y = np.array([0, 1, 0, 0, 1, 0, 0, 0], np.float64)
    loss, dt = oracle.bce_with_logits(np.zeros(n), y)
    assert np.isclose(loss, np.log(2.0), rtol=1e-15)
    assert np.allclose(dt, (0.5 - y) / n)
    t = np.array([-30.0, 30.0, 2.0, -0.5, 0.3, 700.0, -700.0, 1e-9])
    loss, dt = oracle.bce_with_logits(t, y)
    p = 1.0 / (1.0 + np.exp(-np.clip(t, -700, 700)))
    with np.errstate(divide="ignore"):
        want = np.where(y > 0, np.logaddexp(0, -t), np.logaddexp(0, t)).mean()   # -log p / -log(1-p)
    assert np.isclose(loss, want, rtol=1e-13)
    assert np.allclose(dt, (p - y) / n, rtol=1e-12, atol=1e-300)


def test_dense_layer_forward_backward():
    rng = np.random.default_rng(11)
    X, W, b = rng.standard_normal((7, 5)), rng.standard_normal((3, 5)), rng.standard_normal(3)
    Y = oracle.dense_forward(X, W, b, act=1)
    assert np.allclose(Y, np.maximum(X @ W.T + b, 0))
    R = rng.standard_normal(Y.shape)
    dW, db, dX = oracle.dense_backward(R, Y, X, W, act=1)
    dZ = R * (Y > 0)
    assert np.allclose(dW, dZ.T @ X) and np.allclose(db, dZ.sum(0)) and np.allclose(dX, dZ @ W)


# ----------------------------------------------------------------------------- LightGCN

def test_lightgcn_matches_dense_normalised_adjacency_and_is_self_adjoint():
    rng = np.random.default_rng(12)
    n, d, L = 40, 3, 3
    row = rng.integers(0, n - 2, 150).astype(np.int32)         # the last two nodes stay isolated
    col = rng.integers(0, n - 2, 150).astype(np.int32)
    indptr, indices = oracle.csr_from_coo(n, np.concatenate([row, col]), np.concatenate([col, row]))   # symmetric
    A = np.zeros((n, n))
    for u in range(n):
        for e in range(indptr[u], indptr[u + 1]):
            A[u, indices[e]] += 1
    deg = np.diff(indptr).astype(np.float64)
    s = np.where(deg > 0, 1 / np.sqrt(np.maximum(deg, 1)), 0.0)
    Ahat = s[:, None] * A * s[None, :]                             # D^-1/2 A D^-1/2
    H0, G = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    assert np.allclose(oracle.lightgcn_propagate(indptr, indices, H0), Ahat @ H0, atol=1e-13)
    want = sum(np.linalg.matrix_power(Ahat, l) @ H0 for l in range(L + 1)) / (L + 1)
    Y = oracle.lightgcn_forward(indptr, indices, H0, L)
    assert np.allclose(Y, want, atol=1e-13)
    assert np.all(Y[-2:] == H0[-2:] / (L + 1))                     # isolated nodes keep only their own layer-0 term
    # symmetric graph: <Y(H0), G> = <H0, Y(G)>
    assert np.isclose((Y * G).sum(), (H0 * oracle.lightgcn_forward(indptr, indices, G, L)).sum(), rtol=1e-12)
