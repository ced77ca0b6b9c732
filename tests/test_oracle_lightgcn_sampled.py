"""Pins for the oracle's LightGCN on sampled blocks (Eqs. 4-7 on the sampled sub-graph)."""
import numpy as np

import oracle
import synth_inputs as S


def _graph(seed=3, n=60, m=500):
    a, b = S.powerlaw_directed(n, m, 1.1, seed)
    return S.coo_to_csr(n, np.concatenate([a, b]), np.concatenate([b, a]))       # symmetric, parallel edges kept


def _inv_sqrt_deg(indptr):
    deg = np.diff(indptr)
    return np.where(deg > 0, 1.0 / np.sqrt(np.maximum(deg, 1)), 0.0).astype(np.float32)


def test_full_fanout_equals_the_whole_graph_propagation():
    """With fanout >= every degree S(u) = N(u), so the sampled L-layer result on the seeds is the whole-graph
    LightGCN (itself pinned against the dense normalised adjacency) on those rows."""
    indptr, indices = _graph()
    n = indptr.size - 1
    rng = np.random.default_rng(0)
    X = rng.standard_normal((n, 5))
    s = _inv_sqrt_deg(indptr)
    seeds = rng.permutation(n)[:17].astype(np.int32)
    big = int(np.diff(indptr).max())
    for L in (1, 2, 3):
        blocks = oracle.sample_khop(indptr, indices, seeds, (big,) * L, seed=5, step=0)
        Y, _ = oracle.lightgcn_sampled_forward(blocks, X, s)
        want = oracle.lightgcn_forward(indptr, indices, X, L)[seeds]
        assert np.allclose(Y, want, rtol=1e-6, atol=1e-7)        # s is a float32 table: 6e-8 relative per factor


def test_sampled_propagation_is_the_stated_estimator():
    """One block, by hand: out_i = (sqrt|N(i)| / |S(i)|) sum_{v in S(i)} h_v / sqrt|N(v)|."""
    indptr, indices = _graph(seed=4)
    n = indptr.size - 1
    deg = np.diff(indptr)
    rng = np.random.default_rng(1)
    X = rng.standard_normal((n, 3))
    s = _inv_sqrt_deg(indptr)
    seeds = np.flatnonzero(deg > 4)[:6].astype(np.int32)
    blk = oracle.sample_khop(indptr, indices, seeds, (3,), seed=9, step=2)[0]
    Y, _ = oracle.lightgcn_sampled_forward([blk], X, s)
    for i, u in enumerate(seeds):
        picked = blk["nbr_global"][blk["indptr"][i]: blk["indptr"][i + 1]]
        assert picked.size == 3
        prop = np.sqrt(deg[u]) / 3.0 * sum(X[v] * float(s[v]) for v in picked)
        assert np.allclose(Y[i], (X[u] + prop) / 2.0, rtol=1e-6, atol=1e-9)


def test_backward_is_the_adjoint_of_forward():
    indptr, indices = _graph(seed=6, n=80, m=900)
    n = indptr.size - 1
    rng = np.random.default_rng(2)
    X = rng.standard_normal((n, 4))
    s = _inv_sqrt_deg(indptr)
    seeds = rng.permutation(n)[:20].astype(np.int32)
    blocks = oracle.sample_khop(indptr, indices, seeds, (4, 3), seed=1, step=7)
    Y, ctx = oracle.lightgcn_sampled_forward(blocks, X, s)
    dY = rng.standard_normal(Y.shape)
    dX = oracle.lightgcn_sampled_backward(blocks, ctx, dY)
    rows = blocks[-1]["src_nodes"]
    assert np.isclose((Y * dY).sum(), (X[rows] * dX).sum(), rtol=1e-12)
    # and by central differences on a few entries (the map is linear, so the difference quotient is exact)
    for (r, k) in [(0, 0), (5, 2), (rows.size - 1, 3)]:
        Xp = X.copy()
        Xp[rows[r], k] += 1.0
        Yp, _ = oracle.lightgcn_sampled_forward(blocks, Xp, s)
        assert np.isclose(((Yp - Y) * dY).sum(), dX[r, k], rtol=1e-10, atol=1e-12)


def test_isolated_seed_and_bf16_storage():
    indptr, indices = _graph(seed=8, n=200, m=500)
    n = indptr.size - 1
    deg = np.diff(indptr)
    iso = np.flatnonzero(deg == 0)
    assert iso.size > 0
    X = oracle.round_bf16(np.random.default_rng(3).standard_normal((n, 4)))
    s = _inv_sqrt_deg(indptr)
    seeds = np.concatenate([iso[:1], np.flatnonzero(deg > 0)[:5]]).astype(np.int32)
    blocks = oracle.sample_khop(indptr, indices, seeds, (3, 2), seed=2, step=0)
    Y, ctx = oracle.lightgcn_sampled_forward(blocks, X, s)
    assert np.allclose(Y[0], X[iso[0]] / 3.0)                   # an isolated seed only keeps its own layer-0 row
    Yb, _ = oracle.lightgcn_sampled_forward(blocks, X, s, bf16=True)
    assert np.array_equal(Yb, oracle.round_bf16(Yb)) and np.allclose(Yb, Y, rtol=3e-2, atol=3e-2)
    dXb = oracle.lightgcn_sampled_backward(blocks, ctx, np.ones_like(Y), bf16=True)
    assert np.array_equal(dXb, oracle.round_bf16(dXb))
