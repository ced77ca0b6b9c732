"""Pins for the oracle's joint GNN + tower step (CPU only, float64)."""
import numpy as np

import oracle


def _setup(seed=0):
    rng = np.random.default_rng(seed)
    n, m, d = 50, 400, 4
    row, col = rng.integers(0, n, m).astype(np.int32), rng.integers(0, n, m).astype(np.int32)
    indptr, indices = oracle.csr_from_coo(n, row, col)
    X = rng.standard_normal((n, d))
    W_gnn = [rng.standard_normal((5, 2 * d)) / 3, rng.standard_normal((3, 10)) / 3]
    P, dd = 9, 2
    user = rng.integers(0, 20, P).astype(np.int32)
    item = rng.integers(20, n, P).astype(np.int32)
    dense = rng.standard_normal((P, dd))
    labels = (rng.random(P) < 0.4).astype(np.float64)
    zdim = 2 * 3 + dd
    W_t = [rng.standard_normal((6, zdim)) / 2, rng.standard_normal((4, 6)) / 2, rng.standard_normal((1, 4))]
    b_t = [rng.standard_normal(6) / 3, rng.standard_normal(4) / 3, rng.standard_normal(1) / 3]
    return dict(indptr=indptr, indices=indices, X=X, pair_user=user, pair_item=item, dense=dense, labels=labels,
                fanouts=(3, 2), W_gnn=W_gnn, W_tower=W_t, b_tower=b_t, seed=4, step=2)


def _loss(a):
    return oracle.joint_step(**a)["loss"]


def test_joint_forward_is_the_plain_composition():
    a = _setup()
    r = oracle.joint_step(**a)
    seeds = np.unique(np.concatenate([a["pair_user"], a["pair_item"]]))
    assert np.array_equal(r["seeds"], seeds) and np.array_equal(r["blocks"][0]["src_nodes"][: seeds.size], seeds)
    pos = {int(s): i for i, s in enumerate(seeds)}
    H = r["H"]
    z = np.stack([np.concatenate([H[pos[int(u)]], H[pos[int(i)]], b]) for u, i, b in
                  zip(a["pair_user"], a["pair_item"], a["dense"])])
    a1 = np.maximum(z @ a["W_tower"][0].T + a["b_tower"][0], 0)
    a2 = np.maximum(a1 @ a["W_tower"][1].T + a["b_tower"][1], 0)
    t = (a2 @ a["W_tower"][2].T + a["b_tower"][2])[:, 0]
    assert np.allclose(r["logits"], t, rtol=1e-13, atol=1e-13)
    y = a["labels"]
    want = np.mean(np.where(y > 0, np.logaddexp(0, -t), np.logaddexp(0, t)))
    assert np.isclose(r["loss"], want, rtol=1e-13)


def test_joint_gradients_match_central_finite_differences():
    a = _setup(1)
    r = oracle.joint_step(**a)
    eps = 1e-6
    rng = np.random.default_rng(5)

    def fd(apply):
        ap, am = _copy(a), _copy(a)
        apply(ap, +eps)
        apply(am, -eps)
        return (_loss(ap) - _loss(am)) / (2 * eps)

    def _copy(x):
        y = dict(x)
        for k in ("W_gnn", "W_tower", "b_tower"):
            y[k] = [w.copy() for w in x[k]]
        y["X"] = x["X"].copy()
        return y

    for k in range(3):
        W = a["W_tower"][k]
        for _ in range(6):
            i, j = rng.integers(0, W.shape[0]), rng.integers(0, W.shape[1])
            g = fd(lambda q, e: q["W_tower"][k].__setitem__((i, j), q["W_tower"][k][i, j] + e))
            assert np.isclose(r["dW_tower"][k][i, j], g, rtol=2e-5, atol=1e-9)
        o = rng.integers(0, a["b_tower"][k].size)
        g = fd(lambda q, e: q["b_tower"][k].__setitem__(o, q["b_tower"][k][o] + e))
        assert np.isclose(r["db_tower"][k][o], g, rtol=2e-5, atol=1e-9)
    for l in range(2):
        W = a["W_gnn"][l]
        for _ in range(8):
            i, j = rng.integers(0, W.shape[0]), rng.integers(0, W.shape[1])
            g = fd(lambda q, e: q["W_gnn"][l].__setitem__((i, j), q["W_gnn"][l][i, j] + e))
            assert np.isclose(r["dW_gnn"][l][i, j], g, rtol=2e-5, atol=1e-9)
    ids = r["dX_ids"]
    for _ in range(12):
        rr, k = rng.integers(0, ids.size), rng.integers(0, a["X"].shape[1])
        g = fd(lambda q, e: q["X"].__setitem__((ids[rr], k), q["X"][ids[rr], k] + e))
        assert np.isclose(r["dX"][rr, k], g, rtol=2e-5, atol=1e-9)
    assert np.abs(r["dX"]).max() > 0 and all(np.abs(w).max() > 0 for w in r["dW_gnn"])


def test_ranking_loss_reaches_the_gnn_only_through_the_embedding_block():
    """Theorem 1 (i): the GNN gets a gradient from the ranking loss iff the scorer depends on h."""
    a = _setup(2)
    dL = a["W_gnn"][-1].shape[0]
    a["W_tower"][0][:, : 2 * dL] = 0.0           # scorer ignores the embeddings: cascaded-pipeline situation
    r = oracle.joint_step(**a)
    assert all(np.all(w == 0) for w in r["dW_gnn"]) and np.all(r["dX"] == 0)
    assert np.abs(r["dW_tower"][1]).max() > 0    # the tower itself still learns


def _gate_of(a, seed):
    rng = np.random.default_rng(seed)
    zdim = a["W_tower"][0].shape[1]
    return 0.6 * rng.standard_normal((zdim, zdim)), 0.3 * rng.standard_normal(zdim)


def test_gated_joint_step_is_the_plain_step_behind_the_gate():
    """Sec. 4.3.2, concatenation with gating: the tower sees sigmoid(W_g z + b_g) * z.  A gate held open by a large bias
    gives the ungated step; in general the forward pass is the composition written out with numpy."""
    a = _setup(3)
    plain = oracle.joint_step(**a)
    zdim = a["W_tower"][0].shape[1]
    open_gate = (np.zeros((zdim, zdim)), np.full(zdim, 60.0))
    r = oracle.joint_step(**a, gate=open_gate)
    assert np.allclose(r["logits"], plain["logits"], rtol=1e-12, atol=1e-12)
    assert np.allclose(r["dX"], plain["dX"], rtol=1e-9, atol=1e-12)
    Wg, bg = _gate_of(a, 3)
    r = oracle.joint_step(**a, gate=(Wg, bg))
    z = r["trace"]["z"]
    zf = z / (1.0 + np.exp(-(z @ Wg.T + bg)))
    a1 = np.maximum(zf @ a["W_tower"][0].T + a["b_tower"][0], 0)
    a2 = np.maximum(a1 @ a["W_tower"][1].T + a["b_tower"][1], 0)
    t = (a2 @ a["W_tower"][2].T + a["b_tower"][2])[:, 0]
    assert np.allclose(r["logits"], t, rtol=1e-12, atol=1e-12)
    assert not np.allclose(r["logits"], plain["logits"], rtol=1e-3)


def test_gated_joint_gradients_match_central_finite_differences():
    a = _setup(4)
    Wg, bg = _gate_of(a, 4)
    r = oracle.joint_step(**a, gate=(Wg, bg))
    eps = 1e-6
    rng = np.random.default_rng(6)
    loss = lambda args, W_, b_: oracle.joint_step(**args, gate=(W_, b_))["loss"]
    for _ in range(8):                                        # the gate's own parameters
        i, j = rng.integers(0, Wg.shape[0]), rng.integers(0, Wg.shape[1])
        Wp, Wm = Wg.copy(), Wg.copy()
        Wp[i, j] += eps; Wm[i, j] -= eps
        assert np.isclose(r["dW_gate"][i, j], (loss(a, Wp, bg) - loss(a, Wm, bg)) / (2 * eps), rtol=2e-5, atol=1e-9)
    for o in rng.integers(0, bg.size, 4):
        bp, bm = bg.copy(), bg.copy()
        bp[o] += eps; bm[o] -= eps
        assert np.isclose(r["db_gate"][o], (loss(a, Wg, bp) - loss(a, Wg, bm)) / (2 * eps), rtol=2e-5, atol=1e-9)

    def shifted(key, idx, e, l=None):
        b = dict(a)
        if l is None:
            b[key] = a[key].copy()
            b[key][idx] += e
        else:
            b[key] = [w.copy() for w in a[key]]
            b[key][l][idx] += e
        return b

    ids = r["dX_ids"]                                         # through the gate into the encoder and the features
    for _ in range(8):
        rr, k = rng.integers(0, ids.size), rng.integers(0, a["X"].shape[1])
        g = (loss(shifted("X", (ids[rr], k), eps), Wg, bg) - loss(shifted("X", (ids[rr], k), -eps), Wg, bg)) / (2 * eps)
        assert np.isclose(r["dX"][rr, k], g, rtol=2e-5, atol=1e-9)
    for l in range(2):
        W = a["W_gnn"][l]
        for _ in range(5):
            idx = (rng.integers(0, W.shape[0]), rng.integers(0, W.shape[1]))
            g = (loss(shifted("W_gnn", idx, eps, l), Wg, bg) - loss(shifted("W_gnn", idx, -eps, l), Wg, bg)) / (2 * eps)
            assert np.isclose(r["dW_gnn"][l][idx], g, rtol=2e-5, atol=1e-9)
    W = a["W_tower"][0]
    for _ in range(5):
        idx = (rng.integers(0, W.shape[0]), rng.integers(0, W.shape[1]))
        g = (loss(shifted("W_tower", idx, eps, 0), Wg, bg) - loss(shifted("W_tower", idx, -eps, 0), Wg, bg)) / (2 * eps)
        assert np.isclose(r["dW_tower"][0][idx], g, rtol=2e-5, atol=1e-9)


def test_joint_step_with_identity_activations_is_linear_up_to_the_loss():
    """acts 0 everywhere: the logits are a linear map of the features (checked by superposition), and the gradient
    with respect to the features follows from one matrix chain (checked through finite differences of the loss)."""
    a = _setup(5)
    lin = dict(acts_gnn=[0, 0], acts_tower=(0, 0))
    a0 = dict(a); a0["X"] = np.zeros_like(a["X"]); a0["dense"] = np.zeros_like(a["dense"])
    base = oracle.joint_step(**a0, **lin)["logits"]                      # the biases' share
    r1 = oracle.joint_step(**a, **lin)
    a2 = dict(a); a2["X"] = 3.0 * a["X"]; a2["dense"] = 3.0 * a["dense"]
    r3 = oracle.joint_step(**a2, **lin)
    assert np.allclose(r3["logits"] - base, 3.0 * (r1["logits"] - base), rtol=1e-10, atol=1e-10)
    eps = 1e-6
    ids = r1["dX_ids"]
    rng = np.random.default_rng(9)
    for _ in range(6):
        rr, k = rng.integers(0, ids.size), rng.integers(0, a["X"].shape[1])
        ap, am = dict(a), dict(a)
        ap["X"] = a["X"].copy(); am["X"] = a["X"].copy()
        ap["X"][ids[rr], k] += eps; am["X"][ids[rr], k] -= eps
        g = (oracle.joint_step(**ap, **lin)["loss"] - oracle.joint_step(**am, **lin)["loss"]) / (2 * eps)
        assert np.isclose(r1["dX"][rr, k], g, rtol=2e-5, atol=1e-9)
