"""GPU parity of e2egrec_joint_step against the oracle's joint step."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as S
from helpers import assert_blocks_equal, assert_close, tolerance

pytestmark = pytest.mark.gpu


def _inputs(w, n_pairs, dense_dim, h1, h2, seed):
    indptr, indices, (users, items) = S.build_graph(w)
    X, W_gnn = S.build_model(w)
    rng = np.random.default_rng(seed)
    pick = rng.integers(0, users.size, n_pairs)
    pu, pi = users[pick].astype(np.int32), items[pick].astype(np.int32)
    dense = rng.standard_normal((n_pairs, dense_dim)).astype(np.float32)
    labels = S.bernoulli_labels(n_pairs, 0.1, seed)
    zdim = 2 * w.hidden + dense_dim
    W_t = [S.glorot_uniform(h1, zdim, seed, 40), S.glorot_uniform(h2, h1, seed, 41), S.glorot_uniform(1, h2, seed, 42)]
    b_t = [0.1 * rng.standard_normal(h1).astype(np.float32), 0.1 * rng.standard_normal(h2).astype(np.float32),
           0.1 * rng.standard_normal(1).astype(np.float32)]
    if w.dtype == "bf16":
        W_t = [S.to_bf16_values(W) for W in W_t]
    return indptr, indices, X, W_gnn, pu, pi, dense, labels, W_t, b_t


def _run_gpu(w, indptr, indices, X, W_gnn, pu, pi, dense, labels, W_t, b_t, step):
    import paper_2511_20564_b200 as E
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    cu = lambda a, t=None: torch.from_numpy(np.ascontiguousarray(a)).cuda().to(t) if t else torch.from_numpy(np.ascontiguousarray(a)).cuda()
    js = E.JointStep(cu(indptr), cu(indices), cu(X, dt), pu.size, dense.shape[1], w.fanouts, [cu(W, dt) for W in W_gnn],
                     [cu(W, dt) for W in W_t], [cu(b) for b in b_t])
    js.run(cu(pu), cu(pi), cu(dense), cu(labels), w.seed, step)
    torch.cuda.synchronize()
    return js


@pytest.mark.parametrize("name,n_pairs,dense_dim,h1,h2", [("tiny", 96, 8, 48, 24), ("medium_small", 512, 64, 512, 256)])
def test_joint_step_matches_oracle(name, n_pairs, dense_dim, h1, h2):
    w = S.WORKLOADS[name]
    bf16 = w.dtype == "bf16"
    args = _inputs(w, n_pairs, dense_dim, h1, h2, 7)
    indptr, indices, X, W_gnn, pu, pi, dense, labels, W_t, b_t = args
    step = 3
    ora = oracle.joint_step(indptr, indices, X, pu, pi, dense, labels, w.fanouts, W_gnn, W_t, b_t, w.seed, step, bf16=bf16)
    js = _run_gpu(w, *args, step)
    n_rows, status = js.n_rows.tolist()
    assert status == 0
    # integer side: the sampled sub-graph of the distinct endpoints
    assert n_rows == ora["dX_ids"].size and np.array_equal(js.dX_ids[:n_rows].cpu().numpy(), ora["dX_ids"])
    # forward
    logits = js.logits.cpu().numpy().astype(np.float64)
    assert_close("logits", logits, ora["logits"], bf16, np.full(n_pairs, np.linalg.norm(W_t[2])) if bf16 else None)
    assert abs(float(js.loss) - ora["loss"]) <= (2e-2 * abs(ora["loss"]) + 1e-3 if bf16 else 1e-5 * abs(ora["loss"]))
    # gradients
    got = dict(dW_t=[g.cpu().numpy() for g in js.dW_tower], db_t=[g.cpu().numpy() for g in js.db_tower],
               dW_g=[g.cpu().numpy() for g in js.dW_gnn], dX=js.dX_rows[:n_rows].float().cpu().numpy())
    want = dict(dW_t=ora["dW_tower"], db_t=ora["db_tower"], dW_g=ora["dW_gnn"], dX=ora["dX"])
    for key in ("dW_t", "db_t", "dW_g"):
        for k, (g, o) in enumerate(zip(got[key], want[key])):
            _check_grad(f"{key}[{k}]", g, o, bf16)
    _check_grad("dX", got["dX"], want["dX"], bf16)
    # Theorem 1: the ranking loss reaches the encoder
    assert all(np.abs(g).max() > 0 for g in got["dW_g"]) and np.abs(got["dX"]).max() > 0


def _check_grad(name, got, want, bf16):
    """fp32: element-wise at 1e-5 (relative to the tensor's scale).  bf16: the masks of five ReLU layers are
    decided from fp32 sums on one side and float64 sums on the other, and where they differ both gradients
    are valid; the comparison is therefore norm-wise (3e-2) with 99% of the elements inside the element-wise
    tolerance.  The same kernels are held to the element-wise tolerance by the linear-activation and budgeted
    encoder tests."""
    got, want = np.asarray(got, np.float64).reshape(np.shape(want)), np.asarray(want, np.float64)
    assert np.isfinite(got).all(), name
    scale = np.sqrt(np.mean(want ** 2))
    if not bf16:
        bad = np.abs(got - want) > 2e-5 * np.maximum(np.abs(want), scale)
        assert not bad.any(), f"{name}: {bad.sum()} of {bad.size} outside 2e-5"
        return
    rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
    assert rel <= 3e-2, f"{name}: relative Frobenius error {rel:.3e}"
    tol = 1e-3 + 2e-2 * np.abs(want) + 2e-2 * scale
    frac = np.mean(np.abs(got - want) <= tol)
    assert frac >= 0.99, f"{name}: only {frac:.4f} of the elements within tolerance"


def test_joint_step_in_two_phases_equals_the_whole_step():
    """Sampling of a batch on one stream, the rest of its step on another (as a caller that prepares the next batch
    during the current one would issue them): bit-identical to the single call."""
    import paper_2511_20564_b200 as E
    w = S.WORKLOADS["medium_small"]
    args = _inputs(w, 512, 64, 512, 256, 11)
    indptr, indices, X, W_gnn, pu, pi, dense, labels, W_t, b_t = args
    whole = _run_gpu(w, *args, 5)
    dt = torch.bfloat16
    cu = lambda a, t=None: torch.from_numpy(np.ascontiguousarray(a)).cuda().to(t) if t else torch.from_numpy(np.ascontiguousarray(a)).cuda()
    js = E.JointStep(cu(indptr), cu(indices), cu(X, dt), pu.size, dense.shape[1], w.fanouts, [cu(W, dt) for W in W_gnn],
                     [cu(W, dt) for W in W_t], [cu(b) for b in b_t])
    pu_d, pi_d, dense_d, labels_d = cu(pu), cu(pi), cu(dense), cu(labels)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(s2):
        js.run(pu_d, pi_d, dense_d, labels_d, w.seed, 5, phase=1)
    s1.wait_stream(s2)
    with torch.cuda.stream(s1):
        js.run(pu_d, pi_d, dense_d, labels_d, w.seed, 5, phase=2)
    torch.cuda.synchronize()
    assert js.n_rows.tolist() == whole.n_rows.tolist() and js.n_rows.tolist()[1] == 0
    n_rows = js.n_rows.tolist()[0]
    assert torch.equal(js.loss, whole.loss) and torch.equal(js.logits, whole.logits)
    assert torch.equal(js.dX_ids[:n_rows], whole.dX_ids[:n_rows]) and torch.equal(js.dX_rows[:n_rows], whole.dX_rows[:n_rows])
    for a, b in zip(js.dW_gnn + js.dW_tower + js.db_tower, whole.dW_gnn + whole.dW_tower + whole.db_tower):
        assert torch.equal(a, b)
