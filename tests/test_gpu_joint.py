"""GPU parity of e2egrec_joint_step against the oracle's joint step."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as S
from helpers import assert_close, joint_rss_and_budgets

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


def _gate(w, dense_dim, seed):
    zdim = 2 * w.hidden + dense_dim
    Wg = S.glorot_uniform(zdim, zdim, seed, 43)
    bg = 0.1 * np.random.default_rng(seed + 1).standard_normal(zdim).astype(np.float32)
    return (S.to_bf16_values(Wg) if w.dtype == "bf16" else Wg), bg


def _run_gpu(w, indptr, indices, X, W_gnn, pu, pi, dense, labels, W_t, b_t, step, linear=False, gate=None):
    import paper_2511_20564_b200 as E
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    cu = lambda a, t=None: torch.from_numpy(np.ascontiguousarray(a)).cuda().to(t) if t else torch.from_numpy(np.ascontiguousarray(a)).cuda()
    js = E.JointStep(cu(indptr), cu(indices), cu(X, dt), pu.size, dense.shape[1], w.fanouts, [cu(W, dt) for W in W_gnn],
                     [cu(W, dt) for W in W_t], [cu(b) for b in b_t], linear=linear,
                     W_gate=None if gate is None else cu(gate[0], dt), b_gate=None if gate is None else cu(gate[1]))
    js.run(cu(pu), cu(pi), cu(dense), cu(labels), w.seed, step)
    torch.cuda.synchronize()
    return js


def _compare(w, args, step, linear=False, gate=None):
    """One joint step on both sides; every output compared element by element.  Gradients carry the tolerance of their
    last reduction (helpers.tolerance) and, with ReLU on, the budget of the sign decisions that the two sides took
    differently (helpers.joint_rss_and_budgets); with identity activations there is no budget at all."""
    bf16 = w.dtype == "bf16"
    indptr, indices, X, W_gnn, pu, pi, dense, labels, W_t, b_t = args
    acts = 0 if linear else 1
    L = len(W_gnn)
    ora = oracle.joint_step(indptr, indices, X, pu, pi, dense, labels, w.fanouts, W_gnn, W_t, b_t, w.seed, step, bf16=bf16,
                            acts_gnn=[acts] * L, acts_tower=(acts, acts), gate=gate)
    js = _run_gpu(w, *args, step, linear=linear, gate=gate)
    n_rows, status = js.n_rows.tolist()
    assert status == 0
    # integer side: the sampled sub-graph of the distinct endpoints
    assert n_rows == ora["dX_ids"].size and np.array_equal(js.dX_ids[:n_rows].cpu().numpy(), ora["dX_ids"])
    act = js.activations()
    gpu_act = dict(a1=act["a1"].float().cpu().numpy(), a2=act["a2"].float().cpu().numpy(),
                   enc=[h.float().cpu().numpy() for h in act["enc"]])
    rss, bud = joint_rss_and_budgets(ora, W_gnn, W_t, b_t, gpu_act, 2e-2 if bf16 else 1e-5, acts=acts, gate=gate)
    # forward
    # a logit is a 256-term sum over a2, whose elements the two sides store one bf16 step apart in a few percent of the
    # cases (fp32 against float64 sums before the rounding): up to 3.4e-2 of the logits were measured outside the plain
    # tolerance, none by more than 5x, all inside the tolerance scaled by the terms
    assert_close("logits", js.logits.cpu().numpy(), ora["logits"], bf16, rss["logits"], audit_share=6e-2 if bf16 else None)
    assert abs(float(js.loss) - ora["loss"]) <= (2e-2 * abs(ora["loss"]) + 1e-3 if bf16 else 1e-5 * abs(ora["loss"]))
    # gradients
    nt = 3
    for k in range(nt):
        assert_close(f"dW_tower[{k}]", js.dW_tower[k].cpu().numpy(), ora["dW_tower"][k], bf16, rss["dW_t"][k], bud["dW_t"][k])
        assert_close(f"db_tower[{k}]", js.db_tower[k].cpu().numpy(), ora["db_tower"][k], bf16, rss["db_t"][k], bud["db_t"][k])
    if gate is not None:
        assert_close("dW_gate", js.dW_tower[3].cpu().numpy(), ora["dW_gate"], bf16, rss["dW_gate"], bud["dW_gate"])
        assert_close("db_gate", js.db_tower[3].cpu().numpy(), ora["db_gate"], bf16, rss["db_gate"], bud["db_gate"])
    for l in range(L):
        assert_close(f"dW_gnn[{l}]", js.dW_gnn[l].cpu().numpy(), ora["dW_gnn"][l], bf16, rss["dW_g"][l], bud["dW_g"][l])
    dX = js.dX_rows[:n_rows].float().cpu().numpy()
    assert_close("dX", dX, ora["dX"], bf16, rss["dX"], bud["dX"])
    if linear:                                              # no sign decisions: no allowance for them
        assert all(float(np.max(b)) == 0.0 for b in bud["dW_t"] + bud["db_t"] + bud["dW_g"] + [bud["dX"]])
    # Theorem 1: the ranking loss reaches the encoder
    assert all(np.abs(g.cpu().numpy()).max() > 0 for g in js.dW_gnn) and np.abs(dX).max() > 0
    return ora, js


@pytest.mark.parametrize("name,n_pairs,dense_dim,h1,h2", [("tiny", 96, 8, 48, 24), ("medium_small", 512, 64, 512, 256)])
def test_joint_step_matches_oracle(name, n_pairs, dense_dim, h1, h2):
    w = S.WORKLOADS[name]
    _compare(w, _inputs(w, n_pairs, dense_dim, h1, h2, 7), step=3)


@pytest.mark.parametrize("name,n_pairs,dense_dim,h1,h2", [("tiny", 96, 8, 48, 24), ("medium_small", 512, 64, 512, 256)])
def test_joint_step_with_identity_activations_is_strict(name, n_pairs, dense_dim, h1, h2):
    """E2EGREC_JOINT_LINEAR: no ReLU anywhere, so no gradient element gets a sign-decision allowance; the bf16 case
    runs the same tensor-core products, segment reductions and pair -> seed sum as the default step."""
    w = S.WORKLOADS[name]
    _compare(w, _inputs(w, n_pairs, dense_dim, h1, h2, 8), step=1, linear=True)


@pytest.mark.parametrize("name,n_pairs,dense_dim,h1,h2,linear", [("tiny", 96, 8, 48, 24, False),
                                                                 ("medium_small", 512, 64, 512, 256, False),
                                                                 ("medium_small", 384, 64, 256, 128, True)])
def test_gated_joint_step_matches_oracle(name, n_pairs, dense_dim, h1, h2, linear):
    """E2EGREC_JOINT_GATE (Sec. 4.3.2): z_fused = sigmoid(W_g z + b_g) * z feeds the tower; the gate's own gradients and
    everything upstream of it are compared like the rest.  bf16: the gate runs in the epilogue of the W_g product."""
    w = S.WORKLOADS[name]
    _compare(w, _inputs(w, n_pairs, dense_dim, h1, h2, 9), step=2, linear=linear, gate=_gate(w, dense_dim, 9))


def test_joint_step_at_benchmark_size():
    """The joint step of the benchmark in full: 4 096 pairs on the 500 k-node / 20 M-entry graph, d = 128 bf16, fanout
    (15, 10), tower 320-512-256-1, Bernoulli(0.1) labels; every output against the oracle."""
    w = S.WORKLOADS["medium"]
    ora, js = _compare(w, _inputs(w, 4096, 64, 512, 256, 4), step=0)
    assert ora["blocks"][-1]["n_edges"] > 50_000 and ora["seeds"].size > 1_000


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
