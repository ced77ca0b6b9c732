"""GPU parity of the SSL loss, the gradient norms and the GradNorm weight step (Sec. 4.2, Sec. 4.3.1), and of the two-pass backward
that a step with two tasks runs."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as S
from helpers import Case, assert_close, reduction_rss

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,rows,d", [("f32", 300, 64), ("bf16", 4099, 128), ("bf16", 8192, 256)])
def test_ssl_loss_and_gradient_norm(dtype, rows, d):
    import paper_2511_20564_b200 as E
    bf16 = dtype == "bf16"
    dt = torch.bfloat16 if bf16 else torch.float32
    rng = np.random.default_rng(rows)
    n = 20_000
    X = rng.standard_normal((n, d)).astype(np.float32)
    H = rng.standard_normal((rows + 5, d)).astype(np.float32)        # 5 rows beyond the count: must be ignored
    if bf16:
        X, H = S.to_bf16_values(X), S.to_bf16_values(H)
    ids = rng.permutation(n)[: rows + 5].astype(np.int32)
    w = 0.37
    dev = torch.device("cuda")
    n_dev = torch.tensor([rows], dtype=torch.int32, device=dev)
    loss, dH = E.ssl_loss(torch.from_numpy(H).to(dev, dt), torch.from_numpy(X).to(dev, dt), torch.from_numpy(ids).to(dev),
                          n_dev, torch.tensor([w], dtype=torch.float32, device=dev))
    want_loss, want_dH = oracle.ssl_loss(H[:rows], X[ids[:rows]], w, bf16)
    assert abs(float(loss) - want_loss) <= 1e-5 * want_loss
    assert_close("dH_ssl", dH[:rows].float().cpu().numpy(), want_dH, bf16)
    assert not dH[rows:].any()
    norm = E.gradient_norm(dH, n_dev)
    want_norm = oracle.frobenius_norm(dH[:rows].float().cpu().numpy())
    assert abs(float(norm) - want_norm) <= 1e-5 * want_norm
    again = E.gradient_norm(dH, n_dev)
    assert torch.equal(norm, again)                                 # fixed summation order


@pytest.mark.parametrize("case", [([1.0, 1.0], [2.0, 4.0], [4.0, 8.0], [3.0, 3.0], 1.0, 0.025),
                                  ([1.0, 1.0], [1.0, 1.0], [1.0, 1.0], [10.0, 1.0], 1.0, 0.01),
                                  ([0.8, 1.2], [0.5, 0.9], [1.0, 1.0], [4.0, 1.5], 1.0, 1e-3),
                                  ([0.8, 1.2], [0.5, 0.9], [1.0, 2.0], [4.0, 1.5], 0.5, 0.05),
                                  ([0.01, 1.99], [1.0, 1.0], [1.0, 1.0], [1000.0, 0.001], 1.0, 1.0)])
def test_gradnorm_update(case):
    import paper_2511_20564_b200 as E
    w, L, L0, g, gamma, lr = case
    f = lambda v: torch.tensor(v, dtype=torch.float32, device="cuda")
    wd, obj = f(w), f([0.0])
    E.gradnorm_update(wd, f(L), f(L0), f(g), gamma, lr, L_gn=obj)
    want_w, want_obj = oracle.gradnorm_update(w, L, L0, g, gamma, lr)
    assert np.allclose(wd.cpu().numpy(), want_w, rtol=1e-5, atol=1e-7)
    assert abs(float(obj) - want_obj) <= 1e-5 * max(want_obj, 1.0)


def test_two_backward_passes_add_up_to_the_backward_of_the_weighted_sum():
    """A step with two tasks sends each task's gradient through the encoder on its own (their input-gradient norms feed
    GradNorm) and accumulates the weight gradients: the sums equal one backward pass of the summed gradient."""
    import paper_2511_20564_b200 as E
    case = Case(S.WORKLOADS["tiny"], step=1, acts=[0, 0])            # identity activations: the backward is linear
    n_seeds, d = case.seeds.size, case.w.hidden
    rng = np.random.default_rng(3)
    dH_rec = rng.standard_normal((n_seeds, d)).astype(np.float32)
    ora0 = case.run_oracle()
    _, dH_ssl = oracle.ssl_loss(ora0["out"], case.X[case.seeds], 0.6)
    dH_ssl = dH_ssl.astype(np.float32)
    ora = case.run_oracle((dH_rec + dH_ssl).astype(np.float64))
    dev = "cuda"
    indptr, indices = torch.from_numpy(case.indptr).to(dev), torch.from_numpy(case.indices).to(dev)
    X = torch.from_numpy(case.X).to(dev)
    Ws = [torch.from_numpy(W).to(dev) for W in case.Ws]
    blocks = E.Blocks(case.w.n_nodes, n_seeds, case.w.fanouts, dev)
    E.sample_khop(indptr, indices, torch.from_numpy(case.seeds).to(dev), blocks, case.w.seed, case.step)
    H, ctx = E.sage_forward(blocks, X, Ws, acts=case.acts)
    g1 = torch.zeros_like(H); g1[:n_seeds] = torch.from_numpy(dH_rec).to(dev)
    g2 = torch.zeros_like(H); g2[:n_seeds] = torch.from_numpy(dH_ssl).to(dev)
    dWs, dX1 = E.sage_backward(blocks, X, Ws, ctx, g1, acts=case.acts)
    dX1 = dX1.clone()
    dWs, dX2 = E.sage_backward(blocks, X, Ws, ctx, g2, acts=case.acts, dWs=dWs, accumulate=True)
    torch.cuda.synchronize()
    n_src = ora["blocks"][-1]["n_src"]
    rss = reduction_rss(case, ora)
    for l, (gd, od) in enumerate(zip(dWs, ora["dWs"])):
        assert_close(f"dW[{l}]", gd.cpu().numpy(), od, False, 2 * rss["dW"][l])
    assert_close("dX", (dX1 + dX2)[:n_src].cpu().numpy(), ora["dX"], False, 2 * rss["dX"])
    n1 = float(E.gradient_norm(dX1, blocks.counts[-1][1:2].contiguous()))
    assert abs(n1 - oracle.frobenius_norm(dX1[:n_src].cpu().numpy())) <= 1e-5 * n1


@pytest.mark.parametrize("name,cap_seeds", [("tiny", None), ("medium_small", None), ("medium_small", 40000)])
def test_two_gradients_in_one_backward_pass(name, cap_seeds):
    """e2egrec_sage_backward_multi (the two task gradients of Sec. 4.3.1 as two right-hand sides, ReLU on): each input
    gradient equals the oracle's backward pass of that gradient alone, element by element, and -- bit for bit -- what
    e2egrec_sage_backward returns for it alone; the weight gradients are the sums of the two oracle passes.
    cap_seeds = 40000 sizes the blocks for millions of entries (runs of 128 entries, the large workload's launch shapes)."""
    import paper_2511_20564_b200 as E
    from helpers import encoder_flip_budgets, encoder_rss
    w = S.WORKLOADS[name]
    if cap_seeds:
        import dataclasses
        w = dataclasses.replace(S.WORKLOADS["medium"], batch=512)
    case = Case(w, step=2)
    bf16 = case.bf16
    n_seeds, d = case.seeds.size, w.hidden
    rng = np.random.default_rng(11)
    dH_a = case.upstream_grad(n_seeds, d)
    ora0 = case.run_oracle()
    _, dH_b = oracle.ssl_loss(ora0["out"], case.X[case.seeds], 0.7, bf16=bf16)      # the SSL task's gradient 2 w (H - X)
    dH_b = dH_b.astype(np.float32)
    ora_a, ora_b = case.run_oracle(dH_a.astype(np.float64)), case.run_oracle(dH_b.astype(np.float64))
    dev = "cuda"
    dt = torch.bfloat16 if bf16 else torch.float32
    indptr, indices = torch.from_numpy(case.indptr).to(dev), torch.from_numpy(case.indices).to(dev)
    X = torch.from_numpy(case.X).to(dev, dt)
    Ws = [torch.from_numpy(W).to(dev, dt) for W in case.Ws]
    blocks = E.Blocks(w.n_nodes, cap_seeds or n_seeds, w.fanouts, dev)
    E.sample_khop(indptr, indices, torch.from_numpy(case.seeds).to(dev), blocks, w.seed, case.step)
    H, ctx = E.sage_forward(blocks, X, Ws)
    ga, gb = torch.zeros_like(H), torch.zeros_like(H)
    ga[:n_seeds] = torch.from_numpy(dH_a).to(dev, dt)
    gb[:n_seeds] = torch.from_numpy(dH_b).to(dev, dt)
    dWs, (dXa, dXb) = E.sage_backward_multi(blocks, X, Ws, ctx, [ga, gb])
    _, dXa1 = E.sage_backward(blocks, X, Ws, ctx, ga)
    dXa1 = dXa1.clone()
    dWs_b, dXb1 = E.sage_backward(blocks, X, Ws, ctx, gb)
    torch.cuda.synchronize()
    n_src = ora_a["blocks"][-1]["n_src"]
    assert torch.equal(dXa[:n_src], dXa1[:n_src]) and torch.equal(dXb[:n_src], dXb1[:n_src])
    layer_out = [h.float().cpu().numpy() for _, h in E.sage_ctx_views(blocks, X, Ws, ctx)]
    tau = 2e-2 if bf16 else 1e-5
    B_dW_sum, rss_dW_sum = None, None
    for tag, got, ora in (("a", dXa, ora_a), ("b", dXb, ora_b)):
        rss = encoder_rss(case.Ws, None, ora["blocks"], ora["ctx"], ora["trace"])
        B_dW, B_dX = encoder_flip_budgets(case.Ws, None, ora["blocks"], ora["ctx"], ora["trace"], layer_out, tau)
        assert_close(f"dX[{tag}]", got[:n_src].float().cpu().numpy(), ora["dX"], bf16, rss["dX"], B_dX)
        B_dW_sum = B_dW if B_dW_sum is None else [x + y for x, y in zip(B_dW_sum, B_dW)]
        rss_dW_sum = rss["dW"] if rss_dW_sum is None else [np.sqrt(x ** 2 + y ** 2) for x, y in zip(rss_dW_sum, rss["dW"])]
    for l in range(len(Ws)):
        assert_close(f"dW[{l}]", dWs[l].cpu().numpy(), ora_a["dWs"][l] + ora_b["dWs"][l], bf16, rss_dW_sum[l], B_dW_sum[l])


def test_gradient_norms_of_several_matrices_in_one_pass():
    """e2egrec_gradient_norms: the norms of the task gradients of a step in one pass, each equal to the single call's."""
    import paper_2511_20564_b200 as E
    rng = np.random.default_rng(5)
    for dt, rows, d in ((torch.bfloat16, 70_001, 128), (torch.float32, 999, 36)):
        As = [torch.from_numpy(rng.standard_normal((rows, d)).astype(np.float32)).cuda().to(dt) for _ in range(3)]
        n_rows = torch.tensor([rows - 17], dtype=torch.int32, device="cuda")
        got = E.gradient_norms(As, n_rows).cpu().numpy()
        for i, A in enumerate(As):
            want = oracle.frobenius_norm(A[: rows - 17].float().cpu().numpy())
            assert abs(got[i] - want) <= 1e-5 * want
            assert got[i] == float(E.gradient_norm(A, n_rows))
