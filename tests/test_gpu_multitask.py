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
