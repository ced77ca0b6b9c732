"""Pins for the oracle's SSL loss and GradNorm weight update (Sec. 4.2, Sec. 4.3.1)."""
import numpy as np

import oracle


def test_ssl_loss_closed_forms_and_central_differences():
    rng = np.random.default_rng(0)
    X = rng.standard_normal((7, 5))
    loss, dH = oracle.ssl_loss(X, X, 0.7)
    assert loss == 0.0 and not dH.any()                       # perfect reconstruction
    H = rng.standard_normal((7, 5))
    loss, dH = oracle.ssl_loss(H, X, 1.0)
    assert np.isclose(loss, np.linalg.norm(H - X, "fro") ** 2, rtol=1e-14)
    w, eps = 0.3, 1e-6
    _, dHw = oracle.ssl_loss(H, X, w)
    for (i, k) in [(0, 0), (3, 2), (6, 4)]:
        Hp, Hm = H.copy(), H.copy()
        Hp[i, k] += eps
        Hm[i, k] -= eps
        fd = w * (oracle.ssl_loss(Hp, X)[0] - oracle.ssl_loss(Hm, X)[0]) / (2 * eps)
        assert np.isclose(fd, dHw[i, k], rtol=1e-7, atol=1e-9)
    _, dHb = oracle.ssl_loss(H, X, w, bf16=True)
    assert np.array_equal(dHb, oracle.round_bf16(dHb)) and np.allclose(dHb, dHw, rtol=1e-2, atol=1e-6)


def test_frobenius_norm():
    assert oracle.frobenius_norm(np.array([[3.0, 0.0], [0.0, 4.0]])) == 5.0


def test_gradnorm_update_invariants():
    # balanced: both tasks at the same relative rate and the same weighted gradient norm -> nothing moves
    w, L_gn = oracle.gradnorm_update([1.0, 1.0], [2.0, 4.0], [4.0, 8.0], [3.0, 3.0])
    assert L_gn == 0.0 and np.allclose(w, [1.0, 1.0])
    # the task whose weighted gradient is above its target loses weight, the other gains; weights sum to T
    w, L_gn = oracle.gradnorm_update([1.0, 1.0], [1.0, 1.0], [1.0, 1.0], [10.0, 1.0], lr=0.01)
    assert L_gn == 9.0 and w[0] < 1.0 < w[1] and np.isclose(w.sum(), 2.0)
    # a task that trains more slowly (loss ratio higher) gets a larger target: with equal gradients it gains weight
    w, _ = oracle.gradnorm_update([1.0, 1.0], [0.9, 0.1], [1.0, 1.0], [2.0, 2.0], gamma=1.0, lr=0.01)
    assert w[0] > 1.0 > w[1] and np.isclose(w.sum(), 2.0)
    # gamma = 0 ignores the training rates
    w0, _ = oracle.gradnorm_update([1.0, 1.0], [0.9, 0.1], [1.0, 1.0], [2.0, 2.0], gamma=0.0)
    assert np.allclose(w0, [1.0, 1.0])
    # weights stay positive
    w, _ = oracle.gradnorm_update([0.01, 1.99], [1.0, 1.0], [1.0, 1.0], [1000.0, 0.001], lr=1.0)
    assert (w > 0).all() and np.isclose(w.sum(), 2.0)


def test_gradnorm_step_is_the_gradient_of_the_stated_objective():
    """With the targets held constant, L_gn(w) = sum |w_i g_i - c_i|: its difference quotient in w gives the step."""
    w = np.array([0.8, 1.2]); L = np.array([0.5, 0.9]); L0 = np.array([1.0, 1.0]); g = np.array([4.0, 1.5])
    gamma, lr = 1.0, 1e-3
    G = w * g
    r = (L / L0) / (L / L0).mean()
    c = G.mean() * r ** gamma
    grad = np.array([(abs((w[i] + 1e-7) * g[i] - c[i]) - abs((w[i] - 1e-7) * g[i] - c[i])) / 2e-7 for i in range(2)])
    want = w - lr * grad
    want = want * 2 / want.sum()
    got, _ = oracle.gradnorm_update(w, L, L0, g, gamma, lr)
    assert np.allclose(got, want, rtol=1e-6)
