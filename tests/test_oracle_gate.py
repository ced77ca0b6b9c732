"""Pins for the oracle's gated fusion (Sec. 4.3.2, "Concatenation with Gating")."""
import numpy as np

import oracle


def test_gate_closed_forms():
    rng = np.random.default_rng(0)
    F = rng.standard_normal((6, 5))
    fused, g = oracle.gate_fusion_forward(F, np.zeros((5, 5)), np.zeros(5))
    assert np.allclose(g, 0.5) and np.allclose(fused, F / 2)            # sigma(0) = 1/2
    fused, g = oracle.gate_fusion_forward(F, np.zeros((5, 5)), np.full(5, 50.0))
    assert np.allclose(fused, F)                                         # an open gate passes the features
    fused, g = oracle.gate_fusion_forward(F, np.zeros((5, 5)), np.full(5, -800.0))
    assert np.isfinite(g).all() and np.allclose(fused, 0.0)              # a shut one blocks them, no overflow
    Wg = rng.standard_normal((5, 5))
    _, g = oracle.gate_fusion_forward(F, Wg, None)
    assert ((g > 0) & (g < 1)).all()
    assert np.allclose(g[2], 1 / (1 + np.exp(-(Wg @ F[2]))))             # row by row, W applied to the feature vector


def test_gate_backward_by_central_differences():
    rng = np.random.default_rng(1)
    n, d = 5, 4
    F, Wg, bg = rng.standard_normal((n, d)), 0.7 * rng.standard_normal((d, d)), 0.3 * rng.standard_normal(d)
    R = rng.standard_normal((n, d))                                       # loss = <fused, R>
    fused, g = oracle.gate_fusion_forward(F, Wg, bg)
    dF, dW, db = oracle.gate_fusion_backward(R, F, g, Wg)
    loss = lambda F_, W_, b_: float((oracle.gate_fusion_forward(F_, W_, b_)[0] * R).sum())
    eps = 1e-6
    for (i, k) in [(0, 0), (2, 3), (4, 1)]:
        Fp, Fm = F.copy(), F.copy()
        Fp[i, k] += eps; Fm[i, k] -= eps
        assert np.isclose((loss(Fp, Wg, bg) - loss(Fm, Wg, bg)) / (2 * eps), dF[i, k], rtol=1e-6, atol=1e-8)
    for (a, b) in [(0, 0), (1, 2), (3, 3)]:
        Wp, Wm = Wg.copy(), Wg.copy()
        Wp[a, b] += eps; Wm[a, b] -= eps
        assert np.isclose((loss(F, Wp, bg) - loss(F, Wm, bg)) / (2 * eps), dW[a, b], rtol=1e-6, atol=1e-8)
    for a in range(d):
        bp, bm = bg.copy(), bg.copy()
        bp[a] += eps; bm[a] -= eps
        assert np.isclose((loss(F, Wg, bp) - loss(F, Wg, bm)) / (2 * eps), db[a], rtol=1e-6, atol=1e-8)


def test_gate_bf16_storage_points():
    rng = np.random.default_rng(2)
    F = oracle.round_bf16(rng.standard_normal((8, 6)))
    Wg = oracle.round_bf16(0.5 * rng.standard_normal((6, 6)))
    fused, g = oracle.gate_fusion_forward(F, Wg, None, bf16=True)
    assert np.array_equal(fused, oracle.round_bf16(fused)) and np.array_equal(g, oracle.round_bf16(g))
    exact, _ = oracle.gate_fusion_forward(F, Wg, None)
    assert np.allclose(fused, exact, rtol=3e-2, atol=3e-2)
    dF, dW, db = oracle.gate_fusion_backward(np.ones_like(F), F, g, Wg, bf16=True)
    assert np.array_equal(dF, oracle.round_bf16(dF)) and dW.shape == (6, 6) and db.shape == (6,)
