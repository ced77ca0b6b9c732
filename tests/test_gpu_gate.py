"""GPU parity of the gated fusion (Sec. 4.3.2) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as S
from helpers import assert_close

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,n_rows,d", [("f32", 200, 48), ("bf16", 1000, 320), ("bf16", 4096, 128), ("bf16", 77, 40)])
def test_gate_fusion_forward_and_backward(dtype, n_rows, d):
    """tensor-core shapes (d a multiple of 64), a width that is not (fp32-FMA path), a ragged row count."""
    import paper_2511_20564_b200 as E
    bf16 = dtype == "bf16"
    dt = torch.bfloat16 if bf16 else torch.float32
    rng = np.random.default_rng(n_rows + d)
    rows = (n_rows + 127) // 128 * 128
    F = np.zeros((rows, d), np.float32)
    F[:n_rows] = rng.standard_normal((n_rows, d))
    Wg = S.glorot_uniform(d, d, 5, 50) * 2.0
    bg = (0.2 * rng.standard_normal(d)).astype(np.float32)
    R = np.zeros((rows, d), np.float32)
    R[:n_rows] = rng.standard_normal((n_rows, d))
    if bf16:
        F, Wg, R = S.to_bf16_values(F), S.to_bf16_values(Wg), S.to_bf16_values(R)
    cu = lambda a, t=None: torch.from_numpy(np.ascontiguousarray(a)).cuda().to(t) if t else torch.from_numpy(np.ascontiguousarray(a)).cuda()
    Fd, Wd = cu(F, dt), cu(Wg, dt)
    fused, gate, ws = E.gate_fusion_forward(Fd, n_rows, Wd, cu(bg))
    want_fused, want_gate = oracle.gate_fusion_forward(F[:n_rows], Wg, bg, bf16)
    # scale of the terms behind a pre-activation: |F| |Wg|^T; the gate's slope is at most 1/4
    rss_pre = np.sqrt((F[:n_rows].astype(np.float64) ** 2) @ (Wg.astype(np.float64) ** 2).T)
    assert_close("gate", gate[:n_rows].float().cpu().numpy(), want_gate, bf16, 0.25 * rss_pre)
    assert_close("fused", fused[:n_rows].float().cpu().numpy(), want_fused, bf16, 0.25 * rss_pre * np.abs(F[:n_rows]))
    assert not fused[n_rows:].any() and not gate[n_rows:].any()
    # backward from the oracle's gate (the stored gates of the two sides may sit one bf16 step apart)
    gate_in = cu(np.vstack([want_gate, np.zeros((rows - n_rows, d))]).astype(np.float32), dt)
    dF, dWg, dbg = E.gate_fusion_backward(cu(R, dt), Fd, n_rows, gate_in, Wd, ws)
    torch.cuda.synchronize()
    w_dF, w_dW, w_db = oracle.gate_fusion_backward(R[:n_rows], F[:n_rows], want_gate, Wg, bf16)
    dpre = np.abs(R[:n_rows] * F[:n_rows] * want_gate * (1 - want_gate))
    rss_dF = np.sqrt((dpre ** 2) @ (Wg.astype(np.float64) ** 2)) + np.abs(R[:n_rows] * want_gate)
    assert_close("dF", dF[:n_rows].float().cpu().numpy(), w_dF, bf16, rss_dF)
    assert_close("dWg", dWg.cpu().numpy(), w_dW, bf16, np.sqrt((dpre ** 2).T @ (F[:n_rows].astype(np.float64) ** 2)))
    assert_close("dbg", dbg.cpu().numpy(), w_db, bf16, np.sqrt((dpre ** 2).sum(0)))
