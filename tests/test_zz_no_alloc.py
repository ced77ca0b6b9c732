"""The workspace-free aggregation entry point (collected last on purpose).

Some users of the library run where device memory cannot be requested: inside an application that has
already claimed the whole pool, or at a point of their step where an allocation would stall the GPU.
For them e2egrec_aggregate_forward_static keeps its scratch in a fixed buffer inside the library.  It
must give what e2egrec_aggregate_forward gives, also when the buffer still holds the previous call's
partial sums, and must refuse inputs that do not fit instead of overrunning the buffer.
"""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as S
from helpers import assert_close

pytestmark = pytest.mark.gpu


def _graph(n, m, seed):
    dst, src = S.powerlaw_directed(n, m, 1.1, seed)
    return S.coo_to_csr(n, dst, src)


def test_static_scratch_variant_matches_the_workspace_variant_twice_in_a_row():
    import paper_2511_20564_b200 as E
    # two different problems back to back: the second call finds the first call's partial sums in the buffer
    for n, m, d, dtype, seed in ((9_001, 250_000, 64, torch.bfloat16, 3), (4_000, 120_000, 32, torch.float32, 4)):
        indptr, indices = _graph(n, m, seed)
        assert np.diff(indptr).max() > 1000          # hub rows, so partial sums are really used
        X = torch.from_numpy(S.normal_features(n, d, seed)).cuda().to(dtype)
        ip, ix = torch.from_numpy(indptr).cuda(), torch.from_numpy(indices).cuda()
        want, _ = E.aggregate_forward(ip, ix, X)
        out = torch.full((n, d), float("nan"), dtype=dtype, device="cuda")
        E.aggregate_forward_static(ip, ix, X, out)
        torch.cuda.synchronize()
        bf16 = dtype == torch.bfloat16
        # against the other entry point: the same launches on another scratch buffer, so within the tests' tolerance
        # and in fact bit for bit
        assert_close("static vs workspace", out.float().cpu().numpy(), want.float().cpu().numpy()[:n], bf16)
        assert torch.equal(out, want[:n])
        # and against the CPU oracle's mean aggregation (Eq. 2 over whole rows), like every other parity test
        X_h = X.float().cpu().numpy()
        deg = np.maximum(np.diff(indptr), 1).astype(np.float64)[:, None]
        rss = np.sqrt(oracle.mean_aggregate(indptr, indices, X_h.astype(np.float64) ** 2) / deg)
        assert_close("static vs oracle", out.float().cpu().numpy(), oracle.mean_aggregate(indptr, indices, X_h, bf16), bf16, rss)


def _largest_fitting_entries(E, d, dtype, limit):
    """Largest entry count whose scratch (the size e2egrec_aggregate_forward asks for) still fits the built-in buffer."""
    X = torch.zeros(1, d, dtype=dtype, device="cuda")
    need = lambda m: E.binding.aggregate_ws_bytes(m, X)
    lo, hi = 1, 1 << 31
    while hi - lo > 1:
        mid = (lo + hi) // 2
        lo, hi = (mid, hi) if need(mid) <= limit else (lo, mid)
    return lo


def test_static_scratch_variant_at_its_limit_and_beyond():
    """The largest input that fits is computed (and matches the workspace variant bit for bit); one entry more is
    refused with the sizes in the message and nothing is written."""
    import paper_2511_20564_b200 as E
    limit = E.aggregate_forward_static_limit()
    assert limit == 8 << 20
    d, dtype = 1024, torch.float32                      # the widest rows: the limit is reached with few entries
    m = _largest_fitting_entries(E, d, dtype, limit)
    assert m < 2_000_000
    n = 64
    rng = np.random.default_rng(0)
    cuts = np.sort(rng.integers(0, m + 1, n - 1))
    indptr_h = np.concatenate([[0], cuts, [m]]).astype(np.int64)
    indices_h = rng.integers(0, n, m + 1).astype(np.int32)
    X = torch.from_numpy(S.normal_features(n, d, 1)).cuda()
    ip, ix = torch.from_numpy(indptr_h).cuda(), torch.from_numpy(indices_h).cuda()
    out = torch.full((n, d), float("nan"), dtype=dtype, device="cuda")
    E.aggregate_forward_static(ip, ix[:m], X, out)
    want, _ = E.aggregate_forward(ip, ix[:m], X)
    torch.cuda.synchronize()
    assert torch.equal(out, want[:n])
    ip2 = ip.clone()
    ip2[-1] = m + 1
    out.fill_(7.0)
    with pytest.raises(E.E2EGrecError, match="built-in buffer"):
        E.aggregate_forward_static(ip2, ix, X, out)
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
