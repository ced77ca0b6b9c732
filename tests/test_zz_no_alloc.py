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
        assert_close("static vs workspace", out.float().cpu().numpy(), want.float().cpu().numpy()[:n],
                     dtype == torch.bfloat16)


def test_static_scratch_variant_rejects_what_does_not_fit():
    import paper_2511_20564_b200 as E
    limit = E.aggregate_forward_static_limit()
    assert limit == 8 << 20
    d = 256
    m = (limit // (2 * d * 4) + 2) * 128             # one chunk of 128 entries too many
    n = 10
    indptr = torch.zeros(n + 1, dtype=torch.int64, device="cuda")
    indptr[1:] = m
    indices = torch.zeros(m, dtype=torch.int32, device="cuda")
    X = torch.zeros(n, d, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(n, d, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(E.E2EGrecError, match="built-in buffer"):
        E.aggregate_forward_static(indptr, indices, X, out)
