"""GPU parity at the benchmark's full sizes, in the launch configuration that bench.py times.

The oracle cannot run a graph of 10^8 .. 2*10^9 entries whole, so it is given exactly the part of the input it
needs for the outputs that are compared: the rows (or columns) of sampled nodes, cut out of the edge list with
plain numpy / torch indexing (never out of anything the CUDA library produced), and it computes those outputs
one by one.  Integer results are compared bit for bit, floating point at the tolerances of the other tests.
"""
import types

import numpy as np
import pytest
import torch

import oracle
import synth_inputs as S
from helpers import assert_blocks_equal, assert_close
from test_gpu_parity import _check_float

pytestmark = pytest.mark.gpu


def _need(device_gb, host_gb):
    import psutil
    free, _ = torch.cuda.mem_get_info()
    if free < device_gb * 1e9:
        pytest.skip(f"needs {device_gb} GB of free device memory, {free / 1e9:.0f} GB available")
    if psutil.virtual_memory().available < host_gb * 1e9:
        pytest.skip(f"needs {host_gb} GB of host memory")


# ----------------------------------------------------------------------------- whole-graph aggregation, 5 M / 100 M

def test_full_graph_aggregation_at_benchmark_size():
    """5 M nodes, 100 M entries, d = 64 bf16 (the `fullgraph` workload of bench.py): ingest, forward and transpose on
    the device; rows and columns of sampled nodes (the heaviest hubs, random ones, empty ones) against the oracle."""
    import paper_2511_20564_b200 as E
    _need(20, 24)
    n, m, d = 5_000_000, 100_000_000, 64
    dev = torch.device("cuda")
    dst, src = S.powerlaw_directed(n, m, 1.1, 2)
    indptr, indices, st1 = E.graph_from_coo(n, torch.from_numpy(dst).to(dev), torch.from_numpy(src).to(dev))
    indices = indices.contiguous()
    csc_ptr, csc_row, _, st2 = E.csr_transpose(indptr, indices, n)
    csc_row = csc_row.contiguous()
    assert int(st1) == 0 and int(st2) == 0
    deg = np.bincount(dst, minlength=n).astype(np.int64)
    indeg = np.bincount(src, minlength=n).astype(np.int64)
    ip_h = indptr.cpu().numpy()
    assert ip_h[0] == 0 and np.array_equal(np.diff(ip_h), deg)
    assert np.array_equal(np.diff(csc_ptr.cpu().numpy()), indeg)

    X = S.to_bf16_values(S.normal_features(n, d, 2))
    G = S.to_bf16_values(S.normal_features(n, d, 2, stream=11))
    Xd, Gd = torch.from_numpy(X).to(dev, torch.bfloat16), torch.from_numpy(G).to(dev, torch.bfloat16)
    inv_deg = torch.from_numpy(np.where(deg > 0, 1.0 / np.maximum(deg, 1), 0.0).astype(np.float32)).to(dev)
    out, _ = E.aggregate_forward(indptr, indices, Xd)
    dX, _ = E.aggregate_backward(csc_ptr, csc_row, inv_deg, Gd)
    torch.cuda.synchronize()

    rng = np.random.default_rng(7)

    def pick(counts):
        heavy = np.argsort(counts)[-4:]
        empty = np.flatnonzero(counts == 0)[:64]
        return np.unique(np.concatenate([heavy, empty, rng.integers(0, n, 3000)])).astype(np.int64)

    # ---- rows: CSR entries bit for bit, mean rows within the bf16 tolerance
    rows = pick(deg)
    flag = np.zeros(n, bool)
    flag[rows] = True
    keep = flag[dst]
    wide_ptr, sub_idx = oracle.csr_from_coo(n, dst[keep], src[keep])      # all other rows are empty
    sub_ptr = np.concatenate([[0], np.cumsum(np.diff(wide_ptr)[rows])]).astype(np.int64)
    got_idx = torch.cat([indices[int(ip_h[r]): int(ip_h[r + 1])] for r in rows]).cpu().numpy()
    assert np.array_equal(np.diff(sub_ptr), deg[rows]) and np.array_equal(got_idx, sub_idx)
    want = oracle.mean_aggregate(sub_ptr, sub_idx, X, True)
    rss = np.sqrt(oracle.mean_aggregate(sub_ptr, sub_idx, X.astype(np.float64) ** 2) / np.maximum(deg[rows], 1)[:, None])
    assert_close("aggregate_forward rows", out[torch.from_numpy(rows).to(dev)].float().cpu().numpy(), want, True, rss)

    # ---- columns of the transpose: only their entries go to the oracle, with the true row lengths
    cols = pick(indeg)
    flag[:] = False
    flag[cols] = True
    keep = flag[src]
    part_ptr, part_idx = S.coo_to_csr(n, dst[keep], np.searchsorted(cols, src[keep]).astype(np.int32))
    want = oracle.full_aggregate_backward(part_ptr, part_idx, cols.size, G, True, row_len=deg)
    G2 = G.astype(np.float64) ** 2 / np.maximum(deg, 1)[:, None]
    rss = np.sqrt(oracle.full_aggregate_backward(part_ptr, part_idx, cols.size, G2, row_len=deg))
    assert_close("aggregate_backward columns", dX[torch.from_numpy(cols).to(dev)].float().cpu().numpy(), want, True, rss)


# ----------------------------------------------------------------------------- sampled training step, 50 M / 2 * 10^9

def _rows_of(node_ids, row_d, col_d, n, chunk=1 << 28):
    """Canonical CSR (host arrays) that holds the rows of `node_ids` and is empty elsewhere, cut out of the edge
    list on the device with torch indexing and torch.sort."""
    dev = row_d.device
    flag = torch.zeros(n, dtype=torch.bool, device=dev)
    flag[torch.from_numpy(np.ascontiguousarray(node_ids)).to(dev).long()] = True
    keys = []
    for s in range(0, row_d.numel(), chunk):
        r, c = row_d[s: s + chunk], col_d[s: s + chunk]
        keep = flag[r.long()]
        keys.append((r[keep].long() << 32) | c[keep].long())
        del keep
    key = torch.sort(torch.cat(keys))[0]
    del keys
    rows = key >> 32
    indptr = torch.zeros(n + 1, dtype=torch.int64, device=dev)
    indptr[1:] = torch.cumsum(torch.bincount(rows, minlength=n), 0)
    indices = (key & 0xFFFFFFFF).to(torch.int32)
    return indptr.cpu().numpy(), indices.cpu().numpy()


def test_large_workload_at_benchmark_size():
    """50 M nodes, 10^9 interactions (2 * 10^9 CSR entries), d = 256 bf16, fanout [20, 10, 5], batch 8 192 (the `large`
    workload of bench.py).  The sampled blocks of the whole batch are compared bit for bit; the forward rows of the
    first 64 seeds come from the whole-batch launch (a node's sample does not depend on the batch), and a launch
    with the same capacities on those 64 seeds alone is compared in full, forward and backward."""
    import paper_2511_20564_b200 as E
    _need(130, 60)
    w = S.WORKLOADS["large"]
    dev = torch.device("cuda")
    n, L = w.n_nodes, len(w.fanouts)
    users_d, items_d = S.bipartite_interactions_device(w.n_users, w.n_items, w.n_interactions, w.alpha_user,
                                                       w.alpha_item, w.seed, w.q, dev)
    seeds = S.seed_batch_from_interactions_device(users_d, items_d, w.batch, w.seed, 0)
    row_d, col_d = torch.cat([users_d, items_d]), torch.cat([items_d, users_d])
    del users_d, items_d
    indptr, indices, status = E.graph_from_coo(n, row_d, col_d)
    indices = indices.contiguous()
    assert int(status) == 0
    torch.cuda.empty_cache()
    X = S.normal_features_device(n, w.dim, w.seed, torch.bfloat16, dev)
    Ws_h = S.build_weights(w)
    Ws = [torch.from_numpy(W).to(dev, torch.bfloat16) for W in Ws_h]
    step = 0

    def gpu_run(seed_ids, dH):
        blocks = E.Blocks(n, w.batch, w.fanouts, dev)          # capacities of the whole batch, as bench.py allocates
        E.sample_khop(indptr, indices, torch.from_numpy(seed_ids).to(dev), blocks, w.seed, step)
        H, ctx = E.sage_forward(blocks, X, Ws)
        res = dict(blocks=blocks.to_host(), out=H.float().cpu().numpy())
        if dH is not None:
            g = torch.zeros(H.shape, dtype=torch.bfloat16, device=dev)
            g[: dH.shape[0]] = torch.from_numpy(dH).to(dev, torch.bfloat16)
            dWs, dXr = E.sage_backward(blocks, X, Ws, ctx, g)
            n_src = res["blocks"][-1]["n_src"]
            res["dWs"] = [t.float().cpu().numpy() for t in dWs]
            res["dX"] = dXr[:n_src].float().cpu().numpy()
            res["layer_out"] = [h[: res["blocks"][L - 1 - l]["n_dst"]].float().cpu().numpy()
                                for l, (_, h) in enumerate(E.sage_ctx_views(blocks, X, Ws, ctx))]
        torch.cuda.synchronize()
        return res

    # ---- whole batch: blocks bit for bit.  The oracle samples hop h+1 on the rows of its own frontier F_h.
    full = gpu_run(seeds, None)
    frontier, ora_blocks = seeds, None
    for h in range(1, L + 1):
        ip_h, ix_h = _rows_of(frontier, row_d, col_d, n)
        ora_blocks = oracle.sample_khop(ip_h, ix_h, seeds, w.fanouts[:h], w.seed, step)
        frontier = ora_blocks[-1]["src_nodes"]
    assert_blocks_equal(full["blocks"], ora_blocks)
    assert ora_blocks[-1]["n_edges"] > 1_000_000
    del row_d, col_d

    # ---- the first 64 seeds: forward rows of the whole-batch launch, then a launch of their own in full
    sub = np.ascontiguousarray(seeds[:64])
    sub_blocks = oracle.sample_khop(ip_h, ix_h, sub, w.fanouts, w.seed, step)     # their frontiers lie inside F_2
    rows = torch.from_numpy(sub_blocks[-1]["src_nodes"]).to(dev).long()
    X_rows = X[rows].float().cpu().numpy()
    dH = S.to_bf16_values(np.random.default_rng(99).standard_normal((sub.size, w.hidden)).astype(np.float32))
    out, ctx = oracle.sage_forward(sub_blocks, X_rows, Ws_h, bf16=True, gathered=True)
    trace = []
    dWs, _, dXr = oracle.sage_backward(sub_blocks, ctx, Ws_h, dH, bf16=True, trace=trace)
    ora = dict(blocks=sub_blocks, out=out, ctx=ctx, dWs=dWs, dX=dXr, trace=trace)
    case = types.SimpleNamespace(Ws=Ws_h, acts=None, bf16=True, seeds=sub)
    from helpers import reduction_rss
    assert_close("forward rows of the whole batch", full["out"][: sub.size], out, True, reduction_rss(case, ora)["forward"])
    part = gpu_run(sub, dH)
    assert_blocks_equal(part["blocks"], sub_blocks)
    _check_float(case, part, ora)
