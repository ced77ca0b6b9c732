"""GPU parity: the CUDA path through the C ABI against the CPU oracle, same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as S
from helpers import (Case, assert_blocks_equal, assert_close, assert_close_budget, reduction_rss,
                     relu_flip_budgets)

pytestmark = pytest.mark.gpu


def _check_float(case, gpu, ora):
    n_seeds = case.seeds.size
    n_src = ora["blocks"][-1]["n_src"]
    rss = reduction_rss(case, ora)
    assert_close("forward", gpu["out"][:n_seeds], ora["out"], case.bf16, rss["forward"])
    if "dWs" in ora:
        # ReLU decisions that differ between fp32 and float64 sums are accepted only within tau of the kink
        tau = 2e-2 if case.bf16 else 1e-5
        B_dW, B_dX = relu_flip_budgets(case, ora, gpu, tau)
        for l, (g, o) in enumerate(zip(gpu["dWs"], ora["dWs"])):
            assert_close_budget(f"dW[{l}]", g, o, B_dW[l], case.bf16, rss["dW"][l])
        assert_close_budget("dX", gpu["dX"][:n_src], ora["dX"], B_dX, case.bf16, rss["dX"])


@pytest.mark.parametrize("step", [0, 3])
def test_tiny_fp32_sample_forward_backward(step):
    case = Case(S.WORKLOADS["tiny"], step=step)
    dH = case.upstream_grad(case.seeds.size, case.w.hidden)
    ora = case.run_oracle(dH)
    gpu = case.run_gpu(dH)
    assert_blocks_equal(gpu["blocks"], ora["blocks"])
    _check_float(case, gpu, ora)


def test_medium_small_bf16_sample_forward_backward():
    case = Case(S.WORKLOADS["medium_small"], step=1)
    dH = case.upstream_grad(case.seeds.size, case.w.hidden)
    ora = case.run_oracle(dH)
    gpu = case.run_gpu(dH)
    assert_blocks_equal(gpu["blocks"], ora["blocks"])
    _check_float(case, gpu, ora)


def test_blocks_with_capacity_for_millions_of_entries():
    """Block buffers sized for 40 000 seeds on the 500 k-node graph (outer block: 5 M entries of capacity) while the batch
    has 512: the library then cuts the transposed aggregation into runs of 128 entries, the run length of the largest
    workload (256-byte rows: no streaming through shared memory, which the next test covers)."""
    import dataclasses
    w = dataclasses.replace(S.WORKLOADS["medium"], batch=512)
    case = Case(w, step=2)
    dH = case.upstream_grad(case.seeds.size, w.hidden)
    ora = case.run_oracle(dH)
    gpu = case.run_gpu(dH, cap_seeds=40000)
    assert gpu["blocks_obj"].caps[-1][2] >= 1 << 21
    assert_blocks_equal(gpu["blocks"], ora["blocks"])
    _check_float(case, gpu, ora)


def test_wide_rows_with_capacity_for_millions_of_entries():
    """256-value bf16 rows in block buffers sized for 40 000 seeds on the 500 k-node graph (outer block: 5 M entries of
    capacity): the launch shapes of the largest workload, where the aggregation kernels stream their rows through shared
    memory with the TMA unit."""
    import dataclasses
    w = dataclasses.replace(S.WORKLOADS["medium"], dim=256, hidden=256, batch=512)
    case = Case(w, step=2)
    dH = case.upstream_grad(case.seeds.size, w.hidden)
    ora = case.run_oracle(dH)
    gpu = case.run_gpu(dH, cap_seeds=40000)
    assert gpu["blocks_obj"].caps[-1][2] >= 1 << 21
    assert_blocks_equal(gpu["blocks"], ora["blocks"])
    _check_float(case, gpu, ora)


def test_medium_small_bf16_linear_backward_is_strict():
    """Identity activations: no sign decisions, so every gradient element is held to the plain tolerance."""
    case = Case(S.WORKLOADS["medium_small"], step=5, acts=[0, 0])
    dH = case.upstream_grad(case.seeds.size, case.w.hidden)
    ora = case.run_oracle(dH)
    gpu = case.run_gpu(dH)
    assert_blocks_equal(gpu["blocks"], ora["blocks"])
    n_src = ora["blocks"][-1]["n_src"]
    rss = reduction_rss(case, ora)
    assert_close("forward", gpu["out"][: case.seeds.size], ora["out"], True, rss["forward"])
    for l, (g, o) in enumerate(zip(gpu["dWs"], ora["dWs"])):
        assert_close(f"dW[{l}]", g, o, True, rss["dW"][l])
    assert_close("dX", gpu["dX"][:n_src], ora["dX"], True, rss["dX"])


def test_run_to_run_bit_identical():
    case = Case(S.WORKLOADS["medium_small"], step=2)
    dH = case.upstream_grad(case.seeds.size, case.w.hidden)
    a = case.run_gpu(dH)
    b = case.run_gpu(dH)
    assert np.array_equal(a["out"], b["out"]) and np.array_equal(a["dX"], b["dX"])
    for x, y in zip(a["dWs"], b["dWs"]):
        assert np.array_equal(x, y)
    assert_blocks_equal(a["blocks"], b["blocks"])


def test_scratch_is_reusable_across_steps():
    """One Blocks object (one scratch buffer) serves consecutive steps."""
    import paper_2511_20564_b200 as E
    w = S.WORKLOADS["tiny"]
    indptr, indices, _ = S.build_graph(w)
    blocks = E.Blocks(w.n_nodes, w.batch, w.fanouts)
    ip, ix = torch.from_numpy(indptr).cuda(), torch.from_numpy(indices).cuda()
    for step in range(3):
        seeds = S.seed_batch(w.n_nodes, w.batch, w.seed, step)
        E.sample_khop(ip, ix, torch.from_numpy(seeds).cuda(), blocks, w.seed, step)
        ora = oracle.sample_khop(indptr, indices, seeds, w.fanouts, w.seed, step)
        assert_blocks_equal(blocks.to_host(), ora)


def _star_graph(n_leaves):
    row = np.concatenate([np.zeros(n_leaves, np.int32), np.arange(1, n_leaves + 1, dtype=np.int32)])
    col = np.concatenate([np.arange(1, n_leaves + 1, dtype=np.int32), np.zeros(n_leaves, np.int32)])
    return S.coo_to_csr(n_leaves + 3, row, col)       # nodes n_leaves+1, n_leaves+2 are isolated


@pytest.mark.parametrize("fanouts,seeds", [((4, 3), [0, 5, 301]), ((128,), [0, 1, 2]), ((2, 2, 2), [7]),
                                           ((5, 5), [301, 302])])
def test_edge_cases_hub_isolated_and_take_all(fanouts, seeds):
    n_leaves = 300
    graph = _star_graph(n_leaves)
    w = S.Workload("star", 1, n_leaves + 2, 0, None, None, 9, 8, 8, "f32", tuple(fanouts), len(seeds))
    case = Case(w, step=4, seeds=seeds, graph=graph)
    dH = case.upstream_grad(len(seeds), 8)
    ora = case.run_oracle(dH)
    gpu = case.run_gpu(dH)
    assert_blocks_equal(gpu["blocks"], ora["blocks"])
    _check_float(case, gpu, ora)


def test_hub_column_longer_than_a_chunk():
    """Many destinations sample the same hub, so its transposed column spans several warps' chunks."""
    n_leaves = 3000
    graph = _star_graph(n_leaves)
    seeds = np.arange(1, 1201, dtype=np.int32)
    for dtype, d in (("f32", 16), ("bf16", 64)):
        w = S.Workload("star", 1, n_leaves + 2, 0, None, None, 9, d, d, dtype, (3, 2), seeds.size)
        case = Case(w, step=0, seeds=seeds, graph=graph)
        dH = case.upstream_grad(seeds.size, d)
        ora = case.run_oracle(dH)
        gpu = case.run_gpu(dH)
        assert_blocks_equal(gpu["blocks"], ora["blocks"])
        _check_float(case, gpu, ora)


def test_empty_batch():
    graph = _star_graph(10)
    w = S.Workload("star", 1, 12, 0, None, None, 9, 8, 8, "f32", (3, 2), 0)
    case = Case(w, step=0, seeds=np.zeros(0, np.int32), graph=graph)
    gpu = case.run_gpu()
    for b in gpu["blocks"]:
        assert b["n_dst"] == 0 and b["n_src"] == 0 and b["n_edges"] == 0 and b["status"] == 0


def test_empty_and_tiny_batches_in_buffers_for_millions_of_entries():
    """No seed at all, and three seeds, with 256-value bf16 rows in buffers sized for 40 000 seeds: the kernels that stream
    their rows through shared memory see warps without any destination, and a stream of a handful of entries."""
    import dataclasses
    w = dataclasses.replace(S.WORKLOADS["medium"], dim=256, hidden=256, batch=3)
    graph = S.build_graph(w)[:2]
    empty = Case(w, step=0, seeds=np.zeros(0, np.int32), graph=graph)
    dH0 = empty.upstream_grad(0, w.hidden)
    gpu = empty.run_gpu(dH0, cap_seeds=40000)
    assert gpu["blocks_obj"].caps[-1][2] >= 1 << 20
    for b in gpu["blocks"]:
        assert b["n_dst"] == 0 and b["n_src"] == 0 and b["n_edges"] == 0 and b["status"] == 0
    assert all(float(np.abs(g).max()) == 0.0 for g in gpu["dWs"])
    case = Case(w, step=5, graph=graph)
    dH = case.upstream_grad(case.seeds.size, w.hidden)
    ora = case.run_oracle(dH)
    gpu = case.run_gpu(dH, cap_seeds=40000)
    assert_blocks_equal(gpu["blocks"], ora["blocks"])
    _check_float(case, gpu, ora)


def test_out_of_range_seed_sets_status_and_does_not_fault():
    import paper_2511_20564_b200 as E
    indptr, indices = _star_graph(10)
    blocks = E.Blocks(13, 2, (2,))
    seeds = torch.tensor([1, 99], dtype=torch.int32, device="cuda")
    E.sample_khop(torch.from_numpy(indptr).cuda(), torch.from_numpy(indices).cuda(), seeds, blocks, 0, 0)
    assert blocks.to_host()[0]["status"] & 1


def test_host_side_argument_errors():
    import paper_2511_20564_b200 as E
    with pytest.raises(E.E2EGrecError):
        E.sample_khop_workspace(100, 4, [200])          # fanout above the limit
    with pytest.raises(E.E2EGrecError):
        E.sample_khop_workspace(100, 4, [3, 3, 3, 3, 3])  # too many hops
    blocks = E.Blocks(100, 4, (3,))
    X = torch.zeros(100, 6, device="cuda")              # 24-byte rows: not 16-byte aligned
    W = torch.zeros(8, 12, device="cuda")
    with pytest.raises(E.E2EGrecError):
        E.sage_forward(blocks, X, [W])


# ----------------------------------------------------------------------------- whole-graph aggregation

def _powerlaw_graph(n, m, seed):
    dst, src = S.powerlaw_directed(n, m, 1.1, seed)
    return S.coo_to_csr(n, dst, src)


@pytest.mark.parametrize("dtype,d", [("bf16", 64), ("f32", 32), ("bf16", 256), ("f32", 512), ("bf16", 1024),
                                     ("f32", 768), ("f32", 1024)])
def test_full_graph_aggregation_forward_and_transpose(dtype, d):
    """Rows with tens of thousands of entries (split over many warps), empty rows, and a ragged tail; row widths up to
    the documented limit of 1024 values in either dtype (4096-byte rows in fp32)."""
    import paper_2511_20564_b200 as E
    n, m = 20_011, 600_000
    indptr, indices = _powerlaw_graph(n, m, 2)
    assert np.diff(indptr).max() > 20_000 and (np.diff(indptr) == 0).any()
    bf16 = dtype == "bf16"
    dt = torch.bfloat16 if bf16 else torch.float32
    X = S.normal_features(n, d, 5)
    G = S.normal_features(n, d, 6, stream=11)
    if bf16:
        X, G = S.to_bf16_values(X), S.to_bf16_values(G)
    ip, ix = torch.from_numpy(indptr).cuda(), torch.from_numpy(indices).cuda()
    out, _ = E.aggregate_forward(ip, ix, torch.from_numpy(X).cuda().to(dt))
    want = oracle.mean_aggregate(indptr, indices, X, bf16)
    deg = np.diff(indptr).astype(np.float64)[:, None]
    rss_f = np.sqrt(oracle.mean_aggregate(indptr, indices, X.astype(np.float64) ** 2) / np.maximum(deg, 1))
    assert_close("aggregate_forward", out.float().cpu().numpy()[:n], want, bf16, rss_f)
    # transpose through the oracle-built CSC
    cptr, crow, _ = oracle.csr_transpose(n, n, indptr, indices)
    inv_deg = np.where(deg[:, 0] > 0, 1.0 / np.maximum(deg[:, 0], 1), 0.0).astype(np.float32)
    dX, _ = E.aggregate_backward(torch.from_numpy(cptr).cuda(), torch.from_numpy(crow).cuda(),
                                 torch.from_numpy(inv_deg).cuda(), torch.from_numpy(G).cuda().to(dt))
    want = oracle.full_aggregate_backward(indptr, indices, n, G, bf16)
    rss_b = np.sqrt(oracle.full_aggregate_backward(indptr, indices, n, G.astype(np.float64) ** 2 / np.maximum(deg, 1)))
    assert_close("aggregate_backward", dX.float().cpu().numpy()[:n], want, bf16, rss_b)


# ----------------------------------------------------------------------------- graph ingest

@pytest.mark.parametrize("n,m", [(5_000, 80_000), (70_001, 300_007), (3, 0)])
def test_graph_ingest_is_bit_exact(n, m):
    """CSR from an edge list and its transpose: several sort tiles, a ragged tail, parallel edges, empty input."""
    import paper_2511_20564_b200 as E
    rng = np.random.default_rng(n)
    row = S.zipf_ranks(rng, m, n, 1.1).astype(np.int32)
    col = rng.integers(0, n, m).astype(np.int32)
    indptr, indices, status = E.graph_from_coo(n, torch.from_numpy(row).cuda(), torch.from_numpy(col).cuda())
    want_ptr, want_idx = oracle.csr_from_coo(n, row, col)
    assert int(status) == 0
    assert np.array_equal(indptr.cpu().numpy(), want_ptr) and np.array_equal(indices.cpu().numpy(), want_idx)
    cptr, crow, ceid, status = E.csr_transpose(indptr, indices.contiguous(), n)
    w_ptr, w_row, w_eid = oracle.csr_transpose(n, n, want_ptr, want_idx)
    assert int(status) == 0
    assert np.array_equal(cptr.cpu().numpy(), w_ptr) and np.array_equal(crow.cpu().numpy(), w_row)
    assert np.array_equal(ceid.cpu().numpy(), w_eid)


def test_graph_ingest_flags_ids_out_of_range():
    import paper_2511_20564_b200 as E
    row = torch.tensor([0, 1, 7], dtype=torch.int32, device="cuda")
    col = torch.tensor([1, -2, 0], dtype=torch.int32, device="cuda")
    _, _, status = E.graph_from_coo(4, row, col)
    assert int(status) & 1


def test_three_hops_wide_rows_bf16():
    """The shape of the large workload (3 hops, fanout [20,10,5], d = hidden = 256 bf16) on a small graph."""
    base = S.WORKLOADS["medium_small"]
    w = S.Workload("large_shape", base.n_users, base.n_items, base.n_interactions, 1.05, 1.05, 3, 256, 256, "bf16",
                   (20, 10, 5), 128)
    case = Case(w, step=0)
    dH = case.upstream_grad(case.seeds.size, w.hidden)
    ora = case.run_oracle(dH)
    gpu = case.run_gpu(dH)
    assert_blocks_equal(gpu["blocks"], ora["blocks"])
    _check_float(case, gpu, ora)


@pytest.mark.parametrize("dtype,d,fanouts", [("bf16", 512, (6, 4)), ("f32", 256, (3, 3, 3, 3)), ("f32", 768, (4, 3)),
                                             ("f32", 1024, (5,)), ("bf16", 1024, (4, 2))])
def test_widest_rows_and_four_hops(dtype, d, fanouts):
    """Rows of 1 024 to 4 096 bytes (several 16-byte chunks per lane, the large shared-memory form of the segment kernel;
    1024 values per row is the documented limit for both dtypes) and the largest number of hops the library takes."""
    base = S.WORKLOADS["medium_small"]
    w = S.Workload("wide", base.n_users, base.n_items, base.n_interactions, 1.2, 1.2, 1, d, d, dtype, fanouts, 48)
    case = Case(w, step=2)
    dH = case.upstream_grad(case.seeds.size, w.hidden)
    ora = case.run_oracle(dH)
    gpu = case.run_gpu(dH)
    assert_blocks_equal(gpu["blocks"], ora["blocks"])
    _check_float(case, gpu, ora)


# ----------------------------------------------------------------------------- LightGCN

@pytest.mark.parametrize("dtype,d", [("bf16", 64), ("f32", 32)])
def test_lightgcn_forward_and_adjoint(dtype, d):
    """Three propagation layers and the layer mean on a symmetric power-law graph with hubs and isolated nodes."""
    import paper_2511_20564_b200 as E
    n, m, L = 20_011, 300_000, 3
    a, b = S.powerlaw_directed(n, m, 1.1, 7)
    indptr, indices = S.coo_to_csr(n, np.concatenate([a, b]), np.concatenate([b, a]))
    deg = np.diff(indptr)
    assert deg.max() > 10_000 and (deg == 0).any()
    bf16 = dtype == "bf16"
    dt = torch.bfloat16 if bf16 else torch.float32
    H0 = S.normal_features(n, d, 8)
    G = S.normal_features(n, d, 8, stream=12)
    if bf16:
        H0, G = S.to_bf16_values(H0), S.to_bf16_values(G)
    s = np.where(deg > 0, 1.0 / np.sqrt(np.maximum(deg, 1)), 0.0).astype(np.float32)
    ip, ix, sd = torch.from_numpy(indptr).cuda(), torch.from_numpy(indices).cuda(), torch.from_numpy(s).cuda()
    Y, ws = E.lightgcn_forward(ip, ix, sd, L, torch.from_numpy(H0).cuda().to(dt))
    want = oracle.lightgcn_forward(indptr, indices, H0, L, bf16)
    # scale of the terms of one output: s_u * sqrt(sum_i s_i^2 h_i^2) per layer, bounded by the row norm of |H|
    rss = np.sqrt(oracle.lightgcn_propagate(indptr, indices, H0.astype(np.float64) ** 2)) if bf16 else None
    assert_close("lightgcn_forward", Y.float().cpu().numpy(), want, bf16, rss)
    # the graph is stored in both directions, so its CSC arrays are its CSR arrays
    dH0, _ = E.lightgcn_backward(ip, ix, sd, L, torch.from_numpy(G).cuda().to(dt), ws=ws)
    want = oracle.lightgcn_forward(indptr, indices, G, L, bf16)
    rss = np.sqrt(oracle.lightgcn_propagate(indptr, indices, G.astype(np.float64) ** 2)) if bf16 else None
    assert_close("lightgcn_backward", dH0.float().cpu().numpy(), want, bf16, rss)


def test_deferred_transposition_joins_before_use():
    """With the defer flag the csc arrays are complete after e2egrec_sample_join, and the backward pass joins by itself."""
    import paper_2511_20564_b200 as E
    w = S.WORKLOADS["medium_small"]
    case = Case(w, step=6)
    ora = case.run_oracle(case.upstream_grad(case.seeds.size, w.hidden))
    ip, ix = torch.from_numpy(case.indptr).cuda(), torch.from_numpy(case.indices).cuda()
    X = torch.from_numpy(case.X).cuda().to(torch.bfloat16)
    Ws = [torch.from_numpy(W).cuda().to(torch.bfloat16) for W in case.Ws]
    seeds = torch.from_numpy(case.seeds).cuda()
    blocks = E.Blocks(w.n_nodes, case.seeds.size, w.fanouts)
    g = torch.zeros(max(blocks.caps[0][0], 1), w.hidden, dtype=torch.bfloat16, device="cuda")
    g[: case.seeds.size] = torch.from_numpy(case.upstream_grad(case.seeds.size, w.hidden)).cuda().to(torch.bfloat16)
    for _ in range(2):                                       # the second round starts while nothing is pending
        E.sample_khop(ip, ix, seeds, blocks, w.seed, 6, defer_transpose=True)
        H, ctx = E.sage_forward(blocks, X, Ws)
        dWs, dX = E.sage_backward(blocks, X, Ws, ctx, g)     # joins the deferred work itself
        torch.cuda.synchronize()
        assert_blocks_equal(blocks.to_host(), ora["blocks"])
        n_src = ora["blocks"][-1]["n_src"]
        rss = reduction_rss(case, ora)
        for l, (a, b) in enumerate(zip(dWs, ora["dWs"])):
            assert_close(f"dW[{l}]", a.cpu().numpy(), b, True, rss["dW"][l] + 0 * b,
                         budget=relu_flip_budgets(case, ora, dict(layer_out=[h.float().cpu().numpy() for _, h in
                                                                             E.sage_ctx_views(blocks, X, Ws, ctx)]), 2e-2)[0][l])
    E.sample_khop(ip, ix, seeds, blocks, w.seed, 6, defer_transpose=True)
    E.sample_join()
    torch.cuda.synchronize()
    assert_blocks_equal(blocks.to_host(), ora["blocks"])


def test_deferred_transposition_is_joined_from_another_stream():
    """A transposition deferred on one stream is complete for a later-ordered stream once that stream has called
    e2egrec_sample_join (or the backward pass): the join covers everything deferred on the device."""
    import paper_2511_20564_b200 as E
    w = S.WORKLOADS["medium_small"]
    case = Case(w, step=7)
    ora = case.run_oracle()
    ip, ix = torch.from_numpy(case.indptr).cuda(), torch.from_numpy(case.indices).cuda()
    seeds = torch.from_numpy(case.seeds).cuda()
    blocks = E.Blocks(w.n_nodes, case.seeds.size, w.fanouts)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(3):
        with torch.cuda.stream(sa):
            E.sample_khop(ip, ix, seeds, blocks, w.seed, 7, defer_transpose=True)
        sb.wait_stream(sa)
        with torch.cuda.stream(sb):
            E.sample_join()
            snap = [{k: blocks.t[h][k].clone() for k in ("csc_ptr", "csc_row", "csc_eid", "csc_col")}
                    for h in range(len(w.fanouts))]
        sb.synchronize()
        for h, (got, o) in enumerate(zip(snap, ora["blocks"])):
            assert np.array_equal(got["csc_ptr"].cpu().numpy()[: o["n_src"] + 1], o["csc_ptr"])
            for k in ("csc_row", "csc_eid", "csc_col"):
                assert np.array_equal(got[k].cpu().numpy()[: o["n_edges"]], o[k]), f"hop {h}: {k}"
        sa.wait_stream(sb)


def test_sampling_of_the_next_batch_beside_the_current_step():
    """Two sets of block buffers and two streams, as bench.py runs the step: the forward/backward of batch i beside the
    sampling of batch i + 1.  Every step's outputs are bit-identical to the same steps run back to back."""
    import paper_2511_20564_b200 as E
    w = S.WORKLOADS["medium_small"]
    indptr_h, indices_h, _ = S.build_graph(w)
    X_h, Ws_h = S.build_model(w)
    dev = torch.device("cuda")
    indptr, indices = torch.from_numpy(indptr_h).to(dev), torch.from_numpy(indices_h).to(dev)
    X = torch.from_numpy(X_h).to(dev, torch.bfloat16)
    Ws = [torch.from_numpy(W).to(dev, torch.bfloat16) for W in Ws_h]
    n_steps = 4
    seeds = [torch.from_numpy(S.seed_batch(w.n_nodes, w.batch, w.seed, i)).to(dev) for i in range(n_steps + 1)]
    dH = torch.from_numpy(S.to_bf16_values(np.random.default_rng(5).standard_normal((w.batch, w.hidden)).astype(np.float32)))
    dH = dH.to(dev, torch.bfloat16)
    bufs = [E.Blocks(w.n_nodes, w.batch, w.fanouts, dev) for _ in range(2)]

    def compute(b):
        H, ctx = E.sage_forward(b, X, Ws)
        g = torch.zeros(H.shape, dtype=torch.bfloat16, device=dev)
        g[: w.batch] = dH
        dWs, dX = E.sage_backward(b, X, Ws, ctx, g)
        return [H.clone()] + [t.clone() for t in dWs] + [dX.clone(), b.counts.clone()]

    want = []
    for i in range(n_steps):
        E.sample_khop(indptr, indices, seeds[i], bufs[0], w.seed, i)
        want.append(compute(bufs[0]))
    torch.cuda.synchronize()

    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    got = []
    with torch.cuda.stream(s1):
        E.sample_khop(indptr, indices, seeds[0], bufs[0], w.seed, 0)
        for i in range(n_steps):
            s2.wait_stream(s1)
            with torch.cuda.stream(s2):
                E.sample_khop(indptr, indices, seeds[i + 1], bufs[(i + 1) & 1], w.seed, i + 1)
            got.append(compute(bufs[i & 1]))
            s1.wait_stream(s2)
    torch.cuda.synchronize()
    for i in range(n_steps):
        assert int(got[i][-1][:, 3].sum()) == 0
        for a, b in zip(got[i], want[i]):
            assert torch.equal(a, b), f"step {i}"


def test_three_stage_pipeline_sampling_transposition_compute():
    """Three sets of block buffers and three streams, as bench.py runs the step: the hops of batch i + 2, the transposed
    form of batch i + 1 (e2egrec_blocks_transpose) and the forward/backward of batch i side by side.  The blocks of
    the split path equal the oracle's bit for bit; every step's outputs are bit-identical to steps run back to back."""
    import paper_2511_20564_b200 as E
    w = S.WORKLOADS["medium_small"]
    case = Case(w, step=3)
    ora = case.run_oracle(case.upstream_grad(case.seeds.size, w.hidden))
    dev = torch.device("cuda")
    indptr, indices = torch.from_numpy(case.indptr).to(dev), torch.from_numpy(case.indices).to(dev)
    X = torch.from_numpy(case.X).to(dev, torch.bfloat16)
    Ws = [torch.from_numpy(W).to(dev, torch.bfloat16) for W in case.Ws]
    bufs = [E.Blocks(w.n_nodes, w.batch, w.fanouts, dev) for _ in range(3)]

    # the split path alone, against the oracle
    own = E.Blocks(w.n_nodes, case.seeds.size, w.fanouts, dev)
    E.sample_khop(indptr, indices, torch.from_numpy(case.seeds).to(dev), own, w.seed, 3, transpose=False)
    E.blocks_transpose(own)
    torch.cuda.synchronize()
    assert_blocks_equal(own.to_host(), ora["blocks"])

    n_steps = 5
    seeds = [torch.from_numpy(S.seed_batch(w.n_nodes, w.batch, w.seed, i)).to(dev) for i in range(n_steps + 2)]
    dH = torch.from_numpy(S.to_bf16_values(np.random.default_rng(5).standard_normal((w.batch, w.hidden)).astype(np.float32)))
    dH = dH.to(dev, torch.bfloat16)

    def compute(b):
        H, ctx = E.sage_forward(b, X, Ws)
        g = torch.zeros(H.shape, dtype=torch.bfloat16, device=dev)
        g[: w.batch] = dH
        dWs, dX = E.sage_backward(b, X, Ws, ctx, g)
        n_src, n_edges = int(b.counts[-1][1]), int(b.counts[-1][2])
        return [H.clone()] + [t.clone() for t in dWs] + [dX[:n_src].clone(), b.counts.clone()] + \
               [b.t[-1]["csc_row"][:n_edges].clone(), b.t[-1]["csc_ptr"][: n_src + 1].clone()]

    want = []
    for i in range(n_steps):
        E.sample_khop(indptr, indices, seeds[i], bufs[0], w.seed, i)
        want.append(compute(bufs[0]))
    torch.cuda.synchronize()

    s1, s2, s3 = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    got = []
    with torch.cuda.stream(s1):
        E.sample_khop(indptr, indices, seeds[0], bufs[0], w.seed, 0)
        E.sample_khop(indptr, indices, seeds[1], bufs[1], w.seed, 1, transpose=False)
        for i in range(n_steps):
            s2.wait_stream(s1)
            s3.wait_stream(s1)
            with torch.cuda.stream(s2):
                E.sample_khop(indptr, indices, seeds[i + 2], bufs[(i + 2) % 3], w.seed, i + 2, transpose=False)
            with torch.cuda.stream(s3):
                E.blocks_transpose(bufs[(i + 1) % 3])
            got.append(compute(bufs[i % 3]))
            s1.wait_stream(s2)
            s1.wait_stream(s3)
    torch.cuda.synchronize()
    for i in range(n_steps):
        assert int(got[i][-3][:, 3].sum()) == 0
        for a, b in zip(got[i], want[i]):
            assert torch.equal(a, b), f"step {i}"


# ----------------------------------------------------------------------------- weighted sampling

@pytest.mark.parametrize("beta", [0.0, 1.0, 2.5])
def test_weighted_sampling_is_bit_exact(beta):
    """Importance sampling p ~ q (Sec. 4.1): running sums built on the device, blocks against the oracle bit for bit;
    hubs (binary search over tens of thousands of running sums), short rows taken whole, rows of weight zero."""
    import paper_2511_20564_b200 as E
    w = S.WORKLOADS["medium_small"]
    indptr_h, indices_h, _ = S.build_graph(w)
    q = S.edge_weight_units(indptr_h, w.seed, beta)
    deg = np.diff(indptr_h)
    hub = int(np.argmax(deg))
    zero_row = int(np.flatnonzero(deg > 40)[3])
    q[indptr_h[zero_row]: indptr_h[zero_row + 1]] = 0           # sums to zero: drawn uniformly
    q[indptr_h[hub]: indptr_h[hub] + 5] = 0                      # entries that can never be drawn
    dev = torch.device("cuda")
    indptr, indices = torch.from_numpy(indptr_h).to(dev), torch.from_numpy(indices_h).to(dev)
    cum = E.edge_cumulate(indptr, torch.from_numpy(q.view(np.int32)).to(dev))
    want_cum = oracle.edge_cumulate(indptr_h, q)
    assert np.array_equal(cum.cpu().numpy().view(np.uint64), want_cum)
    seeds = np.unique(np.concatenate([S.seed_batch(w.n_nodes, 500, w.seed, 2), [hub, zero_row]])).astype(np.int32)
    blocks = E.Blocks(w.n_nodes, seeds.size, w.fanouts, dev)
    for step in (0, 9):
        E.sample_khop(indptr, indices, torch.from_numpy(seeds).to(dev), blocks, w.seed, step, edge_cum=cum)
        torch.cuda.synchronize()
        want = oracle.sample_khop(indptr_h, indices_h, seeds, w.fanouts, w.seed, step, edge_cum=want_cum)
        assert_blocks_equal(blocks.to_host(), want)
    if beta > 0:
        plain = oracle.sample_khop(indptr_h, indices_h, seeds, w.fanouts, w.seed, 9)
        assert not np.array_equal(plain[0]["nbr_global"], want[0]["nbr_global"])


# ----------------------------------------------------------------------------- LightGCN on sampled blocks

@pytest.mark.parametrize("dtype,d,fanouts", [("bf16", 128, (100,)), ("bf16", 64, (15, 10)), ("f32", 32, (10, 5, 3))])
def test_lightgcn_on_sampled_blocks_forward_and_adjoint(dtype, d, fanouts):
    """Eqs. 4-7 on the sampled sub-graph (one hop x 100 is the paper's default shape): Y on the seeds and the gradient
    with respect to the gathered feature rows, hubs and isolated seeds included."""
    import paper_2511_20564_b200 as E
    base = S.WORKLOADS["medium_small"]
    indptr_h, indices_h, _ = S.build_graph(base)
    n = base.n_nodes
    deg = np.diff(indptr_h)
    bf16 = dtype == "bf16"
    dt = torch.bfloat16 if bf16 else torch.float32
    X_h = S.normal_features(n, d, 31)
    if bf16:
        X_h = S.to_bf16_values(X_h)
    s_h = np.where(deg > 0, 1.0 / np.sqrt(np.maximum(deg, 1)), 0.0).astype(np.float32)
    seeds = np.unique(np.concatenate([S.seed_batch(n, 700, base.seed, 4), [int(np.argmax(deg))],
                                      np.flatnonzero(deg == 0)[:3]])).astype(np.int32)
    dev = torch.device("cuda")
    indptr, indices = torch.from_numpy(indptr_h).to(dev), torch.from_numpy(indices_h).to(dev)
    blocks = E.Blocks(n, seeds.size, fanouts, dev)
    E.sample_khop(indptr, indices, torch.from_numpy(seeds).to(dev), blocks, base.seed, 3)
    X = torch.from_numpy(X_h).to(dev, dt)
    Y, ctx = E.lightgcn_sampled_forward(blocks, X, torch.from_numpy(s_h).to(dev))
    dY_h = np.random.default_rng(8).standard_normal((seeds.size, d)).astype(np.float32)
    if bf16:
        dY_h = S.to_bf16_values(dY_h)
    dY = torch.zeros(Y.shape, dtype=dt, device=dev)
    dY[: seeds.size] = torch.from_numpy(dY_h).to(dev, dt)
    dX, _ = E.lightgcn_sampled_backward(blocks, ctx, dY)
    torch.cuda.synchronize()

    ora_blocks = oracle.sample_khop(indptr_h, indices_h, seeds, fanouts, base.seed, 3)
    assert_blocks_equal(blocks.to_host(), ora_blocks)
    want_Y, octx = oracle.lightgcn_sampled_forward(ora_blocks, X_h, s_h, bf16)
    want_dX = oracle.lightgcn_sampled_backward(ora_blocks, octx, dY_h, bf16)
    # scale of the terms behind an element: the same maps applied to the squares, with squared scales
    s2 = (s_h.astype(np.float64) ** 2).astype(np.float32)
    rssY = rssX = None
    if bf16:
        sq_blocks = ora_blocks
        Y2, c2 = oracle.lightgcn_sampled_forward(sq_blocks, X_h.astype(np.float64) ** 2, s_h)
        rssY = np.sqrt(np.abs(Y2)) + np.abs(want_Y)
        rssX = np.sqrt(np.abs(oracle.lightgcn_sampled_backward(sq_blocks, c2, dY_h.astype(np.float64) ** 2))) + np.abs(want_dX)
    assert_close("lightgcn sampled forward", Y[: seeds.size].float().cpu().numpy(), want_Y, bf16, rssY)
    n_src = ora_blocks[-1]["n_src"]
    assert_close("lightgcn sampled backward", dX[:n_src].float().cpu().numpy(), want_dX, bf16, rssX)
