"""Shared pieces of the GPU parity tests: tolerances, comparisons, running both sides."""
import numpy as np
import torch

import oracle
import synth_inputs as S


def close_f32(got, want, rel=1e-5):
    """fp32 path against the float64 oracle: |a-b| <= rel * max(|b|, rms(b))."""
    want = np.asarray(want, np.float64)
    got = np.asarray(got, np.float64)
    scale = np.sqrt(np.mean(want ** 2)) if want.size else 0.0
    bad = np.abs(got - want) > rel * np.maximum(np.abs(want), scale)
    return bad


def close_bf16(got, want, rel=2e-2, abs_=1e-3):
    """bf16-storage path: |a-b| <= 1e-3 + 2e-2 |b|."""
    want = np.asarray(want, np.float64)
    got = np.asarray(got, np.float64)
    return np.abs(got - want) > abs_ + rel * np.abs(want)


BF16_STEP = 2.0 ** -8


def tolerance(want, bf16, terms_rss=None):
    """Per-element tolerance.

    fp32 path: 1e-5 * max(|b|, rms(b), root-sum-square of the terms of the element's last reduction):
    a long fp32 sum with cancellation is accurate relative to the scale of its terms, not of its result.
    bf16 path: 1e-3 + 2e-2 |b| + 2^-8 * sqrt(sum of squared terms of the element's last reduction).
    The last part covers operands that the two sides stored one bf16 step apart (a value within fp32
    rounding of the midpoint of two bf16 neighbours rounds differently after an fp32 or a float64 sum).
    If every operand were off by a step the bound would be 2^-8 * sum|terms|; the root-sum-square is the
    smaller, statistical form of it and still dominates the effect of any single such operand.
    """
    want = np.asarray(want, np.float64)
    if not bf16:
        scale = np.maximum(np.abs(want), np.sqrt(np.mean(want ** 2)) if want.size else 0.0)
        if terms_rss is not None:
            scale = np.maximum(scale, terms_rss)
        return 1e-5 * scale
    tol = 1e-3 + 2e-2 * np.abs(want)
    if terms_rss is not None:
        tol = tol + BF16_STEP * terms_rss
    return tol


def reduction_rss(case, ora):
    """Root-sum-square of the terms of the last reduction behind every compared output, from oracle tensors:
    forward output, dW per layer, dX rows."""
    Ws, blocks, ctx, L = case.Ws, ora["blocks"], ora["ctx"], len(case.Ws)
    acts = [1] * L if case.acts is None else case.acts
    out = {}
    n0 = blocks[0]["n_dst"]
    cat_top = np.concatenate([ctx["H"][L - 1][:n0], ctx["agg"][L - 1]], axis=1)
    out["forward"] = np.sqrt((cat_top ** 2) @ (np.asarray(Ws[L - 1], np.float64) ** 2).T)
    if "trace" not in ora:
        return out
    out["dW"] = []
    for l in range(L):
        blk = blocks[L - 1 - l]
        n_dst = blk["n_dst"]
        dZ = ora["trace"][l] * ((ctx["H"][l + 1] > 0) if acts[l] else 1.0)
        cat = np.concatenate([ctx["H"][l][:n_dst], ctx["agg"][l]], axis=1)
        out["dW"].append(np.sqrt((dZ ** 2).T @ (cat ** 2)))
        if l == 0:
            W = np.asarray(Ws[0], np.float64)
            d_in = W.shape[1] // 2
            dCat = dZ @ W
            cnt = np.maximum(np.diff(blk["indptr"]), 1).astype(np.float64)[:, None]
            sq_self = np.ascontiguousarray(dCat[:, :d_in] ** 2)
            sq_agg = np.ascontiguousarray(dCat[:, d_in:] ** 2 / cnt)      # the adjoint divides by cnt once more
            S2 = np.zeros((blk["n_src"], d_in))
            ip = blk["indptr"].astype(np.int64)
            oracle.lib().oracle_mean_aggregate_backward(
                oracle._p(ip), oracle._p(blk["col"]), oracle.C.c_int64(n_dst), oracle.C.c_int64(blk["n_src"]),
                oracle._p(sq_self), oracle._p(sq_agg), oracle.C.c_int32(d_in), oracle._p(S2), oracle.C.c_int(0))
            out["dX"] = np.sqrt(S2)
    return out


def assert_close(name, got, want, bf16, terms_rss=None, budget=None):
    """Element-wise tolerance check with a report of the worst element.

    Every element within tolerance(); on the bf16 path at most 1e-4 of the elements may miss it by up
    to 4x (a stored operand one bf16 step apart two layers up, which the last reduction's terms do
    not see).
    """
    want = np.asarray(want, np.float64)
    got = np.asarray(got, np.float64)
    assert got.shape == want.shape, f"{name}: shape {got.shape} vs {want.shape}"
    if want.size == 0:
        return
    assert np.isfinite(got).all(), f"{name}: non-finite values"
    tol = tolerance(want, bf16, terms_rss)
    if budget is not None:
        tol = tol + 1.05 * budget
    err = np.abs(got - want)
    bad = err > tol
    if not bad.any():
        return
    i = np.unravel_index(np.argmax(err / np.maximum(tol, 1e-300)), err.shape)
    msg = (f"{name}: {bad.sum()} of {bad.size} outside tolerance; worst at {i}: got {got[i]!r} want {want[i]!r} "
           f"err {err[i]:.3e} tol {tol[i]:.3e}")
    if bf16 and bad.sum() <= max(1, int(1e-4 * bad.size)) and (err <= 4 * tol).all():
        return
    raise AssertionError(msg)


def assert_blocks_equal(gpu_blocks, ora_blocks):
    assert len(gpu_blocks) == len(ora_blocks)
    for h, (g, o) in enumerate(zip(gpu_blocks, ora_blocks)):
        assert g["status"] == 0, f"hop {h}: device status {g['status']}"
        for k in ("n_dst", "n_src", "n_edges"):
            assert g[k] == o[k], f"hop {h}: {k} {g[k]} != {o[k]}"
        for k in ("indptr", "nbr_global", "src_nodes", "col", "csc_ptr", "csc_row", "csc_eid", "csc_col"):
            assert np.array_equal(g[k], o[k]), f"hop {h}: {k} differs"
        assert np.array_equal(g["inv_cnt"].view(np.uint32), o["inv_cnt"].view(np.uint32)), f"hop {h}: inv_cnt"


def torch_dtype(name):
    return torch.bfloat16 if name == "bf16" else torch.float32


class Case:
    """A graph + model + batch on both sides."""

    def __init__(self, w: S.Workload, step=0, seeds=None, graph=None, acts=None):
        self.w = w
        self.acts = acts
        self.indptr, self.indices = graph if graph is not None else S.build_graph(w)[:2]
        self.X, self.Ws = S.build_model(w)
        self.seeds = S.seed_batch(w.n_nodes, w.batch, w.seed, step) if seeds is None else np.asarray(seeds, np.int32)
        self.step = step
        self.bf16 = w.dtype == "bf16"

    def run_oracle(self, dH=None):
        blocks = oracle.sample_khop(self.indptr, self.indices, self.seeds, self.w.fanouts, self.w.seed, self.step)
        out, ctx = oracle.sage_forward(blocks, self.X, self.Ws, acts=self.acts, bf16=self.bf16)
        res = dict(blocks=blocks, out=out, ctx=ctx)
        if dH is not None:
            res["trace"] = []
            res["dWs"], _, res["dX"] = oracle.sage_backward(blocks, ctx, self.Ws, dH, acts=self.acts, bf16=self.bf16,
                                                            trace=res["trace"])
        return res

    def upstream_grad(self, n_rows, d):
        g = np.random.default_rng(1234 + self.step).standard_normal((n_rows, d)).astype(np.float32)
        return S.to_bf16_values(g) if self.bf16 else g

    def run_gpu(self, dH=None, cap_seeds=None):
        import paper_2511_20564_b200 as E
        dev = "cuda"
        dt = torch_dtype(self.w.dtype)
        indptr = torch.from_numpy(self.indptr).to(dev)
        indices = torch.from_numpy(self.indices).to(dev)
        X = torch.from_numpy(self.X).to(dev, dt)
        Ws = [torch.from_numpy(W).to(dev, dt) for W in self.Ws]
        seeds = torch.from_numpy(self.seeds).to(dev)
        blocks = E.Blocks(self.w.n_nodes, cap_seeds or self.seeds.size, self.w.fanouts, dev)   # capacity may exceed the batch
        E.sample_khop(indptr, indices, seeds, blocks, self.w.seed, self.step)
        H, ctx = E.sage_forward(blocks, X, Ws, acts=self.acts)
        res = dict(blocks_obj=blocks, H=H, ctx=ctx)
        if dH is not None:
            g = torch.zeros(H.shape, dtype=dt, device=dev)
            g[: dH.shape[0]] = torch.from_numpy(dH).to(dev, dt)
            dWs, dX = E.sage_backward(blocks, X, Ws, ctx, g, acts=self.acts)
            res["dWs"] = [w.float().cpu().numpy() for w in dWs]
            res["dX"] = dX.float().cpu().numpy()
        torch.cuda.synchronize()
        res["blocks"] = blocks.to_host()
        res["out"] = H.float().cpu().numpy()
        res["layer_out"] = [h.float().cpu().numpy() for _, h in E.sage_ctx_views(blocks, X, Ws, ctx)]
        return res


def relu_flip_budgets(case, ora, gpu, tau):
    """Upper bounds on how far the gradients may differ because the two sides took a ReLU decision
    differently.

    The derivative of ReLU is decided by the sign of a sum that the GPU forms in fp32 and the oracle in
    float64 (from inputs that may already sit one bf16 step apart), so for pre-activations within `tau`
    of zero the stored masks can differ; both gradients are then valid sub-gradients.  A flipped element
    (i, o) of layer l changes dZ_l[i, o] by at most |dH[i, o]|; that bound is pushed through the same
    linear adjoint with absolute-valued operands.  Flips are only accepted where the oracle's
    pre-activation is within tau of the kink; everything a flip cannot reach keeps the strict tolerance.
    Returns (budget_dW list, budget_dX).
    """
    Ws, blocks, ctx = case.Ws, ora["blocks"], ora["ctx"]
    L = len(Ws)
    acts = [1] * L if case.acts is None else case.acts
    B_dH = np.zeros_like(ora["trace"][L - 1])
    B_dW = [None] * L
    for l in range(L - 1, -1, -1):
        blk = blocks[L - 1 - l]
        n_dst, n_src = blk["n_dst"], blk["n_src"]
        flips = np.zeros(ctx["Z"][l].shape, bool)
        if acts[l]:
            flips = (ctx["H"][l + 1] > 0) != (gpu["layer_out"][l][:n_dst] > 0)
            assert (np.abs(ctx["Z"][l][flips]) <= tau).all(), \
                f"layer {l}: ReLU decision differs where the pre-activation is not near zero"
        B_dZ = B_dH + np.abs(ora["trace"][l]) * flips
        W = np.abs(np.asarray(Ws[l], np.float64))
        d_in = W.shape[1] // 2
        cat = np.abs(np.concatenate([ctx["H"][l][:n_dst], ctx["agg"][l]], axis=1))
        B_dW[l] = B_dZ.T @ cat
        B_dCat = B_dZ @ W
        B_dSelf = np.ascontiguousarray(B_dCat[:, :d_in])
        B_dAgg = np.ascontiguousarray(B_dCat[:, d_in:])
        B_dH = np.zeros((n_src, d_in))
        ip = blk["indptr"].astype(np.int64)
        oracle.lib().oracle_mean_aggregate_backward(
            oracle._p(ip), oracle._p(blk["col"]), oracle.C.c_int64(n_dst), oracle.C.c_int64(n_src),
            oracle._p(B_dSelf), oracle._p(B_dAgg), oracle.C.c_int32(d_in), oracle._p(B_dH), oracle.C.c_int(0))
    return B_dW, B_dH


def assert_close_budget(name, got, want, budget, bf16, terms_rss=None):
    """Tolerance of assert_close widened, per element, by the allowance of relu_flip_budgets."""
    assert_close(name, got, want, bf16, terms_rss=terms_rss, budget=budget)
