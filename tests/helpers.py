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


def encoder_rss(Ws, acts, blocks, ctx, trace=None):
    """Root-sum-square of the terms of the last reduction behind every compared output of the encoder, from oracle
    tensors: forward output, and (given the trace of gradients that arrived at each layer) dW per layer, dX rows."""
    L = len(Ws)
    acts = [1] * L if acts is None else acts
    out = {}
    n0 = blocks[0]["n_dst"]
    cat_top = np.concatenate([ctx["H"][L - 1][:n0], ctx["agg"][L - 1]], axis=1)
    out["forward"] = np.sqrt((cat_top ** 2) @ (np.asarray(Ws[L - 1], np.float64) ** 2).T)
    if trace is None:
        return out
    out["dW"] = []
    for l in range(L):
        blk = blocks[L - 1 - l]
        n_dst = blk["n_dst"]
        dZ = trace[l] * ((ctx["H"][l + 1] > 0) if acts[l] else 1.0)
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


def reduction_rss(case, ora):
    """encoder_rss for a Case and its oracle run."""
    return encoder_rss(case.Ws, case.acts, ora["blocks"], ora["ctx"], ora.get("trace"))


def plain_tolerance(want, bf16):
    """The tolerance as first stated for the two paths, before any allowance: fp32 |a-b| <= 1e-5 max(|b|, rms(b));
    bf16 storage |a-b| <= 1e-3 + 2e-2 |b|."""
    want = np.asarray(want, np.float64)
    if bf16:
        return 1e-3 + 2e-2 * np.abs(want)
    return 1e-5 * np.maximum(np.abs(want), np.sqrt(np.mean(want ** 2)) if want.size else 0.0)


# One record per compared tensor: how many elements needed more than the plain tolerance (with the ReLU-flip budget
# where the test has one, but without the terms-scale or the outlier allowance) and by how much.  conftest.py prints
# the table at the end of the session and writes it to $E2EGREC_PARITY_AUDIT.
AUDIT = []
# ceilings on what may need the allowances at all: share of a tensor's elements (index: bf16?), and the worst ratio
# error / plain tolerance.  Measured on B200: bf16 weight gradients (sums over thousands of rows whose operands the two
# sides stored one bf16 step apart here and there) reach 1.1e-3 of their elements and 12x; everything fp32 stays below
# 5e-6 of the elements and 5x.
AUDIT_MAX_SHARE = {True: 2e-3, False: 1e-4}
AUDIT_MAX_RATIO = {True: 16.0, False: 8.0}


def _audit(name, err, plain, bf16, budget):
    import os
    over = err > plain
    share = float(over.mean())
    ratio = float((err[over] / plain[over]).max()) if over.any() else 0.0
    AUDIT.append(dict(test=os.environ.get("PYTEST_CURRENT_TEST", "").split(" ")[0], tensor=name, dtype="bf16" if bf16 else "f32",
                      elements=int(err.size), outside_plain=int(over.sum()), share=share, worst_ratio=ratio,
                      flip_budget=budget is not None))
    return share, ratio


def assert_close(name, got, want, bf16, terms_rss=None, budget=None, audit_share=None):
    """Element-wise tolerance check with a report of the worst element.

    Every element within tolerance(); on the bf16 path at most 1e-4 of the elements may miss it by up
    to 4x (a stored operand one bf16 step apart two layers up, which the last reduction's terms do
    not see).  Before either allowance is applied the elements outside plain_tolerance() are counted,
    recorded (AUDIT) and held to a ceiling: a small share of the tensor, each within a fixed multiple
    of the plain tolerance, so a widened tolerance cannot hide a wrong row or a mis-scaled column.
    """
    want = np.asarray(want, np.float64)
    got = np.asarray(got, np.float64)
    assert got.shape == want.shape, f"{name}: shape {got.shape} vs {want.shape}"
    if want.size == 0:
        return
    assert np.isfinite(got).all(), f"{name}: non-finite values"
    tol = tolerance(want, bf16, terms_rss)
    plain = plain_tolerance(want, bf16)
    if budget is not None:
        tol = tol + 1.05 * budget
        plain = plain + 1.05 * budget
    err = np.abs(got - want)
    share, ratio = _audit(name, err, plain, bf16, budget)
    note = f"{name}: {share:.2e} of {err.size} elements outside the plain tolerance, worst {ratio:.2f}x"
    assert share <= (audit_share or AUDIT_MAX_SHARE[bf16]) or (err > plain).sum() <= 2, note
    assert ratio <= AUDIT_MAX_RATIO[bf16], note
    bad = err > tol
    if not bad.any():
        return
    i = np.unravel_index(np.argmax(err / np.maximum(tol, 1e-300)), err.shape)
    msg = (f"{name}: {bad.sum()} of {bad.size} outside tolerance; worst at {i}: got {got[i]!r} want {want[i]!r} "
           f"err {err[i]:.3e} tol {tol[i]:.3e}; {note}")
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


def encoder_flip_budgets(Ws, acts, blocks, ctx, trace, gpu_layer_out, tau, B_dH0=None):
    """Upper bounds on how far the encoder's gradients may differ because the two sides took a ReLU decision
    differently.

    The derivative of ReLU is decided by the sign of a sum that the GPU forms in fp32 and the oracle in
    float64 (from inputs that may already sit one bf16 step apart), so for pre-activations within `tau`
    of zero the stored masks can differ; both gradients are then valid sub-gradients.  A flipped element
    (i, o) of layer l changes dZ_l[i, o] by at most |dH[i, o]|; that bound is pushed through the same
    linear adjoint with absolute-valued operands.  Flips are only accepted where the oracle's
    pre-activation is within tau of the kink; everything a flip cannot reach keeps the strict tolerance.
    B_dH0: bound on the difference of the gradient that arrives at the encoder output (zero by default).
    Returns (budget_dW list, budget_dX).
    """
    L = len(Ws)
    acts = [1] * L if acts is None else acts
    B_dH = np.zeros_like(trace[L - 1]) if B_dH0 is None else np.asarray(B_dH0, np.float64)
    B_dW = [None] * L
    for l in range(L - 1, -1, -1):
        blk = blocks[L - 1 - l]
        n_dst, n_src = blk["n_dst"], blk["n_src"]
        flips = np.zeros(ctx["Z"][l].shape, bool)
        if acts[l]:
            flips = (ctx["H"][l + 1] > 0) != (gpu_layer_out[l][:n_dst] > 0)
            assert (np.abs(ctx["Z"][l][flips]) <= tau).all(), \
                f"layer {l}: ReLU decision differs where the pre-activation is not near zero"
        B_dZ = B_dH[:n_dst] + np.abs(trace[l]) * flips
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


def relu_flip_budgets(case, ora, gpu, tau):
    """encoder_flip_budgets for a Case, its oracle run and the GPU's stored layer outputs."""
    return encoder_flip_budgets(case.Ws, case.acts, ora["blocks"], ora["ctx"], ora["trace"], gpu["layer_out"], tau)


def joint_rss_and_budgets(ora, W_gnn, W_tower, b_tower, gpu_act, tau, acts=1, gate=None):
    """For a joint step (oracle result `ora` with its trace; gpu_act = the GPU's stored activations a1, a2 and encoder
    layer outputs): per compared tensor the root-sum-square of the terms of its last reduction and the ReLU-flip
    budget, pushed from the tower's two hidden layers through the pair -> seed sum into the encoder.
    Returns (rss, budget): dicts with logits, dW_t, db_t (lists), dW_g (list), dX, and dW_gate / db_gate with a gate."""
    tr = ora["trace"]
    W1, W2, W3 = (np.asarray(W, np.float64) for W in W_tower[:3])
    b1, b2 = (np.zeros(W.shape[0]) if b is None else np.asarray(b, np.float64) for W, b in zip((W1, W2), b_tower[:2]))
    zf, a1, a2, z = tr["zf"], tr["a1"], tr["a2"], tr["z"]
    P = zf.shape[0]
    m2 = (a2 > 0) if acts else np.ones_like(a2, bool)
    m1 = (a1 > 0) if acts else np.ones_like(a1, bool)
    dz2, dz1 = tr["da2"] * m2, tr["da1"] * m1
    # a logit sums 'a2 * W3' terms; a2 itself already carries the one-step deviations of a1 through its own sum, so the
    # scale of a logit's terms takes the terms of a2's reduction along (where a2 is active)
    rss_a2 = np.sqrt((a1 ** 2) @ (W2 ** 2).T) * m2
    rss = dict(logits=np.sqrt((a2 ** 2 + rss_a2 ** 2) @ (W3 ** 2).T)[:, 0],
               dW_t=[np.sqrt((dz1 ** 2).T @ (zf ** 2)), np.sqrt((dz2 ** 2).T @ (a1 ** 2)), np.sqrt((tr["dt"] ** 2)[None, :] @ (a2 ** 2))],
               db_t=[np.sqrt((dz1 ** 2).sum(0)), np.sqrt((dz2 ** 2).sum(0)), np.sqrt((tr["dt"] ** 2).sum(keepdims=True))])
    f2 = np.zeros_like(m2)
    f1 = np.zeros_like(m1)
    if acts:
        f2 = m2 != (gpu_act["a2"][:P] > 0)
        f1 = m1 != (gpu_act["a1"][:P] > 0)
        assert (np.abs(a1 @ W2.T + b2)[f2] <= tau).all(), "tower layer 2: ReLU decision differs away from the kink"
        assert (np.abs(zf @ W1.T + b1)[f1] <= tau).all(), "tower layer 1: ReLU decision differs away from the kink"
    B_dz2 = np.abs(tr["da2"]) * f2
    B_dz1 = B_dz2 @ np.abs(W2) + np.abs(tr["da1"]) * f1
    B_dzf = B_dz1 @ np.abs(W1)
    bud = dict(logits=None, dW_t=[B_dz1.T @ np.abs(zf), B_dz2.T @ np.abs(a1), np.zeros_like(W3)],
               db_t=[B_dz1.sum(0), B_dz2.sum(0), np.zeros(1)])
    B_dz = B_dzf
    if gate is not None:
        Wg = np.asarray(gate[0], np.float64)
        g = tr["gate"]
        dpre = tr["dzf"] * z * g * (1.0 - g)
        rss["dW_gate"], rss["db_gate"] = np.sqrt((dpre ** 2).T @ (z ** 2)), np.sqrt((dpre ** 2).sum(0))
        B_dpre = B_dzf * np.abs(z) * g * (1.0 - g)
        bud["dW_gate"], bud["db_gate"] = B_dpre.T @ np.abs(z), B_dpre.sum(0)
        B_dz = B_dzf * g + B_dpre @ np.abs(Wg)
    dL = ora["H"].shape[1]
    B_dH = np.zeros_like(ora["H"])
    np.add.at(B_dH, tr["pos_u"], B_dz[:, :dL])
    np.add.at(B_dH, tr["pos_i"], B_dz[:, dL:2 * dL])
    enc_acts = [acts] * len(W_gnn)
    enc = encoder_rss(W_gnn, enc_acts, ora["blocks"], tr["ctx"], tr["enc"])
    rss["dW_g"], rss["dX"] = enc["dW"], enc["dX"]
    bud["dW_g"], bud["dX"] = encoder_flip_budgets(W_gnn, enc_acts, ora["blocks"], tr["ctx"], tr["enc"], gpu_act["enc"], tau, B_dH)
    return rss, bud


def assert_close_budget(name, got, want, budget, bf16, terms_rss=None):
    """Tolerance of assert_close widened, per element, by the allowance of relu_flip_budgets."""
    assert_close(name, got, want, bf16, terms_rss=terms_rss, budget=budget)
