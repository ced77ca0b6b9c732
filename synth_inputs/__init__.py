"""Seeded synthetic inputs: power-law bipartite graphs, features, weights, batches.

This module only *draws inputs*.  It holds none of the method's arithmetic (no
sampling of neighbourhoods, no aggregation, no transforms): both the CUDA path
and the CPU oracle are handed the arrays made here, and neither imports it.

The graphs stand in for the production user-item / item-item graphs of the
paper's experiments (Sec. 4.1 and Sec. 5.1), which are not public: bipartite
interaction lists whose endpoint popularity follows a bounded Zipf(-Mandelbrot)
law, stored in both directions, users numbered first and items after them.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def zipf_ranks(rng: np.random.Generator, size: int, n: int, alpha: float, q: float = 0.0) -> np.ndarray:
    """Ranks in [0, n) with P(rank r) ~ (r + 1 + q)^-alpha (continuous inverse CDF, floored)."""
    u = rng.random(size)
    if abs(alpha - 1.0) < 1e-12:
        lo, hi = np.log(1.0 + q), np.log(n + 1.0 + q)
        r = np.exp(lo + u * (hi - lo)) - q
    else:
        e = 1.0 - alpha
        lo, hi = (1.0 + q) ** e, (n + 1.0 + q) ** e
        r = (lo + u * (hi - lo)) ** (1.0 / e) - q
    r = np.floor(r).astype(np.int64) - 1
    return np.clip(r, 0, n - 1)


def bipartite_interactions(n_users: int, n_items: int, m: int, alpha_user, alpha_item, seed: int,
                           q: float = 0.0, chunk: int = 1 << 24):
    """m (user, item) interactions; ids are global: users [0, U), items [U, U+I).

    alpha None means uniform.  A random permutation scatters the popular ranks over
    the id space so that hubs are not the low ids.
    """
    perm_u = _rng(seed, 1).permutation(n_users).astype(np.int32)
    perm_i = _rng(seed, 2).permutation(n_items).astype(np.int32)
    ru, ri = _rng(seed, 3), _rng(seed, 4)
    users = np.empty(m, np.int32)
    items = np.empty(m, np.int32)
    for s in range(0, m, chunk):
        e = min(m, s + chunk)
        if alpha_user is None:
            ku = ru.integers(0, n_users, e - s)
        else:
            ku = zipf_ranks(ru, e - s, n_users, alpha_user, q)
        if alpha_item is None:
            ki = ri.integers(0, n_items, e - s)
        else:
            ki = zipf_ranks(ri, e - s, n_items, alpha_item, q)
        users[s:e] = perm_u[ku]
        items[s:e] = perm_i[ki] + n_users
    return users, items


def undirected_coo(users: np.ndarray, items: np.ndarray):
    """Both directions of every interaction; multi-edges are kept."""
    row = np.concatenate([users, items])
    col = np.concatenate([items, users])
    return row, col


def powerlaw_directed(n: int, m: int, alpha: float, seed: int):
    """m directed (dst, src) entries with both endpoints Zipf(alpha) over permuted ids."""
    perm = _rng(seed, 1).permutation(n).astype(np.int32)
    dst = perm[zipf_ranks(_rng(seed, 2), m, n, alpha)]
    perm2 = _rng(seed, 5).permutation(n).astype(np.int32)
    src = perm2[zipf_ranks(_rng(seed, 3), m, n, alpha)]
    return dst, src


def coo_to_csr(n: int, row: np.ndarray, col: np.ndarray):
    """Canonical CSR of a COO list: entries ordered by (row, col), duplicates kept."""
    order = np.lexsort((col, row))
    indices = np.ascontiguousarray(col[order], dtype=np.int32)
    counts = np.bincount(row, minlength=n).astype(np.int64)
    indptr = np.zeros(n + 1, np.int64)
    np.cumsum(counts, out=indptr[1:])
    return indptr, indices


def normal_features(n: int, d: int, seed: int, stream: int = 10) -> np.ndarray:
    return _rng(seed, stream).standard_normal((n, d), dtype=np.float32)


def glorot_uniform(d_out: int, d_in: int, seed: int, stream: int) -> np.ndarray:
    lim = np.sqrt(6.0 / (d_in + d_out))
    return _rng(seed, stream).uniform(-lim, lim, (d_out, d_in)).astype(np.float32)


def seed_batch(n: int, batch: int, seed: int, step: int) -> np.ndarray:
    """`batch` distinct node ids, uniform over all nodes, for training step `step`."""
    return _rng(seed, 1000 + step).choice(n, size=batch, replace=False).astype(np.int32)


def seed_batch_from_interactions(users: np.ndarray, items: np.ndarray, batch: int, seed: int, step: int) -> np.ndarray:
    """`batch` distinct node ids met as endpoints of uniformly drawn interactions (users and items in
    turn), so that a node enters a batch in proportion to its activity, as the source nodes of a
    training example stream do."""
    rng = _rng(seed, 2000 + step)
    m = users.size
    got = np.zeros(0, np.int32)
    while got.size < batch:
        idx = rng.integers(0, m, 4 * batch)
        cand = np.empty(2 * idx.size, np.int32)
        cand[0::2] = users[idx]
        cand[1::2] = items[idx]
        got = first_distinct(np.concatenate([got, cand]), len(got) + cand.size)
    return np.ascontiguousarray(got[:batch])


def first_distinct(cand: np.ndarray, batch: int) -> np.ndarray:
    """The first `batch` distinct values of `cand`, in order of first appearance (fewer if there are not enough)."""
    _, first = np.unique(cand, return_index=True)
    return np.ascontiguousarray(cand[np.sort(first)][:batch])


# ----------------------------------------------------------------------------- generation on a device
# The largest workload (10^9 interactions) is drawn with torch on the device that will hold the graph: the host
# arrays alone would take tens of GB and minutes.  Same law as bipartite_interactions, torch's generator
# instead of numpy's, so the two are different (equally valid) graphs of the same shape.

def _torch_gen(device, seed: int, stream: int):
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) * 1_000_003 + int(stream))
    return g


def zipf_ranks_device(gen, size: int, n: int, alpha: float, q: float, device):
    """Device version of zipf_ranks: int64 tensor of ranks in [0, n)."""
    import torch
    u = torch.rand(size, dtype=torch.float64, device=device, generator=gen)
    if abs(alpha - 1.0) < 1e-12:
        lo, hi = np.log(1.0 + q), np.log(n + 1.0 + q)
        r = torch.exp(lo + u * (hi - lo)) - q
    else:
        e = 1.0 - alpha
        lo, hi = (1.0 + q) ** e, (n + 1.0 + q) ** e
        r = torch.pow(lo + u * (hi - lo), 1.0 / e) - q
    return (torch.floor(r).to(torch.int64) - 1).clamp_(0, n - 1)


def bipartite_interactions_device(n_users: int, n_items: int, m: int, alpha_user, alpha_item, seed: int,
                                  q: float, device, chunk: int = 1 << 26):
    """m (user, item) interactions as int32 tensors on `device`; ids are global as in bipartite_interactions."""
    import torch
    perm_u = torch.randperm(n_users, device=device, generator=_torch_gen(device, seed, 1)).to(torch.int32)
    perm_i = torch.randperm(n_items, device=device, generator=_torch_gen(device, seed, 2)).to(torch.int32)
    gu, gi = _torch_gen(device, seed, 3), _torch_gen(device, seed, 4)
    users = torch.empty(m, dtype=torch.int32, device=device)
    items = torch.empty(m, dtype=torch.int32, device=device)
    for s in range(0, m, chunk):
        e = min(m, s + chunk)
        if alpha_user is None:
            ku = torch.randint(0, n_users, (e - s,), device=device, generator=gu)
        else:
            ku = zipf_ranks_device(gu, e - s, n_users, alpha_user, q, device)
        if alpha_item is None:
            ki = torch.randint(0, n_items, (e - s,), device=device, generator=gi)
        else:
            ki = zipf_ranks_device(gi, e - s, n_items, alpha_item, q, device)
        users[s:e] = perm_u[ku]
        items[s:e] = perm_i[ki] + n_users
    return users, items


def normal_features_device(n: int, d: int, seed: int, dtype, device, stream: int = 10, chunk_rows: int = 1 << 22):
    """N(0,1) features drawn on the device in `dtype` (chunked, so that no fp32 copy of the table exists)."""
    import torch
    g = _torch_gen(device, seed, stream)
    X = torch.empty(n, d, dtype=dtype, device=device)
    for s in range(0, n, chunk_rows):
        e = min(n, s + chunk_rows)
        X[s:e] = torch.randn(e - s, d, dtype=torch.float32, device=device, generator=g).to(dtype)
    return X


def seed_batch_from_interactions_device(users, items, batch: int, seed: int, step: int) -> np.ndarray:
    """seed_batch_from_interactions for interaction lists that live on a device (torch tensors)."""
    import torch
    rng = _rng(seed, 2000 + step)
    m = users.numel()
    got = np.zeros(0, np.int32)
    while got.size < batch:
        idx = torch.from_numpy(rng.integers(0, m, 4 * batch)).to(users.device)
        cand = np.empty(2 * idx.numel(), np.int32)
        cand[0::2] = users[idx].cpu().numpy()
        cand[1::2] = items[idx].cpu().numpy()
        got = first_distinct(np.concatenate([got, cand]), batch)
    return got


def edge_weight_units(indptr: np.ndarray, seed: int, beta: float, stream: int = 40, bits: int = 16) -> np.ndarray:
    """Integer sampling weights q_e for every CSR entry: omega_e log-normal (a stand-in for the Swing scores of the
    paper's item graph), q_e = max(1, round(2^bits * (omega_e / max of its row)^beta)).  beta = 0 gives equal
    weights.  Drawn and quantised once, here, so that both sides are handed the same integers."""
    indptr = np.asarray(indptr, np.int64)
    m = int(indptr[-1])
    omega = np.exp(_rng(seed, stream).standard_normal(m))
    deg = np.diff(indptr)
    nz = deg > 0
    row_max = np.ones(indptr.size - 1)
    row_max[nz] = np.maximum.reduceat(omega, indptr[:-1][nz]) if m else 1.0
    rel = omega / np.repeat(row_max, deg)
    return np.maximum(1, np.rint((1 << bits) * rel ** beta)).astype(np.uint32)


def bernoulli_labels(n: int, p: float, seed: int, stream: int = 30) -> np.ndarray:
    return (_rng(seed, stream).random(n) < p).astype(np.float32)


def to_bf16_values(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even onto the bf16 grid; returned as float32 holding bf16 values."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


@dataclass
class Workload:
    """One of the benchmark configurations (shapes only; arrays are built on demand)."""
    name: str
    n_users: int
    n_items: int
    n_interactions: int
    alpha_user: object
    alpha_item: object
    seed: int
    dim: int
    hidden: int
    dtype: str            # "f32" or "bf16"
    fanouts: tuple
    batch: int
    q: float = 0.0
    extra: dict = field(default_factory=dict)

    @property
    def n_nodes(self) -> int:
        return self.n_users + self.n_items


WORKLOADS = {
    "tiny": Workload("tiny", 2_000, 3_000, 40_000, None, 1.2, 0, 64, 64, "f32", (10, 5), 256),
    "medium": Workload("medium", 200_000, 300_000, 10_000_000, 1.2, 1.2, 1, 128, 128, "bf16", (15, 10), 4096),
    "large": Workload("large", 20_000_000, 30_000_000, 1_000_000_000, 1.05, 1.05, 3, 256, 256, "bf16",
                      (20, 10, 5), 8192, q=80.0),
    # `large` at one eighth of its graph (same law, model, batch and fanouts): the feature table (3.2 GB) is still far
    # larger than L2, the whole workload holds under 5 GB on the device; used for counter captures and tests
    "large_eighth": Workload("large_eighth", 2_500_000, 3_750_000, 125_000_000, 1.05, 1.05, 3, 256, 256, "bf16",
                             (20, 10, 5), 8192, q=10.0),
    # the sampler shapes of the paper's experiments (Sec. 5.1: one hop x 100 neighbours, the default; two hops x 25, 15)
    # on the graph and features of `medium`; one GNN layer per hop
    "medium_1hop100": Workload("medium_1hop100", 200_000, 300_000, 10_000_000, 1.2, 1.2, 1, 128, 128, "bf16",
                               (100,), 4096),
    "medium_2hop25_15": Workload("medium_2hop25_15", 200_000, 300_000, 10_000_000, 1.2, 1.2, 1, 128, 128, "bf16",
                                 (25, 15), 4096),
    # the model and batch of `large` on the graph of `medium`: same kernel shapes, a few hundred MB on the device
    "medium_wide": Workload("medium_wide", 200_000, 300_000, 10_000_000, 1.2, 1.2, 1, 256, 256, "bf16",
                            (20, 10, 5), 8192),
    # shape-preserving reductions used where the full size does not fit the time budget of a test
    "medium_small": Workload("medium_small", 20_000, 30_000, 1_000_000, 1.2, 1.2, 1, 128, 128, "bf16",
                             (15, 10), 1024),
}


def build_graph(w: Workload):
    users, items = bipartite_interactions(w.n_users, w.n_items, w.n_interactions, w.alpha_user,
                                          w.alpha_item, w.seed, w.q)
    row, col = undirected_coo(users, items)
    indptr, indices = coo_to_csr(w.n_nodes, row, col)
    return indptr, indices, (users, items)


def build_weights(w: Workload):
    """Layer weights W_l [hidden x 2*d_in] (Glorot); fp32 arrays (bf16 values if w.dtype says so)."""
    Ws = []
    d_in = w.dim
    for l in range(len(w.fanouts)):
        Ws.append(glorot_uniform(w.hidden, 2 * d_in, w.seed, 20 + l))
        d_in = w.hidden
    if w.dtype == "bf16":
        Ws = [to_bf16_values(W) for W in Ws]
    return Ws


def build_model(w: Workload):
    """Features X [n x d] and the layer weights of build_weights."""
    X = normal_features(w.n_nodes, w.dim, w.seed)
    if w.dtype == "bf16":
        X = to_bf16_values(X)
    return X, build_weights(w)
