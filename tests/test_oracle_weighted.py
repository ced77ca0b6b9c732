"""Pins for the oracle's weighted (importance) sampler, p(u -> v) = q_uv / sum_k q_uk (Sec. 4.1 with q for omega^beta)."""
import numpy as np

import oracle
import synth_inputs as S


def _star(deg):
    """Node 0 lists nodes 1..deg (distinct labels, so that a drawn position can be read back); the others are empty."""
    n = deg + 1
    indptr = np.zeros(n + 1, np.int64)
    indptr[1:] = deg
    return indptr, np.arange(1, deg + 1, dtype=np.int32)


def test_running_sums_by_brute_force():
    indptr = np.array([0, 3, 3, 7, 8], np.int64)
    q = np.array([5, 0, 2**32 - 1, 2**32 - 1, 2**32 - 1, 7, 2**32 - 1, 1], np.uint32)      # sums pass 2^32
    cum = oracle.edge_cumulate(indptr, q)
    for u in range(4):
        run = 0
        for e in range(indptr[u], indptr[u + 1]):
            run += int(q[e])
            assert int(cum[e]) == run
    assert cum.dtype == np.uint64 and int(cum[6]) > 2**32


def test_equal_weights_give_the_uniform_sampler_bit_for_bit():
    """floor(floor(r c deg / 2^64) / c) = floor(r deg / 2^64): with q = c on every entry the weighted draw picks the
    entries of the uniform draw, whatever c is."""
    w = S.WORKLOADS["tiny"]
    indptr, indices, _ = S.build_graph(w)
    seeds = S.seed_batch(w.n_nodes, 64, w.seed, 0)
    plain = oracle.sample_khop(indptr, indices, seeds, w.fanouts, w.seed, 3)
    for c in (1, 7, 65536):
        cum = oracle.edge_cumulate(indptr, np.full(indices.size, c, np.uint32))
        got = oracle.sample_khop(indptr, indices, seeds, w.fanouts, w.seed, 3, edge_cum=cum)
        for a, b in zip(got, plain):
            for k in ("indptr", "nbr_global", "src_nodes", "col"):
                assert np.array_equal(a[k], b[k])


def test_draws_follow_the_stated_contract():
    """Recompute the picks of one node from Philox words with Python integers and a linear search."""
    from test_oracle_philox import philox_bigint
    deg, f = 300, 9
    indptr, indices = _star(deg)
    q = np.random.default_rng(1).integers(0, 1000, deg).astype(np.uint32)
    cum = oracle.edge_cumulate(indptr, q)
    seed, step, hop = (0xABCDEF01 << 32) | 0x13579BDF, 5, 1
    blk = oracle.sample_khop(indptr, indices, np.array([0], np.int32), (f,), seed=seed, step=step, edge_cum=cum)[0]
    total = int(q.astype(np.int64).sum())
    want = []
    for j in range(f):
        out = philox_bigint([j >> 1, 0, (1 << 8) | hop, step], [seed & 0xFFFFFFFF, seed >> 32])
        r = (out[2 * (j & 1) + 1] << 32) | out[2 * (j & 1)]
        t, run = (r * total) >> 64, 0
        for p in range(deg):
            run += int(q[p])
            if run > t:
                want.append(p + 1)
                break
    assert blk["nbr_global"].tolist() == want


def test_frequencies_are_proportional_to_the_weights_chi_square():
    deg, f, steps = 8, 4, 6000
    indptr, indices = _star(deg)
    q = np.array([1, 2, 3, 4, 0, 10, 5, 7], np.uint32)
    cum = oracle.edge_cumulate(indptr, q)
    counts = np.zeros(deg, np.int64)
    for t in range(steps):
        blk = oracle.sample_khop(indptr, indices, np.array([0], np.int32), (f,), seed=21, step=t, edge_cum=cum)[0]
        np.add.at(counts, blk["nbr_global"] - 1, 1)
    assert counts[4] == 0                                    # weight 0 is never drawn
    live = q > 0
    expect = steps * f * q[live] / q.sum()
    chi2 = float(((counts[live] - expect) ** 2 / expect).sum())
    assert chi2 < 22.5            # 99.9th percentile of chi-square with 6 degrees of freedom


def test_short_rows_are_taken_whole_and_zero_rows_fall_back_to_uniform():
    deg = 12
    indptr, indices = _star(deg)
    q = np.arange(deg, dtype=np.uint32)
    cum = oracle.edge_cumulate(indptr, q)
    blk = oracle.sample_khop(indptr, indices, np.array([0], np.int32), (20,), seed=1, step=0, edge_cum=cum)[0]
    assert blk["nbr_global"].tolist() == list(range(1, deg + 1))       # deg <= fanout: every neighbour once
    zero = oracle.edge_cumulate(indptr, np.zeros(deg, np.uint32))
    a = oracle.sample_khop(indptr, indices, np.array([0], np.int32), (5,), seed=1, step=0, edge_cum=zero)[0]
    b = oracle.sample_khop(indptr, indices, np.array([0], np.int32), (5,), seed=1, step=0)[0]
    assert np.array_equal(a["nbr_global"], b["nbr_global"])


def test_generated_weight_units_are_positive_and_follow_beta():
    indptr, indices, _ = S.build_graph(S.WORKLOADS["tiny"])
    q0 = S.edge_weight_units(indptr, 0, beta=0.0)
    q1 = S.edge_weight_units(indptr, 0, beta=1.0)
    q2 = S.edge_weight_units(indptr, 0, beta=2.0)
    assert q0.dtype == np.uint32 and (q0 == q0[0]).all() and (q1 >= 1).all()
    # a larger beta concentrates the mass: the share of the heaviest entry of a long row grows
    u = int(np.argmax(np.diff(indptr)))
    s, e = indptr[u], indptr[u + 1]
    assert q2[s:e].max() / q2[s:e].sum() > q1[s:e].max() / q1[s:e].sum()
