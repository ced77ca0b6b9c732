"""Pins for the oracle's graph ingest, sampler, relabel and block transpose (CPU only)."""
import numpy as np
import pytest

import oracle


def _random_coo(rng, n, m):
    return rng.integers(0, n, m).astype(np.int32), rng.integers(0, n, m).astype(np.int32)


def _dense_from_csr(n_rows, n_cols, indptr, indices):
    A = np.zeros((n_rows, n_cols), np.int64)
    for u in range(n_rows):
        for e in range(indptr[u], indptr[u + 1]):
            A[u, indices[e]] += 1
    return A


def test_csr_from_coo_equals_dense_counts_and_is_row_sorted():
    rng = np.random.default_rng(0)
    n, m = 37, 400
    row, col = _random_coo(rng, n, m)
    indptr, indices = oracle.csr_from_coo(n, row, col)
    A = np.zeros((n, n), np.int64)
    np.add.at(A, (row, col), 1)                       # brute-force adjacency with multiplicities
    assert np.array_equal(_dense_from_csr(n, n, indptr, indices), A)
    assert indptr[0] == 0 and indptr[-1] == m and np.all(np.diff(indptr) == A.sum(1))
    for u in range(n):
        seg = indices[indptr[u]:indptr[u + 1]]
        assert np.all(np.diff(seg) >= 0)
    order = np.lexsort((col, row))                    # library routine giving the same canonical order
    assert np.array_equal(indices, col[order])


def test_csr_from_coo_rejects_bad_ids_and_handles_empty():
    with pytest.raises(ValueError):
        oracle.csr_from_coo(4, [0, 5], [1, 1])
    indptr, indices = oracle.csr_from_coo(3, [], [])
    assert indptr.tolist() == [0, 0, 0, 0] and indices.size == 0


def test_transpose_is_dense_transpose_and_round_trips():
    rng = np.random.default_rng(1)
    n, m = 29, 300
    row, col = _random_coo(rng, n, m)
    indptr, indices = oracle.csr_from_coo(n, row, col)
    cptr, crow, ceid = oracle.csr_transpose(n, n, indptr, indices)
    assert np.array_equal(_dense_from_csr(n, n, cptr, crow), _dense_from_csr(n, n, indptr, indices).T)
    # eid points back at the CSR entry, and entries of a column come in CSR order
    rows_of_entry = np.repeat(np.arange(n), np.diff(indptr))
    assert np.array_equal(rows_of_entry[ceid], crow)
    for s in range(n):
        seg = ceid[cptr[s]:cptr[s + 1]]
        assert np.all(indices[seg] == s) and np.all(np.diff(seg) > 0)
    iptr2, idx2, _ = oracle.csr_transpose(n, n, cptr, crow)
    assert np.array_equal(iptr2, indptr) and np.array_equal(idx2, indices)


# ----------------------------------------------------------------------------- sampler

def _graph(rng, n, m):
    row, col = _random_coo(rng, n, m)
    return oracle.csr_from_coo(n, row, col)


def test_sampler_invariants():
    rng = np.random.default_rng(2)
    n = 300
    indptr, indices = _graph(rng, n, 3000)
    indptr = indptr.copy()
    seeds = rng.choice(n, 40, replace=False).astype(np.int32)
    fan = (4, 3)
    blocks = oracle.sample_khop(indptr, indices, seeds, fan, seed=11, step=5)
    dst = seeds
    for h, (blk, f) in enumerate(zip(blocks, fan), start=1):
        assert blk["n_dst"] == dst.size
        deg = (indptr[dst + 1] - indptr[dst]).astype(np.int64)
        cnt = np.diff(blk["indptr"])
        assert np.array_equal(cnt, np.minimum(deg, f))            # |S(u)| = min(deg, k)
        for i, u in enumerate(dst):
            s = blk["nbr_global"][blk["indptr"][i]:blk["indptr"][i + 1]]
            row = indices[indptr[u]:indptr[u + 1]]
            assert np.all(np.isin(s, row))                          # S(u) is drawn from N(u)
            if deg[i] <= f:
                assert np.array_equal(s, row)                       # take-all case: the row verbatim
        src = blk["src_nodes"]
        assert np.array_equal(src[:dst.size], dst)                  # F_h starts with D_h
        tail = src[dst.size:]
        assert np.all(np.diff(tail) > 0) and not np.any(np.isin(tail, dst))
        assert len(set(src.tolist())) == src.size
        assert np.array_equal(src[blk["col"]], blk["nbr_global"])   # col is the position in F_h
        assert set(src.tolist()) == set(dst.tolist()) | set(blk["nbr_global"].tolist())
        dst = src


def test_sampler_is_a_function_of_seed_step_and_node_only():
    rng = np.random.default_rng(3)
    n = 200
    indptr, indices = _graph(rng, n, 4000)
    seeds = rng.choice(n, 30, replace=False).astype(np.int32)
    a = oracle.sample_khop(indptr, indices, seeds, (5,), seed=1, step=0)[0]
    b = oracle.sample_khop(indptr, indices, seeds, (5,), seed=1, step=0)[0]
    c = oracle.sample_khop(indptr, indices, seeds, (5,), seed=1, step=1)[0]
    d = oracle.sample_khop(indptr, indices, seeds, (5,), seed=2, step=0)[0]
    assert np.array_equal(a["nbr_global"], b["nbr_global"])
    assert not np.array_equal(a["nbr_global"], c["nbr_global"])
    assert not np.array_equal(a["nbr_global"], d["nbr_global"])
    # permuting the batch permutes the rows but leaves each node's sample unchanged
    perm = rng.permutation(seeds.size)
    p = oracle.sample_khop(indptr, indices, seeds[perm], (5,), seed=1, step=0)[0]
    for j, i in enumerate(perm):
        sa = a["nbr_global"][a["indptr"][i]:a["indptr"][i + 1]]
        sp = p["nbr_global"][p["indptr"][j]:p["indptr"][j + 1]]
        assert np.array_equal(sa, sp)
    # the two hops of one step use different streams
    two = oracle.sample_khop(indptr, indices, seeds, (5, 5), seed=1, step=0)
    u = int(seeds[0])
    i2 = int(np.where(two[1]["src_nodes"][: two[1]["n_dst"]] == u)[0][0])
    s1 = two[0]["nbr_global"][two[0]["indptr"][0]:two[0]["indptr"][1]]
    s2 = two[1]["nbr_global"][two[1]["indptr"][i2]:two[1]["indptr"][i2 + 1]]
    assert not np.array_equal(s1, s2)


def test_draw_positions_follow_the_stated_counter_contract():
    """Recompute the picks of one node from Philox words with Python integers."""
    from test_oracle_philox import philox_bigint
    deg, f = 1000, 7
    # row 0 lists distinct labels so that the drawn position can be read back
    n = deg + 1
    indptr = np.zeros(n + 1, np.int64)
    indptr[1:] = deg
    indices = np.arange(1, deg + 1, dtype=np.int32)
    seed, step, hop = (0x1234ABCD << 32) | 0x9E3779B1, 77, 1
    blk = oracle.sample_khop(indptr, indices, np.array([0], np.int32), (f,), seed=seed, step=step)[0]
    want = []
    for j in range(f):
        out = philox_bigint([j >> 1, 0, (1 << 8) | hop, step], [seed & 0xFFFFFFFF, seed >> 32])
        r = (out[2 * (j & 1) + 1] << 32) | out[2 * (j & 1)]
        want.append(1 + ((r * deg) >> 64))
    assert blk["nbr_global"].tolist() == want


def test_uniform_draws_on_a_star_chi_square():
    """beta = 0: every stored neighbour of the hub is equally likely (Sec. 4.1 sampling probability)."""
    deg, f, steps = 16, 8, 4000
    n = deg + 1
    indptr = np.zeros(n + 1, np.int64)
    indptr[1:] = deg
    indices = np.arange(1, deg + 1, dtype=np.int32)
    counts = np.zeros(deg, np.int64)
    for t in range(steps):
        blk = oracle.sample_khop(indptr, indices, np.array([0], np.int32), (f,), seed=99, step=t)[0]
        np.add.at(counts, blk["nbr_global"] - 1, 1)
    expect = steps * f / deg
    chi2 = float(((counts - expect) ** 2 / expect).sum())
    assert chi2 < 37.7            # 99.9th percentile of chi-square with 15 degrees of freedom
    # draws within one call are not all identical (slots use distinct counters/words)
    blk = oracle.sample_khop(indptr, indices, np.array([0], np.int32), (f,), seed=99, step=0)[0]
    assert len(set(blk["nbr_global"].tolist())) > 2


def test_block_transpose_is_dense_transpose():
    rng = np.random.default_rng(4)
    n = 120
    indptr, indices = _graph(rng, n, 1500)
    seeds = rng.choice(n, 25, replace=False).astype(np.int32)
    for blk in oracle.sample_khop(indptr, indices, seeds, (6, 4), seed=5, step=2):
        nd, ns = blk["n_dst"], blk["n_src"]
        B = _dense_from_csr(nd, ns, blk["indptr"], blk["col"])
        Bt = _dense_from_csr(ns, nd, blk["csc_ptr"], blk["csc_row"])
        assert np.array_equal(Bt, B.T)
        rows_of_entry = np.repeat(np.arange(nd), np.diff(blk["indptr"]))
        assert np.array_equal(rows_of_entry[blk["csc_eid"]], blk["csc_row"])
        assert np.array_equal(blk["col"][blk["csc_eid"]], np.repeat(np.arange(ns), np.diff(blk["csc_ptr"])))
        for s in range(ns):
            assert np.all(np.diff(blk["csc_eid"][blk["csc_ptr"][s]:blk["csc_ptr"][s + 1]]) > 0)
        cnt = np.diff(blk["indptr"]).astype(np.float32)
        want = np.where(cnt > 0, np.float32(1.0) / np.maximum(cnt, 1), np.float32(0.0)).astype(np.float32)
        assert np.array_equal(blk["inv_cnt"], want)


def test_isolated_and_empty_cases():
    indptr = np.array([0, 0, 2, 2], np.int64)
    indices = np.array([0, 2], np.int32)
    blk = oracle.sample_khop(indptr, indices, np.array([0, 1], np.int32), (3,), seed=0, step=0)[0]
    assert blk["indptr"].tolist() == [0, 0, 2] and blk["inv_cnt"].tolist() == [0.0, 0.5]
    assert blk["src_nodes"].tolist() == [0, 1, 2] and blk["col"].tolist() == [0, 2]
    blk = oracle.sample_khop(indptr, indices, np.array([], np.int32), (3,), seed=0, step=0)[0]
    assert blk["n_dst"] == 0 and blk["n_src"] == 0 and blk["n_edges"] == 0
