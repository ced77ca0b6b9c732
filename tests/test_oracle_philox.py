"""Pins for the oracle's Philox4x32-10 and bf16 rounding (CPU only)."""
import os

import numpy as np
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            w = [int(x, 16) for x in line.split()]
            rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def philox_bigint(ctr, key):
    """Independent restatement with Python integers (no fixed-width arithmetic)."""
    c, k = [int(x) for x in ctr], [int(x) for x in key]
    for _ in range(10):
        p0, p1 = 0xD2511F53 * c[0], 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 % 2**32, (p0 >> 32) ^ c[3] ^ k[1], p0 % 2**32]
        k = [(k[0] + 0x9E3779B9) % 2**32, (k[1] + 0xBB67AE85) % 2**32]
    return c


def test_known_answer_vectors():
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, out in rows:
        assert [int(x) for x in oracle.philox4x32_10(ctr, key)] == out


def test_matches_bigint_restatement():
    rng = np.random.default_rng(7)
    for _ in range(200):
        ctr = rng.integers(0, 2**32, 4, dtype=np.uint64)
        key = rng.integers(0, 2**32, 2, dtype=np.uint64)
        assert [int(x) for x in oracle.philox4x32_10(ctr, key)] == philox_bigint(ctr, key)


def test_counter_and_key_words_all_matter():
    base = [int(x) for x in oracle.philox4x32_10([1, 2, 3, 4], [5, 6])]
    for i in range(4):
        c = [1, 2, 3, 4]
        c[i] ^= 1
        assert [int(x) for x in oracle.philox4x32_10(c, [5, 6])] != base
    for i in range(2):
        k = [5, 6]
        k[i] ^= 1
        assert [int(x) for x in oracle.philox4x32_10([1, 2, 3, 4], k)] != base


def test_round_bf16_matches_torch_conversion():
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-6, 6, 20000),
                        [0.0, 1.0, -1.0, 1.00390625, 1.01171875, 3.0e-5, 65504.0]]).astype(np.float32)
    # exact ties between two bf16 neighbours (9th significant bit set, nothing below)
    ties = (np.arange(256, 512, dtype=np.float64) + 0.5) / 256.0
    x = np.concatenate([x, ties.astype(np.float32), -ties.astype(np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    got = oracle.round_bf16(x.astype(np.float64))
    assert np.array_equal(got, want)
