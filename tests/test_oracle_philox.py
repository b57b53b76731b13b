"""Pins for the oracle's threshold generator (Def. 3: eps ~ U[0,1], independent per element).

The generator is Philox4x32-10.  It is pinned to (a) the published known-answer
vectors, (b) a second implementation written here in Python big integers from
the algorithm's description, and (c) the uniformity Def. 3 asks of eps.
"""
import os
import random

import numpy as np

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

M0, M1 = 0xD2511F53, 0xCD9E8D57
W0, W1 = 0x9E3779B9, 0xBB67AE85
MASK = 0xFFFFFFFF


def philox_py(ctr, key, rounds=10):
    """Independent restatement: ten rounds of two 32x32->64 multiplies and a word shuffle."""
    c = list(ctr)
    k = list(key)
    for r in range(rounds):
        prod0 = M0 * c[0]
        prod1 = M1 * c[2]
        c = [((prod1 >> 32) ^ c[1] ^ k[0]) & MASK, prod1 & MASK,
             ((prod0 >> 32) ^ c[3] ^ k[1]) & MASK, prod0 & MASK]
        k = [(k[0] + W0) & MASK, (k[1] + W1) & MASK]
    return c


def threshold_py(seed, tensor_id, i):
    j = i >> 2
    out = philox_py([j & MASK, (j >> 32) & MASK, tensor_id & MASK, (tensor_id >> 32) & MASK],
                    [seed & MASK, (seed >> 32) & MASK])
    return out[i & 3] >> 8


def _kat():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            w = [int(t, 16) for t in line.split()]
            rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_published_known_answers():
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, expect in rows:
        assert oracle.philox4x32_10(ctr, key) == expect
        assert philox_py(ctr, key) == expect


def test_matches_independent_python_implementation():
    rng = random.Random(1234)
    for _ in range(300):
        ctr = [rng.getrandbits(32) for _ in range(4)]
        key = [rng.getrandbits(32) for _ in range(2)]
        assert oracle.philox4x32_10(ctr, key) == philox_py(ctr, key)


def test_threshold_counter_layout():
    """Block index in words 0-1, tensor_id in words 2-3, seed as key, word i&3, top 24 bits."""
    rng = random.Random(7)
    cases = [(0, 0, 0), (0, 0, 1), (0, 0, 3), (0, 0, 4), (1, 0, 0), (0, 1, 0),
             (2**40 + 5, 2**35 + 3, 2**34 + 2), (2**63 + 9, 2**64 - 1, 2**64 - 1)]
    cases += [(rng.getrandbits(64), rng.getrandbits(64), rng.getrandbits(64)) for _ in range(100)]
    for seed, tid, i in cases:
        assert oracle.threshold_u24(seed, tid, i) == threshold_py(seed, tid, i)
    # the four elements of one block are the four words of one Philox call
    block = philox_py([5, 0, 9, 0], [3, 0])
    assert [oracle.threshold_u24(3, 9, 20 + w) for w in range(4)] == [v >> 8 for v in block]


def test_thresholds_are_uniform_and_uncorrelated():
    n = 1 << 16
    u = np.array([oracle.threshold_u24(11, 5, i) for i in range(n)], dtype=np.float64) / 2.0**24
    # mean of U[0,1): 1/2 with sd 1/sqrt(12 n); variance 1/12
    assert abs(u.mean() - 0.5) < 5.0 / np.sqrt(12.0 * n)
    assert abs(u.var() - 1.0 / 12.0) < 0.002
    # chi-square over 64 equal bins: mean 63, sd sqrt(126)
    hist, _ = np.histogram(u, bins=64, range=(0.0, 1.0))
    chi2 = ((hist - n / 64.0) ** 2 / (n / 64.0)).sum()
    assert chi2 < 63 + 6 * np.sqrt(126.0)
    # neighbouring elements, other tensor_id, other seed: correlation ~ N(0, 1/n)
    v = np.array([oracle.threshold_u24(11, 6, i) for i in range(n)], dtype=np.float64) / 2.0**24
    w = np.array([oracle.threshold_u24(12, 5, i) for i in range(n)], dtype=np.float64) / 2.0**24
    for a, b in ((u[:-1], u[1:]), (u, v), (u, w)):
        assert abs(np.corrcoef(a, b)[0, 1]) < 5.0 / np.sqrt(n)
