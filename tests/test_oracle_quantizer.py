"""Pins for the oracle's quantizer (Def. 1-3) against what the paper and the mathematics fix."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import PER_ROW, PER_TENSOR, RTN, SR, QSpec
from _independent import (qmax_of, quantize_matrix_ref, quantize_scalar_ref, scale_ref,
                          thresholds_u24)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _kv(name):
    d = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, v = line.split()
            d[k] = float(v)
    return d


# ---------------------------------------------------------------- Def. 2: RTN
def test_rtn_tie_table_from_definition():
    with open(os.path.join(GOLDEN, "rtn_ties.txt")) as f:
        rows = [line.split() for line in f if line.strip() and not line.startswith("#")]
    assert len(rows) >= 10
    for t, code in rows:
        # step 1: inv = 1, so t = x
        assert oracle.quantize_scalar(float(t), 1.0, 8, RTN) == int(code), t


def test_rtn_is_floor_of_t_plus_half_in_exact_arithmetic():
    rng = np.random.default_rng(0)
    ts = np.concatenate([rng.uniform(-120, 120, 4000), np.arange(-100, 100) + 0.5,
                         [0.49999997, -0.49999997, 0.50000006, 1e-30, -1e-30]]).astype(np.float32)
    for t in ts:
        expect = math.floor(Fraction(float(t)) + Fraction(1, 2))
        assert oracle.quantize_scalar(float(t), 1.0, 8, RTN) == expect, float(t)


def test_rtn_error_at_most_half_step_and_idempotent():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((64, 96)).astype(np.float32)
    for bits in (8, 6, 4, 3):
        codes, scale, _, _ = oracle.sr_quantize(x, QSpec(bits=bits, round_mode=RTN))
        d = float(scale[0])
        xhat = codes.astype(np.float64) * d
        # |x - xhat| <= D/2 (proof of the bias lemma), up to binary32 rounding of x*inv
        assert np.abs(x - xhat).max() <= d / 2 * (1 + 1e-5)
        again, scale2, _, _ = oracle.sr_quantize((codes.astype(np.float32) * scale[0]),
                                                 QSpec(bits=bits, round_mode=RTN))
        assert np.array_equal(again, codes)


# ---------------------------------------------------------------- worked example
def test_worked_example_sum_of_ten_0p7():
    g = _kv("worked_example_sum_of_0p7.txt")
    terms = int(g["terms"])
    # a tensor holding the ten 0.7s and one element equal to qmax, so that the
    # absmax rule gives exactly the example's step 1
    x = np.array([[127.0] + [g["x"]] * terms], dtype=np.float32)
    codes, scale, _, _ = oracle.sr_quantize(x, QSpec(bits=8, round_mode=RTN))
    assert scale[0] == g["step"]
    assert list(codes[0, 1:]) == [int(g["rtn_code"])] * terms
    assert int(codes[0, 1:].sum()) == int(g["rtn_sum"])
    # SR: exact probability over all 2^24 thresholds (binary32 0.7 = 11744051 / 2^24)
    total = oracle.sum_sr_codes_over_all_thresholds(np.float32(g["x"]), 1.0, 8)
    p_up = Fraction(total, 2 ** 24)
    assert p_up == Fraction(float(np.float32(g["x"])))
    assert abs(float(p_up) - g["sr_prob_up"]) < 2 ** -23
    # Monte Carlo over seeds: sums vary, their mean tends to 7
    sums = []
    for seed in range(4000):
        c, _, _, _ = oracle.sr_quantize(x, QSpec(bits=8, round_mode=SR, seed=seed))
        assert set(np.unique(c[0, 1:])) <= {0, 1}
        sums.append(int(c[0, 1:].sum()))
    sums = np.array(sums)
    sd = math.sqrt(terms * 0.7 * 0.3)
    assert abs(sums.mean() - g["sr_expected_sum"]) < 5 * sd / math.sqrt(len(sums))
    assert abs(sums.var() - terms * 0.21) < 0.25
    assert sums.min() < 7 < sums.max()


# ---------------------------------------------------------------- Def. 3: SR
@pytest.mark.parametrize("t", [0.0, 2.0 ** -24, 0.3, 0.5, 0.7, 1 - 2.0 ** -24, 5.25, -0.3, -7.75,
                               -100.5, 126.999,
                               # fractional parts that binary32 cannot hold (t - floor(t) would round)
                               -2.0 ** -30, -10066331 * 2.0 ** -25, -8388609 * 2.0 ** -25 , 2.0 ** -40,
                               -1e-30, 1e-40, -1e-40])
def test_sr_probability_of_rounding_up_is_the_fraction_exactly(t):
    t32 = np.float32(t)
    f = math.floor(Fraction(float(t32)))
    p = Fraction(float(t32)) - f
    total = oracle.sum_sr_codes_over_all_thresholds(t32, 1.0, 8)
    # eps uniform on k/2^24: P(eps < p) = ceil(p 2^24) / 2^24
    ups = math.ceil(p * 2 ** 24)
    assert total == f * 2 ** 24 + ups
    # hence |E[q] - t| < 2^-24, and = 0 when p is on the lattice
    assert abs(Fraction(total, 2 ** 24) - Fraction(float(t32))) < Fraction(1, 2 ** 24)


def test_sr_grid_exact_inputs_never_move():
    # absmax = qmax * 2^-5  ->  step 2^-5 and 1/step 2^5 exactly
    for bits in (8, 6, 4, 3):
        q = qmax_of(bits)
        k = np.arange(-q, q + 1, dtype=np.float32)
        x = (k * 2.0 ** -5).reshape(1, -1).astype(np.float32)
        for seed in range(20):
            for mode in (SR, RTN):
                c, s, _, _ = oracle.sr_quantize(x, QSpec(bits=bits, round_mode=mode, seed=seed))
                assert s[0] == np.float32(2.0 ** -5)
                assert np.array_equal(c[0].astype(np.float32), k)


def test_sr_output_is_one_of_the_two_neighbours_and_error_below_one_step():
    rng = np.random.default_rng(3)
    x = (rng.standard_normal((37, 53)) * 3).astype(np.float32)
    for bits in (8, 6, 4, 3, 2):
        for seed in range(5):
            c, s, _, _ = oracle.sr_quantize(x, QSpec(bits=bits, seed=seed, tensor_id=seed + 1))
            _, inv = scale_ref(np.abs(x).max(), bits)
            t = x.astype(np.float64) * float(inv)       # exact product of two binary32 values
            lo = np.floor(t)
            q = qmax_of(bits)
            assert np.all((c == np.clip(lo, -q, q)) | (c == np.clip(lo + 1, -q, q)))
            assert np.abs(c.astype(np.float64) * float(s[0]) - x).max() < float(s[0]) * (1 + 1e-5)


def test_sr_codes_match_independent_restatement_with_index_offset():
    rng = np.random.default_rng(4)
    for (rows, cols, off) in [(5, 7, 0), (8, 16, 3), (3, 5, 2 ** 33 + 1), (1, 9, 6), (9, 1, 0)]:
        x = rng.standard_normal((rows, cols)).astype(np.float32)
        for bits in (8, 4):
            seed, tid = 17 + bits, 2 ** 32 + 5
            u = thresholds_u24(seed, tid, off, rows, cols)
            # per tensor, both layouts
            c, s, ct, st = oracle.sr_quantize(
                x, QSpec(bits=bits, seed=seed, tensor_id=tid, index_offset=off), True, True)
            d, inv = scale_ref(np.abs(x).max(), bits)
            ref = quantize_matrix_ref(x, inv, bits, True, u)
            assert s[0] == d and st[0] == d
            assert np.array_equal(c, ref)
            assert np.array_equal(ct, ref.T)
            # spot check single elements through exact rationals
            for (r, cc) in [(0, 0), (rows - 1, cols - 1), (rows // 2, cols // 2)]:
                assert c[r, cc] == quantize_scalar_ref(x[r, cc], inv, bits, True, u[r, cc])
            # per row: the row-major layout scales by row absmax, the transposed layout by
            # column absmax, both with the threshold of the source element
            c, s, ct, st = oracle.sr_quantize(
                x, QSpec(bits=bits, scale_mode=PER_ROW, seed=seed, tensor_id=tid,
                         index_offset=off), True, True)
            sc = [scale_ref(m, bits) for m in np.abs(x).max(axis=1)]
            inv_r = np.array([v[1] for v in sc], dtype=np.float32)[:, None]
            assert np.array_equal(s, np.array([v[0] for v in sc], dtype=np.float32))
            assert np.array_equal(c, quantize_matrix_ref(x, inv_r, bits, True, u))
            sc = [scale_ref(m, bits) for m in np.abs(x).max(axis=0)]
            inv_c = np.array([v[1] for v in sc], dtype=np.float32)[None, :]
            assert np.array_equal(st, np.array([v[0] for v in sc], dtype=np.float32))
            assert np.array_equal(ct, quantize_matrix_ref(x, inv_c, bits, True, u).T)


def test_rtn_matrix_matches_independent_restatement():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((11, 13)).astype(np.float32)
    for bits in (8, 6, 3):
        c, s, ct, st = oracle.sr_quantize(x, QSpec(bits=bits, round_mode=RTN), True, True)
        d, inv = scale_ref(np.abs(x).max(), bits)
        ref = quantize_matrix_ref(x, inv, bits, False, None)
        assert np.array_equal(c, ref) and np.array_equal(ct, ref.T) and s[0] == d


def test_sr_unbiased_and_variance_bound_over_1e4_draws():
    """E[Q(x)] = x within 5 sigma per element; Var = D^2 p(1-p) <= D^2/4 (4096 elements)."""
    rng = np.random.default_rng(6)
    x = rng.standard_normal((1, 4096)).astype(np.float32)
    draws = 10_000
    for bits in (8, 4):
        d, inv = scale_ref(np.abs(x).max(), bits)
        acc = np.zeros(x.shape, dtype=np.float64)
        acc2 = np.zeros(x.shape, dtype=np.float64)
        for seed in range(draws):
            c, s, _, _ = oracle.sr_quantize(x, QSpec(bits=bits, seed=seed, tensor_id=3))
            acc += c
            acc2 += c.astype(np.float64) ** 2
        mean_q = acc / draws
        var_q = acc2 / draws - mean_q ** 2
        t = x.astype(np.float64) * float(inv)
        p = t - np.floor(t)
        sigma = np.sqrt(p * (1 - p) / draws)
        # 5 sigma plus the lattice term, in units of the step
        assert np.all(np.abs(mean_q - t) <= 5 * sigma + 3.0 / draws)
        assert var_q.max() <= 0.25 + 1e-9
        # the variance is the Bernoulli one (loose 6-sigma check on its estimate)
        assert np.abs(var_q - p * (1 - p)).max() < 0.03
        # value domain: mean error in x units
        assert np.abs(mean_q * float(d) - x).max() < float(d) * 0.03


def test_different_tensor_id_or_seed_gives_independent_rounding():
    rng = np.random.default_rng(8)
    x = rng.uniform(-1, 1, (1, 1 << 14)).astype(np.float32)
    d, inv = scale_ref(np.abs(x).max(), 8)
    lo = np.floor(x.astype(np.float64) * float(inv))

    def ups(seed, tid):
        c, _, _, _ = oracle.sr_quantize(x, QSpec(seed=seed, tensor_id=tid))
        return (c - lo).ravel() - (x.astype(np.float64) * float(inv) - lo).ravel()  # centred

    a, b, c2 = ups(1, 1), ups(1, 2), ups(2, 1)
    n = a.size
    assert abs(np.corrcoef(a, b)[0, 1]) < 5 / math.sqrt(n)
    assert abs(np.corrcoef(a, c2)[0, 1]) < 5 / math.sqrt(n)
    assert np.array_equal(ups(1, 1), a)     # deterministic for fixed eps (note under Alg. 1)


# ---------------------------------------------------------------- step size
def test_absmax_matches_numpy_and_handles_pitch():
    rng = np.random.default_rng(9)
    big = rng.standard_normal((19, 40)).astype(np.float32)
    x = big[:, 3:34]                                    # row pitch 40, 31 columns
    assert oracle.absmax(x, "tensor")[0] == np.abs(x).max()
    assert np.array_equal(oracle.absmax(x, "rows"), np.abs(x).max(axis=1))
    assert np.array_equal(oracle.absmax(x, "cols"), np.abs(x).max(axis=0))


def test_scale_rule_and_zero_group():
    from fractions import Fraction
    rng = np.random.default_rng(9)
    for bits in (8, 6, 4, 3, 2):
        q = qmax_of(bits)
        for m in [3.0, 1.0, 127.0] + list(rng.uniform(1e-3, 50, 300).astype(np.float32)):
            d, inv = oracle.scale_from_absmax(float(m), bits)
            assert d == np.float32(m) / np.float32(q)
            # inv is the largest binary32 number <= qmax / m (round toward zero)
            exact = Fraction(q) / Fraction(float(np.float32(m)))
            assert Fraction(float(inv)) <= exact < Fraction(float(np.nextafter(inv, np.float32(np.inf))))
            assert (d, inv) == scale_ref(m, bits)
    # Delta = 0: Q_0 is the identity (note in Def. 1); only an all-zero group reaches it
    d, inv = oracle.scale_from_absmax(0.0, 8)
    assert d == 0 and inv == 0
    z = np.zeros((3, 4), dtype=np.float32)
    c, s, ct, st = oracle.sr_quantize(z, QSpec(bits=8, scale_mode=PER_ROW), True, True)
    assert not c.any() and not ct.any() and not s.any() and not st.any()
    # a group too small for 1/Delta to be finite is flushed the same way
    d, inv = oracle.scale_from_absmax(1e-38, 8)
    assert d == 0 and inv == 0
    # mixed: one zero row among non-zero rows
    x = np.array([[0, 0, 0], [1, -2, 0.5]], dtype=np.float32)
    c, s, _, _ = oracle.sr_quantize(x, QSpec(bits=8, scale_mode=PER_ROW, round_mode=RTN))
    assert s[0] == 0 and not c[0].any() and c[1, 1] == -127


def test_quotient_of_the_extreme_element_never_passes_qmax():
    # Def. 1 has no saturation: |x / D| <= qmax for the whole group.  With the reciprocal rounded
    # toward zero the binary32 quotient of the absmax element itself stays <= qmax, so every code
    # is inside [-qmax, qmax] before any clamp; the extreme element lands on qmax or qmax - 1.
    rng = np.random.default_rng(10)
    ms = rng.uniform(0.1, 10, 2000).astype(np.float32)
    below = False
    for bits in (8, 4):
        q = qmax_of(bits)
        for m in ms:
            d, inv = oracle.scale_from_absmax(float(m), bits)
            t = np.float32(m) * inv
            assert t <= q
            below |= bool(t < q)
            for u in (0, 1, 2 ** 23, 2 ** 24 - 1):
                hi = oracle.quantize_scalar(float(m), float(inv), bits, SR, u)
                lo = oracle.quantize_scalar(-float(m), float(inv), bits, SR, u)
                assert -q <= lo <= -q + 1 and q - 1 <= hi <= q
            assert oracle.quantize_scalar(float(m), float(inv), bits, RTN) == q
            assert oracle.quantize_scalar(-float(m), float(inv), bits, RTN) == -q
    assert below


def test_eight_bit_thresholds_bytes_of_the_philox_stream_and_centred_probabilities():
    """SR with 8 random bits per element: the threshold of element i is byte i & 3 of word (i >> 2) & 3 of
    Philox block i >> 4 (independent numpy Philox), placed at (b + 1/2) / 256; P(up) is then the fraction
    rounded to the nearest multiple of 1/256, and the rounding stays unbiased on average."""
    from _independent import philox_np
    seed, tid, off = 2 ** 40 + 5, 2 ** 33 + 7, 2 ** 36 + 3
    idx = np.arange(off, off + 200, dtype=np.uint64)
    j = idx >> np.uint64(4)
    words = philox_np(j & np.uint64(0xFFFFFFFF), j >> np.uint64(32), np.full_like(j, tid & 0xFFFFFFFF),
                      np.full_like(j, tid >> 32), seed & 0xFFFFFFFF, seed >> 32)
    stacked = np.stack(words, axis=0)
    w = np.take_along_axis(stacked, ((idx >> np.uint64(2)) & np.uint64(3)).astype(np.int64)[None, :], axis=0)[0]
    b = (w >> (np.uint64(8) * (idx & np.uint64(3)))) & np.uint64(0xFF)
    want = (2 * b.astype(np.int64) + 1) << 15
    got = np.array([oracle.threshold_sr8(seed, tid, int(i)) for i in idx])
    assert np.array_equal(got, want)
    # exact probability: thresholds (2b+1) 2^15 for b = 0..255, up iff threshold < frac 2^24
    for p in (0.0, 1 / 512, 1 / 256, 0.3, 0.5, 0.7, 1 - 1 / 512, 1 - 2.0 ** -20):
        ups = sum(oracle.quantize_scalar(2.0 + p, 1.0, 8, oracle.SR8, (2 * bb + 1) << 15) == 3 for bb in range(256))
        assert ups == math.floor(256 * p + 0.5) or (256 * p + 0.5 == math.floor(256 * p + 0.5) and ups == 256 * p - 0.5)
    # matrix form against the restatement, and unbiasedness over seeds
    rng = np.random.default_rng(13)
    x = rng.normal(0, 1, (1, 2048)).astype(np.float32)
    d, inv = scale_ref(np.abs(x).max(), 8)
    u = np.array([oracle.threshold_sr8(3, 9, i) for i in range(2048)]).reshape(1, 2048)
    c, s, _, _ = oracle.sr_quantize(x, QSpec(8, PER_TENSOR, oracle.SR8, 3, 9))
    assert np.array_equal(c, quantize_matrix_ref(x, inv, 8, True, u)) and s[0] == d
    acc = np.zeros((1, 2048))
    draws = 3000
    for seed in range(draws):
        acc += oracle.sr_quantize(x, QSpec(8, PER_TENSOR, oracle.SR8, seed, 9))[0]
    t = x.astype(np.float64) * float(inv)
    p = t - np.floor(t)
    err = acc / draws - t
    assert np.all(np.abs(err) <= 5 * np.sqrt(p * (1 - p) / draws) + 1 / 512 + 3.0 / draws)      # per element: within 2^-9 of unbiased
    assert abs(err.mean()) < 3e-3                                                                  # and no systematic sign
