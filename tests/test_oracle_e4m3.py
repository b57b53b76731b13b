"""Pins of the oracle's E4M3 path from outside the oracle: the format's definition and torch's
float8_e4m3fn (a library routine) for decoding and nearest rounding, exact rationals for the
rounding rule of Def. 1 applied with the local step, Monte Carlo for unbiasedness, numpy's
binary64 matmul for the product."""
from fractions import Fraction

import numpy as np
import torch

import oracle
from oracle import PER_ROW, PER_TENSOR, RTN, SR, QSpec
from _independent import thresholds_u24

ALL = np.arange(256, dtype=np.uint8)
FINITE = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)


def _grid():
    """Sorted distinct finite E4M3 values from the format's definition (no oracle code)."""
    vals = set()
    for ex in range(16):
        for man in range(8):
            if ex == 15 and man == 7:
                continue
            v = Fraction(man, 8) * Fraction(1, 64) if ex == 0 else (1 + Fraction(man, 8)) * Fraction(2) ** (ex - 7)
            vals.add(v)
            vals.add(-v)
    return sorted(vals)


def test_decode_matches_torch_and_known_values():
    got = oracle.e4m3_decode(ALL)
    want = torch.from_numpy(ALL.copy()).view(torch.float8_e4m3fn).double().numpy()
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.array_equal(got[~np.isnan(got)], want[~np.isnan(want)])
    assert oracle.e4m3_decode([0x7E])[0] == 448.0 and oracle.e4m3_decode([0x01])[0] == 2.0 ** -9
    assert oracle.e4m3_decode([0x38])[0] == 1.0 and oracle.e4m3_decode([0xB8])[0] == -1.0
    assert sorted(set(Fraction(float(v)) for v in got[~np.isnan(got)])) == _grid()


def test_grid_values_never_move_under_either_rounding():
    for c in FINITE:
        v = float(oracle.e4m3_decode([c])[0])
        for u in (0, 1, 2 ** 23, 2 ** 24 - 1):
            q = oracle.quantize_e4m3_scalar(v, 1.0, SR, u)
            assert oracle.e4m3_decode([q])[0] == v
        assert oracle.e4m3_decode([oracle.quantize_e4m3_scalar(v, 1.0, RTN)])[0] == v
    assert oracle.quantize_e4m3_scalar(-0.0, 1.0, SR, 5) == 0


def test_rtn_is_torchs_nearest_cast_except_at_ties_which_go_up():
    rng = np.random.default_rng(1)
    t = np.concatenate([rng.uniform(-448, 448, 4000), rng.normal(0, 1, 4000), rng.normal(0, 0.01, 2000)]).astype(np.float32)
    got = np.array([oracle.quantize_e4m3_scalar(float(v), 1.0, RTN) for v in t], dtype=np.uint8)
    want = torch.from_numpy(t).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    gv, wv = oracle.e4m3_decode(got), oracle.e4m3_decode(want)
    grid = _grid()
    for i in np.nonzero(gv != wv)[0]:            # only exact ties may differ, and ours is the upper neighbour
        lo = max(g for g in grid if g <= Fraction(float(t[i])))
        hi = min(g for g in grid if g >= Fraction(float(t[i])))
        assert Fraction(float(t[i])) - lo == hi - Fraction(float(t[i])) and Fraction(float(gv[i])) == hi
    # Def. 2: ties toward +infinity, both signs (torch rounds these to even)
    for tie, want_v in ((1.0625, 1.125), (-1.0625, -1.0), (1.1875, 1.25), (-1.1875, -1.125), (2.0 ** -10, 2.0 ** -9)):
        assert oracle.e4m3_decode([oracle.quantize_e4m3_scalar(tie, 1.0, RTN)])[0] == want_v


def test_sr_goes_to_a_neighbour_with_probability_equal_to_the_fractional_distance():
    grid = _grid()
    rng = np.random.default_rng(2)
    ts = np.concatenate([rng.uniform(-448, 448, 300), rng.normal(0, 1, 300), rng.normal(0, 0.005, 200)]).astype(np.float32)
    for t in ts:
        T = Fraction(float(t))
        lo = max(g for g in grid if g <= T)
        hi = min(g for g in grid if g >= T)
        if lo == hi:
            continue
        P = (T - lo) / (hi - lo) * 2 ** 24        # up iff u24 < P, exactly
        k = -(-P.numerator // P.denominator)      # ceil(P): thresholds 0 .. k-1 go up, k .. 2^24-1 stay
        for u, up in ((0, k > 0), (k - 1, True), (k, False), (2 ** 24 - 1, False)):
            if 0 <= u < 2 ** 24:
                v = Fraction(float(oracle.e4m3_decode([oracle.quantize_e4m3_scalar(float(t), 1.0, SR, u)])[0]))
                assert v == (hi if up else lo), (float(t), u)


def test_scale_rule_keeps_every_quotient_within_448():
    rng = np.random.default_rng(3)
    for m in rng.uniform(1e-3, 100, 500).astype(np.float32):
        d, inv = oracle.scale_e4m3(float(m))
        exact = Fraction(448) / Fraction(float(m))
        assert Fraction(float(inv)) <= exact < Fraction(float(np.nextafter(inv, np.float32(np.inf))))
        assert d == np.float32(m) / np.float32(448) and np.float32(m) * inv <= 448
    assert oracle.scale_e4m3(0.0) == (0, 0) and oracle.scale_e4m3(1e-38) == (0, 0)


def _restate(x, inv, sr, u24):
    """Def. 1 with the local step, in exact rationals (independent of the oracle's arithmetic)."""
    grid = _grid()
    out = np.zeros(x.shape)
    for idx in np.ndindex(x.shape):
        T = Fraction(float(np.float32(x[idx] * np.float32(inv[idx]))))
        lo = max(g for g in grid if g <= T)
        hi = min(g for g in grid if g >= T)
        if lo == hi:
            out[idx] = float(lo)
            continue
        p = (T - lo) / (hi - lo)
        up = Fraction(int(u24[idx]), 2 ** 24) < p if sr else p >= Fraction(1, 2)
        out[idx] = float(hi if up else lo)
    return out


def test_matrix_quantizer_matches_the_restatement_in_both_layouts():
    rng = np.random.default_rng(4)
    x = (rng.normal(0, 1, (9, 14)) * rng.choice([1, 1, 30], (9, 14))).astype(np.float32)
    x[2] = 0
    for mode in (PER_TENSOR, PER_ROW):
        for rnd in (SR, RTN):
            q = QSpec(8, mode, rnd, seed=7, tensor_id=3, index_offset=5)
            crm, srm, ctr, stt = oracle.sr_quantize_e4m3(x, q, True, True)
            u = thresholds_u24(7, 3, 5, 9, 14)
            m_rows = np.abs(x).max(axis=1) if mode == PER_ROW else np.full(9, np.abs(x).max())
            m_cols = np.abs(x).max(axis=0) if mode == PER_ROW else np.full(14, np.abs(x).max())
            inv_r = np.array([oracle.scale_e4m3(float(m))[1] for m in m_rows], dtype=np.float32)
            inv_c = np.array([oracle.scale_e4m3(float(m))[1] for m in m_cols], dtype=np.float32)
            want_rm = _restate(x, np.repeat(inv_r[:, None], 14, 1), rnd == SR, u)
            want_tr = _restate(x, np.repeat(inv_c[None, :], 9, 0), rnd == SR, u)
            assert np.array_equal(oracle.e4m3_decode(crm), want_rm)
            assert np.array_equal(oracle.e4m3_decode(ctr), want_tr.T)
            d_r = np.array([oracle.scale_e4m3(float(m))[0] for m in m_rows], dtype=np.float32)
            assert np.array_equal(srm, d_r if mode == PER_ROW else d_r[:1])


def test_sr_is_unbiased_on_the_e4m3_grid():
    rng = np.random.default_rng(5)
    x = rng.normal(0, 1, (1, 512)).astype(np.float32)
    draws = 2000
    acc = np.zeros((1, 512))
    for seed in range(draws):
        c, s, _, _ = oracle.sr_quantize_e4m3(x, QSpec(8, PER_TENSOR, SR, seed, 1))
        acc += oracle.e4m3_decode(c)
    d, inv = oracle.scale_e4m3(float(np.abs(x).max()))
    t = x.astype(np.float64) * float(inv)
    step = 2.0 ** (np.maximum(np.floor(np.log2(np.abs(t))), -6) - 3)
    p = t / step - np.floor(t / step)
    sigma = step * np.sqrt(p * (1 - p) / draws)
    assert np.all(np.abs(acc / draws - t) <= 5 * sigma + 1e-12)


def test_product_is_the_binary64_matmul_of_the_decoded_codes():
    rng = np.random.default_rng(6)
    a = rng.choice(FINITE, (7, 33)).astype(np.uint8)
    b = rng.choice(FINITE, (5, 33)).astype(np.uint8)
    s_row = rng.uniform(0.5, 2, 7).astype(np.float32)
    s_col = rng.uniform(0.5, 2, 1).astype(np.float32)
    acc, out = oracle.gemm_e4m3_nt(a, b, s_row, s_col)
    want = oracle.e4m3_decode(a) @ oracle.e4m3_decode(b).T
    assert np.array_equal(acc, want)            # sums of this length are exact in binary64
    assert np.array_equal(out, want * (s_row[:, None] * s_col[None, :]).astype(np.float32).astype(np.float64))


# ---------------------------------------------------------------------------------------------
# E4M2, E4M1, E4M0: the E4M3 values with fewer mantissa bits (same exponent field and bias)
# ---------------------------------------------------------------------------------------------
import pytest


def _grid_k(k):
    """Sorted finite values of a format with 1 sign, 4 exponent (bias 7) and k mantissa bits,
    subnormals at exponent field 0, written from that definition (no oracle code).  For k = 3 the
    all-ones code is NaN and is left out."""
    vals = set()
    for ex in range(16):
        for man in range(2 ** k):
            if k == 3 and ex == 15 and man == 7:
                continue
            v = Fraction(man, 2 ** k) * Fraction(1, 64) if ex == 0 else (1 + Fraction(man, 2 ** k)) * Fraction(2) ** (ex - 7)
            vals.add(v)
            vals.add(-v)
    return sorted(vals)


@pytest.mark.parametrize("k", [0, 1, 2, 3])
def test_narrow_grids_are_subsets_of_e4m3_with_the_stated_maxima(k):
    g3, gk = set(_grid_k(3)), _grid_k(k)
    assert set(gk) <= g3                                  # every value has an E4M3 code
    assert max(gk) == Fraction(oracle.e4m_max(k)) == {0: 256, 1: 384, 2: 448, 3: 448}[k]
    # grid values never move, whatever the threshold, and their codes have the low mantissa bits clear
    for v in gk:
        for u in (0, 2 ** 23, 2 ** 24 - 1):
            c = oracle.quantize_e4m_scalar(float(v), 1.0, k, SR, u)
            assert Fraction(float(oracle.e4m3_decode([c])[0])) == v and (c & ((1 << (3 - k)) - 1)) == 0
        assert Fraction(float(oracle.e4m3_decode([oracle.quantize_e4m_scalar(float(v), 1.0, k, RTN)])[0])) == v


@pytest.mark.parametrize("k", [0, 1, 2])
def test_narrow_grids_round_to_a_neighbour_with_the_exact_probability(k):
    grid = _grid_k(k)
    top = float(max(grid))
    rng = np.random.default_rng(10 + k)
    ts = np.concatenate([rng.uniform(-top, top, 300), rng.normal(0, 1, 300), rng.normal(0, 0.01, 200)]).astype(np.float32)
    for t in ts:
        T = Fraction(float(t))
        lo = max(g for g in grid if g <= T)
        hi = min(g for g in grid if g >= T)
        if lo == hi:
            continue
        P = (T - lo) / (hi - lo) * 2 ** 24
        kk = -(-P.numerator // P.denominator)          # ceil(P): thresholds 0 .. kk-1 go up
        for u, up in ((0, kk > 0), (kk - 1, True), (kk, False), (2 ** 24 - 1, False)):
            if 0 <= u < 2 ** 24:
                v = Fraction(float(oracle.e4m3_decode([oracle.quantize_e4m_scalar(float(t), 1.0, k, SR, u)])[0]))
                assert v == (hi if up else lo), (k, float(t), u)
        # Def. 2: the nearer neighbour, the upper one at a tie
        v = Fraction(float(oracle.e4m3_decode([oracle.quantize_e4m_scalar(float(t), 1.0, k, RTN)])[0]))
        assert v == (hi if (T - lo) >= (hi - T) else lo), (k, float(t))


@pytest.mark.parametrize("k", [0, 1, 2])
def test_narrow_grid_scale_rule_and_matrix_form(k):
    top = oracle.e4m_max(k)
    rng = np.random.default_rng(20 + k)
    for m in rng.uniform(1e-3, 100, 200).astype(np.float32):
        d, inv = oracle.scale_e4m(float(m), k)
        exact = Fraction(top) / Fraction(float(m))
        assert Fraction(float(inv)) <= exact < Fraction(float(np.nextafter(inv, np.float32(np.inf))))
        assert d == np.float32(m) / np.float32(top) and np.float32(m) * inv <= top
    assert oracle.scale_e4m(0.0, k) == (0, 0)
    # matrix form against the restatement in exact rationals, both layouts, per row
    grid = _grid_k(k)
    x = (rng.normal(0, 1, (7, 10)) * rng.choice([1, 1, 30], (7, 10))).astype(np.float32)
    x[3] = 0
    q = QSpec(5 + k, PER_ROW, SR, seed=5, tensor_id=2, index_offset=9)
    crm, srm, ctr, stt = oracle.sr_quantize_e4m3(x, q, True, True)
    u = thresholds_u24(5, 2, 9, 7, 10)
    for codes, maxima, axis in ((crm, np.abs(x).max(axis=1), 0), (ctr.T, np.abs(x).max(axis=0), 1)):
        for idx in np.ndindex(x.shape):
            inv = oracle.scale_e4m(float(maxima[idx[axis]]), k)[1]
            T = Fraction(float(np.float32(x[idx] * np.float32(inv))))
            lo = max(g for g in grid if g <= T)
            hi = min(g for g in grid if g >= T)
            want = lo if lo == hi or not Fraction(int(u[idx]), 2 ** 24) < (T - lo) / (hi - lo) else hi
            assert Fraction(float(oracle.e4m3_decode([codes[idx]])[0])) == want
    assert np.array_equal(srm, np.array([oracle.scale_e4m(float(m), k)[0] for m in np.abs(x).max(axis=1)], dtype=np.float32))


def test_sr_is_unbiased_on_e4m1():
    rng = np.random.default_rng(31)
    x = rng.normal(0, 1, (1, 256)).astype(np.float32)
    draws = 2000
    acc = np.zeros((1, 256))
    for seed in range(draws):
        c, s, _, _ = oracle.sr_quantize_e4m3(x, QSpec(6, PER_TENSOR, SR, seed, 1))
        acc += oracle.e4m3_decode(c)
    d, inv = oracle.scale_e4m(float(np.abs(x).max()), 1)
    t = x.astype(np.float64) * float(inv)
    step = 2.0 ** (np.maximum(np.floor(np.log2(np.abs(t))), -6) - 1)
    p = t / step - np.floor(t / step)
    sigma = step * np.sqrt(p * (1 - p) / draws)
    assert np.all(np.abs(acc / draws - t) <= 5 * sigma + 1e-12)
