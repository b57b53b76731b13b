"""Pins for the oracle's integer products, dequantization and the three layer passes
(mixed-precision matmul subsection, Alg. 1, Alg. 2, and the variance lemma)."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import PER_ROW, PER_TENSOR, RTN, SR, QSpec
from _independent import scale_ref
from paper_2511_00874_b200 import synth


# ---------------------------------------------------------------- integer product
def test_gemm_brute_force_tiny_shapes():
    rng = np.random.default_rng(0)
    for (M, N, K) in [(1, 1, 1), (2, 3, 5), (3, 2, 7), (4, 4, 1), (5, 1, 9)]:
        a = rng.integers(-127, 128, (M, K)).astype(np.int8)
        b = rng.integers(-127, 128, (N, K)).astype(np.int8)
        acc = oracle.gemm_i8_nt(a, b)
        for i in range(M):
            for j in range(N):
                assert acc[i, j] == sum(int(a[i, k]) * int(b[j, k]) for k in range(K))


def test_gemm_special_cases_and_library_matmul():
    rng = np.random.default_rng(1)
    # all-ones codes: every entry equals the contraction length
    assert np.all(oracle.gemm_i8_nt(np.ones((5, 33), np.int8), np.ones((7, 33), np.int8)) == 33)
    # identity codes return the other operand (contracted axis last on both)
    b = rng.integers(-127, 128, (6, 9)).astype(np.int8)
    assert np.array_equal(oracle.gemm_i8_nt(np.eye(9, dtype=np.int8), b), b.T.astype(np.int32))
    # a library routine on odd shapes
    a = rng.integers(-127, 128, (37, 129)).astype(np.int8)
    b = rng.integers(-127, 128, (21, 129)).astype(np.int8)
    assert np.array_equal(oracle.gemm_i8_nt(a, b), a.astype(np.int64) @ b.astype(np.int64).T)
    # extreme codes at a long contraction stay inside int32 (65536 * 127^2 < 2^31) ...
    a = np.full((1, 65536), 127, np.int8)
    assert oracle.gemm_i8_nt(a, a)[0, 0] == 65536 * 127 * 127
    # ... and the first length that does not is reported, not wrapped
    a = np.full((1, 133145), 127, np.int8)
    with pytest.raises(OverflowError):
        oracle.gemm_i8_nt(a, a)


def test_dequant_is_two_binary32_multiplies():
    rng = np.random.default_rng(2)
    acc = rng.integers(-2 ** 30, 2 ** 30, (9, 11)).astype(np.int32)
    sr = rng.uniform(1e-3, 1, 9).astype(np.float32)
    sc = rng.uniform(1e-3, 1, 11).astype(np.float32)
    out = oracle.dequant(acc, sr, sc)
    # power-of-two scales make the product exact: only the int->float rounding remains
    out2 = oracle.dequant(acc, np.array([0.5], np.float32), np.array([0.25], np.float32))
    assert np.array_equal(out2, acc.astype(np.float32) * np.float32(0.125))
    # general scales: within 1.5 ulp of the real-number product, and equal to numpy binary32
    exact = acc.astype(np.float64) * sr.astype(np.float64)[:, None] * sc.astype(np.float64)[None, :]
    assert np.all(np.abs(out - exact) <= 1.5 * np.spacing(np.abs(out)))
    assert np.array_equal(out, acc.astype(np.float32) * (sr[:, None] * sc[None, :]))
    # per-tensor on one side, per-row on the other
    out3 = oracle.dequant(acc, sr[:1], sc)
    assert np.array_equal(out3, acc.astype(np.float32) * (sr[0] * sc)[None, :])


# ---------------------------------------------------------------- Alg. 1 and 2
def _inputs(T, N, K, seed=0, std_dy=1.0):
    A, W, dY = synth.layer_inputs(T, N, K, seed, torch.float32, "cpu", std_dy=std_dy)
    return A.numpy(), W.numpy(), dY.numpy()


@pytest.mark.parametrize("mode", [PER_TENSOR, PER_ROW])
def test_layer_passes_compose_quantizer_product_and_dequant(mode):
    T, N, K = 12, 10, 20          # three different extents: a transposed operand cannot pass
    A, W, dY = _inputs(T, N, K)
    qa = QSpec(8, mode, SR, 5, 0)
    qw = QSpec(8, mode, SR, 5, 1)
    qdy = QSpec(6, mode, SR, 5, 4)

    f = oracle.qlinear_fwd(A, W, qa, qw)
    ca, sa, _, _ = oracle.sr_quantize(A, qa)
    cw, sw, cwt, swt = oracle.sr_quantize(W, qw, True, True)
    assert np.array_equal(f.codes_a, ca) and np.array_equal(f.codes_b, cw)
    assert np.array_equal(f.acc, ca.astype(np.int64) @ cw.astype(np.int64).T)
    assert np.array_equal(f.out, oracle.dequant(f.acc, sa, sw))

    bi = oracle.qlinear_bwd_input(dY, W, qdy, qw)
    cdy, sdy, cdyt, sdyt = oracle.sr_quantize(dY, qdy, True, True)
    assert np.array_equal(bi.codes_a, cdy) and np.array_equal(bi.codes_b, cwt)
    assert bi.acc.shape == (T, K)
    assert np.array_equal(bi.acc, cdy.astype(np.int64) @ cwt.astype(np.int64).T)
    assert np.array_equal(bi.out, oracle.dequant(bi.acc, sdy, swt))
    if mode == PER_TENSOR:     # one W-hat serves forward and backward when (seed, id) agree
        assert np.array_equal(cwt, cw.T)

    bw = oracle.qlinear_bwd_weight(dY, A, qdy, qa)
    _, _, cat, sat = oracle.sr_quantize(A, qa, False, True)
    assert np.array_equal(bw.codes_a, cdyt) and np.array_equal(bw.codes_b, cat)
    assert bw.acc.shape == (N, K)
    assert np.array_equal(bw.acc, cdyt.astype(np.int64) @ cat.astype(np.int64).T)
    assert np.array_equal(bw.out, oracle.dequant(bw.acc, sdyt, sat))


@pytest.mark.parametrize("mode", [PER_TENSOR, PER_ROW])
def test_layer_outputs_approach_the_unquantized_products(mode):
    """A-hat B-hat approximates A B (mixed-precision matmul subsection): the error of each
    output entry is bounded by the worst-case rounding of its operands."""
    T, N, K = 24, 18, 40
    A, W, dY = _inputs(T, N, K, seed=1)
    A64, W64, dY64 = A.astype(np.float64), W.astype(np.float64), dY.astype(np.float64)
    for rnd, width in ((SR, 1.0), (RTN, 0.5)):
        qa, qw, qdy = QSpec(8, mode, rnd, 1, 0), QSpec(8, mode, rnd, 1, 1), QSpec(8, mode, rnd, 1, 2)

        def bound(X, Y, sx, sy):
            # |x y - xh yh| <= |x| ey + |y| ex + ex ey, summed along the contraction
            ex = width * sx.astype(np.float64) * (1 + 1e-5)
            ey = width * sy.astype(np.float64) * (1 + 1e-5)
            ex = ex.reshape(-1, 1) if ex.size > 1 else ex.reshape(1, 1)
            ey = ey.reshape(1, -1) if ey.size > 1 else ey.reshape(1, 1)
            L = X.shape[1]
            return (np.abs(X).sum(1)[:, None] * ey + ex * np.abs(Y).sum(1)[None, :] + L * ex * ey)

        f = oracle.qlinear_fwd(A, W, qa, qw)
        assert np.all(np.abs(f.out - A64 @ W64.T) <= bound(A64, W64, f.scale_a, f.scale_b) + 1e-6)
        bi = oracle.qlinear_bwd_input(dY, W, qdy, qw)
        assert np.all(np.abs(bi.out - dY64 @ W64)
                      <= bound(dY64, W64.T, bi.scale_a, bi.scale_b) + 1e-6)
        bw = oracle.qlinear_bwd_weight(dY, A, qdy, qa)
        assert np.all(np.abs(bw.out - dY64.T @ A64)
                      <= bound(dY64.T, A64.T, bw.scale_a, bw.scale_b) + 1e-6)


def test_weight_gradient_is_unbiased_and_its_variance_follows_the_lemma():
    """E[dW_q] = dY^T A (error-decomposition lemma: the cross term vanishes) and
    Var(dW_q[n,k]) = sum_t (A^2 s_dY^2 + dY^2 s_A^2 + s_A^2 s_dY^2) with the per-element SR
    variances s^2 = D^2 p (1 - p) <= D^2 (proof of the batch-size lemma)."""
    T, N, K = 48, 6, 5
    A, W, dY = _inputs(T, N, K, seed=2)
    bits = 4
    draws = 3000
    outs = np.zeros((draws, N, K))
    for seed in range(draws):
        r = oracle.qlinear_bwd_weight(dY, A, QSpec(bits, PER_TENSOR, SR, seed, 4),
                                      QSpec(bits, PER_TENSOR, SR, seed, 2))
        outs[seed] = r.out
    exact = dY.astype(np.float64).T @ A.astype(np.float64)

    def elem_var(X):
        d, inv = scale_ref(np.abs(X).max(), bits)
        t = X.astype(np.float64) * float(inv)
        p = t - np.floor(t)
        return float(d) ** 2 * p * (1 - p), float(d)

    vA, dA_ = elem_var(A)
    vY, dY_ = elem_var(dY)
    # the quantized values are unbiased for x * (inv * D), which is x up to 2^-23 relative
    pred = (dY.astype(np.float64) ** 2).T @ vA + vY.T @ (A.astype(np.float64) ** 2) + vY.T @ vA
    mean = outs.mean(0)
    var = outs.var(0)
    assert np.all(np.abs(mean - exact) <= 5 * np.sqrt(pred / draws) + 1e-4)
    # variance estimate: relative sd about sqrt(2/draws) ~ 2.6 %; allow 6 sd
    assert np.all(np.abs(var / pred - 1) < 6 * math.sqrt(2.0 / draws) + 0.02)
    # the lemma's bound with s^2 <= D^2
    bound = (A.astype(np.float64) ** 2).sum(0)[None, :] * dY_ ** 2 \
        + (dY.astype(np.float64) ** 2).sum(0)[:, None] * dA_ ** 2 + T * dA_ ** 2 * dY_ ** 2
    assert np.all(var <= bound)


def test_one_bit_less_costs_about_four_times_the_variance():
    """The 2^-2B factor of the batch-size lemma: dropping a bit multiplies the SR variance of
    dW by (qmax_b / qmax_{b-1})^2, about 4 (4.06 for 8 -> 7 bits)."""
    T, N, K = 64, 4, 4
    A, W, dY = _inputs(T, N, K, seed=3)
    draws = 1500
    v = {}
    for bits in (8, 7):
        outs = np.zeros((draws, N, K))
        for seed in range(draws):
            outs[seed] = oracle.qlinear_bwd_weight(dY, A, QSpec(bits, PER_TENSOR, SR, seed, 4),
                                                   QSpec(bits, PER_TENSOR, SR, seed, 2)).out
        v[bits] = outs.var(0).mean()
    ratio = v[7] / v[8]
    assert abs(ratio - (127 / 63) ** 2) < 0.6


def test_forward_with_unquantized_activations_reduces_to_known_cases():
    """Sec. 3.3 variant (D_A^fwd = 0): unit-vector activations read out the dequantized weight, and
    activations that already lie on the 8-bit grid give what the fully quantized forward gives."""
    rng = np.random.default_rng(11)
    W = rng.normal(0, 0.02, (12, 16)).astype(np.float32)
    qw = QSpec(8, PER_ROW, SR, 3, 1)
    eye = np.eye(16, dtype=np.float32)
    r = oracle.qlinear_fwd_fp_act(eye, W, qw)
    cw, sw, _, _ = oracle.sr_quantize(W, qw)
    assert np.array_equal(r.out, (cw.astype(np.float64) * sw.astype(np.float64)[:, None]).T)
    A = rng.integers(-127, 128, (9, 16)).astype(np.float32)
    A[0, 0] = 127                                   # absmax 127: step size 1, codes = A
    full = oracle.qlinear_fwd(A, W, QSpec(8, PER_TENSOR, RTN), qw)
    assert full.scale_a[0] == 1 and np.array_equal(full.codes_a, A.astype(np.int8))
    part = oracle.qlinear_fwd_fp_act(A, W, qw)
    assert np.array_equal(part.acc, full.acc.astype(np.float64))
    assert np.array_equal(part.out.astype(np.float32), full.out)


def test_requantization_of_an_output_with_a_supplied_step():
    from fractions import Fraction
    from _independent import thresholds_u24
    rng = np.random.default_rng(12)
    out = (rng.normal(0, 3, (11, 20))).astype(np.float32)
    out[0, :5] = [1000.0, -1000.0, 31.75, -31.75, 0.0]          # far outside, and on the edge of, the range
    step = np.float32(0.25)
    for bits, rnd in ((8, SR), (8, RTN), (4, SR)):
        q = QSpec(bits, PER_TENSOR, rnd, seed=9, tensor_id=4, index_offset=6)
        codes, m = oracle.requantize(out, float(step), q)
        assert m == np.abs(out).max()
        qmax = 2 ** (bits - 1) - 1
        u = thresholds_u24(9, 4, 6, 11, 20)
        inv = np.float32(1) / step
        for idx in np.ndindex(out.shape):                      # Def. 1 in exact rationals after saturation
            t = Fraction(float(np.float32(out[idx] * inv)))
            t = max(Fraction(-qmax), min(Fraction(qmax), t))
            f = t.numerator // t.denominator
            p = t - f
            up = (Fraction(int(u[idx]), 2 ** 24) < p) if rnd == SR else (p >= Fraction(1, 2))
            assert codes[idx] == f + int(up), idx
        assert codes[0, 0] == qmax and codes[0, 1] == -qmax and codes[0, 4] == 0
    # grid values with a power-of-two step are reproduced; a zero step gives zero codes
    grid = (rng.integers(-127, 128, (5, 8)) * 0.5).astype(np.float32)
    codes, _ = oracle.requantize(grid, 0.5, QSpec(8, PER_TENSOR, SR, 1, 1))
    assert np.array_equal(codes, (grid * 2).astype(np.int8))
    assert not oracle.requantize(grid, 0.0, QSpec(8, PER_TENSOR, SR, 1, 1))[0].any()
    # accumulation is one binary32 addition per element
    a, b = rng.normal(0, 1, 50).astype(np.float32), rng.normal(0, 1e-3, 50).astype(np.float32)
    assert np.array_equal(oracle.accumulate(a, b), a + b)
