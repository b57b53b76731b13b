"""Restatements used only by the tests to pin the oracle from outside.

Nothing here is imported by the oracle or by the CUDA package.  The Philox
below is written from the algorithm's published description (vectorised with
numpy uint64 so whole matrices of thresholds can be produced); the quantizer
is Def. 1-3 written with numpy binary32 scalars and exact rationals.
"""
from fractions import Fraction

import numpy as np

M0, M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
W0, W1 = 0x9E3779B9, 0xBB67AE85
MASK = np.uint64(0xFFFFFFFF)
S32 = np.uint64(32)


def philox_np(c0, c1, c2, c3, k0, k1):
    """Vectorised Philox4x32-10; counters are uint64 arrays holding 32-bit words."""
    c0, c1, c2, c3 = [np.asarray(c, dtype=np.uint64) for c in (c0, c1, c2, c3)]
    k0, k1 = int(k0), int(k1)
    for _ in range(10):
        p0 = M0 * c0
        p1 = M1 * c2
        n0 = (p1 >> S32) ^ c1 ^ np.uint64(k0)
        n2 = (p0 >> S32) ^ c3 ^ np.uint64(k1)
        c0, c1, c2, c3 = n0 & MASK, p1 & MASK, n2 & MASK, p0 & MASK
        k0 = (k0 + W0) & 0xFFFFFFFF
        k1 = (k1 + W1) & 0xFFFFFFFF
    return c0, c1, c2, c3


def thresholds_u24(seed, tensor_id, index_offset, rows, cols):
    """u24 of every element of a [rows, cols] tensor, by flat row-major index."""
    i = (np.arange(rows * cols, dtype=np.uint64) + np.uint64(index_offset)).reshape(rows, cols)
    j = i >> np.uint64(2)
    words = philox_np(j & MASK, j >> S32, np.full_like(j, tensor_id & 0xFFFFFFFF),
                      np.full_like(j, (tensor_id >> 32) & 0xFFFFFFFF),
                      seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    sel = (i & np.uint64(3)).astype(np.int64)
    stacked = np.stack(words, axis=0)
    r = np.take_along_axis(stacked, sel[None, ...], axis=0)[0]
    return (r >> np.uint64(8)).astype(np.int64)


def qmax_of(bits):
    return 2 ** (bits - 1) - 1


def scale_ref(m, bits):
    """(Delta, 1/Delta) by the absmax rule: Delta one binary32 division rounded to nearest, the
    reciprocal the largest binary32 number not above qmax / m (found with exact rationals)."""
    m = np.float32(m)
    q = np.float32(qmax_of(bits))
    if m == 0:
        return np.float32(0), np.float32(0)
    with np.errstate(over="ignore"):
        inv = q / m
    if not np.isfinite(inv):
        return np.float32(0), np.float32(0)
    exact = Fraction(int(q)) / Fraction(float(m))
    while Fraction(float(inv)) > exact:
        inv = np.nextafter(inv, np.float32(0))
    while Fraction(float(np.nextafter(inv, np.float32(np.inf)))) <= exact:
        inv = np.nextafter(inv, np.float32(np.inf))
    return np.float32(m / q), np.float32(inv)


def quantize_scalar_ref(x, inv, bits, sr, u24=0):
    """Def. 1 for one element: t in binary32, everything after it in exact rationals."""
    t = Fraction(float(np.float32(np.float32(x) * np.float32(inv))))
    f = t.numerator // t.denominator
    p = t - f
    if sr:
        up = Fraction(int(u24), 2 ** 24) < p
    else:
        up = p >= Fraction(1, 2)
    q = int(f) + int(up)
    return max(-qmax_of(bits), min(qmax_of(bits), q))


def quantize_matrix_ref(x, inv, bits, sr, u24):
    """Def. 1 over a matrix with a broadcastable inv: t in binary32, the threshold comparison in
    exact rationals (slow; for the small matrices of the tests)."""
    x = np.asarray(x, dtype=np.float32)
    t = (x * np.asarray(inv, dtype=np.float32)).astype(np.float32)
    out = np.empty(t.shape, dtype=np.int64)
    flat_t = t.ravel()
    flat_u = None if u24 is None else np.asarray(u24).ravel()
    o = out.ravel()
    for i in range(flat_t.size):
        T = Fraction(float(flat_t[i])) * 2 ** 24            # exact
        f = T.numerator // (T.denominator * 2 ** 24)          # floor(t)
        P = T - f * 2 ** 24                                    # p * 2^24, exact
        if sr:
            up = int(flat_u[i]) < P
        else:
            up = P >= 2 ** 23
        o[i] = f + int(up)
    return np.clip(out, -qmax_of(bits), qmax_of(bits)).astype(np.int8)
