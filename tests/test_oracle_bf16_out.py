"""Pins of the oracle's bfloat16 rounding of a product's results, from outside the oracle: torch's
cast (a library routine), the format's definition in exact rationals, and the tie table."""
from fractions import Fraction

import numpy as np
import torch

import oracle


def _decode(bits):
    return (np.asarray(bits, dtype=np.uint32) << 16).view(np.float32)


def test_matches_the_library_cast_on_random_values_and_every_tie():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(0, 1, 200000), rng.normal(0, 1e-6, 50000), rng.normal(0, 1e6, 50000)]).astype(np.float32)
    # exact ties: every bfloat16 pattern of a few binades with the discarded half set to 0x8000
    keep = np.arange(0x3F00, 0x4100, dtype=np.uint32)
    ties = np.concatenate([(keep << 16) | 0x8000, (keep << 16) | 0x80008000]).astype(np.uint32).view(np.float32)
    x = np.concatenate([x, ties, np.float32([0.0, -0.0, 1.0, -1.0, 3.3895314e38])])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.uint16).numpy()
    assert np.array_equal(oracle.to_bf16(x), want)


def test_result_is_the_nearer_neighbour_and_ties_go_to_the_even_one():
    rng = np.random.default_rng(1)
    for v in rng.normal(0, 3, 400).astype(np.float32):
        got = Fraction(float(_decode(oracle.to_bf16([v]))[0]))
        lo_bits = np.float32(v).view(np.uint32) & np.uint32(0xFFFF0000)          # toward zero
        lo = Fraction(float(np.uint32(lo_bits).view(np.float32)))
        hi = Fraction(float(np.uint32(lo_bits + np.uint32(0x10000)).view(np.float32)))   # away from zero
        x = Fraction(float(v))
        assert got in (lo, hi) and abs(got - x) <= min(abs(lo - x), abs(hi - x))
    # 7 explicit mantissa bits: one unit in the last place at 1.0 is 2^-7
    table = {1 + 2.0 ** -8: 1.0, 1 + 3 * 2.0 ** -8: 1 + 2.0 ** -6, -(1 + 2.0 ** -8): -1.0,
             -(1 + 3 * 2.0 ** -8): -(1 + 2.0 ** -6), 1 + 2.0 ** -8 + 2.0 ** -20: 1 + 2.0 ** -7, 1 + 2.0 ** -8 - 2.0 ** -20: 1.0}
    for v, want in table.items():
        assert _decode(oracle.to_bf16([np.float32(v)]))[0] == np.float32(want)


def test_bfloat16_values_do_not_move():
    bits = np.arange(0, 0x7F80, 7, dtype=np.uint16)            # finite non-negative patterns
    assert np.array_equal(oracle.to_bf16(_decode(bits)), bits)
    assert np.array_equal(oracle.to_bf16(-_decode(bits)), bits | 0x8000)
