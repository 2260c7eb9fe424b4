"""Pins of the oracle's bfloat16 conversions (oracle/bf16_oracle.c), CPU only.

bfloat16 is the upper half of an IEEE-754 binary32: 1 sign, 8 exponent (bias 127), 7 fraction bits.  The
conversions are checked against bit patterns written out by hand from that definition, against invariants that
hold for every pattern, and against exactly constructed midpoints; a dropped tie rule, a wrong bias, a
mishandled subnormal or an off-by-one at a binade boundary each fail at least one of them.
"""
import math

import numpy as np

import oracle


def test_hand_written_bit_patterns():
    cases = [
        (1.0, 0x3F80), (-1.0, 0xBF80), (2.0, 0x4000), (0.5, 0x3F00), (1.5, 0x3FC0),
        (0.0, 0x0000), (-0.0, 0x8000),
        (1.0 + 2.0 ** -7, 0x3F81),                     # one ulp above 1
        (1.0 + 2.0 ** -8, 0x3F80),                     # tie between 0x3F80 (even) and 0x3F81: down
        (1.0 + 3 * 2.0 ** -8, 0x3F82),                 # tie between 0x3F81 and 0x3F82 (even): up
        (1.0 + 2.0 ** -8 + 2.0 ** -40, 0x3F81),        # just above the tie
        (1.0 + 3 * 2.0 ** -8 - 2.0 ** -40, 0x3F81),    # just below the tie
        (2.0 - 2.0 ** -8, 0x4000),                     # tie at the top of a binade: up to 2.0 (even)
        (2.0 - 2.0 ** -7, 0x3FFF),                     # the largest value below 2
        (-(1.0 + 3 * 2.0 ** -8), 0xBF82),              # ties are symmetric in sign
        (3.0e38, 0x7F62),                              # 3e38 = 1.7632 * 2^127 -> fraction 0.7656 = 98/128
        ((2.0 - 2.0 ** -7) * 2.0 ** 127, 0x7F7F),      # largest finite
        ((2.0 - 2.0 ** -8) * 2.0 ** 127, 0x7F80),      # the midpoint to 2^128: ties to even = overflow
        ((2.0 - 2.0 ** -8) * 2.0 ** 127 * (1 - 2.0 ** -30), 0x7F7F),
        (1e39, 0x7F80), (-1e39, 0xFF80), (math.inf, 0x7F80), (-math.inf, 0xFF80),
        (2.0 ** -126, 0x0080),                         # smallest normal
        (2.0 ** -133, 0x0001),                         # smallest subnormal
        (2.0 ** -134, 0x0000),                         # half of it: tie to even = 0
        (1.5 * 2.0 ** -134, 0x0001),
        (3 * 2.0 ** -134, 0x0002),                     # 1.5 quanta: tie between 1 and 2 -> 2
        (127.5 * 2.0 ** -133, 0x0080),                 # tie between the largest subnormal (odd) and the smallest normal
        (1e-45, 0x0000),
    ]
    for x, want in cases:
        got = oracle.double_to_bf16(x)
        assert got == want, (x, hex(got), hex(want))
    assert oracle.double_to_bf16(math.nan) & 0x7FFF == 0x7FC0
    assert oracle.bf16_to_double(0x3F80) == 1.0 and oracle.bf16_to_double(0xC000) == -2.0
    assert oracle.bf16_to_double(0x0001) == 2.0 ** -133 and oracle.bf16_to_double(0x7F7F) == (2.0 - 2.0 ** -7) * 2.0 ** 127
    assert math.isinf(oracle.bf16_to_double(0x7F80)) and math.isnan(oracle.bf16_to_double(0x7FC1))


def test_every_bit_pattern_survives_the_round_trip_and_is_its_binary32_upper_half():
    bits = np.arange(65536, dtype=np.uint16)
    wide = oracle.bf16_widen(bits)
    # the defining property of the format: the pattern is the upper half of the binary32 of the same value
    finite = np.isfinite(wide)
    as32 = (bits.astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(wide[finite], as32[finite])
    back = oracle.bf16_round(wide.astype(np.float64))
    nan = np.isnan(wide)
    assert np.array_equal(back[~nan], bits[~nan])
    assert np.all((back[nan] & 0x7FFF) == 0x7FC0)


def test_midpoints_go_to_the_even_neighbour_and_rounding_is_monotone():
    pos = np.arange(0x0000, 0x7F80, dtype=np.uint16)  # every non-negative finite pattern, ascending in value
    lo = oracle.bf16_widen(pos).astype(np.float64)
    hi = np.append(lo[1:], 2.0 ** 128)
    mid = (lo + hi) / 2  # exact: neighbours differ in at most the last of 9 significant bits
    got = oracle.bf16_round(mid)
    want = np.where(pos % 2 == 0, pos, pos + 1).astype(np.uint16)  # the even fraction (0x7F80 = overflow at the top)
    assert np.array_equal(got, want)
    below = np.nextafter(mid, 0.0)
    above = np.nextafter(mid, np.inf)
    assert np.array_equal(oracle.bf16_round(below), pos)
    assert np.array_equal(oracle.bf16_round(above), (pos + 1).astype(np.uint16))
    assert np.array_equal(oracle.bf16_round(-mid), want | 0x8000)
    rng = np.random.default_rng(1)
    x = np.sort(np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-40, 39, 20000), mid[::97]]))
    r = oracle.bf16_widen(oracle.bf16_round(x)).astype(np.float64)
    assert np.all(np.diff(r) >= 0)
    ok = np.abs(x) < 3.38e38
    assert np.all(np.abs(r[ok] - x[ok]) <= np.maximum(np.abs(x[ok]) * 2.0 ** -8, 2.0 ** -134))


def test_bf16_encode_and_decode_are_the_fp64_formulas_on_the_widened_values_rounded_once():
    rng = np.random.default_rng(3)
    K, W, G, D = 4, 6, 3, 5
    Xb = oracle.bf16_round(rng.standard_normal((G, K, D)))
    exact, rounded = oracle.encode_bf16(K, W, Xb)
    # constants are reproduced exactly (partition of unity) and survive the rounding
    const = np.full((1, K, 2), oracle.double_to_bf16(0.3359375), dtype=np.uint16)  # 43/128: a bfloat16 value
    ce, cr = oracle.encode_bf16(K, W, const)
    assert np.all(np.abs(ce - 0.3359375) < 1e-15) and np.all(cr == const[0, 0, 0])
    assert np.array_equal(rounded, oracle.bf16_round(exact))
    assert np.array_equal(exact, oracle.encode(K, W, oracle.bf16_widen(Xb)))
    mask = np.array([0b111111, 0b101101, 0b011110], dtype=np.uint32)
    Yb = oracle.bf16_round(rng.standard_normal((G, W, 7)))
    de, dr, n_used, status = oracle.decode_bf16(K, W, Yb, mask)
    ref, n_ref, st_ref = oracle.decode(K, W, oracle.bf16_widen(Yb), mask)
    assert np.array_equal(de, ref) and np.array_equal(n_used, n_ref) and np.array_equal(dr, oracle.bf16_round(ref))
