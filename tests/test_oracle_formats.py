"""Pins for the oracle's FP8 decode and encode (CPU only).

What fixes the expected values here: the ranges the paper prints (tests/golden/
paper_constants.txt), PyTorch's float8 dtypes as an outside opinion on the bit layout and
on in-range rounding, exact rational arithmetic for ties, and the two independent search
strategies inside the oracle (every code vs bisection).
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import mor_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def load_constants():
    out = {}
    with open(GOLD) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if line:
                k, v = line.split(None, 1)
                out[k] = eval(v, {"__builtins__": {}})  # exact expressions like 2**-9
    return out


K = load_constants()
E4 = [orc.decode_e4m3(c) for c in range(256)]
E5 = [orc.decode_e5m2(c) for c in range(256)]


def finite(vals):
    return [v for v in vals if np.isfinite(v)]


def test_decode_ranges_match_the_paper():
    pos4 = [v for v in finite(E4) if v > 0]
    pos5 = [v for v in finite(E5) if v > 0]
    assert min(pos4) == K["e4m3_min_positive"] and max(pos4) == K["e4m3_max"]
    assert min(pos5) == K["e5m2_min_positive"] and max(pos5) == K["e5m2_max"]
    # smallest normal of E5M2 = value of exponent field 1, mantissa 0
    assert orc.decode_e5m2(0b0_00001_00) == K["e5m2_min_normal"]
    assert K["eq4_range_bound"] == 939524096


def test_decode_counts_and_specials():
    assert len(finite(E4)) == 254 and len(finite(E5)) == 248
    assert np.isnan(E4[0x7F]) and np.isnan(E4[0xFF])
    assert E5[0x7C] == np.inf and E5[0xFC] == -np.inf
    assert all(np.isnan(E5[c]) for c in (0x7D, 0x7E, 0x7F, 0xFD, 0xFE, 0xFF))
    # sign symmetry and strict monotonicity over the non-negative finite codes
    for tab, n in ((E4, 127), (E5, 124)):
        assert all(tab[c + 1] > tab[c] for c in range(n - 1))
        assert all(tab[c | 0x80] == -tab[c] for c in range(n))
        assert np.signbit(tab[0x80]) and tab[0x80] == 0


def test_decode_matches_torch_float8_layout():
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    t4 = codes.view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    t5 = codes.view(torch.float8_e5m2).float().numpy().astype(np.float64)
    np.testing.assert_array_equal(np.array(E4), t4)
    np.testing.assert_array_equal(np.array(E5), t5)


def test_bit_split_matches_the_paper():
    # mantissa bits = number of equal steps inside one binade
    assert sum(1 for v in finite(E4) if 1.0 <= v < 2.0) == 2 ** K["e4m3_mantissa_bits"]
    assert sum(1 for v in finite(E5) if 1.0 <= v < 2.0) == 2 ** K["e5m2_mantissa_bits"]
    # exponent bits = log2 of the number of distinct exponent fields
    assert len({c >> 3 & 15 for c in range(128)}) == 2 ** K["e4m3_exponent_bits"]
    assert len({c >> 2 & 31 for c in range(128)}) == 2 ** K["e5m2_exponent_bits"]


@pytest.mark.parametrize("enc,tab,n", [(orc.encode_e4m3, E4, 127), (orc.encode_e5m2, E5, 124)])
def test_encode_roundtrip_every_finite_code(enc, tab, n):
    for c in list(range(n)) + [c | 0x80 for c in range(n)]:
        assert enc(tab[c]) == c
        assert enc(tab[c], exhaustive=True) == c


@pytest.mark.parametrize("enc,tab,n", [(orc.encode_e4m3, E4, 127), (orc.encode_e5m2, E5, 124)])
def test_encode_midpoints_go_to_even_and_neighbours_to_nearer(enc, tab, n):
    for c in range(n - 1):
        mid = (Fraction(tab[c]) + Fraction(tab[c + 1])) / 2
        m32 = np.float32(float(mid))
        assert Fraction(float(m32)) == mid, "midpoints of adjacent FP8 values are binary32 numbers"
        even = c if c % 2 == 0 else c + 1
        for sgn, bit in ((1.0, 0), (-1.0, 0x80)):
            assert enc(float(sgn * m32)) == (even | bit)
            assert enc(float(sgn * m32), exhaustive=True) == (even | bit)
            lo = np.nextafter(m32, np.float32(0))
            hi = np.nextafter(m32, np.float32(np.inf))
            assert enc(float(sgn * lo)) == (c | bit)
            assert enc(float(sgn * hi)) == ((c + 1) | bit)


def test_encode_saturates_to_largest_finite():
    big = float(np.finfo(np.float32).max)
    for y in (448.0, float(np.nextafter(np.float32(448), np.float32(1e9))), 464.0, 480.0, 1e6, big, np.inf):
        assert orc.encode_e4m3(y) == 0x7E and orc.encode_e4m3(-y) == 0xFE
    for y in (57344.0, 61440.0, 65536.0, 1e9, big, np.inf):
        assert orc.encode_e5m2(y) == 0x7B and orc.encode_e5m2(-y) == 0xFB
    # just below the last midpoint still rounds down to the value before the largest
    assert orc.encode_e4m3(float(np.nextafter(np.float32(432), np.float32(0)))) == 0x7D
    assert orc.encode_e4m3(432.0) == 0x7E  # tie between 416 (0x7D, odd) and 448 (0x7E, even)


def test_encode_underflow_keeps_sign():
    tiny = float(np.float32(1e-30))
    assert orc.encode_e4m3(0.0) == 0x00 and orc.encode_e4m3(-0.0) == 0x80
    assert orc.encode_e4m3(tiny) == 0x00 and orc.encode_e4m3(-tiny) == 0x80
    assert orc.encode_e5m2(tiny) == 0x00 and orc.encode_e5m2(-tiny) == 0x80
    # half of the smallest positive value is a tie with zero: even code 0 wins
    assert orc.encode_e4m3(2.0 ** -10) == 0x00 and orc.encode_e4m3(float(np.nextafter(np.float32(2.0 ** -10), np.float32(1)))) == 0x01
    assert orc.encode_e5m2(2.0 ** -17) == 0x00 and orc.encode_e5m2(float(np.nextafter(np.float32(2.0 ** -17), np.float32(1)))) == 0x01


def test_encode_nan_is_canonical():
    assert orc.encode_e4m3(float("nan")) == 0x7F
    assert orc.encode_e5m2(float("nan")) == 0x7F


def test_bisection_equals_walk_over_every_code():
    rng = np.random.default_rng(7)
    ys = np.concatenate([
        (rng.standard_normal(20000) * 100).astype(np.float32),
        np.exp2(rng.uniform(-25, 17, 20000)).astype(np.float32) * rng.choice([-1, 1], 20000).astype(np.float32),
        # every BF16 pattern times two scales with full mantissas
        (np.arange(65536, dtype=np.uint32) << 16).view(np.float32) * np.float32(1.337),
        (np.arange(65536, dtype=np.uint32) << 16).view(np.float32) * np.float32(2.9e-3),
    ])
    ys = ys[np.isfinite(ys)]
    L = orc.lib()
    for y in ys[::3]:
        y = float(y)
        assert L.orc_encode_e4m3(y) == L.orc_encode_e4m3_exhaustive(y)
        assert L.orc_encode_e5m2(y) == L.orc_encode_e5m2_exhaustive(y)


def test_encode_matches_torch_cast_in_range():
    # PyTorch rounds binary32 -> float8 to nearest even; its overflow rule differs, so stay in range
    rng = np.random.default_rng(11)
    mag = np.exp2(rng.uniform(-12, np.log2(448), 30000))
    y4 = (mag * rng.choice([-1, 1], mag.size)).astype(np.float32)
    y4 = y4[np.abs(y4) <= 448]
    t4 = torch.from_numpy(y4).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    mag = np.exp2(rng.uniform(-19, np.log2(57344), 30000))
    y5 = (mag * rng.choice([-1, 1], mag.size)).astype(np.float32)
    y5 = y5[np.abs(y5) <= 57344]
    t5 = torch.from_numpy(y5).to(torch.float8_e5m2).view(torch.uint8).numpy()
    L = orc.lib()
    o4 = np.array([L.orc_encode_e4m3(float(v)) for v in y4], dtype=np.uint8)
    o5 = np.array([L.orc_encode_e5m2(float(v)) for v in y5], dtype=np.uint8)
    np.testing.assert_array_equal(o4, t4)
    np.testing.assert_array_equal(o5, t5)


def test_bf16_decode_is_upper_half_of_binary32():
    L = orc.lib()
    for h in (0x0000, 0x8000, 0x3F80, 0xBF80, 0x0001, 0x7F7F, 0x4049, 0x0080):
        ref = torch.tensor([h], dtype=torch.int32).to(torch.int16).view(torch.bfloat16).float().item()
        assert L.orc_bf16_to_float(h) == ref
