"""Pins for the oracle's Group Amax Mantissa scaling (Algorithm 1), CPU only.

Expected values come from exact rational arithmetic, from a worked example derived by hand
from Algorithm 1, and from the properties Section 2 states: no saturation, one shared
23-bit mantissa, one 8-bit exponent per block.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import mor_oracle as orc
from paper_2512_22804_b200 import workloads as wl


def f32(x):
    return float(np.float32(x))


def bits(x):
    return int(np.array([x], dtype=np.float32).view(np.uint32)[0])


def test_hand_worked_example():
    # g_amax = 2.5: s_g = 448/2.5 = 179.2 = 1.4 * 2^7, so the shared mantissa is that of 1.4
    m_g = orc.group_mantissa(2.5)
    assert m_g == bits(f32(179.2)) & 0x7FFFFF
    # block amax 2.0: s_b = 224 = 1.75 * 2^7, m_b (0.75) >= m_g (0.4): keep exponent 7 -> scale 179.2
    s4, e4, s5, e5 = orc.block_scale(2.0, m_g)
    assert s4 == f32(179.2) and e4 == 127 + 7 and 2.0 * s4 <= 448
    # block amax 1.5: s_b = 298.67 = 1.1667 * 2^8, m_b < m_g: exponent 8 - 1 -> scale 179.2 again;
    # keeping exponent 8 would give 1.5 * 358.4 = 537.6 > 448
    s4, e4, s5, e5 = orc.block_scale(1.5, m_g)
    assert s4 == f32(179.2) and e4 == 127 + 7
    assert 1.5 * f32(358.4) > 448
    # block amax 0.5: s_b = 896 = 1.75 * 2^9 -> scale 1.4 * 2^9 = 716.8
    s4, e4, s5, e5 = orc.block_scale(0.5, m_g)
    assert s4 == f32(716.8) and e4 == 127 + 9
    # E5M2 scale: same mantissa, 7 binades up (57344 = 448 * 2^7)
    assert s5 == s4 * 128 and e5 == e4 + 7


def all_positive_bf16():
    h = np.arange(1, 0x7F80, dtype=np.uint32)          # every positive finite BF16
    return (h << 16).view(np.float32)


@pytest.mark.parametrize("g_amax", [1.0, 2.5, 3.0, 0.0123, 1000.0, 3.3e38, 1e-30, 448.0])
def test_scale_is_largest_shared_mantissa_value_below_ideal(g_amax):
    """Algorithm 1 picks, among 1.m_g * 2^k, the largest one not above fl32(448 / b_amax)."""
    g_amax = float(wl.bf16_bits_to_float(wl.to_bf16_bits(np.array([g_amax])))[0])
    m_g = orc.group_mantissa(g_amax)
    sig = Fraction(0x800000 + m_g, 0x800000)            # 1.m_g exactly
    amaxes = all_positive_bf16()
    amaxes = amaxes[amaxes <= np.float32(g_amax)][::37]
    for a in amaxes:
        a = float(a)
        s4, e4, s5, e5 = orc.block_scale(a, m_g)
        with np.errstate(over="ignore"):
            ideal = np.float32(448.0) / np.float32(a)    # one binary32 division
        clamped = not np.isfinite(ideal)
        if clamped:
            ideal = np.finfo(np.float32).max
        ideal = Fraction(float(ideal))
        got = Fraction(s4)
        assert got == sig * Fraction(2) ** (e4 - 127), "scale = shared mantissa joined to the E8M0 exponent"
        assert got <= ideal < got * 2, "largest candidate not above the ideal scale"
        assert 1 <= e4 <= 254
        # no saturation: the block amax lands at or below 448 up to the rounding of the division
        assert Fraction(a) * got <= Fraction(448) * (1 + Fraction(1, 2 ** 23))
        if not clamped:
            assert Fraction(a) * got > Fraction(448) / 2 * (1 - Fraction(1, 2 ** 22))


def test_block_holding_the_tensor_amax_gets_the_group_scale():
    for g in (2.5, 0.0123, 7.0, 1e-20, 3e38):
        g = float(wl.bf16_bits_to_float(wl.to_bf16_bits(np.array([g])))[0])
        m_g = orc.group_mantissa(g)
        s4, e4, _, _ = orc.block_scale(g, m_g)
        s_g = np.float32(448.0) / np.float32(g)
        assert bits(s4) == bits(s_g)


def test_e8m0_mode_is_power_of_two_floor():
    assert orc.group_mantissa(2.5, orc.SCALE_E8M0) == 0
    for a in (2.0, 1.5, 0.3, 100.0, 3e-5):
        a = float(wl.bf16_bits_to_float(wl.to_bf16_bits(np.array([a])))[0])
        s4, e4, s5, e5 = orc.block_scale(a, 0, orc.SCALE_E8M0)
        k = int(np.floor(np.log2(448.0 / a)))
        assert s4 == 2.0 ** k and e4 == 127 + k and s5 == 2.0 ** (k + 7)
        assert a * s4 <= 448 < a * s4 * 2


def test_fp32_amax_mode_is_the_plain_quotient():
    for a in (2.0, 1.5, 0.3, 100.0, 3e-5):
        a = float(wl.bf16_bits_to_float(wl.to_bf16_bits(np.array([a])))[0])
        s4, e4, s5, e5 = orc.block_scale(a, 12345, orc.SCALE_FP32_AMAX)
        assert bits(s4) == bits(np.float32(448.0) / np.float32(a))
        assert s5 == s4 * 128


def test_degenerate_amax():
    # all-zero tensor: mantissa 0; all-zero block: exponent field 127
    assert orc.group_mantissa(0.0) == 0
    s4, e4, s5, e5 = orc.block_scale(0.0, 0)
    assert (s4, e4, s5, e5) == (1.0, 127, 128.0, 134)
    m_g = orc.group_mantissa(2.5)
    s4, e4, _, _ = orc.block_scale(0.0, m_g)
    assert e4 == 127 and bits(s4) == (127 << 23) | m_g
    # quotient overflow: clamp to the largest finite binary32, exponent stays a valid E8M0 byte
    tiny = float(wl.bf16_bits_to_float(np.array([0x0001], dtype=np.uint16))[0])  # smallest BF16 subnormal
    assert orc.group_mantissa(tiny) == 0x7FFFFF
    s4, e4, s5, e5 = orc.block_scale(tiny, 0x7FFFFF)
    assert e4 == 254 and e5 == 254 and np.isfinite(s4) and np.isfinite(s5)
    s4, e4, s5, e5 = orc.block_scale(tiny, 0x000123)
    assert e4 == 254 and bits(s4) == (254 << 23) | 0x123


def test_storage_is_one_byte_per_block_and_one_mantissa_per_tensor():
    x = wl.weight_like(256, 384, seed=5)
    r = orc.run(x, (128, 128), [orc.FMT_E4M3, orc.FMT_BF16], orc.CRIT_BLOCK_VS_E5M2)
    assert r.scale_e8m0.dtype == np.uint8 and r.scale_e8m0.size == 2 * 3
    assert 0 <= r.tensor["group_mantissa"] < 2 ** 23
    # every block scale of the tensor carries the same 23 mantissa bits
    mant = r.blocks["scale_e4m3"].view(np.uint32) & 0x7FFFFF
    assert (mant == r.tensor["group_mantissa"]).all()
    assert ((r.blocks["scale_e4m3"].view(np.uint32) >> 23) == r.blocks["exp_e4m3"]).all()


def test_per_tensor_partition_reduces_to_plain_amax_scaling():
    x = wl.gaussian_outlier_rows(64, 96, n_outlier_rows=2, seed=3)
    r = orc.run(x, (0, 0), [orc.FMT_E4M3, orc.FMT_BF16], orc.CRIT_TENSOR_MEAN_REL)
    amax = np.abs(wl.bf16_bits_to_float(x)).max()
    assert r.tensor["group_amax"] == amax == r.blocks["amax"][0]
    assert bits(r.blocks["scale_e4m3"][0]) == bits(np.float32(448.0) / np.float32(amax))


def test_amax_is_brute_force_max_and_blocks_agree_with_group():
    x = wl.activation_like(130, 300, seed=9)            # ragged in both directions
    vals = np.abs(wl.bf16_bits_to_float(x)).astype(np.float64)
    r = orc.run(x, (128, 128), [orc.FMT_E4M3, orc.FMT_BF16], orc.CRIT_BLOCK_VS_E5M2)
    assert r.grid == (2, 3)
    for bi in range(2):
        for bj in range(3):
            blk = vals[bi * 128:(bi + 1) * 128, bj * 128:(bj + 1) * 128]
            assert r.blocks["amax"][bi * 3 + bj] == blk.max()
    assert r.blocks["amax"].max() == r.tensor["group_amax"] == vals.max()
    assert orc.tensor_amax(x) == vals.max()
