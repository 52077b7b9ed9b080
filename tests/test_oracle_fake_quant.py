"""Pins for the oracle's fake quantisation (quantise, dequantise, de-scale to BF16; Section 4 of the paper).

Expected values come from outside the oracle: PyTorch's float8 and bfloat16 casts and NumPy's binary32
division as a third opinion on in-range data, exact reproduction of FP8-exact data under power-of-two
scales, and the error bound of a 3-bit mantissa followed by a BF16 rounding."""
import numpy as np
import torch

from oracle import mor_oracle as orc
from paper_2512_22804_b200 import workloads as wl

TWO = [orc.FMT_E4M3, orc.FMT_BF16]
THREE = [orc.FMT_E4M3, orc.FMT_E5M2, orc.FMT_BF16]


def vals(bits):
    return wl.bf16_bits_to_float(bits)


def test_third_opinion_from_pytorch_casts_and_numpy_division():
    x = wl.weight_like(128, 256, seed=90)
    res = orc.run(x, (128, 128), TWO, orc.CRIT_BLOCK_VS_E5M2)
    assert (res.sel == orc.FMT_E4M3).all()
    fq = orc.fake_quant(x, res, (128, 128), TWO, orc.CRIT_BLOCK_VS_E5M2)
    for bj in range(2):
        s = np.float32(res.scale_f32[bj])
        blk = vals(x[:, 128 * bj:128 * (bj + 1)])
        y = blk * s                                                    # binary32 products
        assert np.abs(y).max() <= 448.0                                # in range: PyTorch's cast agrees with saturating RNE
        q = torch.from_numpy(y).to(torch.float8_e4m3fn).to(torch.float32).numpy()
        t = (q / s).astype(np.float32)                                 # one binary32 division
        want = torch.from_numpy(t).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        np.testing.assert_array_equal(fq[:, 128 * bj:128 * (bj + 1)], want)


def test_fp8_exact_data_comes_back_unchanged_under_power_of_two_scales():
    rng = np.random.default_rng(91)
    a = np.ldexp(rng.integers(8, 16, size=(64, 256)).astype(np.float64), rng.integers(-5, 3, size=(64, 256)))   # 4 significant bits
    a *= rng.choice([-1.0, 1.0], size=a.shape)
    a[3, 7] = 0.0
    x = wl.to_bf16_bits(a)
    for block in [(1, 128), (64, 64), (0, 0)]:
        res = orc.run(x, block, TWO, orc.CRIT_BLOCK_VS_E5M2 if block != (0, 0) else orc.CRIT_TENSOR_MEAN_REL, scale_mode=orc.SCALE_E8M0)
        fq = orc.fake_quant(x, res, block, TWO, orc.CRIT_BLOCK_VS_E5M2 if block != (0, 0) else orc.CRIT_TENSOR_MEAN_REL,
                            scale_mode=orc.SCALE_E8M0)
        np.testing.assert_array_equal(fq, x)


def test_error_bound_and_copies():
    g = wl.gradient_like(128, 512, seed=92)
    g[5, 9] = 0x7FC0
    g[6, 300] = 0xFF80
    res = orc.run(g, (1, 128), THREE, orc.CRIT_BLOCK_VS_E5M2)
    fq = orc.fake_quant(g, res, (1, 128), THREE, orc.CRIT_BLOCK_VS_E5M2)
    sel = res.sel.reshape(128, 4)
    assert (sel == orc.FMT_BF16).any() and (sel == orc.FMT_E5M2).any()
    a, b = vals(g).astype(np.float64), vals(fq).astype(np.float64)
    for r in range(128):
        for c in range(4):
            sl = (r, slice(128 * c, 128 * (c + 1)))
            if sel[r, c] == orc.FMT_BF16:
                np.testing.assert_array_equal(fq[sl], g[sl])                        # kept blocks are copies, NaN/inf included
                continue
            s = float(res.scale_f32[4 * r + c])
            y = np.abs(a[sl]) * s
            lo = 2.0 ** -14 if sel[r, c] == orc.FMT_E5M2 else 2.0 ** -6            # normal range of the chosen format (scaled domain)
            rel = 2.0 ** -3 if sel[r, c] == orc.FMT_E5M2 else 2.0 ** -4
            ok = y >= lo
            assert (np.abs(a[sl][ok] - b[sl][ok]) <= (rel + 2.0 ** -8) * np.abs(a[sl][ok])).all()
            assert (np.sign(b[sl]) * np.sign(a[sl]) >= 0).all()                     # never flips a sign


def test_tensor_level_decision_writes_e4m3_values_even_when_the_tensor_falls_back():
    x = wl.gaussian_outlier_rows(128, 256, n_outlier_rows=2, seed=93)
    lo = orc.run(x, (128, 128), TWO, orc.CRIT_TENSOR_MEAN_REL, threshold=1e-4)
    hi = orc.run(x, (128, 128), TWO, orc.CRIT_TENSOR_MEAN_REL, threshold=0.5)
    assert lo.tensor["tensor_format"] == orc.FMT_BF16 and hi.tensor["tensor_format"] == orc.FMT_E4M3
    a = orc.fake_quant(x, lo, (128, 128), TWO, orc.CRIT_TENSOR_MEAN_REL, threshold=1e-4)
    b = orc.fake_quant(x, hi, (128, 128), TWO, orc.CRIT_TENSOR_MEAN_REL, threshold=0.5)
    np.testing.assert_array_equal(a, b)
    assert (a != x).any()


def _f32(bits: int) -> float:
    return float(np.array([bits], dtype=np.uint32).view(np.float32)[0])


def test_bf16_rounding_of_every_midpoint_goes_to_even_and_neighbours_to_nearer():
    """The last rounding of fake quantisation (binary32 -> BF16), pinned where it is decided: at exact midpoints
    between neighbouring BF16 values (bit 15 set, bits 0-14 clear) and one binary32 ulp to either side.
    Expected values: exact rationals (the nearer BF16 neighbour; on a tie the one with an even low bit) and
    PyTorch's bfloat16 cast as an outside opinion."""
    from fractions import Fraction

    rng = np.random.default_rng(94)
    # a walk over exponents (subnormal results, the smallest and largest binades included) and mantissas
    his = np.concatenate([np.arange(0, 0x7F7F, 37, dtype=np.uint32), np.array([0, 1, 0x7F, 0x80, 0x7F7E], dtype=np.uint32),
                          rng.integers(0, 0x7F7F, size=400, dtype=np.uint32)])
    pats = []
    for hi in his:
        for low in (0x7FFF, 0x8000, 0x8001):
            for sign in (0, 0x80000000):
                pats.append(int(hi) << 16 | low | sign)
    pats = np.array(pats, dtype=np.uint32)
    got = np.array([orc.f32_to_bf16(_f32(int(p))) for p in pats], dtype=np.uint16)
    torch_bits = torch.from_numpy(pats.view(np.float32).copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(got, torch_bits)
    for p, g in zip(pats.tolist(), got.tolist()):
        v = Fraction(_f32(p & 0x7FFFFFFF))
        lo_bits = (p & 0x7FFFFFFF) >> 16
        lo, hi = Fraction(_f32(lo_bits << 16)), Fraction(_f32((lo_bits + 1) << 16))
        if v - lo < hi - v:
            want = lo_bits
        elif v - lo > hi - v:
            want = lo_bits + 1
        else:
            want = lo_bits if lo_bits % 2 == 0 else lo_bits + 1
        assert g == (want | ((p >> 31) << 15)), hex(p)


def test_bf16_rounding_keeps_specials():
    assert orc.f32_to_bf16(float("inf")) == 0x7F80 and orc.f32_to_bf16(float("-inf")) == 0xFF80
    assert orc.f32_to_bf16(0.0) == 0 and orc.f32_to_bf16(-0.0) == 0x8000
    assert orc.f32_to_bf16(float("nan")) & 0x7FFF > 0x7F80
    assert orc.f32_to_bf16(_f32(0x7F7FFFFF)) == 0x7F80          # the largest binary32 rounds up to infinity
    assert orc.f32_to_bf16(1.0) == 0x3F80


def midpoint_tensor(rows=8, seed=95):
    """BF16 data whose fake-quantised values hit exact BF16 midpoints: every row holds the amax 133 * 2^p, so the
    FP32-amax scale is fl32(448 / (133 * 2^p)) = fl32(64/19) * 2^-p, and every element near 15 * 2^j * 19/64 is
    cast to the E4M3 value 15 * 2^j, whose quotient by the scale is 285 * 2^(j-6): nine significant bits, the
    ninth set, i.e. half way between two BF16 numbers."""
    rng = np.random.default_rng(seed)
    a = np.zeros((rows, 128))
    for r in range(rows):
        p = int(rng.integers(-6, 6))
        j = rng.integers(-4, 4, size=128)
        a[r] = rng.uniform(14.6, 15.4, size=128) * 19.0 / 64.0 * np.ldexp(1.0, j + p - 0) * rng.choice([-1.0, 1.0], size=128)
        a[r, ::3] = rng.standard_normal(a[r, ::3].shape) * np.ldexp(1.0, p)        # ordinary values in between
        a[r, 0] = 133.0 * np.ldexp(1.0, p)
    return wl.to_bf16_bits(a)


def test_fake_quant_on_exact_bf16_midpoints():
    """Element by element against exact rationals on data where the last rounding is a tie for many elements."""
    from fractions import Fraction

    x = midpoint_tensor()
    res = orc.run(x, (1, 128), TWO, orc.CRIT_BLOCK_VS_E5M2, scale_mode=orc.SCALE_FP32_AMAX)
    fq = orc.fake_quant(x, res, (1, 128), TWO, orc.CRIT_BLOCK_VS_E5M2, scale_mode=orc.SCALE_FP32_AMAX)
    ties = 0
    for r in range(x.shape[0]):
        assert res.sel[r] == orc.FMT_E4M3
        s = np.float32(res.scale_f32[r])
        for c in range(128):
            xv = np.float32(vals(x[r:r + 1, c:c + 1])[0, 0])
            y = np.float32(xv * s)
            q = orc.decode_e4m3(orc.encode_e4m3(float(y)))
            t = np.float32(np.float32(q) / s)
            tb = int(np.array([t], dtype=np.float32).view(np.uint32)[0])
            ties += (tb & 0xFFFF) == 0x8000
            lo_bits = (tb & 0x7FFFFFFF) >> 16
            lo, hi = Fraction(_f32(lo_bits << 16)), Fraction(_f32((lo_bits + 1) << 16))
            v = abs(Fraction(float(t)))
            want = lo_bits if (v - lo < hi - v or (v - lo == hi - v and lo_bits % 2 == 0)) else lo_bits + 1
            assert int(fq[r, c]) == (want | ((tb >> 31) << 15))
    assert ties >= 100
