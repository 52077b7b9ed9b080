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
