"""Pins for the oracle's error metric, block decisions and tensor aggregate (CPU only).

Expected values: exact rational brute force on tiny blocks (nearest value searched over a
decode table taken from PyTorch, not from the oracle), the closed-form mean relative
error of round-to-nearest on log-uniform data, the paper's "2.4 % flushed" remark, and
invariants that follow from Eq. 1-4 and Algorithm 2.
"""
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import mor_oracle as orc
from paper_2512_22804_b200 import workloads as wl

TWO = [orc.FMT_E4M3, orc.FMT_BF16]
THREE = [orc.FMT_E4M3, orc.FMT_E5M2, orc.FMT_BF16]


def bf16(a):
    return wl.to_bf16_bits(np.asarray(a, dtype=np.float64))


def vals(bits):
    return wl.bf16_bits_to_float(bits).astype(np.float64)


# ---- brute force in exact arithmetic, with PyTorch's decode table as the value grid ----

_codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
GRID4 = [(c, Fraction(v)) for c, v in enumerate(_codes.view(torch.float8_e4m3fn).float().tolist()) if c < 0x7F]
GRID5 = [(c, Fraction(v)) for c, v in enumerate(_codes.view(torch.float8_e5m2).float().tolist()) if c < 0x7C]


def brute_quant(y, grid):
    """(code, value) of the finite grid point nearest to |y|, ties to the even code."""
    a = abs(Fraction(float(y)))
    best = None
    for c, v in grid:
        d = abs(a - v)
        if best is None or d < best[0] or (d == best[0] and c % 2 == 0 and best[1] % 2 == 1):
            best = (d, c, v)
    return best[1] | (0x80 if math.copysign(1.0, float(y)) < 0 else 0), best[2]


def brute_block(xs, scale4, scale5):
    """Eq. 3 sums, codes and Eq. 4 statistics of one block, in exact rationals."""
    e4 = e5 = Fraction(0)
    n = 0
    c4s, c5s = [], []
    mn = None
    for x in xs:
        y4 = np.float32(x) * np.float32(scale4)          # one binary32 multiply
        y5 = np.float32(x) * np.float32(scale5)
        c4, q4 = brute_quant(y4, GRID4)
        c5, q5 = brute_quant(y5, GRID5)
        c4s.append(c4)
        c5s.append(c5)
        if x != 0:
            n += 1
            e4 += 1 if q4 == 0 else abs(abs(Fraction(float(y4))) - q4) / abs(Fraction(float(y4)))
            e5 += 1 if q5 == 0 else abs(abs(Fraction(float(y5))) - q5) / abs(Fraction(float(y5)))
            mn = abs(x) if mn is None else min(mn, abs(x))
    return e4, e5, n, c4s, c5s, mn


@pytest.mark.parametrize("seed", range(6))
def test_blocks_match_exact_brute_force(seed):
    rng = np.random.default_rng(seed)
    rows, cols = 3, 256
    a = rng.standard_normal((rows, cols)) * np.exp2(rng.integers(-12, 3, size=(rows, cols)))
    a[rng.random((rows, cols)) < 0.1] = 0.0
    if seed % 2:
        a[1, :128] *= 2.0 ** -14                          # a block deep in the flush range
    x = bf16(a)
    r = orc.run(x, (1, 128), THREE, orc.CRIT_BLOCK_VS_E5M2)
    v = vals(x)
    for b in range(rows * 2):
        xs = v[b // 2, (b % 2) * 128:(b % 2 + 1) * 128]
        rec = r.blocks[b]
        e4, e5, n, c4s, c5s, mn = brute_block(xs, rec["scale_e4m3"], rec["scale_e5m2"])
        assert rec["nnz"] == n
        assert abs(rec["sum_rel_e4m3"] - float(e4)) <= 1e-12 * max(1.0, float(e4))
        assert abs(rec["sum_rel_e5m2"] - float(e5)) <= 1e-12 * max(1.0, float(e5))
        assert rec["min_abs_nz"] == (float(mn) if mn is not None else np.inf)
        # Algorithm 2 with M_1 = Eq. 3 (tie keeps E4M3) and M_2 = Eq. 4, from the exact sums
        if e4 <= e5:
            want = orc.FMT_E4M3
        elif mn is not None and Fraction(float(rec["amax"])) / Fraction(float(mn)) < Fraction(57344) * 2 ** 14:
            want = orc.FMT_E5M2
        else:
            want = orc.FMT_BF16
        assert rec["sel"] == want == r.sel[b]
        got = r.codes[b // 2, (b % 2) * 128:(b % 2 + 1) * 128].tolist()
        assert got == (c5s if want == orc.FMT_E5M2 else c4s)
        assert r.scale_e8m0[b] == (rec["exp_e5m2"] if want == orc.FMT_E5M2 else rec["exp_e4m3"])


def test_e5m2_scaled_value_is_128_times_the_e4m3_one():
    rng = np.random.default_rng(2)
    xs = vals(bf16(rng.standard_normal(2000) * 3))
    m_g = orc.group_mantissa(float(np.abs(xs).max()))
    s4, _, s5, _ = orc.block_scale(float(np.abs(xs[:128]).max()), m_g)
    for x in xs[:400]:
        assert orc.scale_value(float(x), s5) == 128.0 * orc.scale_value(float(x), s4)


def test_relative_error_bounds_and_nesting():
    rng = np.random.default_rng(3)
    ys = np.exp2(rng.uniform(-6, math.log2(448), 5000)).astype(np.float32)
    for y in ys:
        r4 = orc.rel_err_e4m3(float(y))
        r5 = orc.rel_err_e5m2(float(np.float32(y) * np.float32(128)))
        assert 0.0 <= r4 <= 2.0 ** -4 and 0.0 <= r5 <= 2.0 ** -3
        assert r5 >= r4          # inside E4M3's normal range its grid contains the E5M2 grid
    # flushed values count fully, exact values not at all
    assert orc.rel_err_e4m3(2.0 ** -11) == 1.0 and orc.rel_err_e4m3(0.0) == 1.0
    assert orc.rel_err_e4m3(1.5) == 0.0 and orc.rel_err_e5m2(3.0 * 128) == 0.0
    assert orc.rel_err_e4m3(-17.0) == 1.0 / 17.0        # 17 lies between 16 and 18: tie to 16


def test_mean_relative_error_closed_form_on_log_uniform_data():
    """Round-to-nearest with p mantissa bits on log-uniform magnitudes: mean |err|/|y| = 2^-(p+3)/ln 2."""
    rng = np.random.default_rng(4)
    n = 1 << 18
    mag = np.exp2(rng.uniform(-6.0, 0.0, n))              # 6 binades below the amax
    a = (mag * rng.choice([-1.0, 1.0], n)).reshape(512, 512)
    a[0, 0] = 1.0
    x = bf16(a)
    r = orc.run(x, (0, 0), TWO, orc.CRIT_TENSOR_MEAN_REL, want_codes=False)
    b = r.blocks[0]
    mean4 = b["sum_rel_e4m3"] / b["nnz"]
    mean5 = b["sum_rel_e5m2"] / b["nnz"]
    assert abs(mean4 - 2.0 ** -6 / math.log(2)) < 0.02 * 2.0 ** -6 / math.log(2)
    assert abs(mean5 - 2.0 ** -5 / math.log(2)) < 0.02 * 2.0 ** -5 / math.log(2)
    assert r.tensor["mean_rel_e4m3"] == mean4 and r.tensor["tensor_format"] == orc.FMT_E4M3


@pytest.mark.parametrize("frac,fmt", [(0.030, orc.FMT_BF16), (0.024, orc.FMT_BF16), (0.018, orc.FMT_E4M3)])
def test_flush_fraction_rule_of_the_paper(frac, fmt):
    """Section 4.1.3: with per-tensor scaling, about 2.4 % of values flushed to zero push the
    mean relative error past the 4.5 % threshold (0.024 + 0.976 * 2.25 % = 4.6 %)."""
    rng = np.random.default_rng(5)
    n = 1 << 18
    mag = np.exp2(rng.uniform(-6.0, 0.0, n))
    flushed = rng.random(n) < frac
    mag[flushed] = 2.0 ** -30                              # far below 2^-10 after scaling by 448
    a = (mag * rng.choice([-1.0, 1.0], n)).reshape(512, 512)
    a[0, 0] = 1.0
    r = orc.run(bf16(a), (0, 0), TWO, orc.CRIT_TENSOR_MEAN_REL, threshold=0.045, want_codes=False)
    assert r.tensor["tensor_format"] == fmt
    expect = flushed.mean() + (1 - flushed.mean()) * 2.0 ** -6 / math.log(2)
    assert abs(r.tensor["mean_rel_e4m3"] - expect) < 0.03 * expect


def test_threshold_is_strict_and_monotone():
    x = wl.gaussian_outlier_rows(128, 128, n_outlier_rows=1, seed=1)
    base = orc.run(x, (0, 0), TWO, orc.CRIT_TENSOR_MEAN_REL, want_codes=False).tensor["mean_rel_e4m3"]
    fmts = []
    for th in (base * 0.5, base * 0.999, base * 1.001, base * 2):
        fmts.append(orc.run(x, (0, 0), TWO, orc.CRIT_TENSOR_MEAN_REL, threshold=th, want_codes=False).tensor["tensor_format"])
    assert fmts == [orc.FMT_BF16, orc.FMT_BF16, orc.FMT_E4M3, orc.FMT_E4M3]
    # an error exactly equal to the threshold is rejected (Eq. 2 uses '<'): one exact element
    # (2.0 -> 448) and one flushed element give a mean of exactly 0.5
    two = bf16(np.array([[2.0, 2.0 ** -20]]))
    r = orc.run(two, (0, 0), TWO, orc.CRIT_TENSOR_MEAN_REL, threshold=0.5, want_codes=False)
    assert r.tensor["mean_rel_e4m3"] == 0.5 and r.tensor["tensor_format"] == orc.FMT_BF16
    r = orc.run(two, (0, 0), TWO, orc.CRIT_TENSOR_MEAN_REL, threshold=0.5000001, want_codes=False)
    assert r.tensor["tensor_format"] == orc.FMT_E4M3


def test_fp8_exact_blocks_choose_e4m3():
    # powers of two and small integers times a power-of-two amax: exact in E4M3 after scaling
    a = np.zeros((1, 256))
    a[0, :128] = np.tile([448.0, 224.0, 112.0, 14.0, -320.0, 0.0, 0.5, -448.0], 16) / 256.0  # amax 1.75 -> scale 256
    a[0, 128:] = 0.0                                                                     # all-zero block
    x = bf16(a)
    for flags, want in ((0, orc.FMT_E4M3),):
        r = orc.run(x, (1, 128), TWO, orc.CRIT_BLOCK_VS_E5M2, flags=flags)
        assert r.blocks["sum_rel_e4m3"][0] == 0.0
        assert list(r.sel) == [want, want]
    # all-zero block: zero codes with the sign of each zero kept, exponent byte 127
    a2 = np.zeros((1, 128)); a2[0, 5] = -0.0
    r = orc.run(bf16(a2), (1, 128), TWO, orc.CRIT_BLOCK_VS_E5M2)
    assert r.sel[0] == orc.FMT_E4M3 and r.scale_e8m0[0] == 127 and r.tensor["group_mantissa"] == 0
    assert r.codes[0, 5] == 0x80 and r.codes.sum() == 0x80
    assert r.tensor["nnz"] == 0 and r.tensor["mean_rel_e4m3"] == 0.0 and r.tensor["tensor_format"] == orc.FMT_E4M3


def test_constant_block_is_a_tie_and_the_flag_makes_it_strict():
    x = bf16(np.full((1, 128), 0.3))
    r = orc.run(x, (1, 128), TWO, orc.CRIT_BLOCK_VS_E5M2)
    assert r.blocks["sum_rel_e4m3"][0] == r.blocks["sum_rel_e5m2"][0]
    assert r.sel[0] == orc.FMT_E4M3
    r = orc.run(x, (1, 128), TWO, orc.CRIT_BLOCK_VS_E5M2, flags=orc.FLAG_STRICT_TIES)
    assert r.sel[0] == orc.FMT_BF16
    r = orc.run(x, (1, 128), THREE, orc.CRIT_BLOCK_VS_E5M2, flags=orc.FLAG_STRICT_TIES)
    assert r.sel[0] == orc.FMT_E5M2 and r.scale_e8m0[0] == r.blocks["exp_e5m2"][0]
    assert (r.codes[0] == orc.encode_e5m2(57344.0)).all()    # constant block: every value lands on the amax


def test_wide_block_rejects_e4m3_and_eq4_gates_e5m2():
    # one large value and many values 2^-20 below it: E4M3 flushes them (error 1 each), E5M2 keeps them
    a = np.full((1, 128), 2.0 ** -20 * 1.3); a[0, 0] = 1.0
    r3 = orc.run(bf16(a), (1, 128), THREE, orc.CRIT_BLOCK_VS_E5M2)
    r2 = orc.run(bf16(a), (1, 128), TWO, orc.CRIT_BLOCK_VS_E5M2)
    assert r3.blocks["sum_rel_e4m3"][0] > r3.blocks["sum_rel_e5m2"][0]
    assert r3.sel[0] == orc.FMT_E5M2 and r2.sel[0] == orc.FMT_BF16
    # widen the range past 57344 / 2^-14: Eq. 4 fails, BF16 even in the three-way recipe
    a[0, 1] = 2.0 ** -31
    r3 = orc.run(bf16(a), (1, 128), THREE, orc.CRIT_BLOCK_VS_E5M2)
    assert r3.blocks["amax"][0] / r3.blocks["min_abs_nz"][0] >= 939524096
    assert r3.sel[0] == orc.FMT_BF16
    # exactly at the bound the strict '<' of Eq. 4 still fails; one BF16 step inside it passes
    a[0, 1] = 1.0 / 939524096.0
    assert orc.run(bf16(a), (1, 128), THREE, orc.CRIT_BLOCK_VS_E5M2).sel[0] == orc.FMT_BF16
    a[0, 1] = 1.0 / 939524096.0 * (1 + 2.0 ** -7)
    assert orc.run(bf16(a), (1, 128), THREE, orc.CRIT_BLOCK_VS_E5M2).sel[0] == orc.FMT_E5M2


def test_eq4_minimum_over_nonzeros_and_the_literal_flag():
    a = np.full((1, 128), 2.0 ** -20 * 1.3); a[0, 0] = 1.0; a[0, 7] = 0.0
    r = orc.run(bf16(a), (1, 128), THREE, orc.CRIT_BLOCK_VS_E5M2)
    assert r.sel[0] == orc.FMT_E5M2
    r = orc.run(bf16(a), (1, 128), THREE, orc.CRIT_BLOCK_VS_E5M2, flags=orc.FLAG_RANGE_MIN_INCLUDES_ZERO)
    assert r.sel[0] == orc.FMT_BF16


def test_tensor_aggregate_is_global_mean_and_order_free():
    x = wl.activation_like(256, 512, seed=21)
    per_tensor_amax = orc.tensor_amax(x)
    r_blk = orc.run(x, (128, 128), TWO, orc.CRIT_TENSOR_MEAN_REL)
    r_row = orc.run(x, (1, 128), TWO, orc.CRIT_TENSOR_MEAN_REL)
    for r in (r_blk, r_row):
        assert r.tensor["nnz"] == r.blocks["nnz"].sum() == np.count_nonzero(x & 0x7FFF)
        assert math.isclose(r.tensor["sum_rel_e4m3"], math.fsum(r.blocks["sum_rel_e4m3"]), rel_tol=1e-12)
        assert math.isclose(r.tensor["mean_rel_e4m3"], math.fsum(r.blocks["sum_rel_e4m3"]) / r.tensor["nnz"], rel_tol=1e-12)
        assert r.tensor["group_amax"] == per_tensor_amax
        assert (r.sel == r.tensor["tensor_format"]).all()
        assert r.tensor["n_blocks"] == r.sel.size
    # finer blocks cannot be worse on heavy-tailed data
    assert r_row.tensor["mean_rel_e4m3"] <= r_blk.tensor["mean_rel_e4m3"]
    # a tensor that is a single block gives the same numbers under either partition
    y = wl.activation_like(128, 128, seed=22)
    a = orc.run(y, (0, 0), TWO, orc.CRIT_TENSOR_MEAN_REL)
    b = orc.run(y, (128, 128), TWO, orc.CRIT_TENSOR_MEAN_REL)
    assert a.tensor == b.tensor and (a.codes == b.codes).all()
    # a subset of blocks with the group amax supplied reproduces the full run's records
    ids = np.array([5, 0, 3])
    sub = orc.run(x, (128, 128), TWO, orc.CRIT_BLOCK_VS_E5M2, ids=ids, group_amax=per_tensor_amax)
    full = orc.run(x, (128, 128), TWO, orc.CRIT_BLOCK_VS_E5M2)
    for i, b in enumerate(ids):
        assert sub.blocks[i] == full.blocks[b]


def test_block_mean_rel_criterion():
    a = np.exp2(np.random.default_rng(8).uniform(-5, 0, (2, 128))); a[1, 1:] *= 2.0 ** -15
    r = orc.run(bf16(a), (1, 128), TWO, orc.CRIT_BLOCK_MEAN_REL, threshold=0.045)
    means = r.blocks["sum_rel_e4m3"] / r.blocks["nnz"]
    assert means[0] < 0.045 < means[1]
    assert list(r.sel) == [orc.FMT_E4M3, orc.FMT_BF16]
    # Eq. 2 on a block is strict as well: one exact element (2.0 -> 448) and one flushed element give a block
    # mean of exactly 0.5, which a threshold of 0.5 rejects and the next larger threshold accepts
    two = bf16(np.array([[2.0, 2.0 ** -20]]))
    r = orc.run(two, (1, 128), TWO, orc.CRIT_BLOCK_MEAN_REL, threshold=0.5)
    assert r.blocks["sum_rel_e4m3"][0] == 1.0 and list(r.sel) == [orc.FMT_BF16]
    r = orc.run(two, (1, 128), TWO, orc.CRIT_BLOCK_MEAN_REL, threshold=0.5000001)
    assert list(r.sel) == [orc.FMT_E4M3]


def test_ragged_edges_behave_like_absent_elements():
    x = wl.weight_like(200, 300, seed=31)
    r = orc.run(x, (128, 128), TWO, orc.CRIT_BLOCK_VS_E5M2)
    assert r.grid == (2, 3) and r.codes.shape == (200, 300)
    # the edge block equals a run on the cut-out piece with the same group amax
    piece = np.ascontiguousarray(x[128:200, 256:300])
    p = orc.run(piece, (128, 128), TWO, orc.CRIT_BLOCK_VS_E5M2, group_amax=r.tensor["group_amax"])
    assert p.blocks[0] == r.blocks[5] and (p.codes == r.codes[128:, 256:]).all()
    # padded rows (ld > cols): the padding is never read
    padded = np.full((200, 320), 0x7FC0, dtype=np.uint16); padded[:, :300] = x
    q = orc.run(padded, (128, 128), TWO, orc.CRIT_BLOCK_VS_E5M2, cols=300)
    assert q.tensor == r.tensor and (q.codes == r.codes).all()
    # empty tensors
    e = orc.run(np.zeros((0, 128), dtype=np.uint16), (1, 128), TWO, orc.CRIT_BLOCK_VS_E5M2)
    assert e.tensor["n_blocks"] == 0 and e.tensor["tensor_format"] == orc.FMT_E4M3


def test_nonfinite_inputs_follow_the_stated_reading():
    a = np.random.default_rng(9).standard_normal((2, 128))
    x = bf16(a)
    x[0, 3] = 0x7FC0; x[0, 4] = 0x7F80; x[0, 5] = 0xFF80   # NaN, +inf, -inf
    r = orc.run(x, (1, 128), TWO, orc.CRIT_BLOCK_VS_E5M2)
    assert r.tensor["n_nonfinite"] == 3 and r.blocks["n_nonfinite"][0] == 3
    assert r.sel[0] == orc.FMT_BF16 and r.tensor["tensor_format"] == orc.FMT_BF16
    assert list(r.codes[0, 3:6]) == [0x7F, 0x7E, 0xFE]
    assert r.blocks["nnz"][0] == 125 and np.isfinite(r.blocks["amax"][0]) and np.isfinite(r.tensor["group_amax"])
    clean = x.copy(); clean[0, 3:6] = 0
    c = orc.run(clean, (1, 128), TWO, orc.CRIT_BLOCK_VS_E5M2)
    assert c.blocks["sum_rel_e4m3"][0] == r.blocks["sum_rel_e4m3"][0]
    assert (np.delete(c.codes[0], [3, 4, 5]) == np.delete(r.codes[0], [3, 4, 5])).all()


def test_unsupported_recipes_are_rejected():
    x = bf16(np.ones((1, 128)))
    with pytest.raises(ValueError):
        orc.run(x, (1, 128), [orc.FMT_E5M2, orc.FMT_E4M3, orc.FMT_BF16], orc.CRIT_BLOCK_VS_E5M2)
    with pytest.raises(ValueError):
        orc.run(x, (1, 128), THREE, orc.CRIT_TENSOR_MEAN_REL)


def test_error_histogram_bins_of_section_4_1_3():
    """Twelve bins of 0.5 % of relative error: the first below 0.5 %, the second from 0.5 % to below 1.0 %,
    the last from 5.5 % up; the 4.5 % threshold is the left edge of the tenth bin."""
    assert orc.error_bin(0.0) == 0 and orc.error_bin(0.0049999) == 0
    assert orc.error_bin(0.005) == 1 and orc.error_bin(0.0099999) == 1
    assert orc.error_bin(0.045) == 9 and orc.error_bin(0.0449999) == 8
    assert orc.error_bin(0.0549999) == 10 and orc.error_bin(0.055) == 11
    assert orc.error_bin(1.0) == 11 and orc.error_bin(37.5) == 11
    # every bin is hit once by its midpoint, and the bin never decreases with the error
    mids = [(k + 0.5) * 0.005 for k in range(12)]
    assert [orc.error_bin(m) for m in mids] == list(range(12))
    xs = np.linspace(0.0, 0.08, 2001)
    bins = [orc.error_bin(float(x)) for x in xs]
    assert all(b1 >= b0 for b0, b1 in zip(bins, bins[1:]))
    # brute force against the definition with exact rationals (edges k/200)
    from fractions import Fraction
    for x in xs:
        k = min(11, int(Fraction(float(x)) / Fraction(0.005)))
        assert orc.error_bin(float(x)) == k
