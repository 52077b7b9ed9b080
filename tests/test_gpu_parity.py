"""Parity of the CUDA path (through the C boundary) with the CPU oracle.  Needs a B200."""
import numpy as np
import pytest

from oracle import mor_oracle as orc
from paper_2512_22804_b200 import binding as mb
from paper_2512_22804_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

TWO = (mb.MOR_FMT_E4M3, mb.MOR_FMT_BF16)
THREE = (mb.MOR_FMT_E4M3, mb.MOR_FMT_E5M2, mb.MOR_FMT_BF16)
KINDS = [(0, 0), (1, 128), (128, 128), (64, 64)]


def recipe(block, formats=TWO, criterion=mb.MOR_CRIT_BLOCK_VS_E5M2, threshold=0.045, scale_mode=mb.MOR_SCALE_GAM, flags=0):
    return mb.Recipe(tuple(block), tuple(formats), criterion, threshold, scale_mode, flags)


# ------------------------------------------------------------ the benchmark configurations, reduced

@pytest.mark.parametrize("cfg,scale", [(0, 1), (0, 4), (1, 8), (2, 8), (3, 8), (4, 16)])
def test_configs_reduced(cfg, scale):
    total = exempt = 0
    for case in wl.config_case(cfg, scale=scale):
        rep = parity.run_and_compare(case.bits, parity.recipe_from_case(case))
        total += rep.n_blocks
        exempt += rep.n_exempt
    assert exempt <= max(1, total // 1000), f"{exempt} of {total} blocks within the tolerance band"


@pytest.mark.parametrize("block", KINDS)
@pytest.mark.parametrize("crit", [mb.MOR_CRIT_TENSOR_MEAN_REL, mb.MOR_CRIT_BLOCK_VS_E5M2, mb.MOR_CRIT_BLOCK_MEAN_REL])
def test_every_partition_with_every_criterion(block, crit):
    x = wl.activation_like(384, 640, seed=41)
    parity.run_and_compare(x, recipe(block, TWO, crit))
    g = wl.gradient_like(256, 512, seed=42)
    parity.run_and_compare(g, recipe(block, TWO, crit, threshold=0.2))


@pytest.mark.parametrize("block", [(1, 128), (128, 128), (64, 64)])
@pytest.mark.parametrize("flags", [0, mb.MOR_FLAG_STRICT_TIES, mb.MOR_FLAG_RANGE_MIN_INCLUDES_ZERO,
                                   mb.MOR_FLAG_STRICT_TIES | mb.MOR_FLAG_RANGE_MIN_INCLUDES_ZERO])
def test_three_way_with_flags(block, flags):
    g = wl.gradient_like(384, 1024, seed=43)
    rep = parity.run_and_compare(g, recipe(block, THREE, flags=flags))
    assert rep.n_exempt <= 2
    # all three formats are exercised by this workload at 1x128
    if block == (1, 128) and flags == 0:
        ref = orc.run(g, block, list(THREE), orc.CRIT_BLOCK_VS_E5M2)
        assert ref.tensor["n_e4m3"] > 0 and ref.tensor["n_e5m2"] > 0 and ref.tensor["n_bf16"] > 0


@pytest.mark.parametrize("block", KINDS)
@pytest.mark.parametrize("mode", [mb.MOR_SCALE_GAM, mb.MOR_SCALE_E8M0, mb.MOR_SCALE_FP32_AMAX])
def test_scale_modes(block, mode):
    x = wl.weight_like(256, 384, seed=44)
    parity.run_and_compare(x, recipe(block, TWO, scale_mode=mode))


@pytest.mark.parametrize("block", [(1, 128), (128, 128), (64, 64)])
@pytest.mark.parametrize("formats", [TWO, THREE])
def test_narrow_range_blocks_next_to_wide_range_blocks(block, formats):
    """Narrow-range blocks (all non-zeros within E4M3's normal range after scaling) keep E4M3 by
    construction (every element's E5M2 error is at least its E4M3 error there); they sit next to
    wide-range blocks that go to E5M2 or BF16.  With and without block statistics, with and without
    strict ties."""
    rng = np.random.default_rng(49)
    a = rng.uniform(0.5, 4.0, size=(384, 512)) * rng.choice([-1.0, 1.0], size=(384, 512))
    a[:, 256:] = wl.bf16_bits_to_float(wl.gradient_like(384, 256, seed=50))      # wide-range half
    a[5, 17] = 0.0
    x = wl.to_bf16_bits(a)
    for stats in (False, True):
        for flags in (0, mb.MOR_FLAG_STRICT_TIES):
            rep = parity.run_and_compare(x, recipe(block, formats, flags=flags), block_stats=stats)
            assert rep.n_exempt <= 1


# ------------------------------------------------------------ sub-column blocks (128 x 1), transposed codes

@pytest.mark.parametrize("shape", [(256, 256), (128, 1), (300, 200), (1, 130), (517, 72)])
@pytest.mark.parametrize("formats", [TWO, THREE])
def test_sub_column_blocks_with_transposed_codes(shape, formats):
    g = wl.gradient_like(shape[0], shape[1], seed=63) if shape[0] > 1 else wl.weight_like(1, shape[1], seed=63)
    if shape[0] > 200:
        g[130:, : shape[1] // 2] = wl.weight_like(shape[0] - 130, shape[1] // 2, seed=64)    # blocks that keep E4M3
        g[3, 5] = 0x7FC0
    ld = (shape[1] + 7) // 8 * 8 + 8
    for flags in (0, mb.MOR_FLAG_STRICT_TIES | mb.MOR_FLAG_RANGE_MIN_INCLUDES_ZERO):
        for mode in (mb.MOR_SCALE_GAM, mb.MOR_SCALE_FP32_AMAX):
            rep = parity.run_and_compare(g, recipe((128, 1), formats, flags=flags, scale_mode=mode), pad_to=ld)
            assert rep.n_exempt <= 2
    parity.run_and_compare(g, recipe((128, 1), TWO, mb.MOR_CRIT_TENSOR_MEAN_REL), pad_to=ld, group_amax_supplied=True)


def test_sub_column_codes_are_the_transpose_of_what_row_blocks_give_for_the_transposed_tensor():
    import torch

    g = wl.activation_like(256, 384, seed=65)
    x = parity.to_device(g)
    xt = parity.to_device(np.ascontiguousarray(g.T))
    a = mb.analyze_quantize(x, recipe((128, 1), THREE))
    b = mb.analyze_quantize(xt, recipe((1, 128), THREE))
    torch.cuda.synchronize()
    assert a.codes.shape == (384, 256) and torch.equal(a.codes, b.codes)          # stored transposed: same bytes
    assert torch.equal(a.sel.t().contiguous(), b.sel) and torch.equal(a.scale_e8m0.t().contiguous(), b.scale_e8m0)


@pytest.mark.parametrize("shape", [(256, 384), (300, 200), (1000, 1160), (130, 2056)])
@pytest.mark.parametrize("formats", [TWO, THREE])
def test_rows_and_columns_of_one_tensor_in_one_call(shape, formats):
    """A batched call that lists the same tensor with 1x128 and with 128x1 blocks reads every tile once and
    serves both; codes, scales, selections and counts of each equal its own single call bit for bit (the error sums
    within the stated tolerance: the two calls may add them in another order) and match the oracle."""
    import torch

    g = wl.gradient_like(shape[0], shape[1], seed=66)
    g[shape[0] // 2:, : shape[1] // 2] = wl.weight_like(shape[0] - shape[0] // 2, shape[1] // 2, seed=67)
    g[3, 5] = 0x7FC0
    x = parity.to_device(g)
    for mode in (mb.MOR_SCALE_GAM, mb.MOR_SCALE_E8M0):
        for supplied, stats in ((False, True), (False, False), (True, True), (True, False)):
            ra, rb = recipe((1, 128), formats, scale_mode=mode), recipe((128, 1), formats, scale_mode=mode)
            ga = None
            if supplied:
                ga = torch.tensor([orc.tensor_amax(g)] * 2, dtype=torch.float32, device="cuda")
            plan = mb.BatchPlan([x, x], [ra, rb], block_stats=stats, group_amax=ga)
            plan.run()
            plan.run()
            torch.cuda.synchronize()
            for r, out, k in ((ra, plan.outs[0], 0), (rb, plan.outs[1], 1)):
                single = mb.analyze_quantize(x, r, block_stats=stats, group_amax=None if ga is None else ga[k:k + 1])
                torch.cuda.synchronize()
                a, b = out.tensor_stats_dict(), single.tensor_stats_dict()
                assert a.keys() == b.keys()
                for key in a:
                    if isinstance(a[key], float):
                        assert a[key] == pytest.approx(b[key], rel=parity.REL_TOL, abs=0.0), key
                    else:
                        assert a[key] == b[key], key
                assert torch.equal(out.codes, single.codes) and torch.equal(out.sel, single.sel)
                assert torch.equal(out.scale_e8m0, single.scale_e8m0)
            for r, out in ((ra, plan.outs[0]), (rb, plan.outs[1])):
                ref = orc.run(g, r.block, list(r.formats), r.criterion, r.threshold, r.scale_mode, r.flags)
                parity.compare(g, r, out, ref)

# ------------------------------------------------------------ fake quantisation (Section 4)

@pytest.mark.parametrize("block", KINDS + [(1, 0), (128, 1)])
def test_fake_quant_output(block):
    g = np.concatenate([wl.gradient_like(150, 1000, seed=58), wl.weight_like(170, 1000, seed=59)])
    g[7, 13] = 0x7FC0
    g[200, 999] = 0xFF80
    whole = block in ((0, 0), (1, 0))
    recipes = [recipe(block, TWO, mb.MOR_CRIT_TENSOR_MEAN_REL)]
    if not whole:
        recipes += [recipe(block, THREE), recipe(block, TWO), recipe(block, TWO, mb.MOR_CRIT_BLOCK_MEAN_REL, threshold=0.03),
                    recipe(block, THREE, scale_mode=mb.MOR_SCALE_E8M0)]
    for r in recipes:
        parity.run_and_compare(g, r, pad_to=1008, block_stats=block != (1, 0), fake_quant=True)
        parity.run_and_compare(g, r, pad_to=1008, block_stats=False, fake_quant=True, group_amax_supplied=True)


def test_fake_quant_where_the_last_rounding_is_a_tie():
    """FP32-amax scaling with a block amax of 133 * 2^p makes the scale fl32(64/19) * 2^-p; elements cast to the
    E4M3 value 15 * 2^j then de-scale to 285 * 2^(j-6), exactly half way between two BF16 numbers, so the
    round-to-nearest-even of the BF16 conversion decides the output bits for over a hundred elements here."""
    from tests.test_oracle_fake_quant import midpoint_tensor

    x = midpoint_tensor(rows=256, seed=96)
    r = recipe((1, 128), TWO, scale_mode=mb.MOR_SCALE_FP32_AMAX)
    ref = orc.run(x, (1, 128), list(TWO), r.criterion, r.threshold, r.scale_mode)
    v = wl.bf16_bits_to_float(x).astype(np.float32) * ref.scale_f32.reshape(-1, 1).astype(np.float32)
    near15 = np.abs(np.abs(v) / np.exp2(np.floor(np.log2(np.maximum(np.abs(v), 1e-30)))) - 1.875) <= 0.0625
    assert near15.sum() > 1000
    parity.run_and_compare(x, r, fake_quant=True)
    parity.run_and_compare(np.tile(x, (1, 2)), recipe((128, 128), TWO, scale_mode=mb.MOR_SCALE_E8M0), fake_quant=True)


# ------------------------------------------------------------ per-channel partition (one block per row)

@pytest.mark.parametrize("shape", [(256, 512), (130, 1000), (1, 128), (300, 72), (5, 2049)])
@pytest.mark.parametrize("mode", [mb.MOR_SCALE_GAM, mb.MOR_SCALE_E8M0, mb.MOR_SCALE_FP32_AMAX])
def test_per_channel_partition_with_the_tensor_level_decision(shape, mode):
    x = wl.activation_like(shape[0], shape[1], n_outlier_cols=min(4, shape[1]), seed=48)
    x[shape[0] // 2, :] = 0                                        # an all-zero channel
    ld = (shape[1] + 7) // 8 * 8 + 8
    for th in (0.045, 0.01):
        r = recipe((1, 0), TWO, mb.MOR_CRIT_TENSOR_MEAN_REL, threshold=th, scale_mode=mode)
        rep = parity.run_and_compare(x, r, pad_to=ld, block_stats=False)
        assert rep.n_blocks == shape[0]
    if shape[0] > 3:
        x[3, shape[1] // 2] = 0x7FC0                               # a NaN in one channel
        parity.run_and_compare(x, recipe((1, 0), TWO, mb.MOR_CRIT_TENSOR_MEAN_REL, scale_mode=mode), pad_to=ld, block_stats=False)
        parity.run_and_compare(x, recipe((1, 0), TWO, mb.MOR_CRIT_TENSOR_MEAN_REL, scale_mode=mode), pad_to=ld, block_stats=False,
                               group_amax_supplied=True)


@pytest.mark.parametrize("shape", [(256, 512), (130, 1000), (300, 72), (5, 2049), (257, 1160)])
@pytest.mark.parametrize("crit", [mb.MOR_CRIT_BLOCK_VS_E5M2, mb.MOR_CRIT_BLOCK_MEAN_REL])
def test_per_channel_partition_with_a_decision_per_row(shape, crit):
    """One block per row, decided row by row (Eq. 3 against E5M2, or Eq. 1-2 on the row): the row's sums are added
    up over its tiles after the main kernel.  Rows that keep E4M3 next to rows that fall back; an all-zero row, a
    row with a NaN; with and without per-row statistics; every scale mode; strict ties."""
    rows, cols = shape
    x = wl.activation_like(rows, cols, n_outlier_cols=min(4, cols), seed=148)
    x[rows // 2, :] = 0                                            # an all-zero channel
    wide = wl.gradient_like(rows, cols, seed=149)
    x[::3, :] = wide[::3, :]                                       # every third row spans many binades
    if rows > 3:
        x[3, cols // 2] = 0x7FC0
    ld = (cols + 7) // 8 * 8 + 8
    for mode in (mb.MOR_SCALE_GAM, mb.MOR_SCALE_E8M0, mb.MOR_SCALE_FP32_AMAX):
        for flags in (0, mb.MOR_FLAG_STRICT_TIES):
            r = recipe((1, 0), TWO, crit, threshold=0.03, scale_mode=mode, flags=flags)
            rep = parity.run_and_compare(x, r, pad_to=ld, block_stats=True)
            assert rep.n_blocks == rows and rep.n_exempt <= 1
    ref = orc.run(x, (1, cols), list(TWO), crit, 0.03)
    if rows >= 100:
        assert ref.tensor["n_e4m3"] > 0 and ref.tensor["n_bf16"] > 0
    parity.run_and_compare(x, recipe((1, 0), TWO, crit, threshold=0.03), pad_to=ld, block_stats=False, group_amax_supplied=True)
    # per-row statistics also with the tensor-level decision
    parity.run_and_compare(x, recipe((1, 0), TWO, mb.MOR_CRIT_TENSOR_MEAN_REL), pad_to=ld, block_stats=True)


@pytest.mark.parametrize("shape", [(256, 512), (1000, 130), (72, 300), (2049, 5), (1160, 257)])
@pytest.mark.parametrize("crit", [mb.MOR_CRIT_TENSOR_MEAN_REL, mb.MOR_CRIT_BLOCK_VS_E5M2, mb.MOR_CRIT_BLOCK_MEAN_REL])
def test_per_channel_partition_along_the_columns(shape, crit):
    """One block per column (the operand whose dot-product dimension runs down the rows): the column's amax spans the
    tile rows, codes come out transposed; tensor-level decision or a decision per column; statistics per column;
    a zero column, a NaN, columns that span many binades; every scale mode; equals the row version of the transpose."""
    import torch

    rows, cols = shape
    x = np.ascontiguousarray(wl.activation_like(cols, rows, n_outlier_cols=min(4, rows), seed=150).T)
    x[:, cols // 2] = 0
    wide = np.ascontiguousarray(wl.gradient_like(cols, rows, seed=151).T)
    x[:, ::3] = wide[:, ::3]
    if cols > 3:
        x[rows // 2, 3] = 0x7FC0
    ld = (cols + 7) // 8 * 8 + 8
    for mode in (mb.MOR_SCALE_GAM, mb.MOR_SCALE_E8M0, mb.MOR_SCALE_FP32_AMAX):
        r = recipe((0, 1), TWO, crit, threshold=0.03, scale_mode=mode)
        rep = parity.run_and_compare(x, r, pad_to=ld, block_stats=True)
        assert rep.n_blocks == cols and rep.n_exempt <= 1
    parity.run_and_compare(x, recipe((0, 1), TWO, crit, threshold=0.03), pad_to=ld, block_stats=False, group_amax_supplied=True)
    if crit == mb.MOR_CRIT_TENSOR_MEAN_REL:
        parity.run_and_compare(x, recipe((0, 1), TWO, crit, threshold=0.03), pad_to=ld, block_stats=False, fake_quant=True)
    # the same bytes as per-row blocks of the transposed tensor (where both leading dimensions are multiples of 8)
    if rows % 8 or cols % 8:
        return
    a = mb.analyze_quantize(parity.to_device(x), recipe((0, 1), TWO, crit, threshold=0.03))
    b = mb.analyze_quantize(parity.to_device(np.ascontiguousarray(x.T)), recipe((1, 0), TWO, crit, threshold=0.03))
    torch.cuda.synchronize()
    assert torch.equal(a.codes[:, :rows], b.codes[:, :rows])
    assert torch.equal(a.sel.reshape(-1), b.sel.reshape(-1)) and torch.equal(a.scale_e8m0.reshape(-1), b.scale_e8m0.reshape(-1))


def test_per_channel_partition_refuses_what_it_cannot_give():
    """Three formats (a row that chose E5M2 would need its codes rewritten after the last tile) and BF16 outputs that
    depend on a per-row decision are refused."""
    import torch

    x = torch.zeros((128, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mb.MorError) as e:
        mb.analyze_quantize(x, recipe((1, 0), THREE, mb.MOR_CRIT_BLOCK_VS_E5M2))
    assert e.value.status == mb.MOR_ERR_UNSUPPORTED
    for kw in (dict(fallback=True), dict(fake_quant=True)):
        with pytest.raises(mb.MorError) as e:
            mb.analyze_quantize(x, recipe((1, 0), TWO, mb.MOR_CRIT_BLOCK_VS_E5M2), **kw)
        assert e.value.status == mb.MOR_ERR_UNSUPPORTED


# ------------------------------------------------------------ ragged, padded, tiny and empty shapes

@pytest.mark.parametrize("block", KINDS)
@pytest.mark.parametrize("shape", [(1, 1), (1, 128), (3, 127), (129, 129), (200, 300), (127, 1000), (257, 8), (5, 2049)])
def test_ragged_shapes(block, shape):
    x = wl.activation_like(shape[0], shape[1], n_outlier_cols=min(4, shape[1]), seed=45)
    ld = (shape[1] + 7) // 8 * 8 + 8
    parity.run_and_compare(x, recipe(block, THREE if block != (0, 0) else TWO), pad_to=ld)


@pytest.mark.parametrize("block", KINDS)
@pytest.mark.parametrize("shape", [(0, 128), (128, 0), (0, 0)])
def test_empty_tensors(block, shape):
    import torch

    x = torch.empty(shape, dtype=torch.bfloat16, device="cuda")
    out = mb.analyze_quantize(x, recipe(block))
    ts = out.tensor_stats_dict()
    assert ts["n_blocks"] == 0 and ts["nnz"] == 0 and ts["mean_rel_e4m3"] == 0.0
    assert ts["tensor_format"] == mb.MOR_FMT_E4M3 and ts["group_amax"] == 0.0 and ts["group_mantissa"] == 0


# ------------------------------------------------------------ degenerate contents

@pytest.mark.parametrize("block", KINDS)
def test_degenerate_blocks(block):
    a = np.zeros((256, 256))
    a[:128, :128] = 0.3                                            # constant block: exact tie in Eq. 3
    a[128:, :128] = np.tile([448.0, 224.0, 14.0, -320.0, 0.0, 0.5, -448.0, 112.0], (128, 16)) / 256.0   # FP8-exact
    a[128:, 128:] = 2.0 ** -20 * 1.3                               # flushed by E4M3 next to the value below
    a[128:, 128] = 1.0
    a[0, 200] = -0.0                                               # all-zero block with a negative zero
    x = wl.to_bf16_bits(a)
    for flags in (0, mb.MOR_FLAG_STRICT_TIES):
        fm = THREE if block != (0, 0) else TWO
        rep = parity.run_and_compare(x, recipe(block, fm, flags=flags))
        assert rep.n_exempt == 0


def test_values_below_binary32_normal_range_after_scaling():
    # a block amax near the top of BF16's range makes the scale tiny; BF16 subnormals times that
    # scale fall below 2^-126 or vanish: they still count as fully flushed non-zeros
    a = np.zeros((4, 256), dtype=np.float64)
    bits = wl.to_bf16_bits(a)
    bits[:, :] = 0x0001                                            # smallest BF16 subnormal
    bits[0, 0] = 0x7F00                                            # 1.7e38
    bits[1, 5] = 0x7E80
    bits[2, 128:] = 0x0040
    bits[2, 130] = 0x7F7F                                          # largest finite BF16
    for block in KINDS:
        fm = THREE if block != (0, 0) else TWO
        rep = parity.run_and_compare(bits, recipe(block, fm))
        assert rep.n_exempt == 0


@pytest.mark.parametrize("block", KINDS)
def test_nonfinite_inputs(block):
    x = wl.activation_like(256, 384, seed=46)
    x[3, 7] = 0x7FC0; x[3, 8] = 0xFFC1; x[130, 200] = 0x7F80; x[255, 383] = 0xFF80; x[131, 0] = 0x7FFF
    fm = THREE if block != (0, 0) else TWO
    parity.run_and_compare(x, recipe(block, fm))
    parity.run_and_compare(x, recipe(block, TWO, mb.MOR_CRIT_TENSOR_MEAN_REL))
    # with the group amax supplied the main kernel finds the block amax itself (no keys from the pre-pass)
    parity.run_and_compare(x, recipe(block, fm), group_amax_supplied=True)


@pytest.mark.parametrize("block", KINDS)
def test_supplied_group_amax_on_ragged_gradient_data(block):
    g = wl.gradient_like(300, 1000, seed=47)
    fm = THREE if block != (0, 0) else TWO
    rep = parity.run_and_compare(g, recipe(block, fm), group_amax_supplied=True, pad_to=1008)
    assert rep.n_exempt <= 2


# ------------------------------------------------------------ the cast itself, exhaustively

@pytest.mark.parametrize("amax_bits", [0x3F80, 0x4049, 0x3C23, 0x4B12, 0x0090, 0x7F00, 0x2D5A])
def test_every_bf16_pattern_through_the_cast(amax_bits):
    """All 65,536 BF16 patterns under several scales (the supplied group amax fixes the shared mantissa; block
    amaxes always come from the data, so finite values never exceed the format's range after scaling and the
    saturating side of the cast is reached by the +-inf patterns only, whose codes the kernel sets explicitly);
    NaN/inf patterns included."""
    import torch

    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16).reshape(512, 128)
    amax = float(wl.bf16_bits_to_float(np.array([amax_bits], dtype=np.uint16))[0])
    for clean in (False, True):
        b = bits.copy()
        if clean:
            b[(b & 0x7F80) == 0x7F80] = 0
        for block, fm in (((0, 0), TWO), ((1, 128), THREE), ((128, 128), THREE), ((64, 64), THREE)):
            r = recipe(block, fm)
            ref = orc.run(b, r.block, list(r.formats), r.criterion, r.threshold, group_amax=amax)
            ga = torch.tensor([amax], dtype=torch.float32, device="cuda")
            out = mb.analyze_quantize(parity.to_device(b), r, group_amax=ga, block_stats=True, scale_f32=True)
            parity.compare(b, r, out, ref)


# ------------------------------------------------------------ row-sharded use, data steps on the GPU

@pytest.mark.parametrize("crit,block", [(mb.MOR_CRIT_BLOCK_VS_E5M2, (128, 128)), (mb.MOR_CRIT_BLOCK_VS_E5M2, (1, 128)),
                                        (mb.MOR_CRIT_TENSOR_MEAN_REL, (128, 128))])
def test_row_sharded_entry_with_its_default_cuda_steps(crit, block):
    """``sharded.analyze_quantize_row_sharded`` with the CUDA functions it uses by default (no process group: one
    rank holds all rows), against the oracle's run over the tensor; then two halves run one after the other with
    the tensor-wide amax, which must give the same codes as the whole."""
    import torch

    from paper_2512_22804_b200 import sharded

    full = wl.activation_like(512, 384, seed=81)
    full[300:, :] = wl.gradient_like(212, 384, seed=82)
    r = recipe(block, TWO, crit)
    ref = orc.run(full, block, list(TWO), crit, 0.045)
    got = sharded.analyze_quantize_row_sharded(parity.to_device(full), r, device=torch.device("cuda"))
    torch.cuda.synchronize()
    assert got.group_amax == ref.tensor["group_amax"]
    parity.compare(full, r, got.outputs, ref)
    assert got.tensor["tensor_format"] == ref.tensor["tensor_format"] and got.tensor["nnz"] == ref.tensor["nnz"]
    # the halves, each given the amax of the whole tensor as a rank of a sharded run would have it
    codes = []
    for half in (full[:256], full[256:]):
        _, out = sharded._cuda_analyze(parity.to_device(half), r, ref.tensor["group_amax"])
        torch.cuda.synchronize()
        codes.append(out.codes_view().cpu().numpy())
    ex = parity.exempt_blocks(ref, r)
    if not ex.any() and crit != mb.MOR_CRIT_TENSOR_MEAN_REL:
        np.testing.assert_array_equal(np.concatenate(codes), ref.codes)


# ------------------------------------------------------------ API behaviour

def test_supplied_group_amax_and_group_amax_entry_point():
    import torch

    xs = [wl.weight_like(256, 256, seed=50), wl.activation_like(130, 200, seed=51), wl.gradient_like(64, 1024, seed=52)]
    dev = [parity.to_device(np.pad(x, ((0, 0), (0, (-x.shape[1]) % 8)))) for x in xs]
    dev = [d[:, :x.shape[1]] for d, x in zip(dev, xs)]
    got = mb.group_amax(dev).cpu().numpy()
    for g, x in zip(got, xs):
        assert g == orc.tensor_amax(x)
    rep = parity.run_and_compare(xs[0], recipe((128, 128)), group_amax_supplied=True)
    assert rep.n_blocks == 4


def test_select_stats_matches_analyze_quantize():
    import torch

    g = wl.gradient_like(256, 1024, seed=53)
    x = parity.to_device(g)
    for block in [(1, 128), (128, 128), (64, 64)]:
        r = recipe(block, THREE)
        a = mb.analyze_quantize(x, r, block_stats=True)
        s = mb.select_stats(x, r)
        torch.cuda.synchronize()
        assert a.tensor_stats_dict() == s.tensor_stats_dict()
        assert torch.equal(a.sel, s.sel) and torch.equal(a.scale_e8m0, s.scale_e8m0)
        assert (a.block_stats_array() == s.block_stats_array()).all()
        ref = orc.run(g, r.block, list(r.formats), r.criterion, r.threshold)
        parity.compare(g, r, s, ref)


@pytest.mark.parametrize("stats", [False, True])
def test_select_stats_batched_matches_the_oracle(stats):
    """Decisions and statistics for several tensors of mixed partitions in one call, without codes; with and without
    block statistics (without: the plain instantiation, whose non-zero counts come from the pre-pass); some with
    the group amax supplied (single read, the kernel scans)."""
    import torch

    cases = [(wl.gradient_like(300, 1000, seed=54), recipe((1, 128), THREE)),
             (wl.weight_like(256, 384, seed=55), recipe((128, 128), TWO)),
             (wl.activation_like(200, 520, seed=56), recipe((64, 64), THREE)),
             (wl.gaussian_outlier_rows(256, 256, seed=57), recipe((0, 0), TWO, mb.MOR_CRIT_TENSOR_MEAN_REL)),
             (wl.weight_like(130, 200, seed=58), recipe((128, 1), TWO)),
             (wl.activation_like(256, 256, seed=59), recipe((1, 128), TWO, scale_mode=mb.MOR_SCALE_E8M0))]
    xs = [parity.to_device(b) for b, _ in cases]
    plan = mb.BatchPlan(xs, [r for _, r in cases], block_stats=stats, stats_only=True)
    plan.run()
    torch.cuda.synchronize()
    for (bits, r), o in zip(cases, plan.outs):
        assert o.codes is None
        ref = orc.run(bits, parity.oracle_block(r.block, bits.shape[1]), list(r.formats), r.criterion, r.threshold, r.scale_mode, r.flags)
        parity.compare(bits, r, o, ref)


def test_bf16_fallback_copies_only_rejected_blocks():
    import torch

    g = np.concatenate([wl.gradient_like(150, 1000, seed=54), wl.weight_like(150, 1000, seed=57)])
    host = np.zeros((300, 1008), dtype=np.uint16); host[:, :1000] = g
    x = parity.to_device(host)
    for block in [(1, 128), (128, 128), (64, 64), (128, 1)]:
        r = recipe(block, THREE)
        out = mb.analyze_quantize(x, r, cols=1000, fallback=True)
        torch.cuda.synchronize()
        fb = out.bf16_fallback.view(torch.int16).cpu().numpy().view(np.uint16)
        sel = out.sel.cpu().numpy()
        assert (sel == mb.MOR_FMT_BF16).any() and (sel != mb.MOR_FMT_BF16).any()
        br, bc = block
        for bi in range(sel.shape[0]):
            for bj in range(sel.shape[1]):
                sl = (slice(bi * br, min((bi + 1) * br, 300)), slice(bj * bc, min((bj + 1) * bc, 1000)))
                want = host[sl] if sel[bi, bj] == mb.MOR_FMT_BF16 else 0
                assert (fb[sl] == want).all()
        assert (fb[:, 1000:] == 0).all()


@pytest.mark.parametrize("block", [(128, 128), (64, 64)])
@pytest.mark.parametrize("formats", [TWO, THREE])
def test_batched_call_mixes_tensors_with_and_without_bf16_copy(block, formats):
    """One launch whose thread blocks walk through tiles of tensors that ask for the BF16 copy or the
    fake-quantised output and of tensors that do not: every tensor equals its own single call."""
    import torch

    n = 6
    host = [wl.gradient_like(2048, 2048, seed=300 + i) if i % 2 else wl.weight_like(2048, 2048, seed=300 + i)
            for i in range(n)]
    xs = [parity.to_device(h) for h in host]
    r = recipe(block, formats)
    fb = [False, True, False, False, True, False]
    fq = [False, False, True, False, True, False]
    plan = mb.BatchPlan(xs, [r] * n, block_stats=True, fallback=fb, fake_quant=fq)
    plan.run()
    plan.run()
    torch.cuda.synchronize()
    for i in range(n):
        single = mb.analyze_quantize(xs[i], r, block_stats=True, fallback=fb[i], fake_quant=fq[i])
        torch.cuda.synchronize()
        o = plan.outs[i]
        assert o.tensor_stats_dict() == single.tensor_stats_dict() and o.tensor_stats_dict()["status"] == 0
        assert torch.equal(o.codes, single.codes) and torch.equal(o.sel, single.sel)
        if fb[i]:
            assert torch.equal(o.bf16_fallback, single.bf16_fallback)
        if fq[i]:
            assert torch.equal(o.fake_quant.view(torch.int16), single.fake_quant.view(torch.int16))
    ref = orc.run(host[4], r.block, list(r.formats), r.criterion, r.threshold, n_threads=8)
    parity.compare(host[4], r, plan.outs[4], ref)


def test_batched_call_equals_single_calls():
    import torch

    cases = wl.llama_layer_cases(scale=16)
    cases += wl.config_case(0, scale=2) + wl.config_case(3, scale=16)
    xs = [parity.to_device(c.bits) for c in cases]
    recipes = [parity.recipe_from_case(c) for c in cases]
    plan = mb.BatchPlan(xs, recipes, block_stats=True)
    plan.run()
    torch.cuda.synchronize()
    for c, x, r, o in zip(cases, xs, recipes, plan.outs):
        single = mb.analyze_quantize(x, r, block_stats=True)
        torch.cuda.synchronize()
        assert o.tensor_stats_dict() == single.tensor_stats_dict(), c.name
        assert torch.equal(o.codes, single.codes) and torch.equal(o.sel, single.sel)
        assert torch.equal(o.scale_e8m0, single.scale_e8m0)
        ref = orc.run(c.bits, r.block, list(r.formats), r.criterion, r.threshold)
        parity.compare(c.bits, r, o, ref)


def test_many_tensors_exceeding_one_launch():
    import torch

    rng = np.random.default_rng(60)
    bits = [wl.weight_like(int(rng.integers(1, 300)), int(rng.integers(1, 40)) * 8, seed=61 + i) for i in range(47)]
    xs = [parity.to_device(b) for b in bits]
    recipes = [recipe(KINDS[i % 4]) for i in range(47)]
    plan = mb.BatchPlan(xs, recipes)
    plan.run()
    torch.cuda.synchronize()
    for b, r, o in zip(bits, recipes, plan.outs):
        ref = orc.run(b, r.block, list(r.formats), r.criterion, r.threshold)
        parity.compare(b, r, o, ref)


def test_error_histogram_counts_one_per_tensor_and_call():
    """Section 4.1.3: every call adds one count to the bin of the tensor's error; the counters persist
    across calls and may be shared by the tensors of a batch."""
    import torch

    cases = [wl.weight_like(512, 512, seed=81), wl.gradient_like(384, 640, seed=82), wl.gaussian_outlier_rows(),
             wl.activation_like(256, 512, seed=83), np.zeros((128, 128), dtype=np.uint16)]
    hist = torch.zeros((mb.MOR_ERROR_BINS,), dtype=torch.int32, device="cuda")
    want = np.zeros(mb.MOR_ERROR_BINS, dtype=np.int64)
    r = recipe((128, 128), TWO)
    for bits in cases:
        out = mb.analyze_quantize(parity.to_device(bits), r, error_histogram=hist)
        torch.cuda.synchronize()
        ref = orc.run(bits, r.block, list(r.formats), r.criterion, r.threshold)
        mean = ref.tensor["mean_rel_e4m3"]
        edge = min(abs(mean - 0.005 * k) for k in range(1, 12))
        assert edge > 1e-5 * max(mean, 1e-30), "a case on a bin edge proves nothing"
        want[orc.error_bin(mean)] += 1
        assert out.tensor_stats_dict()["status"] == 0
    assert hist.cpu().numpy().tolist() == want.tolist() and want.sum() == len(cases)
    assert len(set(np.nonzero(want)[0])) >= 3                          # the cases spread over several bins
    # one shared row of counters for a whole batch, two steps
    per = [torch.zeros((mb.MOR_ERROR_BINS,), dtype=torch.int32, device="cuda") for _ in cases[:4]]
    plan = mb.BatchPlan([parity.to_device(b) for b in cases[:4]], [r] * 4, error_histograms=[hist] * 2 + per[2:])
    plan.run()
    plan.run()
    torch.cuda.synchronize()
    want2 = want.copy()
    for i, bits in enumerate(cases[:4]):
        ref = orc.run(bits, r.block, list(r.formats), r.criterion, r.threshold)
        k = orc.error_bin(ref.tensor["mean_rel_e4m3"])
        if i < 2:
            want2[k] += 2
        else:
            assert per[i].cpu().numpy().tolist() == [2 if j == k else 0 for j in range(mb.MOR_ERROR_BINS)]
    assert hist.cpu().numpy().tolist() == want2.tolist()


def test_two_host_threads_on_two_streams():
    """Calls from two host threads, each with its own stream, tensors, outputs and workspace, may overlap on the
    host and on the GPU; every result equals the single-threaded one."""
    import threading

    import torch

    cases = [(wl.gradient_like(700, 1024, seed=91), recipe((1, 128), THREE)),
             (wl.weight_like(900, 768, seed=92), recipe((128, 128), TWO))]
    xs = [parity.to_device(b) for b, _ in cases]
    want = [mb.analyze_quantize(x, r, block_stats=True) for x, (_, r) in zip(xs, cases)]
    torch.cuda.synchronize()
    plans = [mb.BatchPlan([x], [r], block_stats=True) for x, (_, r) in zip(xs, cases)]
    streams = [torch.cuda.Stream() for _ in cases]
    errors = []

    def work(i):
        try:
            for _ in range(50):
                plans[i].run(streams[i])
            streams[i].synchronize()
        except Exception as e:      # noqa: BLE001
            errors.append(e)

    threads = [threading.Thread(target=work, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for p, w in zip(plans, want):
        o = p.outs[0]
        assert o.tensor_stats_dict() == w.tensor_stats_dict() and o.tensor_stats_dict()["status"] == 0
        assert torch.equal(o.codes, w.codes) and torch.equal(o.sel, w.sel) and torch.equal(o.block_stats, w.block_stats)


def test_step_captured_as_cuda_graph_replays_identically():
    """BatchPlan.capture(): the memset and the three kernels as one CUDA graph; two replays, each checked
    against the oracle after the outputs were overwritten."""
    import torch

    bits = wl.gradient_like(300, 992, seed=77)
    r = recipe((1, 128), THREE)
    plan = mb.BatchPlan([parity.to_device(bits)], [r], block_stats=True)
    graph = plan.capture()
    ref = orc.run(bits, r.block, list(r.formats), r.criterion, r.threshold)
    for _ in range(2):
        plan.outs[0].codes.zero_()
        plan.outs[0].sel.fill_(9)
        plan.outs[0].tensor_stats.zero_()
        graph.replay()
        torch.cuda.synchronize()
        parity.compare(bits, r, plan.outs[0], ref)


def test_runs_are_deterministic():
    import torch

    g = wl.gradient_like(512, 2048, seed=55)
    x = parity.to_device(g)
    for block in KINDS:
        r = recipe(block, THREE if block != (0, 0) else TWO)
        a = mb.analyze_quantize(x, r, block_stats=True)
        b = mb.analyze_quantize(x, r, block_stats=True)
        torch.cuda.synchronize()
        assert torch.equal(a.codes, b.codes) and torch.equal(a.sel, b.sel) and torch.equal(a.tensor_stats, b.tensor_stats)
        assert torch.equal(a.block_stats, b.block_stats)


def test_host_memory_entry_point():
    import ctypes as C
    import torch

    g = wl.gradient_like(300, 1000, seed=56)
    host = np.zeros((300, 1008), dtype=np.uint16); host[:, :1000] = g
    r = recipe((1, 128), THREE)
    hx = torch.from_numpy(host.view(np.int16)).pin_memory()
    d = mb.make_desc(hx.data_ptr(), 300, 1000, 1008, r)
    grid = mb.grid_of(300, 1000, r.block)
    codes = torch.zeros((300, 1000), dtype=torch.uint8).pin_memory()
    scale = torch.zeros(grid, dtype=torch.uint8).pin_memory()
    sel = torch.zeros(grid, dtype=torch.uint8).pin_memory()
    ts = torch.zeros((mb.TENSOR_STATS_DTYPE.itemsize,), dtype=torch.uint8).pin_memory()
    o = mb.mor_outputs_t()
    o.codes, o.codes_ld, o.scale_e8m0, o.sel, o.tensor_stats = codes.data_ptr(), 1000, scale.data_ptr(), sel.data_ptr(), ts.data_ptr()
    nbytes = mb.mor_host_staging_bytes(d)
    staging = torch.empty((nbytes,), dtype=torch.uint8, device="cuda")
    st = mb.mor_analyze_quantize_host(d, o, staging.data_ptr(), nbytes, torch.cuda.current_stream().cuda_stream)
    assert st == mb.MOR_OK
    torch.cuda.synchronize()
    ref = orc.run(host, r.block, list(r.formats), r.criterion, r.threshold, cols=1000)
    np.testing.assert_array_equal(codes.numpy(), ref.codes)
    np.testing.assert_array_equal(sel.numpy().reshape(-1), ref.sel)
    np.testing.assert_array_equal(scale.numpy().reshape(-1), ref.scale_e8m0)
    rec = ts.numpy().view(mb.TENSOR_STATS_DTYPE)[0]
    assert rec["nnz"] == ref.tensor["nnz"] and rec["group_mantissa"] == ref.tensor["group_mantissa"]


def test_invalid_arguments_launch_nothing():
    import torch

    x = torch.zeros((128, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mb.MorError) as e:
        mb.analyze_quantize(x, recipe((32, 32)))
    assert e.value.status == mb.MOR_ERR_UNSUPPORTED
    with pytest.raises(mb.MorError) as e:
        mb.analyze_quantize(x, recipe((1, 128), (mb.MOR_FMT_E5M2, mb.MOR_FMT_E4M3, mb.MOR_FMT_BF16)))
    assert e.value.status == mb.MOR_ERR_UNSUPPORTED
    with pytest.raises(mb.MorError) as e:
        mb.analyze_quantize(x[:, 1:], recipe((1, 128)))                     # misaligned base, odd leading dimension
    assert e.value.status == mb.MOR_ERR_ALIGNMENT
    d = mb.desc_for(x, recipe((1, 128)))
    o = mb.alloc_outputs(128, 256, recipe((1, 128)), x.device)
    assert mb.mor_analyze_quantize(d, o.c_struct, 0, 0) == mb.MOR_ERR_WORKSPACE
    torch.cuda.synchronize()


@pytest.mark.parametrize("shape", [(256, 256), (384, 200), (130, 520), (517, 72), (2560, 2048)])
def test_full_width_column_path_edge_cases(shape):
    """128x1 blocks, plain two-format recipe with the pre-pass (per-column scales prepared by the load warp, four
    columns x 16 rows per thread): columns of zeros, a column piece whose amax is tiny (its scale exponent is beyond
    what the fast conversion takes), NaN and infinities (their blocks stay in BF16, the tile takes the careful path),
    ragged edges in both directions, and more tiles than resident CTAs."""
    rows, cols = shape
    g = wl.weight_like(rows, cols, seed=71)
    g[:, 3] = 0                                   # zeros all the way down
    g[: min(rows, 128), 9] = 0x0001               # smallest subnormal: the largest scale there is
    g[5, 20] = 0x7FC0
    if rows > 140:
        g[140, 21] = 0xFF80
        g[128:, 40] = wl.gradient_like(rows - 128, 1, seed=72)[:, 0]      # a wide spread of exponents down a column
    ld = (cols + 7) // 8 * 8
    for r in (recipe((128, 1), TWO), recipe((128, 1), TWO, mb.MOR_CRIT_TENSOR_MEAN_REL), recipe((128, 1), TWO, scale_mode=mb.MOR_SCALE_E8M0)):
        rep = parity.run_and_compare(g, r, pad_to=ld if ld != cols else None, block_stats=False)
        assert rep.n_exempt <= 2
