"""Parity at the benchmark's full sizes, in the launch configuration that bench.py times.

Small tensors are compared with the oracle element by element elsewhere; here the tensors have
the configurations' real shapes.  Where the oracle finishes in seconds the whole tensor is
compared; for the largest one a seeded sample of blocks is (the oracle computes any listed block
on its own), together with properties that hold at any size.
"""
import numpy as np
import pytest

from oracle import mor_oracle as orc
from paper_2512_22804_b200 import binding as mb
from paper_2512_22804_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

TWO = (mb.MOR_FMT_E4M3, mb.MOR_FMT_BF16)
THREE = (mb.MOR_FMT_E4M3, mb.MOR_FMT_E5M2, mb.MOR_FMT_BF16)


def test_config0_per_tensor_full():
    case = wl.config_case(0)[0]
    rep = parity.run_and_compare(case.bits, parity.recipe_from_case(case))
    assert rep.n_blocks == 1 and not rep.tensor_exempt


def test_config1_batched_launch_as_benchmarked():
    """16 distinct 4096x4096 weight-like tensors in one batched call (bench.py's step); two of them
    compared in full, the others on sampled blocks."""
    import torch

    B = 16
    host = [wl.weight_like(4096, 4096, seed=1 + 1000 * i) for i in range(B)]
    xs = [parity.to_device(h) for h in host]
    r = mb.Recipe((128, 128), TWO, mb.MOR_CRIT_BLOCK_VS_E5M2, 0.045)
    plan = mb.BatchPlan(xs, [r] * B)     # as bench.py builds it: no optional outputs (the plain instantiation)
    plan.run()
    plan.run()                       # the second step must overwrite the first one's results identically
    torch.cuda.synchronize()
    rng = np.random.default_rng(5)
    exempt = 0
    for i in range(B):
        if i in (0, B - 1):
            ref = orc.run(host[i], r.block, list(r.formats), r.criterion, r.threshold, n_threads=8)
            exempt += parity.compare(host[i], r, plan.outs[i], ref).n_exempt
        else:
            ids = np.sort(rng.choice(1024, 24, replace=False))
            ref = orc.run(host[i], r.block, list(r.formats), r.criterion, r.threshold, ids=ids)
            exempt += parity.compare(host[i], r, plan.outs[i], ref, ids=ids).n_exempt
        ts = plan.outs[i].tensor_stats_dict()
        assert ts["n_e4m3"] + ts["n_e5m2"] + ts["n_bf16"] == ts["n_blocks"] == 1024 and ts["status"] == 0
    assert exempt <= 2


def test_config2_activation_1x128_full():
    case = wl.config_case(2)[0]
    r = parity.recipe_from_case(case)
    x = parity.to_device(case.bits)
    out = mb.analyze_quantize(x, r, block_stats=True, scale_f32=True)
    ref = orc.run(case.bits, r.block, list(r.formats), r.criterion, r.threshold, n_threads=8)
    rep = parity.compare(case.bits, r, out, ref)
    assert rep.n_blocks == 8192 * 32 and rep.n_exempt <= 262


@pytest.mark.parametrize("block", [(1, 128), (128, 128)])
def test_config3_gradient_three_way_sampled(block):
    """8192 x 14336, [E4M3, E5M2, BF16]: sampled blocks against the oracle plus whole-tensor properties."""
    g = wl.gradient_like()
    r = mb.Recipe(block, THREE, mb.MOR_CRIT_BLOCK_VS_E5M2, 0.045)
    x = parity.to_device(g)
    out = mb.analyze_quantize(x, r, block_stats=True, scale_f32=True)
    ts = out.tensor_stats_dict()
    grid = mb.grid_of(g.shape[0], g.shape[1], block)
    nb = grid[0] * grid[1]
    rng = np.random.default_rng(11)
    ids = np.sort(rng.choice(nb, 4096 if block == (1, 128) else 96, replace=False))
    ref = orc.run(g, block, list(THREE), r.criterion, r.threshold, ids=ids)
    rep = parity.compare(g, r, out, ref, ids=ids)
    assert rep.n_exempt <= 4
    # properties that need no oracle run over the whole tensor
    assert ts["n_blocks"] == nb == ts["n_e4m3"] + ts["n_e5m2"] + ts["n_bf16"]
    assert ts["nnz"] == int(np.count_nonzero(g & 0x7FFF)) and ts["n_nonfinite"] == 0 and ts["status"] == 0
    assert ts["group_amax"] == orc.tensor_amax(g)
    sel = out.sel.cpu().numpy().reshape(-1)
    assert np.bincount(sel, minlength=3).tolist() == [ts["n_e4m3"], ts["n_e5m2"], ts["n_bf16"]]
    bs = out.block_stats_array()[:nb]
    assert int(bs["nnz"].astype(np.int64).sum()) == ts["nnz"]
    assert abs(float(bs["sum_rel_e4m3"].astype(np.float64).sum()) - ts["sum_rel_e4m3"]) <= 1e-6 * ts["sum_rel_e4m3"]
    # a block kept in E4M3 never has a larger E4M3 error sum than E5M2 error sum (Eq. 3)
    kept = sel == mb.MOR_FMT_E4M3
    assert (bs["sum_rel_e4m3"][kept] <= bs["sum_rel_e5m2"][kept]).all()
    # E8M0 byte of an E5M2 block is 7 above the E4M3 exponent of the same amax (57344 = 448 * 2^7)
    codes = out.codes_view().cpu().numpy()
    assert codes.shape == g.shape


def test_config4_llama_layer_one_batched_call():
    """All 14 operands of one layer in a single batched call, full size; each tensor checked on sampled
    blocks and on its summary's consistency."""
    import torch

    cases = wl.llama_layer_cases()
    xs = [parity.to_device(c.bits) for c in cases]
    recipes = [parity.recipe_from_case(c) for c in cases]
    plan = mb.BatchPlan(xs, recipes)
    plan.run()
    torch.cuda.synchronize()
    rng = np.random.default_rng(13)
    for c, r, o in zip(cases, recipes, plan.outs):
        grid = mb.grid_of(c.bits.shape[0], c.bits.shape[1], r.block)
        nb = grid[0] * grid[1]
        ids = np.sort(rng.choice(nb, 16 if r.block == (128, 128) else 512, replace=False))
        ref = orc.run(c.bits, r.block, list(r.formats), r.criterion, r.threshold, ids=ids)
        parity.compare(c.bits, r, o, ref, ids=ids, check_block_stats=False)
        ts = o.tensor_stats_dict()
        assert ts["n_blocks"] == nb == ts["n_e4m3"] + ts["n_e5m2"] + ts["n_bf16"], c.name
        assert ts["nnz"] == int(np.count_nonzero(c.bits & 0x7FFF)), c.name


@pytest.mark.parametrize("block,formats", [((128, 128), TWO), ((1, 128), THREE)])
def test_tensor_with_more_than_2_31_elements(block, formats):
    """70000 x 33000 (2.31 G elements, 4.6 GB): element offsets pass 2^31 and 2^32 bytes.  Sampled blocks, among
    them the first, the middle and the last ones, against the oracle; counts over the whole tensor."""
    import torch

    rows, cols = 70000, 33000
    gen = torch.Generator(device="cuda").manual_seed(5)
    x = (torch.randn((rows, cols), device="cuda", generator=gen, dtype=torch.float32) * 0.02).to(torch.bfloat16)
    x[rows - 1, cols - 1] = 3.0                     # the amax sits at the very end
    x[12345, 6789] = 0.0
    host = x.view(torch.int16).cpu().numpy().view(np.uint16)
    r = mb.Recipe(block, formats, mb.MOR_CRIT_BLOCK_VS_E5M2, 0.045)
    out = mb.analyze_quantize(x, r, block_stats=True, scale_f32=True)
    torch.cuda.synchronize()
    ts = out.tensor_stats_dict()
    grid = mb.grid_of(rows, cols, block)
    nb = grid[0] * grid[1]
    rng = np.random.default_rng(3)
    ids = np.unique(np.concatenate([rng.choice(nb, 200, replace=False), [0, nb - 1, nb - 2, nb // 2]]))
    ref = orc.run(host, block, list(formats), r.criterion, r.threshold, ids=ids)
    parity.compare(host, r, out, ref, ids=ids)
    assert ts["n_blocks"] == nb == ts["n_e4m3"] + ts["n_e5m2"] + ts["n_bf16"] and ts["status"] == 0
    assert ts["group_amax"] == 3.0 and ts["nnz"] == int(torch.count_nonzero(x).item())


def test_mixed_grid_128x128_three_way_full():
    """A 4096x4096 tensor whose 128x128 tiles differ (E4M3, E5M2 and BF16 blocks side by side), three formats, in
    bench.py's launch configuration (several copies in one batched call, no optional outputs) and with statistics;
    the whole tensor against the oracle."""
    import torch

    bits = wl.mixed_grid()
    r = mb.Recipe((128, 128), THREE, mb.MOR_CRIT_BLOCK_VS_E5M2, 0.045)
    ref = orc.run(bits, r.block, list(r.formats), r.criterion, r.threshold, n_threads=8)
    assert min(ref.tensor["n_e4m3"], ref.tensor["n_e5m2"], ref.tensor["n_bf16"]) > 100      # 459 / 388 / 177 tiles
    xs = [parity.to_device(bits) for _ in range(4)]
    for stats in (False, True):
        plan = mb.BatchPlan(xs, [r] * 4, block_stats=stats)
        plan.run()
        torch.cuda.synchronize()
        ex = sum(parity.compare(bits, r, o, ref).n_exempt for o in (plan.outs[0], plan.outs[3]))
        assert ex <= 4
        del plan
    # the same data with 1x128 and 64x64 blocks, sampled
    for block, nb in (((1, 128), 4096 * 32), ((64, 64), 64 * 64)):
        rr = mb.Recipe(block, THREE, mb.MOR_CRIT_BLOCK_VS_E5M2, 0.045)
        ids = np.sort(np.random.default_rng(6).choice(nb, 2000, replace=False))
        sub = orc.run(bits, block, list(THREE), rr.criterion, rr.threshold, ids=ids)
        out = mb.analyze_quantize(xs[0], rr)
        torch.cuda.synchronize()
        assert parity.compare(bits, rr, out, sub, ids=ids).n_exempt <= 4


def test_rows_and_columns_full_size_plain_paired_call_sampled():
    """8 configs[1]-sized tensors, each with 1x128 and with 128x1 blocks in one paired call of the plain two-format
    recipe (the launch configuration bench.py times for that line): the streaming row path and the full-width
    column path with keys of both directions from one pre-pass.  Sampled blocks of both directions against the
    oracle, whole-tensor counts, and the codes of the column direction as the transpose of what the row direction
    gives for the transposed tensor."""
    import torch

    hosts = [wl.weight_like(4096, 4096, seed=1 + 1000 * i) for i in range(3)]
    hosts[1][17, 4000] = 0x7F80           # an inf: its tile takes the careful path in both directions
    hosts[2][:, 77] = 0                   # a column of zeros
    hosts[2][300:428, 1000:1128] = wl.gradient_like(128, 128, seed=5)     # a tile with tiny and large values side by side
    xs = [parity.to_device(h) for h in hosts]
    rr, rc = mb.Recipe((1, 128), TWO, mb.MOR_CRIT_BLOCK_VS_E5M2, 0.045), mb.Recipe((128, 1), TWO, mb.MOR_CRIT_BLOCK_VS_E5M2, 0.045)
    px, pr = [], []
    for x in xs:
        px += [x, x]
        pr += [rr, rc]
    plan = mb.BatchPlan(px, pr)
    plan.run()
    plan.run()
    torch.cuda.synchronize()
    rng = np.random.default_rng(17)
    for i, h in enumerate(hosts):
        for r, o in ((rr, plan.outs[2 * i]), (rc, plan.outs[2 * i + 1])):
            grid = mb.grid_of(4096, 4096, r.block)
            nb = grid[0] * grid[1]
            ids = rng.choice(nb, 1024, replace=False)
            if i == 1:      # the blocks around the inf
                ids = np.concatenate([ids, [17 * 32 + 31] if r.block == (1, 128) else [0 * 4096 + 4000]])
            if i == 2 and r.block == (128, 1):
                ids = np.concatenate([ids, np.arange(32) * 4096 + 77, 2 * 4096 + 1000 + np.arange(128), 3 * 4096 + 1000 + np.arange(128)])
            ids = np.unique(ids)
            ref = orc.run(h, r.block, list(r.formats), r.criterion, r.threshold, ids=ids)
            parity.compare(h, r, o, ref, ids=ids, check_block_stats=False)
            ts = o.tensor_stats_dict()
            assert ts["status"] == 0 and ts["n_blocks"] == nb == ts["n_e4m3"] + ts["n_e5m2"] + ts["n_bf16"]
            assert ts["nnz"] == int(np.count_nonzero((h & 0x7FFF) != 0) - np.count_nonzero((h & 0x7FFF) >= 0x7F80))
            assert ts["n_nonfinite"] == int(np.count_nonzero((h & 0x7FFF) >= 0x7F80))
        # single calls give the same bytes
        single = mb.analyze_quantize(xs[i], rc)
        torch.cuda.synchronize()
        assert torch.equal(single.codes, plan.outs[2 * i + 1].codes) and torch.equal(single.sel, plan.outs[2 * i + 1].sel)
        xt = parity.to_device(np.ascontiguousarray(h.T))
        tr = mb.analyze_quantize(xt, rr)
        torch.cuda.synchronize()
        assert torch.equal(tr.codes, plan.outs[2 * i + 1].codes)
        assert torch.equal(tr.sel.t().contiguous(), plan.outs[2 * i + 1].sel)
        assert torch.equal(tr.scale_e8m0.t().contiguous(), plan.outs[2 * i + 1].scale_e8m0)
