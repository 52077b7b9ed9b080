"""A bounded device-side wait that runs out: the call returns, reports MOR_ERR_TIMEOUT, and the next call is clean.

Nothing faults here.  A host-set test hook of the library (``mor_test_skip_tile_load``, exported but not part of
mor.h) makes the load warp of the main kernel leave out the TMA load of one tile and shortens the wait limit to
about a millisecond.  The tile's barrier then never completes; the compute warps' waits run out, the CTA sets the
status word and from then on keeps every barrier arrival but skips the work, the other CTAs finish normally, and
the finalise kernel copies the status into ``mor_tensor_stats_t.status``."""
import ctypes as C

import numpy as np
import pytest

from paper_2512_22804_b200 import binding as mb
from paper_2512_22804_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

TWO = (mb.MOR_FMT_E4M3, mb.MOR_FMT_BF16)
THREE = (mb.MOR_FMT_E4M3, mb.MOR_FMT_E5M2, mb.MOR_FMT_BF16)
NONE = 0xFFFFFFFF


def hook(name="mor_test_skip_tile_load"):
    f = getattr(mb.load(), name)
    f.argtypes, f.restype = [C.c_uint32, C.c_longlong], None
    return f


CASES = [
    ("128x128 two-way, keys from the pre-pass (streaming)", (128, 128), TWO, {}, False),
    ("128x128 three-way (stash in the stage, decision round trip)", (128, 128), THREE, {}, False),
    ("1x128 three-way", (1, 128), THREE, {}, False),
    ("1x128 two-way (decisions and metadata in the store warp)", (1, 128), TWO, {}, False),
    ("per channel along the columns, tensor-level decision (full-width column path)", (0, 1), TWO, {}, False),
    ("64x64 with statistics and a fake-quantised output (register path)", (64, 64), THREE, dict(block_stats=True, fake_quant=True), False),
    ("128x128, group amax supplied (the kernel scans, CTA-wide exchange)", (128, 128), TWO, {}, True),
    ("1x128, group amax supplied", (1, 128), TWO, {}, True),
    ("128x1 sub-column blocks", (128, 1), TWO, {}, False),
    ("per tensor", (0, 0), TWO, {}, False),
    ("per channel", (1, 0), TWO, {}, False),
    ("per channel along the columns, a decision per column with statistics", (0, 1), TWO, dict(block_stats=True), False),
]


@pytest.mark.parametrize("name,block,formats,kw,supplied", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("tile", [0, 5, 15])
def test_timeout_is_reported_and_the_workspace_recovers(name, block, formats, kw, supplied, tile):
    import torch

    bits = wl.gradient_like(512, 512, seed=97)                        # 16 tiles, one per thread block
    x = parity.to_device(bits)
    crit = mb.MOR_CRIT_TENSOR_MEAN_REL if block in ((0, 0), (1, 0)) or (block == (0, 1) and not kw) else mb.MOR_CRIT_BLOCK_VS_E5M2
    r = mb.Recipe(block, formats, crit)
    ga = mb.group_amax([x]) if supplied else None
    torch.cuda.synchronize()
    set_hook = hook()
    set_hook(tile, 2_000_000)
    try:
        out = mb.analyze_quantize(x, r, group_amax=ga, **kw)
        torch.cuda.synchronize()                                      # returns: nobody is left waiting
    finally:
        set_hook(NONE, 0)
    assert out.tensor_stats_dict()["status"] == mb.MOR_ERR_TIMEOUT
    # the same tensor again, hook off: everything as the oracle has it
    parity.run_and_compare(bits, r, group_amax_supplied=supplied, block_stats=bool(kw.get("block_stats", False)),
                           fake_quant=bool(kw.get("fake_quant", False)))


def test_timeout_in_a_paired_rows_and_columns_launch():
    import torch

    bits = wl.weight_like(256, 384, seed=98)
    x = parity.to_device(bits)
    rr = mb.Recipe((1, 128), TWO, mb.MOR_CRIT_BLOCK_VS_E5M2)
    rc = mb.Recipe((128, 1), TWO, mb.MOR_CRIT_BLOCK_VS_E5M2)
    plan = mb.BatchPlan([x, x], [rr, rc])
    set_hook = hook()
    set_hook(2, 2_000_000)
    try:
        plan.run()
        torch.cuda.synchronize()
    finally:
        set_hook(NONE, 0)
    assert [o.tensor_stats_dict()["status"] for o in plan.outs] == [mb.MOR_ERR_TIMEOUT, mb.MOR_ERR_TIMEOUT]
    plan.run()
    torch.cuda.synchronize()
    assert [o.tensor_stats_dict()["status"] for o in plan.outs] == [0, 0]
    want = mb.analyze_quantize(x, rr)
    torch.cuda.synchronize()
    assert torch.equal(plan.outs[0].codes, want.codes) and torch.equal(plan.outs[0].sel, want.sel)


@pytest.mark.parametrize("block,formats", [((128, 128), TWO), ((1, 128), THREE), ((128, 1), TWO), ((0, 1), TWO), ((64, 64), TWO)])
@pytest.mark.parametrize("tile", [0, 7, 15])
def test_timeout_in_the_amax_pre_pass(block, formats, tile):
    """The pre-pass streams its tiles through a ring of stages with TMA loads and bounded waits of its own; the
    second hook (``mor_test_skip_prepass_tile_load``) leaves one of its loads out.  Its CTA gives up on that tile, the
    call returns with MOR_ERR_TIMEOUT (the main kernel still runs, on whatever keys there are), and the next call
    is clean."""
    import torch

    bits = wl.gradient_like(512, 512, seed=99)
    x = parity.to_device(bits)
    crit = mb.MOR_CRIT_TENSOR_MEAN_REL if block == (0, 1) else mb.MOR_CRIT_BLOCK_VS_E5M2
    r = mb.Recipe(block, formats, crit)
    set_hook = hook("mor_test_skip_prepass_tile_load")
    set_hook(tile, 2_000_000)
    try:
        out = mb.analyze_quantize(x, r)
        torch.cuda.synchronize()
    finally:
        set_hook(NONE, 0)
    assert out.tensor_stats_dict()["status"] == mb.MOR_ERR_TIMEOUT
    parity.run_and_compare(bits, r)


def test_timeout_in_the_pre_pass_of_a_cta_with_several_tiles():
    """More tiles than resident CTAs: the CTA that loses a tile has others before and after it in its ring."""
    import torch

    bits = wl.weight_like(2560, 2048, seed=100)                       # 320 tiles on at most 296 CTAs
    x = parity.to_device(bits)
    r = mb.Recipe((128, 128), TWO, mb.MOR_CRIT_BLOCK_VS_E5M2)
    set_hook = hook("mor_test_skip_prepass_tile_load")
    set_hook(3, 2_000_000)
    try:
        out = mb.analyze_quantize(x, r)
        torch.cuda.synchronize()
    finally:
        set_hook(NONE, 0)
    assert out.tensor_stats_dict()["status"] == mb.MOR_ERR_TIMEOUT
    parity.run_and_compare(bits, r)
