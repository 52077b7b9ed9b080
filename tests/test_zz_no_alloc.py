"""mor_analyze_quantize_static: the entry point for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits: inside a host runtime that owns all
device memory, in a latency-critical loop that cannot afford the synchronisation an allocation
implies, or under a memory budget fixed at start-up.  For them the library carries its scratch in
a built-in array.  The check here: through the C boundary, the new entry point must give exactly
what mor_analyze_quantize gives with a caller-allocated workspace -- on two calls in a row that
differ in shape and recipe, so that whatever the first call left in the shared array would show
up in the second.  The file sorts last on purpose: a run that stops at the first failure has
already run every other test.
"""
import numpy as np
import pytest

from paper_2512_22804_b200 import binding as mb
from paper_2512_22804_b200 import workloads as wl
from tests import parity

THREE = (mb.MOR_FMT_E4M3, mb.MOR_FMT_E5M2, mb.MOR_FMT_BF16)
TWO = (mb.MOR_FMT_E4M3, mb.MOR_FMT_BF16)


def _both_ways(bits, recipe):
    import torch

    x = parity.to_device(bits)
    want = mb.analyze_quantize(x, recipe, block_stats=True)            # caller-allocated workspace
    d = mb.desc_for(x, recipe)
    got = mb.alloc_outputs(d.rows, d.cols, recipe, x.device, block_stats=True, scale_f32=True)
    stream = torch.cuda.current_stream().cuda_stream
    torch.cuda.synchronize()
    held = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
    st = mb.mor_analyze_quantize_static(d, got.c_struct, stream)
    assert st == mb.MOR_OK, mb.mor_status_string(st)
    torch.cuda.synchronize()
    # the call took no device memory: neither through torch's allocator nor from the driver (the first call of a
    # process may load the kernels' code, which is why the comparison is made on the repeat below as well)
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == held[:2]
    st = mb.mor_analyze_quantize_static(d, got.c_struct, stream)
    assert st == mb.MOR_OK
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    st = mb.mor_analyze_quantize_static(d, got.c_struct, stream)
    assert st == mb.MOR_OK
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    # against the CPU oracle, with the bar every parity test applies
    ob = parity.oracle_block(recipe.block, bits.shape[1])
    ref = parity.orc.run(bits, ob, list(recipe.formats), recipe.criterion, recipe.threshold, recipe.scale_mode, recipe.flags)
    parity.compare(bits, recipe, got, ref)
    # the two runs execute the same kernels on the same bytes: everything is bit-identical,
    # which is inside the tolerance the parity tests allow for the error sums
    assert torch.equal(got.codes, want.codes)
    assert torch.equal(got.sel, want.sel) and torch.equal(got.scale_e8m0, want.scale_e8m0)
    assert torch.equal(got.block_stats, want.block_stats)
    a, b = got.tensor_stats_dict(), want.tensor_stats_dict()
    assert a == b
    return a


@pytest.mark.gpu
def test_static_scratch_matches_workspace_variant_on_two_calls_in_a_row():
    # first call: many tiles, three-way recipe, non-finite inputs (fills the counters in the scratch)
    g = wl.gradient_like(640, 2048, seed=71)
    g[5, 9] = 0x7FC0
    g[600, 2047] = 0xFF80
    first = _both_ways(g, mb.Recipe((1, 128), THREE, mb.MOR_CRIT_BLOCK_VS_E5M2))
    assert first["n_nonfinite"] == 2 and first["n_blocks"] == 640 * 16
    # second call, straight after: fewer tiles, another partition and criterion, clean data
    w = wl.weight_like(300, 520, seed=72)
    second = _both_ways(w, mb.Recipe((128, 128), TWO, mb.MOR_CRIT_TENSOR_MEAN_REL))
    assert second["n_nonfinite"] == 0 and second["n_blocks"] == 3 * 5
    # and the per-tensor partition, whose block amax lives in the scratch
    _both_ways(wl.gaussian_outlier_rows(256, 256, seed=73), mb.Recipe((0, 0), TWO, mb.MOR_CRIT_TENSOR_MEAN_REL))
