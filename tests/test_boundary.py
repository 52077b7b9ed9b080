"""The C boundary without a GPU: the library loads, exports what the header declares, and
rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

from paper_2512_22804_b200 import binding as mb
from paper_2512_22804_b200 import build as mbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    mbuild.build()
    return mb.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "mor.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mor_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_entry_point_is_exported(lib):
    names = declared_functions()
    assert set(names) == set(mb.EXPORTS), "binding and header list the same entry points"
    for n in names:
        assert getattr(lib, n) is not None


def test_nothing_but_the_declared_entry_points_is_exported(lib):
    """The dynamic symbol table holds the mor_* functions of the header and nothing else of this library's
    own code (the CUDA runtime that is linked in statically may add names of its own)."""
    import subprocess

    out = subprocess.run(["nm", "-D", "--defined-only", mb.LIB_PATH], capture_output=True, text=True, check=True).stdout
    names = [line.split()[-1] for line in out.splitlines() if line.strip()]
    ours = [n for n in names if not n.startswith(("cuda", "__cuda", "_init", "_fini", "__bss_start", "_edata", "_end"))]
    hooks = [n for n in ours if n.startswith("mor_test_")]          # test hooks: exported, deliberately not in the header
    assert sorted(hooks) == ["mor_test_skip_prepass_tile_load", "mor_test_skip_tile_load"]
    assert sorted(n for n in ours if n not in hooks) == declared_functions(), ours


def test_version_and_status_strings(lib):
    assert mb.mor_version() >= 100
    seen = {mb.mor_status_string(s) for s in range(0, 8)}
    assert len(seen) == 8 and "ok" in seen


def desc(rows=256, cols=256, ld=None, block=(128, 128), formats=(0, 2), crit=mb.MOR_CRIT_BLOCK_VS_E5M2, x=0x1000):
    r = mb.Recipe(block, formats, crit)
    return mb.make_desc(x, rows, cols, cols if ld is None else ld, r)


def test_workspace_bytes(lib):
    assert mb.mor_workspace_bytes([desc(64 * 128, 64 * 128)]) >= 64 * 64 * 40
    small, big = mb.mor_workspace_bytes([desc(128, 128)]), mb.mor_workspace_bytes([desc(8192, 4096)])
    assert 0 < small < big and small % 256 == 0
    both = mb.mor_workspace_bytes([desc(128, 128), desc(8192, 4096, block=(1, 128))])
    assert both >= big
    assert mb.mor_workspace_bytes([desc(0, 128)]) > 0                     # empty tensors still get their slots
    assert lib.mor_workspace_bytes(None, 1) == 0
    assert mb.mor_workspace_bytes([desc(128, 128, block=(32, 32))]) == 0  # unsupported block shape


def out_struct(codes=0x2000, codes_ld=256, ts=0x3000):
    o = mb.mor_outputs_t()
    o.codes, o.codes_ld, o.tensor_stats = codes, codes_ld, ts
    o.scale_e8m0, o.sel = 0x4000, 0x5000
    return o


@pytest.mark.parametrize("d,o,want", [
    (desc(block=(32, 32)), out_struct(), mb.MOR_ERR_UNSUPPORTED),
    (desc(block=(128, 2)), out_struct(), mb.MOR_ERR_UNSUPPORTED),
    (desc(formats=(1, 0, 2)), out_struct(), mb.MOR_ERR_UNSUPPORTED),       # order is fixed: E4M3 first
    (desc(formats=(0, 1)), out_struct(), mb.MOR_ERR_UNSUPPORTED),
    (desc(formats=(0, 1, 2), crit=mb.MOR_CRIT_TENSOR_MEAN_REL), out_struct(), mb.MOR_ERR_UNSUPPORTED),
    (desc(formats=(0, 1, 2), block=(0, 0)), out_struct(), mb.MOR_ERR_UNSUPPORTED),
    (desc(block=(1, 0), formats=(0, 1, 2)), out_struct(), mb.MOR_ERR_UNSUPPORTED),   # per channel: two formats only
    (desc(rows=512, block=(128, 1)), out_struct(), mb.MOR_ERR_INVALID_ARG),  # transposed codes: codes_ld covers the rows
    (desc(rows=-1), out_struct(), mb.MOR_ERR_INVALID_ARG),
    (desc(ld=128), out_struct(), mb.MOR_ERR_INVALID_ARG),                  # ld < cols
    (desc(ld=260), out_struct(), mb.MOR_ERR_ALIGNMENT),                    # ld not a multiple of 8
    (desc(x=0x1002), out_struct(), mb.MOR_ERR_ALIGNMENT),
    (desc(x=0), out_struct(), mb.MOR_ERR_INVALID_ARG),
    (desc(crit=7), out_struct(), mb.MOR_ERR_INVALID_ARG),
    (desc(), out_struct(ts=0), mb.MOR_ERR_INVALID_ARG),
    (desc(), out_struct(codes=0), mb.MOR_ERR_INVALID_ARG),
    (desc(), out_struct(codes_ld=250), mb.MOR_ERR_INVALID_ARG),
    (desc(cols=250, ld=256), out_struct(codes_ld=250), mb.MOR_ERR_INVALID_ARG),   # codes_ld below roundup(cols, 16)
    (desc(), out_struct(codes=0x2004), mb.MOR_ERR_ALIGNMENT),
    (desc(), out_struct(), mb.MOR_ERR_WORKSPACE),                          # valid, but no workspace given
])
def test_bad_arguments_are_reported_before_any_launch(lib, d, o, want):
    assert mb.mor_analyze_quantize(d, o, 0, 0) == want


def test_threshold_and_flags_are_checked(lib):
    d = desc()
    d.threshold = float("nan")
    assert mb.mor_analyze_quantize(d, out_struct(), 0, 0) == mb.MOR_ERR_INVALID_ARG
    d = desc()
    d.flags = 8
    assert mb.mor_analyze_quantize(d, out_struct(), 0, 0) == mb.MOR_ERR_INVALID_ARG
    d = desc()
    d.scale_mode = mb.MOR_SCALE_FP32_AMAX                                   # needs the scale_f32 output
    assert mb.mor_analyze_quantize(d, out_struct(), 0, 0) == mb.MOR_ERR_INVALID_ARG


def test_misaligned_workspace_is_rejected(lib):
    d = desc()
    need = mb.mor_workspace_bytes([d])
    assert mb.mor_analyze_quantize(d, out_struct(), 0x10010, need) == mb.MOR_ERR_ALIGNMENT
    assert mb.mor_analyze_quantize(d, out_struct(), 0x10000, need - 1) == mb.MOR_ERR_WORKSPACE


def test_group_amax_checks_every_descriptor_before_it_launches(lib):
    """A bad descriptor anywhere in the list is reported although the first ones are fine; only the geometry is
    looked at (formats, criterion and threshold play no part in an amax)."""
    import ctypes as C

    good, bad = desc(), desc(ld=260)
    arr = (mb.mor_tensor_desc_t * 2)(good, bad)
    assert lib.mor_group_amax(arr, 2, C.c_void_p(0x6000), C.c_void_p(0x10000), 1 << 20, None) == mb.MOR_ERR_ALIGNMENT
    odd = desc()
    odd.n_formats = 9                                                        # not looked at by this entry point
    odd.rows = -1
    arr = (mb.mor_tensor_desc_t * 1)(odd)
    assert lib.mor_group_amax(arr, 1, C.c_void_p(0x6000), C.c_void_p(0x10000), 1 << 20, None) == mb.MOR_ERR_INVALID_ARG


def test_static_scratch_refuses_tensors_beyond_its_limit(lib):
    """The size check of mor_analyze_quantize_static comes before any CUDA call, so it can be exercised
    without a device: nothing is looked up, nothing is launched."""
    r = mb.Recipe((128, 128), (0, 2))
    rows = cols = 128 * 200                                              # 40,000 tiles * 56 B > 2 MiB
    d = mb.make_desc(0x10000, rows, cols, cols, r)
    assert mb.mor_workspace_bytes([d]) > mb.MOR_STATIC_SCRATCH_BYTES
    o = mb.mor_outputs_t()
    o.codes, o.codes_ld, o.tensor_stats, o.scale_e8m0, o.sel = 0x20000, cols, 0x30000, 0x40000, 0x50000
    st = mb.mor_analyze_quantize_static(d, o, 0)
    assert st == mb.MOR_ERR_STATIC_SCRATCH
    assert "built-in" in mb.mor_status_string(st)


def test_null_descriptors(lib):
    assert lib.mor_analyze_quantize(None, None, None, 0, None) == mb.MOR_ERR_INVALID_ARG
    assert lib.mor_analyze_quantize_batched(None, None, 3, None, 0, None) == mb.MOR_ERR_INVALID_ARG
    assert lib.mor_select_stats(None, None, None, None, None, None, 0, None) == mb.MOR_ERR_INVALID_ARG
    assert lib.mor_group_amax(None, 2, None, None, 0, None) == mb.MOR_ERR_INVALID_ARG
    assert lib.mor_host_staging_bytes(None) == 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(mb, "_lib", None)
    monkeypatch.setattr(mb, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        mb.load()
