"""ctypes front end of the CPU oracle (``mor_oracle.c``).

TEST INFRASTRUCTURE: imported only by the tests, the smoke check and the benchmark's
CPU-baseline leg.  Nothing here touches the CUDA library or its binding.

The C file is compiled on first use (gcc, -O2, no fast-math, no FMA contraction) into
``libmor_oracle.so`` next to it, and rebuilt when the source is newer than the library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mor_oracle.c")
_LIB = os.path.join(_HERE, "libmor_oracle.so")
# The pins are themselves tested by running them against deliberately wrong copies of the C file
# (tests/test_oracle_planted_mistakes.py); such a run names the source and the library to use here.
if os.environ.get("MOR_ORACLE_SRC") and os.environ.get("MOR_ORACLE_LIB"):
    _SRC, _LIB = os.environ["MOR_ORACLE_SRC"], os.environ["MOR_ORACLE_LIB"]

FMT_E4M3, FMT_E5M2, FMT_BF16 = 0, 1, 2
CRIT_TENSOR_MEAN_REL, CRIT_BLOCK_VS_E5M2, CRIT_BLOCK_MEAN_REL = 0, 1, 2
SCALE_GAM, SCALE_E8M0, SCALE_FP32_AMAX = 0, 1, 2
FLAG_STRICT_TIES, FLAG_RANGE_MIN_INCLUDES_ZERO = 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle if the library is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-Wall", "-Wextra", "-fPIC", "-shared", "-ffp-contract=off",
               "-fopenmp", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB


class Cfg(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64),
                ("block_rows", C.c_int32), ("block_cols", C.c_int32),
                ("n_formats", C.c_int32), ("criterion", C.c_int32),
                ("threshold", C.c_double), ("scale_mode", C.c_int32), ("flags", C.c_uint32),
                ("have_group_amax", C.c_int32), ("group_amax", C.c_float)]


class Block(C.Structure):
    _fields_ = [("amax", C.c_double), ("min_abs_nz", C.c_double), ("nnz", C.c_int64),
                ("sum_rel_e4m3", C.c_double), ("sum_rel_e5m2", C.c_double),
                ("n_nonfinite", C.c_int64), ("scale_e4m3", C.c_float), ("scale_e5m2", C.c_float),
                ("exp_e4m3", C.c_int32), ("exp_e5m2", C.c_int32), ("sel", C.c_int32),
                ("has_zero", C.c_int32)]


class Tensor(C.Structure):
    _fields_ = [("sum_rel_e4m3", C.c_double), ("nnz", C.c_int64), ("mean_rel_e4m3", C.c_double),
                ("group_amax", C.c_float), ("group_mantissa", C.c_uint32),
                ("tensor_format", C.c_int32),
                ("n_blocks", C.c_int64), ("n_e4m3", C.c_int64), ("n_e5m2", C.c_int64),
                ("n_bf16", C.c_int64), ("n_nonfinite", C.c_int64)]


BLOCK_DTYPE = np.dtype([("amax", "f8"), ("min_abs_nz", "f8"), ("nnz", "i8"),
                        ("sum_rel_e4m3", "f8"), ("sum_rel_e5m2", "f8"), ("n_nonfinite", "i8"),
                        ("scale_e4m3", "f4"), ("scale_e5m2", "f4"), ("exp_e4m3", "i4"),
                        ("exp_e5m2", "i4"), ("sel", "i4"), ("has_zero", "i4")])

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        assert L.orc_sizeof_cfg() == C.sizeof(Cfg)
        assert L.orc_sizeof_block() == C.sizeof(Block) == BLOCK_DTYPE.itemsize
        assert L.orc_sizeof_tensor() == C.sizeof(Tensor)
        L.orc_bf16_to_float.restype = C.c_float
        L.orc_bf16_to_float.argtypes = [C.c_uint16]
        for n in ("orc_decode_e4m3", "orc_decode_e5m2"):
            getattr(L, n).restype = C.c_double
            getattr(L, n).argtypes = [C.c_uint8]
        for n in ("orc_encode_e4m3", "orc_encode_e5m2", "orc_encode_e4m3_exhaustive", "orc_encode_e5m2_exhaustive"):
            getattr(L, n).restype = C.c_uint8
            getattr(L, n).argtypes = [C.c_float]
        L.orc_group_mantissa.restype = C.c_uint32
        L.orc_group_mantissa.argtypes = [C.c_float, C.c_int]
        L.orc_block_scale.restype = None
        L.orc_block_scale.argtypes = [C.c_float, C.c_uint32, C.c_int, C.POINTER(C.c_float),
                                      C.POINTER(C.c_int32), C.POINTER(C.c_float), C.POINTER(C.c_int32)]
        L.orc_tensor_amax.restype = C.c_float
        L.orc_tensor_amax.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64]
        L.orc_num_blocks.restype = C.c_int64
        L.orc_num_blocks.argtypes = [C.POINTER(Cfg)]
        L.orc_run_blocks.restype = C.c_int
        L.orc_run_blocks.argtypes = [C.POINTER(Cfg), C.c_void_p, C.c_void_p, C.c_int64,
                                     C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.POINTER(Tensor), C.c_int]
        L.orc_error_bin.restype = C.c_int
        L.orc_error_bin.argtypes = [C.c_double]
        L.orc_fake_quant.restype = C.c_int
        L.orc_fake_quant.argtypes = [C.POINTER(Cfg), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64]
        L.orc_scale_value.restype = C.c_float
        L.orc_scale_value.argtypes = [C.c_float, C.c_float]
        L.orc_f32_to_bf16.restype = C.c_uint16
        L.orc_f32_to_bf16.argtypes = [C.c_float]
        for n in ("orc_rel_err_e4m3", "orc_rel_err_e5m2"):
            getattr(L, n).restype = C.c_double
            getattr(L, n).argtypes = [C.c_float]
        _lib = L
    return _lib


# ----------------------------------------------------------------- element level ----

def decode_e4m3(code: int) -> float:
    return lib().orc_decode_e4m3(code)


def decode_e5m2(code: int) -> float:
    return lib().orc_decode_e5m2(code)


def encode_e4m3(y: float, exhaustive: bool = False) -> int:
    L = lib()
    return (L.orc_encode_e4m3_exhaustive if exhaustive else L.orc_encode_e4m3)(y)


def encode_e5m2(y: float, exhaustive: bool = False) -> int:
    L = lib()
    return (L.orc_encode_e5m2_exhaustive if exhaustive else L.orc_encode_e5m2)(y)


def group_mantissa(g_amax: float, scale_mode: int = SCALE_GAM) -> int:
    return lib().orc_group_mantissa(g_amax, scale_mode)


def block_scale(b_amax: float, m_g: int, scale_mode: int = SCALE_GAM):
    """(scale_e4m3, exp_e4m3, scale_e5m2, exp_e5m2) of Algorithm 1 for one block."""
    s4, s5, e4, e5 = C.c_float(), C.c_float(), C.c_int32(), C.c_int32()
    lib().orc_block_scale(b_amax, m_g, scale_mode, C.byref(s4), C.byref(e4), C.byref(s5), C.byref(e5))
    return s4.value, e4.value, s5.value, e5.value


def scale_value(x: float, scale: float) -> float:
    return lib().orc_scale_value(x, scale)


def f32_to_bf16(f: float) -> int:
    """BF16 bits of a binary32 value, round to nearest even (the last step of fake quantisation)."""
    return lib().orc_f32_to_bf16(f)


def rel_err_e4m3(y: float) -> float:
    return lib().orc_rel_err_e4m3(y)


def rel_err_e5m2(y: float) -> float:
    return lib().orc_rel_err_e5m2(y)


# ------------------------------------------------------------------ tensor level ----

@dataclass
class Result:
    codes: Optional[np.ndarray]       # uint8 [rows, cols] (only listed blocks are written)
    scale_e8m0: np.ndarray            # uint8 [n_blocks_total]
    sel: np.ndarray                   # uint8 [n_blocks_total]
    scale_f32: np.ndarray             # float32 [n_blocks_total]
    blocks: np.ndarray                # BLOCK_DTYPE, one record per listed block
    tensor: dict
    grid: tuple                       # (block rows, block cols) of the block grid
    ids: Optional[np.ndarray]


def make_cfg(rows, cols, ld, block, formats: Sequence[int], criterion, threshold=0.045,
             scale_mode=SCALE_GAM, flags=0, group_amax=None) -> Cfg:
    formats = list(formats)
    if formats not in ([FMT_E4M3, FMT_BF16], [FMT_E4M3, FMT_E5M2, FMT_BF16]):
        raise ValueError("ordered format list must be [E4M3, BF16] or [E4M3, E5M2, BF16]")
    cfg = Cfg()
    cfg.rows, cfg.cols, cfg.ld = rows, cols, ld
    cfg.block_rows, cfg.block_cols = block
    cfg.n_formats, cfg.criterion = len(formats), criterion
    # the boundary carries the threshold as a binary32; compare against that value
    cfg.threshold = float(np.float32(threshold))
    cfg.scale_mode, cfg.flags = scale_mode, flags
    cfg.have_group_amax = 0 if group_amax is None else 1
    cfg.group_amax = 0.0 if group_amax is None else float(group_amax)
    return cfg


def grid_of(rows, cols, block):
    if block == (0, 0):
        return (1, 1) if rows > 0 and cols > 0 else (0, 0)
    if rows == 0 or cols == 0:
        return (0, 0)
    return (-(-rows // block[0]), -(-cols // block[1]))


def run(bits: np.ndarray, block, formats, criterion, threshold=0.045, scale_mode=SCALE_GAM,
        flags=0, group_amax=None, ids=None, want_codes=True, n_threads=1, cols=None) -> Result:
    """Analyse a BF16 tensor given as uint16 bit patterns [rows, ld].

    ``cols`` (default: ld) is the number of valid columns when the rows are padded.
    ``ids`` restricts the work to the listed linear block indices (the group amax is still
    the whole tensor's unless ``group_amax`` is given).
    """
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    assert bits.ndim == 2
    rows, ld_ = bits.shape
    cols = ld_ if cols is None else cols
    cfg = make_cfg(rows, cols, ld_, tuple(block), formats, criterion, threshold, scale_mode, flags, group_amax)
    L = lib()
    nb = int(L.orc_num_blocks(C.byref(cfg)))
    grid = grid_of(rows, cols, tuple(block))
    assert grid[0] * grid[1] == nb
    ids_arr = None if ids is None else np.ascontiguousarray(ids, dtype=np.int64)
    n = nb if ids_arr is None else len(ids_arr)
    codes = np.zeros((rows, cols), dtype=np.uint8) if want_codes else None
    scale = np.zeros(max(nb, 1), dtype=np.uint8)
    sel = np.zeros(max(nb, 1), dtype=np.uint8)
    sf32 = np.zeros(max(nb, 1), dtype=np.float32)
    blocks = np.zeros(max(n, 1), dtype=BLOCK_DTYPE)
    t = Tensor()
    rc = L.orc_run_blocks(C.byref(cfg), bits.ctypes.data,
                          None if ids_arr is None else ids_arr.ctypes.data, n,
                          None if codes is None else codes.ctypes.data, cols,
                          scale.ctypes.data, sel.ctypes.data, sf32.ctypes.data,
                          blocks.ctypes.data, C.byref(t), n_threads)
    if rc != 0:
        raise ValueError(f"oracle rejected the recipe (rc={rc})")
    td = {k: getattr(t, k) for k, _ in Tensor._fields_}
    return Result(codes, scale[:nb], sel[:nb], sf32[:nb], blocks[:n], td, grid, ids_arr)


def error_bin(mean_rel: float) -> int:
    """Bin of the 12-bin relative-error histogram (Section 4.1.3) that a tensor-level error falls into."""
    return int(lib().orc_error_bin(float(mean_rel)))


def fake_quant(bits: np.ndarray, res: Result, block, formats, criterion, threshold=0.045, scale_mode=SCALE_GAM,
               flags=0, cols=None) -> np.ndarray:
    """BF16 bit patterns of the fake-quantised tensor (quantise, dequantise, de-scale) for a finished run."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    rows, ld_ = bits.shape
    cols = ld_ if cols is None else cols
    cfg = make_cfg(rows, cols, ld_, tuple(block), formats, criterion, threshold, scale_mode, flags, None)
    out = np.zeros((rows, cols), dtype=np.uint16)
    sel = np.ascontiguousarray(res.sel, dtype=np.uint8)
    sf = np.ascontiguousarray(res.scale_f32, dtype=np.float32)
    rc = lib().orc_fake_quant(C.byref(cfg), bits.ctypes.data, sel.ctypes.data, sf.ctypes.data, out.ctypes.data, cols)
    assert rc == 0
    return out


def tensor_amax(bits: np.ndarray) -> float:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return lib().orc_tensor_amax(bits.ctypes.data, bits.shape[0], bits.shape[1], bits.shape[1])
