"""ctypes binding of ``libmor_b200.so`` with the same names as the C entry points.

Argument marshalling only: every step of the analyse-and-quantise pass runs in the CUDA
kernels.  PyTorch is used for device memory and streams.  There is no CPU fallback: if the
library has not been built, the first call raises.

Low level (one-to-one with ``include/mor.h``):
    mor_workspace_bytes, mor_analyze_quantize, mor_analyze_quantize_batched,
    mor_analyze_quantize_batched_ex, mor_select_stats, mor_select_stats_batched, mor_group_amax, mor_host_staging_bytes, mor_analyze_quantize_host,
    mor_status_string, mor_version

Helpers that allocate outputs with torch and fill the descriptors:
    Recipe, alloc_outputs, analyze_quantize, select_stats, BatchPlan
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmor_b200.so")

MOR_OK = 0
(MOR_ERR_INVALID_ARG, MOR_ERR_UNSUPPORTED, MOR_ERR_ALIGNMENT, MOR_ERR_WORKSPACE, MOR_ERR_CUDA,
 MOR_ERR_TIMEOUT, MOR_ERR_STATIC_SCRATCH) = range(1, 8)
MOR_STATIC_SCRATCH_BYTES = 2 * 1024 * 1024
MOR_FMT_E4M3, MOR_FMT_E5M2, MOR_FMT_BF16 = 0, 1, 2
MOR_SCALE_GAM, MOR_SCALE_E8M0, MOR_SCALE_FP32_AMAX = 0, 1, 2
MOR_CRIT_TENSOR_MEAN_REL, MOR_CRIT_BLOCK_VS_E5M2, MOR_CRIT_BLOCK_MEAN_REL = 0, 1, 2
MOR_FLAG_STRICT_TIES, MOR_FLAG_RANGE_MIN_INCLUDES_ZERO = 1, 2
MOR_ERROR_BINS = 12


class MorError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {mor_status_string(status)} (status {status})")


class mor_tensor_desc_t(C.Structure):
    _fields_ = [("x", C.c_void_p), ("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64),
                ("block_rows", C.c_int32), ("block_cols", C.c_int32),
                ("n_formats", C.c_int32), ("formats", C.c_int32 * 3),
                ("criterion", C.c_int32), ("threshold", C.c_float),
                ("scale_mode", C.c_int32), ("flags", C.c_uint32), ("group_amax", C.c_void_p)]


class mor_block_stats_t(C.Structure):
    _fields_ = [("amax", C.c_float), ("min_abs_nz", C.c_float), ("nnz", C.c_uint32),
                ("n_nonfinite", C.c_uint32), ("sum_rel_e4m3", C.c_float), ("sum_rel_e5m2", C.c_float)]


class mor_tensor_stats_t(C.Structure):
    _fields_ = [("sum_rel_e4m3", C.c_double), ("nnz", C.c_uint64), ("mean_rel_e4m3", C.c_double),
                ("group_amax", C.c_float), ("group_mantissa", C.c_uint32),
                ("tensor_format", C.c_uint32), ("status", C.c_uint32),
                ("n_blocks", C.c_uint64), ("n_e4m3", C.c_uint64), ("n_e5m2", C.c_uint64),
                ("n_bf16", C.c_uint64), ("n_nonfinite", C.c_uint64)]


class mor_outputs_t(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("codes_ld", C.c_int64), ("scale_e8m0", C.c_void_p),
                ("sel", C.c_void_p), ("scale_f32", C.c_void_p), ("bf16_fallback", C.c_void_p),
                ("block_stats", C.c_void_p), ("tensor_stats", C.c_void_p), ("fake_quant", C.c_void_p),
                ("error_histogram", C.c_void_p)]


class mor_stage_events_t(C.Structure):
    _fields_ = [("amax_begin", C.c_void_p), ("main_begin", C.c_void_p), ("main_end", C.c_void_p),
                ("finalise_end", C.c_void_p)]


BLOCK_STATS_DTYPE = np.dtype([("amax", "f4"), ("min_abs_nz", "f4"), ("nnz", "u4"), ("n_nonfinite", "u4"),
                              ("sum_rel_e4m3", "f4"), ("sum_rel_e5m2", "f4")])
TENSOR_STATS_DTYPE = np.dtype([("sum_rel_e4m3", "f8"), ("nnz", "u8"), ("mean_rel_e4m3", "f8"),
                               ("group_amax", "f4"), ("group_mantissa", "u4"), ("tensor_format", "u4"),
                               ("status", "u4"), ("n_blocks", "u8"), ("n_e4m3", "u8"), ("n_e5m2", "u8"),
                               ("n_bf16", "u8"), ("n_nonfinite", "u8")])
assert BLOCK_STATS_DTYPE.itemsize == C.sizeof(mor_block_stats_t) == 24
assert TENSOR_STATS_DTYPE.itemsize == C.sizeof(mor_tensor_stats_t) == 80

_lib = None


def load():
    """Load the CUDA library; raises if it has not been built (there is no other path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_22804_b200.build` "
                               "(the analyse-and-quantise pass has no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        pd, po = C.POINTER(mor_tensor_desc_t), C.POINTER(mor_outputs_t)
        L.mor_workspace_bytes.restype = C.c_size_t
        L.mor_workspace_bytes.argtypes = [pd, C.c_int]
        L.mor_analyze_quantize.restype = C.c_int
        L.mor_analyze_quantize.argtypes = [pd, po, C.c_void_p, C.c_size_t, C.c_void_p]
        L.mor_analyze_quantize_batched.restype = C.c_int
        L.mor_analyze_quantize_batched.argtypes = [pd, po, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]
        L.mor_analyze_quantize_batched_ex.restype = C.c_int
        L.mor_analyze_quantize_batched_ex.argtypes = [pd, po, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p,
                                                      C.POINTER(mor_stage_events_t)]
        L.mor_select_stats_batched.restype = C.c_int
        L.mor_select_stats_batched.argtypes = [pd, po, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]
        L.mor_select_stats.restype = C.c_int
        L.mor_select_stats.argtypes = [pd, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.mor_group_amax.restype = C.c_int
        L.mor_group_amax.argtypes = [pd, C.c_int, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.mor_host_staging_bytes.restype = C.c_size_t
        L.mor_host_staging_bytes.argtypes = [pd]
        L.mor_analyze_quantize_host.restype = C.c_int
        L.mor_analyze_quantize_host.argtypes = [pd, po, C.c_void_p, C.c_size_t, C.c_void_p]
        L.mor_analyze_quantize_static.restype = C.c_int
        L.mor_analyze_quantize_static.argtypes = [pd, po, C.c_void_p]
        L.mor_status_string.restype = C.c_char_p
        L.mor_status_string.argtypes = [C.c_int]
        L.mor_version.restype = C.c_int
        L.mor_version.argtypes = []
        _lib = L
    return _lib


EXPORTS = ["mor_workspace_bytes", "mor_analyze_quantize", "mor_analyze_quantize_batched",
           "mor_analyze_quantize_batched_ex", "mor_select_stats", "mor_select_stats_batched",
           "mor_group_amax", "mor_host_staging_bytes", "mor_analyze_quantize_host",
           "mor_analyze_quantize_static", "mor_status_string", "mor_version"]


# ------------------------------------------------------------------ C entry points ----

def mor_status_string(status: int) -> str:
    return load().mor_status_string(int(status)).decode()


def mor_version() -> int:
    return load().mor_version()


def _desc_array(descs: Sequence[mor_tensor_desc_t]):
    if isinstance(descs, C.Array):
        return descs, len(descs)
    arr = (mor_tensor_desc_t * len(descs))(*descs)
    return arr, len(descs)


def mor_workspace_bytes(descs) -> int:
    arr, n = _desc_array(descs)
    return int(load().mor_workspace_bytes(arr, n))


def mor_analyze_quantize(desc: mor_tensor_desc_t, out: mor_outputs_t, workspace_ptr: int, workspace_bytes: int,
                         stream_ptr: int = 0) -> int:
    return load().mor_analyze_quantize(C.byref(desc), C.byref(out), workspace_ptr, workspace_bytes, stream_ptr)


def mor_analyze_quantize_batched(descs, outs, workspace_ptr: int, workspace_bytes: int, stream_ptr: int = 0) -> int:
    darr, n = _desc_array(descs)
    oarr = outs if isinstance(outs, C.Array) else (mor_outputs_t * len(outs))(*outs)
    return load().mor_analyze_quantize_batched(darr, oarr, n, workspace_ptr, workspace_bytes, stream_ptr)


def mor_analyze_quantize_batched_ex(descs, outs, workspace_ptr: int, workspace_bytes: int, stream_ptr: int = 0,
                                    events: Optional[mor_stage_events_t] = None) -> int:
    darr, n = _desc_array(descs)
    oarr = outs if isinstance(outs, C.Array) else (mor_outputs_t * len(outs))(*outs)
    return load().mor_analyze_quantize_batched_ex(darr, oarr, n, workspace_ptr, workspace_bytes, stream_ptr,
                                                  None if events is None else C.byref(events))


def mor_select_stats(desc: mor_tensor_desc_t, block_stats_ptr: int, tensor_stats_ptr: int, sel_ptr: int,
                     scale_ptr: int, workspace_ptr: int, workspace_bytes: int, stream_ptr: int = 0) -> int:
    return load().mor_select_stats(C.byref(desc), block_stats_ptr, tensor_stats_ptr, sel_ptr, scale_ptr,
                                   workspace_ptr, workspace_bytes, stream_ptr)


def mor_select_stats_batched(descs, outs, workspace_ptr: int, workspace_bytes: int, stream_ptr: int = 0) -> int:
    darr, n = _desc_array(descs)
    oarr = outs if isinstance(outs, C.Array) else (mor_outputs_t * len(outs))(*outs)
    return load().mor_select_stats_batched(darr, oarr, n, workspace_ptr, workspace_bytes, stream_ptr)


def mor_group_amax(descs, amax_out_ptr: int, workspace_ptr: int, workspace_bytes: int, stream_ptr: int = 0) -> int:
    arr, n = _desc_array(descs)
    return load().mor_group_amax(arr, n, amax_out_ptr, workspace_ptr, workspace_bytes, stream_ptr)


def mor_host_staging_bytes(desc: mor_tensor_desc_t) -> int:
    return int(load().mor_host_staging_bytes(C.byref(desc)))


def mor_analyze_quantize_host(desc: mor_tensor_desc_t, out: mor_outputs_t, staging_ptr: int, staging_bytes: int,
                              stream_ptr: int = 0) -> int:
    return load().mor_analyze_quantize_host(C.byref(desc), C.byref(out), staging_ptr, staging_bytes, stream_ptr)


def mor_analyze_quantize_static(desc: mor_tensor_desc_t, out: mor_outputs_t, stream_ptr: int = 0) -> int:
    """mor_analyze_quantize with the library's built-in scratch array: no workspace to pass, no
    device allocation made; tensors that need more than MOR_STATIC_SCRATCH_BYTES are refused."""
    return load().mor_analyze_quantize_static(C.byref(desc), C.byref(out), stream_ptr)


# ------------------------------------------------------------------------- helpers ----

@dataclass
class Recipe:
    """Partition, ordered format list and acceptance metric (inputs of Algorithm 2)."""
    block: tuple = (128, 128)
    formats: Sequence[int] = (MOR_FMT_E4M3, MOR_FMT_BF16)
    criterion: int = MOR_CRIT_BLOCK_VS_E5M2
    threshold: float = 0.045
    scale_mode: int = MOR_SCALE_GAM
    flags: int = 0


def grid_of(rows: int, cols: int, block) -> tuple:
    if rows == 0 or cols == 0:
        return (0, 0)
    if tuple(block) == (0, 0):
        return (1, 1)
    if tuple(block) == (1, 0):          # per-channel: one block per row
        return (rows, 1)
    if tuple(block) == (0, 1):          # per-channel along the columns: one block per column
        return (1, cols)
    return (-(-rows // block[0]), -(-cols // block[1]))


def make_desc(x_ptr: int, rows: int, cols: int, ld: int, recipe: Recipe, group_amax_ptr: int = 0) -> mor_tensor_desc_t:
    d = mor_tensor_desc_t()
    d.x = x_ptr
    d.rows, d.cols, d.ld = rows, cols, ld
    d.block_rows, d.block_cols = recipe.block
    f = list(recipe.formats)
    d.n_formats = len(f)
    for i in range(3):
        d.formats[i] = f[i] if i < len(f) else 0
    d.criterion, d.threshold = recipe.criterion, recipe.threshold
    d.scale_mode, d.flags = recipe.scale_mode, recipe.flags
    d.group_amax = group_amax_ptr or None
    return d


def desc_for(x, recipe: Recipe, cols: Optional[int] = None, group_amax=None) -> mor_tensor_desc_t:
    """Descriptor of a 2-D torch BF16 CUDA tensor (row stride = leading dimension)."""
    import torch

    assert x.dtype == torch.bfloat16 and x.dim() == 2 and (x.shape[1] == 0 or x.stride(1) == 1)
    rows = x.shape[0]
    ld = x.stride(0) if (rows > 1 and x.shape[1] > 0) else (max(x.shape[1], 1) + 7) // 8 * 8
    return make_desc(x.data_ptr(), rows, x.shape[1] if cols is None else cols, ld, recipe,
                     0 if group_amax is None else group_amax.data_ptr())


@dataclass
class Outputs:
    codes: object = None          # uint8 [rows, codes_ld]
    scale_e8m0: object = None     # uint8 [grid]
    sel: object = None            # uint8 [grid]
    scale_f32: object = None      # float32 [grid]
    bf16_fallback: object = None  # bfloat16, shaped like x
    fake_quant: object = None     # bfloat16, shaped like x
    error_histogram: object = None  # the caller's 12 counters (Section 4.1.3), if given
    block_stats: object = None    # uint8 [n_blocks * 24]
    tensor_stats: object = None   # uint8 [80]
    cols: int = 0
    rows: int = 0
    transposed: bool = False      # (128, 1) sub-column blocks: codes are stored [cols, rows]
    c_struct: mor_outputs_t = field(default_factory=mor_outputs_t)

    def codes_view(self):
        """The codes as a [rows, cols] view, whatever the stored layout."""
        if self.transposed:
            return self.codes[:, :self.rows].t()
        return self.codes[:, :self.cols]

    def tensor_stats_dict(self) -> dict:
        """Copies the summary to the host (synchronises)."""
        rec = self.tensor_stats.cpu().numpy().view(TENSOR_STATS_DTYPE)[0]
        return {k: rec[k].item() for k in TENSOR_STATS_DTYPE.names}

    def block_stats_array(self) -> np.ndarray:
        return self.block_stats.cpu().numpy().view(BLOCK_STATS_DTYPE)


def alloc_outputs(rows: int, cols: int, recipe: Recipe, device, *, codes=True, block_stats=False, fallback_like=None,
                  scale_f32=False, fake_quant_like=None, error_histogram=None) -> Outputs:
    import torch

    g = grid_of(rows, cols, recipe.block)
    nb = g[0] * g[1]
    transposed = tuple(recipe.block) in ((128, 1), (0, 1))     # column blocks: codes are stored [cols, rows]
    o = Outputs(cols=cols, rows=rows, transposed=transposed)
    ld = ((rows if transposed else cols) + 15) // 16 * 16
    u8 = dict(dtype=torch.uint8, device=device)
    if codes:
        o.codes = torch.empty((cols if transposed else rows, ld), **u8)
    o.scale_e8m0 = torch.empty(g, **u8)
    o.sel = torch.empty(g, **u8)
    if scale_f32 or recipe.scale_mode == MOR_SCALE_FP32_AMAX:
        o.scale_f32 = torch.empty(g, dtype=torch.float32, device=device)
    if fallback_like is not None:
        o.bf16_fallback = torch.zeros_like(fallback_like)
    if fake_quant_like is not None:
        o.fake_quant = torch.zeros_like(fake_quant_like)
    if block_stats:
        o.block_stats = torch.empty((max(nb, 1) * BLOCK_STATS_DTYPE.itemsize,), **u8)
    o.tensor_stats = torch.empty((TENSOR_STATS_DTYPE.itemsize,), **u8)
    s = o.c_struct
    s.codes = o.codes.data_ptr() if o.codes is not None and o.codes.numel() else None
    s.codes_ld = ld
    s.scale_e8m0 = o.scale_e8m0.data_ptr() if nb else None
    s.sel = o.sel.data_ptr() if nb else None
    s.scale_f32 = o.scale_f32.data_ptr() if o.scale_f32 is not None and nb else None
    s.bf16_fallback = o.bf16_fallback.data_ptr() if o.bf16_fallback is not None else None
    s.fake_quant = o.fake_quant.data_ptr() if o.fake_quant is not None else None
    if error_histogram is not None:      # the caller's counters (int32 or uint32, MOR_ERROR_BINS of them), kept across calls
        assert error_histogram.numel() == MOR_ERROR_BINS and error_histogram.element_size() == 4 and error_histogram.is_cuda
        o.error_histogram = error_histogram
        s.error_histogram = error_histogram.data_ptr()
    s.block_stats = o.block_stats.data_ptr() if o.block_stats is not None else None
    s.tensor_stats = o.tensor_stats.data_ptr()
    return o


def _stream_ptr(stream) -> int:
    import torch

    return (stream or torch.cuda.current_stream()).cuda_stream


def _workspace(nbytes: int, device):
    import torch

    return torch.empty((max(nbytes, 256),), dtype=torch.uint8, device=device)


def analyze_quantize(x, recipe: Recipe, *, cols=None, group_amax=None, block_stats=False, fallback=False,
                     scale_f32=False, fake_quant=False, error_histogram=None, stream=None) -> Outputs:
    """Run mor_analyze_quantize on one BF16 CUDA tensor; allocates outputs and workspace."""
    d = desc_for(x, recipe, cols, group_amax)
    o = alloc_outputs(d.rows, d.cols, recipe, x.device, block_stats=block_stats,
                      fallback_like=x if fallback else None, scale_f32=scale_f32, fake_quant_like=x if fake_quant else None,
                      error_histogram=error_histogram)
    nbytes = mor_workspace_bytes([d])
    ws = _workspace(nbytes, x.device)
    st = mor_analyze_quantize(d, o.c_struct, ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    if st != MOR_OK:
        raise MorError(st, "mor_analyze_quantize")
    o._keep = (ws, x, group_amax)
    return o


def select_stats(x, recipe: Recipe, *, cols=None, group_amax=None, block_stats=True, stream=None) -> Outputs:
    """Run mor_select_stats: decisions and statistics, no codes."""
    d = desc_for(x, recipe, cols, group_amax)
    o = alloc_outputs(d.rows, d.cols, recipe, x.device, codes=False, block_stats=block_stats)
    ws = _workspace(mor_workspace_bytes([d]), x.device)
    st = mor_select_stats(d, o.c_struct.block_stats or 0, o.c_struct.tensor_stats, o.c_struct.sel or 0,
                          o.c_struct.scale_e8m0 or 0, ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    if st != MOR_OK:
        raise MorError(st, "mor_select_stats")
    o._keep = (ws, x, group_amax)
    return o


def group_amax(xs: Sequence, stream=None):
    """max|x| of each tensor (Algorithm 1's g_amax with the tensor as the group) as a CUDA float tensor."""
    import torch

    r = Recipe()
    descs = [desc_for(x, r) for x in xs]
    out = torch.empty((len(xs),), dtype=torch.float32, device=xs[0].device)
    ws = _workspace(mor_workspace_bytes(descs), xs[0].device)
    st = mor_group_amax(descs, out.data_ptr(), ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    if st != MOR_OK:
        raise MorError(st, "mor_group_amax")
    return out


class BatchPlan:
    """Descriptors, outputs and workspace of a fixed list of tensors, built once so that a
    step is a single call of mor_analyze_quantize_batched."""

    def __init__(self, xs: Sequence, recipes: Sequence[Recipe], *, group_amax=None, block_stats=False,
                 fallback=False, fake_quant=False, error_histograms=None, stats_only=False):
        """`fallback` and `fake_quant` are one flag for all tensors or one flag per tensor; `error_histograms`
        is one tensor of MOR_ERROR_BINS 32-bit counters per tensor (or None)."""
        assert len(xs) == len(recipes) and len(xs) > 0
        self.xs = list(xs)
        self.group_amax = group_amax
        per = lambda f: list(f) if isinstance(f, (list, tuple)) else [bool(f)] * len(xs)
        fallback, fake_quant = per(fallback), per(fake_quant)
        assert len(fallback) == len(xs) == len(fake_quant)
        descs, self.outs = [], []
        for i, (x, r) in enumerate(zip(xs, recipes)):
            ga = None if group_amax is None else group_amax[i:i + 1]
            d = desc_for(x, r, None, ga)
            descs.append(d)
            self.outs.append(alloc_outputs(d.rows, d.cols, r, x.device, block_stats=block_stats, codes=not stats_only,
                                           fallback_like=x if fallback[i] else None,
                                           fake_quant_like=x if fake_quant[i] else None,
                                           error_histogram=None if error_histograms is None else error_histograms[i]))
        self.descs = (mor_tensor_desc_t * len(descs))(*descs)
        self.couts = (mor_outputs_t * len(descs))(*[o.c_struct for o in self.outs])
        self.n = len(descs)
        self.ws = _workspace(mor_workspace_bytes(self.descs), xs[0].device)
        self._fn = load().mor_analyze_quantize_batched_ex
        self.stats_only = stats_only          # decisions and statistics only (mor_select_stats_batched): no codes

    def run(self, stream=None, events: Optional[mor_stage_events_t] = None) -> None:
        if self.stats_only:
            st = load().mor_select_stats_batched(self.descs, self.couts, self.n, self.ws.data_ptr(), self.ws.numel(), _stream_ptr(stream))
            if st != MOR_OK:
                raise MorError(st, "mor_select_stats_batched")
            return
        st = self._fn(self.descs, self.couts, self.n, self.ws.data_ptr(), self.ws.numel(), _stream_ptr(stream),
                      None if events is None else C.byref(events))
        if st != MOR_OK:
            raise MorError(st, "mor_analyze_quantize_batched")

    def capture(self):
        """The step as a CUDA graph (memset, amax pre-pass, main kernel, finalise as graph nodes), for
        launch-bound cases such as a single small tensor.  One ordinary step runs first, so that the library's
        per-device set-up happens outside the capture.  Replay with ``graph.replay()``; the tensors, outputs
        and workspace of this plan are baked in."""
        import torch

        self.run()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.run(torch.cuda.current_stream())
        return graph
