"""Element-by-element comparison of the CUDA path with the CPU oracle (test helper).

The bar (written here so that every parity test applies the same one):
  * FP8 codes, E8M0 scale bytes, selection bytes, group mantissa, group amax, counts of
    non-zeros and non-finites, block amax and block minimum: bit-exact;
  * relative-error sums and means: within REL_TOL = 1e-5 relative (the kernel sums binary32
    terms formed with an approximate reciprocal, the oracle sums exact ratios in double);
  * a block whose deciding quantities lie within 1e-5 relative of each other (Eq. 3), or of
    the threshold (Eq. 2), may legitimately decide either way: it is exempt from the
    comparison of selection, scale byte and codes, and counted.  Exact ties are not exempt.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from oracle import mor_oracle as orc
from paper_2512_22804_b200 import binding as mb

REL_TOL = 1e-5


def to_device(bits: np.ndarray):
    import torch

    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


@dataclass
class Report:
    n_blocks: int
    n_exempt: int
    tensor_exempt: bool


def recipe_from_case(case) -> mb.Recipe:
    return mb.Recipe(block=tuple(case.block), formats=tuple(case.formats), criterion=case.criterion,
                     threshold=case.threshold)


def oracle_block(block, cols, rows=None):
    """The block shape as the oracle takes it: per-channel rows (1, 0) are blocks of one whole row, per-channel
    columns (0, 1) blocks of one whole column (``rows`` needed)."""
    if tuple(block) == (1, 0):
        return (1, cols)
    if tuple(block) == (0, 1):
        return (rows, 1)
    return tuple(block)


def close(a, b, tol=REL_TOL):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return np.abs(a - b) <= tol * np.maximum(np.abs(b), 1e-300)


def exempt_blocks(ref: "orc.Result", recipe: mb.Recipe) -> np.ndarray:
    """Blocks of the oracle run whose decision is within the stated band (exact ties excluded)."""
    b = ref.blocks
    e4, e5 = b["sum_rel_e4m3"], b["sum_rel_e5m2"]
    ex = np.zeros(len(b), dtype=bool)
    if recipe.criterion == mb.MOR_CRIT_BLOCK_VS_E5M2:
        ex = (e4 != e5) & (np.abs(e4 - e5) <= REL_TOL * np.maximum(e4, e5))
    elif recipe.criterion == mb.MOR_CRIT_BLOCK_MEAN_REL:
        th = float(np.float32(recipe.threshold))
        mean = np.where(b["nnz"] > 0, e4 / np.maximum(b["nnz"], 1), 0.0)
        ex = np.abs(mean - th) <= REL_TOL * th
    return ex


def compare(bits: np.ndarray, recipe: mb.Recipe, out: "mb.Outputs", ref: "orc.Result", *, cols=None,
            ids=None, check_block_stats=True) -> Report:
    """Assert parity of one CUDA run with the oracle run ``ref``.

    ``ids``: the oracle analysed only these blocks (sampled parity at full size); the tensor
    summary is then not compared.
    """
    rows = bits.shape[0]
    cols = bits.shape[1] if cols is None else cols
    grid = ref.grid
    nb = grid[0] * grid[1]
    ts = out.tensor_stats_dict()
    sel = out.sel.cpu().numpy().reshape(-1)
    scale = out.scale_e8m0.cpu().numpy().reshape(-1)
    codes = None if out.codes is None else out.codes_view().cpu().numpy()
    idx = np.arange(nb) if ids is None else np.asarray(ids)
    th = float(np.float32(recipe.threshold))

    # ---- Algorithm 1 group quantities: exact
    assert ts["group_amax"] == ref.tensor["group_amax"]
    assert ts["group_mantissa"] == ref.tensor["group_mantissa"]
    assert ts["status"] == 0

    # ---- tensor aggregate (Eq. 1-2)
    tensor_exempt = False
    if ids is None:
        assert ts["n_blocks"] == nb == ref.tensor["n_blocks"]
        assert ts["nnz"] == ref.tensor["nnz"]
        assert ts["n_nonfinite"] == ref.tensor["n_nonfinite"]
        assert close(ts["sum_rel_e4m3"], ref.tensor["sum_rel_e4m3"]), (ts["sum_rel_e4m3"], ref.tensor["sum_rel_e4m3"])
        assert close(ts["mean_rel_e4m3"], ref.tensor["mean_rel_e4m3"])
        tensor_exempt = abs(ref.tensor["mean_rel_e4m3"] - th) <= REL_TOL * th
        if not tensor_exempt:
            assert ts["tensor_format"] == ref.tensor["tensor_format"]

    # ---- per-block outputs
    ex = exempt_blocks(ref, recipe)
    if recipe.criterion == mb.MOR_CRIT_TENSOR_MEAN_REL:
        ex[:] = tensor_exempt
    keep = ~ex
    if nb:
        np.testing.assert_array_equal(sel[idx][keep], ref.sel[idx][keep])
        np.testing.assert_array_equal(scale[idx][keep], ref.scale_e8m0[idx][keep])
        if out.scale_f32 is not None:
            sf = out.scale_f32.cpu().numpy().reshape(-1)
            np.testing.assert_array_equal(sf[idx][keep].view(np.uint32), ref.scale_f32[idx][keep].view(np.uint32))
    if ids is None and not ex.any():
        assert (ts["n_e4m3"], ts["n_e5m2"], ts["n_bf16"]) == (ref.tensor["n_e4m3"], ref.tensor["n_e5m2"], ref.tensor["n_bf16"])

    if codes is not None and nb:
        br, bc = oracle_block(recipe.block, cols, rows) if tuple(recipe.block) != (0, 0) else (rows, cols)
        if ids is None and not ex.any():
            np.testing.assert_array_equal(codes, ref.codes)
        else:
            for j, b in enumerate(idx):
                if ex[j]:
                    continue
                bi, bj = divmod(int(b), grid[1])
                sl = (slice(bi * br, min((bi + 1) * br, rows)), slice(bj * bc, min((bj + 1) * bc, cols)))
                np.testing.assert_array_equal(codes[sl], ref.codes[sl], err_msg=f"codes of block {b}")

    if check_block_stats and out.block_stats is not None and nb:
        bs = out.block_stats_array()[:nb][idx]
        rb = ref.blocks
        np.testing.assert_array_equal(bs["amax"].astype(np.float64), rb["amax"])
        np.testing.assert_array_equal(bs["nnz"].astype(np.int64), rb["nnz"])
        np.testing.assert_array_equal(bs["n_nonfinite"].astype(np.int64), rb["n_nonfinite"])
        assert close(bs["sum_rel_e4m3"], rb["sum_rel_e4m3"]).all()
        assert close(bs["sum_rel_e5m2"], rb["sum_rel_e5m2"]).all()
        if len(recipe.formats) == 3:
            np.testing.assert_array_equal(bs["min_abs_nz"].astype(np.float64), rb["min_abs_nz"])
    return Report(nb, int(ex.sum()), tensor_exempt)


GUARD = 256          # bytes of a known pattern on either side of every output buffer
PATTERN = 0xA5


def _guarded(t):
    """A tensor of the shape and dtype of ``t`` that lies between two guard zones; (view, whole buffer)."""
    import torch

    nbytes = t.numel() * t.element_size()
    buf = torch.full((GUARD + nbytes + GUARD,), PATTERN, dtype=torch.uint8, device=t.device)
    return buf[GUARD:GUARD + nbytes].view(t.dtype).view(t.shape), buf


def guarded_analyze_quantize(x, recipe: mb.Recipe, *, cols=None, group_amax=None, block_stats=True, fake_quant=False):
    """mor_analyze_quantize through the C boundary with every output buffer (codes, scale bytes, selection
    bytes, binary32 scales, block statistics, tensor summary) placed between guard zones and pre-filled with a
    pattern.  After the call the guard zones must still hold the pattern, and so must the padding columns of the
    codes beyond the 16-byte piece that holds a row's last code (that piece is written whole, with the code of
    zero in its unused bytes, as the header states): the library writes nowhere outside what the header says."""
    import torch

    d = mb.desc_for(x, recipe, cols, group_amax)
    o = mb.alloc_outputs(d.rows, d.cols, recipe, x.device, block_stats=block_stats, scale_f32=True,
                         fake_quant_like=x if fake_quant else None)
    if o.codes is not None and o.codes.numel():
        # two more 16-byte pieces per row than the call needs: they must stay untouched
        o.codes = torch.empty((o.codes.shape[0], o.codes.shape[1] + 32), dtype=torch.uint8, device=x.device)
        o.c_struct.codes_ld = o.codes.shape[1]
    bufs = {}
    for name in ("codes", "scale_e8m0", "sel", "scale_f32", "block_stats", "tensor_stats"):
        t = getattr(o, name)
        if t is None:
            continue
        v, buf = _guarded(t)
        v.view(torch.uint8).fill_(PATTERN) if v.numel() else None
        setattr(o, name, v)
        bufs[name] = (buf, t.numel() * t.element_size())
        if getattr(o.c_struct, name):                     # a NULL pointer (no blocks, no codes) stays NULL
            setattr(o.c_struct, name, v.data_ptr())
    ws = torch.empty((max(mb.mor_workspace_bytes([d]), 256),), dtype=torch.uint8, device=x.device)
    st = mb.mor_analyze_quantize(d, o.c_struct, ws.data_ptr(), ws.numel(), torch.cuda.current_stream().cuda_stream)
    if st != mb.MOR_OK:
        raise mb.MorError(st, "mor_analyze_quantize")
    torch.cuda.synchronize()
    o._keep = (ws, x, group_amax, bufs)
    for name, (buf, nbytes) in bufs.items():
        assert (buf[:GUARD] == PATTERN).all() and (buf[GUARD + nbytes:] == PATTERN).all(), f"write outside {name}"
    if o.codes is not None and o.codes.numel():
        used = d.rows if o.transposed else d.cols
        piece = (used + 15) // 16 * 16
        assert (o.codes[:, piece:] == PATTERN).all(), "padding columns of the codes were written"
        assert (o.codes[:, used:piece] == 0).all(), "unused bytes of a row's last 16-byte piece hold the code of zero"
    return o


def run_and_compare(bits: np.ndarray, recipe: mb.Recipe, *, cols=None, block_stats=True, scale_mode=None,
                    group_amax_supplied=False, pad_to=None, fake_quant=False) -> Report:
    """CUDA run + full oracle run on the same bytes, compared."""
    import torch

    if scale_mode is not None:
        recipe = mb.Recipe(recipe.block, recipe.formats, recipe.criterion, recipe.threshold, scale_mode, recipe.flags)
    host = bits
    if pad_to is not None:                       # rows padded with NaN patterns that must never be read
        host = np.full((bits.shape[0], pad_to), 0x7FC1, dtype=np.uint16)
        host[:, :bits.shape[1]] = bits
        cols = bits.shape[1]
    x = to_device(host)
    ga = None
    ref = orc.run(host, oracle_block(recipe.block, host.shape[1] if cols is None else cols, host.shape[0]), list(recipe.formats),
                  recipe.criterion, recipe.threshold, recipe.scale_mode, recipe.flags, cols=cols)
    if group_amax_supplied:
        ga = torch.tensor([ref.tensor["group_amax"]], dtype=torch.float32, device="cuda")
    out = guarded_analyze_quantize(x, recipe, cols=cols, group_amax=ga, block_stats=block_stats, fake_quant=fake_quant)
    rep = compare(host, recipe, out, ref, cols=cols)
    if block_stats and not fake_quant:
        # the same call without the optional outputs runs the plain instantiation of the kernel (no per-thread
        # counts, no keys in the compute threads): same bar
        plain = guarded_analyze_quantize(x, recipe, cols=cols, group_amax=ga, block_stats=False, fake_quant=False)
        compare(host, recipe, plain, ref, cols=cols)
    if fake_quant:
        # the fake-quantised tensor, bit for bit, outside blocks whose decision is within the tolerance band;
        # padding columns must stay untouched (zero-initialised output)
        c = host.shape[1] if cols is None else cols
        ob = oracle_block(recipe.block, c, host.shape[0])
        want = orc.fake_quant(host, ref, ob, list(recipe.formats), recipe.criterion, recipe.threshold, recipe.scale_mode,
                              recipe.flags, cols=cols)
        got = out.fake_quant.view(torch.int16).cpu().numpy().view(np.uint16)
        ex = exempt_blocks(ref, recipe)
        if not ex.any():
            np.testing.assert_array_equal(got[:, :c], want)
        else:
            br, bc = ob if tuple(recipe.block) != (0, 0) else host.shape
            for b in np.nonzero(~ex)[0]:
                bi, bj = divmod(int(b), ref.grid[1])
                sl = (slice(bi * br, min((bi + 1) * br, host.shape[0])), slice(bj * bc, min((bj + 1) * bc, c)))
                np.testing.assert_array_equal(got[sl], want[sl])
        assert (got[:, c:] == 0).all()
    return rep
