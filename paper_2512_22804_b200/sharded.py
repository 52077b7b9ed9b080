"""A tensor whose rows are spread over several ranks (one process per GPU).

Blocks are independent once the shared mantissa of Algorithm 1 is known, so a row-sharded tensor
needs two tiny exchanges and no data movement:

1. ``all_reduce(MAX)`` of one float: the group amax of Algorithm 1 is the maximum over the
   whole tensor, not over the local rows;
2. ``all_reduce(SUM)`` of seven numbers: the Eq. 1-2 numerator, the non-zero count and the block
   counts, from which every rank forms the same tensor-level decision.

Each rank then holds the codes, scale bytes and selection bytes of its own rows.  Shards must
hold whole blocks (a multiple of 128 rows for 128x128 blocks); the single-block partition (0, 0)
cannot be sharded this way because its one scale needs the global amax as the block amax.

In plain data-parallel training every rank quantises its own tensors and none of this is
needed: ranks are replicas and exchange nothing.

The two steps that touch the data are injectable (``amax_fn``, ``analyze_fn``) so that the
exchange logic can be exercised on CPU ranks; by default they are the CUDA entry points.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, Optional

import torch
import torch.distributed as dist

from . import binding as mb

_SUM_FIELDS = ("sum_rel_e4m3", "nnz", "n_blocks", "n_e4m3", "n_e5m2", "n_bf16", "n_nonfinite")


@dataclass
class ShardedResult:
    outputs: object          # what analyze_fn returned for the local rows
    tensor: dict             # tensor-wide summary, identical on every rank
    group_amax: float


def _cuda_amax(x) -> float:
    return float(mb.group_amax([x]).item())


def _cuda_analyze(x, recipe: mb.Recipe, group_amax: float):
    ga = torch.tensor([group_amax], dtype=torch.float32, device=x.device)
    out = mb.analyze_quantize(x, recipe, group_amax=ga)
    return out.tensor_stats_dict(), out


def combine_summaries(local: dict, threshold: float, group: Optional[dist.ProcessGroup] = None,
                      device: Optional[torch.device] = None) -> dict:
    """Sum the additive fields over the ranks and redo Eq. 2 on the totals."""
    t = torch.tensor([float(local[k]) for k in _SUM_FIELDS], dtype=torch.float64, device=device)
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    tot = dict(local)
    for k, v in zip(_SUM_FIELDS, t.tolist()):
        tot[k] = v if k == "sum_rel_e4m3" else int(round(v))
    tot["mean_rel_e4m3"] = tot["sum_rel_e4m3"] / tot["nnz"] if tot["nnz"] else 0.0
    th = float(torch.tensor(threshold, dtype=torch.float32))          # the boundary carries the threshold as binary32
    ok = tot["n_nonfinite"] == 0 and tot["mean_rel_e4m3"] < th
    tot["tensor_format"] = mb.MOR_FMT_E4M3 if ok else mb.MOR_FMT_BF16
    return tot


def analyze_quantize_row_sharded(x_local, recipe: mb.Recipe, *, group: Optional[dist.ProcessGroup] = None,
                                 amax_fn: Callable = _cuda_amax, analyze_fn: Callable = _cuda_analyze,
                                 device: Optional[torch.device] = None) -> ShardedResult:
    """Analyse and quantise this rank's rows of a row-sharded tensor (see the module text)."""
    if tuple(recipe.block) == (0, 0):
        raise ValueError("the per-tensor partition cannot be row-sharded: its one block spans all ranks")
    rows = x_local.shape[0]
    if rows % max(recipe.block[0], 1) != 0:
        raise ValueError("a shard must hold whole blocks")
    a = torch.tensor([amax_fn(x_local)], dtype=torch.float32, device=device)
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(a, op=dist.ReduceOp.MAX, group=group)
    g_amax = float(a.item())
    local, out = analyze_fn(x_local, recipe, g_amax)
    tot = combine_summaries(local, recipe.threshold, group, device)
    tot["group_amax"] = g_amax
    if recipe.criterion == mb.MOR_CRIT_TENSOR_MEAN_REL:
        # one decision for the whole tensor: every local block takes it
        fmt = tot["tensor_format"]
        tot["n_e4m3"] = tot["n_blocks"] if fmt == mb.MOR_FMT_E4M3 else 0
        tot["n_e5m2"] = 0
        tot["n_bf16"] = tot["n_blocks"] if fmt == mb.MOR_FMT_BF16 else 0
        sel = getattr(out, "sel", None)
        if sel is not None:
            sel.fill_(fmt)
    return ShardedResult(out, tot, g_amax)
