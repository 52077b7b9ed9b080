"""Row-sharded use on two CPU ranks (gloo): the exchange logic of ``sharded`` with the data steps
done by the CPU oracle.  The sharded result must equal the oracle's run over the whole tensor:
codes, scale bytes and selection bytes of the shards laid end to end, and the tensor summary."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, crit, block, out_dir):
    if ROOT not in sys.path:
        sys.path.insert(0, ROOT)
    from oracle import mor_oracle as orc
    from paper_2512_22804_b200 import binding as mb
    from paper_2512_22804_b200 import sharded
    from paper_2512_22804_b200 import workloads as wl

    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        full = wl.activation_like(512, 384, seed=81)
        full[300:, :] = wl.gradient_like(212, 384, seed=82)          # the two halves differ a lot: local amax != global amax
        rows = full.shape[0] // world
        mine = full[rank * rows:(rank + 1) * rows]
        recipe = mb.Recipe(block, (mb.MOR_FMT_E4M3, mb.MOR_FMT_BF16), crit, 0.045)

        class Out:
            pass

        def amax_fn(bits):
            return orc.tensor_amax(bits)

        def analyze_fn(bits, r, g_amax):
            res = orc.run(bits, r.block, list(r.formats), r.criterion, r.threshold, group_amax=g_amax)
            o = Out()
            o.codes, o.scale = res.codes, res.scale_e8m0
            o.sel = torch.from_numpy(res.sel.copy())
            return res.tensor, o

        got = sharded.analyze_quantize_row_sharded(mine, recipe, amax_fn=amax_fn, analyze_fn=analyze_fn)
        np.savez(os.path.join(out_dir, f"r{rank}.npz"), codes=got.outputs.codes, scale=got.outputs.scale,
                 sel=got.outputs.sel.numpy(), amax=got.group_amax,
                 summary=np.array([got.tensor[k] for k in ("sum_rel_e4m3", "nnz", "n_blocks", "n_e4m3", "n_e5m2", "n_bf16",
                                                             "n_nonfinite", "mean_rel_e4m3", "tensor_format")], dtype=np.float64))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("crit,block", [(1, (128, 128)), (1, (1, 128)), (0, (128, 128))])
def test_two_ranks_equal_the_unsharded_run(tmp_path, crit, block):
    from oracle import mor_oracle as orc
    from paper_2512_22804_b200 import workloads as wl

    world = 2
    mp.spawn(_worker, args=(world, _free_port(), crit, block, str(tmp_path)), nprocs=world, join=True)
    full = wl.activation_like(512, 384, seed=81)
    full[300:, :] = wl.gradient_like(212, 384, seed=82)
    ref = orc.run(full, block, [0, 2], crit, 0.045)
    parts = [np.load(tmp_path / f"r{r}.npz") for r in range(world)]
    assert all(float(p["amax"]) == ref.tensor["group_amax"] for p in parts)
    np.testing.assert_array_equal(np.concatenate([p["codes"] for p in parts]), ref.codes)
    np.testing.assert_array_equal(np.concatenate([p["scale"] for p in parts]), ref.scale_e8m0)
    np.testing.assert_array_equal(np.concatenate([p["sel"] for p in parts]), ref.sel)
    want = [ref.tensor[k] for k in ("sum_rel_e4m3", "nnz", "n_blocks", "n_e4m3", "n_e5m2", "n_bf16", "n_nonfinite",
                                    "mean_rel_e4m3", "tensor_format")]
    for p in parts:
        np.testing.assert_allclose(p["summary"], want, rtol=1e-12)
    np.testing.assert_array_equal(parts[0]["summary"], parts[1]["summary"])   # every rank holds the same summary


def test_partition_that_cannot_be_sharded_is_refused():
    from paper_2512_22804_b200 import binding as mb
    from paper_2512_22804_b200 import sharded

    with pytest.raises(ValueError):
        sharded.analyze_quantize_row_sharded(np.zeros((128, 128), np.uint16), mb.Recipe((0, 0)), amax_fn=lambda b: 0.0,
                                             analyze_fn=lambda b, r, g: ({}, None))
    with pytest.raises(ValueError):
        sharded.analyze_quantize_row_sharded(np.zeros((100, 128), np.uint16), mb.Recipe((128, 128)), amax_fn=lambda b: 0.0,
                                             analyze_fn=lambda b, r, g: ({}, None))
