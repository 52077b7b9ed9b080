"""Times the main kernel and the whole call on the benchmark configurations, one line per recipe.

    python -m paper_2512_22804_b200.measure [substring ...]

Each configuration gets enough distinct copies of its tensor to exceed the L2 (64 / 16 / 8 / 3), a
``BatchPlan``, 3 warm-up and 10 timed calls of ``mor_analyze_quantize_batched_ex``; the stage events of
that call give the main kernel's time and the whole call's (pre-pass, main kernel, finalise).  GB/s are
algorithmic bytes over the median time: 3 + 2/block bytes per element for the main kernel, 2 more for the
whole call where the amax pre-pass runs.  Arguments select the lines whose name contains one of them.
"""
from __future__ import annotations

import sys

import numpy as np


def main(argv) -> int:
    import torch

    from . import binding as mb
    from . import build
    from . import workloads as wl

    build.build()
    wanted = [a for a in argv if not a.startswith("-")]
    two, three = (mb.MOR_FMT_E4M3, mb.MOR_FMT_BF16), (mb.MOR_FMT_E4M3, mb.MOR_FMT_E5M2, mb.MOR_FMT_BF16)
    eq2, eq3 = mb.MOR_CRIT_TENSOR_MEAN_REL, mb.MOR_CRIT_BLOCK_VS_E5M2

    def device(bits, copies):
        return [torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda().clone() for _ in range(copies)]

    def line(name, bits, recipe, copies):
        if wanted and not any(w in name for w in wanted):
            return
        xs = device(bits, copies)
        plan = mb.BatchPlan(xs, [recipe] * copies)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        for e in ev:
            e.record()
        torch.cuda.synchronize()
        stages = mb.mor_stage_events_t()
        stages.amax_begin, stages.main_begin, stages.main_end, stages.finalise_end = [e.cuda_event for e in ev]
        for _ in range(3):
            plan.run()
        torch.cuda.synchronize()
        t_main, t_call = [], []
        for _ in range(10):
            plan.run(None, stages)
            torch.cuda.synchronize()
            t_main.append(ev[1].elapsed_time(ev[2]))
            t_call.append(ev[0].elapsed_time(ev[3]))
        elements = bits.size * copies
        block = tuple(recipe.block)
        per_block = elements if block == (0, 0) else bits.shape[1] if block == (1, 0) else block[0] * block[1]
        main_bytes = elements * (3.0 + 2.0 / per_block)
        single_read = recipe.scale_mode != mb.MOR_SCALE_GAM and block not in ((0, 0), (1, 0))
        call_bytes = main_bytes + (0.0 if single_read else 2.0 * elements)
        tm, tc = float(np.median(t_main)), float(np.median(t_call))
        st = plan.outs[0].tensor_stats_dict()
        print(f"{name:44s} main {tm * 1e3:7.1f} us {main_bytes / tm / 1e6:6.0f} GB/s | call {tc * 1e3:7.1f} us "
              f"{call_bytes / tc / 1e6:6.0f} GB/s | blocks E4M3 {st['n_e4m3']} E5M2 {st['n_e5m2']} BF16 {st['n_bf16']}, "
              f"Eq.1 error {st['mean_rel_e4m3']:.4f}", flush=True)

    c0, c1, c2, c3 = wl.gaussian_outlier_rows(), wl.weight_like(), wl.activation_like(), wl.gradient_like()
    line("configs[0] x64 per tensor Eq.2", c0, mb.Recipe((0, 0), two, eq2), 64)
    line("configs[0] x1 per tensor Eq.2", c0, mb.Recipe((0, 0), two, eq2), 1)
    line("configs[1] x16 128x128 two-way Eq.3", c1, mb.Recipe((128, 128), two, eq3), 16)
    line("configs[1] x16 128x128 tensor-level Eq.2", c1, mb.Recipe((128, 128), two, eq2), 16)
    line("configs[1] x16 64x64 two-way Eq.3", c1, mb.Recipe((64, 64), two, eq3), 16)
    line("configs[1] x16 128x1 two-way Eq.3", c1, mb.Recipe((128, 1), two, eq3), 16)
    line("configs[1] x16 per channel Eq.2", c1, mb.Recipe((1, 0), two, eq2), 16)
    line("configs[1] x16 128x128 two-way Eq.3 E8M0", c1, mb.Recipe((128, 128), two, eq3, scale_mode=mb.MOR_SCALE_E8M0), 16)
    line("configs[1] x16 128x128 two-way Eq.3 FP32 amax", c1, mb.Recipe((128, 128), two, eq3, scale_mode=mb.MOR_SCALE_FP32_AMAX), 16)
    line("configs[2] x8 1x128 two-way Eq.3", c2, mb.Recipe((1, 128), two, eq3), 8)
    line("configs[2] x8 1x128 two-way Eq.3 E8M0", c2, mb.Recipe((1, 128), two, eq3, scale_mode=mb.MOR_SCALE_E8M0), 8)
    line("configs[2] x8 1x128 two-way Eq.3 FP32 amax", c2, mb.Recipe((1, 128), two, eq3, scale_mode=mb.MOR_SCALE_FP32_AMAX), 8)
    line("configs[3] x3 1x128 three-way", c3, mb.Recipe((1, 128), three, eq3), 3)
    line("configs[3] x3 128x128 three-way", c3, mb.Recipe((128, 128), three, eq3), 3)

    # rows and columns of the same tensors: one call with a pair of entries per tensor against the two calls it replaces
    for name, bits, copies in (("configs[1] x8", c1, 8), ("configs[2] x4", c2, 4)):
        if wanted and not any(w in name + " rows and columns" for w in wanted):
            continue
        xs = device(bits, copies)
        rows, cols = mb.Recipe((1, 128), two, eq3), mb.Recipe((128, 1), two, eq3)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for label, tensors, recipes in (("rows and columns, one call", [x for x in xs for _ in (0, 1)], [rows, cols] * copies),
                                        ("rows only", xs, [rows] * copies), ("columns only", xs, [cols] * copies)):
            plan = mb.BatchPlan(tensors, recipes)
            for _ in range(3):
                plan.run()
            torch.cuda.synchronize()
            ts = []
            for _ in range(10):
                e0.record()
                plan.run()
                e1.record()
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1))
            print(f"{name} {label:28s} call {float(np.median(ts)) * 1e3:7.1f} us", flush=True)
    return 0


if __name__ == "__main__":
    raise SystemExit(main(sys.argv[1:]))
