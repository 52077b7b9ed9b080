#!/usr/bin/env python
"""Throughput of the MoR analyse-and-quantise hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the whole hot path (tensor amax, fused main kernel, finalise) over a
batch of distinct synthetic 4096x4096 weight-like BF16 tensors, 128x128 blocks, two-way
selection [E4M3, BF16] against E5M2 (the benchmark's second configuration), issued as one
batched call.  The batch (512 MiB in, 256 MiB out by default) is larger than L2, so every
step reads its inputs from HBM.

Printed: ONE JSON line.  `value` is GB/s of algorithmic bytes (5 B/element: the amax read,
the main read, the code byte) over all ranks; `roofline` describes the main kernel alone,
timed with CUDA events recorded around it inside the same steps; `e2e` is the same metric
through the host-memory entry point with the copies inside the timed region;
`cpu_baseline` is the CPU oracle timed on this machine's host cores.

With N > 1 (torchrun) every rank runs its own batch: replicas, no collective on the data
path; time is the maximum over ranks.

`--impl reference` times the CPU oracle (the only other implementation of the method that
exists) on a bounded sample per step.
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

ROWS, COLS = 4096, 4096
BLOCK = (128, 128)
ALG_BYTES_MAIN = 2.0 + 1.0 + 2.0 / (BLOCK[0] * BLOCK[1])      # BF16 read + code write + scale and selection bytes
ALG_BYTES_STEP = ALG_BYTES_MAIN + 2.0                           # + the tensor-amax read
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one main-kernel launch: captured on 6 tensors
# (267.5 MB for 100.66 M elements; traffic grows in proportion to the elements) and scaled to the
# 16 tensors of the default batch.  The write part is an undercount: codes still in L2 when the
# kernel ends have not reached DRAM yet.  Must be set back to None when the kernel changes.
MAIN_KERNEL_DRAM_BYTES_PER_LAUNCH = 713.4e6


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clock and throttle-reason samples while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.t.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_step(bits, threads=1):
    from oracle import mor_oracle as orc

    return orc.run(bits, BLOCK, [orc.FMT_E4M3, orc.FMT_BF16], orc.CRIT_BLOCK_VS_E5M2, 0.045, n_threads=threads)


def run_reference(args, rank):
    """The CPU oracle as it stands, on a bounded sample of the workload per step."""
    if rank != 0:
        return
    from paper_2512_22804_b200 import workloads as wl

    sample_rows = 1024
    bits = wl.weight_like(ROWS, COLS, seed=1)[:sample_rows]
    for _ in range(args.warmup):
        oracle_step(bits)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(bits)
    dt = time.perf_counter() - t0
    el = sample_rows * COLS * args.steps
    gbs = el * ALG_BYTES_STEP / dt / 1e9
    line = {"impl": "reference", "metric": "analyse+quantise throughput (algorithmic bytes)", "value": gbs, "unit": "GB/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "configs[1]: 4096x4096 weight-like BF16, 128x128 blocks, [E4M3,BF16] vs E5M2",
                       "sample": f"first {sample_rows} rows of one tensor per step"},
            "elements_per_s": el / dt,
            "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle",
                             "sample": f"{sample_rows}x{COLS} elements per step, {args.steps} steps"},
            "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=16, help="tensors per step")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-variants", action="store_true")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist

    from paper_2512_22804_b200 import binding as mb
    from paper_2512_22804_b200 import build as mbuild
    from paper_2512_22804_b200 import workloads as wl

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        mbuild.build()
    if world > 1:
        dist.barrier()
    mb.load()

    # ---- inputs: `batch` distinct tensors per rank, resident in HBM
    B = args.batch
    host = [wl.weight_like(ROWS, COLS, seed=1 + 1000 * i + 100000 * rank) for i in range(B)]
    xs = [torch.from_numpy(h.view(np.int16)).view(torch.bfloat16).to(dev) for h in host]
    recipe = mb.Recipe(BLOCK, (mb.MOR_FMT_E4M3, mb.MOR_FMT_BF16), mb.MOR_CRIT_BLOCK_VS_E5M2, 0.045)
    plan = mb.BatchPlan(xs, [recipe] * B)
    stream = torch.cuda.current_stream()
    elements = ROWS * COLS * B

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        plan.run(stream)
    sync_all()

    # ---- timed region: K steps, CUDA events on the launching stream, stage events around the main kernel
    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(K)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stage = []
    for a, b in ev:
        a.record(stream); b.record(stream)       # torch creates the CUDA event on first record
        s = mb.mor_stage_events_t()
        s.main_begin, s.main_end = a.cuda_event, b.cuda_event
        assert s.main_begin and s.main_end
        stage.append(s)
    sync_all()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    sync_all()
    t_begin.record(stream)
    for k in range(K):
        plan.run(stream, stage[k])
    t_end.record(stream)
    sync_all()
    clocks = sampler.stop()
    ms_total = t_begin.elapsed_time(t_end)
    ms_main = sum(a.elapsed_time(b) for a, b in ev) / K
    if world > 1:
        t = torch.tensor([ms_total], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
    ms_step = ms_total / K
    value = elements * world * ALG_BYTES_STEP / (ms_step * 1e-3) / 1e9

    stats = [o.tensor_stats_dict() for o in plan.outs]
    n_blocks = sum(s["n_blocks"] for s in stats)
    fp8_frac = sum(s["n_e4m3"] + s["n_e5m2"] for s in stats) / max(n_blocks, 1)
    tensor_fp8 = sum(1 for s in stats if s["tensor_format"] == mb.MOR_FMT_E4M3) / len(stats)

    peak, peak_kind = measured_peak()
    achieved = elements * ALG_BYTES_MAIN / (ms_main * 1e-3) / 1e9
    roofline = {"kernel": "mor_main_kernel<BLK128, yardstick, two-way, store, keys from the pre-pass>", "bound": "hbm", "achieved": achieved,
                "peak": peak, "peak_source": f"{peak_kind} copy bandwidth", "unit": "GB/s", "frac": achieved / peak,
                "frac_of_8TBs": achieved / 8000.0, "ms_per_launch": ms_main,
                "algorithmic_bytes_per_launch": elements * ALG_BYTES_MAIN,
                "traffic": MAIN_KERNEL_DRAM_BYTES_PER_LAUNCH * (B / 16.0) if MAIN_KERNEL_DRAM_BYTES_PER_LAUNCH else None}

    # ---- the same resident tensors under the method's other recipes (main kernel only; context for the
    #      headline, which stays the two-way 128x128 recipe above)
    variants = []
    if rank == 0 and not args.no_variants:
        T = mb.MOR_CRIT_TENSOR_MEAN_REL
        for name, rec in (("128x128, tensor-level Eq.2 (E4M3 only)", mb.Recipe((128, 128), recipe.formats, T, 0.045)),
                          ("1x128, two-way Eq.3", mb.Recipe((1, 128), recipe.formats, mb.MOR_CRIT_BLOCK_VS_E5M2, 0.045)),
                          ("1x128, tensor-level Eq.2 (E4M3 only)", mb.Recipe((1, 128), recipe.formats, T, 0.045)),
                          ("per channel, tensor-level Eq.2 (E4M3 only)", mb.Recipe((1, 0), recipe.formats, T, 0.045)),
                          ("128x128, two-way Eq.3, group amax supplied by the caller (no pre-pass: the main kernel scans the blocks itself)", recipe),
                          ("1x128, two-way Eq.3, group amax supplied by the caller (no pre-pass)", mb.Recipe((1, 128), recipe.formats, mb.MOR_CRIT_BLOCK_VS_E5M2, 0.045))):
            supplied = None
            if "supplied" in name:
                supplied = torch.tensor([o.tensor_stats_dict()["group_amax"] for o in plan.outs], dtype=torch.float32, device=dev)
            vp = mb.BatchPlan(xs, [rec] * B, group_amax=supplied)
            ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ea.record(stream); eb.record(stream)
            sv = mb.mor_stage_events_t()
            sv.main_begin, sv.main_end = ea.cuda_event, eb.cuda_event
            for _ in range(3):
                vp.run(stream)
            tms = []
            for _ in range(5):
                vp.run(stream, sv)
                torch.cuda.synchronize()
                tms.append(ea.elapsed_time(eb))
            nbv = rec.block[0] * rec.block[1] if rec.block[1] else COLS
            gbs = elements * (3.0 + 2.0 / nbv) / (statistics.median(tms) * 1e-3) / 1e9
            variants.append({"recipe": name, "main_kernel_GBs": gbs, "frac_of_measured_copy": gbs / peak, "frac_of_8TBs": gbs / 8000.0})
            del vp

    # ---- mor_select_stats (decisions and statistics, no codes) on the same tensors: one call per tensor
    if rank == 0 and not args.no_variants:
        sd = [mb.desc_for(x, recipe) for x in xs]
        so = [mb.alloc_outputs(ROWS, COLS, recipe, dev, codes=False, block_stats=True) for _ in xs]
        sw = torch.empty((mb.mor_workspace_bytes([sd[0]]),), dtype=torch.uint8, device=dev)

        def stats_step():
            for d, o in zip(sd, so):
                st = mb.mor_select_stats(d, o.c_struct.block_stats, o.c_struct.tensor_stats, o.c_struct.sel,
                                         o.c_struct.scale_e8m0, sw.data_ptr(), sw.numel(), stream.cuda_stream)
                if st != mb.MOR_OK:
                    raise mb.MorError(st, "mor_select_stats")

        for _ in range(3):
            stats_step()
        torch.cuda.synchronize()
        ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        tms = []
        for _ in range(5):
            ea.record(stream); stats_step(); eb.record(stream)
            torch.cuda.synchronize()
            tms.append(ea.elapsed_time(eb))
        gbs = elements * 4.0 / (statistics.median(tms) * 1e-3) / 1e9      # the tensor is read twice, nothing else of size moves
        variants.append({"recipe": "mor_select_stats, 128x128 two-way Eq.3 with block statistics, one call per tensor (whole calls, 4 B/element)",
                         "whole_call_GBs": gbs, "frac_of_measured_copy": gbs / peak, "frac_of_8TBs": gbs / 8000.0})
        del so, sw

    # ---- the same tensors wanted along the rows (1x128) and along the columns (128x1): one call with a pair of
    #      entries per tensor (one read of each tile) against the two calls it replaces; whole calls
    if rank == 0 and not args.no_variants:
        nb2 = min(B, 8)
        rr = mb.Recipe((1, 128), recipe.formats, mb.MOR_CRIT_BLOCK_VS_E5M2, 0.045)
        rc = mb.Recipe((128, 1), recipe.formats, mb.MOR_CRIT_BLOCK_VS_E5M2, 0.045)
        plans = {"one_call_us": [mb.BatchPlan([x for x in xs[:nb2] for _ in (0, 1)], [rr, rc] * nb2)],
                 "two_calls_us": [mb.BatchPlan(xs[:nb2], [rr] * nb2), mb.BatchPlan(xs[:nb2], [rc] * nb2)]}
        both = {"workload": "%d of the tensors, 1x128 and 128x1 blocks, two-way Eq.3" % nb2}
        ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for key, pl in plans.items():
            for _ in range(3):
                for q in pl:
                    q.run(stream)
            torch.cuda.synchronize()
            tms = []
            for _ in range(5):
                ea.record(stream)
                for q in pl:
                    q.run(stream)
                eb.record(stream)
                torch.cuda.synchronize()
                tms.append(ea.elapsed_time(eb) * 1e3)
            both[key] = statistics.median(tms)
        variants.append({"recipe": "rows and columns of the same tensors", **both})
        del plans

    # ---- configs[0]: one 1024x1024 tensor, per-tensor partition: latency of a step, launched directly and
    #      replayed as a CUDA graph (the step is launch-bound at this size)
    small = None
    if rank == 0 and not args.no_variants:
        sb = wl.gaussian_outlier_rows()
        sx = torch.from_numpy(sb.view(np.int16)).view(torch.bfloat16).to(dev)
        sp = mb.BatchPlan([sx], [mb.Recipe((0, 0), recipe.formats, mb.MOR_CRIT_TENSOR_MEAN_REL, 0.045)])
        graph = sp.capture()
        small = {"workload": "configs[0]: one 1024x1024 tensor, per-tensor partition, Eq.2"}
        for key, fn in (("direct_us", lambda: sp.run(torch.cuda.current_stream())), ("cuda_graph_us", graph.replay)):
            for _ in range(5):
                fn()
            torch.cuda.synchronize()
            ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ts = []
            for _ in range(20):
                ea.record(); fn(); eb.record()
                torch.cuda.synchronize()
                ts.append(ea.elapsed_time(eb) * 1e3)
            small[key] = statistics.median(ts)
        del graph, sp

    # ---- end to end through the host-memory entry point: pinned inputs in, codes/scales/selection/stats out
    e2e = None
    if not args.no_e2e:
        Be = min(B, 4)
        pin_in = [torch.from_numpy(h.view(np.int16)).pin_memory() for h in host[:Be]]
        nb = (ROWS // BLOCK[0]) * (COLS // BLOCK[1])
        pin_codes = [torch.empty((ROWS, COLS), dtype=torch.uint8).pin_memory() for _ in range(Be)]
        pin_scale = [torch.empty((nb,), dtype=torch.uint8).pin_memory() for _ in range(Be)]
        pin_sel = [torch.empty((nb,), dtype=torch.uint8).pin_memory() for _ in range(Be)]
        pin_ts = [torch.empty((mb.TENSOR_STATS_DTYPE.itemsize,), dtype=torch.uint8).pin_memory() for _ in range(Be)]
        descs, outs = [], []
        for i in range(Be):
            descs.append(mb.make_desc(pin_in[i].data_ptr(), ROWS, COLS, COLS, recipe))
            o = mb.mor_outputs_t()
            o.codes, o.codes_ld = pin_codes[i].data_ptr(), COLS
            o.scale_e8m0, o.sel, o.tensor_stats = pin_scale[i].data_ptr(), pin_sel[i].data_ptr(), pin_ts[i].data_ptr()
            outs.append(o)
        nbytes = mb.mor_host_staging_bytes(descs[0])
        # two streams, each with its own staging buffer: the host->device copy of one tensor overlaps the
        # device->host copy of the previous one (the link is full duplex); each call is stream-ordered
        side = [torch.cuda.Stream(device=dev) for _ in range(2)]
        staging = [torch.empty((nbytes,), dtype=torch.uint8, device=dev) for _ in range(2)]

        def e2e_step():
            for i in range(Be):
                st = mb.mor_analyze_quantize_host(descs[i], outs[i], staging[i & 1].data_ptr(), nbytes, side[i & 1].cuda_stream)
                if st != mb.MOR_OK:
                    raise mb.MorError(st, "mor_analyze_quantize_host")

        def fork():
            for q in side:
                q.wait_stream(stream)

        def join():
            for q in side:
                stream.wait_stream(q)

        fork()
        for _ in range(3):
            e2e_step()
        join()
        sync_all()
        Ke = max(3, min(K, 10))
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fork()
        for _ in range(Ke):
            e2e_step()
        join()
        b.record(stream)
        sync_all()
        ms_e = a.elapsed_time(b)
        if world > 1:
            t = torch.tensor([ms_e], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms_e = float(t.item())
        el_e = ROWS * COLS * Be
        e2e = {"value": el_e * world * ALG_BYTES_STEP / (ms_e / Ke * 1e-3) / 1e9, "unit": "GB/s",
               "h2d_bytes_per_step": el_e * 2, "d2h_bytes_per_step": el_e + Be * (2 * nb + mb.TENSOR_STATS_DTYPE.itemsize),
               "tensors_per_step": Be, "steps": Ke, "ms_per_step": ms_e / Ke}

    # ---- the oracle on this machine's host cores (rank 0, single GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        reps = 9
        ts_ = []
        for _ in range(reps):
            t0 = time.perf_counter()
            oracle_step(host[0])
            ts_.append(time.perf_counter() - t0)
        dt = statistics.median(ts_)
        cpu = {"value": ROWS * COLS * ALG_BYTES_STEP / dt / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
               "sample": f"one {ROWS}x{COLS} tensor of the batch, median of {reps} runs ({sum(ts_):.1f} s of CPU work)",
               "elements_per_s": ROWS * COLS / dt, "host_cores_available": os.cpu_count()}

    if rank == 0:
        line = {"metric": "analyse+quantise throughput (algorithmic bytes)", "value": value, "unit": "GB/s",
                "n_gpus": world, "steps": K, "warmup": max(3, args.warmup), "ms_per_step": ms_step,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": "configs[1]: 4096x4096 weight-like BF16 N(0,0.02) x per-column 10^U(-1,1), "
                                       "128x128 blocks, candidates [E4M3,BF16], Eq.3 against E5M2, GAM scaling",
                           "tensors_per_step_per_gpu": B, "elements_per_step_per_gpu": elements,
                           "l2": "inputs (512 MiB per step at the default batch) exceed L2; no flush needed",
                           "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
                "elements_per_s": elements * world / (ms_step * 1e-3),
                "frac_of_hbm_peak_8TBs": value / 8000.0, "frac_of_measured_copy": value / peak,
                "fp8_block_fraction": fp8_frac, "fp8_tensor_fraction_eq2": tensor_fp8,
                "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu, "other_recipes_same_tensors": variants, "small_tensor_latency": small,
                "paper_context": "the paper reports no throughput and names no hardware; its own figures are FP8 tensor fractions "
                                 "(98.38 % / 95.93 % per channel, tensor-level MoR, Nemotron-3 8B)",
                "gpu_launches": 3 * K, "clocks": clocks}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
