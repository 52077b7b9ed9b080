#!/usr/bin/env python
"""Throughput of the MoR analyse-and-quantise hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the whole hot path (tensor amax pre-pass, fused main kernel, finalise) over a
batch of distinct synthetic 4096x4096 weight-like BF16 tensors, 128x128 blocks, two-way selection
[E4M3, BF16] against E5M2 with GAM scaling (the benchmark's second configuration), issued as one batched
call.  The batch (512 MiB in, 256 MiB out by default) is larger than L2, so every step reads its inputs
from HBM.

Printed: ONE JSON line.
  value         GB/s of the bytes the RESULT needs (2 B/element read, 1 B/element of codes, scale and selection
                bytes: 3.0001 B/element) over the time of the whole step, all ranks.  GAM scaling needs the tensor
                amax before any block can be scaled (Algorithm 1), so the default path reads the tensor a second
                time in a pre-pass; that second read is paid in time and not counted as useful bytes.
  roofline      the main kernel alone (CUDA events around it inside the same steps), same bytes.
  configs       every benchmark configuration at full size: main kernel with the group amax supplied (single
                read), main kernel fed by the pre-pass, whole default call, decisions-only call; median and
                minimum over timed windows of at least 0.2 s.
  e2e           the same metric through the host-memory entry point, copies inside the timed region.
  cpu_baseline  the CPU oracle on this machine's host cores, one core and all cores.

With N > 1 (torchrun) every rank runs its own batch: replicas, no collective on the data path; time is the
maximum over ranks.  `--impl reference` times the CPU oracle (the only other implementation of the method that
exists) on a bounded sample per step.
"""
from __future__ import annotations

import argparse
import hashlib
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
FALLBACK_HBM_GBS = 6650.0
TARGET_FRAC_OF_8TBS = 0.75
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "main_kernel_blk128_keys_dram_traffic.txt")
WORKLOAD = ("configs[1]: 4096x4096 weight-like BF16 N(0,0.02) x per-column 10^U(-1,1), 128x128 blocks, "
            "candidates [E4M3,BF16], Eq.3 against E5M2, GAM scaling")


def alg_bytes(block, cols) -> float:
    """Bytes per element that the result needs: BF16 read, code write, one scale and one selection byte per block."""
    if tuple(block) == (0, 0):
        return 3.0
    n = block[0] * block[1] if block[1] else cols
    return 3.0 + 2.0 / max(n, 1)


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def csrc_digest() -> str:
    """Hash of the kernel sources: the DRAM counters under profiles/ are valid for exactly one such hash."""
    d = os.path.join(ROOT, "paper_2512_22804_b200", "csrc")
    h = hashlib.sha256()
    for name in sorted(os.listdir(d)):
        if name.endswith((".cu", ".cuh", ".h")):
            h.update(name.encode())
            with open(os.path.join(d, name), "rb") as f:
                h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(elements: int):
    """dram__bytes_read.sum + dram__bytes_write.sum of one main-kernel launch, scaled from the captured launch to this
    one by the elements processed; None when no capture is on file or the kernels have changed since it was taken."""
    try:
        kv = {}
        with open(TRAFFIC_FILE) as f:
            for line in f:
                if ":" in line and not line.lstrip().startswith("#"):
                    k, v = line.split(":", 1)
                    kv[k.strip()] = v.strip()
        if kv["csrc_digest"] != csrc_digest():
            return None
        per_el = (float(kv["dram_bytes_read"]) + float(kv["dram_bytes_write"])) / float(kv["elements"])
        return per_el * elements
    except Exception:
        return None


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
    steps = min(args.steps, 40)                  # bounded: the oracle does about 13 M elements per second per core
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(bits)
    dt = time.perf_counter() - t0
    el = sample_rows * COLS * steps
    gbs = el * alg_bytes(BLOCK, COLS) / dt / 1e9
    sample = f"first {sample_rows} rows of one tensor per step, {steps} steps"
    line = {"impl": "reference", "metric": "analyse+quantise throughput (bytes the result needs: 3.0001 B/element)",
            "value": gbs, "unit": "GB/s", "n_gpus": args.gpus, "steps": steps, "warmup": args.warmup,
            "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
            "elements_per_s": el / dt,
            "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------- timing helpers (GPU) ----

def timed_windows(fn, stage_events=None, min_window_s=0.2, max_calls=4000):
    """Calls ``fn`` back to back in windows of at least ``min_window_s`` in total; per call the CUDA-event time of the
    whole call and, with ``stage_events``, of the main kernel.  Returns medians and minima in microseconds."""
    import torch

    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    whole, main, spent = [], [], 0.0
    while spent < min_window_s and len(whole) < max_calls:
        ea.record(); fn(); eb.record()
        torch.cuda.synchronize()
        ms = ea.elapsed_time(eb)
        whole.append(ms * 1e3)
        if stage_events is not None:
            main.append(stage_events[0].elapsed_time(stage_events[1]) * 1e3)
        spent += ms * 1e-3
    out = {"calls": len(whole), "call_us_median": statistics.median(whole), "call_us_min": min(whole)}
    if main:
        out.update({"main_us_median": statistics.median(main), "main_us_min": min(main)})
    return out


def bench_config(name, tensors, copies, dev, peak, mb):
    """The four figures of one configuration: main kernel with the group amax supplied, main kernel fed by the
    pre-pass, whole default call, decisions-only call.  ``tensors``: list of (bits, recipe)."""
    import torch

    xs, recs = [], []
    for c in range(copies):
        for bits, r in tensors:
            xs.append(torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(dev))
            recs.append(r)
    elements = sum(int(x.numel()) for x in xs)
    nbytes = sum(int(x.numel()) * alg_bytes(r.block, x.shape[1]) for x, r in zip(xs, recs))
    stream = torch.cuda.current_stream()

    def events():
        e = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        for q in e:
            q.record(stream)
        s = mb.mor_stage_events_t()
        s.main_begin, s.main_end = e[0].cuda_event, e[1].cuda_event
        return e, s

    out = {"name": name, "tensors_per_call": len(xs), "elements_per_call": elements, "input_MiB": elements * 2 / 2**20,
           "bytes_needed_per_call": nbytes}

    def rates(us):
        gbs = nbytes / (us * 1e-6) / 1e9
        return {"GBs": gbs, "elements_per_s": elements / (us * 1e-6), "frac_of_measured_copy": gbs / peak, "frac_of_8TBs": gbs / 8000.0}

    # default call: pre-pass + main + finalise
    plan = mb.BatchPlan(xs, recs)
    ev, st = events()
    t = timed_windows(lambda: plan.run(stream, st), ev)
    out["default_call"] = {"us_median": t["call_us_median"], "us_min": t["call_us_min"], "calls": t["calls"], **rates(t["call_us_median"])}
    out["main_kernel_fed_by_pre_pass"] = {"us_median": t["main_us_median"], "us_min": t["main_us_min"], **rates(t["main_us_median"])}
    stats = [o.tensor_stats_dict() for o in plan.outs]
    out["blocks"] = {k: int(sum(s[k] for s in stats)) for k in ("n_blocks", "n_e4m3", "n_e5m2", "n_bf16")}
    out["eq2_mean_rel_error_e4m3"] = [round(float(s["mean_rel_e4m3"]), 6) for s in stats[:len(tensors)]]
    out["eq2_tensor_format"] = [int(s["tensor_format"]) for s in stats[:len(tensors)]]
    assert all(s["status"] == 0 for s in stats)
    ga = torch.tensor([s["group_amax"] for s in stats], dtype=torch.float32, device=dev)
    del plan
    # group amax supplied: no pre-pass, the tensor is read once
    if all(tuple(r.block) not in ((0, 0), (1, 0)) for r in recs):
        plan = mb.BatchPlan(xs, recs, group_amax=ga)
        ev, st = events()
        t = timed_windows(lambda: plan.run(stream, st), ev)
        out["amax_supplied_call"] = {"us_median": t["call_us_median"], "us_min": t["call_us_min"], **rates(t["call_us_median"])}
        out["main_kernel_amax_supplied"] = {"us_median": t["main_us_median"], "us_min": t["main_us_min"], **rates(t["main_us_median"])}
        del plan
    else:
        out["main_kernel_amax_supplied"] = "not applicable: a block that spans tiles takes its amax from the pre-pass"
    # decisions and statistics only (mor_select_stats_batched): 2 B/element read by each of the two kernels, nothing of size written
    plan = mb.BatchPlan(xs, recs, stats_only=True)
    t = timed_windows(lambda: plan.run(stream))
    us = t["call_us_median"]
    out["select_stats_call"] = {"us_median": us, "us_min": t["call_us_min"], "elements_per_s": elements / (us * 1e-6),
                                "GBs_of_2_bytes_per_element": elements * 2.0 / (us * 1e-6) / 1e9}
    del plan, xs
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=16, help="tensors per step")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-configuration table")
    ap.add_argument("--profile", default=None, metavar="RECIPE",
                    help="run only three calls of one recipe on --batch 4096x4096 tensors and exit (the small case that the "
                         "profiler wraps): 128x128, 1x128, 64x64, 128x1, per-tensor, per-channel, rows+cols, each optionally followed by "
                         "-supplied (group amax given: single read) or -three (three formats, gradient-like data)")
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
    peak, peak_kind = measured_peak()
    T2, T3 = (mb.MOR_FMT_E4M3, mb.MOR_FMT_BF16), (mb.MOR_FMT_E4M3, mb.MOR_FMT_E5M2, mb.MOR_FMT_BF16)
    E3 = mb.MOR_CRIT_BLOCK_VS_E5M2

    if args.profile:
        name = args.profile
        three, supplied = name.endswith("-three"), name.endswith("-supplied")
        base = name.replace("-three", "").replace("-supplied", "")
        block = {"128x128": (128, 128), "1x128": (1, 128), "64x64": (64, 64), "128x1": (128, 1), "per-tensor": (0, 0), "per-channel": (1, 0), "rows+cols": (1, 128)}[base]
        crit = mb.MOR_CRIT_TENSOR_MEAN_REL if block in ((0, 0), (1, 0)) else E3
        gen = (lambda i: wl.gradient_like(ROWS, COLS, seed=3 + i)) if three else (lambda i: wl.weight_like(ROWS, COLS, seed=1 + 1000 * i))
        pxs = [torch.from_numpy(gen(i).view(np.int16)).view(torch.bfloat16).to(dev) for i in range(args.batch)]
        ga = mb.group_amax(pxs) if supplied else None
        if base == "rows+cols":        # every tensor with 1x128 and with 128x1 blocks: one paired launch
            pair_x, pair_r = [], []
            for x in pxs:
                pair_x += [x, x]
                pair_r += [mb.Recipe((1, 128), T2, E3, 0.045), mb.Recipe((128, 1), T2, E3, 0.045)]
            pplan = mb.BatchPlan(pair_x, pair_r)
        else:
            pplan = mb.BatchPlan(pxs, [mb.Recipe(block, T3 if three else T2, crit, 0.045)] * args.batch, group_amax=ga)
        for _ in range(3):
            pplan.run(torch.cuda.current_stream())
        torch.cuda.synchronize()
        print(json.dumps({"profile": name, "tensors": args.batch, "elements_per_call": ROWS * COLS * args.batch,
                          "status": [o.tensor_stats_dict()["status"] for o in pplan.outs]}), flush=True)
        return

    # ---- inputs: `batch` distinct tensors per rank, resident in HBM
    B = args.batch
    host = [wl.weight_like(ROWS, COLS, seed=1 + 1000 * i + 100000 * rank) for i in range(B)]
    xs = [torch.from_numpy(h.view(np.int16)).view(torch.bfloat16).to(dev) for h in host]
    recipe = mb.Recipe(BLOCK, T2, E3, 0.045)
    plan = mb.BatchPlan(xs, [recipe] * B)
    stream = torch.cuda.current_stream()
    elements = ROWS * COLS * B
    bpe = alg_bytes(BLOCK, COLS)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    W = max(3, args.warmup)
    for _ in range(W):
        plan.run(stream)
    sync_all()

    # ---- timed region: K steps, CUDA events on the launching stream, stage events around every main kernel,
    #      and an event every K/10 steps so that the spread over ten windows can be reported
    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(K)]
    n_win = 10 if K >= 20 else 1
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_win + 1)]
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
    bounds = [round(i * K / n_win) for i in range(n_win + 1)]
    marks[0].record(stream)
    w = 1
    for k in range(K):
        plan.run(stream, stage[k])
        if k + 1 == bounds[w]:
            marks[w].record(stream)
            w += 1
    sync_all()
    clocks = sampler.stop()
    ms_total = marks[0].elapsed_time(marks[n_win])
    win_ms = [marks[i].elapsed_time(marks[i + 1]) / max(bounds[i + 1] - bounds[i], 1) for i in range(n_win)]
    main_ms = [a.elapsed_time(b) for a, b in ev]
    ms_main = sum(main_ms) / K
    if world > 1:
        t = torch.tensor([ms_total], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
    ms_step = ms_total / K
    value = elements * world * bpe / (ms_step * 1e-3) / 1e9

    stats = [o.tensor_stats_dict() for o in plan.outs]
    n_blocks = sum(s["n_blocks"] for s in stats)
    fp8_frac = sum(s["n_e4m3"] + s["n_e5m2"] for s in stats) / max(n_blocks, 1)
    tensor_fp8 = sum(1 for s in stats if s["tensor_format"] == mb.MOR_FMT_E4M3) / len(stats)

    achieved = elements * bpe / (ms_main * 1e-3) / 1e9
    roofline = {"kernel": "mor_main_kernel<128x128 blocks, Eq.3 yardstick, two formats, codes stored, keys and scales from the pre-pass>",
                "bound": "hbm", "achieved": achieved, "peak": peak, "peak_source": f"{peak_kind} copy bandwidth",
                "unit": "GB/s", "frac": achieved / peak, "frac_of_8TBs": achieved / 8000.0,
                "target_frac_of_8TBs": TARGET_FRAC_OF_8TBS, "target_met": achieved / 8000.0 >= TARGET_FRAC_OF_8TBS,
                "ms_per_launch": ms_main, "ms_per_launch_median": statistics.median(main_ms), "ms_per_launch_min": min(main_ms),
                "algorithmic_bytes_per_launch": elements * bpe, "traffic": recorded_traffic(elements),
                "traffic_source": os.path.relpath(TRAFFIC_FILE, ROOT) + " (null when the kernel sources differ from the captured build)"}

    # ---- every benchmark configuration at full size (rank 0, single-GPU runs)
    configs = []
    if rank == 0 and world == 1 and not args.no_configs:
        del plan
        torch.cuda.empty_cache()
        T = mb.MOR_CRIT_TENSOR_MEAN_REL
        configs.append(bench_config("configs[0] 1024x1024 Gaussian + 8 outlier rows, per tensor, Eq.2 (256 copies per call)",
                                    [(wl.gaussian_outlier_rows(), mb.Recipe((0, 0), T2, T))], 256, dev, peak, mb))
        configs.append(bench_config("configs[1] 4096x4096 weight-like, 128x128, two-way Eq.3 (16 distinct tensors per call)",
                                    [(h, recipe) for h in host], 1, dev, peak, mb))
        configs.append(bench_config("configs[1] tensors with 1x128 blocks, two-way Eq.3",
                                    [(h, mb.Recipe((1, 128), T2, E3)) for h in host], 1, dev, peak, mb))
        configs.append(bench_config("configs[1] tensors with 128x128 blocks, tensor-level Eq.2 only (E4M3 error alone)",
                                    [(h, mb.Recipe((128, 128), T2, T)) for h in host], 1, dev, peak, mb))
        configs.append(bench_config("configs[1] tensors with 128x1 sub-column blocks (transposed codes), two-way Eq.3",
                                    [(h, mb.Recipe((128, 1), T2, E3)) for h in host], 1, dev, peak, mb))
        configs.append(bench_config("configs[1] tensors with 64x64 blocks, two-way Eq.3",
                                    [(h, mb.Recipe((64, 64), T2, E3)) for h in host], 1, dev, peak, mb))
        a = wl.activation_like()
        configs.append(bench_config("configs[2] 8192x4096 activation-like, 1x128, two-way Eq.3 (8 copies per call)",
                                    [(a, mb.Recipe((1, 128), T2, E3))], 8, dev, peak, mb))
        del a
        g = wl.gradient_like()
        configs.append(bench_config("configs[3] 8192x14336 gradient-like, 1x128, three-way (3 copies per call)",
                                    [(g, mb.Recipe((1, 128), T3, E3))], 3, dev, peak, mb))
        configs.append(bench_config("configs[3] 8192x14336 gradient-like, 128x128, three-way (3 copies per call)",
                                    [(g, mb.Recipe((128, 128), T3, E3))], 3, dev, peak, mb))
        # a grid of 128x128 blocks that really is mixed: per-tile exponent spread drawn between 4 and 36 binades
        mixed = wl.mixed_grid()
        configs.append(bench_config("mixed grid: 4096x4096, per-tile spread of 4..36 binades (E4M3, E5M2 and BF16 tiles side by side), 128x128, three-way (16 copies per call)",
                                    [(mixed, mb.Recipe((128, 128), T3, E3))], 16, dev, peak, mb))
        del g, mixed
        cases = wl.config_case(4)
        configs.append(bench_config("configs[4] the 14 operands of one Llama-style layer in one batched call (weights 128x128, activations and output gradients 1x128)",
                                    [(c.bits, mb.Recipe(tuple(c.block), tuple(c.formats), c.criterion, c.threshold)) for c in cases],
                                    1, dev, peak, mb))
        del cases
        # rows and columns of the same tensors: one call with a pair of entries per tensor against the two calls it replaces
        nb2 = min(B, 8)
        rr, rc = mb.Recipe((1, 128), T2, E3), mb.Recipe((128, 1), T2, E3)
        both = {"name": "rows (1x128) and columns (128x1) of %d configs[1] tensors" % nb2}
        for key, pl in (("one_paired_call", [mb.BatchPlan([x for x in xs[:nb2] for _ in (0, 1)], [rr, rc] * nb2)]),
                        ("two_calls", [mb.BatchPlan(xs[:nb2], [rr] * nb2), mb.BatchPlan(xs[:nb2], [rc] * nb2)])):
            t = timed_windows(lambda: [q.run(stream) for q in pl])
            both[key] = {"us_median": t["call_us_median"], "us_min": t["call_us_min"]}
        configs.append(both)
        # one small tensor: launch-bound; launched directly and replayed as a CUDA graph
        sx = torch.from_numpy(wl.gaussian_outlier_rows().view(np.int16)).view(torch.bfloat16).to(dev)
        sp = mb.BatchPlan([sx], [mb.Recipe((0, 0), T2, T)])
        graph = sp.capture()
        small = {"name": "configs[0]: one 1024x1024 tensor per call (latency)"}
        for key, fn in (("direct", lambda: sp.run(torch.cuda.current_stream())), ("cuda_graph", graph.replay)):
            t = timed_windows(fn, min_window_s=0.05)
            small[key] = {"us_median": t["call_us_median"], "us_min": t["call_us_min"]}
        configs.append(small)
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
        Ke = max(3, min(K, 40))
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
        e2e = {"value": el_e * world * bpe / (ms_e / Ke * 1e-3) / 1e9, "unit": "GB/s",
               "h2d_bytes_per_step": el_e * 2, "d2h_bytes_per_step": el_e + Be * (2 * nb + mb.TENSOR_STATS_DTYPE.itemsize),
               "tensors_per_step": Be, "steps": Ke, "ms_per_step": ms_e / Ke,
               "note": "bound by the host link: 2 B/element in, 1 B/element out per tensor, copies in both directions overlapped"}

    # ---- the oracle on this machine's host cores (rank 0, single GPU runs only): one core and all cores
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        def time_oracle(threads, reps):
            ts_ = []
            for _ in range(reps):
                t0 = time.perf_counter()
                oracle_step(host[0], threads)
                ts_.append(time.perf_counter() - t0)
            return statistics.median(ts_), sum(ts_)

        ncores = os.cpu_count() or 1
        dt1, tot1 = time_oracle(1, 9)
        dtn, totn = time_oracle(ncores, 15)
        cpu = {"value": ROWS * COLS * bpe / dt1 / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
               "sample": f"one {ROWS}x{COLS} tensor of the batch, median of 9 runs ({tot1:.1f} s of CPU work)",
               "elements_per_s": ROWS * COLS / dt1,
               "all_cores": {"value": ROWS * COLS * bpe / dtn / 1e9, "unit": "GB/s", "cores": ncores, "elements_per_s": ROWS * COLS / dtn,
                             "sample": f"the same tensor, blocks spread over {ncores} threads, median of 15 runs ({totn:.1f} s wall)"}}

    if rank == 0:
        line = {"metric": "analyse+quantise throughput (bytes the result needs: 3.0001 B/element; the pre-pass read is time, not bytes)",
                "value": value, "unit": "GB/s",
                "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms_step,
                "ms_per_step_windows": {"median": statistics.median(win_ms), "min": min(win_ms), "max": max(win_ms), "windows": n_win},
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": WORKLOAD,
                           "tensors_per_step_per_gpu": B, "elements_per_step_per_gpu": elements,
                           "l2": "inputs (512 MiB per step at the default batch) exceed L2; no flush needed",
                           "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
                "elements_per_s": elements * world / (ms_step * 1e-3),
                "frac_of_hbm_peak_8TBs": value / 8000.0, "frac_of_measured_copy": value / peak,
                "whole_path_note": "GAM scaling (Algorithm 1) needs the tensor amax before any block is scaled: the default call reads the "
                                   "tensor twice (pre-pass + main kernel); with the group amax supplied it is read once (see configs[].amax_supplied_call)",
                "fp8_block_fraction": fp8_frac, "fp8_tensor_fraction_eq2": tensor_fp8,
                "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu, "configs": configs,
                "paper_context": "the paper reports no throughput and names no hardware; its own figures are FP8 tensor fractions "
                                 "(98.38 % / 95.93 % per channel, tensor-level MoR, Nemotron-3 8B)",
                "gpu_launches": 3 * K, "clocks": clocks}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
