#!/usr/bin/env python
"""Benchmark of one rTop-k round (Algorithm 1's communication path) on B200.

A step = rtopk_step over one batch: for W workers, a = g + m, top-r, random k-of-r, messages,
residual update, then the master's average into a dense vector.  Inputs are synthetic (see
paper_2005_10761_b200/workloads.py); the residual is carried from step to step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3_f32] [--impl ours|reference]

Prints one JSON line.  `value` is GB/s of gradient input (W*d*sizeof(g) per step over the device
time of a step, inputs resident in HBM); the timed region of K steps is repeated (`repeats`) and
`ms_per_step` is the median over the repeats, `ms_per_step_min` the fastest; `e2e` is the same
metric through rtopk_step_host with pinned host buffers (host<->device copies inside the timed
region); `roofline` is the dominant kernel's algorithmic bytes over its own event-timed duration
against the measured HBM copy bandwidth; `cpu_baseline` is the CPU oracle timed on a bounded sample
of the same workload; `sweep` holds short runs of the other configurations (the metric is defined
"vs d, W, r, k").  On one GPU the timed rounds are replays of a CUDA graph that holds one round per
resident gradient batch (`--graph 0` launches them on the stream instead); the kernels and their
work are the same, the round number that enters the Philox counter lives in a device word that every
round advances.  With --gpus N > 1 and no launcher in the environment the script starts N ranks
itself (one per GPU, NCCL).
"""
from __future__ import annotations

import argparse
import dataclasses
import hashlib
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "rtopk_step_gradient_input_bandwidth"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
# everything the dominant kernel is compiled from (a change voids the recorded DRAM traffic)
KERNEL_SOURCES = ["common.cuh", "element.cuh", "stream.cuh"]
L2_BYTES = 126 * 1024 * 1024


def load_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def kernel_source_hash() -> str:
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2005_10761_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(launch_bytes: float):
    """DRAM bytes per launch of the streaming kernel from the committed ncu summary, scaled by the
    algorithmic bytes when the capture was taken on a smaller case; None if there is no summary or
    the kernel sources changed since."""
    path = os.path.join(ROOT, "profiles", "k_stream_traffic.txt")
    try:
        kv = {}
        with open(path) as f:
            for line in f:
                if ":" in line and not line.startswith("#"):
                    a, b = line.split(":", 1)
                    kv[a.strip()] = b.strip()
        if kv.get("kernel_source_sha256_16") != kernel_source_hash():
            return None
        return float(kv["dram_bytes_per_launch"]) * launch_bytes / float(kv["algorithmic_bytes_per_launch"])
    except Exception:
        return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.lines, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._pump, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        rows = [l for (t, l) in self.lines if t0 - 0.05 <= t <= t1 + 0.15] or [l for _, l in self.lines]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in rows:
            c = [x.strip() for x in l.split(",")]
            if len(c) < 8:
                continue
            try:
                sm.append(float(c[0])); mx.append(float(c[1]))
            except ValueError:
                continue
            for n, v in zip(names, c[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def pick_workload(name: str, scale_d: int = 0, workers: int = 0):
    from paper_2005_10761_b200 import workloads as wl
    cfgs = wl.configs()
    if name not in cfgs:
        raise SystemExit(f"unknown workload {name!r}; choose from {sorted(cfgs)}")
    cfg = cfgs[name]
    if scale_d or workers:   # same recipe and ratios at another length / row count (small profiling captures)
        cfg = wl.scaled(cfg, d=scale_d or cfg.d, W=workers or cfg.W,
                        name=cfg.name + (f"_d{scale_d}" if scale_d else "") + (f"_W{workers}" if workers else ""))
    return cfg


def resident_batches(cfg, steps: int, warmup: int) -> int:
    gsz = 4 if cfg.grad_dtype == "f32" else 2
    return max(1, min(cfg.steps, int(24e9 // (cfg.W * cfg.ld * gsz)), steps + warmup))


def config_dict(cfg, args, world: int) -> dict:
    """What both arms (ours and --impl reference) print as `config`: the workload and how it is run."""
    seg = cfg.seg_off is not None
    return {"workload": cfg.name, "d": cfg.d, "W_per_gpu": cfg.W, "W_total": cfg.W * world, "r": cfg.r,
            "k": cfg.k_total, "grad_dtype": cfg.grad_dtype, "recipe": cfg.recipe,
            "segments": len(cfg.seg_r) if seg else 1,
            "gradient_batches_resident": resident_batches(cfg, args.steps, args.warmup),
            "residual": "carried across steps", "l2": "inputs larger than L2 (no flush)",
            "parallelism": f"workers sharded x{world}",
            "variant": ("rtopk_step_apply (fused master update)" if args.apply else
                        f"rtopk_step_threshold (theta = {args.threshold})" if args.threshold is not None
                        else "rtopk_step"),
            "select_path": args.select_path, "finish_path": getattr(args, "finish_path", "auto"),
            "reuse_threshold": bool(args.reuse_threshold)}


# ------------------------------------------------------------------------------------ CPU oracle legs
def oracle_sample(cfg, rows: int):
    """Host inputs of the bounded CPU-baseline sample: `rows` workers of step 0, zero residual."""
    import numpy as np
    from paper_2005_10761_b200 import workloads as wl
    g = wl.gradient(cfg, 0, "cpu", workers=range(rows))
    if cfg.grad_dtype == "bf16":
        import torch
        g_np = g.view(torch.int16).numpy().view(np.uint16)
    else:
        g_np = g.numpy()
    return g_np


def time_oracle(cfg, rows: int, threads: int, steps: int = 1, warmup: int = 0):
    """Times the oracle, as it stands, on `rows` rows per step.  Returns seconds per step."""
    import numpy as np
    import oracle
    oracle.set_threads(threads)
    g = oracle_sample(cfg, rows)
    m = np.zeros((rows, cfg.ld), dtype=np.float32)
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        if cfg.seg_off is None:
            idx, val = oracle.sparsify(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, it)
        else:
            idx, val = oracle.sparsify_segmented(g, m, cfg.d, cfg.seg_off, cfg.seg_r, cfg.seg_k, cfg.seed, it)
        oracle.aggregate(idx, val, cfg.d)
        if it >= warmup:
            times.append(time.perf_counter() - t0)
    return sum(times) / len(times)


def cpu_sample_rows(cfg, cores: int) -> int:
    # one full sort of d (key, index) pairs costs roughly 0.12 us per element and core
    per_row_s = max(0.05, cfg.d * 1.3e-7)
    budget_rows = max(1, int(20.0 * cores / per_row_s))
    return max(1, min(cfg.W, budget_rows, 2 * cores))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = pick_workload(args.workload, args.scale_d, args.workers)
    cores = os.cpu_count() or 1
    rows = cpu_sample_rows(cfg, cores)
    threads = min(cores, rows)
    # every step is one bounded sample; the whole run stays within a few minutes
    per_step = max(0.05, cfg.d * 1.3e-7) * ((rows + threads - 1) // threads) * 1.3
    steps = max(1, min(args.steps, int(120.0 / per_step)))
    warmup = min(args.warmup, max(0, int(30.0 / per_step)))
    sec = time_oracle(cfg, rows, threads, steps=steps, warmup=warmup)
    gsz = 4 if cfg.grad_dtype == "f32" else 2
    value = rows * cfg.d * gsz / sec / 1e9
    sample = (f"{rows} of {cfg.W} worker rows per step, step-0 gradient, residual carried; "
              f"{steps} timed steps after {warmup} warm-up steps (bounded to a few minutes of CPU work)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_dict(cfg, args, max(1, args.gpus)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------------ the GPU arm
class Round:
    """Buffers and the step call of one workload on this rank's GPU."""

    def __init__(self, cfg, args, dev, world=1, rank=0, grads=None, n_batches=None):
        import torch
        import paper_2005_10761_b200 as rt
        from paper_2005_10761_b200 import workloads as wl
        from paper_2005_10761_b200 import binding as B
        self.cfg, self.args, self.dev, self.world, self.rank = cfg, args, dev, world, rank
        self.W, self.d, self.ld = cfg.W, cfg.d, cfg.ld
        self.W_total = cfg.W * world
        self.gsz = 4 if cfg.grad_dtype == "f32" else 2
        self.K = cfg.k_total
        self.seg = cfg.seg_off is not None
        self.thr = args.threshold is not None
        self.ctx = rt.RTopK(d_max=self.d, W_max=self.W_total, r_max=min(self.d, 4 * cfg.r) if self.thr else cfg.r,
                            k_max=self.K, segments_max=len(cfg.seg_r) if self.seg else 1, device=dev.index)
        if args.reuse_threshold and args.select_path == "sampled":
            self.ctx.set_option(B.OPT_REUSE_THRESHOLD, 1)
        if args.select_path == "exact":
            self.ctx.set_option(B.OPT_SELECT_PATH, 1)
        if getattr(args, "finish_path", "auto") != "auto":
            self.ctx.set_option(B.OPT_FINISH_PATH, {"cluster": 1, "runs": 2}[args.finish_path])
        if grads is None:
            n_batches = n_batches or resident_batches(cfg, args.steps, args.warmup)
            shard_cfg = cfg if world == 1 else dataclasses.replace(cfg, W=self.W_total)
            rows = range(rank * self.W, rank * self.W + self.W)
            grads = [wl.gradient(shard_cfg, t, dev, workers=rows) for t in range(n_batches)]
        self.grads = grads
        self.n_batches = len(grads)
        self.residual = wl.zero_residual(cfg, dev)
        self.idx = torch.zeros((self.W, self.K), dtype=torch.int32, device=dev)
        self.val = torch.zeros((self.W, self.K), dtype=torch.float32, device=dev)
        # the dense update; with --apply the model weights that the update is applied to
        self.out = torch.zeros(wl.round_up(self.d, 4), dtype=torch.float32, device=dev)
        self.cnt = torch.zeros(self.W, dtype=torch.int32, device=dev)
        self.ones = torch.zeros(self.W, dtype=torch.int32, device=dev)
        self.sharded = world > 1 or bool(getattr(args, "exchange_path", False))
        if self.sharded:
            if self.seg:
                raise SystemExit("the sharded run covers the plain (whole-vector) workloads")
            from paper_2005_10761_b200 import sharded
            self.exchange = sharded.Exchange(self.W_total, self.K, world, rank, dev, always_collective=True)
        self.t_next = 0

    @property
    def n_slices(self):
        return self.W * (len(self.cfg.seg_r) if self.seg else 1)

    def step(self, t: int):
        cfg, ctx, args = self.cfg, self.ctx, self.args
        g = self.grads[t % self.n_batches]
        if not self.sharded:
            if self.seg:
                ctx.step_segmented(g, self.residual, self.d, cfg.seg_off, cfg.seg_r, cfg.seg_k, cfg.seed, t,
                                   self.idx, self.val, self.out)
            elif self.thr:
                ctx.step_threshold(g, self.residual, self.d, args.threshold, cfg.k, cfg.seed, t, self.idx, self.val,
                                   self.cnt, self.ones, self.out)
            elif args.apply:
                ctx.step_apply(g, self.residual, self.d, cfg.r, cfg.k, cfg.seed, t, 0.01, self.idx, self.val, self.out)
            else:
                ctx.step(g, self.residual, self.d, cfg.r, cfg.k, cfg.seed, t, self.idx, self.val, self.out)
        else:
            # workers sharded over the ranks: messages as 8-byte pairs, ONE all-gather, every rank aggregates
            from paper_2005_10761_b200 import sharded

            def sp(gl, ml, wb, pairs):
                ctx.sparsify_pairs(gl, ml, self.d, cfg.r, cfg.k, cfg.seed, t, pairs, worker_base=wb)

            def ag(pairs_all):
                ctx.aggregate_pairs(pairs_all, self.d, self.out)
                return self.out
            sharded.sharded_round(sp, ag, g, self.residual, self.exchange)

    def sync_all(self):
        import torch
        torch.cuda.synchronize()
        if self.sharded:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()

    def timed(self, fn, t_first: int, n: int) -> float:
        """Device time in ms of n consecutive steps (max over ranks)."""
        import torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.sync_all()
        e0.record()
        for t in range(t_first, t_first + n):
            fn(t)
        e1.record()
        self.sync_all()
        ms = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=self.dev)
        if self.sharded:
            import torch.distributed as dist
            dist.all_reduce(ms, op=dist.ReduceOp.MAX)
        return float(ms.item())

    def measure(self, steps: int, warmup: int, repeats: int, graph: bool):
        """Warm-up, then `repeats` timed regions of `steps` steps each.  Returns (ms per step of each
        region, kernels launched per region, launch mode)."""
        import torch
        from paper_2005_10761_b200 import binding as B
        ctx = self.ctx
        for _ in range(warmup):
            self.step(self.t_next); self.t_next += 1
        self.sync_all()
        graphed = graph and not self.sharded and not self.thr   # (the threshold call re-uploads its slice table)
        per_region, launches = [], 0
        if graphed:
            ctx.set_option(B.OPT_DEVICE_STEP, 1)
            ctx.set_device_step(self.t_next)
            graph_len = min(self.n_batches, steps)     # rounds held by the graph
            reps, rem = divmod(steps, graph_len)
            launches_per_graph = 0
            try:
                cap_stream = torch.cuda.Stream()
                g = torch.cuda.CUDAGraph()
                torch.cuda.synchronize()
                l0 = ctx.launch_count()
                with torch.cuda.graph(g, stream=cap_stream):
                    for b in range(graph_len):
                        self.step(b)
                launches_per_graph = ctx.launch_count() - l0
                g.replay()                 # untimed: the first launch of a graph also uploads it
                torch.cuda.synchronize()
            except Exception as ex:        # no capture on this machine: the rounds are launched one by one
                print(f"bench: CUDA graph capture failed ({ex!r}); launching on the stream", file=sys.stderr)
                torch.cuda.synchronize()
                graphed = False
                ctx.set_option(B.OPT_DEVICE_STEP, 0)
        if graphed:
            def graph_rounds(i: int):      # called once per timed step index; replays at the batch boundaries
                if i < reps * graph_len:
                    if i % graph_len == 0:
                        g.replay()
                else:
                    self.step(i)
            for _ in range(repeats):
                l0 = ctx.launch_count()
                per_region.append(self.timed(graph_rounds, 0, steps) / steps)
                launches = ctx.launch_count() - l0 + reps * launches_per_graph
            ctx.set_option(B.OPT_DEVICE_STEP, 0)
            self.t_next += steps * repeats + graph_len
        else:
            for _ in range(repeats):
                l0 = ctx.launch_count()
                per_region.append(self.timed(self.step, self.t_next, steps) / steps)
                launches = ctx.launch_count() - l0
                self.t_next += steps
        ctx.poll_status()
        return per_region, launches, ("cuda graph replay" if graphed else "stream launches")

    def profile_phases(self, n: int):
        """Phase durations (events between the phases of a call), averaged over n more steps, plus how many
        slices fell back to the exact selection and how many brackets were predicted."""
        from paper_2005_10761_b200 import binding as B
        ctx = self.ctx
        ctx.set_option(B.OPT_PROFILE, 1)
        phase_sum, fallbacks, predicted = {}, 0, 0
        for _ in range(n):
            self.step(self.t_next); self.t_next += 1
            for name, ms in ctx.phase_times().items():
                if ms >= 0:
                    phase_sum[name] = phase_sum.get(name, 0.0) + ms
            stats = [ctx.stats(s) for s in range(self.n_slices)]
            fallbacks += sum(s["used_fallback"] for s in stats)
            predicted += sum(s["bracket_predicted"] for s in stats)
        ctx.set_option(B.OPT_PROFILE, 0)
        return {k: v / n for k, v in phase_sum.items()}, fallbacks, predicted

    def step_bytes(self) -> int:
        """Algorithmic bytes of one step: g and m read, m' written, the dense update, messages written and read."""
        upd = 8 * self.W * self.K if self.args.apply else 4 * self.d   # --apply touches only the sent coordinates
        return self.W * self.d * (self.gsz + 8) + upd + 16 * self.W * self.K

    def stream_bytes(self) -> int:
        return self.W * self.d * (self.gsz + 8)

    def close(self):
        self.ctx.close()


def sweep_point(name, args, dev, peak, grads=None, steps=10, warmup=5, repeats=3, select_path=None, cold_l2=False,
                workers=0):
    """One short run of another configuration: the metric "vs d, W, r, k"."""
    import torch
    cfg = pick_workload(name, workers=workers)
    name = cfg.name
    a = argparse.Namespace(**vars(args))
    a.apply, a.threshold = False, None
    a.select_path = select_path or "sampled"
    a.steps, a.warmup = steps, warmup
    try:
        rd = Round(cfg, a, dev, grads=grads)
    except Exception as ex:
        return {"workload": name, "skipped": repr(ex)[:160]}
    try:
        regions, _, mode = rd.measure(steps, warmup, repeats, bool(args.graph))
        phases, fallbacks, _ = rd.profile_phases(5)
        ms = statistics.median(regions)
        e = {"workload": name, "d": cfg.d, "W": cfg.W, "r": cfg.r, "k": cfg.k_total, "dtype": cfg.grad_dtype,
             "select_path": a.select_path, "ms_per_step": ms, "ms_per_step_min": min(regions),
             "gbs_gradient_in": cfg.W * cfg.d * rd.gsz / (ms * 1e-3) / 1e9,
             "step_roofline_frac": rd.step_bytes() / (ms * 1e-3) / 1e9 / peak,
             "kstream_frac": (rd.stream_bytes() / (phases["stream"] * 1e-3) / 1e9 / peak) if phases.get("stream") else None,
             "phases_ms": {k: round(v, 4) for k, v in phases.items()}, "fallback_slices": fallbacks, "launch": mode}
        if cold_l2:
            # every step behind a write of a buffer larger than L2, timed on its own
            flush = torch.empty(2 * L2_BYTES // 4, dtype=torch.float32, device=dev)
            ts = []
            for _ in range(20):
                flush.fill_(1.0)
                ts.append(rd.timed(rd.step, rd.t_next, 1)); rd.t_next += 1
            e["ms_per_step_cold_l2"] = statistics.median(ts)
            del flush
        return e
    except Exception as ex:
        return {"workload": name, "skipped": repr(ex)[:160]}
    finally:
        rd.close()
        del rd
        torch.cuda.empty_cache()


def message_and_master_point(name, args, dev):
    """Times what follows the sparsifier on one configuration: the three message formats (encode, and the
    aggregation with the decoder fused in) and the three master updates.  Device time per call in
    microseconds, median of 20 calls behind a flush of L2 (the messages are a few MB)."""
    import torch
    import paper_2005_10761_b200 as rt
    cfg = pick_workload(name)
    a = argparse.Namespace(**vars(args))
    a.apply, a.threshold, a.select_path, a.steps, a.warmup = False, None, "sampled", 2, 2
    try:
        rd = Round(cfg, a, dev, n_batches=1)
    except Exception as ex:
        return {"workload": name, "skipped": repr(ex)[:160]}
    try:
        ctx, d, W, k = rd.ctx, cfg.d, cfg.W, cfg.k
        for t in range(2):
            rd.step(t)
        bits, lw, lh = rt.packed_layout(d, k)
        spans, ll, lh2 = rt.tiled_layout(d, k)
        pi = torch.zeros((W, lw), dtype=torch.int32, device=dev)
        pv = torch.zeros((W, lh), dtype=torch.int16, device=dev)
        tab = torch.zeros((W, spans + 1), dtype=torch.int32, device=dev)
        low = torch.zeros((W, ll), dtype=torch.int16, device=dev)
        qv = torch.zeros((W, lh2), dtype=torch.int16, device=dev)
        weights = torch.zeros_like(rd.out)
        velocity = torch.zeros_like(rd.out)
        flush = torch.empty(2 * L2_BYTES // 4, dtype=torch.float32, device=dev)
        calls = {
            "encode_packed": lambda: ctx.encode(rd.idx, rd.val, d, pi, pv),
            "encode_span_table": lambda: ctx.encode_tiled(rd.idx, rd.val, d, tab, low, qv),
            "aggregate_plain": lambda: ctx.aggregate(rd.idx, rd.val, d, rd.out),
            "aggregate_packed": lambda: ctx.aggregate_packed(pi, pv, d, k, rd.out),
            "aggregate_span_table": lambda: ctx.aggregate_tiled(tab, low, qv, d, k, rd.out),
            "apply_update": lambda: ctx.apply_update(rd.idx, rd.val, d, 0.01, weights),
            "apply_momentum": lambda: ctx.apply_momentum(rd.idx, rd.val, d, 0.01, 0.9, velocity, weights),
        }
        us = {}
        for label, fn in calls.items():
            fn()
            ts = []
            for _ in range(20):
                flush.fill_(1.0)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); fn(); e1.record()
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1) * 1e3)
            us[label] = round(statistics.median(ts), 2)
        ctx.poll_status()
        return {"workload": name, "kind": "messages_and_master", "d": d, "W": W, "k": k, "us_per_call": us,
                "bytes_per_entry": {"plain": 8.0, "packed": (bits + 16) / 8.0,
                                    "span_table": (4.0 * (spans + 1) + 4.0 * k) / k},
                "momentum_algorithmic_bytes": 16 * d, "l2": "flushed before every call"}
    except Exception as ex:
        return {"workload": name, "skipped": repr(ex)[:160]}
    finally:
        rd.close()
        del rd
        torch.cuda.empty_cache()


def run_sweep(args, dev, peak):
    import torch
    from paper_2005_10761_b200 import workloads as wl
    out = []
    out.append(sweep_point("c1", args, dev, peak, steps=50, warmup=10, cold_l2=True))
    for name in ("c2", "c2_n5", "c3_f32", "c3_bf16", "c4"):
        if name != args.workload:
            out.append(sweep_point(name, args, dev, peak, steps=20, warmup=10))
    for name in ("c2", "c3_f32"):
        out.append(sweep_point(name, args, dev, peak, steps=10, warmup=3, select_path="exact"))
    # one worker row: what each GPU of a job with one worker per GPU runs before the all-gather
    for name in ("c2", "c3_f32", "c3_bf16", "c4"):
        out.append(sweep_point(name, args, dev, peak, steps=50, warmup=10, workers=1))
    for name in ("c2", "c3_f32"):
        out.append(message_and_master_point(name, args, dev))
    # c5: d = 2^28; one gradient batch of the largest row count is generated once and shared (every
    # point reads rows 0..W-1 of it; the vector is 8x the L2 already at W = 1)
    free_b, _ = torch.cuda.mem_get_info()
    d5 = 1 << 28
    W_fit = int((free_b - 12e9) // (d5 * 4 * 2 * 1.08))
    W_all = [W for W in (1, 4, 16, 32) if W <= W_fit]
    if not W_all:
        out.append({"workload": "c5", "skipped": f"free memory {free_b / 1e9:.0f} GB holds no c5 row"})
        return out
    Wg = max(W_all)
    g5 = wl.gradient(dataclasses.replace(wl.configs()["c5_W32_r100_k10"], W=Wg), 0, dev)
    for W in W_all:
        names = [f"c5_W{W}_r{rd}_k{kd}" for rd in (100, 1000) for kd in (10, 4)] + [f"c5_W{W}_topk", f"c5_W{W}_randk"]
        for name in names:
            st = 3 if W >= 16 else 6
            out.append(sweep_point(name, args, dev, peak, grads=[g5[:W]], steps=st, warmup=3, repeats=3))
    if Wg < 32:
        out.append({"workload": "c5_W32_*", "skipped": f"free memory {free_b / 1e9:.0f} GB: W limited to {Wg}"})
    del g5
    torch.cuda.empty_cache()
    return out


def spawn_ranks(args) -> int:
    """--gpus N > 1 without a launcher: start N ranks of this script, one per GPU."""
    import torch
    have = torch.cuda.device_count()
    if have < args.gpus:
        print(f"bench: --gpus {args.gpus} but {have} CUDA devices are visible", file=sys.stderr)
        return 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--repeats", type=int, default=5, help="how many times the timed region of --steps steps is run")
    ap.add_argument("--workload", default="c3_f32")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--scale-d", type=int, default=0, help="run the workload's recipe at this vector length")
    ap.add_argument("--workers", type=int, default=0,
                    help="run the workload's recipe with this many worker rows per GPU (plain workloads)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--sweep", type=int, default=1, choices=[0, 1],
                    help="1 (default, one GPU): also run the other configurations briefly and print them as `sweep`")
    ap.add_argument("--select-path", default="sampled", choices=["sampled", "exact"],
                    help="exact: the multi-pass radix select over the full vector (RTOPK_OPT_SELECT_PATH = 1)")
    ap.add_argument("--finish-path", default="auto", choices=["auto", "cluster", "runs"],
                    help="RTOPK_OPT_FINISH_PATH: which kernels turn the candidates into messages (same result)")
    ap.add_argument("--apply", action="store_true",
                    help="time rtopk_step_apply (master update fused into the aggregation; plain workloads, 1 GPU)")
    ap.add_argument("--threshold", type=float, default=None,
                    help="time rtopk_step_threshold (the threshold-then-subsample encoder) with this theta "
                         "instead of rtopk_step (plain workloads, 1 GPU; message capacity = the workload's k)")
    ap.add_argument("--graph", type=int, default=1, choices=[0, 1],
                    help="1 (default): the timed rounds are replays of a CUDA graph that holds one round per resident "
                         "gradient batch (the round counter lives on the device, RTOPK_OPT_DEVICE_STEP, so every "
                         "replayed round still draws its own subset); 1 GPU")
    ap.add_argument("--exchange-path", action="store_true",
                    help="one GPU under torch.distributed.run with one rank: run the calls of the sharded job "
                         "(messages as pairs, the NCCL all-gather, in-place aggregation) instead of rtopk_step")
    ap.add_argument("--reuse-threshold", type=int, default=1, choices=[0, 1],
                    help="1 (default): the rounds of the loop predict their first threshold from the previous "
                         "rounds (RTOPK_OPT_REUSE_THRESHOLD; results are the same); 0: every round samples")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))

    import torch
    import torch.distributed as dist
    from paper_2005_10761_b200 import build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the product path)")
    if local >= torch.cuda.device_count():
        raise SystemExit(f"rank {rank}: no CUDA device {local} ({torch.cuda.device_count()} visible)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if args.exchange_path and "WORLD_SIZE" not in os.environ:
        raise SystemExit("--exchange-path needs a process group: start bench.py under torch.distributed.run")
    grouped = world > 1 or args.exchange_path
    if grouped:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build()
    if grouped:
        dist.barrier()

    cfg = pick_workload(args.workload, args.scale_d, args.workers)
    seg = cfg.seg_off is not None
    thr = args.threshold is not None
    if (args.apply or thr) and (seg or grouped):
        raise SystemExit("--apply and --threshold cover the plain single-GPU workloads")
    if args.select_path == "exact" and thr:
        raise SystemExit("--threshold runs on the sampled path only")
    rd = Round(cfg, args, dev, world, rank)
    W, d, K, gsz = rd.W, rd.d, rd.K, rd.gsz

    sampler = ClockSampler(local) if rank == 0 else None
    wall0 = time.time()
    regions, gpu_launches, launch_mode = rd.measure(args.steps, args.warmup, max(1, args.repeats), bool(args.graph))
    wall1 = time.time()
    clocks = sampler.stop(wall0, wall1) if sampler else None
    ms_per_step = statistics.median(regions)
    value = rd.W_total * d * gsz / (ms_per_step * 1e-3) / 1e9

    # the dominant kernel's own duration: more steps with events between the phases
    phases, fallbacks, predicted = rd.profile_phases(min(args.steps, 20))
    n_prof = min(args.steps, 20)
    peak, peak_src = load_peak()
    stream_bytes = rd.stream_bytes()
    stream_ms = phases.get("stream")
    achieved = stream_bytes / (stream_ms * 1e-3) / 1e9 if stream_ms else None
    roofline = {"bound": "hbm", "kernel": "k_stream (fused add + write-back + candidate gather)",
                "achieved": achieved, "peak": peak, "peak_source": peak_src, "unit": "GB/s",
                "frac": (achieved / peak) if achieved else None,
                "traffic": recorded_traffic(stream_bytes),
                "algorithmic_bytes_per_launch": stream_bytes, "kernel_ms": stream_ms}
    step_bytes = rd.step_bytes()
    step_gbs = step_bytes / (ms_per_step * 1e-3) / 1e9
    step_frac = step_gbs / peak if world == 1 else None

    # end to end: host gradient in, host messages + update out, through rtopk_step_host
    e2e = None
    if not args.no_e2e and not grouped and not seg and not args.apply and not thr:
        h_grad = rd.grads[0].cpu().pin_memory()
        h_idx = torch.zeros((W, K), dtype=torch.int32).pin_memory()
        h_val = torch.zeros((W, K), dtype=torch.float32).pin_memory()
        h_out = torch.zeros(d, dtype=torch.float32).pin_memory()

        def host_step(t: int):
            rd.ctx.step_host(h_grad, rd.residual, d, cfg.r, cfg.k, cfg.seed, t, h_idx, h_val, h_out)
        for _ in range(3):
            host_step(rd.t_next); rd.t_next += 1
        n_e2e = max(3, min(args.steps, 10))
        ms = rd.timed(host_step, rd.t_next, n_e2e) / n_e2e
        rd.t_next += n_e2e
        e2e = {"value": W * d * gsz / (ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms,
               "h2d_bytes_per_step": W * rd.ld * gsz, "d2h_bytes_per_step": 8 * W * K + 4 * d}
        del h_grad, h_idx, h_val, h_out
    elif not args.no_e2e and grouped and not seg:
        # the sharded job end to end: every rank uploads its rows' gradients from pinned host memory, runs the
        # round (sparsify into pairs, the all-gather, aggregation) and downloads the dense update
        h_grad = rd.grads[0].cpu().pin_memory()
        g_dev = torch.empty_like(rd.grads[0])
        h_out = torch.zeros(rd.out.numel(), dtype=torch.float32).pin_memory()
        kept = rd.grads

        def host_step(t: int):
            g_dev.copy_(h_grad, non_blocking=True)
            rd.step(t)
            h_out.copy_(rd.out, non_blocking=True)
        rd.grads, rd.n_batches = [g_dev], 1
        for _ in range(3):
            host_step(rd.t_next); rd.t_next += 1
        n_e2e = max(3, min(args.steps, 10))
        ms = rd.timed(host_step, rd.t_next, n_e2e) / n_e2e
        rd.t_next += n_e2e
        rd.grads, rd.n_batches = kept, len(kept)
        e2e = {"value": rd.W_total * d * gsz / (ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms,
               "h2d_bytes_per_step": W * rd.ld * gsz * world, "d2h_bytes_per_step": 4 * rd.out.numel() * world}
        del h_grad, g_dev, h_out
    rd.ctx.poll_status()
    rd.close()
    del rd
    torch.cuda.empty_cache()

    sweep = None
    if args.sweep and not grouped and rank == 0 and not (args.apply or thr or args.scale_d or args.workers):
        sweep = run_sweep(args, dev, peak)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cores = os.cpu_count() or 1
        n_rows = cpu_sample_rows(cfg, cores)
        threads = min(cores, n_rows)
        # one step to size the sample, then enough steps for roughly 12 s of CPU work
        sec = time_oracle(cfg, n_rows, threads)
        n_cpu_steps = max(1, min(40, int(12.0 / max(sec, 1e-3))))
        if n_cpu_steps > 1:
            sec = time_oracle(cfg, n_rows, threads, steps=n_cpu_steps)
        cpu = {"value": n_rows * d * gsz / sec / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
               "seconds": sec * n_cpu_steps,
               "sample": f"{n_cpu_steps} steps, {n_rows} of {W} worker rows, step-0 gradient, residual carried"}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "repeats": len(regions), "ms_per_step": ms_per_step,
            "ms_per_step_min": min(regions), "ms_per_step_regions": regions,
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_dict(cfg, args, world),
            "launch": launch_mode if not grouped else launch_mode + "; per round one NCCL all-gather of W*k 8-byte pairs",
            "elements_per_s": W * world * d / (ms_per_step * 1e-3),
            "step_roofline_frac": step_frac, "step_roofline_frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS if world == 1 else None,
            "step_algorithmic_bytes": step_bytes,
            "phases_ms": phases, "fallback_slices": fallbacks,
            "predicted_brackets": {"slices": predicted, "of": W * (len(cfg.seg_r) if seg else 1) * n_prof},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": gpu_launches,
            "clocks": clocks, "sweep": sweep,
        }))
    if grouped:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
