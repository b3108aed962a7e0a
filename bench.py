#!/usr/bin/env python
"""Benchmark of one rTop-k round (Algorithm 1's communication path) on B200.

A step = rtopk_step over one batch: for W workers, a = g + m, top-r, random k-of-r, messages,
residual update, then the master's average into a dense vector.  Inputs are synthetic (see
paper_2005_10761_b200/workloads.py); the residual is carried from step to step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl ours|reference]

Prints one JSON line.  `value` is GB/s of gradient input (W*d*sizeof(g) per step over the device
time of a step, inputs resident in HBM); `e2e` is the same through rtopk_step_host with pinned host
buffers (host<->device copies inside the timed region); `roofline` is the fused streaming kernel's
algorithmic bytes over its own event-timed duration against the measured HBM copy bandwidth;
`cpu_baseline` is the CPU oracle timed on a bounded sample of the same workload.
On one GPU the timed rounds are replays of a CUDA graph that holds one round per resident gradient
batch (`--graph 0` launches them on the stream instead); the kernels and their work are the same, the
round number that enters the Philox counter lives in a device word that every round advances.
"""
from __future__ import annotations

import argparse
import dataclasses
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "rtopk_step_gradient_input_bandwidth"
UNIT = "GB/s"
KERNEL_SOURCES = ["common.cuh", "element.cuh", "stream.cuh"]   # everything k_stream is compiled from


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


def recorded_traffic(workload: str, launch_bytes: float):
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
    sec = time_oracle(cfg, rows, threads, steps=args.steps, warmup=args.warmup)
    gsz = 4 if cfg.grad_dtype == "f32" else 2
    value = rows * cfg.d * gsz / sec / 1e9
    sample = f"{rows} of {cfg.W} worker rows per step, step-0 gradient, residual carried"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "d": cfg.d, "W": rows, "r": cfg.r, "k": cfg.k_total,
                   "grad_dtype": cfg.grad_dtype},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--scale-d", type=int, default=0, help="run the workload's recipe at this vector length")
    ap.add_argument("--workers", type=int, default=0,
                    help="run the workload's recipe with this many worker rows per GPU (plain workloads)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--apply", action="store_true",
                    help="time rtopk_step_apply (master update fused into the aggregation; plain workloads, 1 GPU)")
    ap.add_argument("--threshold", type=float, default=None,
                    help="time rtopk_step_threshold (the threshold-then-subsample encoder) with this theta "
                         "instead of rtopk_step (plain workloads, 1 GPU; message capacity = the workload's k)")
    ap.add_argument("--graph", type=int, default=1, choices=[0, 1],
                    help="1 (default): the timed rounds are replays of a CUDA graph that holds one round per resident "
                         "gradient batch (the round counter lives on the device, RTOPK_OPT_DEVICE_STEP, so every "
                         "replayed round still draws its own subset); 1 GPU")
    ap.add_argument("--reuse-threshold", type=int, default=1, choices=[0, 1],
                    help="1 (default): the rounds of the loop predict their first threshold from the previous "
                         "rounds (RTOPK_OPT_REUSE_THRESHOLD; results are the same); 0: every round samples")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    import paper_2005_10761_b200 as rt
    from paper_2005_10761_b200 import build, sharded, workloads as wl
    from paper_2005_10761_b200.binding import OPT_PROFILE

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the product path)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()

    cfg = pick_workload(args.workload, args.scale_d, args.workers)
    W, d, ld = cfg.W, cfg.d, cfg.ld
    W_total = W * world                      # weak scaling: W workers per GPU
    gsz = 4 if cfg.grad_dtype == "f32" else 2
    K = cfg.k_total
    seg = cfg.seg_off is not None
    thr = args.threshold is not None
    ctx = rt.RTopK(d_max=d, W_max=W_total, r_max=min(d, 4 * cfg.r) if thr else cfg.r, k_max=K,
                   segments_max=len(cfg.seg_r) if seg else 1, device=local)

    if args.reuse_threshold:
        from paper_2005_10761_b200.binding import OPT_REUSE_THRESHOLD
        ctx.set_option(OPT_REUSE_THRESHOLD, 1)

    # gradient batches resident in HBM before timing; the residual is carried across all steps
    batch_bytes = W * ld * gsz
    n_batches = max(1, min(cfg.steps, int(24e9 // batch_bytes), args.steps + args.warmup))
    shard_cfg = cfg if world == 1 else dataclasses.replace(cfg, W=W_total)
    rows = range(rank * W, rank * W + W)
    grads = [wl.gradient(shard_cfg, t, dev, workers=rows) for t in range(n_batches)]
    residual = wl.zero_residual(cfg, dev)
    idx = torch.zeros((W, K), dtype=torch.int32, device=dev)
    val = torch.zeros((W, K), dtype=torch.float32, device=dev)
    # the dense update; with --apply the model weights that the update is applied to
    out = torch.zeros(wl.round_up(d, 4), dtype=torch.float32, device=dev)
    if (args.apply or thr) and (seg or world > 1):
        raise SystemExit("--apply and --threshold cover the plain single-GPU workloads")
    cnt = torch.zeros(W, dtype=torch.int32, device=dev)
    ones = torch.zeros(W, dtype=torch.int32, device=dev)
    base = rank * W

    def one_step(t: int):
        g = grads[t % n_batches]
        if world == 1:
            if seg:
                ctx.step_segmented(g, residual, d, cfg.seg_off, cfg.seg_r, cfg.seg_k, cfg.seed, t, idx, val, out)
            elif thr:
                ctx.step_threshold(g, residual, d, args.threshold, cfg.k, cfg.seed, t, idx, val, cnt, ones, out)
            elif args.apply:
                ctx.step_apply(g, residual, d, cfg.r, cfg.k, cfg.seed, t, 0.01, idx, val, out)
            else:
                ctx.step(g, residual, d, cfg.r, cfg.k, cfg.seed, t, idx, val, out)
        else:
            def sp(gl, ml, wb):
                if seg:
                    ctx.sparsify_segmented(gl, ml, d, cfg.seg_off, cfg.seg_r, cfg.seg_k, cfg.seed, t, idx, val,
                                           worker_base=wb)
                else:
                    ctx.sparsify(gl, ml, d, cfg.r, cfg.k, cfg.seed, t, idx, val, worker_base=wb)
                return idx, val

            def ag(ia, va):
                ctx.aggregate(ia, va, d, out)
                return out
            sharded.sharded_round(sp, ag, g, residual, W_total, world, rank)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, t_first: int, n: int) -> float:
        """Device time in ms of n consecutive steps (max over ranks)."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sync_all()
        e0.record()
        for t in range(t_first, t_first + n):
            fn(t)
        e1.record()
        sync_all()
        ms = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(ms, op=dist.ReduceOp.MAX)
        return float(ms.item())

    t_next = 0
    for _ in range(args.warmup):
        one_step(t_next); t_next += 1
    sync_all()
    sampler = ClockSampler(local) if rank == 0 else None
    wall0 = time.time()
    launches0 = ctx.launch_count()
    graphed = bool(args.graph) and world == 1 and not thr   # (the threshold call re-uploads its slice table)
    if graphed:
        from paper_2005_10761_b200.binding import OPT_DEVICE_STEP
        ctx.set_option(OPT_DEVICE_STEP, 1)
        ctx.set_device_step(t_next)
        graph_len = min(n_batches, args.steps)     # rounds held by the graph
        reps, rem = divmod(args.steps, graph_len)
        launches_per_graph = 0
        if reps:
            try:
                cap_stream = torch.cuda.Stream()
                graph = torch.cuda.CUDAGraph()
                torch.cuda.synchronize()
                l0 = ctx.launch_count()
                with torch.cuda.graph(graph, stream=cap_stream):
                    for b in range(graph_len):
                        one_step(b)
                launches_per_graph = ctx.launch_count() - l0
                graph.replay()             # untimed: the first launch of a graph also uploads it
                torch.cuda.synchronize()
            except Exception as ex:        # no capture on this machine: the rounds are launched one by one
                print(f"bench: CUDA graph capture failed ({ex!r}); launching on the stream", file=sys.stderr)
                torch.cuda.synchronize()
                reps, rem, graphed = 0, args.steps, False

        def graph_rounds(i: int):          # called once per timed "step" index; replays at the batch boundaries
            if i < reps * graph_len:
                if i % graph_len == 0:
                    graph.replay()
            else:
                one_step(i)
        launches0 = ctx.launch_count()
        total_ms = timed(graph_rounds, 0, args.steps)
        gpu_launches = ctx.launch_count() - launches0 + reps * launches_per_graph
    else:
        total_ms = timed(one_step, t_next, args.steps)
        gpu_launches = ctx.launch_count() - launches0   # this library's kernels inside the timed region
    wall1 = time.time()
    t_next += args.steps
    clocks = sampler.stop(wall0, wall1) if sampler else None
    ctx.poll_status()
    ms_per_step = total_ms / args.steps
    value = W_total * d * gsz / (ms_per_step * 1e-3) / 1e9
    n_slices = W * (len(cfg.seg_r) if seg else 1)
    fallbacks = sum(ctx.stats(s)["used_fallback"] for s in range(n_slices))     # of the last timed step
    predicted = 0

    # the streaming kernel's own duration: same steps again with events between the phases
    ctx.set_option(OPT_PROFILE, 1)
    phase_sum, n_prof = {}, 0
    for _ in range(min(args.steps, 20)):
        one_step(t_next); t_next += 1
        for name, ms in ctx.phase_times().items():
            if ms >= 0:
                phase_sum[name] = phase_sum.get(name, 0.0) + ms
        n_prof += 1
        stats = [ctx.stats(s) for s in range(n_slices)]                         # ... and of every profiled step
        fallbacks += sum(s["used_fallback"] for s in stats)
        predicted += sum(s["bracket_predicted"] for s in stats)
    ctx.set_option(OPT_PROFILE, 0)
    phases = {k: v / n_prof for k, v in phase_sum.items()}
    peak, peak_src = load_peak()
    stream_bytes = W * d * (gsz + 8)
    stream_ms = phases.get("stream")
    achieved = stream_bytes / (stream_ms * 1e-3) / 1e9 if stream_ms else None
    roofline = {"bound": "hbm", "kernel": "k_stream (fused add + write-back + candidate gather)",
                "achieved": achieved, "peak": peak, "peak_source": peak_src, "unit": "GB/s",
                "frac": (achieved / peak) if achieved else None,
                "traffic": recorded_traffic(cfg.name, stream_bytes),
                "algorithmic_bytes_per_launch": stream_bytes, "kernel_ms": stream_ms}
    # with --apply the 4 d-byte dense update is not written: 8 bytes per sent coordinate instead
    step_bytes = W * d * (gsz + 8) + (8 * W * K if args.apply else 4 * d) + 16 * W * K
    step_frac = step_bytes / (ms_per_step * 1e-3) / 1e9 / peak if world == 1 else None

    # end to end: host gradient in, host messages + update out, through rtopk_step_host
    e2e = None
    if not args.no_e2e and world == 1 and not seg and not args.apply and not thr:
        h_grad = grads[0].cpu().pin_memory()
        h_idx = torch.zeros((W, K), dtype=torch.int32).pin_memory()
        h_val = torch.zeros((W, K), dtype=torch.float32).pin_memory()
        h_out = torch.zeros(d, dtype=torch.float32).pin_memory()

        def host_step(t: int):
            ctx.step_host(h_grad, residual, d, cfg.r, cfg.k, cfg.seed, t, h_idx, h_val, h_out)
        for _ in range(2):
            host_step(t_next); t_next += 1
        n_e2e = max(3, min(args.steps, 10))
        ms = timed(host_step, t_next, n_e2e) / n_e2e
        t_next += n_e2e
        e2e = {"value": W * d * gsz / (ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms,
               "h2d_bytes_per_step": W * ld * gsz, "d2h_bytes_per_step": 8 * W * K + 4 * d}
    ctx.poll_status()

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
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": cfg.name, "d": d, "W_per_gpu": W, "W_total": W_total, "r": cfg.r, "k": K,
                       "grad_dtype": cfg.grad_dtype, "recipe": cfg.recipe, "segments": len(cfg.seg_r) if seg else 1,
                       "gradient_batches_resident": n_batches, "residual": "carried across steps",
                       "l2": "inputs larger than L2 (no flush)", "parallelism": f"workers sharded x{world}",
                       "variant": ("rtopk_step_apply (fused master update)" if args.apply else
                                   f"rtopk_step_threshold (theta = {args.threshold})" if thr else "rtopk_step"),
                       "launch": "cuda graph replay" if (graphed and reps) else "stream launches",
                       "reuse_threshold": bool(args.reuse_threshold)},
            "elements_per_s": W_total * d / (ms_per_step * 1e-3),
            "step_roofline_frac": step_frac, "step_algorithmic_bytes": step_bytes,
            "phases_ms": phases, "fallback_slices": fallbacks,
            **({"marked_per_worker_last_step": float(ones.float().mean().item()),
                "sent_per_worker_last_step": float(cnt.float().mean().item())} if thr else {}),
            "predicted_brackets": {"slices": predicted, "of": n_slices * n_prof},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": gpu_launches,
            "clocks": clocks,
        }))
    if world > 1:
        dist.destroy_process_group()
    ctx.close()


if __name__ == "__main__":
    main()
