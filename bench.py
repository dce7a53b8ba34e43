#!/usr/bin/env python
"""Benchmark of the resource-constrained submodular partition on B200.

One "step" = one full pass of the hot path over one synthetic dataset: class split, similarity
matrices, and the whole greedy loop of Algorithm 1 (every class, every pick).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C2] [--impl ours|reference]

Prints ONE JSON line.  `value` is samples partitioned per second with the inputs already in HBM;
`e2e` is the same metric through the host-buffer entry point (host->device and device->host
copies inside the timed region).  With N > 1 (torchrun) every rank partitions its own dataset of
the same shape (weak scaling; classes and datasets are independent, no data-path collective).

`--impl reference` times the CPU oracle (the only reference implementation there is: the paper
ships no code) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
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


# DRAM bytes (read + write) of one launch of the dominant kernel under ncu, by (configuration, kernel).
MEASURED_TRAFFIC = {("C2", "greedy_async_kernel"): 41.62e9}     # profiles/greedy_async_kernel_C2.md, capture A


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def measure_yardsticks(rcd, ctx, dev, dtype_code):
    """Times the library's own yardstick kernels with CUDA events: L2-resident and HBM read sweeps (GB/s) and the
    tensor-core peak loop for the feature dtype (TFLOP/s or TOP/s).  Best of three after one warm-up each."""
    import torch
    out = {}
    l2 = int(torch.cuda.get_device_properties(dev).L2_cache_size)

    def best_of(fn, reps=3):
        fn()
        torch.cuda.synchronize(dev)
        best = None
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            work = fn()
            e1.record()
            torch.cuda.synchronize(dev)
            ms = e0.elapsed_time(e1)
            rate = work / (ms * 1e-3)
            best = rate if best is None or rate > best else best
        return best

    small = torch.empty(l2 // 2, dtype=torch.uint8, device=dev).fill_(1)
    out["l2_read_gbs"] = best_of(lambda: rcd.rcd_yardstick_read(ctx, small, repeats=300)) / 1e9
    out["l2_read_buffer_mb"] = small.numel() / 1e6
    big = torch.empty(4 << 30, dtype=torch.uint8, device=dev).fill_(1)
    out["hbm_read_gbs"] = best_of(lambda: rcd.rcd_yardstick_read(ctx, big, repeats=1)) / 1e9
    del small, big
    out["mma_tflops"] = best_of(lambda: rcd.rcd_yardstick_mma(ctx, dtype_code, 20000)) / 1e12
    ctx.sync_status()
    out["mma_dtype"] = "int8" if dtype_code == rcd.RCD_FEAT_I8 else "bf16"
    return out


def oracle_sample(wl, picks: int, threads: int):
    """Times the CPU oracle on a bounded sample: `threads` classes, one per thread, similarity in
    full and the first `picks` picks of Algorithm 1; the oracle's cost per pick is constant (it
    evaluates all M x M terms each pick), so the full-class time is similarity + picks-time * M/picks."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import rcd_oracle as orc
    groups = orc.split_by_label(wl.labels, wl.L)
    classes = [l for l in range(wl.L) if len(groups[l]) > 0][:threads]
    M = len(groups[classes[0]])

    def one(l):
        ids = groups[l]
        t0 = time.perf_counter()
        S = orc.similarity(wl.features[ids])
        t1 = time.perf_counter()
        q = orc.quotas(len(ids), wl.capacities)
        orc.partition_class(S, q, "incremental", max_picks=picks)
        t2 = time.perf_counter()
        return t1 - t0, t2 - t1

    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=len(classes)) as ex:
        times = list(ex.map(one, classes))
    wall = time.perf_counter() - t0
    sim_s = max(t[0] for t in times)
    pick_s = max(t[1] for t in times)
    full_wall = sim_s + pick_s * (M / float(min(picks, M)))       # wall time of the same classes run to the end
    samples = len(classes) * M
    return dict(value=samples / full_wall, wall_sampled_s=wall, classes=len(classes), M=M, picks=min(picks, M),
                cores=len(classes), full_wall_extrapolated_s=full_wall)


def run_reference(args):
    from paper_2211_00839_b200.workloads import make_workload
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = make_workload(args.config, L=args.classes or None)
    cores = min(os.cpu_count() or 1, wl.L)
    vals, walls = [], []
    for i in range(args.warmup + args.steps):
        r = oracle_sample(wl, args.ref_picks, cores)
        if i >= args.warmup:
            vals.append(r["value"])
            walls.append(r["wall_sampled_s"])
    value = statistics.median(vals)
    sample = ("%d of %d classes (one thread each), similarity in full, first %d of %d picks of Algorithm 1; "
              "per-pick cost of the oracle is constant, time scaled by %d/%d"
              % (r["classes"], wl.L, r["picks"], r["M"], r["M"], r["picks"]))
    out = {"impl": "reference", "metric": "samples partitioned/sec", "value": value, "unit": "samples/s",
           "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": 1e3 * statistics.median(walls), "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "int64" if wl.dtype == "int8" else "f64", "data": "synthetic",
           "config": {"workload": workload_name(args.config, wl)},
           "cpu_baseline": {"value": value, "unit": "samples/s", "cores": r["cores"], "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def workload_name(cfg, wl):
    M = wl.N // wl.L
    return "%s: %d classes x %d samples, %s d=%d, W=%d" % (cfg, wl.L, M, wl.dtype, wl.d, wl.W)


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2211_00839_b200 import binding as rcd
    from paper_2211_00839_b200.workloads import make_workload, CONFIGS

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)

    # replicas (default; weak scaling): every rank partitions its own dataset of the same shape (seed differs per rank).
    # --sharding classes (strong scaling): ONE dataset, its classes sharded over the ranks by M^3, one all-gather of
    # the assignment at the end of every step.
    by_classes = args.sharding == "classes"
    wl = make_workload(args.config, L=args.classes or None, seed=CONFIGS[args.config]["seed"] + (0 if by_classes else 1000 * rank))
    M = wl.N // wl.L
    Xh = rcd.features_to_torch(wl.features, pin=True)
    yh = torch.from_numpy(wl.labels).pin_memory()
    Xd, yd = Xh.to(dev), yh.to(dev)
    kind = rcd.RCD_SIM_GAUSSIAN if args.similarity == "gaussian" else rcd.RCD_SIM_DOT
    ctx = rcd.Context(local, sweep_batch_max=args.sweep_batch, profile=1, greedy_path=args.greedy_path, similarity_kind=kind,
                      async_group=args.async_group, async_help_min=args.async_help_min, lazy_mode=args.lazy_mode, lazy_from=args.lazy_from, dense_ring=args.dense_ring, incremental=args.incremental, incremental_max=args.incremental_max,
                      objective=rcd.RCD_OBJ_GRAPH_CUT if args.objective == "cut" else rcd.RCD_OBJ_FACILITY)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def step_device():
        if by_classes:
            from paper_2211_00839_b200.distributed import partition_sharded_gpu
            return partition_sharded_gpu(ctx, Xd, yd, wl.capacities, wl.L)
        out = ctx.rcd_partition(Xd, yd, wl.capacities, wl.L, M_max=M)
        return out

    host_out = None

    def step_host():
        nonlocal host_out
        host_out = ctx.rcd_partition_host(Xh, yh, wl.capacities, wl.L, M_max=M, out=host_out)
        return host_out

    for _ in range(args.warmup):
        step_device()
    ctx.sync_status()
    launches_per_step = int(ctx.profile()["kernel_launches"])

    # Inputs of a step = the similarity matrices every sweep re-reads.  When they exceed L2 nothing survives between
    # steps; when they fit, a buffer larger than L2 is written between the timed steps (outside the event pairs).
    l2_bytes = int(torch.cuda.get_device_properties(local).L2_cache_size)
    s_bytes = 4.0 * wl.L * M * M
    fits_l2 = s_bytes <= l2_bytes
    flush = torch.empty(2 * l2_bytes, dtype=torch.uint8, device=dev) if fits_l2 else None

    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    pairs = []
    for _ in range(args.steps):
        if flush is not None:
            flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        out = step_device()
        e1.record()
        pairs.append((e0, e1))
    barrier()
    ctx.sync_status()
    # (one bracket around all K steps when nothing is flushed in between; the sum of the steps' own brackets otherwise)
    ms = pairs[0][0].elapsed_time(pairs[-1][1]) if flush is None else sum(a.elapsed_time(b) for a, b in pairs)
    prof = ctx.profile()
    # a short timed region leaves the 100 ms clock sampler with nothing: keep the same load running (untimed) until it
    # has a dozen samples, and say so
    extra_steps = 0
    t_guard = time.perf_counter()
    while len(sampler.lines) < 12 and time.perf_counter() - t_guard < 4.0:
        step_device()
        torch.cuda.synchronize()
        extra_steps += 1
    clocks = sampler.stop()
    clocks["sampled_over"] = "the timed steps" if extra_steps == 0 else "the timed steps and %d further identical steps (untimed)" % extra_steps
    ctx.sync_status()
    if world > 1:
        t = torch.tensor([ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    jobs = 1 if by_classes else world                 # datasets partitioned per step, all ranks together
    value = jobs * wl.N * args.steps / (ms * 1e-3)

    # end to end: host buffers in, host buffers out, copies inside the timed region
    for _ in range(max(1, min(args.warmup, 2))):
        step_host()
    barrier()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e2.record()
    for _ in range(args.steps):
        step_host()
    e3.record()
    barrier()
    e2e_wall_ms = (time.perf_counter() - t0) * 1e3
    e2e_ms = max(e2.elapsed_time(e3), 0.0)
    if world > 1:
        t = torch.tensor([e2e_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    e2e_value = jobs * wl.N * args.steps / (e2e_ms * 1e-3)
    h2d = Xh.numel() * Xh.element_size() + yh.numel() * 4
    d2h = sum(t.numel() * t.element_size() for t in host_out)

    # Roofline of the dominant kernel.  The whole greedy loop is ONE launch (greedy_async_kernel when
    # classes are few: pick CTAs and sweep CTAs hand classes back and forth; greedy_persistent_kernel
    # otherwise: sweep phases and pick phases separated by grid barriers); it is HBM-bound through its
    # sweeps.  Algorithmic bytes = for every sweep of a class, the rows of S of its unassigned samples
    # plus the coverage vectors of the blocks refreshed (4*ld*(n_R + n) bytes), summed on the device.
    # Duration = CUDA events around the greedy loop on the launching stream (last timed step).
    peaks = load_peaks()
    yard = measure_yardsticks(rcd, ctx, dev, rcd.RCD_FEAT_I8 if wl.dtype == "int8" else rcd.RCD_FEAT_BF16) if rank == 0 else None
    if world > 1:
        box = [yard]
        dist.broadcast_object_list(box, src=0)
        yard = box[0]
    default_setup = args.classes == 0 and args.sweep_batch in (0, 8) and args.async_group == 0 and args.async_help_min == 0 and args.similarity == "dot"
    loop_s = prof["greedy_ms"] * 1e-3
    achieved = prof["sweep_bytes"] / loop_s / 1e9 if loop_s > 0 else 0.0
    sms = torch.cuda.get_device_properties(local).multi_processor_count
    path = args.greedy_path if args.greedy_path else (3 if wl.L * 4 <= sms else 4)
    if args.objective != "facility":
        kernel_name = "cut_chain_kernel"
    else:
        kernel_name = {1: "sweep_kernel", 2: "greedy_persistent_kernel", 3: "greedy_async_kernel", 4: "greedy_owner_kernel"}[path]
    # S larger than L2: the sweeps stream from HBM (peak: the measured copy bandwidth); S inside L2: they stream from
    # L2 (peak: this library's read-only sweep yardstick over an L2-resident buffer, measured in this run)
    bound = "l2" if fits_l2 else "hbm"
    sweep_peak = yard["l2_read_gbs"] if fits_l2 else peaks["hbm_gbs"]
    roofline = {"bound": bound, "kernel": kernel_name, "achieved": achieved, "peak": sweep_peak,
                "unit": "GB/s", "frac": achieved / sweep_peak,
                "peak_source": ("measured in this run: read-only sweep over %.0f MB (L2-resident)" % yard["l2_read_buffer_mb"]) if fits_l2 else peaks["source"],
                "yardsticks": yard,
                # dram__bytes_read.sum + dram__bytes_write.sum of one launch of that kernel on this workload, from the
                # ncu capture summarised under profiles/ (None: no capture of the kernel as it stands)
                "traffic": MEASURED_TRAFFIC.get((args.config, kernel_name)) if default_setup else None,
                "launch_ms": prof["greedy_ms"], "bytes_per_launch": prof["sweep_bytes"],
                "rounds_with_sweeps": int(prof["sweep_launches"])}
    # the same bytes against the time the kernel spends sweeping (its own clock: the sweep phases of the
    # round-based kernel, the busy time of the first sweep CTA of the asynchronous one)
    if prof["persistent_sweep_ns"] > 0:
        ph = prof["sweep_bytes"] / (prof["persistent_sweep_ns"] * 1e-9) / 1e9
        roofline["sweep_phases"] = {"achieved": ph, "frac": ph / sweep_peak, "ms": prof["persistent_sweep_ns"] * 1e-6,
                                    "pick_phases_ms": prof["persistent_pick_ns"] * 1e-6,
                                    "elem_block_ops_per_s": prof["sweep_elem_ops"] / (prof["persistent_sweep_ns"] * 1e-9)}
    # When the library corrects stored gains in place, the loop reads little and is bound by the latency of its chain of
    # picks.  The same dataset with that correction switched off (every block that received a sample waits for a pass
    # over S: the bandwidth-bound form of the loop) is timed beside it, so that the sweep itself has its roofline too.
    if prof["incremental_updates"] > 0 and args.objective == "facility":
        ctx3 = rcd.Context(local, sweep_batch_max=args.sweep_batch, profile=1, greedy_path=args.greedy_path, similarity_kind=kind, incremental=2)
        for _ in range(2):
            ctx3.rcd_partition(Xd, yd, wl.capacities, wl.L, M_max=M)
        ctx3.sync_status()
        p3 = ctx3.profile()
        a3 = p3["sweep_bytes"] / (p3["greedy_ms"] * 1e-3) / 1e9
        roofline["note"] = ("default run: %d of %d picks correct their block's stored gains in place, so the launch reads %.1fx fewer bytes "
                            "than the passes-only form and is bound by the latency of each class's chain of picks, not by bandwidth; "
                            "the bandwidth-bound form of the same kernel on the same dataset is under passes_only"
                            % (int(prof["incremental_updates"]), wl.N, p3["sweep_bytes"] / max(1.0, prof["sweep_bytes"])))
        roofline["passes_only"] = {"what": "same dataset, in-place correction of stored gains off: every out-of-date block waits for a pass over S",
                                   "ms_per_step": p3["total_ms"], "launch_ms": p3["greedy_ms"], "bytes_per_launch": p3["sweep_bytes"],
                                   "achieved": a3, "frac": a3 / sweep_peak}
        if p3["persistent_sweep_ns"] > 0:
            ph3 = p3["sweep_bytes"] / (p3["persistent_sweep_ns"] * 1e-9) / 1e9
            roofline["passes_only"]["while_sweeping"] = {"achieved": ph3, "frac": ph3 / sweep_peak, "ms": p3["persistent_sweep_ns"] * 1e-6}
        ctx3.close()
    # and with every round's sweep as a launch of its own (sweep_kernel), one CUDA-event pair each
    ctx2 = rcd.Context(local, sweep_batch_max=args.sweep_batch, profile=2, similarity_kind=kind,
                       objective=rcd.RCD_OBJ_GRAPH_CUT if args.objective == "cut" else rcd.RCD_OBJ_FACILITY)
    ctx2.rcd_partition(Xd, yd, wl.capacities, wl.L, M_max=M)
    ctx2.sync_status()
    p2 = ctx2.profile()
    sweep_s = p2["sweep_ms"] * 1e-3
    if sweep_s > 0:
        a2 = p2["sweep_bytes"] / sweep_s / 1e9
        roofline["sweep_kernel_launches"] = {"achieved": a2, "frac": a2 / sweep_peak, "launches": int(p2["sweep_launches"]),
                                             "avg_launch_us": 1e3 * p2["sweep_ms"] / max(1, p2["sweep_launches"]),
                                             "bytes_per_launch": p2["sweep_bytes"] / max(1, p2["sweep_launches"])}
    # similarity GEMM: a dense contraction on the tensor cores.  Peak: this library's tensor-core peak loop for the
    # dtype, measured in this run (the cuBLAS bf16 figure of MEASURED_PEAKS.json is printed beside it).  It also has
    # to write 4*M^2 bytes per class, the tighter bound at d = 512.  Flops by the full-matrix convention 2*M^2*d per
    # class; the kernel computes only the 128 x 128 tiles on or above the diagonal (S is symmetric) and mirrors the
    # stores, so the flops it executes are given as well.
    sim_flops = 2.0 * wl.L * M * M * wl.d
    nt = (M + 127) // 128
    exec_flops = 2.0 * wl.L * (nt * (nt + 1) // 2) * 128 * 128 * wl.d
    sim_s = prof["similarity_ms"] * 1e-3
    tensor_peak = yard["mma_tflops"]
    sim_tflops = sim_flops / sim_s / 1e12 if sim_s > 0 else None
    exec_tflops = exec_flops / sim_s / 1e12 if sim_s > 0 else None
    sim_gbs = 4.0 * wl.L * M * M / sim_s / 1e9 if sim_s > 0 else None
    t_flops = exec_flops / (tensor_peak * 1e12)
    t_bytes = 4.0 * wl.L * M * M / (peaks["hbm_gbs"] * 1e9)
    similarity = {"ms": prof["similarity_ms"], "tensor_core_launches": int(prof["similarity_tc_launches"]),
                  "flops_convention": "full matrix 2*M^2*d per class; the kernel executes the tiles on or above the diagonal only",
                  "tflops": sim_tflops, "executed_tflops": exec_tflops, "tensor_peak_tflops": tensor_peak,
                  "frac_of_tensor_peak": sim_tflops / tensor_peak if sim_tflops else None,
                  "executed_frac_of_tensor_peak": exec_tflops / tensor_peak if exec_tflops else None,
                  "bytes_written_gbs": sim_gbs, "frac_of_hbm_peak": sim_gbs / peaks["hbm_gbs"] if sim_gbs else None,
                  "frac_of_bound": max(t_flops, t_bytes) / sim_s if sim_s > 0 else None,
                  "bound": "tensor" if t_flops >= t_bytes else "hbm-write",
                  "peak_source": "measured in this run: tcgen05 %s peak loop of this library (cuBLAS bf16 in MEASURED_PEAKS.json: %.0f TFLOP/s)"
                                 % (yard["mma_dtype"], peaks["bf16_tflops"])}

    result = {"metric": "samples partitioned/sec", "value": value, "unit": "samples/s", "n_gpus": world,
              "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
              "higher_is_better": True, "scaling": "strong" if by_classes else "weak", "vs_baseline": None,
              "dtype": "int64" if (wl.dtype == "int8" and args.similarity == "dot") else ("f32" if args.objective == "facility" else "f64"),
              "data": "synthetic",
              "config": {"workload": workload_name(args.config, wl),
                         "l2": ("inputs larger than L2 (S: %.0f MB in all, %.1f MB per class, re-read every sweep; L2 %.0f MB)"
                                if not fits_l2 else
                                "S of all classes (%.0f MB, %.1f MB per class) fits in L2 (%.0f MB): a buffer of twice the L2 size is written between timed steps")
                               % (s_bytes * 1e-6, 4e-6 * M * M, l2_bytes * 1e-6),
                         "sweep_batch_max": args.sweep_batch or 8, "similarity": args.similarity, "objective": args.objective,
                         "sharding": ("one dataset, classes sharded over the ranks by M^3, one all-gather of the assignment per step" if by_classes
                                      else "one dataset per rank, no collective")},
              "gain_evals_per_s": jobs * wl.L * M * (M + 1) / 2 * args.steps / (ms * 1e-3),
              "phases_ms": dict({k: prof[k] for k in ("group_ms", "similarity_ms", "greedy_ms", "total_ms")},
                                sweep_phases_ms=prof["persistent_sweep_ns"] * 1e-6, pick_phases_ms=prof["persistent_pick_ns"] * 1e-6,
                                async_lull_ms=prof["async_lull_ns"] * 1e-6, async_visits=int(prof["async_visits"]), async_attempts=int(prof["async_attempts"]),
                                lazy_sweeps=int(prof["lazy_sweeps"]), lazy_misses=int(prof["lazy_misses"]), lazy_rows=int(prof["lazy_rows"]),
                                lazy_rows_skipped=int(prof["lazy_rows_skipped"]),
                                incremental_updates=int(prof["incremental_updates"]), incremental_rows=int(prof["incremental_rows"]),
                                noted_picks=int(prof["noted_picks"]),
                                threshold_pass_ms=prof["threshold_pass_ns"] * 1e-6, threshold_pass_gb=prof["threshold_pass_bytes"] * 1e-9),
              "similarity": similarity,
              "e2e": {"value": e2e_value, "unit": "samples/s", "h2d_bytes_per_step": int(h2d),
                      "d2h_bytes_per_step": int(d2h), "wall_ms_per_step": e2e_wall_ms / args.steps},
              "gpu_launches": launches_per_step * args.steps,
              "clocks": clocks, "roofline": roofline}

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        base_wl = make_workload(args.config, L=args.classes or None)
        cores = min(os.cpu_count() or 1, base_wl.L)
        r = oracle_sample(base_wl, args.ref_picks, cores)
        result["cpu_baseline"] = {
            "value": r["value"], "unit": "samples/s", "cores": r["cores"], "kind": "oracle",
            "sample": "%d of %d classes (one thread each), similarity in full, first %d of %d picks; "
                      "oracle cost per pick is constant, time scaled by %d/%d (%.1f s measured)"
                      % (r["classes"], base_wl.L, r["picks"], r["M"], r["M"], r["picks"], r["wall_sampled_s"])}
    if rank == 0:
        print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="C2", choices=["C1", "C2", "C3", "C4", "C5"])
    ap.add_argument("--classes", type=int, default=0, help="fewer (or more) classes than the configuration names: a reduced copy for profiling")
    ap.add_argument("--sweep-batch", type=int, default=0, help="sweep_batch_max (0 = library default)")
    ap.add_argument("--similarity", default="dot", choices=["dot", "gaussian"], help="similarity of Section 4 item 2")
    ap.add_argument("--objective", default="facility", choices=["facility", "cut"], help="submodular function of Section 4 item 2")
    ap.add_argument("--greedy-path", type=int, default=0,
                    help="0 = chosen by the library, 1 = two launches per round, 2 = one launch with rounds, 3 = one launch, asynchronous classes, 4 = one CTA per class")
    ap.add_argument("--async-help-min", type=int, default=0, help="greedy path 3: row groups left before other classes' CTAs help (0 = default)")
    ap.add_argument("--async-group", type=int, default=0, help="greedy path 3: sweeps served together (0 = library default)")
    ap.add_argument("--sharding", default="replicas", choices=["replicas", "classes"],
                    help="with --gpus N: one dataset per rank (weak scaling), or one dataset with its classes sharded over the ranks (strong scaling)")
    ap.add_argument("--lazy-mode", type=int, default=0, help="1 = threshold passes skip rows below the blocks' floors (exact lazy evaluation), 0 = every pass reads every row")
    ap.add_argument("--incremental", type=int, default=0, help="in-place correction of stored gains: 0 = chosen by the library, 1 = on, 2 = off")
    ap.add_argument("--incremental-max", type=int, default=0, help="most raised columns a pick corrects in place (0 = library default)")
    ap.add_argument("--dense-ring", type=int, default=0, help="0 = dense passes stream through shared-memory rings where they fit, 2 = never")
    ap.add_argument("--lazy-from", type=int, default=0, help="members a block needs before rows are skipped (0 = library default)")
    ap.add_argument("--ref-picks", type=int, default=150, help="picks per class in the CPU-oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
