#!/usr/bin/env python
"""Benchmark of the STAND step (verify + N-gram update + draft) on synthetic workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5] [--impl ours|reference]

Prints ONE JSON line.  A step is one stand_step over one batch of logits [B, N, V].
The timed region runs K steps back to back on one stream over a ring of pre-generated
logit buffers that are resident in HBM (each step's input is far larger than L2 for the
headline workload; smaller workloads use a ring that is larger than L2).
"""
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

from paper_2506_04708_b200 import dist as sd, inputs  # noqa: E402

METRIC = "draft-tree nodes verified/sec at V=151,936 bf16"
UNIT = "nodes/s"
L2_BYTES = 126 * 2 ** 20


def describe(w):
    return (f"{w.name}: B={w.B} N={w.N} (depth {w.D}, <= {w.kb} children) V={w.V} "
            f"{'bf16' if w.dtype == inputs.DTYPE_BF16 else 'fp32'} T={w.T} orders 1-{w.order_max} top-{w.topk} "
            f"table {w.table_slots} slots")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while a region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.times, self.proc = index, [], [], None

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
            self.rows.append([x.strip() for x in line.split(",")])
            self.times.append(time.time())

    def sm_mhz_between(self, t0, t1):
        """Median SM clock of the samples taken in [t0, t1]; the nearest sample when none fell inside."""
        got, near, near_d = [], None, None
        for t, r in zip(list(self.times), list(self.rows)):
            try:
                mhz = float(r[0])
            except Exception:
                continue
            if t0 <= t <= t1:
                got.append(mhz)
            d = min(abs(t - t0), abs(t - t1))
            if near_d is None or d < near_d:
                near, near_d = mhz, d
        return statistics.median(got) if got else near

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.t.join(timeout=2)
        sm, mx, power, reasons = [], [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            try:
                power.append(float(r[2]))
            except Exception:
                pass
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "power_w": statistics.median(power) if power else None}


def physical_gpu_index(local):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


def pregrow(gpu, w, seed, torch):
    """Grows the table to about w.pregrow_contexts contexts with synthetic compressed rows."""
    if not w.pregrow_contexts:
        return 0
    block, fed = 500_000, 0
    for i in range(64):
        if gpu.stats()["inserts"] >= 0.97 * w.pregrow_contexts:
            break
        ctx, ids, probs = inputs.pregrow_records(w, seed + 1000 * i, block)
        gpu.ngram_update_bulk(torch.from_numpy(ctx), torch.from_numpy(ids), torch.from_numpy(probs))
        fed += block
    return gpu.stats()["inserts"]


def workload_of(args):
    """The named workload; --batch scales the number of sequences (for profiling a smaller case of the same kernels)."""
    w = inputs.WORKLOADS[args.workload]
    if args.batch:
        w = inputs.scaled(w, name=f"{w.name}@B={args.batch}", B=args.batch)
    return w


# DRAM bytes per row-pass launch from the ncu capture summarised in profiles/row_pass_kernel_cfg5_B64_ncu_full.md
# (dram__bytes_read.sum + dram__bytes_write.sum = 466.79 MB + 3.6 MB at B=64; traffic grows with the rows, so a
# launch over B sequences moves B/64 times that).  None for shapes that were not captured.
ROW_PASS_TRAFFIC_PER_SEQUENCE = {"cfg5": (466.79e6 + 3.6e6) / 64}


def quick_workload(name, args, dev, peaks):
    """A short closed-loop run of one of the other workloads: nodes/s and logits GB/s (device-timed, warm)."""
    import torch
    from paper_2506_04708_b200.binding import Stand
    w = inputs.WORKLOADS[name]
    parent = inputs.topology(w.N, w.D, w.kb)
    depth = inputs.node_depths(parent)
    esize = 2 if w.dtype == inputs.DTYPE_BF16 else 4
    step_bytes = w.B * w.N * w.V * esize
    ring_n = min(512, max(4, -(-3 * L2_BYTES // step_bytes)))
    steps = max(200, min(2000, int(0.25 / (step_bytes / 5e12 + 40e-6))))
    gpu = Stand(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, args.seed, min(w.table_slots, 1 << 22), parent, device=dev)
    prompt = 8
    streams = inputs.token_streams(w, args.seed, prompt + (ring_n + 4) * (w.D + 2))
    tail = np.ascontiguousarray(streams[:, prompt - w.order_max:prompt])
    gpu.reset_sequences(torch.from_numpy(tail), torch.full((w.B,), prompt, dtype=torch.int64))
    gen = inputs.DeviceLogits(w, streams, depth, args.seed, pool=2, device=dev, peak_mode=args.peak_mode)
    tdtype = torch.bfloat16 if w.dtype == inputs.DTYPE_BF16 else torch.float32
    ring = [torch.empty((w.B, w.N, w.V), dtype=tdtype, device=dev) for _ in range(ring_n)]
    lens = torch.empty(w.B, dtype=torch.int64, device=dev)
    for s in range(ring_n):
        gpu.lens_device(lens)
        gen.make(ring[s], lens, s)
        gpu.step(ring[s])
    for s in range(5):
        gpu.step(ring[s % ring_n])
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    for s in range(steps):
        gpu.step(ring[s % ring_n])
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / steps
    sev = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
    for e in sev:
        e.record()
    k1 = []
    for s in range(20):
        gpu.profile_stages(sev)
        gpu.step(ring[s % ring_n])
        torch.cuda.synchronize()
        k1.append(sev[0].elapsed_time(sev[1]))
    gpu.profile_stages(None)
    st = gpu.stats()
    gpu.close()
    k1_ms = statistics.median(k1)
    return {"workload": describe(w), "steps": steps, "ring_buffers": ring_n, "ms_per_step": ms,
            "nodes_per_s": w.B * w.N / (ms * 1e-3), "logits_gbs": step_bytes / (ms * 1e-3) / 1e9,
            "row_pass_us": k1_ms * 1e3, "row_pass_gbs": step_bytes / (k1_ms * 1e-3) / 1e9,
            "row_pass_frac_of_measured": step_bytes / (k1_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "drops": st["drops"]}


def p80_variant(gpu, w, args, dev, seed, buf=None, steps=200, warm=100):
    """The same step on logits whose planted token holds 70-90 % of its row's mass (peak mode p80), so that drafts
    are accepted, accepted paths are several nodes long and the table is hit: the regime the paper's tables
    report (2.6-3.7 tokens per step).  The table is warmed with the texts of the run first.  The logits are made again before every step (untimed) so that the peaks
    follow the sequences; each step is timed by its own pair of events.  `gpu`: a context whose table is kept
    (None: a fresh one); the sequences restart on fresh streams."""
    import torch
    from paper_2506_04708_b200.binding import Stand
    parent = inputs.topology(w.N, w.D, w.kb)
    depth = inputs.node_depths(parent)
    own = gpu is None
    if own:
        gpu = Stand(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, seed, min(w.table_slots, 1 << 22), parent, device=dev)
    prompt = 8
    streams = inputs.token_streams(w, seed + 1, prompt + (steps + warm + 4) * (w.D + 2))
    tail = np.ascontiguousarray(streams[:, prompt - w.order_max:prompt])
    gpu.reset_sequences(torch.from_numpy(tail), torch.full((w.B,), prompt, dtype=torch.int64))
    # the module has met these texts before (Sec. 5.1: it persists across trajectories): every distinct stream is fed
    # once as synthetic compressed rows, so that drafts are there to be accepted from the first step on
    for row in np.unique(streams, axis=0):
        ctx, ids, probs = inputs.records_from_corpus(w, row, seed + 1)
        gpu.ngram_update_bulk(torch.from_numpy(ctx), torch.from_numpy(ids), torch.from_numpy(probs))
    gen = inputs.DeviceLogits(w, streams, depth, seed + 1, pool=1, device=dev, peak_mode="p80")
    tdtype = torch.bfloat16 if w.dtype == inputs.DTYPE_BF16 else torch.float32
    if buf is None:
        buf = torch.empty((w.B, w.N, w.V), dtype=tdtype, device=dev)
    lens = torch.empty(w.B, dtype=torch.int64, device=dev)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    emitted0 = 0
    for s in range(warm + steps):
        if s == warm:
            emitted0 = gpu.stats()["emitted_tokens"]
        gpu.lens_device(lens)
        gen.make(buf, lens, s)
        if s >= warm:
            evs[s - warm][0].record()
        gpu.step(buf)
        if s >= warm:
            evs[s - warm][1].record()
    torch.cuda.synchronize()
    st = gpu.stats()
    ms = statistics.mean(a.elapsed_time(b) for a, b in evs)
    esize = 2 if w.dtype == inputs.DTYPE_BF16 else 4
    out = {"workload": describe(w), "peak_mode": "p80", "steps": steps, "warm_steps": warm, "ms_per_step": ms,
           "nodes_per_s": w.B * w.N / (ms * 1e-3), "logits_gbs": w.B * w.N * w.V * esize / (ms * 1e-3) / 1e9,
           "acceptance_length": (st["emitted_tokens"] - emitted0) / (steps * w.B), "lookup_hits": st["lookup_hits"],
           "drops": st["drops"], "timing": "one pair of events per step; logits made again between steps (untimed)"}
    del gen
    if own:
        gpu.close()
    return out


def run_ours(args, rank, world, local):
    import torch
    from paper_2506_04708_b200.binding import Stand

    w = workload_of(args)
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    dist = sd.init("nccl", dev)
    seed = sd.replica_seed(args.seed, rank)  # every rank runs its own sequences: independent replicas
    # --sharded: one N-gram module for the sequences of all ranks; the ranks share the seed of the method's random
    # numbers (counters tell the sequences apart) and start from the same table
    lib_seed = args.seed if args.sharded else seed
    parent = inputs.topology(w.N, w.D, w.kb)
    depth = inputs.node_depths(parent)
    esize = 2 if w.dtype == inputs.DTYPE_BF16 else 4
    step_bytes = w.B * w.N * w.V * esize
    ring_n = max(4, min(16, int(40e9 // step_bytes)))
    while ring_n * step_bytes < 3 * L2_BYTES:
        ring_n += 1
    ring_n = min(ring_n, 64)
    if args.ring:
        ring_n = args.ring

    gpu = Stand(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, lib_seed, w.table_slots, parent, device=dev,
                host_staging=True, deterministic=args.deterministic, seq_base=rank * w.B if args.sharded else 0)
    contexts = pregrow(gpu, w, lib_seed, torch)
    # The workload fixes the table's size (cfg5: about 10 M contexts in 16 M slots, 1,024 steps long).  The timed
    # region runs far more steps than that, each adding contexts, so the table is put back to this state whenever
    # it has grown by more than a workload's worth: otherwise the run drifts towards a full table (long probe
    # sequences, dropped updates), which is another workload.
    snapshot = gpu.table_snapshot() if w.pregrow_contexts else None
    growth_limit = max(1, w.pregrow_contexts // 8)

    def keep_table_at_size():
        if snapshot is not None and gpu.stats()["inserts"] - keep_table_at_size.base > growth_limit:
            gpu.table_restore(snapshot)
            keep_table_at_size.base = gpu.stats()["inserts"]
            keep_table_at_size.restores += 1
    keep_table_at_size.base = gpu.stats()["inserts"] if snapshot is not None else 0
    keep_table_at_size.restores = 0
    if args.sharded:
        from paper_2506_04708_b200 import sharded
        step_fn = sharded.ShardedStand(gpu, dist).step
    else:
        step_fn = gpu.step
    prompt = 8
    streams = inputs.token_streams(w, seed, prompt + (ring_n + 4) * (w.D + 2))
    tail = np.full((w.B, w.order_max), -1, np.int32)
    tail[:, :] = streams[:, prompt - w.order_max:prompt]
    gpu.reset_sequences(torch.from_numpy(tail), torch.full((w.B,), prompt, dtype=torch.int64))

    gen = inputs.DeviceLogits(w, streams, depth, seed, pool=2, device=dev, peak_mode=args.peak_mode)
    tdtype = torch.bfloat16 if w.dtype == inputs.DTYPE_BF16 else torch.float32
    ring = [torch.empty((w.B, w.N, w.V), dtype=tdtype, device=dev) for _ in range(ring_n)]
    lens = torch.empty(w.B, dtype=torch.int64, device=dev)
    # closed loop over the ring: every buffer gets its peaks at the positions its step predicts
    for s in range(ring_n):
        gpu.lens_device(lens)
        gen.make(ring[s], lens, s)
        step_fn(ring[s])
    del gen
    torch.cuda.empty_cache()
    for s in range(max(args.warmup, 3)):
        step_fn(ring[s % ring_n])
    torch.cuda.synchronize()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: K steps back to back, repeated until enough device time has been seen ------------
    # Every repeat is exactly K steps between a barrier + device synchronisation on both sides; the slowest
    # rank's time counts.  The line's value is the median repeat: seconds of back-to-back steps are what lets the
    # power limit (if this GPU reaches it) show in the clocks, which are recorded per repeat.
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    time.sleep(0.25)
    launches0 = gpu.launch_count()
    emitted0 = gpu.stats()["emitted_tokens"]
    repeats = []
    total_ms, steps_run = 0.0, 0
    torch.cuda.nvtx.range_push("stand_timed")  # lets a profiler keep to the timed region
    while True:
        keep_table_at_size()  # untimed
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t_host0 = time.time()
        ev0.record()
        for s in range(args.steps):
            step_fn(ring[s % ring_n])
        ev1.record()
        barrier()
        t_host1 = time.time()
        ms = sd.max_over_ranks(dist, ev0.elapsed_time(ev1), dev)
        repeats.append({"ms_total": ms, "t0": t_host0, "t1": t_host1})
        total_ms += ms
        steps_run += args.steps
        if total_ms >= args.min_seconds * 1e3 or len(repeats) >= args.max_repeats:
            break
    torch.cuda.nvtx.range_pop()
    launches = (gpu.launch_count() - launches0) // len(repeats)
    st = gpu.stats()
    accept_len = (st["emitted_tokens"] - emitted0) / (steps_run * w.B)
    ms_total = statistics.median(r["ms_total"] for r in repeats)

    keep_table_at_size()
    # ---- second pass: the row-pass kernel alone, timed by events around it -------------
    n_prof = 200
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_prof)]
    for a, b in evs:  # torch creates the CUDA event at the first record; the library re-records it
        a.record()
        b.record()
    for s in range(n_prof):
        gpu.profile_row_pass(*evs[s])
        step_fn(ring[s % ring_n])
    gpu.profile_row_pass(None, None)
    torch.cuda.synchronize()
    k1_ms = statistics.mean(a.elapsed_time(b) for a, b in evs)
    # the same steps with events at every stage boundary (diagnostic: where the rest of a step goes)
    n_st = 0 if args.sharded else 100  # the stage events belong to the fused step
    sev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(n_st)]
    for row in sev:
        for e in row:
            e.record()
    for s in range(n_st):
        gpu.profile_stages(sev[s])
        step_fn(ring[s % ring_n])
    gpu.profile_stages(None)
    torch.cuda.synchronize()
    stage_us = None if not sev else {name: 1e3 * statistics.mean(row[i].elapsed_time(row[i + 1]) for row in sev)
                                     for i, name in enumerate(("row_pass", "verify", "update", "draft"))}
    per_repeat = []
    for r in repeats:
        mhz = sampler.sm_mhz_between(r["t0"], r["t1"])
        per_repeat.append({"ms_per_step": r["ms_total"] / args.steps, "sm_mhz": mhz,
                           "ms_x_mhz": None if mhz is None else r["ms_total"] / args.steps * mhz})
    clocks = sampler.stop()
    shown = per_repeat if len(per_repeat) <= 32 else [per_repeat[i * (len(per_repeat) - 1) // 31] for i in range(32)]
    all_ms = [r["ms_per_step"] for r in per_repeat]
    timing = {"repeats": len(per_repeat), "steps_per_repeat": args.steps, "timed_seconds": sum(r["ms_total"] for r in repeats) / 1e3,
              "ms_per_step_median": statistics.median(all_ms), "ms_per_step_min": min(all_ms), "ms_per_step_max": max(all_ms),
              "per_repeat": shown, "value_is": "median repeat"}

    ms_per_step = ms_total / args.steps
    nodes_per_step = w.B * w.N * world
    value = sd.whole_job_rate(w.B * w.N, world, args.steps, ms_total)

    # ---- end to end through the C ABI with host buffers ---------------------------------
    # at least 8 steps and about a second (the copy runs at PCIe speed: ~50 GB/s)
    e2e_steps = max(8, min(4096, int(1.0 / (step_bytes / 50e9 + 2 * ms_per_step * 1e-3)) + 1))
    h_logits = torch.empty((w.B, w.N, w.V), dtype=tdtype).pin_memory()
    h_logits.copy_(ring[0])
    h_em = torch.empty((w.B, gpu.D + 1), dtype=torch.int32).pin_memory()
    h_ne = torch.empty(w.B, dtype=torch.int32).pin_memory()
    h_tr = torch.empty((w.B, w.N), dtype=torch.int32).pin_memory()
    def host_step():
        if not args.sharded:
            gpu.step_host(h_logits, h_em, h_ne, h_tr)
            return
        ring[0].copy_(h_logits, non_blocking=True)
        step_fn(ring[0])
        h_em.copy_(gpu.emitted, non_blocking=True)
        h_ne.copy_(gpu.n_emitted, non_blocking=True)
        h_tr.copy_(gpu.tree, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    host_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        host_step()
    barrier()
    e2e_s = time.perf_counter() - t0
    e2e_s = sd.max_over_ranks(dist, e2e_s, dev)
    e2e = {"value": nodes_per_step * e2e_steps / e2e_s, "unit": UNIT, "steps": e2e_steps, "seconds": e2e_s,
           "h2d_bytes_per_step": step_bytes, "d2h_bytes_per_step": (h_em.numel() + h_ne.numel() + h_tr.numel()) * 4}

    peaks, peak_kind = measured_peaks()
    alg_bytes = w.B * w.N * w.V * esize  # every logit is read once; everything else is < 1%
    achieved = alg_bytes / (k1_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "row_pass_kernel", "achieved": achieved, "peak": peaks["hbm_gbs"],
                "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "peak_kind": peak_kind + " copy bandwidth",
                "traffic": None, "kernel_ms": k1_ms, "frac_of_nominal_8TBs": achieved / 8000.0,
                "step_frac": alg_bytes / (ms_per_step * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    if args.workload in ROW_PASS_TRAFFIC_PER_SEQUENCE:
        roofline["traffic"] = ROW_PASS_TRAFFIC_PER_SEQUENCE[args.workload] * w.B
        roofline["traffic_source"] = "ncu capture at B=64 scaled by rows (profiles/row_pass_kernel_cfg5_B64_ncu_full.md)"
    roofline["algorithmic_bytes"] = alg_bytes

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = time_oracle(w, ring[0], args, total_budget_s=12.0, single_thread=True)

    others, p80 = None, None
    if rank == 0 and world == 1 and not args.no_sweep and not args.sharded:
        # the named workload and cfg3 once more in peak mode p80 (deep accepted paths, table hits): labelled, secondary
        if snapshot is not None:
            gpu.table_restore(snapshot)
        p80 = {args.workload: p80_variant(gpu, w, args, dev, seed, buf=ring[0])}
    if rank == 0 and world == 1 and not args.no_sweep:
        # the other four workloads, briefly (secondary figures; the line's value is the named workload's)
        del ring, h_logits
        torch.cuda.empty_cache()
        if p80 is not None and args.workload != "cfg3":
            p80["cfg3"] = p80_variant(None, inputs.WORKLOADS["cfg3"], args, dev, args.seed)
            torch.cuda.empty_cache()
        others = {}
        for name in sorted(inputs.WORKLOADS):
            if name != args.workload:
                others[name] = quick_workload(name, args, dev, peaks)
                torch.cuda.empty_cache()

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3) + ring_n, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": describe(w), "peak_mode": args.peak_mode, "ring_buffers": ring_n,
                       "drafting": "deterministic" if args.deterministic else "stochastic (Gumbel-Top-K)",
                       "l2": f"inputs larger than L2: {step_bytes / 1e6:.0f} MB per step, ring of {ring_n} "
                             f"buffers = {ring_n * step_bytes / 1e9:.2f} GB",
                       "table_contexts_at_start": int(contexts), "table_restores": keep_table_at_size.restores, "multi_gpu": ("sequences sharded over the GPUs, one N-gram module: accepted rows all-gathered every step"
                                     if args.sharded else "independent replicas per GPU" if world > 1 else "single GPU"), "acceptance_length": accept_len},
            "clocks": clocks, "timing": timing, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "logits_gbs": alg_bytes * world / (ms_per_step * 1e-3) / 1e9,
            "stage_us": stage_us,
            "table": {"drops": st["drops"], "max_probe": st["max_probe_seen"], "lookup_hits": st["lookup_hits"],
                      "lookups": st["lookups"]},
        }
        if cpu_baseline is not None:
            line["cpu_baseline"] = cpu_baseline
        if others is not None:
            line["other_workloads"] = others
        if p80 is not None:
            line["p80_variant"] = p80
        print(json.dumps(line))
    gpu.close()
    if dist is not None:
        dist.destroy_process_group()


def _oracle_inputs(w, ws, ring0, args, parent):
    if ring0 is not None:
        import torch
        a = ring0[:ws.B].contiguous().cpu()
        return a.view(torch.int16).numpy().view(np.uint16) if w.dtype == inputs.DTYPE_BF16 else a.numpy()
    streams = inputs.token_streams(ws, args.seed, 64)
    return inputs.logits_numpy(ws, streams, np.full(ws.B, 8), inputs.node_depths(parent), 0, args.seed, args.peak_mode)


def _oracle_run(w, ws, logits, args, parent, n, warmup):
    from oracle import stand_oracle as so
    orc = so.Oracle(ws.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, args.seed, parent)
    orc.reset_sequences(np.full((ws.B, w.order_max), 5, np.int32), np.full(ws.B, 8, np.int64))
    for _ in range(warmup):
        orc.step(logits)
    t0 = time.perf_counter()
    for _ in range(n):
        orc.step(logits)
    dt = time.perf_counter() - t0
    orc.take_margins()
    orc.close()
    return dt


def time_oracle(w, ring0, args, total_budget_s, steps=None, warmup=0, single_thread=False):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: the first B_s sequences,
    B_s chosen so that the whole run takes about total_budget_s on this machine's cores."""
    cores = os.cpu_count() or 1
    parent = inputs.topology(w.N, w.D, w.kb)
    one = inputs.scaled(w, B=1)
    t1 = _oracle_run(w, one, _oracle_inputs(w, one, ring0, args, parent), args, parent, 1, 0)  # one sequence, one step
    if steps is None:
        b = min(w.B, 2 * cores)
        n = max(2, min(64, int(total_budget_s / (t1 * max(1.0, b / cores)))))
    else:
        n = steps
        per_step = total_budget_s / max(1, steps + warmup)
        b = max(1, min(w.B, int(per_step / t1) * cores if per_step >= t1 else 1))
    ws = inputs.scaled(w, B=b)
    dt = _oracle_run(w, ws, _oracle_inputs(w, ws, ring0, args, parent), args, parent, n, warmup)
    out = {"value": ws.B * w.N * n / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"{n} steps of the first {ws.B} of {w.B} sequences ({ws.B * w.N} rows x V={w.V} per step), "
                     f"table not pre-grown, OpenMP over sequences", "ms_per_step": dt / n * 1e3, "steps": n}
    if single_thread:
        # the same oracle on one thread: a few steps of one sequence (one sequence is one unit of its parallel loop)
        n1 = max(2, min(16, int(0.25 * total_budget_s / t1)))
        dt1 = _oracle_run(w, one, _oracle_inputs(w, one, ring0, args, parent), args, parent, n1, 0)
        out["single_thread"] = {"value": w.N * n1 / dt1, "unit": UNIT, "cores": 1,
                                "sample": f"{n1} steps of the first sequence ({w.N} rows x V={w.V} per step)"}
    return out


def run_reference(args, rank, world):
    """The oracle as it stands, on the host cores: the reference arm."""
    if rank != 0:
        return
    w = workload_of(args)
    r = time_oracle(w, None, args, total_budget_s=90.0, steps=args.steps, warmup=args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": describe(w), "peak_mode": args.peak_mode, "sample": r["sample"]},
            "cpu_baseline": {"value": r["value"], "unit": UNIT, "cores": r["cores"], "kind": "oracle",
                             "sample": r["sample"]},
            "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def spawn_ranks(n):
    """`python bench.py --gpus N` outside a launcher: start N ranks of this same command (one process per GPU,
    rendezvous on 127.0.0.1) and pass their output through.  NCCL's communicator set-up is logged to stderr."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.run(cmd, env=env).returncode


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--peak-mode", default="add8", choices=["add8", "p80"])
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--deterministic", action="store_true", help="deterministic drafting (paper Sec. 3.2) instead of stochastic")
    ap.add_argument("--sharded", action="store_true",
                    help="one N-gram module shared by the sequences of all ranks (accepted rows exchanged every step) "
                         "instead of independent replicas")
    ap.add_argument("--no-sweep", action="store_true", help="skip the short runs of the other four workloads")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's number of sequences (profiling)")
    ap.add_argument("--ring", type=int, default=0, help="override the number of logit buffers in the ring (profiling)")
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="repeat the K-step timed region until this much device time has been measured")
    ap.add_argument("--max-repeats", type=int, default=400)
    args = ap.parse_args()
    if args.gpus > 1 and "RANK" not in os.environ and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus))
    rank, world, local = sd.env_ranks()
    if args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world, local)


if __name__ == "__main__":
    main()
