#!/usr/bin/env python
"""Benchmark of the partial causal prefill attention path on B200.

A step is one pass of the whole path over one synthetic long request: host plan, one partial
attention launch per zigzag KV partition, LSE merge of the partials (n-way per group of resident
partials), final output in the input dtype.
Prints one JSON line (see --help for the knobs).  `--impl reference` times the fp64 CPU oracle
on a bounded sample of the same workload instead.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2409_15104_b200 import workloads

METRIC = "causal prefill attention TFLOP/s (tokens/s and % of dense BF16 peak alongside), 1 B200"
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
KERNEL_SOURCES = ("pec_attn_prefill_bf16.cu", "pec_sm100.cuh", "pec_tile.cuh")


def kernel_source_hash():
    """First 16 hex digits of the SHA-256 over the attention kernel's sources: ties a stored profiler
    counter to the kernel revision it was taken on."""
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        h.update(open(os.path.join(ROOT, "paper_2409_15104_b200", "csrc", name), "rb").read())
    return h.hexdigest()[:16]


def stored_counters(workload):
    """Profiler counters of one attention launch of `workload`, read from profiles/attn_counters.txt (taken
    offline with ncu, never in this run).  Returns None when there is no line for the workload, and marks the
    record stale - traffic null - when the kernel sources have changed since the capture."""
    path = os.path.join(ROOT, "profiles", "attn_counters.txt")
    if not os.path.exists(path):
        return None
    for ln in open(path):
        f = ln.split()
        if len(f) >= 6 and not ln.startswith("#") and f[0] == workload:
            rec = {"captured_offline": True, "kernel_source_hash_at_capture": f[1], "dram_bytes_per_launch": float(f[2]),
                   "tensor_pipe_active_pct": float(f[3]), "xu_pipe_pct": float(f[4]), "ms_per_launch_under_ncu": float(f[5]),
                   "note": " ".join(f[6:])}
            rec["stale"] = rec["kernel_source_hash_at_capture"] != kernel_source_hash()
            return rec
    return None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"bf16_burst": d["bf16_tflops"], "bf16_sustained": d["bf16_tflops_sustained"],
                "hbm": d["hbm_gbs"], "source": "measured"}
    return {"bf16_burst": 1590.0, "bf16_sustained": 1400.0, "hbm": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(pw),
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- CPU oracle legs
def oracle_sample(wl, q, k, v, target_s=15.0):
    """Times the fp64 oracle, as it stands, on sampled query rows (all heads) of the workload."""
    import oracle
    S = wl.seq_len
    g = np.random.Generator(np.random.Philox(key=wl.seed))
    probe = sorted(int(x) for x in g.integers(0, S, size=4))
    t0 = time.perf_counter()
    oracle.prefill_attn(q, k, v, seq_len=S, rows=probe)
    t_probe = time.perf_counter() - t0
    n = int(max(4, min(4096, target_s / max(t_probe / len(probe), 1e-6))))
    rows = sorted(int(x) for x in g.integers(0, S, size=n))
    t0 = time.perf_counter()
    oracle.prefill_attn(q, k, v, seq_len=S, rows=rows)
    dt = time.perf_counter() - t0
    pairs = sum(r + 1 for r in rows)
    flops = workloads.attention_flops(pairs, wl.hq)
    return {"seconds": dt, "rows": n, "pairs_per_head": pairs, "tflops": flops / dt / 1e12,
            "tokens_per_s_extrapolated": S / (dt * workloads.causal_pairs(S) / pairs),
            "cores": oracle.oracle_threads()}


def run_reference(args, wl):
    """--impl reference: the oracle on the host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    q, k, v = workloads.qkv(wl.seed, wl.seq_len, wl.hq, wl.hkv, 128, wl.dtype)
    per_step = args.reference_seconds or max(0.15, min(20.0, 90.0 / (args.steps + args.warmup)))   # ~90 s in all
    for _ in range(args.warmup):
        oracle_sample(wl, q, k, v, target_s=per_step)
    res = [oracle_sample(wl, q, k, v, target_s=per_step) for _ in range(args.steps)]
    tflops = sum(r["tflops"] for r in res) / len(res)
    ms = 1e3 * sum(r["seconds"] for r in res) / len(res)
    sample = (f"{res[0]['rows']} seeded random query rows x all {wl.hq} heads per step, full fp64 definition per row; "
              f"tokens/s extrapolated by pair count: {res[0]['tokens_per_s_extrapolated']:.3f}")
    line = {
        "impl": "reference", "metric": METRIC, "value": tflops, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl),
        "cpu_baseline": {"value": tflops, "unit": "TFLOP/s", "cores": res[0]["cores"], "kind": "oracle", "sample": sample},
        "e2e": {"value": tflops, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def workload_config(wl):
    return {"workload": f"{wl.name}: {wl.note}", "seq_len": wl.seq_len, "hq": wl.hq, "hkv": wl.hkv, "head_dim": 128,
            "num_parts": wl.num_parts, "part_align": wl.part_align, "seed": wl.seed,
            "l2": "inputs and partials exceed the 126 MB L2; no explicit flush",
            "flops": "4*D*Hq*(exact causal pairs), attention only, single layer"}


# ----------------------------------------------------------------------------- multi-rank plumbing
def replica_seed(wl, rank):
    """Replicas only: rank r runs the same single-GPU workload on its own seeded request."""
    return wl.seed + 1000 * rank


def max_over_ranks(values, dist, device):
    """Element-wise maximum of per-rank timings (every rank gets the result)."""
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_tflops(flops_per_replica_step, world, ms_per_step):
    """All replicas' work over the slowest rank's time."""
    return world * flops_per_replica_step / (ms_per_step * 1e-3) / 1e12


# ----------------------------------------------------------------------------- GPU arm
def run_ours(args, wl):
    from paper_2409_15104_b200 import binding
    from paper_2409_15104_b200.prefill import PartitionedPrefill
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    binding.load()

    # The extra records come first: they are short workloads, and measured after the headline's half minute at the
    # power cap they would be measured on a hot, clock-limited chip rather than as they run on their own.
    extra = None
    if world == 1 and not args.no_extra and not args.profile:
        extra = {}
        for name, fn in (("c3", extra_partitioned), ("c3_merge_kernel", extra_merge_kernel), ("c4", run_preempted),
                         ("c2", run_short_batch), ("ring", run_ring), ("decode", run_decode), ("linear", run_linear),
                         ("linear_merged", run_linear_merged), ("layer", run_layer)):
            try:
                extra[name] = fn(args)
            except Exception as exc:                       # an extra record must not take the headline with it
                extra[name] = {"error": f"{type(exc).__name__}: {exc}"}
            torch.cuda.empty_cache()

    # Replicas only: every rank runs the same single-GPU workload on its own seeded request.
    seed = replica_seed(wl, rank)
    q_h, k_h, v_h = workloads.qkv(seed, wl.seq_len, wl.hq, wl.hkv, 128, wl.dtype)
    q_h, k_h, v_h = q_h.pin_memory(), k_h.pin_memory(), v_h.pin_memory()
    q, k, v = q_h.to(dev), k_h.to(dev), v_h.to(dev)
    runner = PartitionedPrefill(wl.seq_len, wl.hq, wl.num_parts, wl.dtype, dev, wl.part_align)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        runner.run(q, k, v)
    binding.check_status()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    # Per-launch CUDA events keep a launch from starting on the SMs its predecessor has left.  On launches of tens
    # of milliseconds that overlap is worth nothing, so the events sit inside the timed region; on the short
    # launches of a 32K request it is part of the path, so the K timed steps run without events and the kernel's
    # own time is taken from a few more steps right after them.
    events_inside = wl.seq_len >= 131072
    runner.attn_events, runner.merge_events = [], []
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for _ in range(args.steps):
        runner.run(q, k, v, time_kernels=events_inside)
    t1.record(stream)
    barrier()
    total_ms = t0.elapsed_time(t1)
    if not events_inside:
        for _ in range(max(1, min(args.steps, 3))):
            runner.run(q, k, v, time_kernels=True)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    binding.check_status()
    attn_ms = [a.elapsed_time(b) for a, b in runner.attn_events]
    launches_per_step = runner.launches_per_step()

    if args.profile:
        if rank == 0:
            fl = workloads.attention_flops(workloads.causal_pairs(wl.seq_len), wl.hq)
            print(json.dumps({"profile_run": True, "ms_per_step": total_ms / args.steps,
                              "attn_ms_per_launch": sum(attn_ms) / len(attn_ms),
                              "attn_tflops": fl / wl.num_parts / (sum(attn_ms) / len(attn_ms)) / 1e9,
                              "clocks": clocks}), flush=True)
        if dist is not None:
            dist.destroy_process_group()
        return

    # End to end through the public call sequence with host buffers: every step copies its Q, K, V from pinned
    # host memory, runs the path and copies O and LSE back.  Consecutive steps are pipelined (StreamedPrefill:
    # the copies of neighbouring steps overlap the compute of the current one); the same steps issued one
    # after the other on one stream are timed too and reported beside it.
    from paper_2409_15104_b200.prefill import StreamedPrefill
    o_h = torch.empty((wl.seq_len, wl.hq, 128), dtype=wl.dtype).pin_memory()
    l_h = torch.empty((wl.seq_len, wl.hq), dtype=torch.float32).pin_memory()
    qd, kd, vd = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)

    def serial_step():
        qd.copy_(q_h, non_blocking=True); kd.copy_(k_h, non_blocking=True); vd.copy_(v_h, non_blocking=True)
        o, l = runner.run(qd, kd, vd)
        o_h.copy_(o, non_blocking=True); l_h.copy_(l, non_blocking=True)

    serial_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    serial_steps = max(1, min(args.steps, 3 if wl.seq_len <= 65536 else 1))
    e0.record(stream)
    for _ in range(serial_steps):
        serial_step()
    e1.record(stream)
    barrier()
    serial_ms = e0.elapsed_time(e1) / serial_steps
    del qd, kd, vd

    pipe = StreamedPrefill(runner, wl.hkv, dev)
    pipe.submit(q_h, k_h, v_h, o_h, l_h)
    pipe.drain()
    barrier()
    e2e_steps = max(1, min(args.steps, 20 if wl.seq_len <= 65536 else 8))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(pipe.s_in)                                       # nothing is in flight: first operation of the region
    for _ in range(e2e_steps):
        pipe.submit(q_h, k_h, v_h, o_h, l_h)
    e1.record(pipe.s_out)                                      # after the last step's device-to-host copies
    pipe.drain()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    binding.check_status()

    total_ms, e2e_ms, serial_ms = max_over_ranks([total_ms, e2e_ms, serial_ms], dist, dev)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    pairs = workloads.causal_pairs(wl.seq_len)
    flops_step = workloads.attention_flops(pairs, wl.hq)
    ms_step = total_ms / args.steps
    tflops = whole_job_tflops(flops_step, world, ms_step)
    attn_avg_ms = sum(attn_ms) / len(attn_ms)
    flops_launch = flops_step / wl.num_parts          # zigzag partitions carry equal pair counts
    attn_tflops = flops_launch / (attn_avg_ms * 1e-3) / 1e12
    h2d = q_h.numel() * q_h.element_size() + 2 * k_h.numel() * k_h.element_size()
    d2h = o_h.numel() * o_h.element_size() + l_h.numel() * 4
    del runner, pipe, q, k, v, o_h, l_h
    torch.cuda.empty_cache()

    # Which measured cuBLAS rate the attention kernel is held against follows from the run itself: a timed
    # region of seconds sits at the power cap like the sustained GEMM loop, a shorter one runs at burst clocks.
    timed_s = total_ms * 1e-3
    kind = "sustained" if timed_s >= 2.0 else "burst"
    peak = peaks["bf16_sustained"] if kind == "sustained" else peaks["bf16_burst"]
    counters = stored_counters(wl.name)
    traffic = None if (counters is None or counters["stale"]) else counters["dram_bytes_per_launch"]
    sm_mhz = (clocks or {}).get("sm_mhz")
    roofline = {"bound": "tensor", "kernel": "attn_prefill_bf16_kernel", "achieved": attn_tflops, "peak": peak,
                "unit": "TFLOP/s", "frac": attn_tflops / peak, "traffic": traffic,
                "traffic_unit": "bytes per launch (ncu dram read + write, captured offline)",
                "peak_source": f"{peaks['source']} cuBLAS bf16, {kind} figure (timed region {timed_s:.2f} s)",
                "frac_of_sustained": attn_tflops / peaks["bf16_sustained"], "frac_of_burst": attn_tflops / peaks["bf16_burst"],
                "frac_of_nominal": attn_tflops / NOMINAL_BF16_TFLOPS,
                "flops_per_launch": flops_launch, "ms_per_launch": attn_avg_ms,
                "launch_events": "inside the timed region" if events_inside else "on 3 further steps right after the timed region (events between launches would keep them from overlapping)",
                "ms_per_launch_x_sm_mhz": attn_avg_ms * sm_mhz if sm_mhz else None,
                "launches_timed": len(attn_ms), "ncu": counters}

    cpu = oracle_sample(wl, q_h, k_h, v_h, target_s=15.0)
    line = {
        "metric": METRIC, "value": tflops, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if wl.dtype == torch.bfloat16 else "f32", "data": "synthetic",
        "config": workload_config(wl),
        "tokens_per_s": world * wl.seq_len / (ms_step * 1e-3),
        "frac_of_nominal_bf16_peak": tflops / world / NOMINAL_BF16_TFLOPS,
        "frac_of_measured_bf16_sustained": tflops / world / peaks["bf16_sustained"],
        "attention_only_tflops": attn_tflops,
        "roofline": roofline,
        "cpu_baseline": {"value": cpu["tflops"], "unit": "TFLOP/s", "cores": cpu["cores"], "kind": "oracle",
                         "sample": f"{cpu['rows']} seeded random query rows x {wl.hq} heads of the same request, "
                                   f"{cpu['seconds']:.1f} s; tokens/s extrapolated by pair count: "
                                   f"{cpu['tokens_per_s_extrapolated']:.3f}"},
        "e2e": {"value": whole_job_tflops(flops_step, world, e2e_ms), "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "how": "consecutive steps pipelined on three streams: every step's H2D, compute and D2H are inside the "
                       "timed region; copies of neighbouring steps overlap the compute",
                "one_step_at_a_time": {"value": whole_job_tflops(flops_step, world, serial_ms), "ms_per_step": serial_ms}},
        "gpu_launches": args.steps * launches_per_step,
        "clocks": clocks,
        "extra": extra,
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def _extra_steps(args, cap):
    return max(3, min(args.steps, cap))


def extra_partitioned(args, name="c3"):
    """Extra record: the whole partitioned step of another long configuration (every partition's launch merging
    into the running state), a few steps, with the attention launches timed one by one."""
    from paper_2409_15104_b200 import binding
    from paper_2409_15104_b200.prefill import PartitionedPrefill
    wl = workloads.WORKLOADS[name]
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    q, k, v = (t.to(dev) for t in workloads.qkv(wl.seed, wl.seq_len, wl.hq, wl.hkv, 128, wl.dtype))
    runner = PartitionedPrefill(wl.seq_len, wl.hq, wl.num_parts, wl.dtype, dev, wl.part_align)
    for _ in range(max(args.warmup, 3)):
        runner.run(q, k, v)
    torch.cuda.synchronize()
    steps = _extra_steps(args, 20)
    sampler = ClockSampler(0); sampler.start(); time.sleep(0.2)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        runner.run(q, k, v)
    e1.record()
    torch.cuda.synchronize()
    runner.attn_events = []
    for _ in range(3):                                       # per-launch times: events around every launch, no overlap
        runner.run(q, k, v, time_kernels=True)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    binding.check_status()
    ms = e0.elapsed_time(e1) / steps
    attn_ms = [a.elapsed_time(b) for a, b in runner.attn_events]
    fl = workloads.attention_flops(workloads.causal_pairs(wl.seq_len), wl.hq)
    peaks = load_peaks()
    attn_tf = fl / wl.num_parts / (sum(attn_ms) / len(attn_ms) * 1e-3) / 1e12
    counters = stored_counters(wl.name)
    return {"metric": "whole partitioned step, TFLOP/s (extra record)", "value": fl / (ms * 1e-3) / 1e12, "unit": "TFLOP/s",
            "ms_per_step": ms, "steps": steps, "tokens_per_s": wl.seq_len / (ms * 1e-3),
            "attention_only_tflops": attn_tf, "attention_ms_per_launch": sum(attn_ms) / len(attn_ms),
            "frac_of_burst": attn_tf / peaks["bf16_burst"], "frac_of_sustained": attn_tf / peaks["bf16_sustained"],
            "frac_of_nominal": attn_tf / NOMINAL_BF16_TFLOPS,
            "traffic": None if (counters is None or counters["stale"]) else counters["dram_bytes_per_launch"], "ncu": counters,
            "launches_per_step": runner.launches_per_step(), "clocks": clocks, "config": workload_config(wl)}


def merge_bytes_exact(seq_len, hq, bounds, parts, final_bf16):
    """DRAM bytes one n-way merge launch must move: part p holds keys from bounds[p] on, so under the causal
    mask its rows below bounds[p] are empty and the kernel reads only their LSE; every other (row, head) of a
    part costs 128 fp32 + the LSE, and every (row, head) is written once."""
    total = 0
    for p in parts:
        live = seq_len - bounds[p]
        total += hq * (live * 516 + (seq_len - live) * 4)
    total += seq_len * hq * ((256 if final_bf16 else 512) + 4)
    return total


def extra_merge_kernel(args, name="c3"):
    """Extra record: the n-way LSE merge kernel alone (the path two GPUs' partial outputs take), on the fp32
    partials of every zigzag partition of c3, HBM-bound, with the exact byte count from the plan."""
    from paper_2409_15104_b200 import binding
    wl = workloads.WORKLOADS[name]
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    q, k, v = (t.to(dev) for t in workloads.qkv(wl.seed, wl.seq_len, wl.hq, wl.hkv, 128, wl.dtype))
    P, S = wl.num_parts, wl.seq_len
    parts = [binding.pec_prefill_attn(q, k, v, part_id=p, num_parts=P, part_align=wl.part_align) for p in range(P)]
    out_o = torch.empty((S, wl.hq, 128), dtype=wl.dtype, device=dev)
    out_l = torch.empty((S, wl.hq), dtype=torch.float32, device=dev)
    o_parts, l_parts = [x[0] for x in parts], [x[1] for x in parts]
    for _ in range(3):
        binding.pec_attn_merge_n(o_parts, l_parts, o_out=out_o, lse_out=out_l)
    torch.cuda.synchronize()
    steps = _extra_steps(args, 20)
    evs = []
    for _ in range(steps):                                   # 4.3 GB of partials: far beyond the L2
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); binding.pec_attn_merge_n(o_parts, l_parts, o_out=out_o, lse_out=out_l); e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    binding.check_status()
    ms = statistics.median(a.elapsed_time(b) for a, b in evs)
    bounds = binding.pec_plan_partitions(S, P, 0, wl.part_align, 128, 128, True, tiles=False)["bounds"]
    byts = merge_bytes_exact(S, wl.hq, bounds, range(P), wl.dtype == torch.bfloat16)
    gbs = byts / (ms * 1e-3) / 1e9
    peaks = load_peaks()
    # The two-way kernel (pec_attn_merge) on the same partials: the running merge of part 0's state with parts 1..P-1 in
    # place, P - 1 launches; bytes per launch: state read, part read and state written for the part's live rows, the LSE alone for its empty rows.
    acc_o, acc_l = o_parts[0].clone(), l_parts[0].clone()
    def running():
        for pp in range(1, P):
            binding.pec_attn_merge(acc_o, acc_l, o_parts[pp], l_parts[pp], inplace=True)
    running()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps2 = max(1, steps // 4)
    e0.record()
    for _ in range(reps2):
        running()
    e1.record()
    torch.cuda.synchronize()
    binding.check_status()
    ms2 = e0.elapsed_time(e1) / (reps2 * (P - 1))
    byts2 = sum(wl.hq * ((S - bounds[pp]) * 3 * 516 + bounds[pp] * 8) for pp in range(1, P)) / (P - 1)   # rows the part is empty for: the two LSEs
    return {"metric": "n-way LSE merge kernel, achieved HBM GB/s (extra record)", "value": gbs, "unit": "GB/s", "ms_per_launch": ms,
            "steps": steps, "parts": P,
            "two_way_kernel": {"ms_per_launch": ms2, "gbs": byts2 / (ms2 * 1e-3) / 1e9, "frac": byts2 / (ms2 * 1e-3) / 1e9 / peaks["hbm"],
                               "algorithmic_bytes_per_launch": byts2, "launches": reps2 * (P - 1),
                               "what": "running in-place fp32 merge of the state with parts 1..P-1 (pec_attn_merge)"},
            "roofline": {"bound": "hbm", "kernel": "merge_n_kernel", "achieved": gbs, "peak": peaks["hbm"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm"], "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS, "traffic": None,
                         "algorithmic_bytes": byts, "peak_source": peaks["source"] + " copy bandwidth",
                         "bytes": "exact: rows of a part below its first key are empty and only their LSE is read"},
            "config": {"workload": f"{wl.name}: {P}-way merge of the partitions' fp32 partials into the bf16 output",
                       "l2": "partials (4.3 GB) exceed the L2"}}


def run_decode(args):
    """Extra line (not the headline): split-KV decode of one long request's new token, HBM-bound."""
    from paper_2409_15104_b200 import binding
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    L, hq, hkv = 262144, 64, 8
    seed = workloads.BASE_SEED + 6
    k = workloads.normal_tensor(seed, 2, (L, hkv, 128), torch.bfloat16).to(dev)
    v = workloads.normal_tensor(seed, 3, (L, hkv, 128), torch.bfloat16).to(dev)
    q = workloads.normal_tensor(seed, 1, (hq, 128), torch.bfloat16).to(dev)
    o = torch.empty((hq, 128), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((hq,), dtype=torch.float32, device=dev)
    a = binding.decode_args(q, k, v, o, lse, 0, L)
    ws = torch.empty(max(binding.pec_decode_workspace_size(a), 16), dtype=torch.uint8, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)           # > L2: K/V of one call are 1 GiB anyway
    for _ in range(max(args.warmup, 3)):
        binding.pec_decode_attn(q, k, v, o=o, lse=lse, workspace=ws)
    torch.cuda.synchronize()
    steps = _extra_steps(args, 50)
    evs = []
    for _ in range(steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); binding.pec_decode_attn(q, k, v, o=o, lse=lse, workspace=ws); e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    binding.check_status()
    ms = statistics.median(a_.elapsed_time(b_) for a_, b_ in evs)
    peaks = load_peaks()
    byts = 2 * L * hkv * 128 * 2
    gbs = byts / (ms * 1e-3) / 1e9
    # The same calls one after the other, as a decode loop issues them (the 1 GiB of K/V exceeds the L2 eight times
    # over, so nothing of a call's keys is left for the next): launch latencies then overlap the previous call.
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        binding.pec_decode_attn(q, k, v, o=o, lse=lse, workspace=ws)
    e1.record()
    torch.cuda.synchronize()
    binding.check_status()
    ms_b2b = e0.elapsed_time(e1) / steps
    import oracle
    want = oracle.attn_rows(q.cpu()[None], [L - 1], k.cpu(), v.cpu(), [(0, L)], False)
    err = float(np.abs(o.float().cpu().double().numpy() - want[0][0]).max())
    return {"metric": "split-KV decode attention, achieved HBM GB/s (extra line, not the headline)",
                      "value": gbs, "unit": "GB/s", "ms_per_step": ms, "steps": steps, "n_gpus": 1, "dtype": "bf16",
                      "data": "synthetic", "config": {"workload": f"decode: one token, {hq}/{hkv} heads, {L} cached keys",
                                                       "l2": "256 MiB written between timed calls"},
                      "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm"], "unit": "GB/s",
                                   "frac": gbs / peaks["hbm"], "traffic": None,
                                   "algorithmic_bytes": byts, "peak_source": peaks["source"] + " copy bandwidth"},
                      "back_to_back": {"ms_per_call": ms_b2b, "gbs": byts / (ms_b2b * 1e-3) / 1e9,
                                       "frac": byts / (ms_b2b * 1e-3) / 1e9 / peaks["hbm"],
                                       "l2": "no flush: one call's K/V are 1 GiB"},
                      "max_abs_err_vs_oracle": err}


def _gemm_roofline(tf, timed_ms, peaks, traffic=None):
    """Tensor roofline of a GEMM record: against the burst cuBLAS rate when the timed region was short, the sustained one
    when it lasted seconds (the rule of the headline line); both fractions are printed."""
    kind = "sustained" if timed_ms >= 2000.0 else "burst"
    peak = peaks["bf16_sustained"] if kind == "sustained" else peaks["bf16_burst"]
    return {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak, "traffic": traffic,
            "frac_of_sustained": tf / peaks["bf16_sustained"], "frac_of_burst": tf / peaks["bf16_burst"],
            "peak_source": f"{peaks['source']} cuBLAS bf16, {kind} figure (timed region {timed_ms:.0f} ms)"}


def run_linear(args):
    """Extra line: the QKV-generation GEMM of a Llama-3-8B-shaped layer (Eq. 2) on 32768 tokens."""
    from paper_2409_15104_b200 import binding
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    M, K, N = 32768, 4096, (32 + 2 * 8) * 128
    seed = workloads.BASE_SEED + 7
    x = workloads.normal_tensor(seed, 1, (M, K), torch.bfloat16).to(dev)
    w = (workloads.normal_tensor(seed, 2, (N, K), torch.float32) / K ** 0.5).to(torch.bfloat16).to(dev)
    y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
    for _ in range(max(args.warmup, 3)):
        binding.pec_linear(x, w, y=y)
    torch.cuda.synchronize()
    steps = _extra_steps(args, 50)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        binding.pec_linear(x, w, y=y)
    e1.record()
    torch.cuda.synchronize()
    binding.check_status()
    ms = e0.elapsed_time(e1) / steps
    tf = 2.0 * M * N * K / (ms * 1e-3) / 1e12
    peaks = load_peaks()
    import oracle
    rows = [0, 1, 127, 128, 4095, M - 1]
    want = oracle.linear(x[rows].cpu(), w.cpu())
    err = float(np.abs(y[rows].float().cpu().double().numpy() - want).max())
    # The same GEMM with the rotary position encoding of the query and key heads in its epilogue.
    theta, rot_cols = 500000.0, (32 + 8) * 128
    tables = binding.pec_rope_table(theta, M, dev)
    for _ in range(3):
        binding.pec_linear_rope(x, w, tables, rot_cols, y=y)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        binding.pec_linear_rope(x, w, tables, rot_cols, y=y)
    e1.record()
    torch.cuda.synchronize()
    binding.check_status()
    ms_rope = e0.elapsed_time(e1) / steps
    want = oracle.linear_rope(x[rows].cpu(), w.cpu(), rows, theta, rot_cols)
    err_rope = float(np.abs(y[rows].float().cpu().double().numpy() - want).max())
    return {"metric": "QKV-generation GEMM TFLOP/s (extra line, not the headline)", "value": tf, "unit": "TFLOP/s",
            "with_rotary_encoding": {"ms_per_step": ms_rope, "tflops": 2.0 * M * N * K / (ms_rope * 1e-3) / 1e12,
                                     "max_abs_err_vs_oracle_sampled_rows": err_rope},
                      "ms_per_step": ms, "steps": steps, "n_gpus": 1, "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": f"linear: x [{M},{K}] times w [{N},{K}]^T", "l2": "operands and output (752 MB) exceed L2"},
                      "roofline": _gemm_roofline(tf, ms * steps, peaks),
                      "max_abs_err_vs_oracle_sampled_rows": err}


def run_linear_merged(args):
    """Extra line: Eq. 5 on two unmerged partial results (the two GPUs' outputs of Section 5.2) in one call, beside
    the same work as a merge pass followed by the plain GEMM."""
    from paper_2409_15104_b200 import binding
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    M, hq, N, n = 32768, 32, 4096, 2
    K = hq * 128
    seed = workloads.BASE_SEED + 8
    os_ = [workloads.normal_tensor(seed + i, 1, (M, hq, 128), torch.float32).to(dev) for i in range(n)]
    ls_ = [(workloads.normal_tensor(seed + i, 2, (M, hq), torch.float32) * 2.0).to(dev) for i in range(n)]
    w = (workloads.normal_tensor(seed, 3, (N, K), torch.float32) / K ** 0.5).to(torch.bfloat16).to(dev)
    y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
    o_m = torch.empty((M, hq, 128), dtype=torch.bfloat16, device=dev)
    l_m = torch.empty((M, hq), dtype=torch.float32, device=dev)

    def fused():
        binding.pec_linear_merged(os_, ls_, w, y=y)

    def two_calls():
        binding.pec_attn_merge_n(os_, ls_, out_dtype=torch.bfloat16, o_out=o_m, lse_out=l_m)
        binding.pec_linear(o_m.view(M, K), w, y=y)

    steps = _extra_steps(args, 30)
    ms = {}
    for name, fn in (("two_calls", two_calls), ("fused", fused)):
        for _ in range(max(args.warmup, 3)):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        binding.check_status()
        ms[name] = e0.elapsed_time(e1) / steps
    tf = 2.0 * M * N * K / (ms["fused"] * 1e-3) / 1e12
    peaks = load_peaks()
    import oracle
    rows = [0, 1, 127, 128, 4095, M - 1]
    merged, _ = oracle.merge_n([o[rows].cpu().numpy() for o in os_], [l[rows].cpu().numpy() for l in ls_])
    want = oracle.linear(torch.from_numpy(merged.reshape(len(rows), K)), w.cpu())
    err = float(np.abs(y[rows].float().cpu().double().numpy() - want).max())
    col_tiles = (N + 511) // 512
    l2_bytes = col_tiles * n * M * K * 4 + ((M + 255) // 256) * N * K * 2
    return {"metric": "Eq. 5 on two unmerged partials, TFLOP/s of the GEMM (extra line, not the headline)", "value": tf,
            "unit": "TFLOP/s", "ms_per_step": ms["fused"], "steps": steps, "n_gpus": 1, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"linear_merged: {n} partials [{M},{hq},128] fp32 times w [{N},{K}]^T",
                       "l2": "partials (1.07 GB) exceed L2"},
            "ms_merge_pass_then_gemm": ms["two_calls"],
            "operand_reads_through_l2": {"bytes": l2_bytes, "gbs": l2_bytes / (ms["fused"] * 1e-3) / 1e9,
                                         "note": "every 512-column tile re-reads its rows of the fp32 partials"},
            "roofline": _gemm_roofline(tf, ms["fused"] * steps, peaks),
            "max_abs_err_vs_oracle_sampled_rows": err}


def run_layer(args):
    """Extra line: the attention part of one Llama-3-8B-shaped layer on a 32K-token request, every step through the
    library - QKV generation with rotary encoding (Eq. 2), causal attention over 8 key partitions reading q, k, v as
    strided slices of the fused tensor (Eq. 3-4), the post-attention linear layer (Eq. 5)."""
    from paper_2409_15104_b200 import binding
    from paper_2409_15104_b200.prefill import PartitionedPrefill
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    wl = workloads.WORKLOADS["c3"]
    S, hq, hkv, d = wl.seq_len, wl.hq, wl.hkv, 4096
    seed = workloads.BASE_SEED + 9
    x = workloads.normal_tensor(seed, 1, (S, d), torch.bfloat16).to(dev)
    w_qkv = (workloads.normal_tensor(seed, 2, ((hq + 2 * hkv) * 128, d), torch.float32) / d ** 0.5).to(torch.bfloat16).to(dev)
    w_l = (workloads.normal_tensor(seed, 3, (d, hq * 128), torch.float32) / (hq * 128) ** 0.5).to(torch.bfloat16).to(dev)
    tables = binding.pec_rope_table(500000.0, S, dev)
    qkv = torch.empty((S, (hq + 2 * hkv) * 128), dtype=torch.bfloat16, device=dev)
    y = torch.empty((S, d), dtype=torch.bfloat16, device=dev)
    fused = qkv.view(S, hq + 2 * hkv, 128)
    q, k, v = fused[:, :hq], fused[:, hq:hq + hkv], fused[:, hq + hkv:]
    runner = PartitionedPrefill(S, hq, wl.num_parts, wl.dtype, dev, wl.part_align)

    def step():
        binding.pec_linear_rope(x, w_qkv, tables, (hq + hkv) * 128, y=qkv)
        o, _ = runner.run(q, k, v)
        binding.pec_linear(o.view(S, hq * 128), w_l, y=y)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    steps = _extra_steps(args, 20)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    binding.check_status()
    ms = e0.elapsed_time(e1) / steps
    flops = 2.0 * S * (hq + 2 * hkv) * 128 * d + workloads.attention_flops(workloads.causal_pairs(S), hq) + 2.0 * S * d * hq * 128
    # the last rows of the layer's output against the oracle applied step by step to what each step actually read
    import oracle
    rows = [0, 1, 4095, S - 2, S - 1]
    o_dev = runner.out_o
    want_qkv = oracle.linear_rope(x[rows].cpu(), w_qkv.cpu(), rows, 500000.0, (hq + hkv) * 128)
    err_qkv = float(np.abs(qkv[rows].float().cpu().double().numpy() - want_qkv).max())
    want_o, _ = oracle.prefill_attn(q.cpu(), k.cpu(), v.cpu(), seq_len=S, rows=rows)
    err_o = float(np.abs(o_dev[rows].float().cpu().double().numpy() - want_o).max())
    want_y = oracle.linear(o_dev[rows].reshape(len(rows), hq * 128).cpu(), w_l.cpu())
    err_y = float(np.abs(y[rows].float().cpu().double().numpy() - want_y).max())
    return {"metric": "attention part of one layer (QKV generation + rotary encoding, attention, output projection), TFLOP/s (extra line)",
            "value": flops / (ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": ms, "steps": steps, "n_gpus": 1, "dtype": "bf16",
            "data": "synthetic", "tokens_per_s": S / (ms * 1e-3),
            "config": {"workload": f"layer: S={S}, model width {d}, {hq}/{hkv} heads, {wl.num_parts} key partitions",
                       "l2": "activations exceed the L2"},
            "max_abs_err_vs_oracle_sampled_rows": {"qkv": err_qkv, "o": err_o, "y": err_y}}


def _short_batch(wl, dev, seed_offset=0):
    lens = workloads.short_lengths(wl.seed, wl.short_batch)
    cu = workloads.cu_seqlens(lens)
    q, k, v = workloads.qkv(wl.seed + 100 + seed_offset, cu[-1], wl.hq, wl.hkv, 128, wl.dtype)
    pairs = sum(workloads.causal_pairs(n) for n in lens)
    return (q.to(dev), k.to(dev), v.to(dev), torch.tensor(cu, dtype=torch.int32, device=dev), cu[-1], pairs)


def run_ring(args):
    """Extra line: the P x P (rank, ring step) launches of ring-attention SP over c3's request, every rank
    emulated on this GPU one after the other, beside the planner's per-step work for zigzag and contiguous
    segments (what a real ring's step times would follow)."""
    from paper_2409_15104_b200 import binding
    from paper_2409_15104_b200.prefill import ring_prefill
    wl = workloads.WORKLOADS["c3"]
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    q, k, v = (t.to(dev) for t in workloads.qkv(wl.seed, wl.seq_len, wl.hq, wl.hkv, 128, wl.dtype))
    P = wl.num_parts
    for _ in range(max(args.warmup, 3)):
        _, _, launches = ring_prefill(q, k, v, P, wl.part_align)
    torch.cuda.synchronize()
    evs = []
    for _ in range(_extra_steps(args, 20)):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); ring_prefill(q, k, v, P, wl.part_align); e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    binding.check_status()
    ms = statistics.median(a.elapsed_time(b) for a, b in evs)
    fl = workloads.attention_flops(workloads.causal_pairs(wl.seq_len), wl.hq)
    plans = {name: binding.pec_plan_ring(wl.seq_len, P, wl.part_align, code, True)
             for name, code in (("zigzag", binding.PEC_LAYOUT_ZIGZAG), ("contiguous", binding.PEC_LAYOUT_CONTIGUOUS))}
    total = workloads.causal_pairs(wl.seq_len)
    return {"metric": "ring-attention SP steps of all ranks on one GPU, attention TFLOP/s (extra line, not the headline)",
                      "value": fl / (ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": ms, "n_gpus": 1, "dtype": "bf16",
                      "data": "synthetic", "gpu_launches_per_step": launches,
                      "planned_ring_time_in_pairs": {name: sum(pl["step_max"]) for name, pl in plans.items()},
                      "planned_ring_efficiency": {name: total / (P * sum(pl["step_max"])) for name, pl in plans.items()},
                      "config": {"workload": f"ring: {wl.note}; rank r's query blocks against the keys of rank (r-t) mod P",
                                 "ranks": P, "l2": "inputs and partials exceed the 126 MB L2"}}


def run_short_batch(args, wl=None):
    """Extra record: the packed short-request batch (c2) alone.  A step is what a caller does per batch: build
    the heaviest-first work-list on the host, copy it to the device, launch.  The same batch with every CTA
    searching cu_seqlens instead is timed beside it."""
    from paper_2409_15104_b200 import binding
    from paper_2409_15104_b200.prefill import make_worklist, varlen_prefill
    wl = wl or workloads.WORKLOADS["c2"]
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    q, k, v, cu, T, pairs = _short_batch(wl, dev)
    cu_host = [int(x) for x in cu.cpu()]
    o = torch.empty((T, wl.hq, 128), dtype=wl.dtype, device=dev)
    lse = torch.empty((T, wl.hq), dtype=torch.float32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def with_list():
        varlen_prefill(q, k, v, cu, o=o, lse=lse, worklist=make_worklist(cu_host, wl.dtype, dev))

    def without():
        varlen_prefill(q, k, v, cu, o=o, lse=lse)

    res = {}
    for name, fn in (("worklist", with_list), ("search", without)):
        for _ in range(max(args.warmup, 3)):
            fn()
        torch.cuda.synchronize()
        evs = []
        for _ in range(_extra_steps(args, 50)):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        binding.check_status()
        res[name] = statistics.median(a.elapsed_time(b) for a, b in evs)
    ms = res["worklist"]
    fl = workloads.attention_flops(pairs, wl.hq)
    peaks = load_peaks()
    tf = fl / (ms * 1e-3) / 1e12
    return {"metric": "short-request varlen batch, attention TFLOP/s (extra record)",
            "value": tf, "unit": "TFLOP/s", "ms_per_step": ms, "n_gpus": 1, "dtype": "bf16",
            "data": "synthetic", "tokens_per_s": T / (ms * 1e-3),
            "frac_of_burst": tf / peaks["bf16_burst"], "frac_of_nominal": tf / NOMINAL_BF16_TFLOPS,
            "without_worklist": {"value": fl / (res["search"] * 1e-3) / 1e12, "ms_per_step": res["search"]},
            "config": {"workload": f"{wl.name}: {wl.note}", "requests": wl.short_batch, "tokens": T,
                       "pairs_per_head": pairs, "l2": "256 MiB written between timed calls"}}


def run_preempted(args, wl=None):
    """Extra record: c4 - a long prefill as 16 resumed chunks on a low-priority stream with a short-request
    batch on a high-priority stream, arriving (a) at a chunk boundary and (b) in the middle of a late chunk,
    which is what preemption between kernels costs a short request: the rest of the running chunk at worst."""
    from paper_2409_15104_b200 import binding
    from paper_2409_15104_b200.prefill import chunked_prefill, make_worklist, varlen_prefill
    wl = wl or workloads.WORKLOADS["c4"]
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    S, C = wl.seq_len, wl.chunk_len
    q, k, v = (t.to(dev) for t in workloads.qkv(wl.seed, S, wl.hq, wl.hkv, 128, wl.dtype))
    sq, sk, sv, cu, T, spairs = _short_batch(wl, dev)
    slist = make_worklist([int(x) for x in cu.cpu()], wl.dtype, dev)
    o = torch.empty((S, wl.hq, 128), dtype=wl.dtype, device=dev)
    lse = torch.empty((S, wl.hq), dtype=torch.float32, device=dev)
    so = torch.empty((T, wl.hq, 128), dtype=wl.dtype, device=dev)
    sl = torch.empty((T, wl.hq), dtype=torch.float32, device=dev)
    lo, hi = torch.cuda.Stream(priority=0), torch.cuda.Stream(priority=-1)
    n_chunks = S // C
    late = n_chunks - 4                                       # the chunk the batch interrupts in (b)

    def timed(fn):
        torch.cuda.synchronize()
        t0 = time.perf_counter(); fn(); torch.cuda.synchronize()
        return (time.perf_counter() - t0) * 1e3

    def long_only(events=None):
        chunked_prefill(q, k, v, C, o, lse, stream=lo, events=events)

    def short_only():
        varlen_prefill(sq, sk, sv, cu, o=so, lse=sl, stream=hi, worklist=slist)

    marks = {}

    def short_timed(key):
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record(hi); short_only(); s1.record(hi)
        marks[key] = (s0, s1)

    def at_boundary():
        def arrive(c):
            if c == 3:                                         # the batch starts once chunk 3 has finished
                ev = torch.cuda.Event(); ev.record(lo)
                hi.wait_event(ev)
                short_timed("boundary")
        chunked_prefill(q, k, v, C, o, lse, stream=lo, between_chunks=arrive)

    def mid_chunk():
        started = {}

        def arrive(c):
            if c == late - 1:
                started["ev"] = torch.cuda.Event(); started["ev"].record(lo)
            if c == n_chunks - 1:                              # every chunk is enqueued: now wait, on the host, for chunk
                started["ev"].synchronize()                    # `late` to be the one running, let it run for a while,
                time.sleep(0.003)                              # and only then hand the batch to the GPU
                short_timed("mid")
        chunked_prefill(q, k, v, C, o, lse, stream=lo, between_chunks=arrive)

    for fn in (long_only, short_only, at_boundary, mid_chunk):
        timed(fn)                                              # warm-up
    reps = 3
    chunk_events = []
    t_long = min(timed(lambda: long_only(chunk_events)) for _ in range(reps))
    chunk_ms = [a.elapsed_time(b) for a, b in chunk_events]
    t_short = min(timed(short_only) for _ in range(reps))
    t_both, lat_b, lat_m = [], [], []
    for _ in range(reps):
        t_both.append(timed(at_boundary))
        lat_b.append(marks["boundary"][0].elapsed_time(marks["boundary"][1]))
        timed(mid_chunk)
        lat_m.append(marks["mid"][0].elapsed_time(marks["mid"][1]))
    binding.check_status()
    fl_long = workloads.attention_flops(workloads.causal_pairs(S), wl.hq)
    fl_short = workloads.attention_flops(spairs, wl.hq)
    peaks = load_peaks()
    tf_long = fl_long / (t_long * 1e-3) / 1e12
    return {"metric": "preempted long prefill with a colocated short batch (extra record)",
            "value": (fl_long + fl_short) / (min(t_both) * 1e-3) / 1e12, "unit": "TFLOP/s", "n_gpus": 1,
            "dtype": "bf16", "data": "synthetic",
            "long_alone_ms": t_long, "long_alone_tflops": tf_long, "long_alone_frac_of_nominal": tf_long / NOMINAL_BF16_TFLOPS,
            "long_alone_frac_of_sustained": tf_long / peaks["bf16_sustained"], "long_tokens_per_s": S / (t_long * 1e-3),
            "short_alone_ms": t_short, "interleaved_ms": min(t_both),
            "short_batch_latency_at_chunk_boundary_ms": {"best": min(lat_b), "worst": max(lat_b)},
            "short_batch_latency_arriving_mid_chunk_ms": {"best": min(lat_m), "worst": max(lat_m), "interrupted_chunk": late,
                                                          "that_chunk_alone_ms": chunk_ms[late] if len(chunk_ms) > late else None},
            "longest_chunk_ms": max(chunk_ms) if chunk_ms else None,
            "timing": "host wall clock around a synchronised region (multi-stream); short-batch latency by CUDA events on its "
                      "own stream, from the moment the host hands it over to its completion",
            "config": {"workload": f"{wl.name}: {wl.note}", "chunks": n_chunks, "short_tokens": T}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=["c2", "c3", "c4", "c5", "decode", "linear", "linear_merged", "layer", "ring", "merge"], default="c5",
                    help="c5 (default, the largest single-GPU configuration) and c3 print the full line; the others "
                         "print their extra record alone")
    ap.add_argument("--no-extra", action="store_true", help="skip the extra records nested under the headline line")
    ap.add_argument("--reference-seconds", type=float, default=0.0,
                    help="--impl reference: CPU seconds per step (default: 90 s spread over the steps, 0.15-20 s each)")
    ap.add_argument("--profile", action="store_true",
                    help="profiling runs: skip the end-to-end, extra and CPU-baseline legs (the printed line is not a result)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args, workloads.WORKLOADS[args.workload if args.workload in ("c3", "c5") else "c5"])
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU implementation")
    alone = {"decode": run_decode, "linear": run_linear, "linear_merged": run_linear_merged, "layer": run_layer, "ring": run_ring, "c2": run_short_batch, "c4": run_preempted,
             "merge": extra_merge_kernel}
    if args.workload in alone:
        print(json.dumps(alone[args.workload](args)), flush=True)
        return
    run_ours(args, workloads.WORKLOADS[args.workload])


if __name__ == "__main__":
    main()
