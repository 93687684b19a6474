#!/usr/bin/env python
"""Benchmark of the MCSD verification step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

With --gpus N > 1 and no torchrun around it the script starts its own N ranks (one per GPU).

A step is one pass of the whole hot path (per-node softmax statistics, rejection loop,
endpoint tokens, tree walk, terminal residual) over one batch of synthetic trees whose
logits are already resident in HBM.  The default workload is the largest point of the
throughput sweep (batch 512, k-config 4x4x2x2x1, vocabulary 32000, fp32 logits, 19.5 GB of
logits), which is the configuration the bandwidth target is quoted on.  Prints ONE JSON
line (rank 0).  With --impl reference the CPU oracle is timed on the host cores instead.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2401_06706_b200 import synth

METRIC = "verified_tree_nodes_per_sec"
UNIT = "nodes/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0


# ----------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


TRAFFIC_PROFILES = {"stream_stats_kernel": os.path.join("profiles", "stream_stats_kernel_cfg5_batch16_ncu_full.md"),
                    "node_kernel": os.path.join("profiles", "node_kernel_cfg5_batch16_ncu_full.md")}


def recorded_traffic(kernel: str, units: int):
    """DRAM bytes per launch of a kernel from its committed ncu summary, scaled by the logit rows the
    launch reads (the capture ran a smaller batch of the same workload and the traffic grows in
    proportion to the rows read).  Returns (bytes, source, scale factor); bytes is None when there
    is no summary with a `dram_bytes_per_launch=... units_per_launch=...` line."""
    import re
    prof = TRAFFIC_PROFILES.get(kernel)
    try:
        with open(os.path.join(ROOT, prof)) as f:
            m = re.search(r"dram_bytes_per_launch=(\d+) units_per_launch=(\d+)", f.read())
        scale = units / float(m.group(2))
        return float(m.group(1)) * scale, (f"{prof}: dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture "
                                            f"at {m.group(2)} logit rows per launch, scaled by the rows per launch"), scale
    except Exception:
        return None, "no recorded capture of this kernel", None


def kernel_breakdown(binding, call, n_calls: int):
    """Device time of every kernel of the step, from CUDA events the library records around its own
    launches on the launching stream (MCSD_OPT_TIME_KERNELS), over n_calls further calls; programmatic
    dependent launch is switched off meanwhile so that the intervals do not overlap."""
    names = ("node_kernel", "stream_stats_kernel", "single_decide_kernel", "walk_kernel")
    before = (binding.mcsd_get_option(binding.OPT_TIME_KERNELS), binding.mcsd_get_option(binding.OPT_PDL))
    binding.mcsd_set_option(binding.OPT_TIME_KERNELS, 1)
    binding.mcsd_set_option(binding.OPT_PDL, 0)
    tot, cnt = [0.0] * 4, [0] * 4
    try:
        for _ in range(n_calls):
            call()
            for i, ms in enumerate(binding.mcsd_last_kernel_times()):
                if ms is not None:
                    tot[i] += ms
                    cnt[i] += 1
    finally:
        binding.mcsd_set_option(binding.OPT_TIME_KERNELS, before[0])
        binding.mcsd_set_option(binding.OPT_PDL, before[1])
    return {names[i]: tot[i] / cnt[i] for i in range(4) if cnt[i]}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons, power = [], [], set(), []
        rows = [r for (t, r) in self.rows if t0 <= t <= t1 + 0.15] or [r for (_, r) in self.rows]
        for row in rows:
            parts = [p.strip() for p in row.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def spawn_command(argv, n: int, port: int):
    """The command that starts n ranks of this script on one node (what a plain
    `python bench.py --gpus n` runs when no launcher is around it)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def spawn_ranks(args):
    """--gpus N > 1 without a launcher: start N ranks (one process per GPU) and pass their output on.
    NCCL's log is switched on (to files, so that stdout stays the one JSON line)."""
    if args.impl != "reference" and torch.cuda.device_count() < args.gpus:
        raise SystemExit(f"--gpus {args.gpus}: only {torch.cuda.device_count()} CUDA devices are visible")
    env = dict(os.environ)
    if "NCCL_DEBUG" not in env:
        env["NCCL_DEBUG"] = "INFO"
        env["NCCL_DEBUG_FILE"] = os.path.join(env.get("TMPDIR", "/tmp"), "mcsd_bench_nccl.%h.%p.log")
    if args.impl == "reference":     # only rank 0 works there: it may use every core
        env.setdefault("OMP_NUM_THREADS", str(os.cpu_count() or 1))
    port = 29500 + os.getpid() % 2000
    return subprocess.call(spawn_command(sys.argv[1:], args.gpus, port), env=env)


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def pick_workload(name: str, batch: int = 0, logit_dtype: str = "") -> synth.Workload:
    from dataclasses import replace
    named = synth.named_workloads()
    found = named.get(name)
    if found is None:
        for w in synth.sweep_workloads():
            if w.name == name:
                found = w
    if found is None:
        raise SystemExit(f"unknown workload {name!r}; named: {sorted(named)}")
    if logit_dtype:
        found = replace(found, dtype=logit_dtype)
    return replace(found, batch=batch) if batch > 0 else found


def shard_for_rank(w: synth.Workload, rank: int, world: int) -> synth.Workload:
    """Weak scaling: every rank verifies its own batch of the same shape (sequences are
    independent, so there is no data-path collective); seeds differ per rank."""
    from dataclasses import replace
    return replace(w, seed=w.seed + 7919 * rank) if world > 1 else w


def max_over_ranks(dist, value: float, device) -> float:
    """Largest value any rank holds (elapsed times are reported as the slowest rank's)."""
    if dist is None:
        return float(value)
    tt = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def whole_job_value(world: int, nodes_per_rank_step: int, ms_per_step: float) -> float:
    """Verified tree nodes per second of the whole job: every rank verifies its own batch."""
    return world * nodes_per_rank_step / (ms_per_step * 1e-3)


def oracle_sample(inp: synth.Inputs, n_seq: int):
    """Times the CPU oracle, as it stands, on the first n_seq sequences."""
    import oracle
    w = inp.workload
    n_seq = min(n_seq, w.batch)
    t, d, c, u = inp.host_f32(0, n_seq)
    oracle.verify(t[:1], None if d is None or w.temperature == 0 else d[:1], inp.parent, c[:1], u[:1],
                  w.temperature, w.mode, want_residual=True)          # loads the library
    t0 = time.perf_counter()
    res = oracle.verify(t, d if w.temperature > 0 else None, inp.parent, c, u, w.temperature, w.mode)
    dt = time.perf_counter() - t0
    nodes = n_seq * inp.stats["n_draft"]
    # the same oracle on one thread, on a smaller sample (one sequence at a time leaves OpenMP nothing to split)
    n_one = min(n_seq, 8)
    t1 = time.perf_counter()
    for b in range(n_one):
        oracle.verify(t[b:b + 1], d[b:b + 1] if (d is not None and w.temperature > 0) else None, inp.parent,
                      c[b:b + 1], u[b:b + 1], w.temperature, w.mode)
    dt1 = time.perf_counter() - t1
    return {"value": nodes / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"first {n_seq} of {w.batch} sequences of the same inputs, {dt:.2f} s wall, all-node form, "
                      f"OpenMP over sequences",
            "single_thread": {"value": n_one * inp.stats["n_draft"] / dt1, "unit": UNIT, "cores": 1,
                              "sample": f"first {n_one} sequences one at a time, {dt1:.2f} s wall"}}, res


# ----------------------------------------------------------------------------- reference arm
def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    import oracle
    w = pick_workload(args.workload, args.batch, args.logit_dtype)
    from dataclasses import replace
    # size the per-step sample so that the whole run takes about a minute of wall time
    probe = synth.make_inputs(replace(w, batch=min(w.batch, 8)), "cpu")
    t, d, c, u = probe.host_f32()
    dd = d if w.temperature > 0 else None
    oracle.verify(t[:1], None if dd is None else dd[:1], probe.parent, c[:1], u[:1], w.temperature, w.mode)
    t0 = time.perf_counter()
    oracle.verify(t, dd, probe.parent, c, u, w.temperature, w.mode)
    per_seq = (time.perf_counter() - t0) / t.shape[0]
    budget = 60.0 / max(args.steps + max(args.warmup, 1), 1)
    n_seq = int(max(1, min(w.batch, args.oracle_seqs, budget / max(per_seq, 1e-9))))
    sample = replace(w, batch=n_seq)
    inp = synth.make_inputs(sample, "cpu")
    t, d, c, u = inp.host_f32()
    dd = d if w.temperature > 0 else None
    for _ in range(max(args.warmup, 1)):
        oracle.verify(t, dd, inp.parent, c, u, w.temperature, w.mode)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.verify(t, dd, inp.parent, c, u, w.temperature, w.mode)
    dt = (time.perf_counter() - t0) / args.steps
    value = n_seq * inp.stats["n_draft"] / dt
    desc = f"{n_seq} sequences of workload {w.name} per step (bounded sample of its {w.batch}), generated on the CPU"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, inp.stats, sample_batch=n_seq),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def workload_config(w: synth.Workload, st, **extra):
    cfg = {"workload": w.name, "batch": w.batch, "vocab": w.vocab, "kconfig": w.kconfig,
           "logit_dtype": w.dtype, "draft_nodes_per_tree": st["n_draft"], "target_rows_per_tree": st["n_nodes"],
           "draft_rows_per_tree": st["n_internal"], "temperature": w.temperature,
           "replacement_mode": "without" if w.mode == 1 else "with", "target_dist": w.target_dist,
           "target_scale": w.target_scale, "draft_gain": w.draft_gain, "draft_sigma": w.draft_sigma,
           "seed": w.seed}
    cfg.update(extra)
    return cfg


# ----------------------------------------------------------------------------- CUDA arm
def timed_steps(step, n_steps: int, dist, dev, clock_index):
    """n_steps calls of step(events) between barriers and synchronisations; CUDA events around the whole
    region and around the node stage of every step; clocks sampled meanwhile.  Returns (elapsed ms of
    the slowest rank, node-stage ms per step of this rank, clock record or None)."""
    node_events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in range(n_steps)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(clock_index) if clock_index is not None else None
    if sampler:
        sampler.start()
        time.sleep(0.25)
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    t_host0 = time.time()
    start.record()
    for i in range(n_steps):
        step(node_events[i])
    stop.record()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    t_host1 = time.time()
    elapsed_ms = max_over_ranks(dist, start.elapsed_time(stop), dev)
    node_ms = [a.elapsed_time(b) for a, b in node_events]
    clocks = sampler.stop(t_host0, t_host1) if sampler else None
    return elapsed_ms, node_ms, clocks


def run_cuda(args):
    from paper_2401_06706_b200 import binding
    rank, world, local = dist_env()
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        dist = None
        torch.cuda.set_device(0)
    dev = torch.device("cuda", torch.cuda.current_device())
    binding.load_library()       # raises if the CUDA library is missing: no fallback

    w = shard_for_rank(pick_workload(args.workload, args.batch, args.logit_dtype), rank, world)
    inp = synth.make_inputs(w, dev)
    st = inp.stats
    ver = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[w.dtype], dev)
    draft = inp.draft if w.temperature > 0 else None
    nodes_per_step = w.batch * st["n_draft"]

    def step(events=None):
        if args.form == "path":
            if events is not None:
                events[0].record()
            ver.mcsd_verify_path(inp.target, draft, inp.cand, inp.unif, w.temperature, w.mode)
            if events is not None:
                events[1].record()
            return
        if events is None:
            ver.mcsd_verify(inp.target, draft, inp.cand, inp.unif, w.temperature, w.mode)
            return
        e0, e1 = events
        e0.record()
        ver.mcsd_verify_nodes(inp.target, draft, inp.cand, inp.unif, w.temperature, w.mode)
        e1.record()
        ver.mcsd_verify_walk(inp.target, draft, inp.cand, inp.unif, w.temperature)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    launches_per_step = 0
    if args.form == "path":
        ver.mcsd_verify_path(inp.target, draft, inp.cand, inp.unif, w.temperature, w.mode)
        launches_per_step += binding.mcsd_last_launch_count()
    else:
        ver.mcsd_verify_nodes(inp.target, draft, inp.cand, inp.unif, w.temperature, w.mode)
        launches_per_step += binding.mcsd_last_launch_count()
        ver.mcsd_verify_walk(inp.target, draft, inp.cand, inp.unif, w.temperature)
        launches_per_step += binding.mcsd_last_launch_count()
    torch.cuda.synchronize()

    # timed region: K steps between barriers and synchronisations, CUDA events on the
    # launching stream; the node kernel of every step is bracketed by its own events
    elapsed_ms, node_ms, clocks = timed_steps(step, args.steps, dist, dev, torch.cuda.current_device() if rank == 0 else None)
    status_bits = int(ver.status.max().item()) if w.batch else 0

    ms_per_step = elapsed_ms / args.steps
    value = whole_job_value(world, nodes_per_step, ms_per_step)

    # roofline of the dominant kernel (the per-node kernel): algorithmic bytes per launch =
    # every target row once + every draft row once (none at temperature 0) + 12 bytes of
    # candidate token and uniforms per node
    logit_bytes = inp.logit_bytes()
    algo_bytes = logit_bytes + 12 * w.batch * st["n_nodes"]
    if args.form == "path":
        # only the rows of visited nodes are read: len+1 target rows per sequence and one draft
        # row per visited node that has children (every node above the leaf level)
        ln = ver.accept_len.to(torch.int64)
        rows = int((ln + 1).sum().item()) + (int(torch.clamp(ln + 1, max=st["gamma"]).sum().item())
                                             if w.temperature > 0 else 0)
        algo_bytes = rows * w.vocab * inp.target.element_size()
    node_ms_avg = sum(node_ms) / len(node_ms)
    achieved = algo_bytes / (node_ms_avg * 1e-3) / 1e9
    peak, peak_kind = measured_peaks()
    # The node stage of a large launch is three kernels (the cluster kernel for the nodes with two or
    # more children, the streaming kernel for the rows of all others, the single-test kernel).  The
    # roofline object is for the DOMINANT one, with its own algorithmic bytes and its own duration from
    # CUDA events around it; the whole stage follows under "stage".
    es = inp.target.element_size()
    _, child_count = synth.children_ranges(inp.parent)
    n_keep = int((child_count >= 2).sum())
    n_single = int((child_count == 1).sum())
    n_leaf = st["n_nodes"] - st["n_internal"]
    stage = {"kernels": "argmax_kernel" if w.temperature == 0 else "node_kernel + stream_stats_kernel + single_decide_kernel",
             "ms_avg": node_ms_avg, "ms_min": min(node_ms), "algorithmic_bytes": algo_bytes, "achieved": achieved,
             "frac": achieved / peak, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
             "step_share": node_ms_avg / ms_per_step}
    per_kernel = None
    kernel, k_ms, k_bytes, k_rows = ("node_kernel" if w.temperature > 0 else "argmax_kernel"), node_ms_avg, algo_bytes, None
    if args.form == "all_node" and w.temperature > 0 and world == 1:
        per_kernel = kernel_breakdown(binding, lambda: ver.mcsd_verify(inp.target, draft, inp.cand, inp.unif, w.temperature, w.mode),
                                      min(args.steps, 20))
        split = "stream_stats_kernel" in per_kernel
        rows = {"node_kernel": w.batch * (2 * n_keep if split else st["n_nodes"] + st["n_internal"]),
                "stream_stats_kernel": w.batch * (n_leaf + 2 * n_single)}
        bytes_of = {k: rows[k] * w.vocab * es + (12 * w.batch * (n_keep if split else st["n_nodes"]) if k == "node_kernel" else 0)
                    for k in rows}
        kernel = max((k for k in per_kernel if k in rows), key=lambda k: per_kernel[k])
        k_ms, k_bytes, k_rows = per_kernel[kernel], bytes_of[kernel], rows[kernel]
        stage["per_kernel_ms"] = per_kernel
        stage["per_kernel_gbs"] = {k: bytes_of[k] / (per_kernel[k] * 1e-3) / 1e9 for k in rows if k in per_kernel}
    traffic, traffic_source, traffic_scale = (recorded_traffic(kernel, k_rows)
                                              if (w.name == "cfg5_largest" and w.dtype == "fp32" and k_rows)
                                              else (None, "no capture of this kernel variant and workload", None))
    k_achieved = k_bytes / (k_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": kernel +
                (" (the figure covers the whole call, which is bound by launch and exchange latency, not by HBM)"
                 if args.form == "path" else ""),
                "achieved": k_achieved, "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                "frac": k_achieved / peak, "frac_of_nominal_8TBs": k_achieved / NOMINAL_HBM_GBS,
                "algorithmic_bytes_per_launch": k_bytes, "kernel_ms_avg": k_ms,
                "step_share": k_ms / ms_per_step,
                "traffic": traffic, "traffic_source": traffic_source, "traffic_scale": traffic_scale,
                "stage": stage}

    # the same steps again, many more of them: the power cap pulls the SM clock down after the first
    # hundred milliseconds, and the kernel's time follows the clock.  Clocks come from the sampler;
    # no clock setting is touched.
    sustained = None
    if args.sustained_steps > 0 and world == 1:
        s_ms, s_node, s_clk = timed_steps(step, args.sustained_steps, None, dev, torch.cuda.current_device())
        s_k_ms = sum(s_node) / len(s_node)
        sustained = {"steps": args.sustained_steps, "ms_per_step": s_ms / args.sustained_steps, "stage_ms_avg": s_k_ms,
                     "what": "the whole node stage (all its kernels) over its algorithmic bytes",
                     "achieved": algo_bytes / (s_k_ms * 1e-3) / 1e9, "frac": algo_bytes / (s_k_ms * 1e-3) / 1e9 / peak,
                     "sm_mhz": s_clk["sm_mhz"] if s_clk else None, "reasons": s_clk["reasons"] if s_clk else None,
                     "power_w_max": s_clk.get("power_w_max") if s_clk else None,
                     "stage_ms_x_mhz": (s_k_ms * s_clk["sm_mhz"]) if (s_clk and s_clk["sm_mhz"]) else None,
                     "timed_region_stage_ms_x_mhz": (node_ms_avg * clocks["sm_mhz"]) if (clocks and clocks["sm_mhz"]) else None}

    # end to end through the host-buffer entry point: pinned host inputs, copies inside
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, w, inp, dist, world, dev)

    cpu_baseline = None
    parity = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline, ref = oracle_sample(inp, args.oracle_seqs)
        parity = parity_on_sample(inp, ver, ref, min(args.oracle_seqs, w.batch))
    accept_len_mean = float(ver.accept_len.float().mean().item()) if w.batch else 0.0

    # sub-record: the same workload with 2-byte logits (the precision the paper ran in, Section 4.1)
    half = None
    if (rank == 0 and world == 1 and not args.no_half and w.dtype == "fp32" and args.form == "all_node"
            and w.temperature > 0):
        from dataclasses import replace
        del inp, ver
        torch.cuda.empty_cache()
        half = half_record(replace(w, dtype="bf16"), dev, args, peak)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": workload_config(w, st, form=args.form, parallelism=f"replicas x{world} (batch split, no collective)",
                                          l2="inputs (%.2f GB per GPU) far larger than the 126 MB L2" %
                                          (logit_bytes / 1e9) if logit_bytes > 4 * 126e6 else
                                          "inputs smaller than 4x L2: latency/L2-bound point",
                                          logit_gb_per_gpu=logit_bytes / 1e9),
                "roofline": roofline, "sustained": sustained, "bf16": half, "cpu_baseline": cpu_baseline, "e2e": e2e,
                "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
                "hbm_gbs_whole_step": algo_bytes / (ms_per_step * 1e-3) / 1e9,
                "us_per_call": ms_per_step * 1e3,
                "rows_per_sec": world * w.batch * (st["n_nodes"] + (st["n_internal"] if w.temperature > 0 else 0)) / (ms_per_step * 1e-3),
                "accept_len_mean": accept_len_mean,
                "alpha_hat": parity.get("alpha_hat") if isinstance(parity, dict) else None,
                "device_status_bits": status_bits, "parity_on_oracle_sample": parity}
        print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


def parity_on_sample(inp, ver, ref, n_seq):
    from oracle import compare
    w = inp.workload
    t, d, c, u = inp.host_f32(0, n_seq)
    rep = compare.compare(t, d, inp.parent, c, u, w.temperature, w.mode, w.dtype,
                          accept_len=ver.accept_len[:n_seq].cpu().numpy(), tokens=ver.tokens[:n_seq].cpu().numpy(),
                          residual=ver.residual[:n_seq].cpu().numpy(), status=ver.status[:n_seq].cpu().numpy(),
                          oracle_result=ref)
    out = rep.summary()
    out["ok"] = rep.ok
    out["accept_len_mean"] = float(ref.accept_len.mean())
    # acceptance rate of the synthetic inputs: share of nodes with children that accepted one of their
    # candidates (all nodes of the sampled trees), for comparison with the paper's alpha (Section 4.1)
    n_int = inp.stats["n_internal"]
    out["alpha_hat"] = float((ref.node_accept[:, :n_int] >= 0).mean()) if n_int else None
    return out


def half_record(w, dev, args, peak):
    """Node stage and whole step of the same workload with 2-byte logits: kernel ms, GB/s, fraction of
    the peak, clocks, parity on a sample."""
    from paper_2401_06706_b200 import binding
    inp = synth.make_inputs(w, dev)
    st = inp.stats
    ver = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[w.dtype], dev)

    def step(events):
        e0, e1 = events
        e0.record()
        ver.mcsd_verify_nodes(inp.target, inp.draft, inp.cand, inp.unif, w.temperature, w.mode)
        e1.record()
        ver.mcsd_verify_walk(inp.target, inp.draft, inp.cand, inp.unif, w.temperature)

    dummy = (torch.cuda.Event(), torch.cuda.Event())
    for _ in range(max(args.warmup, 3)):
        step(dummy)
    n = max(20, min(args.steps, 100))
    ms, node_ms, clk = timed_steps(step, n, None, dev, torch.cuda.current_device())
    algo = inp.logit_bytes() + 12 * w.batch * st["n_nodes"]
    k_ms = sum(node_ms) / len(node_ms)
    rec = {"logit_dtype": w.dtype, "steps": n, "ms_per_step": ms / n, "stage_ms_avg": k_ms, "stage_ms_min": min(node_ms),
           "what": "the whole node stage (all its kernels) over its algorithmic bytes",
           "algorithmic_bytes": algo, "achieved": algo / (k_ms * 1e-3) / 1e9, "unit": "GB/s",
           "frac": algo / (k_ms * 1e-3) / 1e9 / peak, "value": w.batch * st["n_draft"] / (ms / n * 1e-3), "clocks": clk,
           "per_kernel_ms": kernel_breakdown(binding, lambda: ver.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif,
                                                                              w.temperature, w.mode), 10)}
    if not args.no_cpu_baseline:
        # cpu_baseline leg of this sub-record: the oracle timed on the first sequences of these inputs;
        # what it computed is then compared with the kernels' output on those sequences
        rec["cpu_baseline"], ref = oracle_sample(inp, min(64, args.oracle_seqs))
        rec["parity_on_oracle_sample"] = parity_on_sample(inp, ver, ref, min(64, args.oracle_seqs, w.batch))
    return rec


def host_mem_available() -> int:
    try:
        with open("/proc/meminfo") as f:
            for line in f:
                if line.startswith("MemAvailable:"):
                    return int(line.split()[1]) * 1024
    except Exception:
        pass
    return 0


def run_e2e(args, w, inp, dist, world, dev):
    """The same metric through mcsd_verify_host: inputs in pinned HOST memory, every copy in both
    directions inside the timed region.  The whole batch of the workload per step when the host can
    pin it, else the largest part that fits (said in the record)."""
    from paper_2401_06706_b200 import binding
    st = inp.stats
    per_seq = inp.logit_bytes() // max(w.batch, 1) + 12 * st["n_nodes"]
    nb, why = w.batch, "the whole batch"
    if args.e2e_batch > 0:
        nb, why = min(w.batch, args.e2e_batch), "--e2e-batch"
    else:
        avail = host_mem_available() // max(world, 1)      # the ranks of one node pin at the same time
        while nb > 1 and avail and 2 * per_seq * nb + (8 << 30) > avail:     # an unpinned copy exists while pinning
            nb //= 2
            why = f"host memory: {avail / 2**30:.0f} GiB available"
    pin = lambda t: None if t is None else t[:nb].cpu().pin_memory()
    target, cand, unif = pin(inp.target), pin(inp.cand), pin(inp.unif)
    draft = pin(inp.draft) if w.temperature > 0 else None
    out = {"accept_len": torch.empty(nb, dtype=torch.int32).pin_memory(),
           "tokens": torch.empty((nb, st["gamma"] + 1), dtype=torch.int32).pin_memory(),
           "residual": torch.empty((nb, w.vocab), dtype=torch.float32).pin_memory(),
           "status": torch.zeros(nb, dtype=torch.int32).pin_memory()}
    h2d = sum(t.numel() * t.element_size() for t in (target, draft, cand, unif) if t is not None)
    d2h = sum(t.numel() * t.element_size() for t in out.values())

    def step():
        binding.mcsd_verify_host(target, draft, inp.parent, cand, unif, w.temperature, w.mode, out=out)

    step()                              # the first call allocates the staging buffers the library then keeps
    steps = max(1, min(args.steps, args.e2e_steps))
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()                      # synchronises internally before it returns
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    dt = max_over_ranks(dist, dt, dev)
    binding.mcsd_release_host_staging()
    value = world * nb * st["n_draft"] * steps / dt
    return {"value": value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "ms_per_step": dt / steps * 1e3, "steps": steps, "batch": nb, "batch_reason": why,
            "h2d_gbs": h2d * steps / dt / 1e9,
            "note": "mcsd_verify_host on pinned host buffers; copies in both directions and kernels inside the timed "
                    "region (the library's device staging buffers are allocated by the untimed first call); bound by "
                    "the host link: h2d_gbs is what the copies achieved"}


# ----------------------------------------------------------------------------- sweep
def sweep_points_done(path: str):
    """Names of the sweep points a (possibly cut-off) output file already holds; a last line that is
    not whole JSON is ignored."""
    names = set()
    with open(path) as f:
        for line in f:
            try:
                names.add(json.loads(line)["workload"])
            except (ValueError, KeyError):
                pass
    return names


def run_sweep(args):
    """The 300-point throughput sweep (dtype x batch x k-config x sigma x mode at vocabulary
    32000, temperature 1).  Every call is timed on its own between CUDA events with L2
    flushed before it (a 256 MB buffer is overwritten), so small points report their
    cold-cache latency; each point is checked against the oracle on its first sequences.
    Writes one JSON line per point to --sweep-out and prints a summary line per point."""
    from paper_2401_06706_b200 import binding
    import oracle
    from oracle import compare
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    binding.load_library()
    peak, peak_kind = measured_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    if args.named:
        # the named configurations 1 to 4 (the latency-bound ones), parity on every sequence
        points = [w for name, w in synth.named_workloads().items() if name != "cfg5_largest" and args.sweep_filter in name]
    else:
        points = [w for w in synth.sweep_workloads() if args.sweep_filter in w.name]
    # --sweep-resume: points already in the output file (one JSON line each, written as they finish) are
    # skipped, so an interrupted sweep goes on where it stopped
    done = set()
    if args.sweep_out and args.sweep_resume and os.path.exists(args.sweep_out):
        done = sweep_points_done(args.sweep_out)
        points = [w for w in points if w.name not in done]
        print(f"resuming: {len(done)} points found in {args.sweep_out}, {len(points)} left", flush=True)
    out = open(args.sweep_out, "a" if done else "w") if args.sweep_out else None
    for w in points:
        inp = synth.make_inputs(w, dev)
        st = inp.stats
        ver = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[w.dtype], dev)
        for _ in range(5):
            ver.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, w.temperature, w.mode)
        # back to back, inputs resident in L2 where they fit: what a decoding loop that verifies the
        # logits it has just produced sees
        torch.cuda.synchronize()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record()
        for _ in range(args.sweep_hot_calls):
            ver.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, w.temperature, w.mode)
        h1.record()
        torch.cuda.synchronize()
        us_hot = h0.elapsed_time(h1) * 1e3 / max(args.sweep_hot_calls, 1)
        # the same call captured in a CUDA graph and replayed: the chain of kernels on the GPU without
        # the host's share (the call neither allocates nor synchronises, so it can be captured)
        us_graph = None
        if args.named:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                ver.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, w.temperature, w.mode)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                ver.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, w.temperature, w.mode)
            graph.replay()
            torch.cuda.synchronize()
            h0.record()
            for _ in range(args.sweep_hot_calls):
                graph.replay()
            h1.record()
            torch.cuda.synchronize()
            us_graph = h0.elapsed_time(h1) * 1e3 / max(args.sweep_hot_calls, 1)
            del graph
        times = []
        for _ in range(args.sweep_calls):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ver.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, w.temperature, w.mode)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        med, best = statistics.median(times), min(times)
        n_par = w.batch if args.named else min(w.batch, args.sweep_parity_seqs)
        # cpu_baseline leg of the point: the oracle on its first sequences, timed; its output is
        # what the kernels' output is compared with
        t, d, c, u = inp.host_f32(0, n_par)
        t_cpu0 = time.time()
        ref = oracle.verify(t, d, inp.parent, c, u, w.temperature, w.mode)
        t_cpu = time.time() - t_cpu0
        rep = compare.compare(t, d, inp.parent, c, u, w.temperature, w.mode, w.dtype, oracle_result=ref,
                              accept_len=ver.accept_len[:n_par].cpu().numpy(), tokens=ver.tokens[:n_par].cpu().numpy(),
                              residual=ver.residual[:n_par].cpu().numpy(), status=ver.status[:n_par].cpu().numpy())
        algo = inp.logit_bytes() + 12 * w.batch * st["n_nodes"]
        rec = {"workload": w.name, "dtype": w.dtype, "batch": w.batch, "kconfig": w.kconfig, "sigma": w.draft_sigma,
               "mode": w.mode, "temperature": w.temperature, "vocab": w.vocab, "algorithmic_mb": algo / 1e6,
               "us_median": med * 1e3, "us_min": best * 1e3, "us_back_to_back": us_hot, "us_graph_replay": us_graph,
               "launches_per_call": binding.mcsd_last_launch_count(),
               "nodes_per_s": w.batch * st["n_draft"] / (med * 1e-3), "gbs": algo / (med * 1e-3) / 1e9,
               "frac_of_peak": algo / (med * 1e-3) / 1e9 / peak, "peak_kind": peak_kind,
               "regime": "hbm" if algo > 4 * 126e6 else "latency/L2-bound point (inputs < 4x L2)",
               "accept_len_mean": float(ver.accept_len.float().mean().item()), "parity_ok": rep.ok,
               "parity": rep.summary(),
               "cpu_baseline": {"value": n_par * st["n_draft"] / max(t_cpu, 1e-9), "unit": UNIT, "cores": oracle.num_threads(),
                                "kind": "oracle", "sample": f"first {n_par} sequences, {t_cpu:.3f} s wall"}}
        if out:
            out.write(json.dumps(rec) + "\n")
            out.flush()
        print(f"{w.name:40s} {rec['algorithmic_mb']:9.1f} MB {rec['us_median']:9.1f} us (hot {us_hot:7.1f}, graph "
              f"{us_graph if us_graph is not None else float('nan'):6.1f}) {rec['gbs']:7.0f} GB/s "
              f"{rec['frac_of_peak']:.3f} tau-1={rec['accept_len_mean']:.2f} parity={'ok' if rep.ok else 'FAIL'}", flush=True)
        del inp, ver
        torch.cuda.empty_cache()
    if out:
        out.close()


def run_stage(args):
    """--stage sample / greedy: one kernel of the wider path on the same workload, one GPU, device
    timed.  sample: mcsd_sample_candidates over all internal nodes (the draft rows once); greedy:
    the verification step at temperature 0 (argmax kernel; the target rows once).  One JSON line."""
    from paper_2401_06706_b200 import binding
    from dataclasses import replace
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (no CPU fallback for the product path)"
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    binding.load_library()
    w = pick_workload(args.workload, args.batch, args.logit_dtype)
    if args.stage == "greedy":
        w = replace(w, temperature=0.0)
    inp = synth.make_inputs(w, dev)
    st = inp.stats
    esize = inp.target.element_size()
    if args.stage == "sample":
        gen = torch.Generator(device=dev)
        gen.manual_seed(w.seed)
        u = synth.open_uniforms((w.batch, st["n_nodes"]), gen, dev)
        cand = torch.full((w.batch, st["n_nodes"]), -1, dtype=torch.int32, device=dev)
        call = lambda: binding.mcsd_sample_candidates(inp.draft, inp.parent, u, w.temperature, w.mode, cand=cand)
        algo = w.batch * st["n_internal"] * w.vocab * esize + 8 * w.batch * st["n_draft"]
        units, metric, unit, kernel = w.batch * st["n_draft"], "sampled_candidate_tokens_per_sec", "tokens/s", "sample_kernel"
    else:
        ver = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[w.dtype], dev, node_outputs=True)
        call = lambda: ver.mcsd_verify_nodes(inp.target, None, inp.cand, None, 0.0, w.mode)
        algo = w.batch * st["n_nodes"] * w.vocab * esize + 4 * w.batch * st["n_nodes"]
        units, metric, unit, kernel = w.batch * st["n_draft"], METRIC, UNIT, "argmax_kernel"
    for _ in range(max(args.warmup, 3)):
        call()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.25)
    torch.cuda.synchronize()
    t_host0 = time.time()
    for e0, e1 in ev:
        e0.record()
        call()
        e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop(t_host0, time.time())
    ms = [a.elapsed_time(b) for a, b in ev]
    ms_avg = sum(ms) / len(ms)
    peak, peak_kind = measured_peaks()
    achieved = algo / (ms_avg * 1e-3) / 1e9
    # CPU baseline leg: the oracle of this stage, as it stands, timed on a bounded sample of the same
    # inputs; what it computed also serves to check the kernel's output on those sequences
    cpu_baseline, parity = None, None
    if not args.no_cpu_baseline:
        import oracle
        n_seq = min(w.batch, args.oracle_seqs if args.stage == "greedy" else max(8, args.oracle_seqs // 8))
        if args.stage == "sample":
            from oracle import compare as cmp
            d_h, u_h = inp.draft[:n_seq].to(torch.float32).cpu().numpy(), u[:n_seq].cpu().numpy()
            t0 = time.time()
            oracle.sample(d_h, inp.parent, u_h, w.temperature, w.mode)
            t1 = time.time()
            rep = cmp.compare_samples(d_h, inp.parent, u_h, w.temperature, w.mode, cand[:n_seq].cpu().numpy(), 0, None)
            parity = {"sequences": n_seq, "draws": rep.n_draws, "tolerated": rep.n_tolerated, "ok": bool(rep.ok)}
        else:
            t, _, c, uu = inp.host_f32(0, n_seq)
            t0 = time.time()
            ref = oracle.verify(t, None, inp.parent, c, uu, 0.0, w.mode, want_residual=False)
            t1 = time.time()
            got = ver.node_accept[:n_seq].cpu().numpy()
            parity = {"sequences": n_seq, "nodes": int(got.size), "ok": bool((got == ref.node_accept).all())}
        cpu_baseline = {"value": n_seq * st["n_draft"] / max(t1 - t0, 1e-9), "unit": unit, "cores": oracle.num_threads(),
                        "kind": "oracle", "sample": f"first {n_seq} of {w.batch} sequences of the same inputs, "
                                                      f"{t1 - t0:.2f} s wall"}
    line = {"metric": metric, "value": units / (ms_avg * 1e-3), "unit": unit, "n_gpus": 1, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_avg, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "stage": args.stage,
            "config": workload_config(w, st, l2="inputs far larger than the 126 MB L2" if algo > 4 * 126e6 else "inputs not much larger than L2"),
            "roofline": {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak, "peak_kind": f"of {peak_kind}",
                         "unit": "GB/s", "frac": achieved / peak, "algorithmic_bytes_per_launch": algo,
                         "kernel_ms_avg": ms_avg, "kernel_ms_min": min(ms), "traffic": None},
            "cpu_baseline": cpu_baseline, "gpu_launches": args.steps, "clocks": clocks,
            "parity_on_oracle_sample": parity}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="cfg5_largest")
    ap.add_argument("--oracle-seqs", type=int, default=256,
                    help="sequences of the workload the CPU oracle is timed on")
    ap.add_argument("--e2e-batch", type=int, default=0,
                    help="sequences per end-to-end step (0: the whole batch if the host has the memory to pin it)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--sustained-steps", type=int, default=300,
                    help="further steps after the timed region for the sustained-clock record (0: none)")
    ap.add_argument("--no-half", action="store_true", help="skip the sub-record with 2-byte logits")
    ap.add_argument("--batch", type=int, default=0, help="override the batch of the workload (profiling)")
    ap.add_argument("--logit-dtype", default="", choices=["", "fp32", "bf16", "fp16"],
                    help="override the logit type of the workload (profiling)")
    ap.add_argument("--form", default="all_node", choices=["all_node", "path"],
                    help="all_node: every node of every tree is evaluated (the measured configuration); "
                         "path: mcsd_verify_path, only the nodes the walks visit, one launch per level")
    ap.add_argument("--stage", default="verify", choices=["verify", "sample", "greedy"],
                    help="verify: the bench line of the verification step (default); sample: time the candidate "
                         "sampler on the workload's draft rows; greedy: the verification step at temperature 0")
    ap.add_argument("--sweep", action="store_true", help="run the throughput sweep instead of the bench line")
    ap.add_argument("--sweep-filter", default="", help="only sweep points whose name contains this text")
    ap.add_argument("--sweep-out", default="", help="file for one JSON line per sweep point")
    ap.add_argument("--sweep-resume", action="store_true", help="skip the points --sweep-out already holds")
    ap.add_argument("--named", action="store_true",
                    help="with --sweep: the named configurations 1 to 4 instead of the sweep points, parity on every sequence")
    ap.add_argument("--sweep-calls", type=int, default=20)
    ap.add_argument("--sweep-hot-calls", type=int, default=100)
    ap.add_argument("--sweep-parity-seqs", type=int, default=16)
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.sweep:
        raise SystemExit(spawn_ranks(args))
    if args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.stage != "verify":
        run_stage(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
