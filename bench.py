#!/usr/bin/env python
"""Benchmark of the CSD verification step (csd_step: verify + memory update, one launch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" is one pass of the whole hot path over one synthetic batch: the streaming
max/arg-max/sum-exp over logits[B,K+1,V], the match test, the OCM look-up, the gate of
Eq. 3, the prefix scan, and the memory update.  Rank 0 prints ONE JSON line:

  value     verified draft positions per second (B*K*steps / time), inputs resident in HBM,
            timed with CUDA events on the launching stream, max over ranks;
  e2e       the same metric through csd_step_host: logits and draft in pinned host memory,
            host->device and device->host copies inside the timed region;
  roofline  achieved logit bytes per second of the step kernel against the measured HBM copy
            bandwidth of this machine;
  cpu_baseline  the CPU oracle timed on this machine's cores on a bounded sample of the workload.

With N > 1 every rank runs an independent replica (own batch, own memory): the path has no
exchange step, so there is no data-path collective; torch.distributed only carries the
barrier and the max over ranks of the elapsed time.
"""

from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verified_draft_positions_per_sec"
UNIT = "positions/s"
FALLBACK_HBM_GBS = 6650.0            # earlier measurement on this machine, used when no measured file exists
DEFAULT_WORKLOAD = "large_batch"
# DRAM bytes per launch of the step kernel from an ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum); a workload is absent where no capture of the current kernel exists.
NCU_TRAFFIC_BYTES = {"large_batch": 596126208, "ocm_contention": 140787712, "batched_serving": 58522880}
# the same for the LM-head GEMM kernels at H = 4096 (profiles/lmhead_stats_kernel_batched_serving_h4096.md), by workload
NCU_TRAFFIC_BYTES_LMHEAD = {"batched_serving": 1252566000 + 4133120, "single_stream": 1051026000 + 3639040}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def workload_config(wl, tau, extra=None):
    cfg = {"workload": f"{wl.name}: B={wl.B} K={wl.K} V={wl.V} {wl.dtype} logits, OCM {wl.ocm_slots} slots, "
                       f"lambda={wl.lam}, tau={tau}",
           "B": wl.B, "K": wl.K, "V": wl.V, "ocm_slots": wl.ocm_slots, "tau": tau, "lambda": wl.lam,
           "logit_bytes_per_step": wl.logit_bytes}
    if extra:
        cfg.update(extra)
    return cfg


def reduce_over_ranks(seconds: float, units: float, dist=None, device=None):
    """Whole-job figures from per-rank ones: elapsed = max over ranks, units = sum over ranks."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return seconds, units
    import torch
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# ---------------------------------------------------------------------------------------
# clocks during the timed region (read-only NVML queries)
# ---------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, device_index: int, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self._nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None
        self.period = period_s

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ---------------------------------------------------------------------------------------
# the CPU oracle leg (also the whole of --impl reference)
# ---------------------------------------------------------------------------------------
class OracleRunner:
    """The CPU oracle on `rows_b` batch rows of the workload (CPU-generated inputs, seed 0)."""

    def __init__(self, wl, tau, rows_b):
        import dataclasses
        from oracle import csd_oracle, row_stats_c
        from synth_inputs import Synth, logits_bits_numpy
        self.o, self.rs = csd_oracle, row_stats_c
        self.wl = dataclasses.replace(wl, B=rows_b)
        self.tau = tau
        self.cores = row_stats_c.max_threads()
        syn = Synth(self.wl, 0, "cpu")
        self.mem = csd_oracle.OCM(wl.ocm_slots, wl.lam)
        self.inputs = []
        for s in range(2):
            z, d = syn.step(s)
            raw, is_bits = logits_bits_numpy(z)
            vals = csd_oracle.bf16_bits_to_f64(raw).astype("float32") if is_bits else raw
            self.inputs.append((vals, raw, is_bits, d.numpy()))
        self.done = 0

    def step(self):
        vals, raw, is_bits, d = self.inputs[self.done % 2]
        stats = self.rs.row_stats_batch(raw, is_bf16_bits=is_bits)
        self.o.step(vals, d, self.mem, self.tau, stats=stats)
        self.done += 1

    def timed(self, n):
        t0 = time.perf_counter()
        for _ in range(n):
            self.step()
        return time.perf_counter() - t0


def oracle_row_seconds(wl, tau):
    """Seconds the oracle needs per batch row of this workload (calibration on a few rows)."""
    rows = min(wl.B, 4)
    r = OracleRunner(wl, tau, rows)
    r.timed(1)
    return r.timed(2) / (2 * rows)


def time_oracle(wl, tau, budget_s=15.0):
    """Oracle positions/s on the host cores over a bounded sample of the workload."""
    t_row = oracle_row_seconds(wl, tau)
    rows_b = wl.B if t_row * wl.B <= budget_s / 3 else max(1, int(budget_s / 3 / t_row))
    n = max(2, min(200, int(budget_s / (t_row * rows_b))))
    r = OracleRunner(wl, tau, rows_b)
    sec = r.timed(n)
    return {"steps": n, "rows_b": rows_b, "seconds": sec, "positions_per_s": rows_b * wl.K * n / sec, "cores": r.cores}


def run_reference(args, wl, tau):
    """--impl reference: the oracle as it stands, timed on the host cores.  Each bench step
    is one oracle step over a bounded number of batch rows, sized so that the whole run
    (warm-up included) stays near two minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    t_row = oracle_row_seconds(wl, tau)
    total = args.steps + args.warmup
    rows_b = max(1, min(wl.B, int(120.0 / (total * t_row))))
    r = OracleRunner(wl, tau, rows_b)
    r.timed(args.warmup)
    sec = r.timed(args.steps)
    value = rows_b * wl.K * args.steps / sec
    sample = f"each step = the oracle on {rows_b} of the workload's {wl.B} batch rows (K+1 logit rows each)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sec / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(wl, tau),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": r.cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------
# the GPU leg
# ---------------------------------------------------------------------------------------
class Bench:
    """One workload's resident inputs, memory and buffers, and the launch plans that replay them."""

    def __init__(self, wl, tau, device, seed=0):
        import torch
        import paper_2604_13634_b200 as pkg
        from synth_inputs import Synth
        self.torch, self.pkg, self.wl, self.tau = torch, pkg, wl, tau
        self.device = device
        l2 = torch.cuda.get_device_properties(device).L2_cache_size
        self.ring_len = max(2, math.ceil(2 * l2 / wl.logit_bytes) + 1)
        syn = Synth(wl, seed, device)
        self.ring = [syn.step(s) for s in range(self.ring_len)]
        self.ocm = pkg.Ocm(wl.ocm_slots, wl.lam, device.index)
        kind, n = wl.prewarm
        if kind == "pairs":
            self.ocm.update(*syn.prewarm_pairs(n))
        self.buf = pkg.StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, device=device)
        if kind == "steps":
            for s in range(n):
                z, d = self.ring[s % self.ring_len]
                pkg.csd_step(z, d, self.ocm, tau, self.buf)
        torch.cuda.synchronize(device)
        self.plan = None          # [(graph, replays)], together exactly the planned number of steps
        self.plan_steps = 0
        self.plan_label = "eager"

    def step(self, i):
        z, d = self.ring[i % self.ring_len]
        self.pkg.csd_step(z, d, self.ocm, self.tau, self.buf)

    def _graph_of(self, n):
        torch = self.torch
        side = torch.cuda.Stream(self.device)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            self.step(0)              # outside the capture: first-use set-up (a workspace clear) must not be captured
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(n):
                self.step(i)
        return g

    def plan_steps_exactly(self, steps, graph_steps=48):
        """CUDA graphs that together enqueue EXACTLY `steps` steps: as many replays of one graph of about
        `graph_steps` steps as fit (consecutive steps overlap only inside one graph launch, so a short graph
        spends a large share of its time on its own start and drain), plus one shorter graph for the rest."""
        replays = max(1, steps // max(1, graph_steps))
        per = steps // replays
        rest = steps - per * replays
        self.plan = [(self._graph_of(per), replays)]
        self.plan_label = f"CUDA graph of {per} steps replayed {replays}x"
        if rest:
            self.plan.append((self._graph_of(rest), 1))
            self.plan_label += f" + one graph of {rest} steps"
        self.plan_steps = steps

    def run(self, steps):
        """Enqueue `steps` steps through the plan (which must have been made for that count), else eagerly."""
        if self.plan is not None and steps == self.plan_steps:
            for g, n in self.plan:
                for _ in range(n):
                    g.replay()
            return
        for i in range(steps):
            self.step(i)

    def launch_label(self, steps):
        return self.plan_label if (self.plan is not None and steps == self.plan_steps) else "eager"

    def timed(self, steps):
        torch = self.torch
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        self.run(steps)
        b.record()
        b.synchronize()
        return a.elapsed_time(b) * 1e-3


def repeats_for(region_s, floor=7, target_s=0.25, cap=201):
    """How often the timed region is repeated: at least `floor` times, more while the whole stays near
    `target_s` (a region of a few milliseconds alone would see one clock sample)."""
    if region_s <= 0:
        return floor
    return int(max(floor, min(cap, math.ceil(target_s / region_s))))


def read_stream_gbs(device):
    """Context for the roofline: a read-only stream (torch.sum over 2 GiB of fp32, best of 5) next to the
    read+write copy that MEASURED_PEAKS.json holds."""
    import torch
    x = torch.empty(1 << 29, dtype=torch.float32, device=device).normal_()
    best = 0.0
    for _ in range(6):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        x.sum()
        b.record()
        b.synchronize()
        best = max(best, x.numel() * 4 / (a.elapsed_time(b) * 1e-3) / 1e9)
    del x
    torch.cuda.empty_cache()
    return best


def standalone_us(pkg, bench, steps=96):
    """Latency of a step that runs alone: overlap off (stream-ordered launches, the 4-blocks-per-SM shape),
    a graph of `steps` steps over the ring, median of 7 replays."""
    import torch
    pkg.csd_set_overlap(False)
    try:
        bench.plan_steps_exactly(steps, steps)
        bench.run(steps)
        torch.cuda.synchronize(bench.device)
        return 1e6 * statistics.median(bench.timed(steps) for _ in range(7)) / steps
    finally:
        bench.plan = None


def time_e2e(wl, tau, device, steps):
    """csd_step_host: pinned host inputs, copies inside the timed region."""
    import torch
    import paper_2604_13634_b200 as pkg
    from synth_inputs import Synth
    syn = Synth(wl, 0, device)
    host = []
    for s in range(2):
        z, d = syn.step(s)
        host.append((z.cpu().pin_memory(), d.cpu().pin_memory()))
    del z, d
    ocm = pkg.Ocm(wl.ocm_slots, wl.lam, device.index)
    hs = pkg.HostStep(wl.B, wl.K, wl.V, wl.torch_dtype, device=device)
    for i in range(2):
        hs(*host[i % 2], ocm, tau)
    torch.cuda.synchronize(device)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(steps):
        hs(*host[i % 2], ocm, tau)
    b.record()
    b.synchronize()
    sec = a.elapsed_time(b) * 1e-3
    ocm.close()
    h2d = wl.logit_bytes + wl.B * wl.K * 4
    d2h = wl.B * 8 + wl.B * wl.K
    return {"value": wl.B * wl.K * steps / sec, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "steps": steps, "ms_per_step": 1e3 * sec / steps}


def run_ours(args, wl, tau):
    import torch
    import torch.distributed as dist

    import paper_2604_13634_b200 as pkg

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path")
    pkg.lib()
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    overlap = not args.no_overlap
    pkg.csd_set_overlap(overlap)
    pkg.csd_set_tuning(args.chunk_bytes, args.ctas_per_sm, args.block_threads)
    bench = Bench(wl, tau, device, seed=rank)
    if not args.eager:
        bench.plan_steps_exactly(args.steps, args.graph_steps)
    warm = max(args.warmup, 3)
    for i in range(warm):                 # warm-up steps are launched one by one
        bench.step(i)
    bench.run(args.steps)                 # and the plan itself once
    torch.cuda.synchronize(device)

    # the timed region (exactly --steps steps, barrier + synchronize on both sides, max over ranks) is
    # taken several times back to back; the line reports the median region
    probe = bench.timed(args.steps)
    repeats = args.repeats if args.repeats > 0 else repeats_for(probe)
    sampler = ClockSampler(local, period_s=0.005)
    sampler.start()
    regions = []
    for _ in range(repeats):
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(device)
        sec_r = bench.timed(args.steps)
        torch.cuda.synchronize(device)
        if world > 1:
            dist.barrier()
        sec_r, positions = reduce_over_ranks(sec_r, wl.B * wl.K * args.steps, dist if world > 1 else None, device)
        regions.append(sec_r)
    clocks = sampler.stop()
    sec = statistics.median(regions)
    launch = bench.launch_label(args.steps)

    st = bench.ocm.stats()
    e2e = time_e2e(wl, tau, device, steps=max(3, min(args.steps, args.e2e_steps)))
    if world > 1:
        _, e2e["value"] = reduce_over_ranks(0.0, e2e["value"], dist, device)

    if rank == 0:
        peak, peak_kind = measured_peak()
        per_launch_s = sec / args.steps
        achieved = wl.logit_bytes / per_launch_s / 1e9
        shape = pkg.csd_launch_shape(wl.B, wl.K, wl.V, 0 if wl.dtype == "f32" else 1)
        line = {
            "metric": METRIC, "value": positions / sec, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": 1e3 * sec / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "repeats": repeats, "value_min": positions / max(regions), "value_max": positions / min(regions),
            "region_ms": {"median": 1e3 * sec, "min": 1e3 * min(regions), "max": 1e3 * max(regions)},
            "config": workload_config(wl, tau, {
                "steps_per_s": args.steps * world / sec, "parallelism": f"replicas x{world}",
                "l2_policy": f"ring of {bench.ring_len} distinct step inputs "
                             f"({bench.ring_len * wl.logit_bytes / 1e6:.0f} MB, > 2x L2)",
                "launch": launch,
                "timing": f"the region of exactly {args.steps} steps timed {repeats} times back to back; value = median",
                "step_overlap": "off" if not overlap else
                                "programmatic dependent launch, one block per SM and launch: a step streams its "
                                "logits while the steps before it finish",
                "kernel_shape": shape}),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": NCU_TRAFFIC_BYTES.get(wl.name), "peak_source": f"of {peak_kind}",
                         "peak_kind": "read+write copy; this kernel only reads, so a fraction slightly above 1 is possible",
                         "kernel": "csd_step_kernel", "bytes_per_launch": wl.logit_bytes,
                         "frac_of_nominal_8TBs": achieved / 8000.0},
            "e2e": e2e, "gpu_launches": args.steps, "clocks": clocks,
            "ocm": {k: st[k] for k in ("n_keys", "n_dropped", "steps", "matches", "rescues", "rejections", "flags")},
        }
        if world == 1 and not args.lean:
            line["roofline"]["read_stream_GBs_torch_sum"] = read_stream_gbs(device)
            us = standalone_us(pkg, bench)
            line["roofline"]["single_step"] = {
                "us_per_step": us, "achieved": wl.logit_bytes / us / 1e3, "frac": wl.logit_bytes / us / 1e3 / peak,
                "what": "a step that runs alone: overlap off, stream-ordered launches, 4 blocks per SM"}
            pkg.csd_set_overlap(overlap)
        if not args.no_cpu_baseline and world == 1:
            r = time_oracle(wl, tau)
            line["cpu_baseline"] = {"value": r["positions_per_s"], "unit": UNIT, "cores": r["cores"], "kind": "oracle",
                                    "sample": f"{r['steps']} oracle steps over {r['rows_b']} of the workload's {wl.B} "
                                              f"batch rows (CPU-generated inputs, same recipe) in {r['seconds']:.1f} s"}
        bench.ocm.close()
        del bench
        torch.cuda.empty_cache()
        if world == 1 and not args.lean:
            names = ("batched_serving", "large_batch", "ocm_contention") + (("single_stream", "tiny") if args.extras else ())
            line["other_workloads"] = run_extras(device, wl.name, peak, names, overlap)
            try:
                line["sampled"] = measure_sampled(args, wl, tau, device, graph_steps=16, min_steps=48, count_draws=True)
            except Exception as e:             # the greedy line stands on its own
                line["sampled"] = {"error": repr(e)}
            try:
                from synth_inputs import WORKLOADS
                torch.cuda.empty_cache()
                line["multi_stream"] = measure_multi_stream(WORKLOADS["batched_serving"], 0.3, device)
                pkg.csd_set_overlap(overlap)
            except Exception as e:
                line["multi_stream"] = {"error": repr(e)}
            try:
                torch.cuda.empty_cache()
                line["early_exit"] = measure_early_exit(wl, tau, device)
                pkg.csd_set_overlap(overlap)
            except Exception as e:
                line["early_exit"] = {"error": repr(e)}
            try:
                from synth_inputs import WORKLOADS
                torch.cuda.empty_cache()
                line["lmhead"] = measure_lmhead(WORKLOADS["batched_serving"], 0.3, device)
                torch.cuda.empty_cache()
                line["lmhead"]["single_stream"] = measure_lmhead(WORKLOADS["single_stream"], 0.3, device)
                pkg.csd_set_overlap(overlap)
            except Exception as e:
                line["lmhead"] = {"error": repr(e)}
        print(json.dumps(line), flush=True)
    else:
        bench.ocm.close()
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------
# --mode sampled: the stochastic verification step (Algorithm 1 at T > 0), a separate line
# ---------------------------------------------------------------------------------------
def measure_sampled(args, wl, tau, device, graph_steps, min_steps, count_draws=True):
    """csd_step_sampled (statistics + decision, races + finalisation, memory update) over a ring of resident
    inputs.  Algorithmic bytes per step: every row of the target and draft logits once, the two rows of
    every position whose residual draw a row needs once more, and the bonus row of every fully accepted
    batch row once more."""
    import torch

    import paper_2604_13634_b200 as pkg
    from synth_inputs import Synth

    T = args.temperature
    syn = Synth(wl, 0, device)
    step_bytes = (wl.rows + wl.B * wl.K) * wl.V * wl.elt_bytes
    l2 = torch.cuda.get_device_properties(device).L2_cache_size
    ring_len = max(2, math.ceil(2 * l2 / step_bytes) + 1)
    ring = [syn.step_sampled(s) for s in range(ring_len)]
    ocm = pkg.Ocm(wl.ocm_slots, wl.lam, device.index)
    kind, n = wl.prewarm
    if kind == "pairs":
        ocm.update(*syn.prewarm_pairs(n))
    diag_buf = pkg.SampledBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, device=device, diag=True)
    for i, (z, y, d, r) in enumerate(ring):                 # warms the memory up
        pkg.csd_step_sampled(z, y, d, r, 1000 + i, T, ocm, tau, diag_buf)
    buf = pkg.SampledBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, device=device, diag=False)

    def step(i):
        z, y, d, r = ring[i % ring_len]
        pkg.csd_step_sampled(z, y, d, r, 1000 + i % ring_len, T, ocm, tau, buf)

    graph_steps = ring_len * max(1, math.ceil(graph_steps / ring_len))
    side = torch.cuda.Stream(device)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step(0)
    torch.cuda.current_stream().wait_stream(side)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(graph_steps):
            step(i)
    steps = max(graph_steps, min_steps - min_steps % graph_steps)
    for _ in range(max(1, math.ceil(max(args.warmup, 3) / graph_steps))):
        g.replay()
    torch.cuda.synchronize(device)
    sampler = ClockSampler(device.index, period_s=0.005)
    sampler.start()
    regions = []
    for _ in range(7):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps // graph_steps):
            g.replay()
        b.record()
        b.synchronize()
        regions.append(a.elapsed_time(b) * 1e-3)
    clocks = sampler.stop()
    sec = statistics.median(regions)
    # how many draws a step makes depends on the memory (rescues let rows go on): counted on one more pass
    # over the ring with the memory as the timed region left it
    failed, draws, bonus = [], [], []
    for i, (z, y, d, r) in enumerate(ring):
        pkg.csd_step_sampled(z, y, d, r, 1000 + i, T, ocm, tau, diag_buf)
        failed.append(int((diag_buf.diag["accepted"] == 0).sum().item()))
        draws.append(int((diag_buf.diag["t_star"] >= 0).sum().item()))
        bonus.append(int((diag_buf.diag["bonus"] >= 0).sum().item()))
    mean = lambda v: sum(v) / len(v)
    # every row of z and y once; z and y again for each residual draw made; z again for each bonus draw made
    rows_per_step = wl.rows + wl.B * wl.K + 2 * mean(draws) + mean(bonus)
    algo_bytes = rows_per_step * wl.V * wl.elt_bytes
    peak, peak_kind = measured_peak()
    achieved = algo_bytes * steps / sec / 1e9
    st = ocm.stats()
    ocm.close()
    launches = pkg.sampled_launches_per_step(wl.B, wl.K, wl.V, wl.torch_dtype)
    return {"positions_per_s": wl.B * wl.K * steps / sec, "us_per_step": 1e6 * sec / steps, "steps": steps, "repeats": 7,
            "temperature": T, "achieved_GBs": achieved, "frac": achieved / peak, "peak_source": f"of {peak_kind}",
            "algorithmic_bytes_per_step": algo_bytes, "failed_positions_per_step": mean(failed),
            "residual_draws_per_step": mean(draws), "bonus_draws_per_step": mean(bonus),
            "launches_per_step": launches, "launch": f"CUDA graph of {graph_steps} steps replayed",
            "ring_len": ring_len, "step_bytes": step_bytes, "clocks": clocks,
            "ocm": {k: st[k] for k in ("n_keys", "n_dropped", "steps", "matches", "rescues", "rejections", "flags")}}


def run_sampled(args, wl, tau):
    """--mode sampled: the stochastic verification step (Algorithm 1 at T > 0) as a bench line of its own."""
    import torch

    import paper_2604_13634_b200 as pkg
    from synth_inputs import Synth

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path")
    pkg.lib()
    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    pkg.csd_set_overlap(not args.no_overlap)     # a step's statistics kernel may run beside the previous step's tail
    m = measure_sampled(args, wl, tau, device, graph_steps=args.graph_steps, min_steps=args.steps)
    T = args.temperature
    line = {"metric": METRIC, "value": m["positions_per_s"], "unit": UNIT, "n_gpus": 1, "steps": m["steps"],
            "warmup": max(args.warmup, 3), "ms_per_step": m["us_per_step"] * 1e-3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic", "repeats": m["repeats"],
            "config": workload_config(wl, tau, {
                "mode": f"stochastic verification (Algorithm 1 at T={T}): acceptance test, residual and bonus draws",
                "draft_logits": "target logits + N(0, 0.3^2), the draft token raised to the row maximum + 1",
                "l2_policy": f"ring of {m['ring_len']} distinct step inputs ({m['ring_len'] * m['step_bytes'] / 1e6:.0f} MB, > 2x L2)",
                "launch": m["launch"] + f" ({m['launches_per_step']} launches per step)",
                "failed_positions_per_step": m["failed_positions_per_step"],
                "residual_draws_per_step": m["residual_draws_per_step"],
                "bonus_draws_per_step": m["bonus_draws_per_step"]}),
            "roofline": {"bound": "hbm", "achieved": m["achieved_GBs"], "peak": measured_peak()[0], "unit": "GB/s",
                         "frac": m["frac"], "traffic": None, "peak_source": m["peak_source"],
                         "kernel": "sampled_stats_kernel + sampled_race_kernel (whole step)",
                         "bytes_per_launch": m["algorithmic_bytes_per_step"]},
            "gpu_launches": m["launches_per_step"] * m["steps"], "clocks": m["clocks"], "ocm": m["ocm"]}
    if not args.no_cpu_baseline:
        import dataclasses
        from oracle import csd_sampled_oracle as so
        from synth_inputs import logits_to_numpy
        rows_b = min(wl.B, 2)
        small = dataclasses.replace(wl, B=rows_b)
        z, y, d, r = Synth(small, 0, "cpu").step_sampled(0)
        zz, yy = logits_to_numpy(z).astype("float64"), logits_to_numpy(y).astype("float64")
        mem = so.OCM(wl.ocm_slots, wl.lam)
        t0 = time.perf_counter()
        n = 0
        while time.perf_counter() - t0 < 10.0:
            so.step(zz, yy, d.numpy(), r.numpy(), n, T, mem, tau)
            n += 1
        secs = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": rows_b * wl.K * n / secs, "unit": UNIT, "cores": 1, "kind": "oracle",
                                "sample": f"{n} oracle steps over {rows_b} of the workload's {wl.B} batch rows in {secs:.1f} s"}
    print(json.dumps(line), flush=True)


def measure_early_exit(wl, tau, device, steps=48):
    """csd_step_early_exit (the step in two phases: batch rows that stop within the first phase are not read any
    further) as a stream-ordered graph over the ring, beside csd_step run the same way; the bytes it reads follow
    from how many batch rows survive the first phase."""
    import torch

    import paper_2604_13634_b200 as pkg
    from synth_inputs import Synth

    l2 = torch.cuda.get_device_properties(device).L2_cache_size
    ring_len = max(2, math.ceil(2 * l2 / wl.logit_bytes) + 1)
    syn = Synth(wl, 0, device)
    ring = [syn.step(s) for s in range(ring_len)]
    pkg.csd_set_overlap(False)

    def prepared():
        ocm = pkg.Ocm(wl.ocm_slots, wl.lam, device.index)
        if wl.prewarm[0] == "pairs":
            ocm.update(*syn.prewarm_pairs(wl.prewarm[1]))
        return ocm

    def graph_time(call):
        side = torch.cuda.Stream(device)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(ring_len):
                call(i)
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(steps):
                call(i)
        g.replay()
        torch.cuda.synchronize(device)
        ts = []
        for _ in range(7):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            g.replay()
            b.record()
            b.synchronize()
            ts.append(a.elapsed_time(b) * 1e-3 / steps)
        return statistics.median(ts)

    ocm = prepared()
    buf = pkg.EarlyExitBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, first=0, device=device)
    first = min(max(1, (wl.K + 1) // 3), wl.K - 1)
    t_two = graph_time(lambda i: pkg.csd_step_early_exit(*ring[i % ring_len], ocm, tau, buf))
    alive = []
    for i in range(ring_len):                      # with the memory as the timed run left it
        pkg.csd_step_early_exit(*ring[i], ocm, tau, buf)
        alive.append(int((buf.accept_len >= first).sum().item()))
    ocm.close()
    ocm = prepared()
    sb = pkg.StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, device=device)
    t_one = graph_time(lambda i: pkg.csd_step(*ring[i % ring_len], ocm, tau, sb))
    ocm.close()
    mean_alive = sum(alive) / len(alive)
    row_bytes = wl.V * wl.elt_bytes
    read = (wl.B * (first + 1) + mean_alive * (wl.K + 1 - first)) * row_bytes
    peak, kind = measured_peak()
    return {"us_per_step": 1e6 * t_two, "csd_step_alone_us_per_step": 1e6 * t_one, "first_phase_positions": first,
            "batch_rows_alive_after_first_phase": mean_alive, "of_batch_rows": wl.B,
            "logit_bytes_read": read, "logit_bytes_of_csd_step": wl.logit_bytes, "bytes_fraction": read / wl.logit_bytes,
            "achieved_GBs": read / t_two / 1e9, "frac_of_measured_peak": read / t_two / 1e9 / peak, "peak_source": f"of {kind}",
            "launch": f"CUDA graph of {steps} steps (3 launches each), stream-ordered, replayed", "repeats": 7}


def measure_multi_stream(wl, tau, device, n_streams=4, steps=48):
    """n_streams serving streams stepping at the same time on ONE shared memory (csd_ocm_set_shared), each with its
    own workspace and outputs, each replaying its own graph of `steps` steps in the overlap launch shape."""
    import torch

    import paper_2604_13634_b200 as pkg
    from synth_inputs import Synth

    l2 = torch.cuda.get_device_properties(device).L2_cache_size
    ring_len = max(2 * n_streams, math.ceil(2 * l2 / wl.logit_bytes) + 1)
    syn = Synth(wl, 0, device)
    ring = [syn.step(s) for s in range(ring_len)]
    ocm = pkg.Ocm(wl.ocm_slots, wl.lam, device.index)
    if wl.prewarm[0] == "pairs":
        ocm.update(*syn.prewarm_pairs(wl.prewarm[1]))
    ocm.set_shared(True)
    pkg.csd_set_overlap(True)
    streams = [torch.cuda.Stream(device) for _ in range(n_streams)]
    bufs = [pkg.StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, device=device) for _ in range(n_streams)]
    graphs = []
    torch.cuda.synchronize(device)
    for s in range(n_streams):
        off = s * (ring_len // n_streams)
        with torch.cuda.stream(streams[s]):
            pkg.csd_step(*ring[off % ring_len], ocm, tau, bufs[s])             # first use of the workspace, outside the capture
        torch.cuda.synchronize(device)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=streams[s]):
            for i in range(steps):
                pkg.csd_step(*ring[(off + i) % ring_len], ocm, tau, bufs[s])
        graphs.append(g)

    def once():
        torch.cuda.synchronize(device)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for s in range(n_streams):
            streams[s].wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(streams[s]):
                graphs[s].replay()
        for s in range(n_streams):
            torch.cuda.current_stream().wait_stream(streams[s])
        b.record()
        b.synchronize()
        return a.elapsed_time(b) * 1e-3

    once()
    sec = statistics.median(once() for _ in range(7))
    st = ocm.stats()
    torch.cuda.synchronize(device)
    ocm.set_shared(False)
    ocm.close()
    peak, kind = measured_peak()
    total_steps = n_streams * steps
    return {"streams": n_streams, "steps_per_stream": steps, "us_per_step_aggregate": 1e6 * sec / total_steps,
            "positions_per_s": wl.B * wl.K * total_steps / sec, "achieved_GBs": wl.logit_bytes * total_steps / sec / 1e9,
            "frac_of_measured_peak": wl.logit_bytes * total_steps / sec / 1e9 / peak, "peak_source": f"of {kind}", "repeats": 7,
            "launch": f"{n_streams} streams, each a CUDA graph of {steps} steps, replayed together on one shared memory",
            "ocm": {k: st[k] for k in ("n_keys", "n_dropped", "rescues", "rejections", "flags")}}


def measure_lmhead(wl, tau, device, H=4096, steps=12, repeats=7):
    """csd_step_lmhead (the step taken straight from the LM head: tcgen05 GEMM with the row statistics in its
    epilogue, decisions, memory update) on hidden[B, K+1, H] and weight[V, H], beside the unfused pair it
    replaces (a library bf16 GEMM that stores the logits, then csd_step on them)."""
    import torch

    import paper_2604_13634_b200 as pkg
    from synth_inputs import Synth

    syn = Synth(wl, 0, device)
    W = syn.lmhead_weight(H)
    ins = [syn.step_lmhead(s, W) for s in range(3)]
    ocm = pkg.Ocm(wl.ocm_slots, wl.lam, device.index)
    buf = pkg.LmheadBuffers(wl.B, wl.K, H, wl.V, device=device)
    R = wl.B * (wl.K + 1)

    def timed(fn):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize(device)
        ts = []
        for _ in range(repeats):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(steps):
                fn(i)
            b.record()
            b.synchronize()
            ts.append(a.elapsed_time(b) * 1e-3 / steps)
        return statistics.median(ts)

    pkg.csd_set_overlap(True)        # the GEMM of a step starts beside the decisions and the update of the step before
    fused = timed(lambda i: pkg.csd_step_lmhead(ins[i % 3][0], W, ins[i % 3][1], ocm, tau, buf))
    pkg.csd_set_overlap(False)       # plain stream-ordered launches: what a loop with other kernels between steps gets
    ordered = timed(lambda i: pkg.csd_step_lmhead(ins[i % 3][0], W, ins[i % 3][1], ocm, tau, buf))
    sb = pkg.StepBuffers(wl.B, wl.K, wl.V, torch.bfloat16, device=device)

    def unfused(i):
        h, d = ins[i % 3]
        z = torch.matmul(h.view(R, H), W.T).view(wl.B, wl.K + 1, wl.V)
        pkg.csd_step(z, d, ocm, tau, sb)
    plain = timed(unfused)
    st = ocm.stats()
    ocm.close()
    hbm, kind = measured_peak()
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            tensor_peak = float(json.load(f)["bf16_tflops"])
    except Exception:
        tensor_peak = 1590.0
    flops = 2.0 * R * H * wl.V
    hbm_bytes = (wl.V + R) * H * 2.0                     # the weight matrix and the hidden states once
    t_bound = max(flops / (tensor_peak * 1e12), hbm_bytes / (hbm * 1e9))
    return {"us_per_step": 1e6 * fused, "positions_per_s": wl.B * wl.K / fused, "steps": steps, "repeats": repeats,
            "H": H, "rows": R, "V": wl.V, "shape": pkg.csd_lmhead_shape(wl.B, wl.K, H, wl.V),
            "tensor_TFLOPs": flops / fused / 1e12, "tensor_frac": flops / fused / 1e12 / tensor_peak,
            "hbm_GBs": hbm_bytes / fused / 1e9, "hbm_frac": hbm_bytes / fused / 1e9 / hbm,
            "bound": "hbm" if hbm_bytes / (hbm * 1e9) >= flops / (tensor_peak * 1e12) else "tensor",
            "roofline_us": 1e6 * t_bound, "frac_of_roofline": t_bound / fused, "peak_source": f"of {kind}",
            "algorithmic_bytes": hbm_bytes, "traffic": NCU_TRAFFIC_BYTES_LMHEAD.get(wl.name) if H == 4096 else None,
            "stream_ordered_us_per_step": 1e6 * ordered, "stream_ordered_frac_of_roofline": t_bound / ordered,
            "unfused_us_per_step": 1e6 * plain,
            "unfused": f"torch.matmul (bf16 logits stored, {R * wl.V * 2 / 1e6:.0f} MB written and read back) followed by csd_step",
            "launches_per_step": 3,
            "launch": "eager, step overlap on (the GEMM launched programmatically behind the step before); "
                      "stream_ordered_*: overlap off",
            "ocm": {k: st[k] for k in ("n_keys", "rescues", "rejections", "flags")}}


def run_lmhead(args, wl, tau):
    """--mode lmhead: a bench line of its own for the step taken straight from the LM head."""
    import torch

    import paper_2604_13634_b200 as pkg
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path")
    pkg.lib()
    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    sampler = ClockSampler(device.index, period_s=0.005)
    sampler.start()
    m = measure_lmhead(wl, tau, device, H=args.hidden, steps=max(3, min(args.steps, 48)))
    if wl.name != "single_stream":
        from synth_inputs import WORKLOADS
        torch.cuda.empty_cache()
        m["single_stream"] = measure_lmhead(WORKLOADS["single_stream"], 0.3, device, H=args.hidden, steps=m["steps"])
    clocks = sampler.stop()
    line = {"metric": METRIC, "value": m["positions_per_s"], "unit": UNIT, "n_gpus": 1, "steps": m["steps"],
            "warmup": 3, "ms_per_step": m["us_per_step"] * 1e-3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "repeats": m["repeats"],
            "config": workload_config(wl, tau, {"mode": "step taken straight from the LM head (logits never stored)",
                                                "H": m["H"], "kernel_shape": m["shape"], "launch": m["launch"],
                                                "l2_policy": "the 1.2 GB weight matrix is larger than L2"}),
            "roofline": {"bound": m["bound"], "achieved": m["hbm_GBs"] if m["bound"] == "hbm" else m["tensor_TFLOPs"],
                         "peak": measured_peak()[0] if m["bound"] == "hbm" else None, "unit": "GB/s" if m["bound"] == "hbm" else "TFLOP/s",
                         "frac": m["frac_of_roofline"], "traffic": m["traffic"], "peak_source": m["peak_source"],
                         "kernel": m["shape"]["kernel"], "tensor_TFLOPs": m["tensor_TFLOPs"], "tensor_frac": m["tensor_frac"]},
            "gpu_launches": 3 * m["steps"], "clocks": clocks, "lmhead": m}
    print(json.dumps(line), flush=True)


def run_extras(device, skip, peak, names, overlap):
    """Short device-resident runs of the other workloads (extra keys, not bench lines): the pipelined loop
    (about a quarter of a second, median of 7 regions) and the latency of a step that runs alone."""
    import torch
    import paper_2604_13634_b200 as pkg
    from synth_inputs import WORKLOADS
    out = {}
    for name in names:
        if name == skip:
            continue
        wl = WORKLOADS[name]
        pkg.csd_set_overlap(overlap)
        b = Bench(wl, wl.taus[0], device)
        steps = 960 if wl.logit_bytes > 100e6 else 1920
        b.plan_steps_exactly(steps, 48)
        b.run(steps)
        torch.cuda.synchronize(device)
        sec = statistics.median(b.timed(steps) for _ in range(7))
        launch = b.launch_label(steps)
        alone = standalone_us(pkg, b)
        out[name] = {"positions_per_s": wl.B * wl.K * steps / sec, "us_per_step": 1e6 * sec / steps,
                     "achieved_GBs": wl.logit_bytes * steps / sec / 1e9,
                     "frac_of_measured_peak": wl.logit_bytes * steps / sec / 1e9 / peak, "steps": steps, "repeats": 7,
                     "launch": launch, "logit_bytes_per_step": wl.logit_bytes,
                     "single_step": {"us_per_step": alone, "achieved_GBs": wl.logit_bytes / alone / 1e3,
                                     "frac_of_measured_peak": wl.logit_bytes / alone / 1e3 / peak}}
        b.ocm.close()
        del b
        torch.cuda.empty_cache()
    pkg.csd_set_overlap(overlap)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=9600)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--tau", type=float, default=None)
    ap.add_argument("--eager", action="store_true", help="launch every step from Python instead of replaying a graph")
    ap.add_argument("--no-overlap", action="store_true",
                    help="plain stream-ordered launches (no programmatic dependent launch between steps)")
    ap.add_argument("--chunk-bytes", type=int, default=0, help="override the automatic chunk size (0 = automatic)")
    ap.add_argument("--ctas-per-sm", type=int, default=0, help="override the resident blocks per SM (0 = automatic)")
    ap.add_argument("--block-threads", type=int, default=0, help="override the threads per block (0 = automatic)")
    ap.add_argument("--graph-steps", type=int, default=48, help="least number of steps captured into the replayed graph")
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--extras", action="store_true", help="also time the two B = 1 workloads (extra keys, same line)")
    ap.add_argument("--lean", action="store_true", help="only the headline measurement: no other workloads, no stand-alone "
                                                         "latency, no stochastic sub-record")
    ap.add_argument("--repeats", type=int, default=0, help="how often the timed region is taken (0 = automatic, at least 7)")
    ap.add_argument("--mode", default="greedy", choices=["greedy", "sampled", "lmhead"],
                    help="sampled: the stochastic verification step; lmhead: the step taken straight from the LM head "
                         "(each its own JSON line; 1 GPU)")
    ap.add_argument("--hidden", type=int, default=4096, help="H of --mode lmhead")
    ap.add_argument("--temperature", type=float, default=0.3, help="T of --mode sampled")
    args = ap.parse_args()

    from synth_inputs import WORKLOADS
    wl = WORKLOADS[args.workload]
    tau = wl.taus[0] if args.tau is None else args.tau
    if args.impl == "reference":
        run_reference(args, wl, tau)
    elif args.mode == "sampled":
        run_sampled(args, wl, tau)
    elif args.mode == "lmhead":
        run_lmhead(args, WORKLOADS["batched_serving"] if args.workload == DEFAULT_WORKLOAD else wl, tau if args.workload != DEFAULT_WORKLOAD else 0.3)
    else:
        run_ours(args, wl, tau)


if __name__ == "__main__":
    main()
