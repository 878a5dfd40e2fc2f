#!/usr/bin/env python
"""Benchmark of the routing + load-control hot path (one B200 per rank).

A step = one pass of the whole path over one fresh synthetic batch:
moe_route_step (router GEMM + sigmoid + biased top-K + gates + load histogram)
followed by moe_controller_update (ID Balancing update and MaxVio/MinVio, one
kernel).  Metric: routed tokens per second, where a routed token is one token
routed through one router layer.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
  python bench.py --impl reference ...     # the CPU oracle, timed as it stands
  python bench.py --aux [--workload NAME]  # the calls that are not on the timed path (quantile update, score
                                           # statistics, diagnostics): microseconds and GB/s of each, own JSON line

The headline workload is the largest single-GPU configuration (`top10_large`: 60 router layers, 65536 tokens,
hidden 4096, Top-10 of 768).  After it the other configurations are timed briefly in the same run and reported
under `all_configs`.  Every timed region lasts at least `--min-region-s` seconds: the K-step loop is repeated
(`repeats`) until it does.  With --gpus N > 1 and no launcher, N ranks are started here (one per GPU).

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2609_39137_b200 import synth

METRIC = "routed_tokens_per_s"
UNIT = "tokens/s"
HEADLINE = "top10_large"
OTHERS = ["tiny_top3", "top10_single", "top3_single", "top5_single", "top10_deep", "top8_of_256"]
# the baseline controllers on the Top-3 workload (the third configuration compares three controllers): the fixed-step
# integral costs what the ID update costs; Quantile Balancing needs the logits dump and the per-token threshold
# from the routing kernel and a selection pass over the dump in the update
CONTROLLER_VARIANTS = [("top3_single", "fixed_step"), ("top3_single", "quantile")]
L2_BYTES = 126e6

# dram__bytes_read.sum + dram__bytes_write.sum of the routing kernels of one moe_route_step, per launch, from ncu
# captures whose summaries are kept with the other profile summaries.  `layers` = router layers of the captured
# launch; the traffic of a launch with more layers of the same shape is scaled by the layer count (every layer
# streams its own x once and re-reads nothing of another layer's).
NCU_TRAFFIC = {
    # routing kernel read + write, merge kernel read + write (2 of the 60 layers: a capture of the full launch
    # would hold 64 GB on the device under the profiler)
    "top10_large": {"bytes": 1148419000 + 79036672 + 31513088 + 256, "layers": 2,
                    "profile": "profiles/route_step_kernel_top10_large.md"},
    "top10_single": {"bytes": 70553344 + 2378496, "layers": 1, "profile": "profiles/route_step_kernel_top10_single.md"},
    "top10_deep": {"bytes": 332765952 + 18158848, "layers": 4, "profile": "profiles/route_step_kernel_top10_deep_4layers.md"},
}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], tflops=d["bf16_tflops"], tflops_sustained=d.get("bf16_tflops_sustained"),
                    source="measured")
    return dict(hbm_gbs=6650.0, tflops=1590.0, tflops_sustained=1400.0, source="fallback")


def ring_size(wl):
    """Distinct input batches cycled through: enough that consecutive steps cannot find their x in L2, at most
    ~70 GB of device memory."""
    batch = wl.L * wl.T * wl.H * 2
    return int(min(512, max(2, math.ceil(3 * L2_BYTES / batch)), max(2, 70e9 // batch)))


def config_dict(wl, world):
    ring = ring_size(wl)
    batch = wl.L * wl.T * wl.H * 2
    return {"workload": wl.name, "T": wl.T, "H": wl.H, "E": wl.E, "K": wl.K, "L": wl.L, "controller": "id",
            "parallelism": f"dp{world}",
            "l2": f"ring of {ring} distinct input batches ({ring * batch / 1e6:.0f} MB) cycled, larger than the "
                  f"126 MB L2; one batch is {batch / 1e6:.0f} MB"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) every few ms."""

    def __init__(self, index):
        self.samples, self.power, self.reasons, self.max_mhz = [], [], set(), None
        self._stop = threading.Event()
        self._th = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "hw_power_brake_slowdown": 0x80, "sw_power_cap": 0x4}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.004)

    def start(self):
        if self.nv is not None:
            self._th = threading.Thread(target=self._run, daemon=True)
            self._th.start()

    def stop(self):
        self._stop.set()
        if self._th is not None:
            self._th.join()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w": statistics.median(self.power) if self.power else None}


def cpu_oracle_rate(wl, threads, tokens_per_thread, keep=False):
    """Routed tokens/s of the CPU oracle (fp64 definition + controller) on a token sample of layer 0."""
    import oracle
    n_tok = min(wl.T, threads * tokens_per_thread)
    xt = synth.hidden_states(wl, 0, 0, "cpu", tokens=n_tok)
    wt = synth.router_weights(wl, 0, "cpu")
    x, w = synth.bf16_bits(xt), synth.bf16_bits(wt)
    b = np.zeros(wl.E, np.float32)
    oracle.route_tokens_f64(x[:threads], w, b, wl.K, threads=1)    # build + page in
    t0 = time.perf_counter()
    r = oracle.route_tokens_f64(x, w, b, wl.K, threads=threads)
    e = oracle.load_error(r["n"])
    oracle.id_update(b, np.zeros_like(b), e, 6e-3, 6e-3, center=True)
    oracle.violations(r["n"])
    dt = time.perf_counter() - t0
    if keep:
        return n_tok / dt, n_tok, dt, (xt, wt, r)
    return n_tok / dt, n_tok, dt


def near_tie_report(wl, sample, dev):
    """Routes the oracle's token sample on the GPU (zero bias, one layer) and counts, against the fp64 definition,
    the tokens whose expert SET differs -- allowed only where the rank-K / rank-K+1 gap is below 1e-4."""
    from paper_2609_39137_b200 import binding
    xt, wt, ref = sample
    n_tok = xt.shape[0]
    r = binding.Router(1, wl.E, wl.K, wl.H, n_tok, device=dev)
    logits = torch.empty(1, n_tok, wl.E, device=dev)
    idx, _ = r.route_step(xt.to(dev)[None].contiguous(), wt.to(dev)[None].contiguous(), logits_out=logits)
    r.poll()
    gi = np.sort(idx[0].cpu().numpy(), 1)
    same = np.all(gi == np.sort(ref["idx"], 1), axis=1)
    near = ref["gap"] < 1e-4
    err = float(np.max(np.abs(logits[0].cpu().numpy().astype(np.float64) - ref["z"])))
    return {"tokens_checked": int(n_tok), "sets_differing": int((~same).sum()),
            "differing_with_clear_gap": int((~same & ~near).sum()),
            "tokens_with_gap_below_1e-4": int(near.sum()),
            "differing_fraction": float((~same).mean()), "budget_fraction": 1e-4,
            "max_abs_logit_error_vs_fp64": err, "logit_tolerance": 1e-4}


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    threads = os.cpu_count() or 1
    per_thread = max(8, int(args.ref_tokens_per_thread))
    for _ in range(max(0, args.warmup)):
        cpu_oracle_rate(wl, threads, 8)
    rates, times, n_tok = [], [], 0
    for _ in range(max(1, args.steps)):
        rate, n_tok, dt = cpu_oracle_rate(wl, threads, per_thread)
        rates.append(rate)
        times.append(dt)
    value = n_tok * len(times) / sum(times)
    sample = f"{n_tok} of {wl.T} tokens of layer 0 per step, all stages (fp64 logits, sort, gates, loads, ID update)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(wl, args.gpus),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_aux(args, wl):
    """Times the calls that work on the logits dump (not part of a step): the routing step with the dump, the
    Quantile Balancing update (single layer), the score statistics, and the small diagnostics calls."""
    from paper_2609_39137_b200 import binding
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    L1 = wl.with_(L=1)
    w = torch.stack([synth.router_weights(L1, 0, dev)]).contiguous()
    xs = [torch.stack([synth.hidden_states(L1, 0, s, dev)]).contiguous() for s in range(4)]
    logits = torch.empty(1, wl.T, wl.E, device=dev)
    alpha = torch.empty(1, wl.T, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # larger than L2

    def timed(fn, reps):
        fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        return statistics.median(ts), min(ts)

    reps = max(3, min(args.steps, 20))
    out = {}
    dump_bytes = wl.T * wl.E * 4
    rq = binding.Router(1, wl.E, wl.K, wl.H, wl.T, controller="quantile", device=dev)
    state = {"i": 0}

    def qb_route():
        rq.route_step(xs[state["i"] % 4], w, logits_out=logits, alpha_out=alpha)
        state["i"] += 1
    med, best = timed(lambda: (qb_route(), rq.controller_update()), reps)
    rs = binding.Router(1, wl.E, wl.K, wl.H, wl.T, controller="id", device=dev)
    r_med, r_best = timed(lambda: rs.route_step(xs[0], w, logits_out=logits, alpha_out=alpha), reps)
    out["route_step_with_dump_us"] = {"median": r_med, "best": r_best}
    out["route_plus_quantile_update_us"] = {"median": med, "best": best}
    out["quantile_update_us"] = {"median": med - r_med, "note": "difference of the two lines above",
                                 "dump_GBps": 4 * dump_bytes / max(1e-9, (med - r_med)) / 1e3}
    rqh = binding.Router(1, wl.E, wl.K, wl.H, wl.T, controller="quantile", qb_hist_bins=1024, device=dev)

    def qbh_route():
        rqh.route_step(xs[state["i"] % 4], w, logits_out=logits, alpha_out=alpha)
        state["i"] += 1
    med_h, _ = timed(lambda: (qbh_route(), rqh.controller_update()), reps)
    out["quantile_update_histogram_estimate_us"] = {
        "median": med_h - r_med, "note": "1024-bin margin histogram, one pass over the dump; difference to the routing call",
        "dump_GBps": dump_bytes / max(1e-9, (med_h - r_med)) / 1e3}
    rqh.poll()
    rs.controller_update()
    idx, gate = rs.route_step(xs[0], w, logits_out=logits)
    loads = rs.loads_peek()
    med, best = timed(lambda: rs.score_stats(logits, loads), reps)
    out["score_stats_us"] = {"median": med, "best": best, "dump_GBps": dump_bytes / best / 1e3}
    med, best = timed(lambda: rs.gate_entropy(gate), reps)
    out["gate_entropy_us"] = {"median": med, "best": best}
    rs.controller_update()
    med, best = timed(lambda: rs.load_diagnostics(), reps)
    out["load_diagnostics_us"] = {"median": med, "best": best}
    rs.poll()
    rq.poll()
    print(json.dumps({"aux": True, "config": {"workload": wl.name, "T": wl.T, "H": wl.H, "E": wl.E, "K": wl.K, "L": 1},
                      "l2": "256 MB written between timed calls", "reps": reps, "calls": out}), flush=True)


class Job:
    """Inputs, outputs and context of one workload on one rank."""

    chunk_split = 0      # moe_route_config.chunk_split of every context made here (0 = the library chooses)

    def __init__(self, wl, dev, rank, world, dist, controller="id"):
        from paper_2609_39137_b200 import binding, dp
        self.controller = controller
        self.wl, self.dev, self.dist, self.dp = wl, dev, dist, dp
        self.ring = ring_size(wl)
        # seeded, synthetic; each rank draws its own token shard (step index offset by the rank)
        self.w = torch.stack([synth.router_weights(wl, l, dev) for l in range(wl.L)]).contiguous()
        self.xs = []
        for s in range(self.ring):
            x = torch.empty(wl.L, wl.T, wl.H, dtype=torch.bfloat16, device=dev)
            for l in range(wl.L):
                x[l] = synth.hidden_states(wl, l, s * world + rank, dev)
            self.xs.append(x)
        self.idx = torch.empty(wl.L, wl.T, wl.K, dtype=torch.int32, device=dev)
        self.gate = torch.empty(wl.L, wl.T, wl.K, dtype=torch.float32, device=dev)
        self.router = binding.Router(wl.L, wl.E, wl.K, wl.H, wl.T, controller=controller, device=dev,
                                     chunk_split=Job.chunk_split)
        self.logits = self.alpha = None
        if controller == "quantile":     # Eq. 7 needs every token's scores and its threshold
            self.logits = torch.empty(wl.L, wl.T, wl.E, dtype=torch.float32, device=dev)
            self.alpha = torch.empty(wl.L, wl.T, dtype=torch.float32, device=dev)

    def step(self, i):
        self.router.route_step(self.xs[i % self.ring], self.w, self.idx, self.gate, logits_out=self.logits,
                               alpha_out=self.alpha)
        if self.dist is not None:
            self.dp.allreduce_loads(self.router, self.dist)   # Algorithm 1 line 4: counts summed over the DP group
        self.router.controller_update()

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        torch.cuda.synchronize()

    def prewarm(self, seconds, warmup):
        t_end = time.perf_counter() + seconds
        i = 0
        while time.perf_counter() < t_end:
            self.step(i)
            i += 1
            if i % 16 == 0:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        # estimate of one step for sizing the timed region
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = max(3, warmup)
        e0.record()
        for i in range(n):
            self.step(i)
        e1.record()
        self.router.poll()
        self.barrier()
        return e0.elapsed_time(e1) / n

    def timed(self, steps, repeats):
        """`repeats` back-to-back runs of the `steps`-step loop; events on the launching stream.  A few routing
        launches are bracketed by their own event pair (an event between two kernels switches the overlap of
        consecutive launches off for that launch, so most run without one)."""
        total_steps = steps * repeats
        stride = 1 if total_steps <= 16 else max(8, total_steps // 16)
        ev = {i: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for i in range(0, total_steps, stride)}
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = self.router.launch_count()
        self.barrier()
        t0.record()
        i = 0
        for _ in range(repeats):
            for _ in range(steps):
                probe = ev.get(i)
                if probe is not None:
                    probe[0].record()
                self.router.route_step(self.xs[i % self.ring], self.w, self.idx, self.gate, logits_out=self.logits,
                                       alpha_out=self.alpha)
                if probe is not None:
                    probe[1].record()
                if self.dist is not None:
                    self.dp.allreduce_loads(self.router, self.dist)
                self.router.controller_update()
                i += 1
        t1.record()
        self.barrier()
        launches = self.router.launch_count() - launches0
        self.router.poll()
        total_ms = t0.elapsed_time(t1)
        route_ms = [a.elapsed_time(b) for a, b in ev.values()]
        return total_ms, route_ms, launches

    def breakdown(self, n_break):
        """Every step bracketed by events, so the two calls are serialised: median and best step and the two
        calls separately (after the timed region, not part of `value`)."""
        bev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_break)]
        for i in range(n_break):
            bev[i][0].record()
            self.router.route_step(self.xs[i % self.ring], self.w, self.idx, self.gate, logits_out=self.logits,
                                   alpha_out=self.alpha)
            bev[i][1].record()
            if self.dist is not None:
                self.dp.allreduce_loads(self.router, self.dist)
            self.router.controller_update()
            bev[i][2].record()
        self.barrier()
        self.router.poll()
        br_route = sorted(a.elapsed_time(b) for a, b, _ in bev)
        br_ctrl = sorted(b.elapsed_time(c) for _, b, c in bev)
        br_step = sorted(a.elapsed_time(c) for a, _, c in bev)
        return {"steps": n_break, "serialised": True,
                "step_ms_median": statistics.median(br_step), "step_ms_best": br_step[0],
                "route_step_ms_median": statistics.median(br_route), "route_step_ms_best": br_route[0],
                "controller_update_ms_median": statistics.median(br_ctrl), "controller_update_ms_best": br_ctrl[0]}


def roofline_of(wl, total_ms, steps_total, route_ms, pk):
    flops = 2.0 * wl.L * wl.T * wl.H * wl.E
    bracketed_ms = sum(route_ms) / len(route_ms)
    # Consecutive launches overlap (the next routing kernel's prologue and loads run under the controller update
    # of the step before), and an event pair around a launch switches that overlap off for it.  The launch
    # duration used for the roofline is therefore the smaller of the bracketed time and the whole step's time
    # (events around the timed region / steps), which contains the routing launch plus the controller kernel.
    avg_route_ms = min(bracketed_ms, total_ms / steps_total)
    achieved = flops / (avg_route_ms * 1e-3) / 1e12
    cap = NCU_TRAFFIC.get(wl.name)
    if cap is not None:
        traffic = cap["bytes"] * wl.L / cap["layers"]
        traffic_note = (f"ncu capture of {cap['layers']} layer(s) of this shape scaled to {wl.L} "
                        f"({cap['profile']})") if cap["layers"] != wl.L else cap["profile"]
    else:
        traffic, traffic_note = None, "no ncu capture of this workload"
    algo_bytes = wl.L * (wl.T * wl.H * 2 + wl.E * wl.H * 2 + wl.T * wl.K * 8)
    # Denominator: the measured cuBLAS figure for the regime the kernel was timed in -- the sustained one when the
    # timed region is a long stretch of back-to-back launches under the power cap, the burst one for a short region.
    region_s = total_ms * 1e-3
    long_region = region_s >= 0.25 and bool(pk.get("tflops_sustained"))
    peak = pk["tflops_sustained"] if long_region else pk["tflops"]
    which = (f"sustained bf16: the timed region is {region_s:.2f} s of back-to-back launches" if long_region
             else "burst bf16: short timed region")
    return {"kernel": "route_step_kernel (+ route_merge_kernel under chunk-split scheduling)", "bound": "tensor",
            "achieved": achieved, "peak": peak,
            "unit": "TFLOP/s", "frac": achieved / peak, "peak_source": f"{pk['source']} ({which})",
            "frac_of_burst": achieved / pk["tflops"], "peak_burst": pk["tflops"],
            "frac_of_sustained": (achieved / pk["tflops_sustained"]) if pk.get("tflops_sustained") else None,
            "avg_launch_ms": avg_route_ms, "bracketed_launch_ms": bracketed_ms,
            "best_bracketed_launch_ms": min(route_ms), "launches_bracketed": len(route_ms),
            "algorithmic_flops_per_launch": flops, "algorithmic_bytes_per_launch": algo_bytes,
            "traffic": traffic, "traffic_note": traffic_note}


def library_gemm_leg(wl, job, local_rank, seconds=1.5):
    """Yardstick, not part of the path: the logits GEMM alone ([T x H] x [H x E] bf16 -> fp32-accumulated bf16
    logits written to HBM, no score, no selection, no histogram) through torch.matmul on the job's own inputs,
    layer after layer over the input ring, back to back for `seconds` under the same power cap, with the clock it
    ran at.  What a fused routing step is worth is read against this on the same GPU: the library call still
    needs a pass over its logits before it has routed anything."""
    out = torch.empty(wl.T, wl.E, dtype=torch.bfloat16, device=job.dev)
    wt = [job.w[l].t() for l in range(wl.L)]

    def sweep(i):
        x = job.xs[i % job.ring]
        for l in range(wl.L):
            torch.matmul(x[l], wt[l], out=out)
    sweep(0)
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n, t0 = 0, time.perf_counter()
    e0.record()
    while time.perf_counter() - t0 < seconds:
        sweep(n)
        n += 1
        torch.cuda.synchronize()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / n
    return {"what": "torch.matmul of the same [T x H] x [H x E] bf16 problem per layer on the same inputs, logits "
                    "written as bf16, nothing routed; yardstick only",
            "ms_per_step": ms, "tflops": 2.0 * wl.L * wl.T * wl.H * wl.E / ms / 1e9, "seconds": seconds,
            "sm_mhz": clocks.get("sm_mhz"), "power_w": clocks.get("power_w")}


def e2e_leg(wl, job, dev, world, steps_hint):
    """Same step through moe_route_step_host: pinned host x and W_r in, indices, gates and MaxVio/MinVio out,
    all copies inside the timed region."""
    from paper_2609_39137_b200 import binding
    batch = wl.L * wl.T * wl.H * 2
    note = None
    try:
        import psutil
        avail = psutil.virtual_memory().available
    except Exception:
        avail = 64e9
    L = wl.L
    if batch * world > 0.45 * avail:
        L = max(1, int(0.45 * avail / (world * wl.T * wl.H * 2)))
        note = (f"host memory allows {L} of {wl.L} layers per step in pinned buffers; tokens/s of those layers")
    wle = wl.with_(L=L)
    rh = binding.Router(L, wl.E, wl.K, wl.H, wl.T, controller="id", host_staging=True, device=dev)
    xh = torch.empty(L, wl.T, wl.H, dtype=torch.bfloat16, pin_memory=True)
    for l in range(L):
        xh[l].copy_(job.xs[0][l])
    wh = torch.empty(L, wl.E, wl.H, dtype=torch.bfloat16, pin_memory=True)
    wh.copy_(job.w[:L])
    ih = torch.empty(L, wl.T, wl.K, dtype=torch.int32, pin_memory=True)
    gh = torch.empty(L, wl.T, wl.K, dtype=torch.float32, pin_memory=True)
    vio_h = torch.empty(2, L, dtype=torch.float32, pin_memory=True)
    torch.cuda.synchronize()

    def e2e_step():
        rh.route_step_host(xh, wh, ih, gh)
        if job.dist is not None:
            job.dp.allreduce_loads(rh, job.dist)
        rh.controller_update()
        _, _, mx, mn = rh.load_stats()
        vio_h[0].copy_(mx, non_blocking=True)
        vio_h[1].copy_(mn, non_blocking=True)

    e2e_step()
    job.barrier()
    est = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    est[0].record()
    e2e_step()
    est[1].record()
    job.barrier()
    one_ms = est[0].elapsed_time(est[1])
    n = int(max(3, min(steps_hint, 30, math.ceil(3000.0 / max(one_ms, 1e-3)))))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        e2e_step()
    e1.record()
    job.barrier()
    ms = e0.elapsed_time(e1)
    rh.poll()
    h2d = L * wl.T * wl.H * 2 + L * wl.E * wl.H * 2
    d2h = 2 * L * wl.T * wl.K * 4 + 2 * L * 4
    return ms, n, wle, h2d, d2h, note


def spawn_ranks(n):
    """No launcher around us: start one rank per GPU here and wait for them."""
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env))
    rc = 0
    for p in procs:
        rc = max(rc, abs(p.wait()))
    sys.exit(rc)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=HEADLINE, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--layers", type=int, default=0, help="override the number of router layers (0 = workload's)")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--ref-tokens-per-thread", type=int, default=1024)
    ap.add_argument("--prewarm-s", type=float, default=0.5, help="untimed seconds of steps before the warm-up")
    ap.add_argument("--min-region-s", type=float, default=0.5, help="shortest timed region; the step loop is repeated")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-all-configs", action="store_true", help="time only the chosen workload")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-library-gemm", action="store_true", help="skip the torch.matmul yardstick of the same problem")
    ap.add_argument("--chunk-split", type=int, default=0, choices=[0, 1, 2],
                    help="scheduling of the expert chunks (moe_route_config.chunk_split); 0 = the library chooses")
    ap.add_argument("--aux", action="store_true", help="time the calls outside the step (one GPU) and exit")
    args = ap.parse_args()

    wl = synth.WORKLOADS[args.workload]
    if args.layers > 0:
        wl = wl.with_(L=args.layers)
    if args.impl == "reference":
        run_reference(args, wl)
        return
    if args.aux:
        run_aux(args, wl)
        return

    env_world = os.environ.get("WORLD_SIZE")
    if env_world is None and args.gpus > 1:
        if torch.cuda.device_count() < args.gpus:
            raise SystemExit(f"--gpus {args.gpus}: only {torch.cuda.device_count()} CUDA device(s) visible")
        spawn_ranks(args.gpus)
    world = int(env_world or "1")
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} does not match WORLD_SIZE={world} of the launcher")

    from paper_2609_39137_b200 import binding     # fails loudly if the CUDA library is missing

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (sm_100a); there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    pk = peaks()
    sampler = ClockSampler(local_rank)
    Job.chunk_split = args.chunk_split

    # ---- headline workload
    job = Job(wl, dev, rank, world, dist)
    est_ms = job.prewarm(args.prewarm_s, args.warmup)
    repeats = max(1, math.ceil(args.min_region_s * 1e3 / max(1e-6, est_ms * args.steps)))
    sampler.start()
    total_ms, route_ms, launches = job.timed(args.steps, repeats)
    while total_ms < args.min_region_s * 1e3:          # the estimate was too high: time a longer region
        repeats = max(repeats + 1, math.ceil(1.1 * repeats * args.min_region_s * 1e3 / total_ms))
        total_ms, route_ms, launches = job.timed(args.steps, repeats)
    clocks = sampler.stop()
    loads, bias, maxvio, minvio = job.router.load_stats()
    gate_open = int(job.router.gate_stats().sum())
    breakdown = job.breakdown(max(3, min(args.steps, 24)))
    lib_gemm = None
    if rank == 0 and world == 1 and not args.no_library_gemm:
        lib_gemm = library_gemm_leg(wl, job, local_rank)
    e2e = None
    if not args.no_e2e:
        e2e = e2e_leg(wl, job, dev, world, args.steps)

    if dist is not None:
        t = torch.tensor([total_ms, e2e[0] if e2e else 0.0], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t[0])
        if e2e:
            e2e = (float(t[1]),) + tuple(e2e[1:])
    steps_total = args.steps * repeats
    tokens_per_step = wl.L * wl.T * world
    value = tokens_per_step * steps_total / (total_ms * 1e-3)
    last_step = {"maxvio_max": float(maxvio.max()), "minvio_max": float(minvio.max()),
                 "open_derivative_gates": gate_open}
    headline_roofline = roofline_of(wl, total_ms, steps_total, route_ms, pk) if rank == 0 else None
    del job
    torch.cuda.empty_cache()

    # ---- the other configurations, briefly (same run, same rules; one entry each)
    others = []
    if not args.no_all_configs and args.layers == 0:
        for name, ctrl in [(n, "id") for n in OTHERS] + CONTROLLER_VARIANTS:
            if name == wl.name and ctrl == "id":
                continue
            if ctrl == "quantile" and world > 1:
                continue          # Eq. 7 ranks the tokens of one rank's dump; not a data-parallel configuration here
            o = synth.WORKLOADS[name]
            oj = Job(o, dev, rank, world, dist, controller=ctrl)
            o_est = oj.prewarm(0.2, 3)
            o_steps = max(3, args.steps)
            o_rep = max(1, math.ceil(args.min_region_s * 1e3 / max(1e-6, o_est * o_steps)))
            o_sampler = ClockSampler(local_rank)
            o_sampler.start()
            o_ms, o_route, _ = oj.timed(o_steps, o_rep)
            while o_ms < args.min_region_s * 1e3:
                o_rep = max(o_rep + 1, math.ceil(1.1 * o_rep * args.min_region_s * 1e3 / o_ms))
                o_ms, o_route, _ = oj.timed(o_steps, o_rep)
            o_clocks = o_sampler.stop()
            oj.router.poll()
            if dist is not None:
                t = torch.tensor([o_ms], device=dev, dtype=torch.float64)
                dist.all_reduce(t, op=dist.ReduceOp.MAX)
                o_ms = float(t[0])
            if rank == 0:
                rf = roofline_of(o, o_ms, o_steps * o_rep, o_route, pk)
                others.append({"workload": name, "controller": ctrl, "L": o.L, "T": o.T, "H": o.H, "E": o.E, "K": o.K,
                               "steps": o_steps, "repeats": o_rep, "timed_region_s": o_ms * 1e-3,
                               "ms_per_step": o_ms / (o_steps * o_rep),
                               "tokens_per_s": o.L * o.T * world * o_steps * o_rep / (o_ms * 1e-3),
                               "tflops": rf["achieved"], "frac_of_burst": rf["frac_of_burst"],
                               "frac_of_sustained": rf["frac_of_sustained"], "ring": oj.ring,
                               "traffic": rf["traffic"], "sm_mhz": o_clocks.get("sm_mhz"),
                               "power_w": o_clocks.get("power_w"), "clock_reasons": o_clocks.get("reasons")})
            del oj
            torch.cuda.empty_cache()

    if rank == 0:
        cpu = near = None
        if not args.no_cpu_baseline:
            threads = os.cpu_count() or 1
            rate, n_tok, dt, sample = cpu_oracle_rate(wl, threads, args.ref_tokens_per_thread, keep=True)
            rate1, n_tok1, dt1 = cpu_oracle_rate(wl, 1, max(64, args.ref_tokens_per_thread // 4))
            cpu = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle",
                   "sample": f"{n_tok} of {wl.T} tokens of layer 0, all stages, {dt:.1f} s",
                   "single_thread": {"value": rate1, "sample": f"{n_tok1} tokens, {dt1:.1f} s"}}
            near = near_tie_report(wl, sample, dev)
        cfg = config_dict(wl, world)
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": total_ms / steps_total, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": cfg, "repeats": repeats, "timed_steps": steps_total, "timed_region_s": total_ms * 1e-3,
                "roofline": headline_roofline, "cpu_baseline": cpu, "near_tie": near,
                "gpu_launches": int(launches), "clocks": clocks, "breakdown": breakdown,
                "last_step": last_step, "all_configs": others}
        if lib_gemm:
            # > 1: a whole routing step (logits, scores, top-K, gates, loads, controller) takes less time than
            # the library's logits GEMM alone
            lib_gemm["library_gemm_ms_over_routing_step_ms"] = lib_gemm["ms_per_step"] / (total_ms / steps_total)
            line["library_gemm"] = lib_gemm
        if e2e:
            ms, n, wle, h2d, d2h, note = e2e
            line["e2e"] = {"value": wle.L * wl.T * world * n / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                           "d2h_bytes_per_step": d2h, "steps": n, "ms_per_step": ms / n, "layers": wle.L}
            if note:
                line["e2e"]["note"] = note
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
