#!/usr/bin/env python
"""Benchmark of the routing + load-control hot path (one B200 per rank).

A step = one pass of the whole path over one fresh synthetic batch:
moe_route_step (router GEMM + sigmoid + biased top-K + gates + load histogram,
one fused kernel) followed by moe_controller_update (ID Balancing update and
MaxVio/MinVio, one kernel).  Metric: routed tokens per second, where a routed
token is one token routed through one router layer.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
  python bench.py --impl reference ...     # the CPU oracle, timed as it stands
  python bench.py --aux [--workload NAME]  # the calls that are not on the timed path (quantile update, score
                                           # statistics, diagnostics): microseconds and GB/s of each, own JSON line

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
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
RING = 8   # distinct input batches cycled through, so every timed step reads x from HBM

# dram__bytes_read.sum + dram__bytes_write.sum of one route_step_kernel launch, from an ncu capture of
# this command on the same workload (the summary is kept with the other profile summaries); None = no capture
NCU_TRAFFIC_BYTES = {"top10_single": 70629376 + 1660928}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], tflops=d["bf16_tflops"], tflops_sustained=d.get("bf16_tflops_sustained"),
                    source="measured")
    return dict(hbm_gbs=6650.0, tflops=1590.0, tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) every few ms."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
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
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def cpu_oracle_rate(wl, threads, tokens_per_thread):
    """Routed tokens/s of the CPU oracle (fp64 definition + controller) on a token sample."""
    import oracle
    n_tok = min(wl.T, threads * tokens_per_thread)
    x = synth.bf16_bits(synth.hidden_states(wl, 0, 0, "cpu", tokens=n_tok))
    w = synth.bf16_bits(synth.router_weights(wl, 0, "cpu"))
    b = np.zeros(wl.E, np.float32)
    oracle.route_tokens_f64(x[:threads], w, b, wl.K, threads=1)    # build + page in
    t0 = time.perf_counter()
    r = oracle.route_tokens_f64(x, w, b, wl.K, threads=threads)
    e = oracle.load_error(r["n"])
    oracle.id_update(b, np.zeros_like(b), e, 6e-3, 6e-3, center=True)
    oracle.violations(r["n"])
    dt = time.perf_counter() - t0
    return n_tok / dt, n_tok, dt


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
            "config": {"workload": wl.name, "T": wl.T, "H": wl.H, "E": wl.E, "K": wl.K, "L": wl.L},
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
    out["quantile_update_us"] = {"median": med - r_med, "note": "difference of the two lines above; 4 passes over the dump",
                                 "dump_GBps": 4 * dump_bytes / max(1e-9, (med - r_med)) / 1e3}
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="top10_single", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--layers", type=int, default=0, help="override the number of router layers (0 = workload's)")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--ref-tokens-per-thread", type=int, default=1024)
    ap.add_argument("--prewarm-s", type=float, default=0.5, help="untimed seconds of steps before the warm-up")
    ap.add_argument("--no-cpu-baseline", action="store_true")
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

    from paper_2609_39137_b200 import binding, dp     # fails loudly if the CUDA library is missing

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (sm_100a); there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    # ---- inputs (seeded, synthetic; each rank draws its own token shard: step index offset by rank)
    ring = min(RING, max(2, int(6e9 // max(1, wl.L * wl.T * wl.H * 2))))
    w = torch.stack([synth.router_weights(wl, l, dev) for l in range(wl.L)]).contiguous()
    xs = [torch.stack([synth.hidden_states(wl, l, s * world + rank, dev) for l in range(wl.L)]).contiguous()
          for s in range(ring)]
    idx = torch.empty(wl.L, wl.T, wl.K, dtype=torch.int32, device=dev)
    gate = torch.empty(wl.L, wl.T, wl.K, dtype=torch.float32, device=dev)
    router = binding.Router(wl.L, wl.E, wl.K, wl.H, wl.T, controller="id", device=dev)

    def step(i):
        router.route_step(xs[i % ring], w, idx, gate)
        if dist is not None:
            dp.allreduce_loads(router, dist)     # Algorithm 1 line 4: counts summed over the data-parallel group
        router.controller_update()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    # pre-warm: bring clocks up and fault everything in (untimed, before the W warm-up steps)
    t_end = time.perf_counter() + args.prewarm_s
    i = 0
    while time.perf_counter() < t_end:
        step(i)
        i += 1
        if i % 64 == 0:
            torch.cuda.synchronize()
    for i in range(args.warmup):
        step(i)
    router.poll()
    barrier()

    # ---- timed region: device-resident inputs
    # the routing launch is bracketed by events on every `stride`-th step only (16 brackets per run): an event between two kernels
    # keeps the second from overlapping the first one's tail, so most steps run without any
    stride = 1 if args.steps <= 16 else max(8, args.steps // 16)
    ev = {i: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
          for i in range(0, args.steps, stride)}
    t_all0, t_all1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = router.launch_count()
    sampler.start()
    barrier()
    t_all0.record()
    for i in range(args.steps):
        probe = ev.get(i)
        if probe is not None:
            probe[0].record()
        router.route_step(xs[i % ring], w, idx, gate)
        if probe is not None:
            probe[1].record()
        if dist is not None:
            dp.allreduce_loads(router, dist)
        router.controller_update()
    t_all1.record()
    barrier()
    launches = router.launch_count() - launches0
    total_ms = t_all0.elapsed_time(t_all1)
    router.poll()
    route_ms = [a.elapsed_time(b) for a, b in ev.values()]
    loads, bias, maxvio, minvio = router.load_stats()

    # ---- per-call breakdown (after the timed region, not part of `value`): every step bracketed by events, so the
    # two calls are serialised; median and best step, and the two calls separately
    n_break = max(3, min(args.steps, 48))
    bev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_break)]
    for i in range(n_break):
        bev[i][0].record()
        router.route_step(xs[i % ring], w, idx, gate)
        bev[i][1].record()
        if dist is not None:
            dp.allreduce_loads(router, dist)
        router.controller_update()
        bev[i][2].record()
    barrier()
    router.poll()
    br_route = sorted(a.elapsed_time(b) for a, b, _ in bev)
    br_ctrl = sorted(b.elapsed_time(c) for _, b, c in bev)
    br_step = sorted(a.elapsed_time(c) for a, _, c in bev)
    breakdown = {"steps": n_break, "serialised": True,
                 "step_ms_median": statistics.median(br_step), "step_ms_best": br_step[0],
                 "route_step_ms_median": statistics.median(br_route), "route_step_ms_best": br_route[0],
                 "controller_update_ms_median": statistics.median(br_ctrl), "controller_update_ms_best": br_ctrl[0]}

    # ---- end-to-end: host buffers in, host results out, through moe_route_step_host
    e2e_steps = max(3, min(args.steps, 30))
    rh = binding.Router(wl.L, wl.E, wl.K, wl.H, wl.T, controller="id", host_staging=True, device=dev)
    xh = [x.cpu().pin_memory() for x in xs[:2]]
    wh = w.cpu().pin_memory()
    ih = torch.empty(wl.L, wl.T, wl.K, dtype=torch.int32).pin_memory()
    gh = torch.empty(wl.L, wl.T, wl.K, dtype=torch.float32).pin_memory()
    vio_h = torch.empty(2, wl.L, dtype=torch.float32).pin_memory()

    def e2e_step(i):
        rh.route_step_host(xh[i % 2], wh, ih, gh)
        if dist is not None:
            dp.allreduce_loads(rh, dist)
        rh.controller_update()
        _, _, mx, mn = rh.load_stats()
        vio_h[0].copy_(mx, non_blocking=True)
        vio_h[1].copy_(mn, non_blocking=True)

    for i in range(3):
        e2e_step(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    rh.poll()
    clocks = sampler.stop()

    # ---- max over ranks
    if dist is not None:
        t = torch.tensor([total_ms, e2e_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms, e2e_ms = t.tolist()
    tokens_per_step = wl.L * wl.T * world
    value = tokens_per_step * args.steps / (total_ms * 1e-3)
    e2e_value = tokens_per_step * e2e_steps / (e2e_ms * 1e-3)

    if rank == 0:
        pk = peaks()
        flops = 2.0 * wl.L * wl.T * wl.H * wl.E
        bracketed_ms = sum(route_ms) / len(route_ms)
        # Consecutive launches overlap (the next routing kernel's prologue and loads run under the controller
        # update of the step before), and an event pair around a launch switches that overlap off for it.
        # The launch duration used for the roofline is therefore the smaller of the bracketed time and the
        # whole step's time (events around the timed region / steps), which contains exactly one routing launch
        # plus the controller kernel.
        avg_route_ms = min(bracketed_ms, total_ms / args.steps)
        achieved = flops / (avg_route_ms * 1e-3) / 1e12
        roofline = {"kernel": "route_step_kernel", "bound": "tensor", "achieved": achieved, "peak": pk["tflops"],
                    "unit": "TFLOP/s", "frac": achieved / pk["tflops"], "peak_source": pk["source"] + " (burst bf16)",
                    "frac_of_sustained": (achieved / pk["tflops_sustained"]) if pk.get("tflops_sustained") else None,
                    "avg_launch_ms": avg_route_ms, "bracketed_launch_ms": bracketed_ms, "best_bracketed_launch_ms": min(route_ms),
                    "launches_bracketed": len(route_ms),
                    "algorithmic_flops_per_launch": flops,
                    "traffic": NCU_TRAFFIC_BYTES.get(wl.name)}
        cpu = None
        if not args.no_cpu_baseline:
            threads = os.cpu_count() or 1
            rate, n_tok, dt = cpu_oracle_rate(wl, threads, args.ref_tokens_per_thread)
            rate1, n_tok1, dt1 = cpu_oracle_rate(wl, 1, max(64, args.ref_tokens_per_thread // 4))
            cpu = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle",
                   "sample": f"{n_tok} of {wl.T} tokens of layer 0, all stages, {dt:.1f} s",
                   "single_thread": {"value": rate1, "sample": f"{n_tok1} tokens, {dt1:.1f} s"}}
        h2d = wl.L * wl.T * wl.H * 2 + wl.L * wl.E * wl.H * 2
        d2h = 2 * wl.L * wl.T * wl.K * 4 + 2 * wl.L * 4
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": wl.name, "T": wl.T, "H": wl.H, "E": wl.E, "K": wl.K, "L": wl.L,
                           "controller": "id", "parallelism": f"dp{world}",
                           "l2": f"ring of {ring} distinct input batches ({ring * wl.L * wl.T * wl.H * 2 / 1e6:.0f} MB) "
                                 "cycled, larger than the 126 MB L2"},
                "roofline": roofline, "cpu_baseline": cpu,
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                        "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps},
                "gpu_launches": int(launches), "clocks": clocks, "breakdown": breakdown,
                "last_step": {"maxvio_max": float(maxvio.max()), "minvio_max": float(minvio.max())}}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
