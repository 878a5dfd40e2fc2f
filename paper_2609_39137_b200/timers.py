"""Cycle accounting of the routing kernel per warp role, from the instrumented build (-DMOE_KERNEL_TIMERS).

    python -m paper_2609_39137_b200.timers [workload] [layers]

Builds libmoe_route_b200_timers.so if needed, runs a few routing steps of the named synthetic workload and
prints, per CTA and per epilogue warp, where the cycles went (waits, issue, the epilogue's phases) and the
timeline of the first CTA pair's last item.  A development aid: the instrumented kernel is a few per cent slower
than the production build and its numbers are clock64 cycles, not profiler counters.
"""
from __future__ import annotations

import ctypes as C
import sys

import numpy as np
import torch

from . import binding, build, synth


def main(argv):
    name = argv[1] if len(argv) > 1 else "top10_single"
    wl = synth.WORKLOADS[name]
    if len(argv) > 2:
        wl = wl.with_(L=int(argv[2]))
    binding.LIB_PATH = build.build(timers=True)
    lib = binding.load()
    lib.moe_debug_read_timers.argtypes = [C.c_void_p, C.c_int]
    lib.moe_debug_read_marks.argtypes = [C.c_void_p]
    dev = "cuda"
    w = torch.stack([synth.router_weights(wl, l, dev) for l in range(wl.L)])
    xs = [torch.stack([synth.hidden_states(wl, l, s, dev) for l in range(wl.L)]) for s in range(3)]
    r = binding.Router(wl.L, wl.E, wl.K, wl.H, wl.T)
    for i in range(5):
        r.route_step(xs[i % 3], w)
        r.controller_update()
    r.poll()
    acc = (C.c_longlong * 32)()
    lib.moe_debug_read_timers(acc, 1)                       # reset
    n = 10
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(n):
        r.route_step(xs[i % 3], w)
        r.controller_update()
    e1.record()
    torch.cuda.synchronize()
    lib.moe_debug_read_timers(acc, 0)
    t = np.array(list(acc), dtype=np.float64)
    tile_pairs = wl.L * ((wl.T + 255) // 256)
    pairs = min(74, tile_pairs)
    ctas, items = 2 * pairs, tile_pairs / pairs
    print(f"{name} L={wl.L}: {e0.elapsed_time(e1) / n * 1e3:.1f} us per step (instrumented build), "
          f"{ctas} CTAs with work, {items:.1f} tiles per pair")
    kc = lambda v, per: v / n / per / 1e3
    print("producer, kcycles per CTA:      wait for a free stage %.1f, issue %.1f" % (kc(t[0], ctas), kc(t[1], ctas)))
    print("MMA issuer, kcycles per pair:   wait for a free accumulator %.1f, wait for a full stage %.1f, issue %.1f"
          % (kc(t[8], pairs), kc(t[9], pairs), kc(t[10], pairs)))
    ew = ctas * 8
    names = ["wait for accumulators", "seed pass", "scan", "fallback drain", "selection and outputs",
             "between items (layer change, decode)"]
    print("epilogue, kcycles per warp:     " + ", ".join(f"{nm} {kc(t[16 + i], ew):.1f}" for i, nm in enumerate(names)))
    print("per CTA (us): set-up %.1f, role loops %.1f, teardown %.1f" % (t[26] / n / ctas / 1e3, t[27] / n / ctas / 1e3,
                                                                       t[28] / n / ctas / 1e3))
    marks = (C.c_ulonglong * 32)()
    lib.moe_debug_read_marks(marks)
    m = np.array(list(marks), dtype=np.float64)
    labels = {1: "set-up done", 2: "first stage full", 3: "chunk 1 issued", 4: "chunk 2 issued", 5: "chunk 3 issued",
              6: "chunk 1 accumulators ready", 7: "chunk 2 ready", 8: "chunk 3 ready", 9: "chunk 1 scanned",
              10: "chunk 2 scanned", 11: "chunk 3 scanned", 12: "selection and outputs done", 13: "role loops left",
              14: "end of the CTA"}
    print("first CTA pair, last item of the last launch (us after the CTA's start):")
    for k in sorted(labels, key=lambda k: m[k]):
        if m[k] >= m[0] > 0:
            print(f"  {labels[k]:28s} {(m[k] - m[0]) / 1e3:8.2f}")


if __name__ == "__main__":
    main(sys.argv)
