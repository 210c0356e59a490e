"""Phase table of the fused decode kernel from its global-timer stamps.

    python -m paper_2501_10054_b200.phase_stamps [workload] [--batch B] [--layers L] [--calls N]

Builds libtardis_stamps.so (the library compiled with -DTARDIS_PHASE_STAMPS), runs batch-B decode calls that
rotate over L independently seeded layers (so that a call finds its state in HBM, not in L2), reads the stamps
of the last launch through tardis_debug_phase_stamps and prints, per phase boundary, the distribution over the
CTAs of the time since the first CTA had x.  Profiling aid only: the stamped kernel is a little slower than
the ordinary one (the mean time per call of both is printed).
"""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

SLOTS = {0: "kernel entry", 1: "x loaded", 2: "fixed-point x ready", 3: "predictor done",
         4: "folded product done (first streaming warp)", 5: "flagged list complete", 6: "result fixing done",
         7: "CTA counted", 8: "y written (last CTA)"}


def time_calls(T, handles, x, y, batch, calls):
    n = x.shape[0] // batch
    def run(k):
        for i in range(k):
            j = (i % n) * batch
            T.tardis_ffn_forward(handles[i % len(handles)], x[j:j + batch], y[j:j + batch])
    run(30)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    run(calls)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / calls


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("workload", nargs="?", default="decode_7b")
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--calls", type=int, default=200)
    args = ap.parse_args()
    import paper_2501_10054_b200 as T
    from paper_2501_10054_b200 import build as tbuild
    import workloads as W
    cfg = W.CONFIGS[args.workload]
    dev = torch.device("cuda", 0)
    x = W.make_tokens(cfg, 64, 0, device=dev)
    y = torch.empty_like(x)
    layers = [W.make_layer(cfg, seed=l, device=dev) for l in range(args.layers)]

    tbuild.build()
    T.load_library()
    hs = [T.fold_layer(L) for L in layers]
    us_plain = time_calls(T, hs, x, y, args.batch, args.calls)
    for h in hs:
        T.tardis_destroy(h)

    T._lib = None
    T.LIB_PATH = tbuild.build(stamps=True)
    T.load_library()
    hs = [T.fold_layer(L) for L in layers]
    us = time_calls(T, hs, x, y, args.batch, args.calls)
    buf = T.tardis_debug_phase_stamps(512)
    grid = int((buf[:, 0] != 0).sum())
    buf = buf[:grid]
    t0 = buf[:, 1].min()
    print("%s, batch %d, %d layers in rotation: %.2f us per call (%.2f us with the stamps compiled in); grid %d CTAs"
          % (cfg.name, args.batch, args.layers, us_plain, us, grid))
    print("time since the first CTA had x [us]:  %-46s %7s %7s %7s %7s %7s" % ("", "min", "p10", "median", "p90", "max"))
    for slot, name in SLOTS.items():
        v = buf[:, slot]
        v = (v[v != 0] - t0) / 1e3
        if slot == 8:
            v = v[v > 0][-1:] if (v > 0).any() else v[:0]      # only the last CTA of the last launch writes it
        if len(v):
            print("  %-82s %7.2f %7.2f %7.2f %7.2f %7.2f" % (name, v.min(), np.percentile(v, 10), np.median(v), np.percentile(v, 90), v.max()))
    nfl = buf[:, 9]
    print("flagged neurons per CTA: mean %.2f, max %d, total %d" % (nfl.mean(), nfl.max(), nfl.sum()))
    for h in hs:
        T.tardis_destroy(h)


if __name__ == "__main__":
    main()
