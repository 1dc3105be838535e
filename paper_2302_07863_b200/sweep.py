"""Threshold sweep (the shape of the paper's Figure 10 trade-off curves): tokens/s, fallback
and rollback rate of the BiLD loop over a grid of (alpha_FB, alpha_RB).

    python -m paper_2302_07863_b200.sweep --workload t5_long

The two encoders run once; every grid point is one device-side generation of the workload's
length, timed with CUDA events on the context's stream (mean of `--reps` runs after one untimed
run).  The grid is centred on the thresholds stored with the workload's oracle run: alpha_FB
scaled by the factors of `--fb`, alpha_RB by those of `--rb`.  One JSON line per point, or one row of a
markdown table with `--md`.  `--max-draft` overrides the workload's cap on consecutive drafted tokens (the fallback
rate cannot go below 1 / (cap + 1): after `cap` drafts the hand-over is forced).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="t5_long")
    ap.add_argument("--fb", default="0.2,0.45,0.7,1.0,1.4")
    ap.add_argument("--rb", default="0.95,1.0,1.15,1.3,1.8")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--max-draft", type=int, default=0)
    ap.add_argument("--md", action="store_true")
    a = ap.parse_args()
    import torch
    assert torch.cuda.is_available(), "needs a CUDA device"
    from workloads import WORKLOADS
    from paper_2302_07863_b200 import MODE_BILD, MODE_LARGE_ONLY, build
    from paper_2302_07863_b200.synthetic import make_context
    build.build()
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with open(os.path.join(root, "tests", "golden", a.workload + ".json")) as f:
        g = json.load(f)
    wl = WORKLOADS[a.workload]
    ctx, ids, _ = make_context(a.workload, g["scale_small"]["scale"], g["scale_large"]["scale"],
                               max_draft=a.max_draft or None)
    ctx.encode(ids)
    th = g["thresholds"]

    def timed(mode, afb, arb):
        r = ctx.generate(mode, afb, arb, wl.gen_len)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(a.reps):
            ctx.generate_async(mode, afb, arb, wl.gen_len)
        e1.record()
        e1.synchronize()
        return r, e0.elapsed_time(e1) / a.reps

    r, ms = timed(MODE_LARGE_ONLY, 0.0, float("inf"))
    large_tps = len(r["tokens"]) / ms * 1e3
    if a.md:
        print(f"Large model alone: {large_tps:.0f} tokens/s ({ms:.1f} ms for {len(r['tokens'])} tokens); "
              f"cap on consecutive drafts: {a.max_draft or wl.max_draft}.\n")
        print("| alpha_FB | alpha_RB | tokens/s | speed-up vs large | fallback rate | rollback rate | agreement with large |")
        print("|---|---|---|---|---|---|---|")
    else:
        print(json.dumps({"point": "large model alone", "tokens_per_s": large_tps, "ms": ms}))
    for fs in [float(x) for x in a.fb.split(",")]:
        for rs in [float(x) for x in a.rb.split(",")]:
            afb, arb = th["alpha_fb"] * fs, th["alpha_rb"] * rs
            r, ms = timed(MODE_BILD, afb, arb)
            st, n = r["stats"], len(r["tokens"])
            rec = ({"alpha_fb": afb, "alpha_rb": arb, "tokens_per_s": n / ms * 1e3, "ms": ms,
                              "fallback_rate": (st["fallbacks"] + st["forced"]) / max(1, n),
                              "rollback_rate": st["rollbacks"] / max(1, n),
                              "speedup_vs_large": n / ms * 1e3 / large_tps,
                              "agree_with_large": sum(x == y for x, y in zip(r["tokens"], g["large_only"]["tokens"])) / max(1, n)})
            if a.md:
                print(f"| {afb:.3f} | {arb:.1f} | {rec['tokens_per_s']:.0f} | {rec['speedup_vs_large']:.2f}x | "
                      f"{100 * rec['fallback_rate']:.1f} % | {100 * rec['rollback_rate']:.1f} % | "
                      f"{100 * rec['agree_with_large']:.1f} % |", flush=True)
            else:
                print(json.dumps(rec), flush=True)


if __name__ == "__main__":
    main()
