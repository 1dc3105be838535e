"""The two ablations of the paper's Section 4.4 on a synthetic pair, as speed / agreement curves:

  * no rollback policy: alpha_RB = +inf, alpha_FB swept (the large model's predictions only
    take effect at fallbacks);
  * no fallback policy: alpha_FB = 0 and a hand-over to the large model after a fixed number of
    small-model steps (window 3..10 = the context's max_draft), alpha_RB as stored.

    python -m paper_2302_07863_b200.ablation --workload t5_sum

Quality metrics need trained models and datasets and are out of scope; the columns here are
tokens/s, speed-up over the large model alone, fallback / rollback rates and the fraction of
positions whose token equals the large model's own greedy output.  One JSON line per point.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="t5_sum")
    ap.add_argument("--fb", default="0.5,0.75,1.0,1.25,1.5", help="factors on the stored alpha_FB")
    ap.add_argument("--windows", default="3,4,5,6,7,8,9,10")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--md", action="store_true", help="rows of a markdown table instead of JSON lines")
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
    th = g["thresholds"]
    inf = float("inf")

    def timed(ctx, mode, afb, arb):
        r = ctx.generate(mode, afb, arb, wl.gen_len)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(a.reps):
            ctx.generate_async(mode, afb, arb, wl.gen_len)
        e1.record()
        e1.synchronize()
        return r, e0.elapsed_time(e1) / a.reps

    def line(variant, extra, r, ms, large_tps):
        st, n = r["stats"], len(r["tokens"])
        rec = {"variant": variant, "tokens_per_s": n / ms * 1e3, "speedup_vs_large": n / ms * 1e3 / large_tps,
               "fallback_rate": (st["fallbacks"] + st["forced"]) / max(1, n), "rollback_rate": st["rollbacks"] / max(1, n),
               "agree_with_large": sum(x == y for x, y in zip(r["tokens"], g["large_only"]["tokens"])) / max(1, n)}
        rec.update(extra)
        if a.md:
            second = f"window {rec['window']} (alpha_RB {rec['alpha_rb']:.1f})" if "window" in rec else (
                "inf" if rec["alpha_rb"] == "inf" else f"{rec['alpha_rb']:.1f}")
            print(f"| {variant} | {rec.get('alpha_fb', 0):.3g} | {second} | {rec['tokens_per_s']:.0f} | "
                  f"{rec['speedup_vs_large']:.2f}x | {100 * rec['fallback_rate']:.1f} % | "
                  f"{100 * rec['rollback_rate']:.1f} % |", flush=True)
        else:
            print(json.dumps(rec), flush=True)

    ctx, ids, _ = make_context(a.workload, g["scale_small"]["scale"], g["scale_large"]["scale"])
    ctx.encode(ids)
    r, ms = timed(ctx, MODE_LARGE_ONLY, 0.0, inf)
    large_tps = len(r["tokens"]) / ms * 1e3
    if a.md:
        print(f"Large model alone: {large_tps:.0f} tokens/s.\n")
        print("| variant | alpha_FB | alpha_RB / window | tokens/s | speed-up vs large | fallback rate | rollback rate |")
        print("|---|---|---|---|---|---|---|", flush=True)
    else:
        print(json.dumps({"variant": "large model alone", "tokens_per_s": large_tps}), flush=True)
    for f in [float(x) for x in a.fb.split(",")]:
        afb = th["alpha_fb"] * f
        r, ms = timed(ctx, MODE_BILD, afb, th["alpha_rb"])
        line("fallback + rollback", {"alpha_fb": afb, "alpha_rb": th["alpha_rb"]}, r, ms, large_tps)
        r, ms = timed(ctx, MODE_BILD, afb, inf)
        line("no rollback", {"alpha_fb": afb, "alpha_rb": "inf"}, r, ms, large_tps)
    ctx.close()
    for w in [int(x) for x in a.windows.split(",")]:
        ctx, ids, _ = make_context(a.workload, g["scale_small"]["scale"], g["scale_large"]["scale"], max_draft=w)
        ctx.encode(ids)
        r, ms = timed(ctx, MODE_BILD, 0.0, th["alpha_rb"])
        line("no fallback policy, fixed window", {"window": w, "alpha_rb": th["alpha_rb"]}, r, ms, large_tps)
        ctx.close()


if __name__ == "__main__":
    main()
