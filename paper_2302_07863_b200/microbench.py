"""Per-pass micro-benchmark of the decoder passes (time, achieved HBM GB/s, fraction of peak).

    python -m paper_2302_07863_b200.microbench --workload t5_sum --k 1,2,4,8,16 --cache 64,256,1024

For every (k, cache length) it replays the large model's block pass as a CUDA graph
(bild_time_pass) and prints one JSON line; `--small` adds the small model's single step.
Bytes are the algorithmic bytes of the pass: every weight matrix and the LM head once, the
cached self-attention rows and the cross-attention K/V of every layer, the k embedding rows.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def pass_bytes(s, w_bytes, kv_bytes, cache_rows, enc_len, k):
    g = 3 if s.ffn == "gated_gelu" else 2
    I, d, F, V, L = s.inner, s.d_model, s.d_ff, s.vocab, s.n_layers
    weights = w_bytes * (L * (6 * I * d + g * d * F) + V * d)
    kv = kv_bytes * L * (2 * (cache_rows + k) * I + 2 * enc_len * I)
    return weights + kv + w_bytes * k * d


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="t5_sum")
    ap.add_argument("--k", default="1,2,4,8,16")
    ap.add_argument("--cache", default="64,256,1024")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--small", action="store_true")
    ap.add_argument("--dist", type=int, default=0, help="also time N single passes per point: median, p10, p90")
    ap.add_argument("--peak-gbs", type=float, default=0.0)
    ap.add_argument("--tuning", default="", help="bild_tuning fields, e.g. pdl=0,fused=1")
    a = ap.parse_args()
    import torch
    assert torch.cuda.is_available(), "needs a CUDA device"
    from workloads import MODEL_SHAPES, WORKLOADS
    from paper_2302_07863_b200 import build
    from paper_2302_07863_b200.synthetic import make_context
    build.build()
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with open(os.path.join(root, "tests", "golden", a.workload + ".json")) as f:
        g = json.load(f)
    peak = a.peak_gbs
    if not peak:
        p = os.path.join(root, "MEASURED_PEAKS.json")
        peak = float(json.load(open(p))["hbm_gbs"]) if os.path.exists(p) else 6650.0
    tf_peak = 1590.0
    pk = os.path.join(root, "MEASURED_PEAKS.json")
    if os.path.exists(pk):
        tf_peak = float(json.load(open(pk)).get("bf16_tflops", tf_peak))
    ks = [int(x) for x in a.k.split(",")]
    caches = [int(x) for x in a.cache.split(",")]
    wl = WORKLOADS[a.workload]
    tuning = {kv.split("=")[0]: int(kv.split("=")[1]) for kv in a.tuning.split(",") if kv}
    ctx, ids, _ = make_context(a.workload, g["scale_small"]["scale"], g["scale_large"]["scale"],
                               max_dec_len=max(caches) + 16 + 1, tuning=tuning or None)
    ctx.encode(ids)
    wb = 2 if wl.dtype == "bf16" else 4
    sS, sL = MODEL_SHAPES[wl.small], MODEL_SHAPES[wl.large]
    def dist(which, k, cache, cold_after=None):
        """median / p10 / p90 (us) of a.dist single passes; cold_after: run that large pass before each one"""
        if not a.dist:
            return {}
        ts = []
        for _ in range(a.dist):
            if cold_after is not None:
                ctx.time_pass(1, cold_after, cache, 1)
                ts.append(ctx.time_pass(which, k, cache, -1) * 1e3)
            else:
                ts.append(ctx.time_pass(which, k, cache, 1) * 1e3)
        ts.sort()
        q = lambda f: ts[min(len(ts) - 1, int(f * len(ts)))]
        return {"median_us": q(0.5), "p10_us": q(0.1), "p90_us": q(0.9), "n": len(ts)}

    nominal = 8000.0   # GB/s, the nominal HBM3e figure
    for cache in caches:
        if a.small:
            ms = ctx.time_pass(0, 1, cache, a.iters)
            b = pass_bytes(sS, wb, wb, cache, wl.enc_len, 1)
            rec = {"pass": "small step", "k": 1, "cache": cache, "us": ms * 1e3, "GBs": b / ms / 1e6,
                   "frac_of_peak": b / ms / 1e6 / peak, "frac_of_nominal": b / ms / 1e6 / nominal, "bytes": b}
            rec.update(dist(0, 1, cache))
            print(json.dumps(rec))
            if a.dist:   # the small model's weights fit in L2: time the step right after a large pass as well
                rec = {"pass": "small step after a large pass (L2-cold)", "k": 1, "cache": cache, "bytes": b}
                rec.update(dist(0, 1, cache, cold_after=4))
                print(json.dumps(rec))
        for k in ks:
            ms = ctx.time_pass(1, k, cache, a.iters)
            b = pass_bytes(sL, wb, wb, cache, wl.enc_len, k)
            # tensor-pipe utilisation, derived: the pass's matrix products (2 k flops per weight; single-row passes run
            # them on the plain ALUs) over its duration, against the measured dense bf16 rate
            g = 3 if sL.ffn == "gated_gelu" else 2
            flops = 2.0 * k * (sL.n_layers * (6 * sL.inner * sL.d_model + g * sL.d_model * sL.d_ff) + sL.vocab * sL.d_model)
            rec = {"pass": "large block pass", "k": k, "cache": cache, "us": ms * 1e3, "GBs": b / ms / 1e6,
                   "frac_of_peak": b / ms / 1e6 / peak, "frac_of_nominal": b / ms / 1e6 / nominal, "bytes": b,
                   "tensor_util_derived": (flops / (ms * 1e-3) / 1e12 / tf_peak) if k > 1 else 0.0}
            rec.update(dist(1, k, cache))
            print(json.dumps(rec))


if __name__ == "__main__":
    main()
