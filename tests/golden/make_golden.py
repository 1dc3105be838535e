"""Writes tests/golden/<workload>.json by running ONLY the CPU oracle.

    python tests/golden/make_golden.py tiny odd odd_bf16 tiny_bf16 t5_sum mt5_mt

Per workload: the calibrated logit scales and thresholds (oracle/calibrate.py),
the oracle's BiLD tokens / trace / counters / decision margins, the two greedy
baselines, and a sample of the logits of every model call of the BiLD run
(arg-max, log-sum-exp, max probability and the logits at a fixed set of
vocabulary indices), which the GPU parity tests compare against without having
to re-run the oracle at full size.  If the file exists already, its calibration
(logit scales, thresholds) is kept and only the oracle runs are repeated
(`--recalibrate` calibrates afresh).  No value here comes from the CUDA path.
The paper prints no numeric worked example, so none of these are the paper's.
"""
import json
import math
import os
import sys
import time

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))

from oracle import bild, calibrate                                   # noqa: E402
from oracle.t5 import Model                                          # noqa: E402
from workloads import MODEL_SHAPES, WORKLOADS, gen_ids, gen_model    # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))
N_SAMPLE = 24

BANDS = {   # (fallback band, rollback band, min margin, max runs)
    "tiny": ((0.15, 0.25), (0.05, 0.15), 1e-3, 400),
    "odd": ((0.15, 0.25), (0.05, 0.15), 1e-3, 400),
    "odd_bf16": ((0.15, 0.25), (0.05, 0.15), 1e-3, 400),
    "tiny_bf16": ((0.15, 0.25), (0.05, 0.15), 1e-3, 400),
    "t5_sum": ((0.15, 0.25), (0.01, 0.08), 0.0, 60),
    "mt5_mt": ((0.15, 0.25), (0.01, 0.08), 0.0, 12),
    "t5_long": ((0.15, 0.25), (0.01, 0.08), 0.0, 6),
}


def sample_rows(r, vocab, seed):
    rng = np.random.default_rng(seed)
    idx = np.sort(rng.choice(vocab, size=min(N_SAMPLE, vocab), replace=False))
    out = []
    for tag, first, Z in r["logits"]:
        Z2 = Z[None] if Z.ndim == 1 else Z
        for i, z in enumerate(Z2):
            t, pmax, lse, gap = bild.max_prob(z)
            out.append(dict(model=tag, first=int(first), row=i, argmax=t, pmax=pmax, lse=lse, gap=gap,
                            zmax=float(z[t]), z=[float(v) for v in z[idx]]))
    return [int(i) for i in idx], out


def fin(v):
    """JSON has no infinity: margins that do not apply are stored as null."""
    return None if math.isinf(v) else float(v)


def main(names):
    recal = "--recalibrate" in names
    for name in [n for n in names if not n.startswith("--")]:
        t0 = time.time()
        wl = WORKLOADS[name]
        sS, sL = MODEL_SHAPES[wl.small], MODEL_SHAPES[wl.large]
        S = Model(sS, gen_model(sS, wl.seed, wl.dtype))
        L = Model(sL, gen_model(sL, wl.seed, wl.dtype))
        ids = gen_ids(sS.vocab, wl.enc_len, wl.seed)
        print(f"[{name}] models ready {time.time() - t0:.1f}s", flush=True)
        path = os.path.join(HERE, name + ".json")
        old = None
        if os.path.exists(path) and not recal:
            with open(path) as f:
                old = json.load(f)
            cs, cl, th = old["scale_small"], old["scale_large"], old["thresholds"]
            S.logit_scale, L.logit_scale = float(cs["scale"]), float(cl["scale"])
        else:
            cs = calibrate.calibrate_scale(S, ids, wl.gen_len)
            cl = calibrate.calibrate_scale(L, ids, wl.gen_len)
            print(f"[{name}] scales {cs} {cl} {time.time() - t0:.1f}s", flush=True)
            fb, rb, mm, runs = BANDS[name]
            th = calibrate.calibrate_thresholds(S, L, ids, wl.gen_len, wl.max_draft, fb, rb, mm, runs)
        print(f"[{name}] thresholds {th} {time.time() - t0:.1f}s", flush=True)
        r = bild.generate(S, L, ids, th["alpha_fb"], th["alpha_rb"], wl.gen_len, max_draft=wl.max_draft,
                          keep_logits=True)
        idx, rows = sample_rows(r, sS.vocab, wl.seed)
        rs = bild.generate(S, L, ids, 0.0, math.inf, wl.gen_len, mode="small")
        rl = bild.generate(S, L, ids, 0.0, math.inf, wl.gen_len, mode="large")
        out = dict(
            workload=name, seed=wl.seed, enc_len=wl.enc_len, gen_len=wl.gen_len, max_draft=wl.max_draft,
            scale_small=cs, scale_large=cl, thresholds=th,
            bild=dict(tokens=r["tokens"], trace=[list(t) for t in r["trace"]], stats=r["stats"],
                      margins={k: float(v) for k, v in r["margins"].items()},
                      trace_margins=[[fin(v) for v in t] for t in r["trace_margins"]]),
            small_only=dict(tokens=rs["tokens"], argmax_margin=float(rs["margins"]["argmax"]),
                            gaps=[float(t[0]) for t in rs["trace_margins"]]),
            large_only=dict(tokens=rl["tokens"], argmax_margin=float(rl["margins"]["argmax"]),
                            gaps=[float(t[0]) for t in rl["trace_margins"]]),
            sample_idx=idx, sample_rows=rows)
        if old is not None:   # same calibration, same oracle: the runs must come out as before
            assert old["bild"]["tokens"] == out["bild"]["tokens"] and old["bild"]["stats"] == out["bild"]["stats"], name
        with open(path, "w") as f:
            json.dump(out, f)
        print(f"[{name}] done {time.time() - t0:.1f}s  stats {r['stats']}", flush=True)


if __name__ == "__main__":
    main(sys.argv[1:] or ["tiny", "odd", "odd_bf16", "tiny_bf16"])
