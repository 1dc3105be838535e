"""CPU oracle, part 3: calibration of the synthetic workloads.

TEST INFRASTRUCTURE ONLY: see the header of oracle/t5.py.

The paper sweeps the two thresholds on trained models (evaluation details in
the supplementary material) and reports the resulting fallback and rollback
percentages (comparison table with speculative sampling).  Random models have
no trained confidence, so two things are chosen here, by running the oracle:

* a logit scale per model such that the median of max-softmax-probability over
  that model's own greedy decode is 0.5 (arg-max does not depend on a positive
  scale, so one greedy run suffices);
* (alpha_FB, alpha_RB) such that the realised fallback and rollback rates of
  the BiLD run fall in a requested band.  Rates are events per generated token.
"""
from __future__ import annotations

import math

import numpy as np

from . import bild
from .t5 import Model


def pmax_at_scale(z: np.ndarray, s: float) -> float:
    zz = s * z
    return 1.0 / float(np.sum(np.exp(zz - zz.max())))


def calibrate_scale(model: Model, enc_ids, gen_len: int, target_median: float = 0.5) -> dict:
    """Bisection on the logit scale; returns scale and the p_max percentiles."""
    model.logit_scale = 1.0
    r = bild.generate(model, None, enc_ids, 0.0, math.inf, gen_len, mode="small", keep_logits=True)
    zs = [z for _, _, z in r["logits"]]
    lo, hi = 1e-3, 1e4
    for _ in range(60):
        mid = math.sqrt(lo * hi)
        med = float(np.median([pmax_at_scale(z, mid) for z in zs]))
        lo, hi = (mid, hi) if med < target_median else (lo, mid)
    s = float(np.float32(math.sqrt(lo * hi)))       # representable in the fp32 config field
    pm = [pmax_at_scale(z, s) for z in zs]
    model.logit_scale = s
    return dict(scale=s, pmax_pct_5_50_95=[float(v) for v in np.percentile(pm, [5, 50, 95])],
                distinct_tokens=len(set(r["tokens"])))


def _between(values, q: float) -> float:
    """A threshold at quantile level q that sits half-way between two
    neighbouring observed values (so that no observed value ties with it),
    rounded to fp32."""
    a = np.sort(np.asarray(values, dtype=np.float64))
    if len(a) == 1:
        return float(np.float32(a[0] * 0.999))
    i = int(min(max(math.floor(q * (len(a) - 1)), 0), len(a) - 2))
    return float(np.float32(0.5 * (a[i] + a[i + 1])))


def rates(r: dict) -> tuple:
    n = max(1, len(r["tokens"]))
    st = r["stats"]
    return (st["fallbacks"] + st["forced"]) / n, st["rollbacks"] / n


def calibrate_thresholds(small: Model, large: Model, enc_ids, gen_len: int, max_draft: int,
                         fb_band=(0.15, 0.25), rb_band=(0.05, 0.15), min_margin: float = 0.0,
                         max_runs: int = 60) -> dict:
    """Try quantile levels of the observed p_max (for alpha_FB) and of the
    drafted tokens' distances (for alpha_RB), nearest to the band centres first,
    until the BiLD run's realised rates land in both bands and every decision
    margin exceeds min_margin.  Thresholds are rounded to fp32 so that the C ABI
    passes them exactly.  Returns the first hit, else the closest miss."""
    r0 = bild.generate(small, large, enc_ids, 0.0, math.inf, gen_len, max_draft=max_draft)
    pm = np.array([t[5] for t in r0["trace"] if t[0] == bild.KIND_SMALL_ACCEPT])
    c_fb, c_rb = 0.5 * sum(fb_band), 0.5 * sum(rb_band)
    levels_fb = sorted(np.linspace(0.02, 0.40, 20), key=lambda q: abs(q - c_fb))
    levels_rb = sorted(np.linspace(0.005, 0.30, 20), key=lambda q: abs(q - 0.5 * c_rb))
    best, runs = None, 0
    for q_fb in levels_fb:
        a_fb = _between(pm, q_fb)
        r1 = bild.generate(small, large, enc_ids, a_fb, math.inf, gen_len, max_draft=max_draft,
                           keep_logits=True)
        d_pool = _draft_distances(r1)       # distances of every drafted token, no-rollback run
        if len(d_pool) == 0:
            continue
        for q_rb in levels_rb:
            a_rb = _between(d_pool, 1.0 - q_rb)
            r = bild.generate(small, large, enc_ids, a_fb, a_rb, gen_len, max_draft=max_draft)
            runs += 1
            fb, rb = rates(r)
            ok = (fb_band[0] <= fb <= fb_band[1] and rb_band[0] <= rb <= rb_band[1]
                  and min(r["margins"].values()) > min_margin)
            miss = abs(fb - c_fb) / c_fb + abs(rb - c_rb) / c_rb + (0 if ok else 10)
            cand = dict(alpha_fb=a_fb, alpha_rb=a_rb, fallback_rate=fb, rollback_rate=rb,
                        margins={k: float(v) for k, v in r["margins"].items()}, in_band=ok,
                        runs=runs, miss=miss)
            if best is None or miss < best["miss"]:
                best = cand
            if ok or runs >= max_runs:
                best["runs"] = runs
                return best
            if rb < rb_band[0] and fb > fb_band[1]:
                break               # more rollbacks only add fallbacks: next alpha_FB
    return best


def _draft_distances(r: dict) -> np.ndarray:
    out = []
    y = [0] + list(r["tokens"])
    for tag, first, Z in r["logits"]:
        if tag != "L":
            continue
        for i in range(Z.shape[0] - 1):
            z = Z[i]
            lse = z.max() + math.log(np.sum(np.exp(z - z.max())))
            out.append(lse - z[y[first + i + 1]])
    return np.array(out)
