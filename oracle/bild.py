"""CPU oracle, part 2: the Big Little Decoder loop (Algorithm 1) with the
fallback policy (Section 3.3) and the rollback policy (Section 3.4, Eq. 3).

TEST INFRASTRUCTURE ONLY: see the header of oracle/t5.py.

BiLD is a policy, not a faster route to a closed-form result, so this file is
the algorithm taken step by step in the paper's order.  Readings of the places
where the paper is loose (each is a deliberate choice):

* fallback iff  max_y p_S(y | y_1:n-1) < alpha_FB  (the boxed policy of
  Section 3.3; equality keeps the small model's token);
* the distance d is the cross entropy between the small model's hard label and
  the large model's soft label, d = -ln p_L(y_S) (Sections 3.4 and 4.1, and the
  evaluation details of the supplementary material);
* rollback iff d > alpha_RB (Eq. 3, strict), at the smallest such position;
* only the pending, not yet verified small-model tokens are scanned; a token
  emitted by the large model is never re-judged;
* sample() is arg-max with the lowest index on ties (greedy decoding), or, for the
  sampling variant of the supplementary material ("BiLD with Sampling"), nucleus
  sampling from both models with the same two policies: the fallback test still uses
  the small model's maximum probability, the rollback distance is still -ln p_L of
  the token the small model drew.  The uniform numbers are INPUTS (one per model and
  output position: a token drawn again for the same position after a rollback uses
  the same number), so a run is a deterministic function of its arguments;
* the small model keeps at most `max_draft` tokens in a row (supplementary
  material, "maximum generation length of the small model"): once that many
  drafts are pending, the next small step still runs but control goes to the
  large model whatever its confidence ("forced fallback");
* the loop stops as soon as max_len tokens exist or the last token is EOS,
  even if drafts are pending;
* on rollback both models' caches are cut back to the replaced position.

Trace records are (kind, pos, token, k, m, value):
  kind 0 small-accept : token written at y[pos], value = p_max
  kind 1 fallback     : small model's rejected candidate for y[pos], value = p_max
  kind 2 forced       : same, but p_max was above the threshold
  kind 3 verify, no rollback : large model's token written at y[pos], k = block
                        size, m = -1, value = largest distance scanned (0 if none)
  kind 4 verify, rollback    : large model's token written at y[pos], m = index of
                        the first violating row, value = its distance
"""
from __future__ import annotations

import math

import numpy as np

from .t5 import Model

KIND_SMALL_ACCEPT, KIND_FALLBACK, KIND_FORCED, KIND_VERIFY_OK, KIND_ROLLBACK = 0, 1, 2, 3, 4


def max_prob(z: np.ndarray):
    """(argmax, max softmax probability, log-sum-exp, margin to runner-up)."""
    t = int(np.argmax(z))                       # lowest index on ties
    zmax = float(z[t])
    sumexp = float(np.sum(np.exp(z - zmax)))
    second = float(np.max(np.delete(z, t))) if z.size > 1 else -math.inf
    return t, 1.0 / sumexp, zmax + math.log(sumexp), zmax - second


def nucleus_sample(z: np.ndarray, top_p: float, u: float):
    """Nucleus (top-p) sampling of one token from softmax(z) with the uniform number u in [0, 1).

    The tokens are put in order of decreasing probability (equal probabilities: lower index first); the
    nucleus is the shortest prefix of that order whose probabilities add up to at least top_p; the drawn token
    is the first of the prefix at which the running sum exceeds u times the prefix's total (inverse CDF of the
    renormalised prefix).  Returns (token, nucleus size, margin), margin = how close (in probability) the two
    threshold comparisons came to going the other way."""
    zmax = float(np.max(z))
    e = np.exp(z - zmax)
    p = e / float(np.sum(e))
    order = np.argsort(-p, kind="stable")
    c = np.cumsum(p[order])
    hit = np.nonzero(c >= top_p)[0]
    n = int(hit[0]) + 1 if hit.size else int(z.size)            # rounding may keep the total just below 1
    target = u * float(c[n - 1])
    i = int(np.searchsorted(c[:n], target, side="right"))       # first running sum > target
    i = min(i, n - 1)
    near = [abs(float(c[n - 1]) - top_p), abs(float(c[i]) - target)]
    if n > 1:
        near.append(abs(float(c[n - 2]) - top_p))
    if i > 0:
        near.append(abs(float(c[i - 1]) - target))
    return int(order[i]), n, min(near)


def generate(small: Model, large: Model, enc_ids, alpha_fb: float, alpha_rb: float,
             max_len: int, max_draft: int = 10, mode: str = "bild",
             start_id: int = 0, eos_id: int = -1, keep_logits: bool = False,
             top_p: float = 0.0, u_small=None, u_large=None):
    """Run Algorithm 1.  Returns a dict with
    tokens  : y[1..n] (the start symbol is not included),
    trace   : list of (kind, pos, token, k, m, value),
    stats   : counters,
    margins : smallest decision margins seen (top-1 vs top-2 logit of every
              arg-max that was used, |p_max - alpha_FB|, |d - alpha_RB|),
    trace_margins : one (arg-max gap, |p_max - alpha_FB|, min |d_i - alpha_RB|) triple
              per trace record: the margins of the decisions that produced that
              record (inf where the record did not depend on such a decision),
    logits  : (if keep_logits) list of ("S"|"L", first position, array).

    top_p > 0 selects the sampling variant: every token is drawn by nucleus_sample with u_small[pos] (small
    model) or u_large[pos] (large model), pos = the position in y the token is written to; the trace margins
    then carry a fourth entry, the sampling margin of the record's token (in probability).
    """
    sampling = top_p > 0.0

    def pick(z, arg, u):   # the token a model emits: arg-max, or a draw
        if not sampling:
            return arg, math.inf
        tok, _, near = nucleus_sample(z, top_p, float(u))
        return tok, near
    assert mode in ("bild", "small", "large")
    cap = max_len + 1
    stS = small.start(enc_ids, cap) if mode != "large" else None
    stL = large.start(enc_ids, cap) if mode != "small" else None
    y = [start_id]
    n = 0                       # index of the last token in y
    L_len = 0                   # tokens the large model has consumed
    drafts = 0
    trace, logits, tmg = [], [], []
    stats = dict(small_steps=0, large_calls=0, fallbacks=0, forced=0, rollbacks=0,
                 discarded=0, sum_k=0)
    mg = dict(argmax=math.inf, fallback=math.inf, rollback=math.inf)

    while n < max_len and y[n] != eos_id:
        if mode != "large":
            zS = small.forward_one(stS, y[n])                       # Alg. 1: p_S <- SmallModel(y)
            stats["small_steps"] += 1
            if keep_logits:
                logits.append(("S", n, zS.copy()))
            t, pmax, _, gap = max_prob(zS)
            t, smg = pick(zS, t, u_small[n + 1] if sampling else 0.0)
            if sampling:
                gap = math.inf                                      # no arg-max decision is taken
            if mode == "small":
                mg["argmax"] = min(mg["argmax"], gap)
                y.append(t); n += 1
                trace.append((KIND_SMALL_ACCEPT, n, t, 0, -1, pmax))
                tmg.append((gap, math.inf, math.inf) + ((smg,) if sampling else ()))
                continue
            mg["fallback"] = min(mg["fallback"], abs(pmax - alpha_fb))
            confident = not (pmax < alpha_fb)                       # Section 3.3
            if confident and drafts < max_draft:
                mg["argmax"] = min(mg["argmax"], gap)
                y.append(t); n += 1; drafts += 1
                trace.append((KIND_SMALL_ACCEPT, n, t, 0, -1, pmax))
                tmg.append((gap, abs(pmax - alpha_fb), math.inf) + ((smg,) if sampling else ()))
                continue
            if confident:
                stats["forced"] += 1
                trace.append((KIND_FORCED, n + 1, t, 0, -1, pmax))
            else:
                stats["fallbacks"] += 1
                trace.append((KIND_FALLBACK, n + 1, t, 0, -1, pmax))
            tmg.append((gap, abs(pmax - alpha_fb), math.inf) + ((smg,) if sampling else ()))   # the record names the rejected candidate
        # ---- the large model reads every token it has not seen yet ----------
        k = n - L_len + 1
        ZL = large.forward_block(stL, y[L_len:n + 1])              # Alg. 1: p_L <- LargeModel(y)
        stats["large_calls"] += 1
        stats["sum_k"] += k
        if keep_logits:
            logits.append(("L", L_len, ZL.copy()))
        rows = [max_prob(ZL[i]) for i in range(k)]
        m_star, d_star, d_max, rb_here = -1, 0.0, 0.0, math.inf
        for i in range(k - 1):                                      # pending drafts only
            d_i = rows[i][2] - float(ZL[i][y[L_len + i + 1]])       # -ln p_L(y_S)
            mg["rollback"] = min(mg["rollback"], abs(d_i - alpha_rb))
            rb_here = min(rb_here, abs(d_i - alpha_rb))
            d_max = max(d_max, d_i)
            if d_i > alpha_rb:                                      # Eq. 3, first violation
                m_star, d_star = i, d_i
                break
        if m_star >= 0:                                             # rollback
            j = L_len + m_star + 1
            stats["rollbacks"] += 1
            stats["discarded"] += n - j + 1
            tokL, smg = pick(ZL[m_star], rows[m_star][0], u_large[j] if sampling else 0.0)
            gapL = math.inf if sampling else rows[m_star][3]
            mg["argmax"] = min(mg["argmax"], gapL)
            del y[j:]
            y.append(tokL); n = j
            stL.rewind(j)
            stS.rewind(j)
            L_len = j
            trace.append((KIND_ROLLBACK, j, y[j], k, m_star, d_star))
            tmg.append((gapL, math.inf, rb_here) + ((smg,) if sampling else ()))
        else:
            tokL, smg = pick(ZL[k - 1], rows[k - 1][0], u_large[n + 1] if sampling else 0.0)
            gapL = math.inf if sampling else rows[k - 1][3]
            mg["argmax"] = min(mg["argmax"], gapL)
            y.append(tokL); n += 1
            L_len = n
            trace.append((KIND_VERIFY_OK, n, y[n], k, -1, d_max))
            tmg.append((gapL, math.inf, rb_here) + ((smg,) if sampling else ()))
        drafts = 0
    return dict(tokens=y[1:], trace=trace, stats=stats, margins=mg, logits=logits, trace_margins=tmg)
