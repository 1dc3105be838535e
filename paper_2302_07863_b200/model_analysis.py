"""Analytic FLOPs, memory operations and arithmetic intensity of a stored run, normalised by the
large model alone (the quantities of the paper's "Model Analysis" appendix figure).

    python -m paper_2302_07863_b200.model_analysis --workload t5_sum

No GPU is needed: the counts come from the model shapes and from the event sequence of the
workload's stored oracle run (small steps, large passes and their block sizes).

  FLOPs of a pass over k rows with c cached rows and E encoder positions
      = 2 k (weights of the decoder stack + LM head) + attention 4 I (sum over rows of keys seen)
  memory operations (bytes) of the same pass
      = every weight once + the cached keys / values read + k embedding rows
  (the byte model that bench.py and microbench.py use).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def pass_counts(s, w_bytes, kv_bytes, cache_rows, enc_len, k):
    """(flops, bytes) of one decoder pass of shape `s` over k rows."""
    g = 3 if s.ffn == "gated_gelu" else 2
    I, d, F, V, L = s.inner, s.d_model, s.d_ff, s.vocab, s.n_layers
    params = L * (6 * I * d + g * d * F) + V * d
    self_keys = sum(cache_rows + i + 1 for i in range(k))          # causal inside the block
    flops = 2 * k * params + 4 * I * L * (self_keys + k * enc_len)
    mem = w_bytes * params + kv_bytes * L * (2 * (cache_rows + k) * I + 2 * enc_len * I) + w_bytes * k * d
    return flops, mem


def analyse(workload: str):
    from workloads import MODEL_SHAPES, WORKLOADS
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with open(os.path.join(root, "tests", "golden", workload + ".json")) as f:
        g = json.load(f)
    wl = WORKLOADS[workload]
    sS, sL = MODEL_SHAPES[wl.small], MODEL_SHAPES[wl.large]
    wb = 2 if wl.dtype == "bf16" else 4
    E = wl.enc_len
    n_tok = len(g["bild"]["tokens"])
    # the large model alone: one single-row pass per token
    fl_v = mem_v = 0
    for t in range(len(g["large_only"]["tokens"])):
        f, m = pass_counts(sL, wb, 4, t, E, 1)
        fl_v += f; mem_v += m
    fl_v /= len(g["large_only"]["tokens"]); mem_v /= len(g["large_only"]["tokens"])
    # BiLD: replay the trace (kinds 0..2 are small steps at position pos - 1 ... ; 3 / 4 large passes of k rows)
    fl_b = mem_b = 0
    S_len = L_len = 0
    for kind, pos, tok, k, m, val in g["bild"]["trace"]:
        if kind in (0, 1, 2):
            f, mm = pass_counts(sS, wb, 4, S_len, E, 1)
            S_len += 1
        else:
            f, mm = pass_counts(sL, wb, 4, L_len, E, k)
            if kind == 4:
                S_len = L_len = pos
            else:
                L_len += k
        fl_b += f; mem_b += mm
    fl_b /= n_tok; mem_b /= n_tok
    return {"workload": workload, "tokens": n_tok,
            "large_alone": {"flops_per_token": fl_v, "bytes_per_token": mem_v, "flops_per_byte": fl_v / mem_v},
            "bild": {"flops_per_token": fl_b, "bytes_per_token": mem_b, "flops_per_byte": fl_b / mem_b},
            "normalised": {"flops": fl_b / fl_v, "memory_operations": mem_b / mem_v,
                           "arithmetic_intensity": (fl_b / mem_b) / (fl_v / mem_v)}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="t5_sum")
    a = ap.parse_args()
    print(json.dumps(analyse(a.workload)))


if __name__ == "__main__":
    main()
