"""Times the set-up step (both encoders and the cross-attention K/V of every decoder layer).

    python -m paper_2302_07863_b200.encode_time --workload t5_sum

Three untimed calls of Context.encode, then the mean of `--reps` calls (CUDA events)."""
from __future__ import annotations

import argparse
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="t5_sum")
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--tuning", default="", help="bild_tuning fields, e.g. enc_split_k=0,enc_parallel=0")
    a = ap.parse_args()
    import torch
    assert torch.cuda.is_available(), "needs a CUDA device"
    from paper_2302_07863_b200 import build
    from paper_2302_07863_b200.synthetic import make_context
    build.build()
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with open(os.path.join(root, "tests", "golden", a.workload + ".json")) as f:
        g = json.load(f)
    tuning = {k: int(v) for k, v in (kv.split("=") for kv in a.tuning.split(",") if kv)} or None
    ctx, ids, wl = make_context(a.workload, g["scale_small"]["scale"], g["scale_large"]["scale"], tuning=tuning)
    for _ in range(3):
        ctx.encode(ids)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.reps):
        ctx.encode(ids)
    e1.record()
    e1.synchronize()
    print(json.dumps({"workload": a.workload, "enc_len": wl.enc_len, "encode_ms": e0.elapsed_time(e1) / a.reps}))


if __name__ == "__main__":
    main()
