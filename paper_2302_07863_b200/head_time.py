"""Times the LM-head kernels alone through the single-operation entry points (CUDA events, L2 flushed before each call):

    python -m paper_2302_07863_b200.head_time

ncu does not profile graph nodes that can set conditional handles, which the head kernels do, so the launch lists
under profiles/ do not contain them."""
import os, sys
sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from paper_2302_07863_b200 import build
build.build()
import numpy as np, torch
from paper_2302_07863_b200.binding import op_lm_head, op_lm_head_sliced, op_lm_head_stream
def bench(fn, n=30):
    flush = torch.empty(160 << 20, dtype=torch.uint8, device="cuda")
    ts = []
    for i in range(n):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); fn(); e1.record(); torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1) * 1e3)
    ts.sort(); return ts[len(ts) // 2]
# "stream": bild_op_lm_head_stream (single rows: two blocks per SM walk the vocabulary); "rows": bild_op_lm_head (single rows: weights of a warp's vocabulary rows in registers); "sliced": the streaming tensor-core head
for V, K, M, which in [(32128, 512, 1, "stream"), (32128, 1024, 1, "stream"), (250112, 512, 1, "stream"), (250112, 1024, 1, "stream"),
                       (32128, 512, 1, "rows"), (32128, 512, 1, "sliced"), (32128, 1024, 1, "rows"), (32128, 1024, 1, "sliced"), (32128, 1024, 5, "sliced"),
                       (250112, 512, 1, "rows"), (250112, 512, 1, "sliced"), (250112, 1024, 1, "rows"), (250112, 1024, 1, "sliced"),
                       (250112, 1024, 5, "sliced")]:
    W = (torch.randn(V, K, device="cuda") * 0.05).to(torch.bfloat16)
    X = torch.randn(M, K, device="cuda"); g = torch.ones(K, device="cuda"); t = torch.zeros(M, dtype=torch.int32, device="cuda")
    f = ((lambda: op_lm_head(W, X, g, 1e-6, 5.0, t, M, V, K)) if which == "rows" else
         (lambda: op_lm_head_stream(W, X, g, 1e-6, 5.0, t, V, K)) if which == "stream" else
         (lambda: op_lm_head_sliced(W, X, g, 1e-6, 5.0, t, M, V, K)))
    us = bench(f)
    print(f"V={V} K={K} M={M} {which}: {us:.1f} us (L2 flushed; includes the entry point's small copies) -> {V*K*2/us/1e3:.0f} GB/s")
