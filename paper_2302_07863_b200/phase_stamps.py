"""Cycle stamps of the fused sub-layer kernels, phase by phase (per launch: block 0 / mean of all blocks / the longest
any block took in any launch):

    python -m paper_2302_07863_b200.phase_stamps [workload] [k,...]

Builds a second copy of the library with -DBILD_STAMPS (libbild_stamps.so beside libbild.so: the same kernels plus
clock64() reads at the phase boundaries and a debug entry point that returns the sums) and replays the small step
and the large pass for the given row counts, then the set-up step (phases of the encoder GEMM's blocks, T5-large shapes
at 512 tokens).  The stamped build is a few percent slower than the product build."""
import ctypes as C, json, os, sys
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import paper_2302_07863_b200.binding as B
import subprocess
HERE = os.path.dirname(os.path.abspath(__file__))
B.LIB_PATH = os.path.join(HERE, "libbild_stamps.so")
subprocess.run([os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc"), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3",
                "-std=c++17", "-shared", "-Xcompiler", "-fPIC", "-DBILD_STAMPS", "-I", os.path.join(ROOT, "include"), "-I",
                os.path.join(HERE, "csrc"), "-o", B.LIB_PATH, os.path.join(HERE, "csrc", "bild.cu"),
                os.path.join(HERE, "csrc", "no_alloc.cu"), "-lcuda"], check=True)
from paper_2302_07863_b200.synthetic import make_context
wlname = sys.argv[1] if len(sys.argv) > 1 else "t5_sum"
ks = [int(x) for x in (sys.argv[2] if len(sys.argv) > 2 else "1,5").split(",")]
g = json.load(open(os.path.join(ROOT, "tests", "golden", wlname + ".json")))
ctx, ids, wl = make_context(wlname, g["scale_small"]["scale"], g["scale_large"]["scale"], max_dec_len=64 + 17)
ctx.encode(ids)
L = B.lib()
L.bild_debug_stamps.argtypes = [C.POINTER(C.c_ulonglong), C.c_int]
names = {0: ["P0 init", "P1 copies", "P2 loads", "arrive", "dep wait", "rows+norm", "weights wait", "qkv products", "exch stores", "cluster bar 1", "B1 staged", "B2 scores", "B3 softmax", "attention(pv)", "rec stores", "cluster bar 2", "merge", "oproj+red"],
         1: None, 2: ["prologue", "dep wait", "rows+norm", "weights wait", "hidden", "out+red"]}
names[1] = names[0]
def run(which, k):
    buf = (C.c_ulonglong * 288)()
    L.bild_debug_stamps(buf, 1)
    us = ctx.time_pass(which, k, 64, 10) * 1000
    L.bild_debug_stamps(buf, 0)
    print(f"== model {which} k={k}: {us:.1f} us per pass")
    for kind, nm in (("self", 0), ("cross", 1), ("ffn", 2)):
        n0, na = buf[nm * 24 + 23], buf[96 + nm * 24 + 23]
        if not n0: continue
        # single-row kernels have no separate soft-max phase (it is part of the value phase)
        nms = [x for x in names[nm] if not (k == 1 and x == "B3 softmax")]
        ph0 = [buf[nm * 24 + i] / n0 / 1965.0 for i in range(len(nms))]
        pha = [buf[96 + nm * 24 + i] / na / 1965.0 for i in range(len(nms))]
        phm = [buf[192 + nm * 24 + i] / 1965.0 for i in range(len(nms))]
        off = 5 if nm < 2 else 2
        print(f"  {kind:5s} after wait: block 0 {sum(ph0[off:]):.2f} us, mean of blocks {sum(pha[off:]):.2f} us | " +
              " ".join(f"{a}={b:.2f}/{c:.2f}/{e:.2f}" for a, b, c, e in zip(nms, ph0, pha, phm)))
run(0, 1)
for k in ks: run(1, k)

# ---- encoder GEMM: phases of a block (sources of 512 ids) ----
import torch
L.bild_debug_gemm_stamps.argtypes = [C.POINTER(C.c_ulonglong), C.c_int]
gb = (C.c_ulonglong * 48)()
for _ in range(3): ctx.encode(ids)
torch.cuda.synchronize()
L.bild_debug_gemm_stamps(gb, 1)
for _ in range(5): ctx.encode(ids)
torch.cuda.synchronize()
L.bild_debug_gemm_stamps(gb, 0)
for cls, nm in enumerate(["QKV (24 x 4 tiles)", "FFN-up (32 x 4)", "residual (8 x 4, K split)"]):
    n = gb[cls * 16 + 15]
    if not n: continue
    f = lambda i: gb[cls * 16 + i] / n / 1965.0
    print(f"== encoder GEMM {nm}: {n} blocks | start -> tensor memory allocated {f(0):.2f} us | -> dependency wait returned {f(1):.2f} | "
          f"-> all MMAs done {f(2):.2f} (MMA thread: wait -> first stage full {f(8):.2f}, first -> last MMA issued {f(9):.2f}; "
          f"producer: wait -> last copy issued {f(12):.2f}) | epilogue {f(3):.2f} (loads from tensor memory {f(4):.2f})")
