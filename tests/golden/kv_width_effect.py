"""How far the ORACLE's logits move when the self- and cross-attention K/V caches are rounded to bf16 on write
(everything else unchanged): the measurement behind keeping the caches in fp32 on the GPU.  Calls only oracle/ and
workloads/; teacher-forced over the first positions of the stored run.

    python tests/golden/kv_width_effect.py [workload] [positions] [large|small]

t5_sum, 10 positions, large model (about two minutes on 8 cores): max |dz| 2.3e-2 at the first position, 4.6e-2 to
5.7e-2 from the second on, for logits of magnitude 30 -- above the 2e-2 the logits are allowed to differ by."""
import json, sys, os, time
import numpy as np
sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
from oracle.t5 import Model, DecState
from workloads import MODEL_SHAPES, WORKLOADS, gen_ids, gen_model
from workloads.gen import bf16_round_bits, bf16_bits_to_f32
def rb(a):
    return bf16_bits_to_f32(bf16_round_bits(a.astype(np.float32))).astype(np.float64)
wlname = sys.argv[1] if len(sys.argv) > 1 else "t5_sum"
npos = int(sys.argv[2]) if len(sys.argv) > 2 else 12
which = sys.argv[3] if len(sys.argv) > 3 else "large"
wl = WORKLOADS[wlname]; g = json.load(open(os.path.join(os.path.dirname(os.path.abspath(__file__)), wlname + ".json")))
shape = MODEL_SHAPES[wl.large if which == "large" else wl.small]
t0 = time.time()
m = Model(shape, gen_model(shape, wl.seed, wl.dtype), g["scale_large" if which == "large" else "scale_small"]["scale"])
ids = gen_ids(shape.vocab, wl.enc_len, wl.seed)
print("model built", round(time.time() - t0, 1), "s")
toks = [0] + g["bild"]["tokens"][:npos]
stA = m.start(ids, npos + 2); stB = m.start(ids, npos + 2)
stB.ck = [rb(x) for x in stB.ck]; stB.cv = [rb(x) for x in stB.cv]
worst = 0.0
for i in range(npos):
    zA = m.forward_block(stA, [toks[i]])[0]
    zB = m.forward_block(stB, [toks[i]])[0]
    for l in range(len(stB.k)):
        stB.k[l][stB.len - 1] = rb(stB.k[l][stB.len - 1]); stB.v[l][stB.len - 1] = rb(stB.v[l][stB.len - 1])
    d = float(np.max(np.abs(zA - zB))); worst = max(worst, d)
    srt = np.sort(zA)
    print(i, "max |dz| =", f"{d:.3e}", "max |z| =", f"{np.max(np.abs(zA)):.2f}", "top-2 gap", f"{srt[-1]-srt[-2]:.3f}", "argmax same", int(np.argmax(zA)) == int(np.argmax(zB)), flush=True)
print("worst", worst)
