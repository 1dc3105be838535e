"""Benchmark of the BiLD decode loop (libbild) on synthetic T5-shaped workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload t5_sum] [--impl ours|reference]

One step = one pass of the whole hot path over one input: Algorithm 1 from the start
symbol to gen_len tokens (small-model steps with the fused fallback test, large-model
block passes with the fused rollback test, cache rewinds), with the encoder results
already resident (`value`), or including the host->device copy of the ids, both encoders
and the device->host copy of tokens and trace (`e2e`).  Prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC, UNIT = "BiLD tokens/s at batch 1", "tokens/s"


def load_golden(name):
    with open(os.path.join(ROOT, "tests", "golden", name + ".json")) as f:
        return json.load(f)


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def measured_traffic(workload, kernel):
    """DRAM bytes of one launch sequence of `kernel` from the committed ncu summary (profiles/dram_traffic.json:
    dram__bytes_read.sum + dram__bytes_write.sum), or None where it was not measured for this workload and kernel."""
    p = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(p):
        return None
    with open(p) as f:
        t = json.load(f)
    e = t.get(workload, {}).get(kernel)
    return float(e["bytes"]) if e else None


def pass_bytes(s, w_bytes, kv_bytes, cache_rows, enc_len, k):
    """Algorithmic bytes one decoder pass must read: every weight matrix once, the LM head,
    the self cache rows it attends to and the cross K/V (per layer), the k embedding rows."""
    g = 3 if s.ffn == "gated_gelu" else 2
    I, d, F, V, L = s.inner, s.d_model, s.d_ff, s.vocab, s.n_layers
    weights = w_bytes * (L * (6 * I * d + g * d * F) + V * d)
    kv = kv_bytes * L * (2 * (cache_rows + k) * I + 2 * enc_len * I)
    return weights + kv + w_bytes * k * d


class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "200"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 8:
                continue
            try:
                sm.append(float(c[0])); mx.append(float(c[1]))
            except ValueError:
                continue
            for n, v in zip(names, c[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        os.unlink(self.f.name)
        if sm:
            sm.sort()
            out = {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}
        return out


def oracle_models(wl, g):
    from oracle.t5 import Model
    from workloads import MODEL_SHAPES, gen_ids, gen_model
    S = Model(MODEL_SHAPES[wl.small], gen_model(MODEL_SHAPES[wl.small], wl.seed, wl.dtype), g["scale_small"]["scale"])
    L = Model(MODEL_SHAPES[wl.large], gen_model(MODEL_SHAPES[wl.large], wl.seed, wl.dtype), g["scale_large"]["scale"])
    return S, L, gen_ids(S.s.vocab, wl.enc_len, wl.seed)


def time_oracle(wl, g, n_tokens, steps, warmup):
    """The CPU oracle as it stands, timed on the host cores: BiLD generation of n_tokens
    tokens per step (encoder results reused, as in the GPU arm's `value`)."""
    from oracle import bild as obild
    S, L, ids = oracle_models(wl, g)
    th = g["thresholds"]
    # encoders once, outside the timed region (the GPU arm's `value` also excludes them)
    orig_start = (S.start, L.start)
    stS, stL = S.start(ids, wl.gen_len + 1), L.start(ids, wl.gen_len + 1)

    def restart(model, st):
        def f(enc_ids, cap):
            st.len = 0
            return st
        return f
    S.start, L.start = restart(S, stS), restart(L, stL)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        r = obild.generate(S, L, ids, th["alpha_fb"], th["alpha_rb"], n_tokens, max_draft=wl.max_draft)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    S.start, L.start = orig_start
    total = sum(times)
    return len(r["tokens"]) * len(times) / total, total / len(times) * 1e3


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="t5_sum")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--oracle-tokens", type=int, default=16)
    a = ap.parse_args()
    a.warmup = max(a.warmup, 3) if a.impl == "ours" else a.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    from workloads import MODEL_SHAPES, WORKLOADS
    wl = WORKLOADS[a.workload]
    g = load_golden(a.workload)
    th = g["thresholds"]
    cores = len(os.sched_getaffinity(0))
    cfg_common = {"workload": f"{a.workload}: {wl.small}/{wl.large} pair, {wl.dtype}, batch 1, enc {wl.enc_len} ids, "
                              f"{wl.gen_len} generated tokens, alpha_fb={th['alpha_fb']:.4f} alpha_rb={th['alpha_rb']:.3f}",
                  "fallback_rate": th["fallback_rate"], "rollback_rate": th["rollback_rate"]}

    if a.impl == "reference":
        if rank != 0:
            return
        ntok = min(a.oracle_tokens, wl.gen_len)
        tps, ms = time_oracle(wl, g, ntok, a.steps, a.warmup)
        sample = f"oracle BiLD loop, first {ntok} tokens of the workload per step, encoders outside the timed region"
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": a.gpus, "steps": a.steps,
            "warmup": a.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": cfg_common,
            "cpu_baseline": {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    import numpy as np
    import torch
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    from paper_2302_07863_b200 import MODE_BILD, MODE_LARGE_ONLY, build
    from paper_2302_07863_b200.synthetic import make_context
    build.build()
    ctx, ids, _ = make_context(a.workload, g["scale_small"]["scale"], g["scale_large"]["scale"], device=f"cuda:{local}")
    ids_pinned = torch.from_numpy(np.ascontiguousarray(ids)).pin_memory()
    ctx.encode(ids_pinned.numpy())
    torch.cuda.synchronize()

    from paper_2302_07863_b200 import replicas

    def barrier():
        replicas.barrier(dist if world > 1 else None, world)
        torch.cuda.synchronize()

    def run(fn, steps, warmup):
        for _ in range(warmup):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        return replicas.max_over_ranks(dist if world > 1 else None, world, e0.elapsed_time(e1), device="cuda")

    def step_resident():
        ctx.generate_async(MODE_BILD, th["alpha_fb"], th["alpha_rb"], wl.gen_len)

    res = {}

    def step_e2e():
        ctx.encode(ids_pinned.numpy())
        res["r"] = ctx.generate(MODE_BILD, th["alpha_fb"], th["alpha_rb"], wl.gen_len)

    sampler = ClockSampler(local) if rank == 0 else None
    ctx.generate(MODE_BILD, th["alpha_fb"], th["alpha_rb"], wl.gen_len)
    l0 = ctx.launch_count()
    ms = run(step_resident, a.steps, a.warmup)
    r = ctx.fetch_result(wl.gen_len)
    launches = (ctx.launch_count() - l0) * a.steps // (a.steps + a.warmup)
    ntok = len(r["tokens"])
    ms_e2e = run(step_e2e, max(2, a.steps // 4), 1)
    e2e_steps = max(2, a.steps // 4)
    clocks = sampler.stop() if sampler else None
    ms_large_only = run(lambda: ctx.generate_async(MODE_LARGE_ONLY, 0.0, math.inf, wl.gen_len), max(2, a.steps // 4), 1)
    large_steps = max(2, a.steps // 4)

    # per-pass latencies and the roofline of the dominant pass (the large-model block pass)
    st = r["stats"]
    k_mean = max(1, round(st["sum_k"] / max(1, st["large_calls"])))
    cache_mid = wl.gen_len // 2
    sS, sL = MODEL_SHAPES[wl.small], MODEL_SHAPES[wl.large]
    wb = 2 if wl.dtype == "bf16" else 4
    t_small = ctx.time_pass(0, 1, cache_mid, 50)
    t_large = ctx.time_pass(1, k_mean, cache_mid, 20)
    t_large1 = ctx.time_pass(1, 1, cache_mid, 20)
    # algorithmic bytes: keys / values at the weights' width (what the method has to move); the caches are kept in
    # fp32 here, so the passes read somewhat more than that ("stored" figures below)
    b_small = pass_bytes(sS, wb, wb, cache_mid, wl.enc_len, 1)
    b_large = pass_bytes(sL, wb, wb, cache_mid, wl.enc_len, k_mean)
    b_small_st = pass_bytes(sS, wb, 4, cache_mid, wl.enc_len, 1)
    b_large_st = pass_bytes(sL, wb, 4, cache_mid, wl.enc_len, k_mean)
    peak, peak_kind = peaks()
    time_small_total = st["small_steps"] * t_small
    time_large_total = st["large_calls"] * t_large
    dom_large = time_large_total >= time_small_total
    ach = (b_large / (t_large * 1e-3) if dom_large else b_small / (t_small * 1e-3)) / 1e9

    if rank != 0:
        return
    out = {
        "metric": METRIC, "value": replicas.whole_job_rate(ntok * a.steps, world, ms), "unit": UNIT, "n_gpus": world,
        "steps": a.steps, "warmup": a.warmup, "ms_per_step": ms / a.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 weights, f32 activations and KV cache" if wb == 2 else "f32",
        "data": "synthetic", "gpu_launches": int(launches),
        "config": dict(cfg_common, l2="inputs larger than L2: every step re-reads "
                       f"{(b_large_st + b_small_st) / 1e6:.0f} MB of weights and K/V", parallelism="replicas only"),
        "e2e": {"value": replicas.whole_job_rate(ntok * e2e_steps, world, ms_e2e), "unit": UNIT,
                "h2d_bytes_per_step": int(ids_pinned.numel() * 4),
                "d2h_bytes_per_step": int(4 * ntok + 24 * r["n_trace"] + 2 * 96)},
        "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": ("large-model block pass, k=%d" % k_mean) if dom_large else "small-model step",
                     "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak, "peak_kind": peak_kind,
                     "frac_with_fp32_kv_bytes": (b_large_st / t_large if dom_large else b_small_st / t_small) / 1e6 / peak,
                     "traffic": measured_traffic(a.workload, ("large_block_pass_k%d" % k_mean) if dom_large else "small_step"),
                     "note": "a pass is a chain of dependent kernels replayed as one CUDA graph; its duration is "
                             "measured with CUDA events over back-to-back replays"},
        "passes": {"small_step_us": t_small * 1e3, "small_step_GBs": b_small / t_small / 1e6,
                   "small_step_frac": b_small / t_small / 1e6 / peak,
                   "verify_us": t_large * 1e3, "verify_k": k_mean, "verify_GBs": b_large / t_large / 1e6,
                   "verify_frac": b_large / t_large / 1e6 / peak, "verify_k1_us": t_large1 * 1e3,
                   "large_only_tokens_per_s": ntok * large_steps / (ms_large_only * 1e-3),
                   "speedup_vs_large_only": (ntok * a.steps / ms) / (ntok * large_steps / ms_large_only),
                   "stats": st},
    }
    if world == 1 and not a.no_cpu_baseline:
        nt = min(a.oracle_tokens, wl.gen_len)
        tps, _ = time_oracle(wl, g, nt, 1, 0)
        out["cpu_baseline"] = {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle",
                               "sample": f"oracle BiLD loop over the first {nt} tokens of the same workload, one run, "
                                         "encoders outside the timed region"}
    print(json.dumps(out))


if __name__ == "__main__":
    main()
