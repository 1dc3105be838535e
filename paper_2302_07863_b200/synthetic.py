"""Contexts for the named synthetic workloads (random T5 / mT5-shaped pairs)."""
from __future__ import annotations

from workloads import MODEL_SHAPES, WORKLOADS, gen_ids, gen_model

from .binding import BF16, FP32, Config, Context, model_cfg, upload_model


def make_context(workload: str, scale_small: float, scale_large: float, device="cuda:0", max_enc_len=None,
                 max_dec_len=None, eos_id=-1, max_draft=None, tuning=None, early_exit_layers=0):
    """Generate the workload's two models on the host, upload them, create a Context.
    Returns (context, encoder ids, workload).  early_exit_layers > 0: the early-exit configuration of Section 4.4,
    the small model being the first layers of the workload's LARGE model (its own small model is not used)."""
    import dataclasses
    wl = WORKLOADS[workload]
    sS, sL = MODEL_SHAPES[wl.small], MODEL_SHAPES[wl.large]
    devL = upload_model(gen_model(sL, wl.seed, wl.dtype), device)
    if early_exit_layers > 0:
        sS, devS = dataclasses.replace(sL, n_layers=early_exit_layers), devL
    else:
        devS = upload_model(gen_model(sS, wl.seed, wl.dtype), device)
    cfg = Config(model_cfg(sS, scale_small), model_cfg(sL, scale_large), BF16 if wl.dtype == "bf16" else FP32,
                 max_enc_len or wl.enc_len, max_dec_len or wl.gen_len + 1, max_draft or wl.max_draft, 0, eos_id,
                 early_exit_layers)
    ctx = Context(cfg, sS, devS, sL, devL, device, tuning=tuning)
    return ctx, gen_ids(sS.vocab, wl.enc_len, wl.seed), wl
