"""Synthetic model pairs and encoder inputs with the shapes of the paper's workloads.

The paper evaluates T5-small/large on summarization and mT5-small/large on
translation (Section 4.1; model-size table in the supplementary material).
Neither the checkpoints nor the datasets are available offline, so random
models of the same shapes and random token ids of representative lengths stand
in for them.  Every tensor has its own counter-based stream keyed by
(seed, model name, tensor name), so a tensor's values do not depend on the
order or the subset in which tensors are generated.

This module draws numbers and rounds weights to their storage type once.  It
contains none of the decoder's or the policy's arithmetic.
"""
from __future__ import annotations

import zlib
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    d_kv: int
    d_ff: int
    ffn: str            # "relu" (T5) or "gated_gelu" (mT5)
    vocab: int
    tied_head: bool     # LM head shares the embedding matrix
    rel_buckets: int = 32
    rel_max_dist: int = 128
    eps: float = 1e-6

    @property
    def inner(self) -> int:
        return self.n_heads * self.d_kv


# layers / d_model / heads / d_kv / d_ff follow the supplementary model table
# (24/1024/2816 and 8/512/1024 for mT5; 24/1024/4096 and 6/512/2048 for T5).
MODEL_SHAPES = {
    "tiny_s": ModelShape("tiny_s", 2, 64, 4, 16, 256, "relu", 512, False),
    "tiny_l": ModelShape("tiny_l", 4, 128, 4, 32, 512, "relu", 512, False),
    # odd sizes on purpose: inner != d_model, vocab not a multiple of any tile,
    # d_ff not a power of two, gated FFN.
    "odd_s": ModelShape("odd_s", 2, 64, 3, 16, 136, "gated_gelu", 773, False),
    "odd_l": ModelShape("odd_l", 3, 128, 6, 16, 328, "gated_gelu", 773, False),
    # small pair with the 64-channel heads of the T5 / mT5 shapes (no stored run: live parity tests only)
    "wide_s": ModelShape("wide_s", 2, 128, 2, 64, 264, "relu", 520, False),
    "wide_l": ModelShape("wide_l", 3, 256, 4, 64, 520, "gated_gelu", 520, False),
    "t5_s": ModelShape("t5_s", 6, 512, 8, 64, 2048, "relu", 32128, False),
    "t5_l": ModelShape("t5_l", 24, 1024, 16, 64, 4096, "relu", 32128, False),
    "mt5_s": ModelShape("mt5_s", 8, 512, 6, 64, 1024, "gated_gelu", 250112, False),
    "mt5_l": ModelShape("mt5_l", 24, 1024, 16, 64, 2816, "gated_gelu", 250112, False),
}


@dataclass(frozen=True)
class Workload:
    name: str
    small: str
    large: str
    dtype: str          # "fp32" or "bf16" (storage type of weight matrices)
    enc_len: int
    gen_len: int
    seed: int = 0
    max_draft: int = 10


WORKLOADS = {
    "tiny": Workload("tiny", "tiny_s", "tiny_l", "fp32", 32, 32),
    "odd": Workload("odd", "odd_s", "odd_l", "fp32", 19, 40),
    "odd_bf16": Workload("odd_bf16", "odd_s", "odd_l", "bf16", 19, 40),
    "tiny_bf16": Workload("tiny_bf16", "tiny_s", "tiny_l", "bf16", 32, 32),
    "wide_bf16": Workload("wide_bf16", "wide_s", "wide_l", "bf16", 80, 100, max_draft=15),
    "t5_sum": Workload("t5_sum", "t5_s", "t5_l", "bf16", 512, 64),
    "mt5_mt": Workload("mt5_mt", "mt5_s", "mt5_l", "bf16", 64, 64),
    "t5_long": Workload("t5_long", "t5_s", "t5_l", "bf16", 1024, 256),
}


def bf16_round_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> the fp32 values they denote (exact)."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def tensor_names(s: ModelShape) -> dict:
    """name -> (shape, kind); kind in {"embedding", "matrix", "gain", "bias"}."""
    d, inner, f, v = s.d_model, s.inner, s.d_ff, s.vocab
    t = {"emb": ((v, d), "embedding")}
    if not s.tied_head:
        t["lm_head"] = ((v, d), "matrix")
    for stack in ("enc", "dec"):
        t[f"{stack}.rel_bias"] = ((s.rel_buckets, s.n_heads), "bias")
        t[f"{stack}.final_ln"] = ((d,), "gain")
        for l in range(s.n_layers):
            p = f"{stack}.{l}."
            t[p + "ln1"] = ((d,), "gain")
            t[p + "wqkv"] = ((3 * inner, d), "matrix")      # rows: q, then k, then v
            t[p + "wo"] = ((d, inner), "matrix")
            t[p + "ln2"] = ((d,), "gain")
            if stack == "dec":
                t[p + "wcq"] = ((inner, d), "matrix")
                t[p + "wckv"] = ((2 * inner, d), "matrix")  # rows: k, then v
                t[p + "wco"] = ((d, inner), "matrix")
                t[p + "ln3"] = ((d,), "gain")
            t[p + "wi0"] = ((f, d), "matrix")
            if s.ffn == "gated_gelu":
                t[p + "wi1"] = ((f, d), "matrix")
            t[p + "wfo"] = ((d, f), "matrix")
    return t


def _stream(seed: int, model: str, tensor: str) -> np.random.Generator:
    key = zlib.crc32(f"{model}/{tensor}".encode())
    return np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64(key)]))


def _gen_one(s: ModelShape, seed: int, dtype: str, name: str, shape, kind):
    g = _stream(seed, s.name, name)
    n = int(np.prod(shape))
    x = g.standard_normal(n, dtype=np.float32)
    if kind in ("matrix", "embedding"):
        # Matrices are N(0, 0.02).  The embedding table is N(0, 1), T5's own
        # initialisation: with a 0.02 table the token identity drowns in the
        # sub-layer outputs and greedy decoding of a random model collapses onto
        # a fixed point within a few tokens, so the confidence never varies.
        if kind == "matrix":
            x *= np.float32(0.02)
        x = x.reshape(shape)
        return bf16_round_bits(x).reshape(shape) if dtype == "bf16" else x
    if kind == "gain":          # 1 + N(0, 0.02): a dropped gain multiply is visible
        return (np.float32(1.0) + np.float32(0.02) * x).reshape(shape)
    return x.reshape(shape)     # bias table, N(0, 1): a wrong bucket is visible


def gen_model(s: ModelShape, seed: int, dtype: str, only=None, threads: int = 8) -> dict:
    """All tensors of one encoder-decoder model.

    Matrices and the embedding table are fp32 arrays (dtype "fp32") or uint16
    bf16 bit patterns (dtype "bf16"); gains and relative-position bias tables
    are always fp32.  `only` restricts generation to names with one of the
    given prefixes.
    """
    assert dtype in ("fp32", "bf16")
    todo = [(n, sh, k) for n, (sh, k) in tensor_names(s).items()
            if only is None or any(n.startswith(p) for p in only)]
    with ThreadPoolExecutor(max_workers=threads) as ex:
        vals = list(ex.map(lambda a: _gen_one(s, seed, dtype, *a), todo))
    return {n: v for (n, _, _), v in zip(todo, vals)}


def gen_ids(vocab: int, n: int, seed: int) -> np.ndarray:
    """Encoder input: n token ids uniform on [2, vocab) (0 = start/pad, 1 = EOS)."""
    g = _stream(seed, "input", f"ids{n}")
    return g.integers(2, vocab, size=n, dtype=np.int64).astype(np.int32)


def gen_uniforms(n: int, seed: int, tag: str) -> np.ndarray:
    """n uniform numbers in [0, 1) as fp32 (multiples of 2^-24, so exact in either precision): the random
    input of the sampling variant, one per output position; `tag` names the stream ("small" / "large")."""
    g = _stream(seed, "uniform", tag)
    return (g.integers(0, 1 << 24, size=n, dtype=np.int64).astype(np.float64) / float(1 << 24)).astype(np.float32)
