"""CPU oracle, part 1: a T5-shaped encoder-decoder forward pass in fp64.

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain reference that the
CUDA library is checked against; nothing in the product path may import it.
It shares no code with the CUDA path.

The paper treats its two models as black boxes and only names them (T5 and
mT5, small and large; Section 4.1 and the model-size table of the
supplementary material).  The forward pass below is therefore the published
T5 / mT5 architecture written out as plain mathematics:

* pre-norm residual blocks; RMS norm  y = x * g / sqrt(mean(x^2) + eps),
  no mean subtraction, no bias anywhere;
* attention scores are NOT divided by sqrt(d_kv);
* an additive relative-position bias on self-attention only, one table
  [buckets][heads] per stack, shared by all layers of that stack;
* cross-attention has neither bias nor mask (batch 1, no padding);
* feed-forward: ReLU (T5) or tanh-approximated GELU gate (mT5);
* final RMS norm, then logits = logit_scale * W_lm h.

Weights arrive as fp32 arrays or as bf16 bit patterns (uint16); both are
upcast exactly to fp64 and every operation runs in fp64.
"""
from __future__ import annotations

import functools
import math

import numpy as np


def to_f64(a: np.ndarray) -> np.ndarray:
    """fp32 array, or uint16 bf16 bit patterns, to fp64 (exact)."""
    if a.dtype == np.uint16:
        a = (a.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return a.astype(np.float64)


# --------------------------------------------------------------------------
# relative-position buckets (integer arithmetic only, so no log rounding)
# --------------------------------------------------------------------------
def _log_bucket(dist: int, max_exact: int, n_log: int, max_dist: int) -> int:
    """For dist >= max_exact: max_exact + floor(n_log * ln(dist/max_exact) /
    ln(max_dist/max_exact)), capped at max_exact + n_log - 1.  Evaluated as the
    largest j with (dist/max_exact)^n_log >= (max_dist/max_exact)^j, in exact
    integers."""
    j = 0
    while (j + 1 <= n_log - 1 and
           dist ** n_log * max_exact ** (j + 1) >= max_dist ** (j + 1) * max_exact ** n_log):
        j += 1
    return max_exact + j


@functools.lru_cache(maxsize=None)
def decoder_bucket(delta: int, n_buckets: int = 32, max_dist: int = 128) -> int:
    """Unidirectional bucket of delta = query_pos - key_pos >= 0."""
    assert delta >= 0
    max_exact = n_buckets // 2
    if delta < max_exact:
        return delta
    return _log_bucket(delta, max_exact, n_buckets - max_exact, max_dist)


@functools.lru_cache(maxsize=None)
def encoder_bucket(rel: int, n_buckets: int = 32, max_dist: int = 128) -> int:
    """Bidirectional bucket of rel = key_pos - query_pos (any sign)."""
    half = n_buckets // 2
    off = half if rel > 0 else 0
    dist = abs(rel)
    max_exact = half // 2
    if dist < max_exact:
        return off + dist
    return off + _log_bucket(dist, max_exact, half - max_exact, max_dist)


# --------------------------------------------------------------------------
# building blocks
# --------------------------------------------------------------------------
def rms_norm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x * g / np.sqrt(ms + eps)


def softmax(s: np.ndarray) -> np.ndarray:
    e = np.exp(s - np.max(s, axis=-1, keepdims=True))
    return e / np.sum(e, axis=-1, keepdims=True)


def gelu_tanh(u: np.ndarray) -> np.ndarray:
    return 0.5 * u * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (u + 0.044715 * u ** 3)))


def attend(q: np.ndarray, K: np.ndarray, V: np.ndarray, bias=None) -> np.ndarray:
    """One head, one query: softmax(q.K^T + bias) V.  K, V: [n][d_kv]."""
    s = K @ q
    if bias is not None:
        s = s + bias
    return softmax(s) @ V


class Model:
    """One encoder-decoder model with fp64 weights."""

    def __init__(self, shape, tensors: dict, logit_scale: float = 1.0, exit_layers: int = 0):
        """exit_layers > 0: the early-exit "small model" of Section 4.4: the same encoder, embedding, final norm and
        prediction head, but only the first `exit_layers` decoder layers."""
        self.s = shape
        self.w = {k: to_f64(v) for k, v in tensors.items()}
        self.logit_scale = float(logit_scale)
        self.lm = self.w["emb"] if shape.tied_head else self.w["lm_head"]
        self.dec_layers = exit_layers if exit_layers > 0 else shape.n_layers
        assert 1 <= self.dec_layers <= shape.n_layers

    def early_exit(self, exit_layers: int, logit_scale: float = None) -> "Model":
        """The model that shares every tensor with this one and stops after `exit_layers` decoder layers."""
        m = Model.__new__(Model)
        m.s, m.w, m.lm = self.s, self.w, self.lm
        m.logit_scale = self.logit_scale if logit_scale is None else float(logit_scale)
        m.dec_layers = exit_layers
        assert 1 <= exit_layers <= self.s.n_layers
        return m

    # ---- feed-forward -----------------------------------------------------
    def _ffn(self, p: str, h: np.ndarray) -> np.ndarray:
        w = self.w
        if self.s.ffn == "relu":
            u = np.maximum(h @ w[p + "wi0"].T, 0.0)
        else:
            u = gelu_tanh(h @ w[p + "wi0"].T) * (h @ w[p + "wi1"].T)
        return u @ w[p + "wfo"].T

    # ---- encoder ----------------------------------------------------------
    def encode(self, ids) -> np.ndarray:
        """Encoder memory [E][d] for the input ids (bidirectional attention)."""
        s, w = self.s, self.w
        E, H, dk = len(ids), s.n_heads, s.d_kv
        I = H * dk
        x = w["emb"][np.asarray(ids)]
        rb = w["enc.rel_bias"]
        # bias[h][i][j] = table[bucket(j - i)][h]
        tab = np.array([encoder_bucket(r, s.rel_buckets, s.rel_max_dist) for r in range(-(E - 1), E)])
        rel = np.arange(E)[None, :] - np.arange(E)[:, None]
        bias = rb[tab[rel + (E - 1)]].transpose(2, 0, 1)
        for l in range(s.n_layers):
            p = f"enc.{l}."
            h = rms_norm(x, w[p + "ln1"], s.eps)
            qkv = h @ w[p + "wqkv"].T
            q, k, v = qkv[:, :I], qkv[:, I:2 * I], qkv[:, 2 * I:]
            a = np.empty((E, I))
            for hd in range(H):
                sl = slice(hd * dk, (hd + 1) * dk)
                a[:, sl] = softmax(q[:, sl] @ k[:, sl].T + bias[hd]) @ v[:, sl]
            x = x + a @ w[p + "wo"].T
            x = x + self._ffn(p, rms_norm(x, w[p + "ln2"], s.eps))
        return rms_norm(x, w["enc.final_ln"], s.eps)

    # ---- decoder with caches ----------------------------------------------
    def start(self, enc_ids, cap: int) -> "DecState":
        """Run the encoder and project the per-layer cross-attention K/V."""
        s, w = self.s, self.w
        mem = self.encode(enc_ids)
        st = DecState(s, cap)
        st.mem = mem
        for l in range(self.dec_layers):
            kv = mem @ w[f"dec.{l}.wckv"].T
            st.ck.append(kv[:, :s.inner].copy())
            st.cv.append(kv[:, s.inner:].copy())
        return st

    def forward_block(self, st: "DecState", tokens) -> np.ndarray:
        """Feed k tokens at positions st.len .. st.len+k-1 in one pass.

        Row i of the result holds the logits of the distribution over the token
        that follows tokens[i], given everything up to and including tokens[i].
        Appends k rows to the self-attention cache."""
        s, w = self.s, self.w
        k, c, H, dk, I = len(tokens), st.len, s.n_heads, s.d_kv, s.inner
        assert c + k <= st.cap
        x = w["emb"][np.asarray(tokens)]
        rb = w["dec.rel_bias"]
        for l in range(self.dec_layers):
            p = f"dec.{l}."
            qkv = rms_norm(x, w[p + "ln1"], s.eps) @ w[p + "wqkv"].T
            q = qkv[:, :I]
            st.k[l][c:c + k] = qkv[:, I:2 * I]
            st.v[l][c:c + k] = qkv[:, 2 * I:]
            a = np.empty((k, I))
            for i in range(k):
                n_keys = c + i + 1          # causal: keys 0 .. own position
                pos = c + i
                bk = [decoder_bucket(pos - j, s.rel_buckets, s.rel_max_dist) for j in range(n_keys)]
                for hd in range(H):
                    sl = slice(hd * dk, (hd + 1) * dk)
                    a[i, sl] = attend(q[i, sl], st.k[l][:n_keys, sl], st.v[l][:n_keys, sl], rb[bk, hd])
            x = x + a @ w[p + "wo"].T
            qc = rms_norm(x, w[p + "ln2"], s.eps) @ w[p + "wcq"].T
            cc = np.empty((k, I))
            for i in range(k):
                for hd in range(H):
                    sl = slice(hd * dk, (hd + 1) * dk)
                    cc[i, sl] = attend(qc[i, sl], st.ck[l][:, sl], st.cv[l][:, sl])
            x = x + cc @ w[p + "wco"].T
            x = x + self._ffn(p, rms_norm(x, w[p + "ln3"], s.eps))
        st.len = c + k
        return self.logit_scale * (rms_norm(x, w["dec.final_ln"], s.eps) @ self.lm.T)

    def forward_one(self, st: "DecState", token: int) -> np.ndarray:
        return self.forward_block(st, [token])[0]

    # ---- cache-less recomputation (used only to pin the cached path) -------
    def forward_full(self, st: "DecState", tokens) -> np.ndarray:
        """Logits for every prefix of `tokens`, recomputed from position 0 with
        whole-sequence masked attention; touches no self-attention cache."""
        s, w = self.s, self.w
        n, H, dk, I = len(tokens), s.n_heads, s.d_kv, s.inner
        x = w["emb"][np.asarray(tokens)]
        rb = w["dec.rel_bias"]
        bias = np.full((H, n, n), -np.inf)
        for i in range(n):
            for j in range(i + 1):
                bias[:, i, j] = rb[decoder_bucket(i - j, s.rel_buckets, s.rel_max_dist)]
        for l in range(self.dec_layers):
            p = f"dec.{l}."
            qkv = rms_norm(x, w[p + "ln1"], s.eps) @ w[p + "wqkv"].T
            q = qkv[:, :I].reshape(n, H, dk).transpose(1, 0, 2)
            kk = qkv[:, I:2 * I].reshape(n, H, dk).transpose(1, 0, 2)
            vv = qkv[:, 2 * I:].reshape(n, H, dk).transpose(1, 0, 2)
            a = softmax(q @ kk.transpose(0, 2, 1) + bias) @ vv
            x = x + a.transpose(1, 0, 2).reshape(n, I) @ w[p + "wo"].T
            qc = (rms_norm(x, w[p + "ln2"], s.eps) @ w[p + "wcq"].T).reshape(n, H, dk).transpose(1, 0, 2)
            ck = st.ck[l].reshape(-1, H, dk).transpose(1, 0, 2)
            cv = st.cv[l].reshape(-1, H, dk).transpose(1, 0, 2)
            cc = softmax(qc @ ck.transpose(0, 2, 1)) @ cv
            x = x + cc.transpose(1, 0, 2).reshape(n, I) @ w[p + "wco"].T
            x = x + self._ffn(p, rms_norm(x, w[p + "ln3"], s.eps))
        return self.logit_scale * (rms_norm(x, w["dec.final_ln"], s.eps) @ self.lm.T)


class DecState:
    """Per-sequence decoder state: self-attention K/V caches with a length
    counter (rewinding = lowering `len`; later appends overwrite) and the
    per-layer cross-attention K/V of the encoder memory."""

    def __init__(self, shape, cap: int):
        self.cap = cap
        self.len = 0
        self.k = [np.zeros((cap, shape.inner)) for _ in range(shape.n_layers)]
        self.v = [np.zeros((cap, shape.inner)) for _ in range(shape.n_layers)]
        self.ck, self.cv = [], []
        self.mem = None

    def rewind(self, new_len: int) -> None:
        assert 0 <= new_len <= self.len
        self.len = new_len
