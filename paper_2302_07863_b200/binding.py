"""ctypes binding of libbild.so: the same names and arguments as include/bild.h.

Only argument marshalling happens here; every step of the decode path runs in the
library's CUDA kernels.  PyTorch is used for device memory and streams only.  There
is no fallback: a missing library raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libbild.so")

BILD_OK = 0
ERR = {-1: "BILD_ERR_ARG", -2: "BILD_ERR_WORKSPACE", -3: "BILD_ERR_STATE", -4: "BILD_ERR_CAPACITY",
       -5: "BILD_ERR_CUDA", -6: "BILD_ERR_TIMEOUT"}
FP32, BF16 = 0, 1
FFN_RELU, FFN_GATED_GELU = 0, 1
MODE_BILD, MODE_SMALL_ONLY, MODE_LARGE_ONLY = 0, 1, 2
MAX_BLOCK = 16

EXPORTS = ["bild_query_workspace", "bild_create", "bild_create_tuned", "bild_tuning_default", "bild_destroy", "bild_encode", "bild_reset",
           "bild_small_step", "bild_large_verify", "bild_rewind", "bild_generate", "bild_generate_async",
           "bild_fetch_result", "bild_time_pass", "bild_uses_tensor_cores", "bild_launch_count", "bild_last_error", "bild_op_linear",
           "bild_op_lm_head_scratch_bytes", "bild_op_lm_head", "bild_op_lm_head_static", "bild_debug_bucket",
           "bild_debug_read_cache", "bild_op_lm_head_sliced", "bild_op_lm_head_stream", "bild_op_sublayer_scratch_bytes", "bild_op_attn_sublayer",
           "bild_op_ffn_sublayer", "bild_generate_sampled"]


class ModelCfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "d_kv", "d_ff", "ffn_kind", "vocab",
                                         "rel_buckets", "rel_max_dist")] + [("ln_eps", C.c_float),
                                                                            ("logit_scale", C.c_float)]


class Config(C.Structure):
    _fields_ = [("small_cfg", ModelCfg), ("large_cfg", ModelCfg)] + [
        (n, C.c_int32) for n in ("dtype", "max_enc_len", "max_dec_len", "max_draft", "start_id", "eos_id", "early_exit_layers")]


class EncLayer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("ln1", "wqkv", "wo", "ln2", "wi0", "wi1", "wfo")]


class DecLayer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("ln1", "wqkv", "wo", "ln2", "wcq", "wckv", "wco", "ln3",
                                          "wi0", "wi1", "wfo")]


class Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("emb", "lm_head", "enc_rel_bias", "dec_rel_bias", "enc_final_ln",
                                          "dec_final_ln")] + [("enc_layers", C.POINTER(EncLayer)),
                                                              ("dec_layers", C.POINTER(DecLayer))]


class Tuning(C.Structure):
    """bild_tuning: kernel selection and debugging switches (defaults from bild_tuning_default)."""
    _fields_ = [(n, C.c_int32) for n in ("host_loop", "pdl", "fused", "ffn_parts", "block_simt", "slice_mode", "slice_min_kb",
                                         "slice_mma_min", "slice_head", "slice_head_min_mb", "unit_attn", "umma", "enc_gemm",
                                         "enc_attn_mma", "enc_parallel", "spin_limit", "debug_skip_copies", "attn_all_keys", "graph_switch", "enc_split_k", "head_stream", "enc_attn_groups")]


class StepOut(C.Structure):
    _fields_ = [("argmax", C.c_int32), ("max_logit", C.c_float), ("lse", C.c_float), ("pmax", C.c_float),
                ("fallback", C.c_int32)]


class VerifyOut(C.Structure):
    _fields_ = [("argmax", C.c_int32 * MAX_BLOCK), ("lse", C.c_float * MAX_BLOCK), ("d", C.c_float * MAX_BLOCK),
                ("first_violation", C.c_int32), ("next_token", C.c_int32)]


class TraceRec(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("kind", "pos", "token", "k", "m")] + [("value", C.c_float)]


class Stats(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("small_steps", "large_calls", "fallbacks", "forced", "rollbacks",
                                         "discarded", "sum_k")]


_lib = None


def lib() -> C.CDLL:
    """The loaded library; raises if it has not been built (python -m paper_2302_07863_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python paper_2302_07863_b200/build.py`; "
                               "there is no fallback path")
        L = C.CDLL(LIB_PATH)
        vp, i32, f32 = C.c_void_p, C.c_int, C.c_float
        L.bild_query_workspace.argtypes = [C.POINTER(Config), C.POINTER(C.c_size_t)]
        L.bild_create.argtypes = [C.POINTER(Config), C.POINTER(Weights), C.POINTER(Weights), vp, C.c_size_t, vp,
                                  C.POINTER(vp)]
        L.bild_create_tuned.argtypes = [C.POINTER(Config), C.POINTER(Weights), C.POINTER(Weights), vp, C.c_size_t, vp,
                                        C.POINTER(Tuning), C.POINTER(vp)]
        L.bild_tuning_default.argtypes = [C.POINTER(Tuning)]
        L.bild_tuning_default.restype = None
        L.bild_destroy.argtypes = [vp]
        L.bild_destroy.restype = None
        L.bild_encode.argtypes = [vp, C.POINTER(C.c_int32), i32]
        L.bild_reset.argtypes = [vp]
        L.bild_small_step.argtypes = [vp, C.c_int32, f32, C.POINTER(StepOut), vp]
        L.bild_large_verify.argtypes = [vp, C.POINTER(C.c_int32), i32, f32, C.POINTER(VerifyOut), vp]
        L.bild_rewind.argtypes = [vp, i32, i32]
        L.bild_generate.argtypes = [vp, i32, f32, f32, i32, C.POINTER(C.c_int32), C.POINTER(i32),
                                    C.POINTER(TraceRec), i32, C.POINTER(i32), C.POINTER(Stats)]
        L.bild_generate_async.argtypes = [vp, i32, f32, f32, i32]
        L.bild_fetch_result.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(i32), C.POINTER(TraceRec), i32,
                                        C.POINTER(i32), C.POINTER(Stats)]
        L.bild_time_pass.argtypes = [vp, i32, i32, i32, i32, C.POINTER(f32)]
        L.bild_uses_tensor_cores.argtypes = [vp]
        L.bild_launch_count.argtypes = [vp]
        L.bild_launch_count.restype = C.c_int64
        L.bild_last_error.argtypes = [vp]
        L.bild_last_error.restype = C.c_char_p
        L.bild_op_linear.argtypes = [vp, i32, vp, vp, f32, vp, i32, i32, i32, vp]
        L.bild_op_lm_head_scratch_bytes.argtypes = [i32]
        L.bild_op_lm_head_scratch_bytes.restype = C.c_size_t
        L.bild_op_lm_head.argtypes = [vp, i32, vp, vp, f32, f32, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        L.bild_op_lm_head_static.argtypes = [vp, i32, vp, vp, f32, f32, vp, i32, i32, i32, vp, vp, vp, vp, vp]
        L.bild_debug_bucket.argtypes = [i32, i32, i32, i32]
        _lib = L
    return _lib


class BildError(RuntimeError):
    def __init__(self, code, msg=""):
        super().__init__(f"{ERR.get(code, code)}: {msg}")
        self.code = code


def model_cfg(shape, logit_scale: float) -> ModelCfg:
    """ModelCfg from any object with the fields of workloads.ModelShape."""
    return ModelCfg(shape.n_layers, shape.d_model, shape.n_heads, shape.d_kv, shape.d_ff,
                    FFN_RELU if shape.ffn == "relu" else FFN_GATED_GELU, shape.vocab, shape.rel_buckets,
                    shape.rel_max_dist, shape.eps, logit_scale)


def upload_model(tensors: dict, device):
    """numpy tensors (fp32, or uint16 bf16 bit patterns) -> torch tensors on the device."""
    import torch
    out = {}
    for k, v in tensors.items():
        if v.dtype == np.uint16:
            out[k] = torch.from_numpy(v.view(np.int16)).to(device).view(torch.bfloat16)
        else:
            out[k] = torch.from_numpy(np.ascontiguousarray(v, dtype=np.float32)).to(device)
    return out


def make_weights(shape, dev: dict):
    """Weights struct of device pointers for one model; returns (struct, keep-alive list)."""
    p = lambda name: dev[name].data_ptr()
    L = shape.n_layers
    enc = (EncLayer * L)()
    dec = (DecLayer * L)()
    gated = shape.ffn != "relu"
    for l in range(L):
        e, d = f"enc.{l}.", f"dec.{l}."
        enc[l] = EncLayer(p(e + "ln1"), p(e + "wqkv"), p(e + "wo"), p(e + "ln2"), p(e + "wi0"),
                          p(e + "wi1") if gated else None, p(e + "wfo"))
        dec[l] = DecLayer(p(d + "ln1"), p(d + "wqkv"), p(d + "wo"), p(d + "ln2"), p(d + "wcq"), p(d + "wckv"),
                          p(d + "wco"), p(d + "ln3"), p(d + "wi0"), p(d + "wi1") if gated else None, p(d + "wfo"))
    w = Weights(p("emb"), p("lm_head") if "lm_head" in dev else p("emb"), p("enc.rel_bias"), p("dec.rel_bias"),
                p("enc.final_ln"), p("dec.final_ln"), enc, dec)
    return w, [enc, dec, dev]


class Context:
    """Owns the workspace tensor and keeps the weight tensors alive; methods mirror the C calls."""

    def __init__(self, cfg: Config, small_shape, small_dev: dict, large_shape, large_dev: dict, device="cuda:0",
                 stream=None, tuning: dict | None = None):
        import torch
        self.L = lib()
        self.cfg = cfg
        self.device = torch.device(device)
        nbytes = C.c_size_t()
        self._check(self.L.bild_query_workspace(C.byref(cfg), C.byref(nbytes)), "bild_query_workspace")
        self.workspace_bytes = nbytes.value
        self.workspace = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        ws, self._keep_s = make_weights(small_shape, small_dev)
        wl, self._keep_l = make_weights(large_shape, large_dev)
        self.stream = stream
        sp = stream.cuda_stream if stream is not None else None
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            if tuning:   # bild_tuning: the defaults with the given fields replaced
                t = Tuning()
                self.L.bild_tuning_default(C.byref(t))
                for key, val in tuning.items():
                    if key not in dict(Tuning._fields_):
                        raise KeyError(f"bild_tuning has no field {key!r}")
                    setattr(t, key, int(val))
                rc = self.L.bild_create_tuned(C.byref(cfg), C.byref(ws), C.byref(wl), base, nbytes.value, sp, C.byref(t),
                                              C.byref(h))
            else:
                rc = self.L.bild_create(C.byref(cfg), C.byref(ws), C.byref(wl), base, nbytes.value, sp, C.byref(h))
        if rc != BILD_OK:
            raise BildError(rc, "bild_create")
        self.h = h

    def _check(self, rc, what=""):
        if rc != BILD_OK:
            msg = self.L.bild_last_error(self.h).decode() if getattr(self, "h", None) else what
            raise BildError(rc, msg)

    def close(self):
        if getattr(self, "h", None):
            self.L.bild_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()

    def encode(self, ids):
        a = np.ascontiguousarray(ids, dtype=np.int32)
        self._check(self.L.bild_encode(self.h, a.ctypes.data_as(C.POINTER(C.c_int32)), len(a)))

    def reset(self):
        self._check(self.L.bild_reset(self.h))

    def small_step(self, token: int, alpha_fb: float, logits_dbg=None) -> StepOut:
        out = StepOut()
        self._check(self.L.bild_small_step(self.h, int(token), alpha_fb, C.byref(out),
                                           logits_dbg.data_ptr() if logits_dbg is not None else None))
        return out

    def large_verify(self, tokens, alpha_rb: float, logits_dbg=None) -> VerifyOut:
        a = np.ascontiguousarray(tokens, dtype=np.int32)
        out = VerifyOut()
        self._check(self.L.bild_large_verify(self.h, a.ctypes.data_as(C.POINTER(C.c_int32)), len(a), alpha_rb,
                                             C.byref(out), logits_dbg.data_ptr() if logits_dbg is not None else None))
        return out

    def rewind(self, which: int, new_len: int):
        self._check(self.L.bild_rewind(self.h, which, new_len))

    def generate(self, mode: int, alpha_fb: float, alpha_rb: float, max_len: int):
        toks = (C.c_int32 * max(1, max_len))()
        n = C.c_int()
        cap = (max_len + 1) * (self.cfg.max_draft + 3)
        tr = (TraceRec * cap)()
        nt = C.c_int()
        st = Stats()
        self._check(self.L.bild_generate(self.h, mode, alpha_fb, alpha_rb, max_len, toks, C.byref(n), tr, cap,
                                         C.byref(nt), C.byref(st)))
        return self._unpack(toks, n, tr, nt, cap, st)

    def generate_sampled(self, mode: int, alpha_fb: float, alpha_rb: float, max_len: int, top_p: float, u_small, u_large):
        """bild_generate_sampled: nucleus sampling from both models; u_small / u_large: max_len + 1 uniform numbers each."""
        toks = (C.c_int32 * max(1, max_len))()
        n = C.c_int()
        cap = (max_len + 1) * (self.cfg.max_draft + 3)
        tr = (TraceRec * cap)()
        nt = C.c_int()
        st = Stats()
        us = np.ascontiguousarray(u_small, dtype=np.float32)
        ul = np.ascontiguousarray(u_large, dtype=np.float32)
        assert len(us) >= max_len + 1 and len(ul) >= max_len + 1
        fp = C.POINTER(C.c_float)
        self.L.bild_generate_sampled.argtypes = [C.c_void_p, C.c_int, C.c_float, C.c_float, C.c_int, C.c_float, fp, fp,
                                                 C.POINTER(C.c_int32), C.POINTER(C.c_int), C.POINTER(TraceRec), C.c_int,
                                                 C.POINTER(C.c_int), C.POINTER(Stats)]
        self._check(self.L.bild_generate_sampled(self.h, mode, alpha_fb, alpha_rb, max_len, top_p, us.ctypes.data_as(fp),
                                                 ul.ctypes.data_as(fp), toks, C.byref(n), tr, cap, C.byref(nt), C.byref(st)))
        return self._unpack(toks, n, tr, nt, cap, st)

    def generate_async(self, mode: int, alpha_fb: float, alpha_rb: float, max_len: int):
        self._check(self.L.bild_generate_async(self.h, mode, alpha_fb, alpha_rb, max_len))

    def fetch_result(self, max_len: int):
        toks = (C.c_int32 * max(1, max_len))()
        n = C.c_int()
        cap = (max_len + 1) * (self.cfg.max_draft + 3)
        tr = (TraceRec * cap)()
        nt = C.c_int()
        st = Stats()
        self._check(self.L.bild_fetch_result(self.h, toks, C.byref(n), tr, cap, C.byref(nt), C.byref(st)))
        return self._unpack(toks, n, tr, nt, cap, st)

    @staticmethod
    def _unpack(toks, n, tr, nt, cap, st):
        trace = [(r.kind, r.pos, r.token, r.k, r.m, r.value) for r in tr[:min(nt.value, cap)]]
        stats = {f: getattr(st, f) for f, _ in Stats._fields_}
        return dict(tokens=list(toks[:n.value]), trace=trace, stats=stats, n_trace=nt.value)

    def time_pass(self, which: int, k: int, cache_len: int, iters: int) -> float:
        ms = C.c_float()
        self._check(self.L.bild_time_pass(self.h, which, k, cache_len, iters, C.byref(ms)))
        return ms.value

    def read_cache(self, which: int, what: int, layer: int, n_heads: int, capacity: int, d_kv: int):
        """One layer's cached keys / values [n_heads][capacity][d_kv] as a numpy array (what: 0 / 1 cross K / V, 2 / 3 self)."""
        out = np.empty((n_heads, capacity, d_kv), dtype=np.float32)
        self.L.bild_debug_read_cache.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_size_t]
        self._check(self.L.bild_debug_read_cache(self.h, which, what, layer, out.ctypes.data, out.size))
        return out

    def uses_tensor_cores(self) -> bool:
        return bool(self.L.bild_uses_tensor_cores(self.h))

    def launch_count(self) -> int:
        return self.L.bild_launch_count(self.h)


def op_linear(W, X, gain, eps, M, N, K, stream=None):
    """Y[M][N] = rms?(X) W^T through the library's kernel; W bf16 or fp32 torch tensor."""
    import torch
    Y = torch.empty((M, N), dtype=torch.float32, device=X.device)
    dt = BF16 if W.dtype == torch.bfloat16 else FP32
    rc = lib().bild_op_linear(W.data_ptr(), dt, X.data_ptr(), gain.data_ptr() if gain is not None else None, eps,
                              Y.data_ptr(), M, N, K, stream.cuda_stream if stream is not None else None)
    if rc != BILD_OK:
        raise BildError(rc, "bild_op_linear")
    return Y


def op_lm_head(W, X, gain, eps, scale, target, M, V, K, want_logits=False, stream=None):
    import torch
    dev = X.device
    nb = lib().bild_op_lm_head_scratch_bytes(V)
    scratch = torch.zeros(nb + 256, dtype=torch.uint8, device=dev)
    sp = (scratch.data_ptr() + 255) // 256 * 256
    am = torch.empty(M, dtype=torch.int32, device=dev)
    mx = torch.empty(M, dtype=torch.float32, device=dev)
    lse = torch.empty(M, dtype=torch.float32, device=dev)
    ga = torch.zeros(M, dtype=torch.float32, device=dev)
    lg = torch.empty((M, V), dtype=torch.float32, device=dev) if want_logits else None
    dt = BF16 if W.dtype == torch.bfloat16 else FP32
    rc = lib().bild_op_lm_head(W.data_ptr(), dt, X.data_ptr(), gain.data_ptr() if gain is not None else None, eps,
                               scale, target.data_ptr() if target is not None else None, M, V, K, am.data_ptr(),
                               mx.data_ptr(), lse.data_ptr(), ga.data_ptr(), lg.data_ptr() if lg is not None else None,
                               sp, stream.cuda_stream if stream is not None else None)
    if rc != BILD_OK:
        raise BildError(rc, "bild_op_lm_head")
    return am, mx, lse, ga, lg


def op_lm_head_sliced(W, X, gain, eps, scale, target, M, V, K, want_logits=False):
    """bild_op_lm_head_sliced: the tensor-core head of the bf16 decoder passes (bf16 weights only)."""
    import torch
    dev = X.device
    L = lib()
    L.bild_op_lm_head_scratch_bytes.restype = C.c_size_t
    nb = L.bild_op_lm_head_scratch_bytes(V)
    scratch = torch.zeros(nb + 512, dtype=torch.uint8, device=dev)
    sp = (scratch.data_ptr() + 255) // 256 * 256
    am = torch.empty(M, dtype=torch.int32, device=dev)
    mx = torch.empty(M, dtype=torch.float32, device=dev)
    lse = torch.empty(M, dtype=torch.float32, device=dev)
    ga = torch.zeros(M, dtype=torch.float32, device=dev)
    lg = torch.empty((M, V), dtype=torch.float32, device=dev) if want_logits else None
    vp = C.c_void_p
    L.bild_op_lm_head_sliced.argtypes = [vp, vp, vp, C.c_float, C.c_float, vp, C.c_int, C.c_int, C.c_int, vp, vp, vp, vp, vp, vp, vp]
    rc = L.bild_op_lm_head_sliced(W.data_ptr(), X.data_ptr(), gain.data_ptr() if gain is not None else None, eps, scale,
                                  target.data_ptr() if target is not None else None, M, V, K, am.data_ptr(), mx.data_ptr(),
                                  lse.data_ptr(), ga.data_ptr(), lg.data_ptr() if lg is not None else None, sp, None)
    if rc != BILD_OK:
        raise BildError(rc, "bild_op_lm_head_sliced")
    return am, mx, lse, ga, lg


def op_lm_head_stream(W, X, gain, eps, scale, target, V, K, want_logits=False):
    """bild_op_lm_head_stream: the streaming head of the bf16 single-row passes (one row, bf16 weights, K <= 1024)."""
    import torch
    dev = X.device
    L = lib()
    L.bild_op_lm_head_scratch_bytes.restype = C.c_size_t
    nb = L.bild_op_lm_head_scratch_bytes(V)
    scratch = torch.zeros(nb + 512, dtype=torch.uint8, device=dev)
    sp = (scratch.data_ptr() + 255) // 256 * 256
    am = torch.empty(1, dtype=torch.int32, device=dev)
    mx = torch.empty(1, dtype=torch.float32, device=dev)
    lse = torch.empty(1, dtype=torch.float32, device=dev)
    ga = torch.zeros(1, dtype=torch.float32, device=dev)
    lg = torch.empty((1, V), dtype=torch.float32, device=dev) if want_logits else None
    vp = C.c_void_p
    L.bild_op_lm_head_stream.argtypes = [vp, vp, vp, C.c_float, C.c_float, vp, C.c_int, C.c_int, vp, vp, vp, vp, vp, vp, vp]
    rc = L.bild_op_lm_head_stream(W.data_ptr(), X.data_ptr(), gain.data_ptr() if gain is not None else None, eps, scale,
                                  target.data_ptr() if target is not None else None, V, K, am.data_ptr(), mx.data_ptr(),
                                  lse.data_ptr(), ga.data_ptr(), lg.data_ptr() if lg is not None else None, sp, None)
    if rc != BILD_OK:
        raise BildError(rc, "bild_op_lm_head_stream")
    return am, mx, lse, ga, lg


def _sub_scratch(d, F, dev):
    import torch
    L = lib()
    L.bild_op_sublayer_scratch_bytes.restype = C.c_size_t
    L.bild_op_sublayer_scratch_bytes.argtypes = [C.c_int, C.c_int]
    scratch = torch.zeros(L.bild_op_sublayer_scratch_bytes(d, F) + 256, dtype=torch.uint8, device=dev)
    return scratch, (scratch.data_ptr() + 255) // 256 * 256


def op_ffn_sublayer(Wi0, Wi1, Wfo, gain, eps, x_in, M, d, F, parts=0):
    """x_in + FFN(rms_norm(x_in)) on the fused feed-forward kernel; returns x_out [M][d]."""
    import torch
    scratch, sp = _sub_scratch(d, F, x_in.device)
    x_out = torch.empty((M, d), dtype=torch.float32, device=x_in.device)
    vp = C.c_void_p
    L = lib()
    L.bild_op_ffn_sublayer.argtypes = [vp, vp, vp, vp, C.c_float, vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp]
    rc = L.bild_op_ffn_sublayer(Wi0.data_ptr(), Wi1.data_ptr() if Wi1 is not None else None, Wfo.data_ptr(), gain.data_ptr(), eps,
                                x_in.data_ptr(), x_out.data_ptr(), M, d, F, parts, sp, None)
    if rc != BILD_OK:
        raise BildError(rc, "bild_op_ffn_sublayer")
    return x_out


def op_attn_sublayer(self_attn, Wp, Wo, gain, eps, x_in, kc, vc, cap, n_before, bias, M, d, H, dkv):
    """x_in + W_o Attention(...) on the fused attention kernel; kc / vc [H][cap][dkv] fp32 (appended to for self-attention)."""
    import torch
    scratch, sp = _sub_scratch(d, 0, x_in.device)
    x_out = torch.empty((M, d), dtype=torch.float32, device=x_in.device)
    vp = C.c_void_p
    L = lib()
    L.bild_op_attn_sublayer.argtypes = [C.c_int, vp, vp, vp, C.c_float, vp, vp, vp, vp, C.c_int, C.c_int, vp, C.c_int, C.c_int,
                                        C.c_int, C.c_int, vp, vp]
    rc = L.bild_op_attn_sublayer(1 if self_attn else 0, Wp.data_ptr(), Wo.data_ptr(), gain.data_ptr(), eps, x_in.data_ptr(),
                                 x_out.data_ptr(), kc.data_ptr(), vc.data_ptr(), cap, n_before,
                                 bias.data_ptr() if bias is not None else None, M, d, H, dkv, sp, None)
    if rc != BILD_OK:
        raise BildError(rc, "bild_op_attn_sublayer")
    return x_out


def op_lm_head_static(W, X, gain, eps, scale, target, M, V, K, stream=None):
    """bild_op_lm_head_static: the fused LM head for callers that cannot allocate scratch
    (a worker inside a process whose allocator owns the device, or a loop that must not
    hit cudaMalloc's device-wide synchronisation).  Only the four small output tensors are
    created here, by the test harness; the library call itself allocates nothing."""
    import torch
    dev = X.device
    am = torch.empty(M, dtype=torch.int32, device=dev)
    mx = torch.empty(M, dtype=torch.float32, device=dev)
    lse = torch.empty(M, dtype=torch.float32, device=dev)
    ga = torch.zeros(M, dtype=torch.float32, device=dev)
    dt = BF16 if W.dtype == torch.bfloat16 else FP32
    rc = lib().bild_op_lm_head_static(W.data_ptr(), dt, X.data_ptr(), gain.data_ptr() if gain is not None else None,
                                      eps, scale, target.data_ptr() if target is not None else None, M, V, K,
                                      am.data_ptr(), mx.data_ptr(), lse.data_ptr(), ga.data_ptr(),
                                      stream.cuda_stream if stream is not None else None)
    if rc != BILD_OK:
        raise BildError(rc, "bild_op_lm_head_static")
    return am, mx, lse, ga
