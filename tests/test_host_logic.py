"""CPU-only checks of the library's host side: it builds, loads, exports every symbol the
header declares, validates configurations, and its relative-position buckets equal the
oracle's exact integer rule.  No compute call is made (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

from oracle.t5 import decoder_bucket, encoder_bucket
from workloads import MODEL_SHAPES

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2302_07863_b200 import build, binding
    build.build()
    return binding.lib()


def test_exports_every_declared_symbol(L):
    hdr = open(os.path.join(ROOT, "include", "bild.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(bild_[a-z_0-9]+)\s*\(", hdr))
    assert {"bild_create", "bild_encode", "bild_small_step", "bild_large_verify", "bild_generate"} <= names
    from paper_2302_07863_b200.binding import EXPORTS
    assert names == set(EXPORTS)
    for n in names:
        assert getattr(L, n) is not None


def test_bucket_tables_equal_oracle(L):
    for nb, md in ((32, 128), (16, 64), (8, 20)):
        for delta in range(0, 600):
            assert L.bild_debug_bucket(0, delta, nb, md) == decoder_bucket(delta, nb, md)
        for rel in range(-600, 600):
            assert L.bild_debug_bucket(1, rel, nb, md) == encoder_bucket(rel, nb, md)
    assert L.bild_debug_bucket(0, -1, 32, 128) == -1
    assert L.bild_debug_bucket(0, 1, 5, 128) == -1


def _cfg(**over):
    from paper_2302_07863_b200.binding import Config, model_cfg
    c = Config(model_cfg(MODEL_SHAPES["t5_s"], 1.0), model_cfg(MODEL_SHAPES["t5_l"], 1.0), 1, 512, 65, 10, 0, -1)
    for k, v in over.items():
        setattr(c, k, v)
    return c


def test_workspace_query_and_validation(L):
    n = C.c_size_t()
    assert L.bild_query_workspace(C.byref(_cfg()), C.byref(n)) == 0
    s, l = MODEL_SHAPES["t5_s"], MODEL_SHAPES["t5_l"]
    # at least the self- and cross-attention K/V of both models (fp32)
    need = sum(2 * m.n_layers * m.inner * (65 + 512) * 4 for m in (s, l))
    # ... plus two re-ordered copies of the feed-forward output matrices of both decoders (bf16 configurations)
    need += sum(2 * m.n_layers * m.d_ff * m.d_model * 2 for m in (s, l))
    # ... plus activations, per-model encoder temporaries (fp32 and bf16 pairs), head partials
    assert need <= n.value <= need + 96 * 2 ** 20
    n2 = C.c_size_t()
    assert L.bild_query_workspace(C.byref(_cfg(max_dec_len=257)), C.byref(n2)) == 0 and n2.value > n.value
    for bad in (dict(max_draft=0), dict(max_draft=16), dict(max_enc_len=0), dict(max_dec_len=1), dict(dtype=7),
                dict(start_id=-1), dict(max_dec_len=100000)):
        assert L.bild_query_workspace(C.byref(_cfg(**bad)), C.byref(n)) == -1, bad
    c = _cfg()
    c.small_cfg.vocab = 100
    assert L.bild_query_workspace(C.byref(c), C.byref(n)) == -1      # vocabularies must agree
    c = _cfg()
    c.large_cfg.d_kv = 48
    assert L.bild_query_workspace(C.byref(c), C.byref(n)) == -1
    assert L.bild_query_workspace(None, C.byref(n)) == -1
    assert L.bild_query_workspace(C.byref(_cfg()), None) == -1


def test_create_rejects_bad_arguments_without_a_gpu(L):
    from paper_2302_07863_b200.binding import Weights
    h = C.c_void_p()
    w = Weights()
    assert L.bild_create(C.byref(_cfg()), C.byref(w), C.byref(w), None, 0, None, C.byref(h)) == -1
    assert L.bild_create(C.byref(_cfg()), C.byref(w), C.byref(w), 12345, 1 << 40, None, C.byref(h)) == -2  # misaligned
    assert L.bild_create(C.byref(_cfg()), C.byref(w), C.byref(w), 4096, 16, None, C.byref(h)) == -2        # too small
    assert not h.value
    assert L.bild_encode(None, None, 0) == -1
    assert L.bild_launch_count(None) == 0
    assert L.bild_last_error(None) == b"null context"
    assert L.bild_op_linear(None, 0, None, None, 0.0, None, 1, 1, 8, None) == -1
    assert L.bild_op_lm_head_scratch_bytes(32128) > 0


def test_model_analysis_counts():
    """Analytic FLOPs / memory operations of the stored runs: the byte model agrees with the one the
    benchmarks use, and BiLD trades slightly more FLOPs for several times fewer memory operations
    than the large model alone (the direction of the paper's model-analysis figure)."""
    from workloads import MODEL_SHAPES
    from paper_2302_07863_b200 import microbench, model_analysis
    s = MODEL_SHAPES["t5_l"]
    for k, cache in [(1, 0), (5, 64), (16, 1024)]:
        assert model_analysis.pass_counts(s, 2, 4, cache, 512, k)[1] == microbench.pass_bytes(s, 2, 4, cache, 512, k)
    # one row, no cache, no encoder: 2 flops per weight plus one key
    f, _ = model_analysis.pass_counts(s, 2, 4, 0, 0, 1)
    params = s.n_layers * (6 * s.inner * s.d_model + 2 * s.d_model * s.d_ff) + s.vocab * s.d_model
    assert f == 2 * params + 4 * s.inner * s.n_layers
    r = model_analysis.analyse("t5_sum")["normalised"]
    assert 1.0 < r["flops"] < 1.5
    assert r["memory_operations"] < 0.5
    assert abs(r["arithmetic_intensity"] - r["flops"] / r["memory_operations"]) < 1e-9
