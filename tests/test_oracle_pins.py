"""Pins for the CPU oracle: it is checked against things other than itself
(closed forms, library routines, an independent library model built from a
config, brute force without caches, special cases of the policy that reduce
to plain greedy decoding, a post-hoc certificate of a finished run)."""
import dataclasses
import math

import numpy as np
import pytest
import torch

from oracle import bild
from oracle.t5 import (Model, attend, decoder_bucket, encoder_bucket, gelu_tanh, rms_norm, softmax)
from workloads import MODEL_SHAPES, WORKLOADS, gen_ids, gen_model, gen_uniforms

INF = math.inf


def make_pair(wl_name, scale_s=25.0, scale_l=15.0):
    wl = WORKLOADS[wl_name]
    S = Model(MODEL_SHAPES[wl.small], gen_model(MODEL_SHAPES[wl.small], wl.seed, wl.dtype), scale_s)
    L = Model(MODEL_SHAPES[wl.large], gen_model(MODEL_SHAPES[wl.large], wl.seed, wl.dtype), scale_l)
    ids = gen_ids(S.s.vocab, wl.enc_len, wl.seed)
    return wl, S, L, ids


@pytest.fixture(scope="module", params=["tiny", "odd_bf16"])
def pair(request):
    return make_pair(request.param)


# ---- policy special cases that reduce to plain greedy decoding ---------------
def test_never_fallback_equals_small_greedy(pair):
    wl, S, L, ids = pair
    ref = bild.generate(S, L, ids, 0.0, INF, wl.gen_len, mode="small")
    got = bild.generate(S, L, ids, 0.0, INF, wl.gen_len, max_draft=10 ** 9)
    assert got["tokens"] == ref["tokens"]
    assert got["stats"]["large_calls"] == 0
    # and it really is arg-max decoding of the small model, recomputed without caches
    st = S.start(ids, wl.gen_len + 1)
    Z = S.forward_full(st, [0] + ref["tokens"][:-1])
    assert [int(np.argmax(z)) for z in Z] == ref["tokens"]


@pytest.mark.parametrize("alpha_rb", [0.0, 3.0, INF])
def test_always_fallback_equals_large_greedy(pair, alpha_rb):
    wl, S, L, ids = pair
    ref = bild.generate(S, L, ids, 0.0, INF, wl.gen_len, mode="large")
    got = bild.generate(S, L, ids, 2.0, alpha_rb, wl.gen_len)
    assert got["tokens"] == ref["tokens"]
    assert got["stats"]["rollbacks"] == 0 and got["stats"]["sum_k"] == wl.gen_len
    st = L.start(ids, wl.gen_len + 1)
    Z = L.forward_full(st, [0] + ref["tokens"][:-1])
    assert [int(np.argmax(z)) for z in Z] == ref["tokens"]


@pytest.mark.parametrize("alpha_fb,max_draft", [(0.0, 10), (0.3, 3), (0.6, 10), (0.0, 1)])
def test_negative_rollback_threshold_equals_large_greedy(pair, alpha_fb, max_draft):
    """d >= 0 > alpha_RB: the first pending draft is always replaced by the large
    model's arg-max, so the output is the large model's greedy decode whatever
    the small model does (up to drafts still pending when the loop stops).
    Exercises rollback and cache rewinding heavily."""
    wl, S, L, ids = pair
    ref = bild.generate(S, L, ids, 0.0, INF, wl.gen_len, mode="large")
    got = bild.generate(S, L, ids, alpha_fb, -1.0, wl.gen_len, max_draft=max_draft)
    # the loop may stop with unverified drafts pending; everything up to the last
    # position written by the large model must be the large model's greedy decode
    verified = max(t[1] for t in got["trace"] if t[0] in (bild.KIND_VERIFY_OK, bild.KIND_ROLLBACK))
    assert verified >= wl.gen_len - max_draft
    assert got["tokens"][:verified] == ref["tokens"][:verified]
    if alpha_fb == 0.0 and max_draft == 10:
        assert got["stats"]["rollbacks"] > 0


# ---- block pass == token-by-token == cache-less recomputation -----------------
@pytest.mark.parametrize("split", [(1,) * 12, (5, 7), (12,), (3, 1, 8)])
def test_block_equals_sequential_equals_full(pair, split):
    wl, S, L, ids = pair
    rng = np.random.default_rng(5)
    toks = [0] + [int(t) for t in rng.integers(2, L.s.vocab, 11)]
    st0 = L.start(ids, 16)
    full = L.forward_full(st0, toks)
    st = L.start(ids, 16)
    rows, pos = [], 0
    for k in split:
        rows.append(L.forward_block(st, toks[pos:pos + k]))
        pos += k
    got = np.concatenate(rows)
    assert np.max(np.abs(got - full)) < 1e-10


def test_rewind_then_refeed_matches_fresh_run(pair):
    wl, S, L, ids = pair
    toks = [0, 7, 9, 11, 13, 17, 19]
    st = L.start(ids, 16)
    L.forward_block(st, toks)
    st.rewind(3)
    again = L.forward_block(st, [50, 51])
    fresh = L.forward_full(L.start(ids, 16), toks[:3] + [50, 51])[3:]
    assert np.max(np.abs(again - fresh)) < 1e-10


# ---- post-hoc certificate of finished runs -----------------------------------
@pytest.mark.parametrize("alpha_fb,alpha_rb,max_draft", [(0.3, 16.0, 10), (0.25, 17.5, 4), (0.5, 15.0, 10),
                                                          (0.0, 16.5, 5)])
def test_certificate(pair, alpha_fb, alpha_rb, max_draft):
    """Recompute both models on the final sequence without caches and check
    every token against the policy that its trace record claims."""
    wl, S, L, ids = pair
    r = bild.generate(S, L, ids, alpha_fb, alpha_rb, wl.gen_len, max_draft=max_draft)
    y = [0] + r["tokens"]
    assert len(r["tokens"]) == wl.gen_len
    # who wrote each surviving position: replay the trace
    owner, verified = {}, 0
    for kind, pos, tok, k, m, val in r["trace"]:
        if kind == bild.KIND_SMALL_ACCEPT:
            owner[pos] = "S"
        elif kind in (bild.KIND_VERIFY_OK, bild.KIND_ROLLBACK):
            for p in [p for p in owner if p > pos]:
                del owner[p]
            owner[pos] = "L"
            verified = pos
    assert sorted(owner) == list(range(1, wl.gen_len + 1))
    ZS = S.forward_full(S.start(ids, len(y)), y[:-1])
    ZL = L.forward_full(L.start(ids, len(y)), y[:-1])
    for j in range(1, len(y)):
        zs, zl = ZS[j - 1], ZL[j - 1]
        if owner[j] == "S":
            assert int(np.argmax(zs)) == y[j]
            assert softmax(zs).max() >= alpha_fb
            if j <= verified:
                d = -math.log(softmax(zl)[y[j]])
                assert d <= alpha_rb
        else:
            assert int(np.argmax(zl)) == y[j]
    # progress: every large call consumes at least one token; drafts are capped
    run = 0
    for kind, *_ in r["trace"]:
        run = run + 1 if kind == bild.KIND_SMALL_ACCEPT else 0
        assert run <= max_draft
    assert r["stats"]["large_calls"] <= wl.gen_len
    assert r["stats"]["sum_k"] >= r["stats"]["large_calls"]


def test_threshold_endpoints_and_equality(pair):
    wl, S, L, ids = pair
    r = bild.generate(S, L, ids, 0.0, INF, 8, max_draft=100)
    pm = [t[5] for t in r["trace"]]
    # equality keeps the small model's token (fallback only if strictly below)
    r_eq = bild.generate(S, L, ids, pm[0], INF, 1, max_draft=100)
    assert r_eq["trace"][0][0] == bild.KIND_SMALL_ACCEPT
    r_above = bild.generate(S, L, ids, np.nextafter(pm[0], 1.0), INF, 1, max_draft=100)
    assert r_above["trace"][0][0] == bild.KIND_FALLBACK


def test_rollback_threshold_is_strict(pair):
    """Eq. 3 rolls back when the distance is strictly above alpha_RB: a threshold equal to the first scanned
    distance leaves that draft in place, the next representable value below it rolls it back."""
    wl, S, L, ids = pair
    base = bild.generate(S, L, ids, 0.0, INF, 4, max_draft=2)            # two drafts, then a forced hand-over
    v = next(t for t in base["trace"] if t[0] in (bild.KIND_VERIFY_OK, bild.KIND_ROLLBACK))
    assert v[0] == bild.KIND_VERIFY_OK and v[3] == 3
    # the distances of the two scanned drafts, recomputed from the large model alone
    st = L.start(ids, 8)
    Z = L.forward_block(st, [0] + base["tokens"][:2])
    d = [bild.max_prob(Z[i])[2] - Z[i][base["tokens"][i]] for i in range(2)]
    assert abs(max(d) - v[5]) < 1e-12
    r_eq = bild.generate(S, L, ids, 0.0, d[0], 4, max_draft=2)
    first = next(t for t in r_eq["trace"] if t[0] in (bild.KIND_VERIFY_OK, bild.KIND_ROLLBACK))
    assert not (first[0] == bild.KIND_ROLLBACK and first[4] == 0)          # d_0 == alpha_RB: no violation at row 0
    r_below = bild.generate(S, L, ids, 0.0, np.nextafter(d[0], -INF), 4, max_draft=2)
    first = next(t for t in r_below["trace"] if t[0] in (bild.KIND_VERIFY_OK, bild.KIND_ROLLBACK))
    assert first[0] == bild.KIND_ROLLBACK and first[4] == 0 and first[5] == d[0]


def test_trace_margins_line_up_with_the_trace(pair):
    """One margin triple per trace record; their minima are the global margins."""
    wl, S, L, ids = pair
    r = bild.generate(S, L, ids, 0.3, 16.0, 24, max_draft=4)
    tm = r["trace_margins"]
    assert len(tm) == len(r["trace"])
    assert min(t[1] for t in tm) == r["margins"]["fallback"] and min(t[2] for t in tm) == r["margins"]["rollback"]
    # the per-record gaps also cover the rejected candidates a fallback record names
    used = [t[0] for rec, t in zip(r["trace"], tm) if rec[0] not in (bild.KIND_FALLBACK, bild.KIND_FORCED)]
    assert min(used) == r["margins"]["argmax"] and min(t[0] for t in tm) <= r["margins"]["argmax"]
    for rec, t in zip(r["trace"], tm):
        if rec[0] in (bild.KIND_FALLBACK, bild.KIND_FORCED, bild.KIND_SMALL_ACCEPT):
            assert t[1] == abs(rec[5] - 0.3) and t[2] == INF
        else:
            assert t[1] == INF and (t[2] < INF) == (rec[3] > 1)


def test_bf16_bit_helpers_against_torch():
    """The shared generator's fp32 -> bf16 rounding (nearest, ties to even) and the oracle's bf16 -> fp64
    widening, against torch's bfloat16 conversions: random values, values next to a rounding boundary,
    exact ties, signed zeros, subnormals."""
    import torch
    from oracle.t5 import to_f64
    from workloads import bf16_bits_to_f32, bf16_round_bits
    rng = np.random.default_rng(7)
    x = (rng.standard_normal(20000) * np.exp(rng.uniform(-30, 30, 20000))).astype(np.float32)
    base = (rng.integers(0, 1 << 15, 4000).astype(np.uint32) << 16)             # exactly representable
    ties = (base | 0x8000).view(np.float32)                                        # half-way cases
    near = np.concatenate([(base | 0x7FFF).view(np.float32), (base | 0x8001).view(np.float32)])
    special = np.array([0.0, -0.0, 1e-40, -1e-40, 1.0, -1.0, 65504.0, 3.3895314e38], dtype=np.float32)
    x = np.concatenate([x, ties, -ties, near, -near, special])
    x = x[np.isfinite(x)]
    bits = bf16_round_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16)
    assert np.array_equal(bits.view(np.int16), ref.view(torch.int16).numpy())
    assert np.array_equal(bf16_bits_to_f32(bits).view(np.uint32), ref.float().numpy().view(np.uint32))
    assert np.array_equal(to_f64(bits), ref.double().numpy())
    # a truncating conversion or a wrong shift would differ on the ties / near-boundary values
    assert np.any(bits != (x.view(np.uint32) >> 16).astype(np.uint16))
    f = rng.standard_normal(100).astype(np.float32)
    assert np.array_equal(to_f64(f), f.astype(np.float64))


def test_forced_fallback_after_max_draft(pair):
    wl, S, L, ids = pair
    r = bild.generate(S, L, ids, 0.0, INF, 12, max_draft=3)
    kinds = [t[0] for t in r["trace"]]
    assert kinds[:5] == [0, 0, 0, bild.KIND_FORCED, bild.KIND_VERIFY_OK]
    assert r["trace"][4][3] == 4          # k = 3 drafts + the current token


def test_eos_stops_the_loop(pair):
    wl, S, L, ids = pair
    ref = bild.generate(S, L, ids, 0.0, INF, 10, mode="small")["tokens"]
    r = bild.generate(S, L, ids, 0.0, INF, 10, mode="small", eos_id=ref[4])
    assert r["tokens"] == ref[:5]


# ---- sampling variant (supplementary material, "BiLD with Sampling") -----------------------
def test_nucleus_sample_against_its_definition():
    """Small vocabularies, every decision by brute force: the nucleus is the shortest prefix of the tokens sorted by
    decreasing probability (ties: lower index) with mass >= top_p; over a fine grid of u the tokens come out with
    frequencies proportional to their probabilities inside the nucleus and never from outside it."""
    rng = np.random.default_rng(3)
    for V, top_p in [(5, 0.8), (17, 0.8), (64, 0.5), (64, 1.0), (9, 0.95)]:
        z = rng.normal(size=V) * 2
        z[3] = z[1]                                    # a tie, resolved by index
        p = np.exp(z) / np.exp(z).sum()
        ranked = sorted(range(V), key=lambda i: (-p[i], i))
        mass, keep = 0.0, []
        for i in ranked:                               # plain loop: add tokens until the mass reaches top_p
            keep.append(i); mass += p[i]
            if mass >= top_p:
                break
        assert mass - p[keep[-1]] < top_p <= mass or len(keep) == V
        N = 20000
        counts = np.zeros(V)
        for j in range(N):
            tok, n, _ = bild.nucleus_sample(z, top_p, (j + 0.5) / N)
            assert n == len(keep) and tok in keep
            counts[tok] += 1
        for i in range(V):                             # the u's that give token i form one interval of length p_i / mass
            want = N * p[i] / mass if i in keep else 0.0
            assert abs(counts[i] - want) <= 1.0 + 1e-9, (V, top_p, i)
    # u = 0 gives the most probable token; top_p -> 0 keeps only that token
    z = rng.normal(size=40)
    assert bild.nucleus_sample(z, 0.8, 0.0)[0] == int(np.argmax(z))
    assert all(bild.nucleus_sample(z, 1e-12, u)[:2] == (int(np.argmax(z)), 1) for u in (0.0, 0.3, 0.999999))


def test_sampling_with_a_vanishing_nucleus_is_greedy(pair):
    wl, S, L, ids = pair
    uS, uL = gen_uniforms(wl.gen_len + 2, 1, "small"), gen_uniforms(wl.gen_len + 2, 1, "large")
    ref = bild.generate(S, L, ids, 0.3, 16.0, wl.gen_len, max_draft=5)
    got = bild.generate(S, L, ids, 0.3, 16.0, wl.gen_len, max_draft=5, top_p=1e-12, u_small=uS, u_large=uL)
    assert got["tokens"] == ref["tokens"] and got["trace"] == ref["trace"] and got["stats"] == ref["stats"]


@pytest.mark.parametrize("alpha_fb,alpha_rb,max_draft", [(0.3, 16.0, 10), (0.5, 14.0, 4), (0.0, 15.0, 3)])
def test_certificate_of_a_sampled_run(pair, alpha_fb, alpha_rb, max_draft):
    """Sampling changes how tokens are drawn and nothing else: recomputed from scratch on the final sequence, every token
    the trace attributes to the small model is the nucleus draw from p_S with that position's number and passed the
    fallback test; every large-model token is the nucleus draw from p_L with the large model's number of that position."""
    wl, S, L, ids = pair
    n = wl.gen_len
    uS, uL = gen_uniforms(n + 2, 2, "small"), gen_uniforms(n + 2, 2, "large")
    r = bild.generate(S, L, ids, alpha_fb, alpha_rb, n, max_draft=max_draft, top_p=0.8, u_small=uS, u_large=uL)
    y = [0] + r["tokens"]
    assert len(r["trace_margins"]) == len(r["trace"]) and all(len(t) == 4 for t in r["trace_margins"])
    ZS = S.forward_full(S.start(ids, len(y)), y[:-1])
    ZL = L.forward_full(L.start(ids, len(y)), y[:-1])
    owner = {}
    for kind, pos, tok, k, m, val in r["trace"]:
        if kind == bild.KIND_SMALL_ACCEPT:
            owner[pos] = "S"
        elif kind in (bild.KIND_VERIFY_OK, bild.KIND_ROLLBACK):
            for q in [q for q in owner if q > pos]:
                del owner[q]
            owner[pos] = "L"
    assert sorted(owner) == list(range(1, n + 1))
    for j in range(1, len(y)):
        if owner[j] == "S":
            assert y[j] == bild.nucleus_sample(ZS[j - 1], 0.8, float(uS[j]))[0]
            assert bild.max_prob(ZS[j - 1])[1] >= alpha_fb
        else:
            assert y[j] == bild.nucleus_sample(ZL[j - 1], 0.8, float(uL[j]))[0]
    assert any(bild.max_prob(ZS[j - 1])[0] != y[j] for j in range(1, len(y)) if owner[j] == "S") or alpha_fb > 0.45
    assert r["tokens"] != bild.generate(S, L, ids, alpha_fb, alpha_rb, n, max_draft=max_draft)["tokens"]


# ---- early-exit configuration (Section 4.4) -------------------------------------------------
def test_early_exit_model_is_the_prefix_of_the_decoder(pair):
    """The early-exit small model shares everything with the large model and stops after its first layers: exiting
    after the last layer is the model itself; exiting after layer 1 equals the full model whose later layers are
    made the identity (their three output matrices set to zero)."""
    wl, S, L, ids = pair
    toks = [0, 5, 9, 3, 7]
    full = L.forward_block(L.start(ids, 8), toks)
    same = L.early_exit(L.s.n_layers)
    assert np.array_equal(same.forward_block(same.start(ids, 8), toks), full)
    t = gen_model(MODEL_SHAPES[wl.large], wl.seed, wl.dtype)
    for l in range(1, L.s.n_layers):
        for name in ("wo", "wco", "wfo"):
            t[f"dec.{l}.{name}"] = np.zeros_like(t[f"dec.{l}.{name}"])
    ident = Model(MODEL_SHAPES[wl.large], t, L.logit_scale)
    e1 = L.early_exit(1)
    z1 = e1.forward_block(e1.start(ids, 8), toks)
    assert np.max(np.abs(z1 - ident.forward_block(ident.start(ids, 8), toks))) < 1e-10
    assert np.max(np.abs(z1 - full)) > 1e-2                      # and it is not the full model
    assert np.max(np.abs(e1.forward_full(e1.start(ids, 8), toks) - z1)) < 1e-10


def test_bild_with_an_early_exit_draft_model(pair):
    """Algorithm 1 with the small model = first layer of the large one: with the exit after the LAST layer the drafts
    are the large model's own tokens, so nothing is ever rolled back for alpha_RB above their distances and the output
    is the large model's greedy decode; with the exit after layer 1 the certificate of finished runs still holds."""
    wl, S, L, ids = pair
    ref = bild.generate(S, L, ids, 0.0, INF, wl.gen_len, mode="large")
    same = L.early_exit(L.s.n_layers)
    got = bild.generate(same, L, ids, 0.3, 50.0, wl.gen_len, max_draft=4)
    assert got["tokens"] == ref["tokens"] and got["stats"]["rollbacks"] == 0
    e1 = L.early_exit(1, logit_scale=2.0 * L.logit_scale)
    r = bild.generate(e1, L, ids, 0.3, 16.0, wl.gen_len, max_draft=4)
    y = [0] + r["tokens"]
    ZS = e1.forward_full(e1.start(ids, len(y)), y[:-1])
    ZL = L.forward_full(L.start(ids, len(y)), y[:-1])
    owner = {}
    for kind, pos, tok, k, m, val in r["trace"]:
        if kind == bild.KIND_SMALL_ACCEPT:
            owner[pos] = "S"
        elif kind in (bild.KIND_VERIFY_OK, bild.KIND_ROLLBACK):
            for q in [q for q in owner if q > pos]:
                del owner[q]
            owner[pos] = "L"
    for j in range(1, len(y)):
        assert y[j] == int(np.argmax(ZS[j - 1] if owner[j] == "S" else ZL[j - 1]))
    assert r["stats"]["small_steps"] > 0 and r["stats"]["large_calls"] > 0


# ---- closed forms --------------------------------------------------------------
def test_softmax_identities():
    rng = np.random.default_rng(0)
    z = rng.normal(size=300) * 4
    t, pmax, lse, gap = bild.max_prob(z)
    p = np.exp(z) / np.exp(z).sum()
    assert abs(p.sum() - 1) < 1e-12 and t == int(np.argmax(p))
    assert abs(pmax - p.max()) < 1e-14
    assert abs(lse - math.log(np.exp(z).sum())) < 1e-12
    assert all(lse - z >= 0)
    srt = np.sort(z)
    assert abs(gap - (srt[-1] - srt[-2])) < 1e-14
    onehot = np.full(10, -1e4); onehot[3] = 0.0
    assert bild.max_prob(onehot)[1] == 1.0 and bild.max_prob(onehot)[2] == 0.0
    assert bild.max_prob(np.array([1.0, 2.0, 2.0, 0.0]))[0] == 1     # lowest index on ties


def test_block_closed_forms():
    d = 24
    g = np.linspace(0.5, 1.5, d)
    assert np.allclose(rms_norm(np.ones(d), g, 1e-6), g / math.sqrt(1 + 1e-6), atol=1e-15)
    x = np.arange(1, d + 1, dtype=float)
    assert np.allclose(rms_norm(x, np.ones(d), 0.0), x / math.sqrt(np.mean(x ** 2)))
    V = np.arange(12.0).reshape(3, 4)
    q = np.array([1.0, -2.0, 0.5, 3.0])
    assert np.allclose(attend(q, V[:1], V[:1] + 5), V[0] + 5)                 # one key
    assert np.allclose(attend(q, np.tile(q, (3, 1)), V), V.mean(axis=0))      # equal keys
    assert np.allclose(attend(q, np.zeros((3, 4)), V, np.array([0.0, 50.0, 0.0])), V[1], atol=1e-9)
    assert gelu_tanh(np.array([0.0]))[0] == 0.0
    assert abs(gelu_tanh(np.array([30.0]))[0] - 30.0) < 1e-12
    assert abs(gelu_tanh(np.array([-30.0]))[0]) < 1e-12
    # Taylor: gelu(u) ~ u/2 + u^2 * sqrt(2/pi)/2 near 0
    u = 1e-4
    assert abs(gelu_tanh(np.array([u]))[0] - (u / 2 + u * u * math.sqrt(2 / math.pi) / 2)) < 1e-15


def test_bucket_tables():
    for delta in range(16):
        assert decoder_bucket(delta) == delta
    tab = [decoder_bucket(i) for i in range(400)]
    assert all(b2 >= b1 for b1, b2 in zip(tab, tab[1:]))
    # last boundary is 16 * 8^(15/16) = 112.4
    assert tab[112] == 30 and all(b == 31 for b in tab[113:])
    assert set(tab) == set(range(32))
    for delta in range(16, 128):          # log form; no integer hits a boundary here
        assert decoder_bucket(delta) == 16 + int(math.floor(16 * math.log(delta / 16) / math.log(8)))
    # bidirectional: exact at |rel| = 16, 32, 64 where 8 * 16^(j/8) is an integer
    assert [encoder_bucket(-r) for r in (8, 16, 32, 64, 128, 500)] == [8, 10, 12, 14, 15, 15]
    assert [encoder_bucket(-r) for r in (15, 31, 63, 127)] == [9, 11, 13, 15]
    for r in range(1, 300):
        assert encoder_bucket(r) == encoder_bucket(-r) + 16
        if r < 8:
            assert encoder_bucket(-r) == r
    assert encoder_bucket(0) == 0
    for r in (9, 11, 13, 20, 45, 90, 100):
        assert encoder_bucket(-r) == 8 + int(math.floor(8 * math.log(r / 8) / math.log(16)))


# ---- library routines ----------------------------------------------------------
def test_blocks_against_torch_fp64():
    rng = np.random.default_rng(1)
    x = rng.normal(size=(5, 48)); g = rng.normal(size=48)
    ref = torch.nn.functional.rms_norm(torch.tensor(x), (48,), torch.tensor(g), eps=1e-6).numpy()
    assert np.max(np.abs(rms_norm(x, g, 1e-6) - ref)) < 1e-13
    u = rng.normal(size=100) * 3
    ref = torch.nn.functional.gelu(torch.tensor(u), approximate="tanh").numpy()
    assert np.max(np.abs(gelu_tanh(u) - ref)) < 1e-13
    q = rng.normal(size=16); K = rng.normal(size=(9, 16)); V = rng.normal(size=(9, 16)); b = rng.normal(size=9)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(q)[None, None], torch.tensor(K)[None], torch.tensor(V)[None],
        attn_mask=torch.tensor(b)[None, None], scale=1.0)[0, 0].numpy()
    assert np.max(np.abs(attend(q, K, V, b) - ref)) < 1e-13
    ref = torch.softmax(torch.tensor(u), 0).numpy()
    assert np.max(np.abs(softmax(u) - ref)) < 1e-15


@pytest.mark.parametrize("shape_name", ["tiny_s", "odd_l"])
def test_whole_model_against_library_t5(shape_name):
    """Build the installed transformers T5 from a config (no checkpoint), load
    the synthetic weights, and compare encoder memory and teacher-forced decoder
    logits in fp64.  Pins the architecture reading (norm, no attention scaling,
    bucketed bias shared across layers, GELU flavour)."""
    from transformers import T5Config, T5ForConditionalGeneration
    # this library version always shares the LM head with the embedding table (and,
    # given tie_word_embeddings=False, applies no output scaling), so compare a
    # tied-head variant of the shape with logit_scale 1
    s = dataclasses.replace(MODEL_SHAPES[shape_name], tied_head=True)
    w = gen_model(s, 3, "fp32")
    w["emb"] = w["emb"] * np.float32(0.05)     # keeps tied-head logits O(1)
    m = Model(s, w, logit_scale=1.0)
    cfg = T5Config(vocab_size=s.vocab, d_model=s.d_model, d_kv=s.d_kv, d_ff=s.d_ff, num_layers=s.n_layers,
                   num_decoder_layers=s.n_layers, num_heads=s.n_heads,
                   relative_attention_num_buckets=s.rel_buckets, relative_attention_max_distance=s.rel_max_dist,
                   dropout_rate=0.0, layer_norm_epsilon=s.eps,
                   feed_forward_proj="relu" if s.ffn == "relu" else "gated-gelu",
                   tie_word_embeddings=False, decoder_start_token_id=0, pad_token_id=0)
    hf = T5ForConditionalGeneration(cfg).double().eval()
    sd = {}
    T = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))
    I = s.inner
    for name in ("shared.weight", "encoder.embed_tokens.weight", "decoder.embed_tokens.weight", "lm_head.weight"):
        sd[name] = T(w["emb"])
    for stack, hs in (("enc", "encoder"), ("dec", "decoder")):
        sd[f"{hs}.final_layer_norm.weight"] = T(w[f"{stack}.final_ln"])
        sd[f"{hs}.block.0.layer.0.SelfAttention.relative_attention_bias.weight"] = T(w[f"{stack}.rel_bias"])
        for l in range(s.n_layers):
            p, b = f"{stack}.{l}.", f"{hs}.block.{l}.layer."
            qkv = w[p + "wqkv"]
            for i, n in enumerate("qkv"):
                sd[b + f"0.SelfAttention.{n}.weight"] = T(qkv[i * I:(i + 1) * I])
            sd[b + "0.SelfAttention.o.weight"] = T(w[p + "wo"])
            sd[b + "0.layer_norm.weight"] = T(w[p + "ln1"])
            f = 1
            if stack == "dec":
                sd[b + "1.EncDecAttention.q.weight"] = T(w[p + "wcq"])
                sd[b + "1.EncDecAttention.k.weight"] = T(w[p + "wckv"][:I])
                sd[b + "1.EncDecAttention.v.weight"] = T(w[p + "wckv"][I:])
                sd[b + "1.EncDecAttention.o.weight"] = T(w[p + "wco"])
                sd[b + "1.layer_norm.weight"] = T(w[p + "ln2"])
                sd[b + "2.layer_norm.weight"] = T(w[p + "ln3"])
                f = 2
            else:
                sd[b + "1.layer_norm.weight"] = T(w[p + "ln2"])
            if s.ffn == "relu":
                sd[b + f"{f}.DenseReluDense.wi.weight"] = T(w[p + "wi0"])
            else:
                sd[b + f"{f}.DenseReluDense.wi_0.weight"] = T(w[p + "wi0"])
                sd[b + f"{f}.DenseReluDense.wi_1.weight"] = T(w[p + "wi1"])
            sd[b + f"{f}.DenseReluDense.wo.weight"] = T(w[p + "wfo"])
    own = dict(hf.state_dict())
    sd = {k: v for k, v in sd.items() if k in own}
    assert {k for k in own if "embed_tokens" not in k and k != "lm_head.weight"} <= set(sd)
    hf.load_state_dict(sd, strict=False)
    ids = gen_ids(s.vocab, 40, 3)       # long enough to reach log-spaced buckets on both sides
    dec = [0] + [int(t) for t in gen_ids(s.vocab, 37, 4)]
    with torch.no_grad():
        out = hf(input_ids=torch.tensor(ids, dtype=torch.long)[None],
                 decoder_input_ids=torch.tensor(dec, dtype=torch.long)[None])
    mem = m.encode(ids)
    # the library's norm takes its mean of squares in fp32 even in a double model,
    # which leaves ~1e-7 of noise; an architectural difference would be >= 1e-2
    assert np.max(np.abs(mem - out.encoder_last_hidden_state[0].numpy())) < 1e-5
    st = m.start(ids, 64)
    Z = np.concatenate([m.forward_block(st, dec[:20]), m.forward_block(st, dec[20:])])
    assert np.max(np.abs(Z)) > 0.5
    assert np.max(np.abs(Z - out.logits[0].numpy())) < 1e-5


# ---- the tests can see every component -----------------------------------------
@pytest.mark.parametrize("mutation", ["dec.rel_bias", "enc.rel_bias", "dec.1.ln1", "dec.0.ln2", "dec.1.ln3",
                                      "dec.final_ln", "enc.final_ln", "dec.0.wo", "dec.1.wco", "dec.0.wfo",
                                      "enc.0.wo", "enc.1.wfo"])
def test_mutations_move_logits(mutation):
    """Neutralising any one component (bias table -> 0, gain -> 1, a residual
    branch -> 0) moves the logits by at least ten times the 1e-4 parity
    tolerance of the fp32 configuration (the unit-variance embedding dominates
    the residual stream, so single sub-layers move logits by 1e-3 .. 1e-1)."""
    s = MODEL_SHAPES["tiny_l"]
    w = gen_model(s, 0, "fp32")
    ids = gen_ids(s.vocab, 32, 0)
    toks = [0, 5, 9, 200, 31, 77, 8, 300, 12, 44, 101, 19, 23, 29, 31, 37, 41, 43, 47, 53]
    base = Model(s, w, 15.0)
    z0 = base.forward_block(base.start(ids, 32), toks)
    w2 = dict(w)
    if "rel_bias" in mutation or mutation.split(".")[-1].startswith("w"):
        w2[mutation] = np.zeros_like(w[mutation])
    else:
        w2[mutation] = np.ones_like(w[mutation])
    mut = Model(s, w2, 15.0)
    z1 = mut.forward_block(mut.start(ids, 32), toks)
    assert np.max(np.abs(z1 - z0)) > 1e-3
