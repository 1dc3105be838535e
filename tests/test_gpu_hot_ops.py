"""GPU parity of the hot kernels of the bf16 decoder passes, one operation at a time, against plain fp64 numpy
at the shapes of the paper's models (Table of model sizes in the supplementary material): the fused attention
sub-layer (self and cross), the fused feed-forward sub-layer (ReLU and gated GELU), and the tensor-core LM head
over the whole vocabulary.  Every output element is compared."""
import numpy as np
import pytest

from oracle.t5 import gelu_tanh, rms_norm
from workloads import bf16_bits_to_f32, bf16_round_bits

pytestmark = pytest.mark.gpu


def _bf16(torch, rng, shape, scale):
    w = (rng.standard_normal(shape) * scale).astype(np.float32)
    bits = bf16_round_bits(w)
    return bf16_bits_to_f32(bits).astype(np.float64), torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("M", [1, 2, 5, 8])
@pytest.mark.parametrize("d,F,gated,parts", [(1024, 4096, False, 0), (1024, 2816, True, 0), (512, 2048, False, 0),
                                             (512, 1024, True, 2), (128, 264, False, 0)])
def test_ffn_sublayer_matches_numpy(M, d, F, gated, parts):
    import torch
    from paper_2302_07863_b200.binding import op_ffn_sublayer
    rng = np.random.default_rng(M * 7 + d + F)
    Wi0, Wi0d = _bf16(torch, rng, (F, d), 0.03)
    Wi1, Wi1d = _bf16(torch, rng, (F, d), 0.03) if gated else (None, None)
    Wfo, Wfod = _bf16(torch, rng, (d, F), 0.03)
    g = (1 + 0.1 * rng.standard_normal(d)).astype(np.float32)
    x = (rng.standard_normal((M, d)) * 2).astype(np.float32)
    h = rms_norm(x.astype(np.float64), g.astype(np.float64), 1e-6)
    u = gelu_tanh(h @ Wi0.T) * (h @ Wi1.T) if gated else np.maximum(h @ Wi0.T, 0.0)
    ref = x.astype(np.float64) + u @ Wfo.T
    got = op_ffn_sublayer(Wi0d, Wi1d, Wfod, torch.from_numpy(g).cuda(), 1e-6, torch.from_numpy(x).cuda(), M, d, F, parts)
    err = float(np.max(np.abs(got.cpu().numpy() - ref)))
    assert err <= 5e-5 * max(1.0, float(np.max(np.abs(ref)))), err


def _ref_attention(self_attn, x, g, Wp, Wo, K, V, n_before, bias, H, dkv):
    """x + W_o Attention(rms_norm(x)) written out per head; returns (output, new keys, new values)."""
    M, d = x.shape
    I = H * dkv
    h = rms_norm(x, g, 1e-6)
    proj = h @ Wp.T
    q = proj[:, :I]
    out = np.zeros((M, I))
    knew = vnew = None
    if self_attn:
        knew, vnew = proj[:, I:2 * I], proj[:, 2 * I:]
    for hd in range(H):
        sl = slice(hd * dkv, (hd + 1) * dkv)
        for m in range(M):
            if self_attn:
                keys = np.concatenate([K[hd, :n_before], knew[:m + 1, sl]])
                vals = np.concatenate([V[hd, :n_before], vnew[:m + 1, sl]])
                b = np.array([bias[hd, n_before + m - j] for j in range(n_before + m + 1)])
            else:
                keys, vals, b = K[hd, :n_before], V[hd, :n_before], 0.0
            s = keys @ q[m, sl] + b
            p = np.exp(s - s.max())
            out[m, sl] = (p / p.sum()) @ vals
    return x + out @ Wo.T, knew, vnew


@pytest.mark.parametrize("M", [1, 3, 8])
@pytest.mark.parametrize("self_attn,d,H,dkv,cap,n_before", [
    (True, 1024, 16, 64, 81, 0), (True, 1024, 16, 64, 81, 64), (True, 1024, 16, 64, 1040, 1000),
    (False, 1024, 16, 64, 512, 512), (False, 1024, 16, 64, 1024, 1000), (False, 512, 8, 64, 512, 512),
    (True, 512, 6, 64, 300, 257), (False, 512, 6, 64, 64, 64), (True, 128, 4, 32, 40, 7), (False, 64, 4, 16, 32, 19),
    # around the key count up to which every block of a head attends over all keys (one staged chunk)
    (True, 1024, 16, 64, 200, 72), (True, 1024, 16, 64, 200, 75), (True, 512, 8, 64, 257, 100), (False, 1024, 16, 64, 96, 70)])
def test_attention_sublayer_matches_numpy(M, self_attn, d, H, dkv, cap, n_before):
    import torch
    from paper_2302_07863_b200.binding import op_attn_sublayer
    rng = np.random.default_rng(M + d + H + cap + n_before)
    I = H * dkv
    Wp, Wpd = _bf16(torch, rng, ((3 if self_attn else 1) * I, d), 0.03)
    Wo, Wod = _bf16(torch, rng, (d, I), 0.03)
    g = (1 + 0.1 * rng.standard_normal(d)).astype(np.float32)
    x = (rng.standard_normal((M, d)) * 2).astype(np.float32)
    K = rng.standard_normal((H, cap, dkv)).astype(np.float32)
    V = rng.standard_normal((H, cap, dkv)).astype(np.float32)
    bias = rng.standard_normal((H, cap)).astype(np.float32) if self_attn else None
    ref, knew, vnew = _ref_attention(self_attn, x.astype(np.float64), g.astype(np.float64), Wp, Wo, K.astype(np.float64),
                                     V.astype(np.float64), n_before, bias, H, dkv)
    Kd, Vd = torch.from_numpy(K).cuda(), torch.from_numpy(V).cuda()
    got = op_attn_sublayer(self_attn, Wpd, Wod, torch.from_numpy(g).cuda(), 1e-6, torch.from_numpy(x).cuda(), Kd, Vd, cap,
                           n_before, torch.from_numpy(bias).cuda() if self_attn else None, M, d, H, dkv)
    err = float(np.max(np.abs(got.cpu().numpy() - ref)))
    assert err <= 5e-5 * max(1.0, float(np.max(np.abs(ref)))), err
    if self_attn:   # the rows appended to the cache, and nothing else touched
        Kg, Vg = Kd.cpu().numpy(), Vd.cpu().numpy()
        for hd in range(H):
            sl = slice(hd * dkv, (hd + 1) * dkv)
            assert np.max(np.abs(Kg[hd, n_before:n_before + M] - knew[:, sl])) <= 2e-5 * max(1.0, np.max(np.abs(knew)))
            assert np.max(np.abs(Vg[hd, n_before:n_before + M] - vnew[:, sl])) <= 2e-5 * max(1.0, np.max(np.abs(vnew)))
        assert np.array_equal(Kg[:, :n_before], K[:, :n_before]) and np.array_equal(Kg[:, n_before + M:], K[:, n_before + M:])


@pytest.mark.parametrize("M,V,K", [(1, 32128, 1024), (5, 32128, 1024), (16, 32128, 1024), (1, 250112, 512), (1, 250112, 1024),
                                   (5, 250112, 1024), (16, 250112, 1024), (3, 773, 64)])
def test_sliced_head_matches_numpy_over_the_whole_vocabulary(M, V, K):
    """All V logits of every row (debug dump), arg-max, max, log-sum-exp and gathered logit against fp64."""
    import torch
    from paper_2302_07863_b200.binding import op_lm_head_sliced
    rng = np.random.default_rng(V + K + M)
    W, Wd = _bf16(torch, rng, (V, K), 0.05)
    X = rng.standard_normal((M, K)).astype(np.float32)
    g = (1 + 0.1 * rng.standard_normal(K)).astype(np.float32)
    tgt = rng.integers(0, V, M).astype(np.int32)
    scale = 9.0
    Z = scale * (rms_norm(X.astype(np.float64), g.astype(np.float64), 1e-6) @ W.T)
    am, mx, lse, ga, lg = op_lm_head_sliced(Wd, torch.from_numpy(X).cuda(), torch.from_numpy(g).cuda(), 1e-6, scale,
                                            torch.from_numpy(tgt).cuda(), M, V, K, want_logits=True)
    torch.cuda.synchronize()
    assert np.max(np.abs(lg.cpu().numpy() - Z)) <= 2e-4          # every logit: a dropped tile or row would show here
    for m in range(M):
        srt = np.sort(Z[m])
        if srt[-1] - srt[-2] > 1e-3:
            assert int(am[m]) == int(np.argmax(Z[m]))
        zmax = Z[m].max()
        assert abs(float(mx[m]) - zmax) <= 2e-4
        assert abs(float(lse[m]) - (zmax + np.log(np.exp(Z[m] - zmax).sum()))) <= 2e-4
        assert abs(float(ga[m]) - Z[m][tgt[m]]) <= 2e-4


@pytest.mark.parametrize("V,K", [(32128, 512), (32128, 1024), (250112, 512), (250112, 1024), (1001, 264), (40, 64), (5000, 256)])
def test_streaming_head_matches_numpy_over_the_whole_vocabulary(V, K):
    """The single-row streaming head: all V logits (debug dump), arg-max, max, log-sum-exp and gathered logit against
    fp64; vocabularies that do not fill the grid or the last batch of a warp included."""
    import torch
    from paper_2302_07863_b200.binding import op_lm_head_stream
    rng = np.random.default_rng(V + K)
    W, Wd = _bf16(torch, rng, (V, K), 0.05)
    X = rng.standard_normal((1, K)).astype(np.float32)
    g = (1 + 0.1 * rng.standard_normal(K)).astype(np.float32)
    tgt = rng.integers(0, V, 1).astype(np.int32)
    scale = 9.0
    Z = scale * (rms_norm(X.astype(np.float64), g.astype(np.float64), 1e-6) @ W.T)
    am, mx, lse, ga, lg = op_lm_head_stream(Wd, torch.from_numpy(X).cuda(), torch.from_numpy(g).cuda(), 1e-6, scale,
                                            torch.from_numpy(tgt).cuda(), V, K, want_logits=True)
    torch.cuda.synchronize()
    assert np.max(np.abs(lg.cpu().numpy() - Z)) <= 2e-4          # every logit: a skipped row or batch would show here
    srt = np.sort(Z[0])
    if srt[-1] - srt[-2] > 1e-3:
        assert int(am[0]) == int(np.argmax(Z[0]))
    zmax = Z[0].max()
    assert abs(float(mx[0]) - zmax) <= 2e-4
    assert abs(float(lse[0]) - (zmax + np.log(np.exp(Z[0] - zmax).sum()))) <= 2e-4
    assert abs(float(ga[0]) - Z[0][tgt[0]]) <= 2e-4
