"""bild_op_lm_head_static against bild_op_lm_head and against a plain fp64 computation.

The static variant serves callers that cannot allocate device memory for the kernel's
scratch - a worker inside a serving process whose allocator already owns the GPU, or a
latency-critical loop that must avoid cudaMalloc's device-wide synchronisation - by keeping
that scratch in a fixed array inside the library.  Because the array is shared by every
call and keeps the previous call's contents, the check is made on two different calls in a
row: the second must not see anything of the first.  Collected last on purpose."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _case(torch, seed, M, V, K, bf16):
    from workloads import bf16_bits_to_f32, bf16_round_bits
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((V, K)) * 0.05).astype(np.float32)
    if bf16:
        bits = bf16_round_bits(W)
        Wd = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    else:
        Wd = torch.from_numpy(W).cuda()
    X = torch.from_numpy(rng.standard_normal((M, K)).astype(np.float32)).cuda()
    g = torch.from_numpy((1 + 0.1 * rng.standard_normal(K)).astype(np.float32)).cuda()
    t = torch.from_numpy(rng.integers(0, V, M).astype(np.int32)).cuda()
    return Wd, X, g, t


def _plain(Wd, X, g, t, scale, eps, bf16):
    """The head written out in fp64: rms-norm, scaled logits, arg-max, max, log-sum-exp, gathered logit."""
    W = (Wd.float() if bf16 else Wd).cpu().numpy().astype(np.float64)
    x = X.cpu().numpy().astype(np.float64)
    h = x / np.sqrt((x * x).mean(axis=1, keepdims=True) + eps) * g.cpu().numpy().astype(np.float64)
    z = scale * (h @ W.T)
    zmax = z.max(axis=1)
    lse = zmax + np.log(np.exp(z - zmax[:, None]).sum(axis=1))
    srt = np.sort(z, axis=1)
    return z.argmax(axis=1), zmax, lse, z[np.arange(len(z)), t.cpu().numpy()], srt[:, -1] - srt[:, -2]


def test_static_scratch_head_matches_regular_head_twice_in_a_row():
    import torch
    assert torch.cuda.is_available()
    from paper_2302_07863_b200 import BildError
    from paper_2302_07863_b200.binding import op_lm_head, op_lm_head_static
    # two calls in a row with different shapes, rows and weight types
    for seed, (M, V, K, bf16) in enumerate([(16, 40013, 512, True), (1, 32128, 1024, False), (5, 773, 64, True)]):
        Wd, X, g, t = _case(torch, seed, M, V, K, bf16)
        ref = op_lm_head(Wd, X, g, 1e-6, 7.0, t, M, V, K)
        got = op_lm_head_static(Wd, X, g, 1e-6, 7.0, t, M, V, K)
        torch.cuda.synchronize()
        assert got[0].tolist() == ref[0].tolist()                       # arg-max
        for a, b in zip(got[1:], ref[1:4]):                             # max, lse, gathered logit
            assert float((a - b).abs().max()) <= 1e-4
        am, zmax, lse, gat, gap = _plain(Wd, X, g, t, 7.0, 1e-6, bf16)   # and an independent computation
        for m in range(M):
            if gap[m] > 1e-3:
                assert int(got[0][m]) == int(am[m])
        for a, b in zip(got[1:], (zmax, lse, gat)):
            assert float(np.abs(a.cpu().numpy().astype(np.float64) - b).max()) <= 1e-4
    # sizes beyond the built-in scratch are refused, not truncated
    Wd, X, g, t = _case(torch, 9, 1, 64, 8, False)
    with pytest.raises(BildError) as e:
        op_lm_head_static(Wd, X, g, 1e-6, 1.0, t, 1, (1 << 20) + 1, 8)
    assert e.value.code == -4
    with pytest.raises(BildError):
        op_lm_head_static(Wd, X, g, 1e-6, 1.0, t, 17, 64, 8)
    # two or more rows of 4096 columns: the staged rows exceed a block's shared memory -> capacity, not a CUDA error
    Wd, X, g, t = _case(torch, 10, 2, 64, 4096, True)
    for fn, extra in ((op_lm_head_static, ()), (op_lm_head, ())):
        with pytest.raises(BildError) as e:
            fn(Wd, X, g, 1e-6, 1.0, t, 2, 64, 4096)
        assert e.value.code == -4
    # and the context is unharmed: a call that fits still gives the right answer
    Wd, X, g, t = _case(torch, 11, 2, 300, 64, False)
    got = op_lm_head_static(Wd, X, g, 1e-6, 3.0, t, 2, 300, 64)
    torch.cuda.synchronize()
    am, zmax, lse, gat, gap = _plain(Wd, X, g, t, 3.0, 1e-6, False)
    assert float(np.abs(got[2].cpu().numpy() - lse).max()) <= 1e-4
