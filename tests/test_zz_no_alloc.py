"""bild_op_lm_head_static against bild_op_lm_head.

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
    # sizes beyond the built-in scratch are refused, not truncated
    Wd, X, g, t = _case(torch, 9, 1, 64, 8, False)
    with pytest.raises(BildError) as e:
        op_lm_head_static(Wd, X, g, 1e-6, 1.0, t, 1, (1 << 20) + 1, 8)
    assert e.value.code == -4
    with pytest.raises(BildError):
        op_lm_head_static(Wd, X, g, 1e-6, 1.0, t, 17, 64, 8)
