"""The allocation-free split-K entry point (collected last on purpose: a run that stops at the first
failure has then already run every other test).

trdq_linear_splitk_static is for callers that cannot allocate device memory at the call site, such as a
server whose memory pool already owns the whole GPU.  It must give exactly what trdq_linear_splitk gives
with a caller workspace, on repeated calls that reuse the library's built-in scratch array, and it must
refuse problems that do not fit that array.
"""
import numpy as np
import pytest

from paper_2503_06564_b200 import workloads as WL
from tests.util import to_dev_bf16

pytestmark = pytest.mark.gpu


def _layer(N, K, seed):
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(seed)
    signs = (rng.integers(0, 2, (2, K)) * 2 - 1).astype(np.int8)
    smooth = rng.uniform(0.5, 2.0, (2, K)).astype(np.float32)
    rot = trdq.Rotation(K, [0, 500, 1000], signs, smooth)
    w = WL.to_bf16_bits(rng.standard_normal((N, K)) * 0.02)
    bias = WL.to_bf16_bits(rng.standard_normal(N) * 0.01)
    return rot, trdq.trdq_prepare_weights(rot, to_dev_bf16(w), 8), to_dev_bf16(bias)


def _codes(rot, t, M, K, seed):
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, K))
    x[:, rng.choice(K, K // 100, replace=False)] *= 30.0
    return trdq.trdq_rotate_quantize(rot, t, to_dev_bf16(WL.to_bf16_bits(x)))


def test_static_scratch_matches_workspace_version_on_consecutive_calls():
    import torch
    from paper_2503_06564_b200 import trdq
    N, K = 1152, 8192
    rot, wts, bias = _layer(N, K, 7)
    # first call: 200 rows; second call: other data and FEWER rows, so stale partial sums of the first call
    # sit in the scratch array right where (and beyond where) the second call works
    free_after_first = None
    for call, (M, t) in enumerate([(200, 100), (96, 900)]):
        codes, scales = _codes(rot, t, M, K, 40 + call)
        splits, nbytes = trdq.trdq_linear_splitk_workspace(wts, M)
        assert splits > 1 and splits * M * N <= trdq.STATIC_SCRATCH_ELEMS
        expected = trdq.trdq_linear_splitk(wts, t, codes, scales, bias)         # caller-allocated workspace
        out = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        trdq.trdq_linear_splitk_static(wts, t, codes, scales, bias, out)
        torch.cuda.synchronize()
        free_after = torch.cuda.mem_get_info()[0]
        assert torch.equal(out, expected)                                        # integer partial sums: bit-identical
        # The built-in array is part of the library's GEMM module and is reserved when that module is first used on the
        # device (trdq_prepare_weights above already did); from then on no call, not even the first one, which looks
        # up the array's address, changes the device's free memory.
        assert free_after == free_before
        if call == 0:
            free_after_first = free_after
        else:
            assert free_after == free_after_first
    assert trdq.trdq_device_status() == 0


def test_static_scratch_refuses_what_does_not_fit():
    import torch
    from paper_2503_06564_b200 import trdq
    N, K = 1152, 8192
    rot, wts, bias = _layer(N, K, 9)
    M = 1000                                   # 8 x 9 tiles, two k ranges: 2 * 1000 * 1152 > 2 Mi elements
    codes, scales = _codes(rot, 0, M, K, 3)
    splits, _ = trdq.trdq_linear_splitk_workspace(wts, M)
    assert splits > 1 and splits * M * N > trdq.STATIC_SCRATCH_ELEMS
    out = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_linear_splitk_static(wts, 0, codes, scales, bias, out)
    assert e.value.status == 11
    assert not out.any().item()                # nothing was launched
    # a shape for which split-K does not pay needs no scratch at all and simply runs the ordinary linear
    rot2, wts2, bias2 = _layer(1152, 1152, 11)
    c2, s2 = _codes(rot2, 0, 300, 1152, 5)
    out2 = torch.empty((300, 1152), dtype=torch.bfloat16, device="cuda")
    trdq.trdq_linear_splitk_static(wts2, 0, c2, s2, bias2, out2)
    assert torch.equal(out2, trdq.trdq_linear(wts2, 0, c2, s2, bias2))
