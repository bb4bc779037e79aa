"""GPU parity: INT8 tcgen05 GEMM (raw accumulators and dequantizing epilogue) against the CPU oracle."""
import numpy as np
import pytest

from oracle import trdq_oracle as O
from paper_2503_06564_b200 import workloads as WL
from tests.util import bf16_to_f32_np, check_output, to_dev_bf16

pytestmark = pytest.mark.gpu


def _setup(N, K, G, seed, wbits=8):
    """A prepared layer on the device plus the oracle's own codes for every group."""
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(seed)
    signs = (rng.integers(0, 2, (G, K)) * 2 - 1).astype(np.int8)
    smooth = rng.uniform(0.5, 2.0, (G, K)).astype(np.float32)
    bounds = WL.group_bounds(G)
    rot = trdq.Rotation(K, bounds, signs, smooth)
    w = WL.to_bf16_bits(rng.standard_normal((N, K)) * 0.02)
    bias = WL.to_bf16_bits(rng.standard_normal(N) * 0.01)
    wts = trdq.trdq_prepare_weights(rot, to_dev_bf16(w), wbits)
    ref = []
    for g in range(G):
        act, wv = O.fused_vectors(signs[g], smooth[g])
        ref.append((act, *(O.prepare_w8(w, wv) if wbits == 8 else O.prepare_w4(w, wv))))
    return rot, wts, bounds, bias, ref


def _acts(M, K, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, K))
    x[:, rng.choice(K, max(1, K // 100), replace=False)] *= 30.0
    return WL.to_bf16_bits(x)


@pytest.mark.parametrize("M,N,K", [
    (256, 1024, 1024),     # single-layer configuration: two row tiles
    (300, 1152, 1152),     # ragged rows, 9 k-blocks
    (129, 3456, 1152),     # one row past a tile
    (200, 1152, 4608),     # 36 k-blocks: the stage ring wraps many times
    (1, 16, 128),          # smallest legal problem
    (77, 1040, 256),       # N is not a multiple of any tile width
    (520, 4608, 1152),
])
def test_int32_accumulators_bit_exact(M, N, K):
    import torch
    from paper_2503_06564_b200 import trdq
    G = 2
    rot, wts, bounds, _, ref = _setup(N, K, G, 100 + N + K)
    x = _acts(M, K, 7 + M)
    for g in range(G):
        act, qw_ref, sw_ref = ref[g]
        q_ref, _ = O.rotate_quantize(x, act)
        # the GEMM is judged on the oracle's codes, so that only the contraction is under test
        wq_dev, _ = wts.view_tensors(g)
        assert np.array_equal(wq_dev.cpu().numpy(), qw_ref)
        acc = trdq.trdq_gemm_i32(wts, int(bounds[g]), torch.from_numpy(q_ref).cuda())
        acc_ref = O.gemm_i32(q_ref, qw_ref)
        assert np.array_equal(acc.cpu().numpy(), acc_ref)
    assert trdq.trdq_device_status() == 0


def test_int32_accumulators_extreme_codes():
    """All codes at +-127 with K = 4608: |acc| reaches 74 million (> 2^24), exact in int32."""
    import torch
    from paper_2503_06564_b200 import trdq
    N, K, M = 64, 4608, 130
    signs = np.ones((1, K), np.int8)
    rot = trdq.Rotation(K, [0, 1000], signs, np.full((1, K), np.float32(2.0 ** 3.5), np.float32))
    # weights whose rotated rows are +-c in every position: a single non-zero per 128-block
    w = np.zeros((N, K))
    rng = np.random.default_rng(0)
    for n in range(N):
        for b in range(K // 128):
            w[n, b * 128 + rng.integers(0, 128)] = rng.choice([-1.0, 1.0])
    wb = WL.to_bf16_bits(w)
    wts = trdq.trdq_prepare_weights(rot, to_dev_bf16(wb), 8)
    _, wv = O.fused_vectors(signs[0], np.full(K, np.float32(2.0 ** 3.5), np.float32))
    qw_ref, sw_ref = O.prepare_w8(wb, wv)
    assert set(np.unique(qw_ref).tolist()) == {-127, 127}
    q = (rng.integers(0, 2, (M, K)) * 254 - 127).astype(np.int8)
    q[0] = qw_ref[0]                      # one row fully aligned with a weight row: acc = K * 127^2
    acc = trdq.trdq_gemm_i32(wts, 0, torch.from_numpy(q).cuda()).cpu().numpy()
    acc_ref = q.astype(np.int64) @ qw_ref.astype(np.int64).T
    assert acc_ref[0, 0] == K * 127 * 127 and acc_ref.max() < 2 ** 31
    assert np.array_equal(acc.astype(np.int64), acc_ref)
    # epilogue on accumulators that do not fit fp32 exactly
    sx = rng.uniform(0.01, 0.02, M).astype(np.float32)
    y = trdq.trdq_linear(wts, 0, torch.from_numpy(q).cuda(), torch.from_numpy(sx).cuda())
    y_ref = O.epilogue(acc_ref.astype(np.int32), sx, sw_ref, None)
    check_output(bf16_to_f32_np(y), y_ref, max_ulp=1.0)


@pytest.mark.parametrize("M,N,K,with_bias", [
    (256, 1024, 1024, True),
    (300, 1152, 1152, True),
    (129, 3456, 1152, False),
    (200, 1152, 4608, True),
    (1, 16, 128, True),
    (77, 1040, 256, True),
    (2304, 1152, 1152, True),    # enough rows for the CTA-pair kernel: nine 256-row tiles
    (2100, 1040, 256, False),    # pair kernel, ragged: the last pair's second CTA has no valid row; N not a tile multiple
])
def test_linear_matches_oracle(M, N, K, with_bias):
    import torch
    from paper_2503_06564_b200 import trdq
    G = 2
    rot, wts, bounds, bias, ref = _setup(N, K, G, 200 + N + K)
    x = _acts(M, K, 17 + M)
    xd = to_dev_bf16(x)
    bias_d = to_dev_bf16(bias) if with_bias else None
    for g in range(G):
        t = int(bounds[g])
        act, qw_ref, sw_ref = ref[g]
        q_ref, sx_ref = O.rotate_quantize(x, act)
        codes, scales = trdq.trdq_rotate_quantize(rot, t, xd)
        assert np.array_equal(codes.cpu().numpy(), q_ref) and np.array_equal(scales.cpu().numpy(), sx_ref)
        y = trdq.trdq_linear(wts, t, codes, scales, bias_d)
        y_ref = O.linear_w8_rows(q_ref, sx_ref, qw_ref, sw_ref, bias if with_bias else None, np.arange(M))
        l2, ulps = check_output(bf16_to_f32_np(y), y_ref, max_ulp=2.0, rel_l2=2e-3)
        assert ulps <= 1.0      # the epilogue is accurate to half a bf16 step plus fp32 noise
    assert trdq.trdq_device_status() == 0


def test_epilogue_cancellation_against_bias():
    """Outputs where acc*sx*sw and the bias cancel to almost nothing must still be within 2 bf16
    steps of the exact value: the scale product is carried as an exact two-term sum."""
    import torch
    from paper_2503_06564_b200 import trdq
    N, K, M = 16, 128, 128
    signs = np.ones((1, K), np.int8)
    rot = trdq.Rotation(K, [0, 1000], signs, np.full((1, K), np.float32(2.0 ** 3.5), np.float32))
    w = np.zeros((N, K))
    w[:, 0] = 1.0                                    # rotated rows are all ones -> codes all 127
    wb = WL.to_bf16_bits(w)
    wts = trdq.trdq_prepare_weights(rot, to_dev_bf16(wb), 8)
    _, wv = O.fused_vectors(signs[0], np.full(K, np.float32(2.0 ** 3.5), np.float32))
    qw_ref, sw_ref = O.prepare_w8(wb, wv)
    rng = np.random.default_rng(4)
    q = rng.integers(-127, 128, (M, K)).astype(np.int8)
    acc = q.astype(np.int64) @ qw_ref.astype(np.int64).T
    sx = rng.uniform(0.003, 0.03, M).astype(np.float32)
    # bias = bf16 value closest to -acc*sx*sw of row n (so row n, column n nearly cancels)
    exact = acc.astype(np.float64) * sx[:, None].astype(np.float64) * sw_ref[None, :].astype(np.float64)
    bias = WL.to_bf16_bits(-np.diag(exact[:N, :N]))
    y = trdq.trdq_linear(wts, 0, torch.from_numpy(q).cuda(), torch.from_numpy(sx).cuda(), to_dev_bf16(bias))
    y_ref = O.epilogue(acc.astype(np.int32), sx, sw_ref, bias)
    d = np.abs(np.diag(y_ref[:N, :N]))
    assert (d < 1e-2 * np.abs(np.diag(exact[:N, :N]))).all()     # the cancellation really happens
    check_output(bf16_to_f32_np(y), y_ref, max_ulp=2.0)


def test_linear_strided_output_and_cfg_segments():
    import torch
    from paper_2503_06564_b200 import trdq
    M, N, K = 300, 1152, 1152
    rot, wts, bounds, bias, ref = _setup(N, K, 2, 321)
    x = _acts(M, K, 3)
    t = int(bounds[1])
    codes, scales = trdq.trdq_rotate_quantize(rot, t, to_dev_bf16(x))
    bias_d = to_dev_bf16(bias)
    y = trdq.trdq_linear(wts, t, codes, scales, bias_d)
    # output rows with a larger stride; the padding must stay untouched
    wide = torch.full((M, N + 24), 7.0, dtype=torch.bfloat16, device="cuda")
    trdq.trdq_linear(wts, t, codes, scales, bias_d, out=wide[:, :N])
    assert torch.equal(wide[:, :N], y) and bool((wide[:, N:] == 7.0).all())
    # conditional / unconditional halves stored apart, one launch
    mc = 171
    halves = trdq.trdq_linear_cfg(wts, t, [codes[:mc].contiguous(), codes[mc:].contiguous()],
                                  [scales[:mc].contiguous(), scales[mc:].contiguous()], bias_d)
    assert torch.equal(torch.cat(halves), y)
    empty = trdq.trdq_linear_cfg(wts, t, [codes[:0], codes], [scales[:0], scales], bias_d)
    assert empty[0].shape[0] == 0 and torch.equal(empty[1], y)
    # M == 0
    assert trdq.trdq_linear(wts, t, codes[:0], scales[:0], bias_d).shape == (0, N)
    # the same through the CTA-pair kernel (>= 2048 rows in total): two segments of 1300 and 1100 rows
    xl = _acts(2400, K, 8)
    cl, sl = trdq.trdq_rotate_quantize(rot, t, to_dev_bf16(xl))
    yl = trdq.trdq_linear(wts, t, cl, sl, bias_d)
    hl = trdq.trdq_linear_cfg(wts, t, [cl[:1300].contiguous(), cl[1300:].contiguous()], [sl[:1300].contiguous(), sl[1300:].contiguous()],
                              bias_d)
    assert torch.equal(torch.cat(hl), yl)
    act_l, qw_l, sw_l = ref[1]
    rows = np.concatenate([np.arange(0, 300), np.arange(1200, 1400), np.arange(2300, 2400)])
    q_l, sx_l = O.rotate_quantize(xl, act_l)
    y_l_ref = O.linear_w8_rows(q_l, sx_l, qw_l, sw_l, bias, rows)
    check_output(bf16_to_f32_np(yl)[rows], y_l_ref, max_ulp=1.0)
    # errors
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_linear(wts, 5000, codes, scales, bias_d)
    assert e.value.status == 4
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_linear(wts, t, codes, scales, bias_d, out=torch.empty((M, N + 4), dtype=torch.bfloat16, device="cuda")[:, :N])
    assert e.value.status == 3
    assert trdq.trdq_device_status() == 0


@pytest.mark.parametrize("M,N,K,with_bias", [
    (300, 1152, 1152, True),     # 9 scale groups, ragged rows
    (129, 1168, 4608, True),     # 36 groups: accumulators rotate many times; N is not a multiple of the tile
    (1, 16, 128, False),         # one group, smallest problem
    (260, 3456, 1152, False),
    (40, 128, 12416, True),      # 97 groups: the multiplier table no longer fits shared memory
])
def test_linear_w4a8_matches_oracle(M, N, K, with_bias):
    """int4 weights with one scale per (channel, 128 k): per-group integer sums, scaled and added."""
    from paper_2503_06564_b200 import trdq
    G = 2
    rot, wts, bounds, bias, ref = _setup(N, K, G, 400 + N + K, wbits=4)
    assert wts.wbits == 4
    x = _acts(M, K, 27 + M)
    xd = to_dev_bf16(x)
    bias_d = to_dev_bf16(bias) if with_bias else None
    for g in range(G):
        t = int(bounds[g])
        act, packed_ref, sw4_ref = ref[g]
        packed_dev, sw4_dev = wts.view_tensors(g)
        assert np.array_equal(packed_dev.cpu().numpy(), packed_ref) and np.array_equal(sw4_dev.cpu().numpy(), sw4_ref)
        q_ref, sx_ref = O.rotate_quantize(x, act)
        codes, scales = trdq.trdq_rotate_quantize(rot, t, xd)
        assert np.array_equal(codes.cpu().numpy(), q_ref)
        y = trdq.trdq_linear(wts, t, codes, scales, bias_d)
        y_ref = O.linear_w4_rows(q_ref, sx_ref, packed_ref, sw4_ref, bias if with_bias else None, np.arange(M))
        l2, ulps = check_output(bf16_to_f32_np(y), y_ref, max_ulp=2.0, rel_l2=2e-3)
        assert ulps <= 1.0
    assert trdq.trdq_device_status() == 0


def test_linear_w4a8_group_scales_of_very_different_size():
    """Channels whose group scales span many binades (one huge weight in one block): the common-grid
    integer multipliers lose low bits of the small scales only, far below a bf16 step of the result."""
    from paper_2503_06564_b200 import trdq
    M, N, K = 140, 128, 1024
    rng = np.random.default_rng(77)
    signs = (rng.integers(0, 2, (1, K)) * 2 - 1).astype(np.int8)
    rot = trdq.Rotation(K, [0, 1000], signs, None)
    w = rng.standard_normal((N, K)) * 0.02
    w[:, 0:128] *= 3000.0          # group 0 is 3000 x larger than the others
    w[5, 256:384] = 0.0            # an all-zero group: scale 0, codes 0
    wb = WL.to_bf16_bits(w)
    wts = trdq.trdq_prepare_weights(rot, to_dev_bf16(wb), 4)
    act, wv = O.fused_vectors(signs[0], None)
    packed_ref, sw4_ref = O.prepare_w4(wb, wv)
    assert sw4_ref[5, 2] == 0.0
    x = _acts(M, K, 5)
    q_ref, sx_ref = O.rotate_quantize(x, act)
    codes, scales = trdq.trdq_rotate_quantize(rot, 0, to_dev_bf16(x))
    y = trdq.trdq_linear(wts, 0, codes, scales, None)
    y_ref = O.linear_w4_rows(q_ref, sx_ref, packed_ref, sw4_ref, None, np.arange(M))
    check_output(bf16_to_f32_np(y), y_ref, max_ulp=1.0)


def test_small_shapes_through_the_cta_pair_kernel():
    """The CTA-pair kernel normally serves problems of >= 2048 rows.  Re-run this file's 8-bit cases in a
    child process with the threshold lowered to one row (the library reads TRDQ_PAIR_MIN_M once), so that
    every small and ragged shape above also goes through the pair kernel."""
    import os
    import subprocess
    import sys
    env = dict(os.environ, TRDQ_PAIR_MIN_M="1")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, "-m", "pytest", os.path.abspath(__file__), "-m", "gpu", "-x", "-q", "-k",
                          "not w4a8 and not through_the_cta_pair"], cwd=root, env=env,
                         capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]


@pytest.mark.parametrize("M,N,K", [
    (130, 272, 8192),      # ragged rows and columns, 64 k-blocks over eight ranges
    (64, 1152, 16384),     # nine tiles, 128 k-blocks
    (200, 1024, 9088),     # 71 k-blocks: the last range is shorter than the others
    (960, 1152, 4096),     # cross-attention K / V projection: the reduction is too short to pay, one range
    (4096, 1152, 1152),    # enough tiles: split-K declines and the call is the ordinary GEMM
])
def test_linear_splitk_is_bit_identical(M, N, K):
    """Partial int32 sums from several CTAs per tile, added by a second kernel: integer addition does not
    depend on the order, so the output must equal trdq_linear bit for bit."""
    import torch
    from paper_2503_06564_b200 import trdq
    rot, wts, bounds, bias, ref = _setup(N, K, 2, 500 + N + K)
    x = _acts(M, K, 31 + M)
    t = int(bounds[1])
    codes, scales = trdq.trdq_rotate_quantize(rot, t, to_dev_bf16(x))
    bias_d = to_dev_bf16(bias)
    y = trdq.trdq_linear(wts, t, codes, scales, bias_d)
    splits, nbytes = trdq.trdq_linear_splitk_workspace(wts, M)
    if K < 8192:
        assert splits == 1 and nbytes == 0
    else:
        assert splits >= 2 and nbytes == splits * M * N * 4
    ws = torch.full((max(nbytes, 16),), 0x5A, dtype=torch.uint8, device="cuda")    # stale contents must not matter
    y2 = trdq.trdq_linear_splitk(wts, t, codes, scales, bias_d, workspace=ws)
    assert torch.equal(y2, y)
    y3 = trdq.trdq_linear_splitk(wts, t, codes, scales, None, workspace=ws)
    assert torch.equal(y3, trdq.trdq_linear(wts, t, codes, scales, None))
    if splits > 1:
        with pytest.raises(trdq.TrdqError) as e:
            trdq.trdq_linear_splitk(wts, t, codes, scales, bias_d, workspace=ws[:nbytes - 16])
        assert e.value.status == 8
    assert trdq.trdq_device_status() == 0


def test_an_expired_wait_is_reported_and_the_device_stays_usable():
    """Every barrier wait in the kernels has a time limit.  The self-test kernel waits on a barrier nothing signals:
    the wait gives up after 20 ms, the status word carries its bit, and ordinary work runs fine afterwards."""
    import torch
    from paper_2503_06564_b200 import trdq
    assert trdq.trdq_device_status() == 0
    trdq.trdq_selftest_wait_expiry()
    word = trdq.trdq_device_status()               # synchronises
    assert word == 1 << 31
    assert trdq.trdq_device_status() == 0          # reading clears it
    rot, wts, bounds, bias, ref = _setup(256, 256, 1, 9)
    x = _acts(64, 256, 2)
    codes, scales = trdq.trdq_rotate_quantize(rot, 0, to_dev_bf16(x))
    act, qw_ref, sw_ref = ref[0]
    q_ref, sx_ref = O.rotate_quantize(x, act)
    assert np.array_equal(codes.cpu().numpy(), q_ref)
    y = trdq.trdq_linear(wts, 0, codes, scales, to_dev_bf16(bias))
    y_ref = O.linear_w8_rows(q_ref, sx_ref, qw_ref, sw_ref, bias, np.arange(64))
    check_output(bf16_to_f32_np(y), y_ref, max_ulp=1.0)
    assert trdq.trdq_device_status() == 0


@pytest.mark.parametrize("M,K,N,wbits", [(300, 256, 400, 8), (4096, 1152, 4608, 8), (260, 384, 272, 4)])
def test_linear_with_gelu_epilogue(M, K, N, wbits):
    """trdq_linear_act: GELU (tanh form) folded into the epilogue, all three GEMM kernels (M >= 2048 takes the CTA-pair one),
    against the oracle's double evaluation on the same codes; act = 0 must equal trdq_linear bit for bit."""
    import torch
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(90 + N)
    signs = (rng.integers(0, 2, (1, K)) * 2 - 1).astype(np.int8)
    rot = trdq.Rotation(K, [0, 1000], signs)
    x = WL.to_bf16_bits(rng.standard_normal((M, K)) * 2.0)
    w_bits = WL.to_bf16_bits(rng.standard_normal((N, K)) * 0.06)        # pre-activations of a few units: both GELU tails are hit
    bias_bits = WL.to_bf16_bits(rng.standard_normal(N) * 0.5)
    w = trdq.trdq_prepare_weights(rot, to_dev_bf16(w_bits), wbits)
    codes, scales = trdq.trdq_rotate_quantize(rot, 0, to_dev_bf16(x))
    bias = to_dev_bf16(bias_bits)
    y = trdq.trdq_linear_act(w, 0, codes, scales, bias)
    wq, sw = w.view_tensors(0)
    rows = np.unique(np.concatenate([np.arange(0, M, max(1, M // 48)), [M - 1]])).astype(np.int64)
    fn = O.linear_w8_rows if wbits == 8 else O.linear_w4_rows
    y_ref = fn(codes.cpu().numpy(), scales.cpu().numpy(), wq.cpu().numpy(), sw.cpu().numpy(), bias_bits, rows, act=1)
    pre = fn(codes.cpu().numpy(), scales.cpu().numpy(), wq.cpu().numpy(), sw.cpu().numpy(), bias_bits, rows, act=0)
    assert pre.max() > 3.0 and pre.min() < -3.0
    check_output(bf16_to_f32_np(y)[rows], y_ref, tiny=2.0 ** -100)   # GELU of x < -8.5 lies below 2^-100
    plain = trdq.trdq_linear(w, 0, codes, scales, bias)
    assert torch.equal(trdq.trdq_linear_act(w, 0, codes, scales, bias, act=trdq.ACT_NONE), plain)
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_linear_act(w, 0, codes, scales, bias, act=7)
    assert e.value.status == 2
    assert trdq.trdq_device_status() == 0


@pytest.mark.parametrize("wbits", [8, 4])
def test_maximum_k(wbits):
    """K = 131072, the largest row the interface accepts (the bound that keeps |sum q * qw| <= K * 127^2 below 2^31):
    1024 blocks per row through the wide-row rotate kernel, 1024 k-blocks through the GEMM.  With every activation and
    weight code at +-127 in a worst-case row the accumulator reaches K * 127^2 = 2 114 060 288 exactly."""
    from paper_2503_06564_b200 import trdq
    K, M, N = 131072, 5, 32
    rng = np.random.default_rng(77)
    signs = np.ones((1, K), np.int8)
    rot = trdq.Rotation(K, [0, 1000], signs, np.full((1, K), 2.0 ** 3.5, np.float32))     # fused vector exactly +1
    x = rng.standard_normal((M, K))
    w = rng.standard_normal((N, K)) * 0.05
    # one token and one output channel made of a single spike per block: the transform of a spike is flat, so every
    # rotated value of that row is +-amax and every code +-127
    spike = np.zeros(K)
    spike[::128] = 3.0
    x[0] = spike
    w[0] = spike * 0.01
    x_bits, w_bits = WL.to_bf16_bits(x), WL.to_bf16_bits(w)
    wts = trdq.trdq_prepare_weights(rot, to_dev_bf16(w_bits), wbits)
    codes, scales = trdq.trdq_rotate_quantize(rot, 0, to_dev_bf16(x_bits))
    act, wv = O.fused_vectors(signs[0], np.full(K, 2.0 ** 3.5, np.float32))
    q_ref, sx_ref = O.rotate_quantize(x_bits, act)
    assert np.array_equal(codes.cpu().numpy(), q_ref) and np.array_equal(scales.cpu().numpy(), sx_ref)
    assert np.all(np.abs(q_ref[0]) == 127)                                  # the flat row
    y = trdq.trdq_linear(wts, 0, codes, scales, None)
    rows = np.arange(M)
    if wbits == 8:
        qw_ref, sw_ref = O.prepare_w8(w_bits, wv)
        acc = trdq.trdq_gemm_i32(wts, 0, codes).cpu().numpy()
        acc_ref = O.gemm_i32(q_ref, qw_ref)
        assert np.array_equal(acc, acc_ref)
        assert abs(int(acc_ref[0, 0])) == K * 127 * 127                     # the int32 bound is reached, not exceeded
        y_ref = O.linear_w8_rows(q_ref, sx_ref, qw_ref, sw_ref, None, rows)
    else:
        pk_ref, sw4_ref = O.prepare_w4(w_bits, wv)
        y_ref = O.linear_w4_rows(q_ref, sx_ref, pk_ref, sw4_ref, None, rows)
    check_output(bf16_to_f32_np(y), y_ref)
    assert trdq.trdq_device_status() == 0


def test_every_linear_entry_point_validates_on_the_host():
    """Bad pointers, strides and time-steps are reported by the host code of every linear entry point (the plain one,
    the two split-K forms and the asymmetric one) before anything is launched: the output stays untouched and the
    device healthy.  Called through the C ABI directly so that misaligned addresses can be passed."""
    import ctypes as C
    import torch
    from paper_2503_06564_b200 import trdq
    lib = trdq.lib()
    N, K, M = 1152, 8192, 128                        # a shape for which split-K is chosen, so those paths do their own checks
    rot, wts, _, bias_bits, _ = _setup(N, K, 2, seed=21)
    x_bits = _acts(M, K, 22)
    codes, scales = trdq.trdq_rotate_quantize(rot, 0, to_dev_bf16(x_bits))
    bias = to_dev_bf16(bias_bits)
    assert trdq.trdq_linear_splitk_workspace(wts, M)[0] > 1
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty((8 * M * N * 4,), dtype=torch.uint8, device="cuda")
    zp = torch.zeros((M,), dtype=torch.int32, device="cuda")
    h, st = wts._h, trdq._stream()
    c, sc, b, yp, wp, z = (t.data_ptr() for t in (codes, scales, bias, y, ws, zp))

    def calls(c=c, sc=sc, b=b, yp=yp, ldy=N, t=0, M=M):
        return {
            "linear": lib.trdq_linear(h, t, c, sc, M, b, yp, ldy, st),
            "act": lib.trdq_linear_act(h, t, c, sc, M, b, yp, ldy, 0, st),
            "splitk": lib.trdq_linear_splitk(h, t, c, sc, M, b, yp, ldy, wp, ws.numel(), st),
            "static": lib.trdq_linear_splitk_static(h, t, c, sc, M, b, yp, ldy, st),
            "asym": lib.trdq_linear_asym(h, t, c, sc, z, M, b, yp, ldy, st),
        }

    def all_equal(result, status):
        assert set(result.values()) == {status}, result

    all_equal(calls(M=-1), 2)                 # negative row count
    all_equal(calls(t=1000), 4)               # time-step outside the covered range
    all_equal(calls(t=-1), 4)
    all_equal(calls(c=None), 1)
    all_equal(calls(sc=None), 1)
    all_equal(calls(yp=None), 1)
    all_equal(calls(ldy=N - 8), 2)            # rows of Y would overlap
    all_equal(calls(ldy=N + 4), 3)            # rows of Y not 16-byte aligned
    all_equal(calls(c=c + 8), 3)
    all_equal(calls(yp=yp + 2), 3)
    all_equal(calls(sc=sc + 2), 3)            # the kernels read sx[m] as a 4-byte float
    all_equal(calls(sc=sc + 1), 3)
    all_equal(calls(b=b + 1), 3)              # ... and bias[n] as a 2-byte bf16
    assert lib.trdq_linear_splitk(h, 0, c, sc, M, b, yp, N, wp + 4, ws.numel(), st) == 3
    assert lib.trdq_linear_splitk(h, 0, c, sc, M, b, yp, N, None, ws.numel(), st) == 1
    assert lib.trdq_linear_splitk(h, 0, c, sc, M, b, yp, N, wp, 16, st) == 8
    assert lib.trdq_linear_asym(h, 0, c, sc, z + 2, M, b, yp, N, st) == 3
    assert lib.trdq_linear_asym(h, 0, c, sc, None, M, b, yp, N, st) == 1
    torch.cuda.synchronize()
    assert not y.any().item()                 # none of the refused calls launched anything
    # M = 0 is a valid empty call everywhere, and an odd but 2-byte aligned bias address is accepted
    all_equal(calls(M=0), 0)
    bias_odd = torch.zeros((N + 1,), dtype=torch.bfloat16, device="cuda")
    bias_odd[1:] = bias
    expected = trdq.trdq_linear(wts, 0, codes, scales, bias)
    assert lib.trdq_linear_splitk_static(h, 0, c, sc, M, bias_odd.data_ptr() + 2, yp, N, st) == 0
    assert torch.equal(y, expected)
    assert trdq.trdq_device_status() == 0


def test_prepare_then_use_on_one_stream_without_synchronisation():
    """Weight preparation, rotate + quantize and the linear enqueued back to back on one stream, nothing synchronised in
    between, several fresh weight sets in a row: the GEMM requests weight tiles before its dependent-launch wait, which
    is only correct if the preparation's last kernel fully orders the code-writing kernels before anything that follows."""
    import torch
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(77)
    M, K = 2304, 1152                                   # enough rows for the CTA-pair kernel
    x_bits = _acts(M, K, 78)
    xd = to_dev_bf16(x_bits)
    rows = np.arange(0, M, 53, dtype=np.int64)
    signs = (rng.integers(0, 2, (1, K)) * 2 - 1).astype(np.int8)
    rot = trdq.Rotation(K, [0, 1000], signs)
    act, wv = O.fused_vectors(signs[0], None)
    q_ref, sx_ref = O.rotate_quantize(x_bits, act)
    cases = []
    for i, (N, wbits) in enumerate([(1152, 8), (256, 8), (3456, 8), (640, 4), (1152, 8), (128, 8)]):
        w_bits = WL.to_bf16_bits(rng.standard_normal((N, K)) * 0.03)
        bias_bits = WL.to_bf16_bits(rng.standard_normal(N) * 0.01)
        cases.append((N, wbits, w_bits, bias_bits, to_dev_bf16(w_bits), to_dev_bf16(bias_bits)))
    torch.cuda.synchronize()
    outs = []
    for N, wbits, w_bits, bias_bits, wd, bd in cases:    # no synchronisation from here to the end of the loop
        wts = trdq.trdq_prepare_weights(rot, wd, wbits)
        codes, scales = trdq.trdq_rotate_quantize(rot, 0, xd)
        outs.append((wts, trdq.trdq_linear(wts, 0, codes, scales, bd)))
    torch.cuda.synchronize()
    for (N, wbits, w_bits, bias_bits, wd, bd), (wts, y) in zip(cases, outs):
        if wbits == 8:
            qw, sw = O.prepare_w8(w_bits, wv)
            y_ref = O.linear_w8_rows(q_ref, sx_ref, qw, sw, bias_bits, rows)
        else:
            pk, sw4 = O.prepare_w4(w_bits, wv)
            y_ref = O.linear_w4_rows(q_ref, sx_ref, pk, sw4, bias_bits, rows)
        check_output(bf16_to_f32_np(y)[rows], y_ref)
    assert trdq.trdq_device_status() == 0


def test_kernel_choice_and_tensor_pipe_ceiling():
    """The two reporting aids: the library names the kernel a shape gets (the same functions the launchers use), and
    the MMA-only kernel runs to completion and reports the operations it performed."""
    import torch
    from paper_2503_06564_b200 import trdq
    assert trdq.trdq_kernel_choice(0, 256, 1024) == "rotate_quantize_rows_kernel"
    assert trdq.trdq_kernel_choice(0, 32768, 1152) == "rotate_quantize_team_kernel"
    assert trdq.trdq_kernel_choice(0, 8, 17408) == "rotate_quantize_kernel"
    assert trdq.trdq_kernel_choice(1, 32768, 1152, 4608, 8).startswith("gemm_w8a8_pair_kernel<")
    import os
    small_is_pair = int(os.environ.get("TRDQ_PAIR_MIN_M", "2048")) <= 960      # the child run of this file lowers the threshold
    assert trdq.trdq_kernel_choice(1, 960, 4096, 1152, 8).startswith("gemm_w8a8_pair_kernel<" if small_is_pair else "gemm_w8a8_kernel<")
    assert trdq.trdq_kernel_choice(1, 16384, 1152, 4608, 4) == "gemm_w4a8_kernel"
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_kernel_choice(1, 128, 1152, 1152, 6)
    assert e.value.status == 6
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    trdq.trdq_measure_mma_ceiling(4096)
    e0.record()
    ops = trdq.trdq_measure_mma_ceiling(16384)
    e1.record()
    torch.cuda.synchronize()
    assert trdq.trdq_device_status() == 0
    tops = ops / (e0.elapsed_time(e1) * 1e-3) / 1e12
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    per_cluster = 16384 * 2 * 256 * 256 * 32
    assert ops % per_cluster == 0 and 1 <= ops // per_cluster <= sms // 2
    assert 1000.0 < tops < 6000.0, tops           # the tensor pipe alone: a few PTOPS on this part


def test_debug_mode_reports_at_the_call():
    """TRDQ_DEBUG=1 (read once per process, hence a child process): every online call waits for its own work, so the
    self-test's expired wait comes back from that very call, the word is cleared, and ordinary calls still return OK."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = (
        "import numpy as np, torch\n"
        "from paper_2503_06564_b200 import trdq\n"
        "lib = trdq.lib()\n"
        "st = trdq._stream()\n"
        "assert lib.trdq_selftest_wait_expiry(st) == 9\n"
        "assert trdq.trdq_device_status() == 0\n"
        "rot = trdq.Rotation(1152, [0, 1000], np.ones((1, 1152), np.int8))\n"
        "x = torch.randn((3000, 1152), device='cuda').to(torch.bfloat16)\n"
        "w = trdq.trdq_prepare_weights(rot, (torch.randn((256, 1152), device='cuda') * 0.02).to(torch.bfloat16), 8)\n"
        "c, s = trdq.trdq_rotate_quantize(rot, 0, x)\n"
        "y = trdq.trdq_linear(w, 0, c, s, None)\n"
        "assert torch.isfinite(y.float()).all().item() and trdq.trdq_device_status() == 0\n"
        "print('debug ok')\n")
    res = subprocess.run([sys.executable, "-c", code], cwd=root, env=dict(os.environ, TRDQ_DEBUG="1"), capture_output=True, text=True,
                         timeout=600)
    assert res.returncode == 0 and "debug ok" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]
