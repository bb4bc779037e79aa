"""GPU parity of the literal asymmetric activation quantizer (Eq. 1-3) and the linear layer that consumes it."""
import numpy as np
import pytest

from oracle import trdq_oracle as O
from paper_2503_06564_b200 import workloads as WL
from tests.util import bf16_to_f32_np, check_output, to_dev_bf16

pytestmark = pytest.mark.gpu


def _spec(K, G, seed):
    rng = np.random.default_rng(seed)
    signs = (rng.integers(0, 2, (G, K)) * 2 - 1).astype(np.int8)
    smooth = rng.uniform(0.5, 2.0, (G, K)).astype(np.float32)
    return signs, smooth


def _acts(M, K, seed, shift=0.7):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, K)) + shift          # a non-zero mean: what the zero point is for
    x[:, rng.choice(K, max(1, K // 100), replace=False)] *= 20.0
    return WL.to_bf16_bits(x)


@pytest.mark.parametrize("M,K,G", [(300, 1152, 2), (70, 4608, 1), (5, 128, 2), (33, 384, 1), (1000, 1024, 1)])
def test_asymmetric_codes_match_oracle(M, K, G):
    from paper_2503_06564_b200 import trdq
    signs, smooth = _spec(K, G, 80 + K)
    bounds = WL.group_bounds(G)
    rot = trdq.Rotation(K, bounds, signs, smooth)
    x = _acts(M, K, 4 + M)
    x[min(3, M - 1)] = WL.to_bf16_bits(np.full(K, 0.0))      # an all-zero token: scale 0, z 0, codes 0
    xd = to_dev_bf16(x)
    for g in range(G):
        codes, scales, zp = trdq.trdq_rotate_quantize_asym(rot, int(bounds[g]), xd)
        act, _ = O.fused_vectors(signs[g], smooth[g])
        c_ref, s_ref, z_ref = O.rotate_quantize_asym(x, act)
        assert np.array_equal(scales.cpu().numpy(), s_ref)
        assert np.array_equal(zp.cpu().numpy(), z_ref)
        assert np.array_equal(codes.cpu().numpy(), c_ref)
    assert trdq.trdq_device_status() == 0


@pytest.mark.parametrize("M,N,K", [(260, 1152, 1152), (129, 1040, 256), (2304, 1152, 1152), (1, 16, 128)])
def test_asymmetric_linear_matches_oracle(M, N, K):
    import torch
    from paper_2503_06564_b200 import trdq
    G = 2
    signs, smooth = _spec(K, G, 90 + K)
    bounds = WL.group_bounds(G)
    rot = trdq.Rotation(K, bounds, signs, smooth)
    rng = np.random.default_rng(6)
    w = WL.to_bf16_bits(rng.standard_normal((N, K)) * 0.02)
    bias = WL.to_bf16_bits(rng.standard_normal(N) * 0.01)
    wts = trdq.trdq_prepare_weights(rot, to_dev_bf16(w), 8)
    x = _acts(M, K, 11)
    xd, bias_d = to_dev_bf16(x), to_dev_bf16(bias)
    for g in range(G):
        t = int(bounds[g])
        act, wv = O.fused_vectors(signs[g], smooth[g])
        q_ref, sx_ref, z_ref = O.rotate_quantize_asym(x, act)
        qw_ref, sw_ref = O.prepare_w8(w, wv)
        codes, scales, zp = trdq.trdq_rotate_quantize_asym(rot, t, xd)
        assert np.array_equal(codes.cpu().numpy(), q_ref) and np.array_equal(zp.cpu().numpy(), z_ref)
        y = trdq.trdq_linear_asym(wts, t, codes, scales, zp, bias_d)
        rows = np.arange(M) if M <= 300 else np.concatenate([np.arange(200), np.arange(M - 200, M)])
        y_ref = O.linear_asym_rows(q_ref, sx_ref, z_ref, qw_ref, sw_ref, bias, rows)
        l2, ulps = check_output(bf16_to_f32_np(y)[rows], y_ref, max_ulp=2.0, rel_l2=2e-3)
        assert ulps <= 1.0
    # not available for 4-bit weights or together with the full transform
    w4 = trdq.trdq_prepare_weights(rot, to_dev_bf16(w), 4)
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_linear_asym(w4, 0, codes, scales, zp, bias_d)
    assert e.value.status == 6
    rot_full = trdq.Rotation(K, bounds, signs, smooth, perm=np.stack([np.arange(K, dtype=np.int32)] * G))
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_rotate_quantize_asym(rot_full, 0, xd)
    assert e.value.status == 2
    assert trdq.trdq_device_status() == 0
