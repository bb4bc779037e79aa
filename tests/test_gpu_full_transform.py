"""GPU parity of the full balancing transform (Eq. 9: rotation, zigzag permutation, second rotation)
against the CPU oracle: activation codes, prepared weights, and the linear layer built on both."""
import numpy as np
import pytest

from oracle import trdq_oracle as O
from paper_2503_06564_b200 import workloads as WL
from tests.util import bf16_to_f32_np, check_output, to_dev_bf16

pytestmark = pytest.mark.gpu


def _spec(K, G, seed):
    rng = np.random.default_rng(seed)
    d1 = (rng.integers(0, 2, (G, K)) * 2 - 1).astype(np.int8)
    d2 = (rng.integers(0, 2, (G, K)) * 2 - 1).astype(np.int8)
    smooth = rng.uniform(0.25, 4.0, (G, K)).astype(np.float32)
    return d1, d2, smooth


def _acts(M, K, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, K))
    x[:, :128] *= 15.0                                   # a hot block: what the permutation is for
    x[:, rng.choice(K, max(1, K // 100), replace=False)] *= 30.0
    return WL.to_bf16_bits(x)


def _zigzag_per_group(x, d1, smooth):
    """Calibration stand-in: permutation of each group from the channel maxima after that group's first rotation."""
    perms = []
    for g in range(d1.shape[0]):
        a1, _ = O.fused_vectors(d1[g], smooth[g])
        perms.append(O.zigzag_permutation(np.abs(O.rotate(x[:64], a1)).max(axis=0)))
    return np.stack(perms)


@pytest.mark.parametrize("M,K,G", [(300, 1152, 2), (70, 4608, 1), (9, 128, 2), (33, 384, 1), (5, 16384, 1)])
def test_full_transform_codes_match_oracle(M, K, G):
    from paper_2503_06564_b200 import trdq
    d1, d2, smooth = _spec(K, G, 60 + K)
    x = _acts(M, K, 3 + M)
    perm = _zigzag_per_group(x, d1, smooth)
    bounds = WL.group_bounds(G)
    rot = trdq.Rotation(K, bounds, d1, smooth, perm=perm, signs2=d2)
    xd = to_dev_bf16(x)
    for g in range(G):
        codes, scales = trdq.trdq_rotate_quantize(rot, int(bounds[g]), xd)
        a1, _ = O.fused_vectors(d1[g], smooth[g])
        c_ref, s_ref = O.rotate2_quantize(x, a1, perm[g], O.second_vector(d2[g], K))
        assert np.array_equal(scales.cpu().numpy(), s_ref)
        assert np.array_equal(codes.cpu().numpy(), c_ref)
    # without signs2 the second rotation uses all +1
    rot1 = trdq.Rotation(K, bounds, d1, smooth, perm=perm)
    codes, scales = trdq.trdq_rotate_quantize(rot1, 0, xd)
    a1, _ = O.fused_vectors(d1[0], smooth[0])
    c_ref, s_ref = O.rotate2_quantize(x, a1, perm[0], O.second_vector(None, K))
    assert np.array_equal(codes.cpu().numpy(), c_ref) and np.array_equal(scales.cpu().numpy(), s_ref)
    assert trdq.trdq_device_status() == 0


@pytest.mark.parametrize("wbits", [8, 4])
def test_full_transform_linear_matches_oracle(wbits):
    """Weights prepared with R2^T P^T R1^T Delta^-1 (same pipeline on the rows of W), then the unchanged GEMM."""
    from paper_2503_06564_b200 import trdq
    M, N, K, G = 260, 1152, 1152, 2
    d1, d2, smooth = _spec(K, G, 77)
    rng = np.random.default_rng(5)
    x = _acts(M, K, 9)
    w = WL.to_bf16_bits(rng.standard_normal((N, K)) * 0.02)
    bias = WL.to_bf16_bits(rng.standard_normal(N) * 0.01)
    perm = _zigzag_per_group(x, d1, smooth)
    bounds = WL.group_bounds(G)
    rot = trdq.Rotation(K, bounds, d1, smooth, perm=perm, signs2=d2)
    wts = trdq.trdq_prepare_weights(rot, to_dev_bf16(w), wbits)
    xd, bias_d = to_dev_bf16(x), to_dev_bf16(bias)
    for g in range(G):
        t = int(bounds[g])
        a1, b1 = O.fused_vectors(d1[g], smooth[g])
        v2 = O.second_vector(d2[g], K)
        q_ref, sx_ref = O.rotate2_quantize(x, a1, perm[g], v2)
        wq_dev, sw_dev = wts.view_tensors(g)
        if wbits == 8:
            qw_ref, sw_ref = O.rotate2_quantize(w, b1, perm[g], v2)
            y_ref = O.linear_w8_rows(q_ref, sx_ref, qw_ref, sw_ref, bias, np.arange(M))
        else:
            qw_ref, sw_ref = O.prepare2_w4(w, b1, perm[g], v2)
            y_ref = O.linear_w4_rows(q_ref, sx_ref, qw_ref, sw_ref, bias, np.arange(M))
        assert np.array_equal(wq_dev.cpu().numpy(), qw_ref) and np.array_equal(sw_dev.cpu().numpy(), sw_ref)
        codes, scales = trdq.trdq_rotate_quantize(rot, t, xd)
        assert np.array_equal(codes.cpu().numpy(), q_ref)
        y = trdq.trdq_linear(wts, t, codes, scales, bias_d)
        l2, ulps = check_output(bf16_to_f32_np(y), y_ref, max_ulp=2.0, rel_l2=2e-3)
        assert ulps <= 1.0
        # the transform is an exact change of basis: the quantized product stays close to the fp64 linear layer
        y64 = WL.bf16_bits_to_f32(x).astype(np.float64) @ WL.bf16_bits_to_f32(w).astype(np.float64).T + WL.bf16_bits_to_f32(bias)
        rel = np.linalg.norm(bf16_to_f32_np(y) - y64) / np.linalg.norm(y64)
        assert rel < (0.06 if wbits == 8 else 0.6)
    assert trdq.trdq_device_status() == 0
