"""GPU parity of the LayerNorm + modulation + rotation + quantizer kernel against the CPU oracle.

Tolerance.  The oracle forms h in double and rounds once; the kernel forms it in fp32: the row sum passes through at most
16 + 3 + K/128 additions, so mean and variance carry a relative error of about (19 + K/128) * 2^-24, and h three more
roundings.  Allowed here: |h_gpu - h_ref| <= 2^-17 * (|h - shift| + |shift| + |1 + scale| * rstd * mean|x|), a factor of
a few above that estimate.  It propagates through the rotation as sum_i tol_h[i] * |vec[i]| over the block; scales and codes
are then compared as for any path whose pre-quantization values carry a tolerance (tests/util.py).  Rows whose arithmetic
is exact in both evaluations (see the test) must match bit for bit."""
import numpy as np
import pytest

from oracle import trdq_oracle as O
from paper_2503_06564_b200 import workloads as WL
from tests.util import check_codes_with_tolerance, to_dev_bf16

pytestmark = pytest.mark.gpu


def reference(x_bits, shift_bits, scale_bits, rps, eps, act_vec):
    K = x_bits.shape[1]
    h = O.norm_modulate(x_bits, shift_bits, scale_bits, rps, eps)
    v = O.rotate_f32(h, act_vec)
    x = WL.bf16_bits_to_f32(x_bits).astype(np.float64)
    M = x.shape[0]
    sh = np.zeros((M, K)) if shift_bits is None else np.repeat(WL.bf16_bits_to_f32(shift_bits).astype(np.float64), rps, axis=0)[:M]
    sc = np.zeros((M, K)) if scale_bits is None else np.repeat(WL.bf16_bits_to_f32(scale_bits).astype(np.float64), rps, axis=0)[:M]
    rstd = 1.0 / np.sqrt(x.var(axis=1) + eps)
    tol_h = 2.0 ** -17 * (np.abs(h - sh) + np.abs(sh) + np.abs(1.0 + sc) * (rstd * np.abs(x).mean(axis=1))[:, None])
    a = np.abs(act_vec.astype(np.float64))
    tol_v = np.repeat((tol_h * a[None, :]).reshape(M, K // 128, 128).sum(axis=2), 128, axis=1)
    return v, tol_v


@pytest.mark.parametrize("M,K,rps,G", [(300, 1152, 64, 2), (37, 4608, 16, 1), (5, 128, 2, 1), (1024, 1152, 256, 1), (64, 8192, 64, 1),
                                       # thousands of rows: samples that are not a multiple of the row tile, a ragged last sample,
                                       # 32- and 36-block rows, and samples of only four rows
                                       (8192, 1152, 256, 2), (5000, 1152, 1000, 1), (3000, 4096, 64, 1), (2400, 4608, 100, 1), (4000, 1152, 4, 1)])
def test_norm_fused_codes_match_oracle(M, K, rps, G):
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(200 + K + M)
    signs = (rng.integers(0, 2, (G, K)) * 2 - 1).astype(np.int8)
    smooth = rng.uniform(0.5, 2.0, (G, K)).astype(np.float32)
    bounds = WL.group_bounds(G)
    rot = trdq.Rotation(K, bounds, signs, smooth)
    x = rng.standard_normal((M, K)) * 2.0 + 0.7
    x[:, rng.choice(K, max(1, K // 100), replace=False)] *= 20.0
    x_bits = WL.to_bf16_bits(x)
    S = (M + rps - 1) // rps
    shift_bits = WL.to_bf16_bits(rng.standard_normal((S, K)) * 0.2)
    scale_bits = WL.to_bf16_bits(rng.standard_normal((S, K)) * 0.2)
    eps = 1e-6
    total = 0
    for g in range(G):
        codes, scales = trdq.trdq_norm_rotate_quantize(rot, int(bounds[g]), to_dev_bf16(x_bits), to_dev_bf16(shift_bits),
                                                       to_dev_bf16(scale_bits), rps, eps)
        a, _ = O.fused_vectors(signs[g], smooth[g])
        v, tol_v = reference(x_bits, shift_bits, scale_bits, rps, eps, a)
        total += check_codes_with_tolerance(codes.cpu().numpy(), scales.cpu().numpy(), v, tol_v)
    # no modulation: plain LayerNorm in front of the rotation
    codes, scales = trdq.trdq_norm_rotate_quantize(rot, 0, to_dev_bf16(x_bits), None, None, rps, eps)
    a, _ = O.fused_vectors(signs[0], smooth[0])
    v, tol_v = reference(x_bits, None, None, rps, eps, a)
    total += check_codes_with_tolerance(codes.cpu().numpy(), scales.cpu().numpy(), v, tol_v)
    assert trdq.trdq_device_status() == 0
    print(f"M={M} K={K}: {total} of {(G + 1) * M * K} codes off by one")


def test_norm_fused_exact_rows_and_determinism():
    """Rows of +-c in equal numbers have mean 0 and variance c^2 exactly; with eps = 0, scale = -1 + 2^p and a power-of-two shift
    every intermediate is exact in fp32 and in double, so the codes must equal the oracle's bit for bit.  Repeated launches give
    identical results (ordered reductions)."""
    import torch
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(9)
    K, M = 512, 40
    signs = (rng.integers(0, 2, (1, K)) * 2 - 1).astype(np.int8)
    rot = trdq.Rotation(K, [0, 1000], signs, np.full((1, K), 2.0 ** 3.5, np.float32))   # fused vector = +-1 exactly
    c = 2.0 ** rng.integers(-2, 3, M).astype(np.float64)
    x = np.where(rng.permuted(np.tile(np.array([1.0, -1.0]), (M, K // 2)), axis=1) > 0, 1.0, -1.0) * c[:, None]
    x_bits = WL.to_bf16_bits(x)
    scale_bits = WL.to_bf16_bits(np.full((1, K), -1.0 + 2.0 ** -1))      # 1 + scale = 0.5
    shift_bits = WL.to_bf16_bits(np.full((1, K), 0.25))
    codes, scales = trdq.trdq_norm_rotate_quantize(rot, 0, to_dev_bf16(x_bits), to_dev_bf16(shift_bits), to_dev_bf16(scale_bits), M, 0.0)
    a, _ = O.fused_vectors(signs[0], np.full(K, 2.0 ** 3.5, np.float32))
    assert np.all(np.abs(a) == 1.0)
    h = O.norm_modulate(x_bits, shift_bits, scale_bits, M, 0.0)
    assert set(np.unique(h)) <= {np.float32(0.75), np.float32(-0.25)}
    c_ref, s_ref = O.quantize_rows(O.rotate_f32(h, a))
    assert np.array_equal(codes.cpu().numpy(), c_ref) and np.array_equal(scales.cpu().numpy(), s_ref)
    # the same exact rows sixty times over, in samples of 70 rows (35 rows of each sign pattern pair do not align with any row tile)
    reps = 60
    xb_big = np.tile(x_bits, (reps, 1))
    cb, sb = trdq.trdq_norm_rotate_quantize(rot, 0, to_dev_bf16(xb_big), to_dev_bf16(np.tile(shift_bits, (35, 1))),
                                            to_dev_bf16(np.tile(scale_bits, (35, 1))), 70, 0.0)
    assert np.array_equal(cb.cpu().numpy(), np.tile(c_ref, (reps, 1))) and np.array_equal(sb.cpu().numpy(), np.tile(s_ref, reps))
    xr_big = to_dev_bf16(WL.to_bf16_bits(rng.standard_normal((M * reps, K)) * 3.0))
    c1, s1 = trdq.trdq_norm_rotate_quantize(rot, 0, xr_big, None, None, 70, 1e-6)
    for _ in range(3):
        c2, s2 = trdq.trdq_norm_rotate_quantize(rot, 0, xr_big, None, None, 70, 1e-6)
        assert torch.equal(c1, c2) and torch.equal(s1, s2)
    # determinism on ordinary data
    xr = to_dev_bf16(WL.to_bf16_bits(rng.standard_normal((M, K)) * 3.0))
    c1, s1 = trdq.trdq_norm_rotate_quantize(rot, 0, xr, None, None, M, 1e-6)
    for _ in range(3):
        c2, s2 = trdq.trdq_norm_rotate_quantize(rot, 0, xr, None, None, M, 1e-6)
        assert torch.equal(c1, c2) and torch.equal(s1, s2)
    assert trdq.trdq_device_status() == 0


def test_norm_fused_argument_errors():
    import torch
    from paper_2503_06564_b200 import trdq
    K = 256
    rot = trdq.Rotation(K, [0, 1000], np.ones((1, K), np.int8))
    x = torch.zeros((8, K), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_norm_rotate_quantize(rot, 0, x, None, None, 0, 1e-6)
    assert e.value.status == 2
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_norm_rotate_quantize(rot, 0, x, None, None, 8, -1.0)
    assert e.value.status == 2
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_norm_rotate_quantize(rot, 2000, x, None, None, 8, 1e-6)
    assert e.value.status == 4
    full = trdq.Rotation(K, [0, 1000], np.ones((1, K), np.int8), perm=np.arange(K, dtype=np.int32)[None, :])
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_norm_rotate_quantize(full, 0, x, None, None, 8, 1e-6)
    assert e.value.status == 10
    # a constant row: zero deviation, the output is the shift alone; all-zero result quantizes to scale 0
    codes, scales = trdq.trdq_norm_rotate_quantize(rot, 0, x + 3.0, None, None, 8, 1e-6)
    assert not codes.any() and not scales.any()
