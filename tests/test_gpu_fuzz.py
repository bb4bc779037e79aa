"""Seeded random shapes through the whole path (rotate + quantize, both GEMM kernels, 8- and 4-bit weights,
with and without smoothing and bias) against the oracle: small problems, many corner combinations."""
import os

import numpy as np
import pytest

from oracle import trdq_oracle as O
from paper_2503_06564_b200 import workloads as WL
from tests.util import bf16_to_f32_np, check_output, to_dev_bf16

pytestmark = pytest.mark.gpu
LARGE_SEEDS = int(os.environ.get("TRDQ_FUZZ_SEEDS", "10"))   # more seeds for a soak run


@pytest.mark.parametrize("seed", list(range(12)))
def test_random_problem(seed):
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(1000 + seed)
    K = 128 * int(rng.integers(1, 13))
    N = 16 * int(rng.integers(1, 40))
    M = int(rng.integers(1, 420))
    G = int(rng.integers(1, 4))
    wbits = 4 if seed % 3 == 2 else 8
    with_smooth = bool(rng.integers(0, 2))
    with_bias = bool(rng.integers(0, 2))
    signs = (rng.integers(0, 2, (G, K)) * 2 - 1).astype(np.int8)
    smooth = rng.uniform(0.3, 3.0, (G, K)).astype(np.float32) if with_smooth else None
    bounds = np.sort(rng.choice(np.arange(1, 1000), G - 1, replace=False)) if G > 1 else np.array([], np.int64)
    bounds = np.concatenate([[0], bounds, [1000]]).astype(np.int32)
    x = rng.standard_normal((M, K)) * rng.uniform(0.1, 5.0)
    x[:, rng.choice(K, max(1, K // 64), replace=False)] *= 25.0
    if M > 2:
        x[1] = 0.0
    x = WL.to_bf16_bits(x)
    w = WL.to_bf16_bits(rng.standard_normal((N, K)) * 0.05)
    bias = WL.to_bf16_bits(rng.standard_normal(N) * 0.02)
    rot = trdq.Rotation(K, bounds, signs, smooth)
    wts = trdq.trdq_prepare_weights(rot, to_dev_bf16(w), wbits)
    xd = to_dev_bf16(x)
    bias_d = to_dev_bf16(bias) if with_bias else None
    g = int(rng.integers(0, G))
    t = int(rng.integers(bounds[g], bounds[g + 1]))
    assert rot.group_of(t) == g == O.group_of(bounds, t)
    act, wv = O.fused_vectors(signs[g], None if smooth is None else smooth[g])
    q_ref, sx_ref = O.rotate_quantize(x, act)
    codes, scales = trdq.trdq_rotate_quantize(rot, t, xd)
    assert np.array_equal(codes.cpu().numpy(), q_ref) and np.array_equal(scales.cpu().numpy(), sx_ref)
    y = trdq.trdq_linear(wts, t, codes, scales, bias_d)
    rows = np.arange(M)
    if wbits == 8:
        qw_ref, sw_ref = O.prepare_w8(w, wv)
        y_ref = O.linear_w8_rows(q_ref, sx_ref, qw_ref, sw_ref, bias if with_bias else None, rows)
        assert np.array_equal(trdq.trdq_gemm_i32(wts, t, codes).cpu().numpy(), O.gemm_i32(q_ref, qw_ref))
    else:
        pk_ref, sw4_ref = O.prepare_w4(w, wv)
        y_ref = O.linear_w4_rows(q_ref, sx_ref, pk_ref, sw4_ref, bias if with_bias else None, rows)
    wq_dev, sw_dev = wts.view_tensors(g)
    assert np.array_equal(wq_dev.cpu().numpy(), qw_ref if wbits == 8 else pk_ref)
    l2, ulps = check_output(bf16_to_f32_np(y), y_ref, max_ulp=2.0, rel_l2=2e-3)
    assert ulps <= 1.0
    assert trdq.trdq_device_status() == 0


@pytest.mark.parametrize("seed", list(range(LARGE_SEEDS)))
def test_random_large_rotate_quantize(seed):
    """Row counts in the thousands with random row widths (1 to 80 blocks), row strides and group vectors: the shapes that
    go to the one-thread-per-block team kernel with every team size it has, ragged last tiles included."""
    import torch
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(5000 + seed)
    nb = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 9, 11, 16, 18, 24, 32, 33, 36, 40, 64, 72, 80]))
    K = 128 * nb
    M = int(rng.integers(150, max(151, min(30000, 24_000_000 // K))))
    pad = int(rng.choice([0, 8, 64, 136]))
    signs = (rng.integers(0, 2, (1, K)) * 2 - 1).astype(np.int8)
    smooth = rng.uniform(0.3, 3.0, (1, K)).astype(np.float32) if rng.integers(0, 2) else None
    rot = trdq.Rotation(K, [0, 1000], signs, smooth)
    x = rng.standard_normal((M, K)).astype(np.float32) * np.float32(rng.uniform(0.1, 5.0))
    x[:, rng.choice(K, max(1, K // 64), replace=False)] *= 25.0
    x[rng.integers(0, M)] = 0.0
    xb = WL.to_bf16_bits(x.astype(np.float64))
    wide = torch.zeros((M, K + pad), dtype=torch.bfloat16, device="cuda")
    wide[:, :K] = to_dev_bf16(xb)
    codes, scales = trdq.trdq_rotate_quantize(rot, 0, wide[:, :K])
    act, _ = O.fused_vectors(signs[0], None if smooth is None else smooth[0])
    q_ref, s_ref = O.rotate_quantize(xb, act)
    assert np.array_equal(scales.cpu().numpy(), s_ref), (M, K, pad, trdq.trdq_kernel_choice(0, M, K))
    assert np.array_equal(codes.cpu().numpy(), q_ref), (M, K, pad, trdq.trdq_kernel_choice(0, M, K))
    assert trdq.trdq_device_status() == 0


@pytest.mark.parametrize("seed", list(range(8)))
def test_random_problem_dense_rotation_and_fusions(seed):
    """Random shapes through the paths with a derived tolerance: dense block rotation (tensor-core accumulation order),
    LayerNorm + modulation in front of the rotation (fp32 row statistics), and the GELU epilogue on top of either."""
    from paper_2503_06564_b200 import trdq
    from tests.util import check_codes_with_tolerance
    rng = np.random.default_rng(3000 + seed)
    nb = int(rng.integers(1, 11))
    K = 128 * nb
    N = 16 * int(rng.integers(1, 30))
    M = int(rng.integers(1, 500))
    x = rng.standard_normal((M, K)) * rng.uniform(0.2, 4.0) + rng.uniform(-1.0, 1.0)
    x[:, rng.choice(K, max(1, K // 64), replace=False)] *= 20.0
    x_bits = WL.to_bf16_bits(x)
    xd = to_dev_bf16(x_bits)
    w_bits = WL.to_bf16_bits(rng.standard_normal((N, K)) * 0.05)
    bias_bits = WL.to_bf16_bits(rng.standard_normal(N) * 0.3)
    smooth = rng.uniform(0.5, 2.0, (1, K)).astype(np.float32)
    rows = np.arange(M)
    if seed % 2 == 0:
        # dense blocks
        blocks = np.empty((1, nb, 128, 128), np.float32)
        for b in range(nb):
            q, _ = np.linalg.qr(rng.standard_normal((128, 128)))
            blocks[0, b] = q
        rot = trdq.DenseRotation(K, [0, 1000], blocks, smooth)
        codes, scales = trdq.trdq_rotate_dense_quantize(rot, 3, xd)
        stored = O.dense_stored_blocks(blocks[0], smooth[0])
        v = O.rotate_dense(x_bits, stored)
        xa = np.abs(WL.bf16_bits_to_f32(x_bits).astype(np.float64))
        sa = np.abs(WL.bf16_bits_to_f32(stored).astype(np.float64))
        mass = np.concatenate([xa[:, 128 * b:128 * (b + 1)] @ sa[b] for b in range(nb)], axis=1)
        check_codes_with_tolerance(codes.cpu().numpy(), scales.cpu().numpy(), v, 2.0 ** -20 * mass)
    else:
        # LayerNorm + modulation in front of the Hadamard rotation
        signs = (rng.integers(0, 2, (1, K)) * 2 - 1).astype(np.int8)
        rot = trdq.Rotation(K, [0, 1000], signs, smooth)
        rps = int(rng.integers(1, M + 1))
        S = (M + rps - 1) // rps
        shift_bits = WL.to_bf16_bits(rng.standard_normal((S, K)) * 0.3)
        scale_bits = WL.to_bf16_bits(rng.standard_normal((S, K)) * 0.3)
        eps = 1e-5
        codes, scales = trdq.trdq_norm_rotate_quantize(rot, 3, xd, to_dev_bf16(shift_bits), to_dev_bf16(scale_bits), rps, eps)
        a, _ = O.fused_vectors(signs[0], smooth[0])
        h = O.norm_modulate(x_bits, shift_bits, scale_bits, rps, eps)
        v = O.rotate_f32(h, a)
        xf = WL.bf16_bits_to_f32(x_bits).astype(np.float64)
        sh = np.repeat(WL.bf16_bits_to_f32(shift_bits).astype(np.float64), rps, axis=0)[:M]
        sc = np.repeat(WL.bf16_bits_to_f32(scale_bits).astype(np.float64), rps, axis=0)[:M]
        rstd = 1.0 / np.sqrt(xf.var(axis=1) + eps)
        tol_h = 2.0 ** -17 * (np.abs(h - sh) + np.abs(sh) + np.abs(1.0 + sc) * (rstd * np.abs(xf).mean(axis=1))[:, None])
        tol_v = np.repeat((tol_h * np.abs(a.astype(np.float64))[None, :]).reshape(M, nb, 128).sum(axis=2), 128, axis=1)
        check_codes_with_tolerance(codes.cpu().numpy(), scales.cpu().numpy(), v, tol_v)
    # the linear layer with the GELU epilogue on the codes the GPU produced (exact function of the codes)
    wts = trdq.trdq_prepare_weights(rot, to_dev_bf16(w_bits), 8)
    act = int(rng.integers(0, 2))
    y = trdq.trdq_linear_act(wts, 3, codes, scales, to_dev_bf16(bias_bits), act=act)
    wq, sw = wts.view_tensors(0)
    y_ref = O.linear_w8_rows(codes.cpu().numpy(), scales.cpu().numpy(), wq.cpu().numpy(), sw.cpu().numpy(), bias_bits, rows, act=act)
    check_output(bf16_to_f32_np(y), y_ref, tiny=2.0 ** -100 if act else 0.0)
    assert trdq.trdq_device_status() == 0
