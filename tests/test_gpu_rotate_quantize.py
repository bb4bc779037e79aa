"""GPU parity: fused rotate + quantize kernel and the offline weight preparation against the CPU oracle."""
import numpy as np
import pytest

from oracle import trdq_oracle as O
from paper_2503_06564_b200 import workloads as WL
from tests.util import check_codes, to_dev_bf16

pytestmark = pytest.mark.gpu


def _rot(K, G, seed, with_smooth):
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(seed)
    signs = (rng.integers(0, 2, (G, K)) * 2 - 1).astype(np.int8)
    smooth = rng.uniform(0.25, 4.0, (G, K)).astype(np.float32) if with_smooth else None
    bounds = WL.group_bounds(G)
    return trdq.Rotation(K, bounds, signs, smooth), signs, smooth, bounds


def _x(M, K, seed, outliers=True):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, K))
    if outliers and K >= 128:
        x[:, rng.choice(K, max(1, K // 100), replace=False)] *= 40.0
    return WL.to_bf16_bits(x)


@pytest.mark.parametrize("M,K,G,smooth", [
    (256, 1024, 2, False),      # the single-layer configuration
    (300, 1152, 5, True),       # 9 blocks, ragged row count
    (37, 4608, 3, True),        # 36 blocks, one row per tile
    (130, 4096, 4, False),
    (1, 128, 1, False),         # smallest legal problem
    (5, 128, 2, True),
    (33, 384, 2, True),         # 3 blocks: lane groups do not fill a warp multiple
    (3, 17408, 1, True),        # 136 blocks: several blocks per lane group
    (100, 640, 2, True),        # 5 blocks: 56 rows per tile, the last warp is partly idle, ragged last tile
    (9, 4736, 1, True),         # 37 blocks: too wide for one thread per block, lane-group kernel
    (600, 1152, 1, False),
    (9500, 1152, 1, True),      # team kernel, one-warp teams of 3 rows (27 of 32 lanes): 3167 tiles over 1776 teams, ragged tail
    (28500, 1152, 1, True),     # same, five to six tiles per team: both ring stages wrap several times
    (2100, 1152, 1, True),      # too few tiles for one-warp teams: two-warp teams of 7 rows (named barrier between the warps)
    (7200, 4608, 1, False),     # 36 blocks: four-warp teams of 3 rows, three teams per CTA
    (50000, 640, 2, True),      # 5 blocks: one-warp teams of 6 rows, eleven teams (shared memory bound)
    (4000, 4096, 1, True),      # 32 blocks: one row per warp, ten teams
    (5000, 2048, 1, False),     # 16 blocks: two rows per warp
    (3000, 8192, 1, True),      # 64 blocks: two-warp teams of one row
    (1500, 10240, 1, True),     # 80 blocks: three-warp teams of one row (80 of 96 lanes), three teams
    (149, 1152, 1, True),       # just over one tile per SM with the widest team: team kernel, most teams idle
])
def test_rotate_quantize_matches_oracle(M, K, G, smooth):
    from paper_2503_06564_b200 import trdq
    rot, signs, sm, bounds = _rot(K, G, 11 + K + M, smooth)
    x = _x(M, K, 5 + M)
    xd = to_dev_bf16(x)
    for g in range(G):
        t = int(bounds[g])
        codes, scales = trdq.trdq_rotate_quantize(rot, t, xd)
        act, _ = O.fused_vectors(signs[g], None if sm is None else sm[g])
        c_ref, s_ref = O.rotate_quantize(x, act)
        v_ref = O.rotate(x, act)
        amax = np.abs(v_ref).max(axis=1)
        inv = np.where(amax > 0, np.float32(127.0) / amax, 0).astype(np.float32)
        assert np.array_equal(scales.cpu().numpy(), s_ref), "per-token scales must be bit-exact"
        assert check_codes(codes.cpu().numpy(), c_ref, v_ref, inv) == 0
    assert trdq.trdq_device_status() == 0


def test_rotate_quantize_strided_rows_zero_rows_and_group_switch():
    import torch
    from paper_2503_06564_b200 import trdq
    K, M, G = 1152, 70, 2
    rot, signs, sm, bounds = _rot(K, G, 3, True)
    x = _x(M, K, 9)
    x[7] = 0          # all-zero token: scale 0, codes 0
    x[M - 1] = 0
    wide = torch.zeros((M, K + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :K] = to_dev_bf16(x)
    view = wide[:, :K]                      # row stride K + 64
    results = []
    for g in range(G):
        codes, scales = trdq.trdq_rotate_quantize(rot, int(bounds[g]) + 1, view)
        act, _ = O.fused_vectors(signs[g], sm[g])
        c_ref, s_ref = O.rotate_quantize(x, act)
        assert np.array_equal(codes.cpu().numpy(), c_ref) and np.array_equal(scales.cpu().numpy(), s_ref)
        assert scales[7].item() == 0.0 and not codes[7].any().item()
        results.append(codes.cpu().numpy())
    assert not np.array_equal(results[0], results[1])       # another group, another parameter set
    # any time-step of one group selects the same parameter set
    a, _ = trdq.trdq_rotate_quantize(rot, int(bounds[1]), view)
    b, _ = trdq.trdq_rotate_quantize(rot, int(bounds[2]) - 1, view)
    assert torch.equal(a, b)
    # M == 0 is a no-op
    trdq.trdq_rotate_quantize(rot, 0, wide[:0, :K])


def test_team_kernel_strided_rows_zero_rows_and_ties():
    """The same special cases at row counts that go to the one-thread-per-block team kernel: a row stride wider than K,
    all-zero tokens scattered through the tiles (scale 0, codes 0), and exact rounding ties (half to even)."""
    import torch
    from paper_2503_06564_b200 import trdq
    K, M = 1152, 9001
    assert trdq.trdq_kernel_choice(0, M, K) == "rotate_quantize_team_kernel"
    rot, signs, sm, bounds = _rot(K, 1, 5, True)
    x = _x(M, K, 10)
    zero_rows = [0, 4, 5, 3000, M - 1]
    x[zero_rows] = 0
    wide = torch.zeros((M, K + 128), dtype=torch.bfloat16, device="cuda")
    wide[:, :K] = to_dev_bf16(x)
    codes, scales = trdq.trdq_rotate_quantize(rot, 0, wide[:, :K])
    act, _ = O.fused_vectors(signs[0], sm[0])
    c_ref, s_ref = O.rotate_quantize(x, act)
    assert np.array_equal(codes.cpu().numpy(), c_ref) and np.array_equal(scales.cpu().numpy(), s_ref)
    assert not scales[zero_rows].any().item() and not codes[zero_rows].any().item()
    # ties: the five exact rows of test_rounding_ties_on_device repeated 2000 times (K = 128: 32 rows per one-warp team)
    K2, reps = 128, 2000
    assert trdq.trdq_kernel_choice(0, 5 * reps, K2) == "rotate_quantize_team_kernel"
    rot2 = trdq.Rotation(K2, [0, 1000], np.ones((1, K2), np.int8), np.full((1, K2), np.float32(2.0 ** 3.5), np.float32))
    base = np.zeros((5, K2))
    base[0, :4] = [201, 150, 99, 58]
    base[1, :4] = [-201, -150, -99, -58]
    base[2, :2] = [255, 253]
    base[3, :4] = [131, 130, 126, 121]
    base[4, :4] = [-131, -130, -126, -121]
    xb = WL.to_bf16_bits(np.tile(base, (reps, 1)))
    c2, s2 = trdq.trdq_rotate_quantize(rot2, 0, to_dev_bf16(xb))
    c2 = c2.cpu().numpy().reshape(reps, 5, K2)
    assert np.all(s2.cpu().numpy() == 4.0)
    i = np.arange(K2) & 3
    expect = np.stack([np.array(v)[i] for v in ([127, 23, 48, 2], [-127, -23, -48, -2], [127, 0, 127, 0], [127, 2, 4, -1], [-127, -2, -4, 1])])
    assert np.array_equal(c2, np.broadcast_to(expect, c2.shape))
    assert trdq.trdq_device_status() == 0


def test_rounding_ties_on_device():
    """With Delta = 2^3.5 the fused vector is exactly +-1 and small-integer rows transform exactly.
    Rows whose absmax is 508 = 127 * 4 are scaled by exactly 1/4, so transformed values that are
    2 mod 4 land on exact halves: ties must go to the even code."""
    from paper_2503_06564_b200 import trdq
    K = 128
    signs = np.ones((1, K), np.int8)
    smooth = np.full((1, K), np.float32(2.0 ** 3.5), np.float32)
    rot = trdq.Rotation(K, [0, 1000], signs, smooth)
    x = np.zeros((5, K))
    x[0, :4] = [201, 150, 99, 58]      # transform by (i & 3): 508, 92, 194, 10  -> 127, 23, 48.5, 2.5
    x[1, :4] = [-201, -150, -99, -58]
    x[2, :2] = [255, 253]              # 508, 2 -> 127, 0.5
    x[3, :4] = [131, 130, 126, 121]    # 508, 6, 14, -4 -> 127, 1.5, 3.5, -1
    x[4, :4] = [-131, -130, -126, -121]
    xb = WL.to_bf16_bits(x)
    assert np.array_equal(WL.bf16_bits_to_f32(xb).astype(np.float64), x), "test rows must be exact in bf16"
    codes, scales = trdq.trdq_rotate_quantize(rot, 0, to_dev_bf16(xb))
    codes = codes.cpu().numpy()
    assert scales.cpu().numpy().tolist() == [4.0] * 5
    i = np.arange(K) & 3
    assert np.array_equal(codes[0], np.array([127, 23, 48, 2])[i])
    assert np.array_equal(codes[1], np.array([-127, -23, -48, -2])[i])
    assert np.array_equal(codes[2], np.array([127, 0, 127, 0])[i])
    assert np.array_equal(codes[3], np.array([127, 2, 4, -1])[i])
    assert np.array_equal(codes[4], np.array([-127, -2, -4, 1])[i])
    act, _ = O.fused_vectors(signs[0], smooth[0])
    assert np.all(act == np.float32(1.0))
    c_ref, s_ref = O.rotate_quantize(xb, act)
    assert np.array_equal(codes, c_ref) and np.array_equal(scales.cpu().numpy(), s_ref)


@pytest.mark.parametrize("N,K,G", [(1024, 1024, 2), (1152, 1152, 3), (272, 4608, 2), (16, 128, 1)])
def test_prepare_weights_w8_matches_oracle(N, K, G):
    from paper_2503_06564_b200 import trdq
    rot, signs, sm, _ = _rot(K, G, 21 + N, True)
    rng = np.random.default_rng(N + K)
    w = WL.to_bf16_bits(rng.standard_normal((N, K)) * 0.02)
    wts = trdq.trdq_prepare_weights(rot, to_dev_bf16(w), 8)
    assert (wts.N, wts.K, wts.wbits, wts.num_groups) == (N, K, 8, G)
    for g in range(G):
        _, wv = O.fused_vectors(signs[g], sm[g])
        c_ref, s_ref = O.prepare_w8(w, wv)
        codes, scales = wts.view_tensors(g)
        assert np.array_equal(scales.cpu().numpy(), s_ref)
        assert np.array_equal(codes.cpu().numpy(), c_ref)


@pytest.mark.parametrize("N,K,G", [(1152, 1152, 2), (144, 4608, 1), (16, 256, 2)])
def test_prepare_weights_w4_matches_oracle(N, K, G):
    from paper_2503_06564_b200 import trdq
    rot, signs, sm, _ = _rot(K, G, 31 + N, True)
    rng = np.random.default_rng(N + K + 1)
    w = WL.to_bf16_bits(rng.standard_normal((N, K)) * 0.02)
    wts = trdq.trdq_prepare_weights(rot, to_dev_bf16(w), 4)
    for g in range(G):
        _, wv = O.fused_vectors(signs[g], sm[g])
        p_ref, s_ref = O.prepare_w4(w, wv)
        packed, scales = wts.view_tensors(g)
        assert np.array_equal(scales.cpu().numpy(), s_ref)
        assert np.array_equal(packed.cpu().numpy(), p_ref)


def test_argument_errors_are_reported_not_launched():
    import torch
    from paper_2503_06564_b200 import trdq
    rot, *_ = _rot(256, 2, 1, False)
    x = torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_rotate_quantize(rot, 1000, x)
    assert e.value.status == 4
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_rotate_quantize(rot, -1, x)
    assert e.value.status == 4
    flat = torch.zeros(4 * 256 + 8, dtype=torch.bfloat16, device="cuda")
    mis = flat[1:1 + 4 * 256].view(4, 256)          # 2-byte offset: not 16-byte aligned
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_rotate_quantize(rot, 0, mis)
    assert e.value.status == 3
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_prepare_weights(rot, torch.zeros((24, 256), dtype=torch.bfloat16, device="cuda"), 8)   # N % 16
    assert e.value.status == 2
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_prepare_weights(rot, torch.zeros((32, 256), dtype=torch.bfloat16, device="cuda"), 6)
    assert e.value.status == 6
