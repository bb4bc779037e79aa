"""Pins for the CPU oracle: every check compares it with something other than itself
(a textbook definition, a closed form, an invariant the paper states, a library
routine it does not use, or brute force on tiny inputs)."""
import os

import numpy as np
import pytest

from oracle import trdq_oracle as O
from paper_2503_06564_b200 import workloads as WL

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
C_NORM = 2.0 ** -3.5


def bf16(x):
    return WL.to_bf16_bits(np.asarray(x, dtype=np.float64))


def f32_of(bits):
    return WL.bf16_bits_to_f32(bits)


def unit_vectors(K=128):
    return bf16(np.eye(K))


def identity_vec_smooth():
    """smooth value that makes the fused *activation* vector exactly +-1.0f."""
    return np.float32(2.0 ** 3.5)


# --------------------------------------------------------------------------- #
# rotation (Eq. 8, Eq. 10)
# --------------------------------------------------------------------------- #
def test_fused_vectors_values():
    rng = np.random.default_rng(1)
    K = 256
    signs = (rng.integers(0, 2, K) * 2 - 1).astype(np.int8)
    a, b = O.fused_vectors(signs, None)
    # Delta = 1: both vectors are d * 2^-3.5 rounded to fp32
    assert np.array_equal(a, b)
    assert np.array_equal(np.sign(a).astype(np.int8), signs)
    assert np.allclose(a.astype(np.float64) ** 2 * 128.0, 1.0, rtol=2e-7)
    smooth = rng.uniform(0.05, 20.0, K).astype(np.float32)
    a, b = O.fused_vectors(signs, smooth)
    # act carries Delta, weight carries 1/Delta: a*b = 1/128, a/b = Delta^2
    assert np.allclose(a.astype(np.float64) * b.astype(np.float64) * 128.0, 1.0, rtol=3e-7)
    assert np.allclose(a.astype(np.float64) / b.astype(np.float64), smooth.astype(np.float64) ** 2, rtol=3e-7)
    assert np.array_equal(np.sign(a).astype(np.int8), signs)
    assert np.array_equal(np.sign(b).astype(np.int8), signs)


def test_unit_act_vector_trick():
    signs = np.ones(128, np.int8)
    a, _ = O.fused_vectors(signs, np.full(128, identity_vec_smooth(), np.float32))
    assert np.all(a == np.float32(1.0))
    _, b = O.fused_vectors(signs, np.full(128, np.float32(2.0 ** -3.5), np.float32))
    assert np.all(b == np.float32(1.0))


def test_butterfly_is_sylvester_natural_order():
    """Row j of the transform of the identity is (-1)^popcount(i & j): natural order, no bit reversal."""
    ones = np.ones(128, np.float32)
    v = O.rotate(unit_vectors(), ones)          # v[j, i] = H[j][i]
    i = np.arange(128)
    pop = np.array([[bin(a & b).count("1") for a in i] for b in i])
    assert np.array_equal(v, ((-1.0) ** pop).astype(np.float32))
    golden = np.loadtxt(os.path.join(GOLDEN, "hadamard8_sylvester.txt"))
    assert np.array_equal(v[:8, :8], golden.astype(np.float32))


def test_butterfly_closed_forms():
    ones = np.ones(128, np.float32)
    x = np.zeros((3, 128))
    x[0, 0] = 3.0            # H(alpha e0) = alpha * ones
    x[1, :] = 1.0            # H(ones) = 128 e0
    x[2, 5] = -2.0
    v = O.rotate(bf16(x), ones)
    assert np.array_equal(v[0], np.full(128, 3.0, np.float32))
    e0 = np.zeros(128, np.float32); e0[0] = 128.0
    assert np.array_equal(v[1], e0)
    # involution: H(H(x)) = 128 x  (values stay small integers => exact in bf16/fp32)
    rng = np.random.default_rng(7)
    xi = rng.integers(-1, 2, size=(4, 128)).astype(np.float64)
    once = O.rotate(bf16(xi), ones)
    assert np.all(np.abs(once) <= 128)
    twice = O.rotate(bf16(once.astype(np.float64) / 128.0), ones)   # /128 exact; bf16 holds k/128, |k|<=128
    assert np.array_equal(twice, xi.astype(np.float32))


def test_dense_rotation_is_orthogonal():
    rng = np.random.default_rng(3)
    K = 384
    signs = (rng.integers(0, 2, K) * 2 - 1).astype(np.int8)
    R = O.dense_rotation(signs)
    assert np.max(np.abs(R @ R.T - np.eye(K))) < 1e-6
    assert np.max(np.abs(R.T @ R - np.eye(K))) < 1e-6
    # block-diagonal: nothing outside the 128 x 128 diagonal blocks
    mask = np.kron(np.eye(K // 128), np.ones((128, 128))) > 0
    assert np.all(R[~mask] == 0.0)
    assert np.allclose(np.abs(R[mask]), C_NORM)


def test_computational_invariance_fp64():
    """(X Delta R)(R^T Delta^-1 W) = X W  (Eq. 9 / Eq. 10) in double to 1e-10."""
    rng = np.random.default_rng(4)
    M, K, N = 8, 256, 24
    signs = (rng.integers(0, 2, K) * 2 - 1).astype(np.int8)
    delta = rng.uniform(0.1, 8.0, K)
    X = rng.standard_normal((M, K))
    W = rng.standard_normal((K, N))            # paper orientation: C_in x C_out
    R = O.dense_rotation(signs)
    G = O.matmul_f64(X * delta[None, :], R)
    H = O.matmul_f64(np.ascontiguousarray(R.T), W / delta[:, None])
    Y = O.matmul_f64(G, H)
    ref = X @ W
    assert np.max(np.abs(Y - ref)) / np.max(np.abs(ref)) < 1e-10


def test_butterfly_matches_dense_fp64_product():
    """fp32 butterfly vs. the fp64 dense product, within the fp32 summation bound."""
    rng = np.random.default_rng(5)
    M, K = 16, 384
    signs = (rng.integers(0, 2, K) * 2 - 1).astype(np.int8)
    smooth = rng.uniform(0.2, 5.0, K).astype(np.float32)
    xb = bf16(rng.standard_normal((M, K)) * 3.0)
    a, b = O.fused_vectors(signs, smooth)
    v = O.rotate(xb, a).astype(np.float64)
    x = f32_of(xb).astype(np.float64)
    R = O.dense_rotation(signs)
    dense = (x * smooth.astype(np.float64)[None, :]) @ R
    # bound: 8 roundings along each path, each relative 2^-24, on sum_j |x_j a_j|
    mag = np.abs(x * a.astype(np.float64)[None, :]).reshape(M, K // 128, 128).sum(axis=2)
    bound = np.repeat(mag, 128, axis=1) * 128 * 2.0 ** -24 + 1e-12
    assert np.all(np.abs(v - dense) <= bound)
    assert np.max(np.abs(v - dense)) > 0      # the two paths are really different computations
    # weight side uses 1/Delta
    vw = O.rotate(xb, b).astype(np.float64)
    dense_w = (x / smooth.astype(np.float64)[None, :]) @ R
    assert np.all(np.abs(vw - dense_w) <= np.repeat(
        np.abs(x * b.astype(np.float64)[None, :]).reshape(M, K // 128, 128).sum(axis=2), 128, axis=1) * 128 * 2.0 ** -24 + 1e-12)


def test_block_diagonal_locality():
    rng = np.random.default_rng(6)
    K = 512
    a, _ = O.fused_vectors(np.ones(K, np.int8), None)
    x = rng.standard_normal((1, K))
    x2 = x.copy()
    x2[0, 128 + 17] += 5.0
    v1 = O.rotate(bf16(x), a)
    v2 = O.rotate(bf16(x2), a)
    changed = np.nonzero(v1[0] != v2[0])[0]
    assert changed.min() >= 128 and changed.max() < 256 and changed.size == 128


# --------------------------------------------------------------------------- #
# quantizer (Eq. 1-2, symmetric signed form; per token)
# --------------------------------------------------------------------------- #
def test_quantizer_error_bound_and_extremes():
    rng = np.random.default_rng(8)
    v = (rng.standard_normal((64, 256)) * rng.uniform(0.01, 100.0, (64, 1))).astype(np.float32)
    q, s = O.quantize_rows(v)
    assert q.dtype == np.int8 and s.shape == (64,)
    amax = np.abs(v).max(axis=1)
    assert np.allclose(s.astype(np.float64) * 127.0, amax.astype(np.float64), rtol=1e-6)
    err = np.abs(v.astype(np.float64) - s.astype(np.float64)[:, None] * q.astype(np.float64))
    assert np.all(err <= s.astype(np.float64)[:, None] * (0.5 + 1e-5))
    assert q.min() >= -127 and q.max() <= 127
    rows = np.arange(64)
    arg = np.abs(v).argmax(axis=1)
    assert np.all(np.abs(q[rows, arg]) == 127)
    assert np.array_equal(np.sign(q[rows, arg]), np.sign(v[rows, arg]).astype(np.int8))


def test_quantizer_zero_row_and_row_independence():
    rng = np.random.default_rng(9)
    v = rng.standard_normal((5, 128)).astype(np.float32)
    v[2] = 0.0
    q, s = O.quantize_rows(v)
    assert s[2] == 0.0 and np.all(q[2] == 0)
    # dynamic per-token scale: a row's result does not depend on the other rows
    perm = np.array([4, 0, 3, 1, 2])
    q2, s2 = O.quantize_rows(v[perm])
    assert np.array_equal(q2, q[perm]) and np.array_equal(s2, s[perm])
    v3 = v.copy(); v3[0] *= 1000.0
    q3, s3 = O.quantize_rows(v3)
    assert np.array_equal(q3[1:], q[1:]) and np.array_equal(s3[1:], s[1:])


def test_quantizer_round_half_to_even():
    table = np.loadtxt(os.path.join(GOLDEN, "rounding_ties.txt"))
    vals, expect = table[:, 0], table[:, 1].astype(np.int64)
    for p in (-3, 0, 5):
        row = np.zeros(128, np.float32)
        row[0] = 127.0 * 2.0 ** p           # absmax => inverse scale is exactly 2^-p
        row[1:1 + vals.size] = (vals * 2.0 ** p).astype(np.float32)
        q, s = O.quantize_rows(row[None, :])
        assert s[0] == np.float32(2.0 ** p)
        assert q[0, 0] == 127
        assert np.array_equal(q[0, 1:1 + vals.size].astype(np.int64), expect)


def test_rotate_quantize_equals_its_two_steps():
    rng = np.random.default_rng(10)
    xb = bf16(rng.standard_normal((9, 256)))
    a, _ = O.fused_vectors((rng.integers(0, 2, 256) * 2 - 1).astype(np.int8), None)
    q, s = O.rotate_quantize(xb, a)
    q2, s2 = O.quantize_rows(O.rotate(xb, a))
    assert np.array_equal(q, q2) and np.array_equal(s, s2)


# --------------------------------------------------------------------------- #
# integer GEMM and epilogue (Eq. 10)
# --------------------------------------------------------------------------- #
def test_int_gemm_brute_force_and_numpy():
    q = np.array([[1, -2, 3, 4], [127, 127, -127, 0]], np.int8)
    w = np.array([[1, 1, 1, 1], [0, -1, 2, -3], [127, 127, -127, 5]], np.int8)
    acc = O.gemm_i32(q, w)
    # written out by hand
    assert acc.tolist() == [[6, -4, -488], [127, -381, 48387]]
    rng = np.random.default_rng(11)
    q = rng.integers(-127, 128, (37, 384), dtype=np.int8)
    w = rng.integers(-127, 128, (29, 384), dtype=np.int8)
    assert np.array_equal(O.gemm_i32(q, w).astype(np.int64), q.astype(np.int64) @ w.astype(np.int64).T)
    # extreme magnitude stays exact in int32
    q = np.full((1, 4096), 127, np.int8); w = np.full((1, 4096), -127, np.int8)
    assert O.gemm_i32(q, w)[0, 0] == -4096 * 127 * 127


def test_epilogue_special_cases():
    rng = np.random.default_rng(12)
    acc = rng.integers(-256, 257, (6, 10)).astype(np.int32)
    ones_m, ones_n = np.ones(6, np.float32), np.ones(10, np.float32)
    assert np.array_equal(O.epilogue(acc, ones_m, ones_n, None), acc.astype(np.float32))
    bias = bf16(rng.standard_normal(10))
    y = O.epilogue(np.zeros((6, 10), np.int32), ones_m, ones_n, bias)
    assert np.array_equal(y, np.broadcast_to(f32_of(bias), (6, 10)))
    # per-token scale acts on rows, per-channel scale on columns (powers of two: exact)
    sx = np.array([1, 2, 4, 8, 16, 32], np.float32)
    sw = (2.0 ** -np.arange(10)).astype(np.float32)
    y = O.epilogue(acc, sx, sw, None)
    assert np.array_equal(y, (acc * sx[:, None] * sw[None, :]).astype(np.float32))
    y_rows = O.linear_w8_rows(np.eye(6, 128, dtype=np.int8), sx, np.ones((10, 128), np.int8), sw, None, np.array([5, 0]))
    assert np.array_equal(y_rows, np.stack([32.0 * sw, 1.0 * sw]).astype(np.float32))


def _w8a8(xb, wb, biasb, signs, smooth):
    a, b = O.fused_vectors(signs, smooth)
    q, sx = O.rotate_quantize(xb, a)
    qw, sw = O.prepare_w8(wb, b)
    return O.epilogue(O.gemm_i32(q, qw), sx, sw, biasb)


def test_end_to_end_close_to_fp64_linear():
    """The whole quantised path reproduces X W + bias up to quantisation noise (Eq. 10)."""
    wl = WL.WORKLOADS[0]
    li = WL.make_layer_inputs(wl, 0, M=32)
    x = f32_of(li.x).astype(np.float64); w = f32_of(li.w).astype(np.float64)
    ref = x @ w.T + f32_of(li.bias).astype(np.float64)[None, :]
    rng = np.random.default_rng(13)
    smooth = rng.uniform(0.5, 2.0, (1, li.layer.K)).astype(np.float32)
    for sm in (None, smooth[0]):
        y = _w8a8(li.x, li.w, li.bias, li.signs[0], sm).astype(np.float64)
        rel = np.linalg.norm(y - ref) / np.linalg.norm(ref)
        assert rel < 0.02, rel
    rows = np.array([3, 31, 0])
    a, b = O.fused_vectors(li.signs[1], None)
    q, sx = O.rotate_quantize(li.x, a); qw, sw = O.prepare_w8(li.w, b)
    full = O.epilogue(O.gemm_i32(q, qw), sx, sw, li.bias)
    assert np.array_equal(O.linear_w8_rows(q, sx, qw, sw, li.bias, rows), full[rows])


def test_rotation_reduces_outliers_and_error():
    """Sec. 3.2: rotation spreads massive outliers, shrinking the per-token range and the W8A8 error."""
    wl = WL.WORKLOADS[0]
    li = WL.make_layer_inputs(wl, 0, M=64)
    x = f32_of(li.x).astype(np.float64); w = f32_of(li.w).astype(np.float64)
    a, b = O.fused_vectors(li.signs[0], None)
    v = O.rotate(li.x, a)
    before = np.abs(x).max(axis=1).mean()
    after = np.abs(v).max(axis=1).mean()
    assert before / after > 3.0
    ref = x @ w.T
    y_rot = O.epilogue(O.gemm_i32(*[t for t in (O.rotate_quantize(li.x, a)[0], O.prepare_w8(li.w, b)[0])]),
                       O.rotate_quantize(li.x, a)[1], O.prepare_w8(li.w, b)[1], None)
    qx, sx = O.quantize_rows(f32_of(li.x)); qw, sw = O.quantize_rows(f32_of(li.w))
    y_plain = O.epilogue(O.gemm_i32(qx, qw), sx, sw, None)
    e_rot = np.linalg.norm(y_rot - ref); e_plain = np.linalg.norm(y_plain - ref)
    assert e_rot < 0.5 * e_plain


# --------------------------------------------------------------------------- #
# 4-bit weights
# --------------------------------------------------------------------------- #
def _w4_rows_for_pairs():
    """Rows whose rotated values are the period-4 pattern (a, b, +-7, r): exact small numbers."""
    pairs = [(a, b) for a in range(-7, 8) for b in range(-7, 8)]
    idx = np.arange(128)
    s = np.zeros((len(pairs), 128))
    for r, (a, b) in enumerate(pairs):
        s2 = (a - 7) / 2.0 if b <= a else (a + 7) / 2.0
        s[r, 1] = (a - b) / 2.0
        s[r, 2] = s2
        s[r, 0] = (a + b) / 2.0 - s2
    return pairs, s


def test_w4_pack_exhaustive_nibble_pairs():
    pairs, s = _w4_rows_for_pairs()
    _, wvec = O.fused_vectors(np.ones(128, np.int8), np.full(128, np.float32(2.0 ** -3.5), np.float32))
    assert np.all(wvec == np.float32(1.0))
    sb = bf16(s)
    assert np.array_equal(f32_of(sb).astype(np.float64), s)      # inputs are exact in bf16
    v = O.rotate(sb, wvec)
    packed, scales = O.prepare_w4(sb, wvec)
    assert packed.shape == (len(pairs), 64) and scales.shape == (len(pairs), 1)
    assert np.all(scales == np.float32(1.0))
    for r, (a, b) in enumerate(pairs):
        assert v[r, 0] == a and v[r, 1] == b and abs(v[r, 2]) == 7
        assert packed[r, 0] == ((a & 0xF) | ((b & 0xF) << 4))
        assert packed[r, 1] == ((int(v[r, 2]) & 0xF) | ((int(v[r, 3]) & 0xF) << 4))
    assert np.array_equal(O.unpack_w4(packed).astype(np.float32), v)


def test_w4_group_scales_and_linear():
    rng = np.random.default_rng(14)
    N, K, M = 12, 384, 7
    wb = bf16(rng.standard_normal((N, K)) * 0.02)
    signs = (rng.integers(0, 2, K) * 2 - 1).astype(np.int8)
    a, b = O.fused_vectors(signs, None)
    packed, sw4 = O.prepare_w4(wb, b)
    v = O.rotate(wb, b).reshape(N, K // 128, 128)
    amax = np.abs(v).max(axis=2)
    assert np.allclose(sw4.astype(np.float64) * 7.0, amax.astype(np.float64), rtol=1e-6)
    q4 = O.unpack_w4(packed).reshape(N, K // 128, 128)
    assert q4.min() >= -7 and q4.max() <= 7
    assert np.all(np.abs(v - sw4[:, :, None] * q4) <= sw4[:, :, None] * (0.5 + 1e-5))
    # linear: sum over k-groups of exact int partials times the group scale
    xb = bf16(rng.standard_normal((M, K)))
    q, sx = O.rotate_quantize(xb, a)
    bias = bf16(rng.standard_normal(N) * 0.01)
    y = O.linear_w4_rows(q, sx, packed, sw4, bias, np.arange(M))
    deq = (q4.astype(np.float64) * sw4.astype(np.float64)[:, :, None]).reshape(N, K)
    ref = sx.astype(np.float64)[:, None] * (q.astype(np.float64) @ deq.T) + f32_of(bias).astype(np.float64)[None, :]
    assert np.allclose(y, ref, rtol=1e-6, atol=1e-9)
    x = f32_of(xb).astype(np.float64); w = f32_of(wb).astype(np.float64)
    full = x @ w.T + f32_of(bias).astype(np.float64)[None, :]
    assert np.linalg.norm(y - full) / np.linalg.norm(full) < 0.15


# --------------------------------------------------------------------------- #
# time-step groups (Sec. 3.2, Time-Rotation)
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("G", [1, 2, 3, 4, 5])
def test_group_of_exhaustive(G):
    bounds = WL.group_bounds(G)
    assert bounds[0] == 0 and bounds[-1] == 1000 and np.all(np.diff(bounds) > 0)
    t = np.arange(1000)
    got = np.array([O.group_of(bounds, int(ti)) for ti in t])
    assert np.array_equal(got, np.searchsorted(bounds, t, side="right") - 1)
    assert O.group_of(bounds, -1) == -1 and O.group_of(bounds, 1000) == -1


def test_time_step_selects_parameter_set():
    wl = WL.WORKLOADS[0]
    li = WL.make_layer_inputs(wl, 0, M=8)
    codes = {}
    for t in (0, 250, 499, 500, 750, 999):
        g = O.group_of(li.t_bounds, t)
        a, _ = O.fused_vectors(li.signs[g], None)
        codes[t] = O.rotate_quantize(li.x, a)[0]
    assert np.array_equal(codes[0], codes[250]) and np.array_equal(codes[250], codes[499])
    assert np.array_equal(codes[500], codes[750]) and np.array_equal(codes[750], codes[999])
    assert not np.array_equal(codes[499], codes[500])


# --------------------------------------------------------------------------- #
# full balancing transform (Eq. 9): second rotation after the zigzag permutation
# --------------------------------------------------------------------------- #
def _full_setup(K, seed, with_smooth=True):
    rng = np.random.default_rng(seed)
    d1 = (rng.integers(0, 2, K) * 2 - 1).astype(np.int8)
    d2 = (rng.integers(0, 2, K) * 2 - 1).astype(np.int8)
    smooth = rng.uniform(0.25, 4.0, K).astype(np.float32) if with_smooth else None
    perm = rng.permutation(K).astype(np.int32)
    return d1, d2, smooth, perm


def test_zigzag_is_the_serpentine_deal():
    """Sec. 3.2: highest channel to the first block, next ones to the following blocks, direction reversing at
    the last block.  Slot r of every block therefore holds the channels ranked r*B .. r*B+B-1, in block order
    on even rounds and in reverse block order on odd rounds."""
    rng = np.random.default_rng(5)
    for K in (256, 1152):
        B = K // 128
        mag = rng.gamma(2.0, 1.0, K).astype(np.float32)
        perm = O.zigzag_permutation(mag)
        assert sorted(perm.tolist()) == list(range(K))                       # a permutation
        rank = np.empty(K, np.int64)
        rank[np.argsort(-mag.astype(np.float64), kind="stable")] = np.arange(K)
        slots = rank[perm].reshape(B, 128)                                   # rank of the channel in (block, slot)
        for r in range(128):
            expect = np.arange(r * B, (r + 1) * B)
            assert np.array_equal(slots[:, r], expect if r % 2 == 0 else expect[::-1])
        # balance: block totals differ by less than the spread of single channels, unlike a contiguous deal
        sums = mag[perm].astype(np.float64).reshape(B, 128).sum(axis=1)
        contiguous = np.sort(mag.astype(np.float64))[::-1].reshape(B, 128).sum(axis=1)
        assert sums.max() - sums.min() <= mag.max() - mag.min()
        assert sums.max() - sums.min() < 0.05 * (contiguous.max() - contiguous.min())
    # a hand-checkable case: two blocks, magnitudes descending with the channel index
    perm = O.zigzag_permutation(np.arange(256, 0, -1).astype(np.float32))
    assert perm[:4].tolist() == [0, 3, 4, 7] and perm[128:132].tolist() == [1, 2, 5, 6]


def test_permutation_and_full_rotation_are_orthogonal():
    K = 256
    d1, d2, _, perm = _full_setup(K, 11)
    P = O.dense_permutation(perm)
    assert np.array_equal(P @ P.T, np.eye(K)) and np.array_equal(P.sum(axis=0), np.ones(K))
    v = np.arange(K, dtype=np.float64)
    assert np.array_equal(v @ P, v[perm])                                    # (v P)[j] = v[perm[j]]
    R = O.dense_rotation(d1) @ P @ O.dense_rotation(d2)
    assert np.abs(R @ R.T - np.eye(K)).max() < 1e-6


def test_full_transform_invariance_fp64():
    """Eq. 9: [(X Delta) R1 P R2] . [R2^T P^T R1^T (Delta^-1 W)] = X W."""
    K, M, N = 256, 6, 5
    d1, d2, smooth, perm = _full_setup(K, 12)
    rng = np.random.default_rng(3)
    X = rng.standard_normal((M, K))
    W = rng.standard_normal((K, N))
    R = O.dense_rotation(d1) @ O.dense_permutation(perm) @ O.dense_rotation(d2)
    delta = smooth.astype(np.float64)
    G = O.matmul_f64(X * delta, R)
    H = O.matmul_f64(np.ascontiguousarray(R.T), W / delta[:, None])
    ref = X @ W
    assert np.abs(O.matmul_f64(G, H) - ref).max() <= 1e-10 * np.abs(ref).max()


def test_rotate2_matches_dense_fp64_and_its_parts():
    K, M = 384, 9
    d1, d2, smooth, perm = _full_setup(K, 13)
    x = bf16(np.random.default_rng(8).standard_normal((M, K)) * 3.0)
    a1, _ = O.fused_vectors(d1, smooth)
    a2 = O.second_vector(d2, K)
    assert np.array_equal(a2, (d2.astype(np.float64) * C_NORM).astype(np.float32))
    v = O.rotate2(x, a1, perm, a2)
    R = O.dense_rotation(d1) @ O.dense_permutation(perm) @ O.dense_rotation(d2)
    ref = (f32_of(x).astype(np.float64) * smooth.astype(np.float64)) @ R
    bound = 4.0 * 128 * 2.0 ** -24 * np.abs(ref).max() * np.sqrt(128)
    assert np.abs(v - ref).max() <= bound
    # composition of the single-stage pieces: rotate, gather by perm, scale, rotate
    v1 = O.rotate(x, a1)
    v2 = (v1[:, perm] * a2[None, :]).astype(np.float32)
    ones = np.ones(K, np.float32)
    # feed v2 through the butterfly with a unit vector: v2 is fp32, not bf16, so compare block by block via the dense H
    Hm = O.rotate(unit_vectors(128), np.ones(128, np.float32)).astype(np.float64)
    ref2 = np.concatenate([v2[:, c:c + 128].astype(np.float64) @ Hm for c in range(0, K, 128)], axis=1)
    assert np.abs(v - ref2).max() <= 128 * 2.0 ** -23 * np.abs(ref2).max()
    codes, scales = O.rotate2_quantize(x, a1, perm, a2)
    c2, s2 = O.quantize_rows(v)
    assert np.array_equal(codes, c2) and np.array_equal(scales, s2)


def test_full_transform_identity_special_case():
    """perm = identity, d2 = +1, Delta = 1: (H/sqrt(128))^2 = I, so G(X) = X diag(d1) up to fp32 rounding."""
    K = 256
    rng = np.random.default_rng(2)
    d1 = (rng.integers(0, 2, K) * 2 - 1).astype(np.int8)
    x = bf16(rng.standard_normal((4, K)))
    a1, _ = O.fused_vectors(d1, None)
    v = O.rotate2(x, a1, np.arange(K, dtype=np.int32), O.second_vector(None, K))
    ref = f32_of(x).astype(np.float64) * d1
    assert np.abs(v - ref).max() <= 2.0 ** -20 * np.abs(ref).max()


def test_second_rotation_balances_blocks():
    """Sec. 3.2: after the first rotation outliers are spread inside their block only; the zigzag permutation
    deals strong channels over all blocks and the second rotation flattens them further."""
    K, M = 1024, 64
    rng = np.random.default_rng(21)
    x = rng.standard_normal((M, K))
    x[:, :128] *= 20.0                                  # one whole block is hot
    xb = bf16(x)
    d1, d2, _, _ = _full_setup(K, 14, with_smooth=False)
    a1, _ = O.fused_vectors(d1, None)
    v1 = O.rotate(xb, a1)
    perm = O.zigzag_permutation(np.abs(v1).max(axis=0))
    v3 = O.rotate2(xb, a1, perm, O.second_vector(d2, K))
    assert np.abs(v3).max(axis=1).mean() < 0.6 * np.abs(v1).max(axis=1).mean()
    # quantisation error of the rows drops accordingly
    def rel_err(v):
        q, s = O.quantize_rows(v)
        return np.linalg.norm(q * s[:, None] - v) / np.linalg.norm(v)
    assert rel_err(v3) < 0.7 * rel_err(v1)


# --------------------------------------------------------------------------- #
# literal asymmetric quantizer (Eq. 1-3)
# --------------------------------------------------------------------------- #
def test_asymmetric_quantizer_eq1_to_eq3():
    rng = np.random.default_rng(31)
    v = (rng.standard_normal((40, 256)) * rng.uniform(0.1, 30.0, (40, 1)) + rng.uniform(-5, 5, (40, 1))).astype(np.float32)
    q, s, z = O.quantize_rows_asym(v)
    assert q.dtype == np.uint8
    rng_ = v.max(axis=1) - v.min(axis=1)
    assert np.array_equal(s, (rng_ / np.float32(255.0)).astype(np.float32))               # Eq. 2
    deq = s[:, None].astype(np.float64) * (q.astype(np.float64) - z[:, None])
    # nearest rounding (Eq. 1): error at most half a step, plus the half step the zero point itself was rounded by
    assert np.all(np.abs(deq - v) <= s[:, None].astype(np.float64) * (1.0 + 1e-4))
    # the minimum maps to code 0 and the maximum to 255 (Eq. 1-3 with z = -round(min / s))
    assert np.all(q[np.arange(40), v.argmin(axis=1)] == 0) and np.all(q[np.arange(40), v.argmax(axis=1)] == 255)
    # z is where the real value 0 lands
    zero_code = np.rint(0.0 * 0 + z)
    assert np.all(np.abs(s * (zero_code - z)) == 0)
    # a closed-form case: values 0..255 -> s = 1, z = 0, codes = values; shifted by -100: z = 100
    ramp = np.arange(256, dtype=np.float32)[None, :]
    q1, s1, z1 = O.quantize_rows_asym(ramp)
    assert s1[0] == 1.0 and z1[0] == 0 and np.array_equal(q1[0], np.arange(256))
    q2, s2, z2 = O.quantize_rows_asym(ramp - 100.0)
    assert s2[0] == 1.0 and z2[0] == 100 and np.array_equal(q2[0], np.arange(256))
    # ties go to the even integer: range 510 -> inv = 0.5, values 2k+1 land on halves
    odd = np.array([[0.0, 1.0, 3.0, 5.0, 510.0]], np.float32)
    q3, s3, z3 = O.quantize_rows_asym(odd)
    assert s3[0] == 2.0 and z3[0] == 0 and q3[0].tolist() == [0, 0, 2, 2, 255]
    # constant row
    q4, s4, z4 = O.quantize_rows_asym(np.full((1, 128), 3.5, np.float32))
    assert s4[0] == 0.0 and z4[0] == 0 and not q4.any()


def test_asymmetric_linear_brute_force_and_accuracy():
    rng = np.random.default_rng(32)
    M, N, K = 6, 5, 128
    q = rng.integers(0, 256, (M, K)).astype(np.uint8)
    z = rng.integers(0, 256, M).astype(np.int32)
    qw = rng.integers(-127, 128, (N, K)).astype(np.int8)
    sx = rng.uniform(0.01, 0.1, M).astype(np.float32)
    sw = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    y = O.linear_asym_rows(q, sx, z, qw, sw, None, np.arange(M))
    ref = ((q.astype(np.int64) - z[:, None]) @ qw.astype(np.int64).T).astype(np.float64) * sx[:, None] * sw[None, :]
    assert np.allclose(y, ref, rtol=1e-6, atol=0)
    # equals the "accumulate unsigned codes, subtract z * column sums" form used on the tensor cores
    acc_u = q.astype(np.int64) @ qw.astype(np.int64).T
    colsum = qw.astype(np.int64).sum(axis=1)
    assert np.array_equal(acc_u - z[:, None] * colsum[None, :], (q.astype(np.int64) - z[:, None]) @ qw.astype(np.int64).T)
    # on shifted activations (a positive mean, as after a GELU) the asymmetric quantizer is the more accurate one
    K2 = 1024
    x = WL.to_bf16_bits(np.abs(rng.standard_normal((32, K2))) + 0.5)
    act = np.ones(K2, np.float32)
    v = O.rotate(x, act) * 0 + WL.bf16_bits_to_f32(x)          # no rotation: quantise the raw values
    qa, sa, za = O.quantize_rows_asym(v)
    qs, ss = O.quantize_rows(v)
    err_a = np.linalg.norm(sa[:, None] * (qa.astype(np.float64) - za[:, None]) - v)
    err_s = np.linalg.norm(ss[:, None] * qs.astype(np.float64) - v)
    assert err_a < 0.6 * err_s


# --------------------------------------------------------------------------- #
# dense block rotations (Eq. 6-8)
# --------------------------------------------------------------------------- #
def _random_orthogonal_blocks(nb, seed):
    rng = np.random.default_rng(seed)
    out = np.empty((nb, 128, 128), np.float32)
    for b in range(nb):
        q, r = np.linalg.qr(rng.standard_normal((128, 128)))
        out[b] = (q * np.sign(np.diag(r))).astype(np.float32)
    return out


def _sylvester(n):
    H = np.ones((1, 1))
    while H.shape[0] < n:
        H = np.block([[H, H], [H, -H]])
    return H


def test_dense_blocks_are_stored_as_nearest_bf16():
    rng = np.random.default_rng(40)
    blocks = _random_orthogonal_blocks(2, 41)
    smooth = rng.uniform(0.1, 8.0, 256).astype(np.float32)
    stored = f32_of(O.dense_stored_blocks(blocks, smooth)).astype(np.float64)
    exact = blocks.astype(np.float64) * smooth.astype(np.float64).reshape(2, 128, 1)  # row i of block b scaled by Delta[128 b + i]
    # nearest bf16: the error is at most half a unit of the last of the 8 significand bits
    ulp = 2.0 ** (np.floor(np.log2(np.abs(stored))) - 7)
    assert np.all(np.abs(stored - exact) <= ulp / 2)
    assert np.max(np.abs(stored - exact) / ulp) > 0.49            # and the bound is attained: it is not a finer format
    assert np.array_equal(bf16(stored), O.dense_stored_blocks(blocks, smooth))   # the stored values are bf16 numbers
    # without smoothing the blocks themselves are rounded
    assert np.array_equal(O.dense_stored_blocks(blocks, None), bf16(blocks))
    # ties go to even: 1 + 2^-8 lies midway between 1 and 1 + 2^-7 -> 1; 1 + 3 * 2^-8 -> 1 + 2^-6
    tie = np.zeros((1, 128, 128), np.float32)
    tie[0, 0, 0] = 1.0 + 2.0 ** -8
    tie[0, 0, 1] = 1.0 + 3 * 2.0 ** -8
    tie[0, 1, 0] = 3.0                      # times Delta = 1/3 rounded to fp32: product needs the double
    sm = np.ones(128, np.float32)
    got = f32_of(O.dense_stored_blocks(tie, sm))
    assert got[0, 0, 0] == 1.0 and got[0, 0, 1] == np.float32(1.0 + 2.0 ** -6)


def test_dense_rotation_is_the_matrix_product():
    rng = np.random.default_rng(42)
    K, M = 384, 24
    blocks = _random_orthogonal_blocks(K // 128, 43)
    smooth = rng.uniform(0.2, 5.0, K).astype(np.float32)
    stored_bits = O.dense_stored_blocks(blocks, smooth)
    S = f32_of(stored_bits).astype(np.float64)
    x_bits = bf16(rng.standard_normal((M, K)) * 3.0)
    x = f32_of(x_bits).astype(np.float64)
    v = O.rotate_dense(x_bits, stored_bits).astype(np.float64)
    ref = np.concatenate([x[:, 128 * b:128 * (b + 1)] @ S[b] for b in range(K // 128)], axis=1)  # BLAS, another summation order
    bound = np.concatenate([np.abs(x[:, 128 * b:128 * (b + 1)]) @ np.abs(S[b]) for b in range(K // 128)], axis=1)
    assert np.all(np.abs(v - ref) <= bound * 2.0 ** -23)       # one fp32 rounding of an (almost) exact sum
    # a transposed operand would fail this by O(1)
    wrong = np.concatenate([x[:, 128 * b:128 * (b + 1)] @ S[b].T for b in range(K // 128)], axis=1)
    assert np.max(np.abs(v - wrong)) > 0.5


def test_dense_rotation_with_hadamard_block_equals_the_butterfly():
    # S = H_128 / 8 is bf16-exact; with small integer rows both evaluations are exact, so the dense product must
    # equal the butterfly of the single-rotation path bit for bit (two structurally different routes).
    rng = np.random.default_rng(44)
    H = _sylvester(128)
    blocks = np.stack([H / 8.0, -H / 8.0]).astype(np.float32)
    stored = O.dense_stored_blocks(blocks, None)
    x_bits = bf16(rng.integers(-9, 10, (16, 256)).astype(np.float64))
    vec = np.concatenate([np.full(128, 0.125, np.float32), np.full(128, -0.125, np.float32)])
    assert np.array_equal(O.rotate_dense(x_bits, stored), O.rotate(x_bits, vec))


def test_dense_block_inverse_and_invariance_fp64():
    rng = np.random.default_rng(45)
    K, M, N = 256, 12, 20
    blocks = _random_orthogonal_blocks(K // 128, 46)
    smooth = rng.uniform(0.05, 20.0, K).astype(np.float32)
    stored_bits = O.dense_stored_blocks(blocks, smooth)
    S = f32_of(stored_bits).astype(np.float64)
    inv = O.invert_blocks(stored_bits)
    for b in range(K // 128):
        assert np.max(np.abs(S[b] @ inv[b] - np.eye(128))) < 1e-10
        assert np.max(np.abs(inv[b] - np.linalg.inv(S[b]))) < 1e-9 * np.max(np.abs(inv[b]))   # LAPACK's LU, not Gauss-Jordan
    # Eq. 9 / Eq. 10: (X S)(S^-1 W^T) = X W^T
    x_bits = bf16(rng.standard_normal((M, K)))
    w_bits = bf16(rng.standard_normal((N, K)) * 0.05)
    x = f32_of(x_bits).astype(np.float64)
    w = f32_of(w_bits).astype(np.float64)
    xs = np.concatenate([x[:, 128 * b:128 * (b + 1)] @ S[b] for b in range(K // 128)], axis=1)
    wr = O.prepare_dense_rotate(w_bits, inv).astype(np.float64)
    wr_ref = np.concatenate([w[:, 128 * b:128 * (b + 1)] @ np.linalg.inv(S[b]).T for b in range(K // 128)], axis=1)
    assert np.max(np.abs(wr - wr_ref)) <= 2.0 ** -22 * np.max(np.abs(wr_ref))
    y = xs @ wr.T
    y_ref = x @ w.T
    assert np.max(np.abs(y - y_ref)) <= 1e-5 * np.max(np.abs(y_ref))   # wr is rounded to fp32: 2^-24 per term
    # a singular block is reported
    bad = stored_bits.copy()
    bad[1, :, 5] = bad[1, :, 7]
    with pytest.raises(ValueError):
        O.invert_blocks(bad)


def test_quantize_w4_rows_matches_the_hadamard_path_format():
    # the stand-alone 4-bit quantiser must produce what prepare_w4 produces from the same rotated rows
    rng = np.random.default_rng(47)
    N, K = 16, 256
    signs = (rng.integers(0, 2, K) * 2 - 1).astype(np.int8)
    _, wv = O.fused_vectors(signs, None)
    w_bits = bf16(rng.standard_normal((N, K)) * 0.02)
    packed_ref, scales_ref = O.prepare_w4(w_bits, wv)
    packed, scales = O.quantize_w4_rows(O.rotate(w_bits, wv))
    assert np.array_equal(packed, packed_ref) and np.array_equal(scales, scales_ref)


def test_greedy_block_single_outlier_closed_form():
    # one massive column d, everything else zero: C1 moves it to position 0, the uniform first row of Q spreads
    # it as a / sqrt(128) over all outputs, C2 swaps two equal entries -> every entry equals a / sqrt(128).
    rng = np.random.default_rng(48)
    Mc, d = 6, 37
    a = rng.uniform(20.0, 50.0, Mc) * np.where(rng.random(Mc) < 0.5, -1.0, 1.0)
    X = np.zeros((Mc, 128))
    X[:, d] = a
    R, n, trace = O.greedy_block(X, rng.standard_normal((1, 128, 128)))
    assert n == 1
    assert np.max(np.abs(R @ R.T - np.eye(128))) < 1e-12
    Y = X @ R
    assert np.allclose(Y, np.repeat((a / np.sqrt(128.0))[:, None], 128, axis=1), rtol=0, atol=1e-12)
    assert np.isclose(trace[0], np.max(np.abs(a)) / np.sqrt(128.0))


def test_greedy_block_eq6_structure_and_eq7_choice():
    rng = np.random.default_rng(49)
    Mc, steps = 64, 6
    X = rng.standard_normal((Mc, 128))
    X[:, 11] *= 60.0
    X[:, 90] *= 25.0
    G = rng.standard_normal((steps, 128, 128))
    R, n, trace = O.greedy_block(X, G)
    assert np.max(np.abs(R @ R.T - np.eye(128))) < 1e-11            # product of orthogonal factors
    assert 1 <= n <= steps and n == int(np.argmin(trace)) + 1        # Eq. 7: the first k reaching the minimum
    assert np.isclose(np.max(np.abs(X @ R)), trace[n - 1], rtol=1e-12)
    assert trace[n - 1] < 0.25 * np.max(np.abs(X))                   # the massive outliers are gone
    # rebuild the first factor from Eq. 6 with numpy: Q by QR of [uniform row; G rows] (Gram-Schmidt up to row signs)
    d = int(np.argmax(np.max(np.abs(X), axis=0)))
    assert d == 11
    A = G[0].copy()
    A[0] = 1.0 / np.sqrt(128.0)
    q, r = np.linalg.qr(A.T)
    Q = (q * np.sign(np.diag(r))).T                                   # rows orthonormal, row 0 = +uniform
    C = np.eye(128)
    C[[0, d]] = C[[d, 0]]
    R1 = C @ Q @ C
    R_one, n_one, _ = O.greedy_block(X, G[:1])
    assert n_one == 1 and np.max(np.abs(R_one - R1)) < 1e-10


# --------------------------------------------------------------------------- #
# activation folded into the epilogue
# --------------------------------------------------------------------------- #
def test_linear_with_gelu_is_gelu_of_the_linear():
    import torch
    rng = np.random.default_rng(50)
    M, N, K = 6, 40, 128
    q = rng.integers(-127, 128, (M, K)).astype(np.int8)
    qw = rng.integers(-127, 128, (N, K)).astype(np.int8)
    sx = rng.uniform(2e-3, 8e-3, M).astype(np.float32)       # outputs spread over about [-8, 8]
    sw = rng.uniform(2e-3, 8e-3, N).astype(np.float32)
    bias = bf16(rng.standard_normal(N))
    rows = np.arange(M, dtype=np.int64)
    acc = q.astype(np.int64) @ qw.astype(np.int64).T
    pre = acc * sx.astype(np.float64)[:, None] * sw.astype(np.float64)[None, :] + f32_of(bias).astype(np.float64)[None, :]
    assert np.abs(pre).max() > 4 and np.abs(pre).min() < 0.05
    got = O.linear_w8_rows(q, sx, qw, sw, bias, rows, act=1).astype(np.float64)
    # library routine 1: torch's fp64 GELU (tanh form).  It evaluates 0.5 x (1 + tanh u) as printed, which cancels for
    # x < -4, so it pins the bulk; library routine 2: scipy's logistic function through 0.5 (1 + tanh u) = expit(2u),
    # accurate on both tails, pins the whole range.
    ref_torch = torch.nn.functional.gelu(torch.from_numpy(pre), approximate="tanh").numpy()
    bulk = pre > -4.0
    assert np.max(np.abs(got - ref_torch)[bulk] / np.maximum(np.abs(ref_torch[bulk]), 1e-30)) < 2.0 ** -22
    from scipy.special import expit
    ref = pre * expit(2.0 * np.sqrt(2.0 / np.pi) * (pre + 0.044715 * pre ** 3))
    assert np.max(np.abs(got - ref) / np.maximum(np.abs(ref), 1e-300)) < 2.0 ** -22
    assert np.min(pre) < -6.0 and np.min(np.abs(ref)) < 1e-10          # the deep tail is in the sample
    assert np.array_equal(O.linear_w8_rows(q, sx, qw, sw, bias, rows, act=0), pre.astype(np.float32))
    # closed-form anchors of the function itself: gelu(0) = 0, gelu(x) -> x for large x, -> 0 for very negative x,
    # and gelu(x) - gelu(-x) = x
    one = np.ones((1, 1), np.int8)
    for x in (0.0, 12.0, -12.0, 0.75):
        s = np.float32(abs(x)) if x != 0 else np.float32(0.0)
        y_pos = O.linear_w8_rows(one * (1 if x >= 0 else -1), [s], one, [1.0], None, [0], act=1)[0, 0]
        y_neg = O.linear_w8_rows(one * (-1 if x >= 0 else 1), [s], one, [1.0], None, [0], act=1)[0, 0]
        assert abs((y_pos - y_neg) - x) <= 1e-6 * max(1.0, abs(x))
    assert O.linear_w8_rows(one, [12.0], one, [1.0], None, [0], act=1)[0, 0] == np.float32(12.0)
    assert abs(O.linear_w8_rows(-one, [12.0], one, [1.0], None, [0], act=1)[0, 0]) < 1e-30


# --------------------------------------------------------------------------- #
# LayerNorm + modulation folded in front of the rotation
# --------------------------------------------------------------------------- #
def test_norm_modulate_is_layer_norm_then_modulation():
    import torch
    rng = np.random.default_rng(51)
    M, K, rps, eps = 12, 256, 4, 1e-6
    x_bits = bf16(rng.standard_normal((M, K)) * 3.0 + 1.5)
    shift_bits = bf16(rng.standard_normal((M // rps, K)) * 0.3)
    scale_bits = bf16(rng.standard_normal((M // rps, K)) * 0.3)
    x = torch.from_numpy(f32_of(x_bits).astype(np.float64))
    ln = torch.nn.functional.layer_norm(x, (K,), eps=eps).numpy()                      # library routine, fp64
    sc = np.repeat(f32_of(scale_bits).astype(np.float64), rps, axis=0)
    sh = np.repeat(f32_of(shift_bits).astype(np.float64), rps, axis=0)
    ref = ln * (1.0 + sc) + sh
    h = O.norm_modulate(x_bits, shift_bits, scale_bits, rps, eps).astype(np.float64)
    assert np.max(np.abs(h - ref)) <= 2.0 ** -23 * np.max(np.abs(ref))
    # without modulation it is the plain normalisation: zero mean, unit variance
    h0 = O.norm_modulate(x_bits, None, None, rps, eps).astype(np.float64)
    assert np.max(np.abs(h0 - ln)) <= 2.0 ** -22 and np.max(np.abs(h0.mean(axis=1))) < 1e-6
    assert np.max(np.abs(h0.var(axis=1) - 1.0)) < 1e-5
    # a constant row has no deviation: the output is the shift; scale = -1 removes the normalised part as well
    const = bf16(np.full((rps, K), 2.5))
    assert np.array_equal(O.norm_modulate(const, shift_bits[:1], scale_bits[:1], rps, eps), np.repeat(f32_of(shift_bits[:1]), rps, axis=0))
    minus_one = bf16(np.full((1, K), -1.0))
    assert np.array_equal(O.norm_modulate(x_bits[:rps], shift_bits[:1], minus_one, rps, eps), np.repeat(f32_of(shift_bits[:1]), rps, axis=0))
    # the sample index: rows of the second sample use the second modulation row
    swapped = O.norm_modulate(x_bits[rps:2 * rps], shift_bits[1:2], scale_bits[1:2], rps, eps)
    assert np.array_equal(swapped, O.norm_modulate(x_bits, shift_bits, scale_bits, rps, eps)[rps:2 * rps])


def test_rotate_f32_equals_rotate_on_bf16_values():
    rng = np.random.default_rng(52)
    x_bits = bf16(rng.standard_normal((5, 384)))
    signs = (rng.integers(0, 2, 384) * 2 - 1).astype(np.int8)
    a, _ = O.fused_vectors(signs, rng.uniform(0.5, 2.0, 384).astype(np.float32))
    assert np.array_equal(O.rotate_f32(f32_of(x_bits), a), O.rotate(x_bits, a))


# --------------------------------------------------------------------------- #
# composite entry points used only by the GPU parity tests
# --------------------------------------------------------------------------- #
def test_prepare2_w4_closed_form_and_composition():
    """Weight side of Eq. 9 with 4-bit storage.  A weight row that is a scaled Hadamard row per block becomes a single spike
    after the first rotation; the permutation moves the spike (to another block), and the second rotation spreads it into a
    block of equal magnitudes, so every code is +-7 with the sign pattern of one Hadamard column: a closed form that a wrong
    permutation direction, nibble order or scale stride breaks."""
    K = 256
    unit_w = np.full(K, np.float32(2.0 ** -3.5), np.float32)          # weight vector d / Delta * 2^-3.5 = exactly 1.0
    _, vec1 = O.fused_vectors(np.ones(K, np.int8), unit_w)
    assert np.all(vec1 == np.float32(1.0))
    d2 = np.ones(K, np.int8)
    d2[[5, 130, 131]] = -1
    vec2 = O.second_vector(d2, K)
    c2 = np.float32(2.0 ** -3.5)
    assert np.array_equal(vec2, (d2.astype(np.float32) * c2))
    # spikes: block 0 gets 3 at local index 9, block 1 gets -5 at local index 70 (after the first rotation)
    j0, m0, j1, m1 = 9, 3.0, 70, -5.0
    idx = np.arange(128)
    h = lambda j: np.array([(-1.0) ** bin(int(i) & j).count("1") for i in idx])
    w = np.concatenate([h(j0) * m0 / 128.0, h(j1) * m1 / 128.0])[None, :]
    wb = bf16(w)
    assert np.array_equal(f32_of(wb).astype(np.float64), w)
    v1 = O.rotate(wb, vec1)[0]
    expect_v1 = np.zeros(K); expect_v1[j0] = m0; expect_v1[128 + j1] = m1
    assert np.array_equal(v1.astype(np.float64), expect_v1)
    # (vP)[j] = v[perm[j]]: output slot 131 (block 1, local 3) takes the block-0 spike, slot 5 (block 0) takes the block-1 spike
    perm = np.arange(K, dtype=np.int32)
    # (a 4-cycle, so that reading the index vector in the other direction gives a different result)
    perm[131], perm[j0], perm[5], perm[128 + j1] = j0, 5, 128 + j1, 131
    assert not np.array_equal(perm[perm], np.arange(K))
    packed, scales = O.prepare2_w4(wb, vec1, perm, vec2)
    assert packed.shape == (1, K // 2) and scales.shape == (1, 2)
    # block 0 of the result holds |m1| * c2 everywhere, block 1 holds |m0| * c2
    a0 = np.float32(abs(m1)) * c2
    a1 = np.float32(abs(m0)) * c2
    assert scales[0, 0] == a0 / np.float32(7.0) and scales[0, 1] == a1 / np.float32(7.0)
    sign0 = np.sign(m1) * d2[5] * h(5)         # column 5 of the Hadamard block
    sign1 = np.sign(m0) * d2[131] * h(3)       # column 3
    codes = np.concatenate([7 * sign0, 7 * sign1]).astype(np.int64)
    expect = ((codes[0::2] & 0xF) | ((codes[1::2] & 0xF) << 4)).astype(np.uint8)   # even k in the low nibble, two's complement
    assert np.array_equal(packed[0], expect)
    assert np.array_equal(O.unpack_w4(packed)[0], codes)
    # on random rows it is the 4-bit quantiser applied to the full transform's rows
    rng = np.random.default_rng(77)
    K2, N2 = 384, 10
    d1, d2r, smooth, permr = _full_setup(K2, 78)
    _, wv = O.fused_vectors(d1, smooth)
    v2 = O.second_vector(d2r, K2)
    wb2 = bf16(rng.standard_normal((N2, K2)) * 0.02)
    p_a, s_a = O.prepare2_w4(wb2, wv, permr, v2)
    p_b, s_b = O.quantize_w4_rows(O.rotate2(wb2, wv, permr, v2))
    assert np.array_equal(p_a, p_b) and np.array_equal(s_a, s_b)
    # and not the single-rotation path's result (the permutation and second rotation do something)
    p_c, _ = O.prepare_w4(wb2, wv)
    assert not np.array_equal(p_a, p_c)


def test_rotate_quantize_asym_ramp_and_composition():
    """Eq. 1-3 applied to the rotated token (Eq. 10's G_t): input rows whose rotation is a known ramp."""
    K = 256
    signs = np.ones(K, np.int8)
    signs[[0, 2, 133]] = -1
    act, _ = O.fused_vectors(signs, np.full(K, identity_vec_smooth(), np.float32))
    assert np.array_equal(act, signs.astype(np.float32))
    # rotated row: block 0 = 0, 2, .., 254, block 1 = 1, 3, .., 255.  The inverse transform of a ramp 2 i + c is
    # (127 + c) at index 0 and -2^b at index 2^b (the normalisation is folded into the unit vector above).
    def block(c):
        x = np.zeros(128)
        x[0] = 127.0 + c
        for b in range(7):
            x[1 << b] = -(2.0 ** b)
        return x
    for shift, z_expect in ((0.0, 0), (-100.0, 100)):
        x = np.concatenate([block(0.0 + shift), block(1.0 + shift)]) * signs     # the sign diagonal is undone by the vector
        xb = bf16(x[None, :])
        assert np.array_equal(f32_of(xb).astype(np.float64)[0], x)
        v = O.rotate(xb, act)[0]
        ramp = np.concatenate([2.0 * np.arange(128), 2.0 * np.arange(128) + 1.0]) + shift
        assert np.array_equal(v.astype(np.float64), ramp)
        q, s, z = O.rotate_quantize_asym(xb, act)
        assert q.dtype == np.uint8 and s[0] == np.float32(1.0) and z[0] == z_expect
        assert np.array_equal(q[0].astype(np.float64), ramp - shift)
    # on random rows: the asymmetric quantiser applied to the rotated rows, and it depends on the vector
    rng = np.random.default_rng(79)
    K2, M2 = 384, 9
    d = (rng.integers(0, 2, K2) * 2 - 1).astype(np.int8)
    smooth = rng.uniform(0.25, 4.0, K2).astype(np.float32)
    a2, _ = O.fused_vectors(d, smooth)
    xb2 = bf16(rng.standard_normal((M2, K2)) + 0.7)
    q_a, s_a, z_a = O.rotate_quantize_asym(xb2, a2)
    q_b, s_b, z_b = O.quantize_rows_asym(O.rotate(xb2, a2))
    assert np.array_equal(q_a, q_b) and np.array_equal(s_a, s_b) and np.array_equal(z_a, z_b)
    a3, _ = O.fused_vectors(d, None)
    q_c, _, _ = O.rotate_quantize_asym(xb2, a3)
    assert not np.array_equal(q_a, q_c)
