"""CPU-side checks of the C ABI: the shared library builds, loads without a GPU, exports every
symbol the header declares, and validates arguments on the host before touching CUDA."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2503_06564_b200 import build, trdq
    build.build()
    return trdq.lib()


def test_every_declared_symbol_is_exported(lib):
    from paper_2503_06564_b200 import trdq
    header = open(os.path.join(ROOT, "include", "trdq.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(trdq_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(trdq.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    from paper_2503_06564_b200 import trdq
    seen = set()
    for code in range(0, 12):
        s = trdq.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 12
    assert trdq.status_string(99) == "unknown status"
    assert lib.trdq_version() >= 100


@pytest.mark.parametrize("G", [1, 2, 3, 4, 5])
def test_find_group_exhaustive(lib, G):
    from paper_2503_06564_b200 import trdq, workloads as WL
    b = WL.group_bounds(G)
    for t in range(1000):
        g = trdq.trdq_find_group(b, t)
        assert b[g] <= t < b[g + 1]
    for t in (-1, 1000, 12345):
        with pytest.raises(trdq.TrdqError) as e:
            trdq.trdq_find_group(b, t)
        assert e.value.status == 4
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_find_group([0, 10, 10], 5)
    assert e.value.status == 5


def test_host_side_validation_needs_no_device(lib):
    """Bad specifications are rejected before any CUDA call, so the codes are the same on a CPU-only box."""
    from paper_2503_06564_b200 import trdq
    ones = np.ones((2, 256), np.int8)

    def status_of(**kw):
        args = dict(K=256, t_bounds=[0, 500, 1000], signs=ones, smooth=None, block=128)
        args.update(kw)
        try:
            trdq.Rotation(**args)
        except trdq.TrdqError as e:
            return e.status
        return 0

    assert status_of(K=200) == 2
    assert status_of(K=0) == 2
    assert status_of(block=64) == 2
    assert status_of(K=131072 + 128, signs=np.ones((2, 131072 + 128), np.int8)) == 2
    assert status_of(t_bounds=[0, 500, 400]) == 5
    bad = ones.copy()
    bad[1, 5] = 0
    assert status_of(signs=bad) == 5
    assert status_of(smooth=np.zeros((2, 256), np.float32)) == 5
    # null handles
    g = C.c_int32()
    assert lib.trdq_group_of(None, 0, C.byref(g)) == 1
    assert lib.trdq_rotate_quantize(None, 0, None, 0, 0, None, None, None) == 1
    assert lib.trdq_linear(None, 0, None, None, 0, None, None, 0, None) == 1
    assert lib.trdq_weights_info(None, None, None, None, None) == 1
    # the split-K entry points (caller workspace / built-in scratch) and the asymmetric one take a null handle the same way
    assert lib.trdq_linear_splitk(None, 0, None, None, 0, None, None, 0, None, 0, None) == 1
    assert lib.trdq_linear_splitk_static(None, 0, None, None, 0, None, None, 0, None) == 1
    assert lib.trdq_linear_splitk_workspace(None, 0, None, None) == 1
    assert lib.trdq_linear_asym(None, 0, None, None, None, 0, None, None, 0, None) == 1
    # reporting aids: argument checks come before any device query
    name = C.create_string_buffer(96)
    assert lib.trdq_kernel_choice(0, 128, 1152, 0, 8, None, 96) == 1
    assert lib.trdq_kernel_choice(0, 128, 1152, 0, 8, name, 8) == 2          # buffer too small for a kernel name
    assert lib.trdq_kernel_choice(0, 0, 1152, 0, 8, name, 96) == 2
    assert lib.trdq_kernel_choice(0, 128, 1000, 0, 8, name, 96) == 2         # K not a multiple of the block
    assert lib.trdq_measure_mma_ceiling(1024, None, None) == 1
    clusters = C.c_int32(0)
    assert lib.trdq_measure_mma_ceiling(4, C.byref(clusters), None) == 2     # fewer than eight MMAs
    assert lib.trdq_measure_mma_ceiling(1 << 23, C.byref(clusters), None) == 2
    assert lib.trdq_rotation_destroy(None) == 0 and lib.trdq_weights_destroy(None) == 0
    import torch
    if not torch.cuda.is_available():
        # a valid specification cannot be realised without a device, and says so
        assert status_of() == 7


def test_binding_fails_loudly_without_the_library(tmp_path, monkeypatch):
    from paper_2503_06564_b200 import trdq
    monkeypatch.setattr(trdq, "_lib", None)
    monkeypatch.setattr(trdq, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(ImportError):
        trdq.lib()


def test_zigzag_permutation_matches_the_oracle_and_rejects_bad_input(lib):
    """Host-only: the library's zigzag deal equals the oracle's on random magnitudes, ties included."""
    from oracle import trdq_oracle as O
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(0)
    for K in (128, 256, 1152, 4608):
        mag = rng.gamma(2.0, 1.0, K).astype(np.float32)
        mag[rng.choice(K, K // 10, replace=False)] = mag[0]          # ties
        assert np.array_equal(trdq.trdq_zigzag_permutation(mag), O.zigzag_permutation(mag))
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_zigzag_permutation(np.ones(100, np.float32))
    assert e.value.status == 2
    # a full-transform specification with a non-permutation is refused on the host
    with pytest.raises(trdq.TrdqError) as e:
        trdq.Rotation(256, [0, 1000], np.ones((1, 256), np.int8), perm=np.zeros((1, 256), np.int32))
    assert e.value.status == 5


def test_greedy_rotation_block_matches_oracle(lib):
    """Eq. 6-7 on the host: the library's construction against the oracle's on the same calibration rows and draws."""
    from oracle import trdq_oracle as O
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(5)
    x = rng.standard_normal((48, 128)).astype(np.float32)
    x[:, 17] *= 70.0
    x[:, 101] *= 30.0
    gauss = rng.standard_normal((5, 128, 128))
    R, n = trdq.trdq_greedy_rotation_block(x, gauss)
    R_ref, n_ref, trace = O.greedy_block(x.astype(np.float64), gauss)
    assert n == n_ref
    assert np.max(np.abs(R.astype(np.float64) - R_ref)) <= 2.0 ** -24 + 1e-9   # one rounding to fp32 of entries below 1
    assert np.max(np.abs(R.astype(np.float64) @ R.astype(np.float64).T - np.eye(128))) < 1e-5
    assert np.max(np.abs(x.astype(np.float64) @ R_ref)) < 0.2 * np.max(np.abs(x))
    # argument errors are found on the host
    assert lib.trdq_greedy_rotation_block(None, 4, 1, None, None, None) == 1
    bad = x.copy()
    bad[0, 0] = np.inf
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_greedy_rotation_block(bad, gauss)
    assert e.value.status == 5


def test_dense_rotation_and_fusion_calls_validate_on_the_host(lib):
    """The newer entry points reject bad arguments before any CUDA call: the dense-block specification (shape, bounds,
    smoothing values, singular or non-finite blocks), and null handles of the dense, norm-fused and activation calls."""
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(3)
    q, _ = np.linalg.qr(rng.standard_normal((128, 128)))
    blocks = np.stack([q, q.T]).astype(np.float32)[None]           # K = 256, one group

    def status_of(K=256, bounds=(0, 1000), blk=blocks, smooth=None):
        try:
            trdq.DenseRotation(K, list(bounds), blk, smooth)
        except trdq.TrdqError as e:
            return e.status
        return 0

    b = np.ascontiguousarray([0, 1000], np.int32)
    f = blocks.ctypes.data_as(C.POINTER(C.c_float))
    h = C.c_void_p()
    assert lib.trdq_rotation_create_dense(200, 1, b.ctypes.data_as(C.POINTER(C.c_int32)), f, None, C.byref(h)) == 2
    assert lib.trdq_rotation_create_dense(256, 0, b.ctypes.data_as(C.POINTER(C.c_int32)), f, None, C.byref(h)) == 5
    assert lib.trdq_rotation_create_dense(256, 1, None, f, None, C.byref(h)) == 1
    assert status_of(bounds=(10, 10)) == 5
    assert status_of(smooth=np.full((1, 256), -1.0, np.float32)) == 5
    singular = blocks.copy()
    singular[0, 1, :, 3] = singular[0, 1, :, 40]
    assert status_of(blk=singular) == 5
    inf = blocks.copy()
    inf[0, 0, 7, 7] = np.inf
    assert status_of(blk=inf) == 5
    import torch
    if not torch.cuda.is_available():
        assert status_of() in (7, 8)                                 # a valid specification needs a device and says so
    n = C.c_uint64()
    assert lib.trdq_rotate_dense_workspace(None, 16, C.byref(n)) == 1
    assert lib.trdq_rotate_dense_quantize(None, 0, None, 0, 0, None, None, None, 0, None) == 1
    assert lib.trdq_norm_rotate_quantize(None, 0, None, 0, 0, None, None, 1, C.c_float(1e-6), None, None, None) == 1
    assert lib.trdq_linear_act(None, 0, None, None, 0, None, None, 0, 7, None) == 2      # unknown activation
    assert lib.trdq_linear_act(None, 0, None, None, 0, None, None, 0, 1, None) == 1
    assert lib.trdq_run_layers(None, 3, 0, None) == 1 and lib.trdq_run_layers(None, 0, 0, None) == 0
