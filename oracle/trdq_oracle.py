"""numpy/ctypes front end of the CPU oracle (test infrastructure only).

Every function marshals numpy arrays into the C++ oracle library built from
``trdq_oracle.cpp``; no arithmetic of the method happens in this file.  The CUDA
library never imports this module.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


def _lib() -> C.CDLL:
    global _LIB
    if _LIB is None:
        from . import build as _build
        _LIB = C.CDLL(_build.build())
        _LIB.oracle_group_of.restype = C.c_int
        _LIB.oracle_num_threads.restype = C.c_int
        _LIB.oracle_invert_blocks.restype = C.c_int
        _LIB.oracle_greedy_block.restype = C.c_int
    return _LIB


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(_lib().oracle_num_threads())


def group_of(t_bounds, t: int) -> int:
    b = _c(t_bounds, np.int32)
    return int(_lib().oracle_group_of(_p(b), C.c_int(len(b) - 1), C.c_int(int(t))))


def fused_vectors(signs_g, smooth_g=None) -> Tuple[np.ndarray, np.ndarray]:
    """(act_vec, weight_vec) fp32 [K] of one group."""
    s = _c(signs_g, np.int8)
    K = s.shape[0]
    sm = None if smooth_g is None else _c(smooth_g, np.float32)
    act = np.empty(K, np.float32)
    wv = np.empty(K, np.float32)
    _lib().oracle_fused_vectors(_p(s), _p(sm), C.c_int(K), _p(act), _p(wv))
    return act, wv


def rotate(x_bits, vec) -> np.ndarray:
    x = _c(x_bits, np.uint16)
    M, K = x.shape
    v = np.empty((M, K), np.float32)
    _lib().oracle_rotate(_p(x), C.c_int64(K), C.c_int(M), C.c_int(K), _p(_c(vec, np.float32)), _p(v))
    return v


def quantize_rows(v) -> Tuple[np.ndarray, np.ndarray]:
    v = _c(v, np.float32)
    M, K = v.shape
    codes = np.empty((M, K), np.int8)
    scales = np.empty(M, np.float32)
    _lib().oracle_quantize_rows(_p(v), C.c_int(M), C.c_int(K), _p(codes), _p(scales))
    return codes, scales


def rotate_quantize(x_bits, act_vec) -> Tuple[np.ndarray, np.ndarray]:
    x = _c(x_bits, np.uint16)
    M, K = x.shape
    codes = np.empty((M, K), np.int8)
    scales = np.empty(M, np.float32)
    _lib().oracle_rotate_quantize(_p(x), C.c_int64(K), C.c_int(M), C.c_int(K),
                                  _p(_c(act_vec, np.float32)), _p(codes), _p(scales))
    return codes, scales


def prepare_w8(w_bits, weight_vec) -> Tuple[np.ndarray, np.ndarray]:
    w = _c(w_bits, np.uint16)
    N, K = w.shape
    codes = np.empty((N, K), np.int8)
    scales = np.empty(N, np.float32)
    _lib().oracle_prepare_w8(_p(w), C.c_int(N), C.c_int(K), _p(_c(weight_vec, np.float32)), _p(codes), _p(scales))
    return codes, scales


def prepare_w4(w_bits, weight_vec) -> Tuple[np.ndarray, np.ndarray]:
    w = _c(w_bits, np.uint16)
    N, K = w.shape
    packed = np.empty((N, K // 2), np.uint8)
    scales = np.empty((N, K // 128), np.float32)
    _lib().oracle_prepare_w4(_p(w), C.c_int(N), C.c_int(K), _p(_c(weight_vec, np.float32)), _p(packed), _p(scales))
    return packed, scales


def unpack_w4(packed) -> np.ndarray:
    p = _c(packed, np.uint8)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), np.int8)
    _lib().oracle_unpack_w4(_p(p), C.c_int64(out.size), _p(out))
    return out


def gemm_i32(q, qw) -> np.ndarray:
    q = _c(q, np.int8)
    qw = _c(qw, np.int8)
    M, K = q.shape
    N = qw.shape[0]
    assert qw.shape[1] == K
    acc = np.empty((M, N), np.int32)
    _lib().oracle_gemm_i32(_p(q), _p(qw), C.c_int(M), C.c_int(N), C.c_int(K), _p(acc))
    return acc


def epilogue(acc, sx, sw, bias_bits=None) -> np.ndarray:
    acc = _c(acc, np.int32)
    M, N = acc.shape
    b = None if bias_bits is None else _c(bias_bits, np.uint16)
    y = np.empty((M, N), np.float32)
    _lib().oracle_epilogue(_p(acc), _p(_c(sx, np.float32)), _p(_c(sw, np.float32)), _p(b), C.c_int(M), C.c_int(N), _p(y))
    return y


def linear_w8_rows(q, sx, qw, sw, bias_bits, rows, act: int = 0) -> np.ndarray:
    q = _c(q, np.int8)
    qw = _c(qw, np.int8)
    rows = _c(rows, np.int64)
    K = q.shape[1]
    N = qw.shape[0]
    b = None if bias_bits is None else _c(bias_bits, np.uint16)
    y = np.empty((rows.size, N), np.float32)
    _lib().oracle_linear_w8_rows_act(_p(q), _p(_c(sx, np.float32)), _p(qw), _p(_c(sw, np.float32)), _p(b),
                                     _p(rows), C.c_int(rows.size), C.c_int(N), C.c_int(K), C.c_int(int(act)), _p(y))
    return y


def linear_w4_rows(q, sx, packed, sw4, bias_bits, rows, act: int = 0) -> np.ndarray:
    q = _c(q, np.int8)
    packed = _c(packed, np.uint8)
    rows = _c(rows, np.int64)
    K = q.shape[1]
    N = packed.shape[0]
    b = None if bias_bits is None else _c(bias_bits, np.uint16)
    y = np.empty((rows.size, N), np.float32)
    _lib().oracle_linear_w4_rows_act(_p(q), _p(_c(sx, np.float32)), _p(packed), _p(_c(sw4, np.float32)), _p(b),
                                     _p(rows), C.c_int(rows.size), C.c_int(N), C.c_int(K), C.c_int(int(act)), _p(y))
    return y


def dense_rotation(signs_g) -> np.ndarray:
    s = _c(signs_g, np.int8)
    K = s.shape[0]
    R = np.empty((K, K), np.float64)
    _lib().oracle_dense_rotation(_p(s), C.c_int(K), _p(R))
    return R


def matmul_f64(A, B) -> np.ndarray:
    A = _c(A, np.float64)
    B = _c(B, np.float64)
    M, K = A.shape
    N = B.shape[1]
    out = np.empty((M, N), np.float64)
    _lib().oracle_matmul_f64(_p(A), _p(B), C.c_int(M), C.c_int(K), C.c_int(N), _p(out))
    return out


def second_vector(signs2_g, K: int) -> np.ndarray:
    s2 = None if signs2_g is None else _c(signs2_g, np.int8)
    out = np.empty(K, np.float32)
    _lib().oracle_second_vector(_p(s2), C.c_int(K), _p(out))
    return out


def zigzag_permutation(magnitude) -> np.ndarray:
    m = _c(magnitude, np.float32)
    perm = np.empty(m.shape[0], np.int32)
    _lib().oracle_zigzag_permutation(_p(m), C.c_int(m.shape[0]), _p(perm))
    return perm


def rotate2(x_bits, vec1, perm, vec2) -> np.ndarray:
    x = _c(x_bits, np.uint16)
    M, K = x.shape
    v = np.empty((M, K), np.float32)
    _lib().oracle_rotate2(_p(x), C.c_int64(K), C.c_int(M), C.c_int(K), _p(_c(vec1, np.float32)), _p(_c(perm, np.int32)),
                          _p(_c(vec2, np.float32)), _p(v))
    return v


def rotate2_quantize(x_bits, vec1, perm, vec2) -> Tuple[np.ndarray, np.ndarray]:
    x = _c(x_bits, np.uint16)
    M, K = x.shape
    codes = np.empty((M, K), np.int8)
    scales = np.empty(M, np.float32)
    _lib().oracle_rotate2_quantize(_p(x), C.c_int64(K), C.c_int(M), C.c_int(K), _p(_c(vec1, np.float32)), _p(_c(perm, np.int32)),
                                   _p(_c(vec2, np.float32)), _p(codes), _p(scales))
    return codes, scales


def prepare2_w4(w_bits, vec1, perm, vec2) -> Tuple[np.ndarray, np.ndarray]:
    w = _c(w_bits, np.uint16)
    N, K = w.shape
    packed = np.empty((N, K // 2), np.uint8)
    scales = np.empty((N, K // 128), np.float32)
    _lib().oracle_prepare2_w4(_p(w), C.c_int(N), C.c_int(K), _p(_c(vec1, np.float32)), _p(_c(perm, np.int32)),
                              _p(_c(vec2, np.float32)), _p(packed), _p(scales))
    return packed, scales


def dense_permutation(perm) -> np.ndarray:
    pm = _c(perm, np.int32)
    K = pm.shape[0]
    P = np.empty((K, K), np.float64)
    _lib().oracle_dense_permutation(_p(pm), C.c_int(K), _p(P))
    return P


def quantize_rows_asym(v) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    v = _c(v, np.float32)
    M, K = v.shape
    codes = np.empty((M, K), np.uint8)
    scales = np.empty(M, np.float32)
    zp = np.empty(M, np.int32)
    _lib().oracle_quantize_rows_asym(_p(v), C.c_int(M), C.c_int(K), _p(codes), _p(scales), _p(zp))
    return codes, scales, zp


def rotate_quantize_asym(x_bits, act_vec) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    x = _c(x_bits, np.uint16)
    M, K = x.shape
    codes = np.empty((M, K), np.uint8)
    scales = np.empty(M, np.float32)
    zp = np.empty(M, np.int32)
    _lib().oracle_rotate_quantize_asym(_p(x), C.c_int64(K), C.c_int(M), C.c_int(K), _p(_c(act_vec, np.float32)), _p(codes),
                                       _p(scales), _p(zp))
    return codes, scales, zp


def linear_asym_rows(q, sx, zp, qw, sw, bias_bits, rows) -> np.ndarray:
    q = _c(q, np.uint8)
    qw = _c(qw, np.int8)
    rows = _c(rows, np.int64)
    K = q.shape[1]
    N = qw.shape[0]
    b = None if bias_bits is None else _c(bias_bits, np.uint16)
    y = np.empty((rows.size, N), np.float32)
    _lib().oracle_linear_asym_rows(_p(q), _p(_c(sx, np.float32)), _p(_c(zp, np.int32)), _p(qw), _p(_c(sw, np.float32)), _p(b),
                                   _p(rows), C.c_int(rows.size), C.c_int(N), C.c_int(K), _p(y))
    return y


# ---- dense block rotations (Eq. 6-8) -------------------------------------------------------------

def dense_stored_blocks(blocks, smooth_g=None) -> np.ndarray:
    """bf16 bit patterns [K/128, 128, 128] of Delta-scaled blocks, as applied to the activations."""
    b = _c(blocks, np.float32)
    nb = b.shape[0]
    sm = None if smooth_g is None else _c(smooth_g, np.float32)
    out = np.empty((nb, 128, 128), np.uint16)
    _lib().oracle_dense_stored_blocks(_p(b), _p(sm), C.c_int(nb * 128), _p(out))
    return out


def rotate_dense(x_bits, stored) -> np.ndarray:
    x = _c(x_bits, np.uint16)
    M, K = x.shape
    v = np.empty((M, K), np.float32)
    _lib().oracle_rotate_dense(_p(x), C.c_int64(K), C.c_int(M), C.c_int(K), _p(_c(stored, np.uint16)), _p(v))
    return v


def invert_blocks(stored) -> np.ndarray:
    s = _c(stored, np.uint16)
    inv = np.empty(s.shape, np.float64)
    rc = int(_lib().oracle_invert_blocks(_p(s), C.c_int(s.shape[0]), _p(inv)))
    if rc != 0:
        raise ValueError(f"block {rc - 1} is singular")
    return inv


def prepare_dense_rotate(w_bits, inv) -> np.ndarray:
    w = _c(w_bits, np.uint16)
    N, K = w.shape
    wr = np.empty((N, K), np.float32)
    _lib().oracle_prepare_dense_rotate(_p(w), C.c_int(N), C.c_int(K), _p(_c(inv, np.float64)), _p(wr))
    return wr


def quantize_w4_rows(wr) -> Tuple[np.ndarray, np.ndarray]:
    wr = _c(wr, np.float32)
    N, K = wr.shape
    packed = np.empty((N, K // 2), np.uint8)
    scales = np.empty((N, K // 128), np.float32)
    _lib().oracle_quantize_w4_rows(_p(wr), C.c_int(N), C.c_int(K), _p(packed), _p(scales))
    return packed, scales


def greedy_block(x_calib, gauss) -> Tuple[np.ndarray, int, np.ndarray]:
    """(R [128,128] fp64, n, per-step maxima) of Eq. 6-7 for one block."""
    x = _c(x_calib, np.float64)
    g = _c(gauss, np.float64)
    steps = g.shape[0]
    R = np.empty((128, 128), np.float64)
    trace = np.empty(steps, np.float64)
    n = int(_lib().oracle_greedy_block(_p(x), C.c_int(x.shape[0]), C.c_int(steps), _p(g), _p(R), _p(trace)))
    return R, n, trace


# ---- LayerNorm + modulation in front of the rotation ---------------------------------------------

def norm_modulate(x_bits, shift_bits, scale_bits, rows_per_sample: int, eps: float) -> np.ndarray:
    x = _c(x_bits, np.uint16)
    M, K = x.shape
    sh = None if shift_bits is None else _c(shift_bits, np.uint16)
    sc = None if scale_bits is None else _c(scale_bits, np.uint16)
    h = np.empty((M, K), np.float32)
    _lib().oracle_norm_modulate(_p(x), C.c_int64(K), C.c_int(M), C.c_int(K), _p(sh), _p(sc), C.c_int(int(rows_per_sample)),
                                C.c_double(float(eps)), _p(h))
    return h


def rotate_f32(h, vec) -> np.ndarray:
    h = _c(h, np.float32)
    M, K = h.shape
    v = np.empty((M, K), np.float32)
    _lib().oracle_rotate_f32(_p(h), C.c_int(M), C.c_int(K), _p(_c(vec, np.float32)), _p(v))
    return v
