"""ctypes binding of ``libtrdq.so``: argument marshalling only.

Every function here has the name of the C entry point it calls (``include/trdq.h``)
and does nothing but turn torch tensors into pointers, sizes and the current
stream.  All arithmetic runs in the CUDA kernels of the library; if the shared
object is missing the import of this module's library handle fails loudly, and
there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtrdq.so")

OK = 0
STATUS_NAMES = {0: "TRDQ_OK", 1: "TRDQ_ERR_NULL", 2: "TRDQ_ERR_SHAPE", 3: "TRDQ_ERR_ALIGN", 4: "TRDQ_ERR_TIMESTEP",
                5: "TRDQ_ERR_GROUP", 6: "TRDQ_ERR_WBITS", 7: "TRDQ_ERR_CUDA", 8: "TRDQ_ERR_NOMEM", 9: "TRDQ_ERR_TIMEOUT",
                10: "TRDQ_ERR_MISMATCH", 11: "TRDQ_ERR_SCRATCH"}

EXPORTS = (
    "trdq_status_string", "trdq_version", "trdq_rotation_create", "trdq_rotation_destroy", "trdq_group_of",
    "trdq_find_group", "trdq_prepare_weights", "trdq_weights_destroy", "trdq_weights_info", "trdq_weights_view",
    "trdq_weights_export",
    "trdq_rotate_quantize", "trdq_linear", "trdq_linear_cfg", "trdq_gemm_i32", "trdq_device_status",
    "trdq_run_layers", "trdq_linear_splitk_workspace", "trdq_linear_splitk", "trdq_linear_splitk_static",
    "trdq_rotation_create_full", "trdq_zigzag_permutation", "trdq_rotate_quantize_asym", "trdq_linear_asym",
    "trdq_selftest_wait_expiry", "trdq_rotation_create_dense", "trdq_rotate_dense_workspace", "trdq_rotate_dense_quantize",
    "trdq_greedy_rotation_block", "trdq_linear_act", "trdq_norm_rotate_quantize", "trdq_kernel_choice",
    "trdq_measure_mma_ceiling",
)


class TrdqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {STATUS_NAMES.get(self.status, self.status)} ({status_string(self.status)})")


class RotationSpec(C.Structure):
    _fields_ = [("K", C.c_int32), ("block", C.c_int32), ("num_groups", C.c_int32),
                ("t_bounds", C.POINTER(C.c_int32)), ("signs", C.POINTER(C.c_int8)), ("smooth", C.POINTER(C.c_float))]


class LayerOp(C.Structure):
    _fields_ = [("rot", C.c_void_p), ("w", C.c_void_p), ("X_bf16", C.c_void_p), ("ldx", C.c_int64), ("M", C.c_int32),
                ("codes", C.c_void_p), ("scales", C.c_void_p), ("bias_bf16", C.c_void_p), ("Y_bf16", C.c_void_p),
                ("ldy", C.c_int64), ("act", C.c_int32), ("workspace", C.c_void_p), ("workspace_bytes", C.c_uint64)]


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """The loaded library.  Raises if it has not been built: there is no other code path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2503_06564_b200.build`")
        l = C.CDLL(LIB_PATH)
        l.trdq_status_string.restype = C.c_char_p
        l.trdq_status_string.argtypes = [C.c_int]
        l.trdq_version.restype = C.c_int32
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        l.trdq_rotation_create.argtypes = [C.POINTER(RotationSpec), C.POINTER(vp)]
        l.trdq_rotation_create_full.argtypes = [C.POINTER(RotationSpec), C.POINTER(i32), C.POINTER(C.c_int8), C.POINTER(vp)]
        l.trdq_zigzag_permutation.argtypes = [C.POINTER(C.c_float), i32, C.POINTER(i32)]
        l.trdq_rotation_destroy.argtypes = [vp]
        l.trdq_group_of.argtypes = [vp, i32, C.POINTER(i32)]
        l.trdq_find_group.argtypes = [C.POINTER(i32), i32, i32, C.POINTER(i32)]
        l.trdq_prepare_weights.argtypes = [vp, vp, i32, i32, C.POINTER(vp), vp]
        l.trdq_weights_destroy.argtypes = [vp]
        l.trdq_weights_info.argtypes = [vp, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
        l.trdq_weights_view.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp)]
        l.trdq_weights_export.argtypes = [vp, i32, vp, vp, vp]
        l.trdq_rotate_quantize.argtypes = [vp, i32, vp, i64, i32, vp, vp, vp]
        l.trdq_linear.argtypes = [vp, i32, vp, vp, i32, vp, vp, i64, vp]
        l.trdq_norm_rotate_quantize.argtypes = [vp, i32, vp, i64, i32, vp, vp, i32, C.c_float, vp, vp, vp]
        l.trdq_linear_act.argtypes = [vp, i32, vp, vp, i32, vp, vp, i64, i32, vp]
        l.trdq_kernel_choice.argtypes = [i32, i32, i32, i32, i32, C.c_char_p, i32]
        l.trdq_measure_mma_ceiling.argtypes = [i32, C.POINTER(i32), vp]
        l.trdq_linear_cfg.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(i32), vp, C.POINTER(vp),
                                      C.POINTER(i64), vp]
        l.trdq_gemm_i32.argtypes = [vp, i32, vp, i32, vp, i64, vp]
        l.trdq_run_layers.argtypes = [C.POINTER(LayerOp), i32, i32, vp]
        l.trdq_linear_splitk_workspace.argtypes = [vp, i32, C.POINTER(i32), C.POINTER(C.c_uint64)]
        l.trdq_linear_splitk.argtypes = [vp, i32, vp, vp, i32, vp, vp, i64, vp, C.c_uint64, vp]
        l.trdq_linear_splitk_static.argtypes = [vp, i32, vp, vp, i32, vp, vp, i64, vp]
        l.trdq_rotate_quantize_asym.argtypes = [vp, i32, vp, i64, i32, vp, vp, vp, vp]
        l.trdq_linear_asym.argtypes = [vp, i32, vp, vp, vp, i32, vp, vp, i64, vp]
        l.trdq_selftest_wait_expiry.argtypes = [vp]
        l.trdq_rotation_create_dense.argtypes = [i32, i32, C.POINTER(i32), C.POINTER(C.c_float), C.POINTER(C.c_float), C.POINTER(vp)]
        l.trdq_rotate_dense_workspace.argtypes = [vp, i32, C.POINTER(C.c_uint64)]
        l.trdq_rotate_dense_quantize.argtypes = [vp, i32, vp, i64, i32, vp, vp, vp, C.c_uint64, vp]
        l.trdq_greedy_rotation_block.argtypes = [C.POINTER(C.c_float), i32, i32, C.POINTER(C.c_double), C.POINTER(C.c_float),
                                                 C.POINTER(i32)]
        l.trdq_device_status.argtypes = [C.POINTER(C.c_uint32)]
        _lib = l
    return _lib


def status_string(status: int) -> str:
    return lib().trdq_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise TrdqError(status, where)


def _stream() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def trdq_find_group(t_bounds: Sequence[int], t: int) -> int:
    b = np.ascontiguousarray(t_bounds, dtype=np.int32)
    g = C.c_int32(-1)
    _check(lib().trdq_find_group(b.ctypes.data_as(C.POINTER(C.c_int32)), len(b) - 1, int(t), C.byref(g)), "trdq_find_group")
    return g.value


def trdq_zigzag_permutation(magnitude) -> np.ndarray:
    """Zigzag channel permutation (int32 [K]) from per-channel magnitudes; host only."""
    m = np.ascontiguousarray(magnitude, dtype=np.float32)
    perm = np.empty(m.shape[0], np.int32)
    _check(lib().trdq_zigzag_permutation(m.ctypes.data_as(C.POINTER(C.c_float)), int(m.shape[0]),
                                         perm.ctypes.data_as(C.POINTER(C.c_int32))), "trdq_zigzag_permutation")
    return perm


class Rotation:
    """Handle of a trdq_rotation (per-group device tables of one C_in)."""

    def __init__(self, K: int, t_bounds, signs, smooth=None, block: int = 128, perm=None, signs2=None):
        """perm (int32 [G][K]) selects the full transform of Eq. 9: rotation, zigzag permutation, second rotation
        (signs2: its +-1 vector, int8 [G][K] or None)."""
        self._h = C.c_void_p()
        b = np.ascontiguousarray(t_bounds, dtype=np.int32)
        s = np.ascontiguousarray(signs, dtype=np.int8)
        sm = None if smooth is None else np.ascontiguousarray(smooth, dtype=np.float32)
        spec = RotationSpec(int(K), int(block), int(len(b) - 1), b.ctypes.data_as(C.POINTER(C.c_int32)),
                            s.ctypes.data_as(C.POINTER(C.c_int8)),
                            None if sm is None else sm.ctypes.data_as(C.POINTER(C.c_float)))
        if perm is None:
            _check(lib().trdq_rotation_create(C.byref(spec), C.byref(self._h)), "trdq_rotation_create")
        else:
            pm = np.ascontiguousarray(perm, dtype=np.int32)
            s2 = None if signs2 is None else np.ascontiguousarray(signs2, dtype=np.int8)
            _check(lib().trdq_rotation_create_full(C.byref(spec), pm.ctypes.data_as(C.POINTER(C.c_int32)),
                                                   None if s2 is None else s2.ctypes.data_as(C.POINTER(C.c_int8)),
                                                   C.byref(self._h)), "trdq_rotation_create_full")
        self.K = int(K)
        self.num_groups = int(len(b) - 1)

    def group_of(self, t: int) -> int:
        g = C.c_int32(-1)
        _check(lib().trdq_group_of(self._h, int(t), C.byref(g)), "trdq_group_of")
        return g.value

    def close(self) -> None:
        if self._h:
            lib().trdq_rotation_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class DenseRotation(Rotation):
    """Handle of a trdq_rotation made of dense 128 x 128 blocks (Eq. 6-8): blocks fp32 [G][K/128][128][128]."""

    def __init__(self, K: int, t_bounds, blocks, smooth=None):
        self._h = C.c_void_p()
        b = np.ascontiguousarray(t_bounds, dtype=np.int32)
        G = int(len(b) - 1)
        blk = np.ascontiguousarray(blocks, dtype=np.float32)
        assert blk.shape == (G, int(K) // 128, 128, 128), blk.shape
        sm = None if smooth is None else np.ascontiguousarray(smooth, dtype=np.float32)
        _check(lib().trdq_rotation_create_dense(int(K), G, b.ctypes.data_as(C.POINTER(C.c_int32)),
                                                blk.ctypes.data_as(C.POINTER(C.c_float)),
                                                None if sm is None else sm.ctypes.data_as(C.POINTER(C.c_float)),
                                                C.byref(self._h)), "trdq_rotation_create_dense")
        self.K = int(K)
        self.num_groups = G


class Weights:
    """Handle of a trdq_weights (H_t(W) of one layer, quantized for every group)."""

    def __init__(self, handle: C.c_void_p):
        self._h = handle
        n, k, wb, g = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int32()
        _check(lib().trdq_weights_info(self._h, C.byref(n), C.byref(k), C.byref(wb), C.byref(g)), "trdq_weights_info")
        self.N, self.K, self.wbits, self.num_groups = n.value, k.value, wb.value, g.value

    def view(self, g: int) -> Tuple[int, int]:
        """(device pointer of the codes, device pointer of the scales) of group g."""
        wq, sc = C.c_void_p(), C.c_void_p()
        _check(lib().trdq_weights_view(self._h, int(g), C.byref(wq), C.byref(sc)), "trdq_weights_view")
        return wq.value, sc.value

    def view_tensors(self, g: int):
        """Copies of group g's codes and scales as torch tensors (device)."""
        import torch
        if self.wbits == 8:
            codes = torch.empty((self.N, self.K), dtype=torch.int8, device="cuda")
            scales = torch.empty((self.N,), dtype=torch.float32, device="cuda")
        else:
            codes = torch.empty((self.N, self.K // 2), dtype=torch.uint8, device="cuda")
            scales = torch.empty((self.N, self.K // 128), dtype=torch.float32, device="cuda")
        _check(lib().trdq_weights_export(self._h, int(g), _ptr(codes), _ptr(scales), _stream()), "trdq_weights_export")
        return codes, scales

    def close(self) -> None:
        if self._h:
            lib().trdq_weights_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def trdq_prepare_weights(rot: Rotation, W_bf16, wbits: int = 8) -> Weights:
    assert W_bf16.is_cuda and W_bf16.is_contiguous() and W_bf16.dim() == 2 and W_bf16.element_size() == 2
    if W_bf16.shape[1] != rot.K:
        raise TrdqError(2, "trdq_prepare_weights (K of W differs from the rotation's)")
    h = C.c_void_p()
    _check(lib().trdq_prepare_weights(rot._h, _ptr(W_bf16), int(W_bf16.shape[0]), int(wbits), C.byref(h), _stream()),
           "trdq_prepare_weights")
    return Weights(h)


def trdq_rotate_quantize(rot: Rotation, t: int, X_bf16, codes=None, scales=None):
    """codes int8 [M,K], scales fp32 [M] of the rotated activations at time-step t."""
    import torch
    assert X_bf16.is_cuda and X_bf16.dim() == 2 and X_bf16.element_size() == 2 and X_bf16.stride(1) == 1
    M = int(X_bf16.shape[0])
    if codes is None:
        codes = torch.empty((M, rot.K), dtype=torch.int8, device=X_bf16.device)
    if scales is None:
        scales = torch.empty((M,), dtype=torch.float32, device=X_bf16.device)
    ldx = int(X_bf16.stride(0)) if M > 1 else rot.K
    _check(lib().trdq_rotate_quantize(rot._h, int(t), _ptr(X_bf16), ldx, M, _ptr(codes), _ptr(scales), _stream()),
           "trdq_rotate_quantize")
    return codes, scales


def trdq_norm_rotate_quantize(rot: Rotation, t: int, X_bf16, shift_bf16=None, scale_bf16=None, rows_per_sample: Optional[int] = None,
                              eps: float = 1e-6, codes=None, scales=None):
    """LayerNorm + per-sample modulation + rotation + per-token quantizer in one kernel."""
    import torch
    assert X_bf16.is_cuda and X_bf16.dim() == 2 and X_bf16.element_size() == 2 and X_bf16.stride(1) == 1
    M = int(X_bf16.shape[0])
    if rows_per_sample is None:
        rows_per_sample = max(M, 1)
    if codes is None:
        codes = torch.empty((M, rot.K), dtype=torch.int8, device=X_bf16.device)
    if scales is None:
        scales = torch.empty((M,), dtype=torch.float32, device=X_bf16.device)
    ldx = int(X_bf16.stride(0)) if M > 1 else rot.K
    _check(lib().trdq_norm_rotate_quantize(rot._h, int(t), _ptr(X_bf16), ldx, M, _ptr(shift_bf16), _ptr(scale_bf16),
                                           int(rows_per_sample), float(eps), _ptr(codes), _ptr(scales), _stream()),
           "trdq_norm_rotate_quantize")
    return codes, scales


def trdq_rotate_dense_workspace(rot: Rotation, M: int) -> int:
    n = C.c_uint64(0)
    _check(lib().trdq_rotate_dense_workspace(rot._h, int(M), C.byref(n)), "trdq_rotate_dense_workspace")
    return int(n.value)


def trdq_rotate_dense_quantize(rot: Rotation, t: int, X_bf16, codes=None, scales=None, workspace=None):
    """codes int8 [M,K], scales fp32 [M] of the activations rotated by the dense blocks of time-step t."""
    import torch
    assert X_bf16.is_cuda and X_bf16.dim() == 2 and X_bf16.element_size() == 2 and X_bf16.stride(1) == 1
    M = int(X_bf16.shape[0])
    if codes is None:
        codes = torch.empty((M, rot.K), dtype=torch.int8, device=X_bf16.device)
    if scales is None:
        scales = torch.empty((M,), dtype=torch.float32, device=X_bf16.device)
    if workspace is None:
        workspace = torch.empty((max(1, trdq_rotate_dense_workspace(rot, M)),), dtype=torch.uint8, device=X_bf16.device)
    ldx = int(X_bf16.stride(0)) if M > 1 else rot.K
    _check(lib().trdq_rotate_dense_quantize(rot._h, int(t), _ptr(X_bf16), ldx, M, _ptr(codes), _ptr(scales), _ptr(workspace),
                                            int(workspace.numel() * workspace.element_size()), _stream()),
           "trdq_rotate_dense_quantize")
    return codes, scales


def trdq_greedy_rotation_block(x_calib, gauss) -> Tuple[np.ndarray, int]:
    """(R fp32 [128,128], n) of Eq. 6-7 for one block; host only."""
    x = np.ascontiguousarray(x_calib, dtype=np.float32)
    g = np.ascontiguousarray(gauss, dtype=np.float64)
    assert x.ndim == 2 and x.shape[1] == 128 and g.ndim == 3 and g.shape[1:] == (128, 128)
    R = np.empty((128, 128), np.float32)
    n = C.c_int32(0)
    _check(lib().trdq_greedy_rotation_block(x.ctypes.data_as(C.POINTER(C.c_float)), int(x.shape[0]), int(g.shape[0]),
                                            g.ctypes.data_as(C.POINTER(C.c_double)), R.ctypes.data_as(C.POINTER(C.c_float)),
                                            C.byref(n)), "trdq_greedy_rotation_block")
    return R, int(n.value)


def trdq_linear(w: Weights, t: int, codes, scales, bias_bf16=None, out=None):
    """bf16 [M,N] output of the integer GEMM with the dequantizing epilogue."""
    import torch
    M = int(codes.shape[0])
    if out is None:
        out = torch.empty((M, w.N), dtype=torch.bfloat16, device=codes.device)
    ldy = int(out.stride(0)) if M > 1 else w.N
    _check(lib().trdq_linear(w._h, int(t), _ptr(codes), _ptr(scales), M, _ptr(bias_bf16), _ptr(out), ldy, _stream()),
           "trdq_linear")
    return out


ACT_NONE, ACT_GELU_TANH = 0, 1


def trdq_linear_act(w: Weights, t: int, codes, scales, bias_bf16=None, out=None, act: int = ACT_GELU_TANH):
    """trdq_linear with the following activation (GELU, tanh form) folded into the epilogue."""
    import torch
    M = int(codes.shape[0])
    if out is None:
        out = torch.empty((M, w.N), dtype=torch.bfloat16, device=codes.device)
    ldy = int(out.stride(0)) if M > 1 else w.N
    _check(lib().trdq_linear_act(w._h, int(t), _ptr(codes), _ptr(scales), M, _ptr(bias_bf16), _ptr(out), ldy, int(act), _stream()),
           "trdq_linear_act")
    return out


def trdq_linear_cfg(w: Weights, t: int, codes2, scales2, bias_bf16=None, out2=None):
    """Two row segments (conditional, unconditional) through one launch."""
    import torch
    Ms = [int(c.shape[0]) for c in codes2]
    if out2 is None:
        out2 = [torch.empty((m, w.N), dtype=torch.bfloat16, device=codes2[0].device) for m in Ms]
    vp2, i32_2, i64_2 = C.c_void_p * 2, C.c_int32 * 2, C.c_int64 * 2
    _check(lib().trdq_linear_cfg(w._h, int(t), vp2(*[_ptr(c) for c in codes2]), vp2(*[_ptr(s) for s in scales2]),
                                 i32_2(*Ms), _ptr(bias_bf16), vp2(*[_ptr(o) for o in out2]),
                                 i64_2(*[int(o.stride(0)) if m > 1 else w.N for o, m in zip(out2, Ms)]), _stream()),
           "trdq_linear_cfg")
    return out2


def trdq_linear_splitk_workspace(w: Weights, M: int) -> Tuple[int, int]:
    """(number of k ranges, workspace bytes) the split-K call would use for M rows."""
    splits, nbytes = C.c_int32(0), C.c_uint64(0)
    _check(lib().trdq_linear_splitk_workspace(w._h, int(M), C.byref(splits), C.byref(nbytes)), "trdq_linear_splitk_workspace")
    return splits.value, nbytes.value


def trdq_linear_splitk(w: Weights, t: int, codes, scales, bias_bf16=None, out=None, workspace=None):
    """trdq_linear with the reduction split over several CTAs per tile; `workspace` is a device tensor of at least
    the size trdq_linear_splitk_workspace reports (allocated here when omitted)."""
    import torch
    M = int(codes.shape[0])
    if out is None:
        out = torch.empty((M, w.N), dtype=torch.bfloat16, device=codes.device)
    splits, nbytes = trdq_linear_splitk_workspace(w, M)
    if workspace is None and nbytes:
        workspace = torch.empty((nbytes,), dtype=torch.uint8, device=codes.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    ldy = int(out.stride(0)) if M > 1 else w.N
    _check(lib().trdq_linear_splitk(w._h, int(t), _ptr(codes), _ptr(scales), M, _ptr(bias_bf16), _ptr(out), ldy, _ptr(workspace),
                                    ws_bytes, _stream()), "trdq_linear_splitk")
    return out


STATIC_SCRATCH_ELEMS = 2 * 1024 * 1024


def trdq_linear_splitk_static(w: Weights, t: int, codes, scales, bias_bf16, out):
    """Split-K linear whose partial sums go to the library's built-in scratch array: the call allocates nothing,
    so `out` must be passed in.  For callers that cannot allocate device memory where they call this."""
    M = int(codes.shape[0])
    ldy = int(out.stride(0)) if M > 1 else w.N
    _check(lib().trdq_linear_splitk_static(w._h, int(t), _ptr(codes), _ptr(scales), M, _ptr(bias_bf16), _ptr(out), ldy, _stream()),
           "trdq_linear_splitk_static")
    return out


def trdq_rotate_quantize_asym(rot: Rotation, t: int, X_bf16):
    """Asymmetric per-token quantizer of Eq. 1-3: (codes uint8 [M,K], scales fp32 [M], zero points int32 [M])."""
    import torch
    M = int(X_bf16.shape[0])
    codes = torch.empty((M, rot.K), dtype=torch.uint8, device=X_bf16.device)
    scales = torch.empty((M,), dtype=torch.float32, device=X_bf16.device)
    zp = torch.empty((M,), dtype=torch.int32, device=X_bf16.device)
    ldx = int(X_bf16.stride(0)) if M > 1 else rot.K
    _check(lib().trdq_rotate_quantize_asym(rot._h, int(t), _ptr(X_bf16), ldx, M, _ptr(codes), _ptr(scales), _ptr(zp), _stream()),
           "trdq_rotate_quantize_asym")
    return codes, scales, zp


def trdq_linear_asym(w: Weights, t: int, codes, scales, zero_points, bias_bf16=None, out=None):
    import torch
    M = int(codes.shape[0])
    if out is None:
        out = torch.empty((M, w.N), dtype=torch.bfloat16, device=codes.device)
    ldy = int(out.stride(0)) if M > 1 else w.N
    _check(lib().trdq_linear_asym(w._h, int(t), _ptr(codes), _ptr(scales), _ptr(zero_points), M, _ptr(bias_bf16), _ptr(out), ldy,
                                  _stream()), "trdq_linear_asym")
    return out


def trdq_gemm_i32(w: Weights, t: int, codes, out=None):
    """Raw int32 accumulators [M,N] of the integer GEMM (8-bit weights only)."""
    import torch
    M = int(codes.shape[0])
    if out is None:
        out = torch.empty((M, w.N), dtype=torch.int32, device=codes.device)
    ld = int(out.stride(0)) if M > 1 else w.N
    _check(lib().trdq_gemm_i32(w._h, int(t), _ptr(codes), M, _ptr(out), ld, _stream()), "trdq_gemm_i32")
    return out


class LayerList:
    """A fixed list of trdq_layer_op records (one denoising step's quantized linears).  Holds
    references to every tensor and handle it points to."""

    def __init__(self):
        self._keep = []
        self._extra = []
        self._ops = []
        self._array = None

    def add(self, rot: Rotation, w: Weights, X_bf16, codes, scales, bias_bf16, Y_bf16, act: int = 0, workspace=None) -> None:
        M = int(X_bf16.shape[0])
        assert X_bf16.stride(1) == 1 and Y_bf16.stride(1) == 1 and codes.is_contiguous()
        self._ops.append(LayerOp(rot._h, w._h, _ptr(X_bf16), int(X_bf16.stride(0)) if M > 1 else rot.K, M, _ptr(codes),
                                 _ptr(scales), _ptr(bias_bf16), _ptr(Y_bf16), int(Y_bf16.stride(0)) if M > 1 else w.N, int(act),
                                 _ptr(workspace), 0 if workspace is None else int(workspace.numel() * workspace.element_size())))
        self._keep.append((rot, w, X_bf16, codes, scales, bias_bf16, Y_bf16))
        self._extra.append(workspace)
        self._array = None

    def __len__(self) -> int:
        return len(self._ops)

    def array(self):
        if self._array is None:
            self._array = (LayerOp * len(self._ops))(*self._ops)
        return self._array


def trdq_run_layers(layers: LayerList, t: int, first: int = 0, count: Optional[int] = None) -> None:
    """All (or a slice of) the layer ops at time-step t on the current stream."""
    n = len(layers) - first if count is None else count
    arr = layers.array()
    ptr = C.cast(C.byref(arr, first * C.sizeof(LayerOp)), C.POINTER(LayerOp))
    _check(lib().trdq_run_layers(ptr, int(n), int(t), _stream()), "trdq_run_layers")


def trdq_kernel_choice(stage: int, M: int, K: int, N: int = 0, wbits: int = 8) -> str:
    """Name of the kernel trdq_rotate_quantize (stage 0) or trdq_linear (stage 1) runs for this shape on the current device."""
    buf = C.create_string_buffer(96)
    _check(lib().trdq_kernel_choice(int(stage), int(M), int(K), int(N), int(wbits), buf, 96), "trdq_kernel_choice")
    return buf.value.decode()


def trdq_measure_mma_ceiling(mmas_per_cluster: int) -> int:
    """Launches the tensor-pipe-only kernel on the current stream; returns the integer operations the launch performs."""
    clusters = C.c_int32(0)
    _check(lib().trdq_measure_mma_ceiling(int(mmas_per_cluster), C.byref(clusters), _stream()), "trdq_measure_mma_ceiling")
    return clusters.value * int(mmas_per_cluster) * 2 * 256 * 256 * 32


def trdq_selftest_wait_expiry() -> None:
    """Launches the kernel whose only barrier is never signalled (its wait expires after 20 ms)."""
    _check(lib().trdq_selftest_wait_expiry(_stream()), "trdq_selftest_wait_expiry")


def trdq_device_status() -> int:
    """Synchronises; returns the raw status word (0 = no bounded wait expired) and clears it."""
    word = C.c_uint32(0)
    st = lib().trdq_device_status(C.byref(word))
    if st not in (0, 9):
        raise TrdqError(st, "trdq_device_status")
    return word.value
