"""Seeded synthetic inputs shaped like the paper's image- and video-DiT workloads.

This module only *draws numbers and lists shapes*.  It performs none of the
method's arithmetic (no rotation, no quantizer, no GEMM): the CPU oracle and the
CUDA library both receive the arrays produced here and each does its own
computation.  numpy is the only dependency, so the module can be imported by the
CPU-only tests, by the GPU tests and by the benchmark alike.

The paper evaluates on PixArt-alpha (images) and Open-Sora (video) with real
prompts (Sec. 4.2, "Setting up").  Neither weights nor datasets are available,
so the generators below stand in for them: same tensor shapes, Gaussian bulk,
and a small set of heavy "massive outlier" channels, which is the structure the
method targets (Sec. 3.2, "Massive Outliers").

bf16 tensors are returned as ``uint16`` arrays holding the bf16 bit patterns
(numpy has no bf16 type).  Values are drawn in fp64, converted to fp32 and then
rounded to bf16 with round-half-to-even.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

BLOCK = 128           # Hadamard block size (Eq. 8: blocks of 2^n x 2^n, n = 7)
T_RANGE = 1000        # diffusion time-steps live in [0, 1000)


# --------------------------------------------------------------------------- #
# bf16 helpers (bit manipulation only)
# --------------------------------------------------------------------------- #
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 -> bf16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + np.uint32(0x7FFF) + lsb
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_bf16_bits(x64: np.ndarray) -> np.ndarray:
    return f32_to_bf16_bits(np.asarray(x64, dtype=np.float64).astype(np.float32))


# --------------------------------------------------------------------------- #
# keyed random streams
# --------------------------------------------------------------------------- #
_TENSOR_IDS = {"x": 1, "w": 2, "bias": 3, "signs": 4, "outlier_channels": 5, "x_text": 6,
               "sample": 7, "aux": 8}


def stream(seed: int, config: int, layer: int, tensor: str, group: int = 0) -> np.random.Generator:
    """Independent generator keyed by (seed, config, layer, tensor, group).

    Philox is counter based, so every key owns a reproducible stream no matter
    in which order tensors are drawn.
    """
    ss = np.random.SeedSequence([int(seed), int(config), int(layer), _TENSOR_IDS[tensor], int(group)])
    return np.random.Generator(np.random.Philox(ss))


# --------------------------------------------------------------------------- #
# workload descriptions
# --------------------------------------------------------------------------- #
@dataclass(frozen=True)
class Layer:
    name: str
    K: int              # input features  (C_in)
    N: int              # output features (C_out)
    M: Optional[int] = None   # rows, when different from the config's M (cross-attention text tokens)


@dataclass(frozen=True)
class Workload:
    index: int                    # position in the list of benchmark configurations
    name: str
    M: int                        # tokens per launch, both CFG halves stacked
    layers: Tuple[Layer, ...]
    num_groups: int               # time-step groups G
    steps: int                    # sampling steps S
    blocks: int                   # transformer blocks per denoising step
    wbits: int = 8
    outlier: str = "none"         # "fixed50" | "student_t3" | "scale30"
    seed: int = 0
    extra_layers: Tuple[Layer, ...] = field(default_factory=tuple)

    @property
    def t_bounds(self) -> np.ndarray:
        return group_bounds(self.num_groups)

    def timesteps(self) -> np.ndarray:
        return sampling_timesteps(self.steps)


DIT_XL2_LAYERS = (
    Layer("qkv", 1152, 3456),
    Layer("proj", 1152, 1152),
    Layer("fc1", 1152, 4608),
    Layer("fc2", 4608, 1152),
)

WORKLOADS: Tuple[Workload, ...] = (
    Workload(0, "single-w8a8-256x1024x1024", 256, (Layer("linear", 1024, 1024),), 2, 2, 1,
             outlier="fixed50"),
    Workload(1, "dit-xl2-256px-b8-cfg", 4096, DIT_XL2_LAYERS, 5, 50, 28, outlier="student_t3"),
    Workload(2, "dit-xl2-512px-b8-cfg", 16384, DIT_XL2_LAYERS, 5, 50, 28, outlier="student_t3"),
    Workload(3, "pixart-1024px-b4-cfg", 32768, DIT_XL2_LAYERS, 4, 20, 28, outlier="student_t3",
             extra_layers=(Layer("xattn_k", 4096, 1152, M=960), Layer("xattn_v", 4096, 1152, M=960))),
    Workload(4, "video-dit-16f-b2-cfg-w4a8", 16384, DIT_XL2_LAYERS, 3, 30, 28, wbits=4,
             outlier="scale30"),
)


def group_bounds(num_groups: int) -> np.ndarray:
    """G contiguous, equal-width intervals of [0, 1000): bounds[g] <= t < bounds[g+1]."""
    g = np.arange(num_groups + 1, dtype=np.int64)
    return ((g * T_RANGE) // num_groups).astype(np.int32)


def sampling_timesteps(steps: int) -> np.ndarray:
    """Descending time-step of sampling step i = 0..S-1: floor((S-1-i) * 1000 / S)."""
    i = np.arange(steps, dtype=np.int64)
    return (((steps - 1 - i) * T_RANGE) // steps).astype(np.int32)


# --------------------------------------------------------------------------- #
# tensors
# --------------------------------------------------------------------------- #
def outlier_channels(wl: Workload, layer_idx: int, K: int) -> np.ndarray:
    if wl.outlier == "fixed50":
        # one fixed channel in each of the first eight 128-blocks
        return np.array([(131 * i + 7) % K for i in range(8)], dtype=np.int64)
    if wl.outlier in ("student_t3", "scale30"):
        n = int(np.ceil(0.01 * K))
        rng = stream(wl.seed, wl.index, layer_idx, "outlier_channels")
        return np.sort(rng.choice(K, size=n, replace=False)).astype(np.int64)
    return np.zeros(0, dtype=np.int64)


def make_x(wl: Workload, layer_idx: int, M: int, K: int, group: int = 0) -> np.ndarray:
    """Activations [M, K] as bf16 bits: N(0,1) bulk plus the workload's outlier channels."""
    rng = stream(wl.seed, wl.index, layer_idx, "x", group)
    x = rng.standard_normal((M, K))
    ch = outlier_channels(wl, layer_idx, K)
    if ch.size:
        if wl.outlier == "fixed50":
            x[:, ch] *= 50.0
        elif wl.outlier == "scale30":
            x[:, ch] *= 30.0
        elif wl.outlier == "student_t3":
            z = rng.standard_normal((M, ch.size))
            chi2 = rng.chisquare(3.0, size=(M, ch.size))
            x[:, ch] = z / np.sqrt(chi2 / 3.0)
    return to_bf16_bits(x)


def make_w(wl: Workload, layer_idx: int, N: int, K: int) -> np.ndarray:
    """Weights [N, K] (K contiguous) as bf16 bits, N(0, 0.02)."""
    rng = stream(wl.seed, wl.index, layer_idx, "w")
    return to_bf16_bits(rng.standard_normal((N, K)) * 0.02)


def make_bias(wl: Workload, layer_idx: int, N: int) -> np.ndarray:
    rng = stream(wl.seed, wl.index, layer_idx, "bias")
    return to_bf16_bits(rng.standard_normal(N) * 0.01)


def make_signs(wl: Workload, layer_idx: int, K: int) -> np.ndarray:
    """Per-group random +-1 diagonal d_g, int8 [G, K]."""
    out = np.empty((wl.num_groups, K), dtype=np.int8)
    for g in range(wl.num_groups):
        rng = stream(wl.seed, wl.index, layer_idx, "signs", g)
        out[g] = (rng.integers(0, 2, size=K, dtype=np.int8) * 2 - 1)
    return out


def group_alphas(num_groups: int) -> np.ndarray:
    """Migration strengths (the per-group hyper-parameter), evenly spread over [0.4, 0.6]."""
    if num_groups == 1:
        return np.array([0.5])
    return np.linspace(0.4, 0.6, num_groups)


def make_smooth(wl: Workload, layer_idx: int, x_bits: np.ndarray, w_bits: np.ndarray) -> np.ndarray:
    """Per-group channel multipliers applied to X, fp32 [G, K].

    A stand-in for calibration: channel maxima of the synthetic X and W are
    combined as in the channel-smoothing formula (Eq. 5) with the group's
    alpha, and the *reciprocal* is returned because the online transform
    multiplies X by this vector (Eq. 10) whereas Eq. 4 divides by it.
    """
    ax = np.abs(bf16_bits_to_f32(x_bits).astype(np.float64)).max(axis=0)
    aw = np.abs(bf16_bits_to_f32(w_bits).astype(np.float64)).max(axis=0)
    ax = np.maximum(ax, 1e-5)
    aw = np.maximum(aw, 1e-5)
    out = np.empty((wl.num_groups, x_bits.shape[1]), dtype=np.float32)
    for g, alpha in enumerate(group_alphas(wl.num_groups)):
        delta = ax ** alpha / aw ** (1.0 - alpha)
        out[g] = (1.0 / delta).astype(np.float32)
    return out


@dataclass
class LayerInputs:
    layer: Layer
    M: int
    x: np.ndarray                 # uint16 [M, K]  (bf16 bits)
    w: np.ndarray                 # uint16 [N, K]
    bias: np.ndarray              # uint16 [N]
    signs: np.ndarray             # int8   [G, K]
    smooth: Optional[np.ndarray]  # fp32   [G, K] or None
    t_bounds: np.ndarray          # int32  [G+1]


def make_layer_inputs(wl: Workload, layer_idx: int, *, M: Optional[int] = None,
                      with_smooth: bool = True, group: int = 0) -> LayerInputs:
    layers = wl.layers + wl.extra_layers
    layer = layers[layer_idx]
    rows = M if M is not None else (layer.M if layer.M is not None else wl.M)
    if layer.M is not None:
        # text embeddings: plain N(0,1) without outlier channels
        rng = stream(wl.seed, wl.index, layer_idx, "x_text", group)
        x = to_bf16_bits(rng.standard_normal((rows, layer.K)))
    else:
        x = make_x(wl, layer_idx, rows, layer.K, group)
    w = make_w(wl, layer_idx, layer.N, layer.K)
    bias = make_bias(wl, layer_idx, layer.N)
    signs = make_signs(wl, layer_idx, layer.K)
    smooth = make_smooth(wl, layer_idx, x, w) if (with_smooth and wl.index != 0) else None
    return LayerInputs(layer, rows, x, w, bias, signs, smooth, wl.t_bounds)


def sample_rows(wl: Workload, layer_idx: int, M: int, count: int, tile: int = 128) -> np.ndarray:
    """Row subset for full-size checks: first and last tile plus a seeded sample."""
    rng = stream(wl.seed, wl.index, layer_idx, "sample")
    edge = np.concatenate([np.arange(min(tile, M)), np.arange(max(0, M - tile), M)])
    extra = rng.choice(M, size=min(count, M), replace=False)
    return np.unique(np.concatenate([edge, extra])).astype(np.int64)
