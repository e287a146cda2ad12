"""Seeded synthetic inputs for the LoRaQ fused-linear hot path.

This module holds none of the method's arithmetic (no quantizer, no matmul of
the layer, no calibration).  It only draws tensors whose shapes and outlier
structure imitate the PixArt-class and SANA-class diffusion-transformer linears
the paper evaluates (Section 4.1, "Models"); the real activations and weights
are not available offline, so these stand in for them.  Both the CUDA path and
the CPU oracle are fed the arrays produced here, so the random-number code is
never a parity risk.

Generator: a counter-based stream.  Element ``i`` of the tensor with 64-bit key
``k`` is ``splitmix64(k + i * GOLDEN)``; two such words give one normal deviate
through Box-Muller.  The same (seed, config, layer, tag) always yields the same
array on every machine.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _splitmix64(z: np.ndarray) -> np.ndarray:
    z = z.astype(np.uint64, copy=True)
    z ^= z >> np.uint64(30)
    z *= _M1
    z ^= z >> np.uint64(27)
    z *= _M2
    z ^= z >> np.uint64(31)
    return z


def tensor_key(seed: int, config: int, layer: str, tag: str) -> int:
    """64-bit key of one tensor: a hash of (base seed, config number, layer name, tag)."""
    h = hashlib.sha256(f"{seed}/{config}/{layer}/{tag}".encode()).digest()
    return int.from_bytes(h[:8], "little")


def uniform01(key: int, n: int, stream: int = 0) -> np.ndarray:
    """n doubles in (0, 1), element i depends only on (key, stream, i)."""
    with np.errstate(over="ignore"):
        ctr = (np.arange(n, dtype=np.uint64) * np.uint64(2) + np.uint64(stream)) * _GOLDEN
        w = _splitmix64(ctr + np.uint64(key & 0xFFFFFFFFFFFFFFFF))
    return ((w >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(key: int, n: int) -> np.ndarray:
    """n standard-normal doubles (Box-Muller on two counter-based uniform streams)."""
    u1 = uniform01(key, n, 0)
    u2 = uniform01(key, n, 1)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def permutation(key: int, n: int) -> np.ndarray:
    """Seeded permutation of range(n) (argsort of a uniform stream)."""
    return np.argsort(uniform01(key ^ 0x5DEECE66D, n, 0), kind="stable")


def _gelu(z: np.ndarray) -> np.ndarray:
    # tanh form; this only shapes an input distribution, it is not part of the method
    return 0.5 * z * (1.0 + np.tanh(0.7978845608028654 * (z + 0.044715 * z ** 3)))


def make_activations(seed: int, config: int, layer: str, M: int, K: int,
                     n_outlier: int, outlier_scale: float = 20.0,
                     gelu_shaped: bool = False) -> np.ndarray:
    """X fp16 [M, K] ~ N(0,1) (or GELU(N(0,1)): non-negative-skewed, as an MLP's
    second linear sees), with ``n_outlier`` seeded channels scaled by ``outlier_scale``."""
    key = tensor_key(seed, config, layer, "X")
    x = normal(key, M * K).reshape(M, K)
    if gelu_shaped:
        x = _gelu(x)
    ch = permutation(key, K)[:n_outlier]
    x[:, ch] *= outlier_scale
    return x.astype(np.float16)


def make_weight(seed: int, config: int, layer: str, K: int, N: int,
                n_outlier: int, std: float = 0.02, outlier_scale: float = 10.0) -> np.ndarray:
    """W fp16 [K, N] (the paper's d x n orientation, Section 3.1) ~ N(0, std^2) with
    ``n_outlier`` seeded input channels (rows) scaled by ``outlier_scale``."""
    key = tensor_key(seed, config, layer, "W")
    w = normal(key, K * N).reshape(K, N) * std
    ch = permutation(key, K)[:n_outlier]
    w[ch, :] *= outlier_scale
    return w.astype(np.float16)


def make_bias(seed: int, config: int, layer: str, N: int, std: float = 0.02) -> np.ndarray:
    key = tensor_key(seed, config, layer, "b")
    return (normal(key, N) * std).astype(np.float16)


@dataclass(frozen=True)
class LayerSpec:
    name: str
    K: int
    N: int
    gelu_in: bool = False


# hidden 1152, MLP 4608 (PixArt-class block linears)
PIXART_LAYERS = (
    LayerSpec("qkv", 1152, 3456),
    LayerSpec("attn_out", 1152, 1152),
    LayerSpec("fc1", 1152, 4608),
    LayerSpec("fc2", 4608, 1152, gelu_in=True),
)

# hidden 2240, MLP 5600 (SANA-class linear-attention block; pointwise convs as linears)
SANA_LAYERS = (
    LayerSpec("qkv", 2240, 6720),
    LayerSpec("out", 2240, 2240),
    LayerSpec("mlp_up", 2240, 5600),
    LayerSpec("mlp_down", 5600, 2240),
)


@dataclass(frozen=True)
class Workload:
    config: int
    layers: tuple
    M: int
    rank: int
    branch: str            # "w8a8" | "w6a6" | "w4a8" | "w16a16" | "none"
    act_outliers: object   # int, or callable K -> int
    w_outliers: object

    def n_act_outliers(self, K: int) -> int:
        return self.act_outliers(K) if callable(self.act_outliers) else int(self.act_outliers)

    def n_w_outliers(self, K: int) -> int:
        return self.w_outliers(K) if callable(self.w_outliers) else int(self.w_outliers)


def _one_percent(K: int) -> int:
    return max(1, K // 100)


def workload(config: int, branch: str | None = None, rank: int = 32, M: int | None = None) -> Workload:
    """The five benchmark configurations (shapes, row counts, outlier recipe)."""
    if config == 0:
        return Workload(0, (LayerSpec("linear", 1152, 1152),), M or 256, rank, branch or "w8a8", 8, 4)
    if config in (1, 2):
        return Workload(config, PIXART_LAYERS, M or 8192, rank, branch or "w8a8", 8, 4)
    if config == 3:
        return Workload(3, SANA_LAYERS, M or 8192, rank, branch or "w4a8", _one_percent, _one_percent)
    if config == 4:
        return Workload(4, PIXART_LAYERS, M or 32768, rank, branch or "w8a8", 8, 4)
    raise ValueError(f"unknown config {config}")


def layer_inputs(wl: Workload, spec: LayerSpec, seed: int = 0, M: int | None = None,
                 with_bias: bool = False):
    """(X fp16 [M,K], W fp16 [K,N], bias fp16 [N] or None) for one layer of a workload.
    Configs 1, 2 and 4 share tensors (same seeds), as the sweep configs require."""
    cfg_key = 1 if wl.config in (1, 2, 4) else wl.config
    m = M or wl.M
    X = make_activations(seed, cfg_key, spec.name, m, spec.K, wl.n_act_outliers(spec.K),
                         gelu_shaped=spec.gelu_in)
    W = make_weight(seed, cfg_key, spec.name, spec.K, spec.N, wl.n_w_outliers(spec.K))
    b = make_bias(seed, cfg_key, spec.name, spec.N) if with_bias else None
    return X, W, b
