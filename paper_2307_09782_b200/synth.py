"""Seeded synthetic inputs shaped like the paper's OPT / LLaMA linear layers.

This module only draws random tensors and converts their storage type.  It holds none of the
method's arithmetic (no quantizer, no scale rule, no number-format encoder), so that the CPU
oracle and the CUDA path can both be fed from it without sharing any code of the method.

Value structure (Section 2, "Distribution of Activations", Fig. 1): activations are close to
normal after layer-norm, with a few channels of much larger magnitude; here those are a seeded
random subset of columns multiplied by a constant factor.  Weights and the two LoRC factors
(Section 3) are zero-mean normal.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np

# tensor ids used to derive independent sub-streams from one seed
_T_X, _T_W, _T_U, _T_V, _T_OUTLIER = 1, 2, 3, 4, 5


@dataclass(frozen=True)
class LayerShape:
    K: int
    N: int
    name: str = ""


@dataclass(frozen=True)
class Workload:
    """One of the five configurations: a set of layer shapes, token counts and quantizer settings."""
    name: str
    seed: int
    shapes: Tuple[LayerShape, ...]
    Ms: Tuple[int, ...]
    modes: Tuple[str, ...]            # subset of ("none", "M1", "M2")
    lorc_rank: int                    # 0 = no LoRC
    outlier_frac: float = 0.0         # fraction of channels that are outliers ...
    outlier_count: int = 0            # ... or an absolute count (used when > 0)
    outlier_factor: float = 20.0
    sigma_w: float = 0.02
    group: int = 128

    def n_outliers(self, K: int) -> int:
        if self.outlier_count > 0:
            return min(self.outlier_count, K)
        return int(round(self.outlier_frac * K))


WORKLOADS = {
    "opt125m": Workload("opt125m", 0, (LayerShape(768, 768, "proj"),), (16,), ("none",), 0,
                        outlier_count=8, outlier_factor=20.0, sigma_w=0.02),
    "opt1.3b": Workload("opt1.3b", 1,
                        (LayerShape(2048, 2048, "qkvo"), LayerShape(2048, 8192, "fc1"),
                         LayerShape(8192, 2048, "fc2")),
                        (1, 16, 128), ("M1",), 8, outlier_frac=0.01),
    "llama7b": Workload("llama7b", 2,
                        (LayerShape(4096, 4096, "qkvo"), LayerShape(4096, 11008, "gate_up"),
                         LayerShape(11008, 4096, "down")),
                        (1, 16, 128, 2048), ("none", "M1", "M2"), 8, outlier_frac=0.01),
    "llama30b": Workload("llama30b", 3,
                         (LayerShape(6656, 17920, "gate_up"), LayerShape(17920, 6656, "down")),
                         (4096,), ("M2",), 8, outlier_frac=0.005, outlier_factor=50.0,
                         sigma_w=0.015),
    "opt30b": Workload("opt30b", 4,
                       (LayerShape(7168, 28672, "fc1"), LayerShape(28672, 7168, "fc2")),
                       (1, 8, 32, 128, 512, 2048, 8192), ("M2",), 8, outlier_frac=0.01),
}


def _rng(seed: int, tensor_id: int, *extra: int) -> np.random.Generator:
    ss = np.random.SeedSequence([int(seed), int(tensor_id), *[int(e) for e in extra]])
    return np.random.Generator(np.random.Philox(ss))


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Storage conversion fp32 -> bfloat16 bit patterns (round to nearest, ties to even)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def outlier_channels(seed: int, K: int, count: int) -> np.ndarray:
    if count <= 0:
        return np.zeros((0,), dtype=np.int64)
    return np.sort(_rng(seed, _T_OUTLIER, K).choice(K, size=count, replace=False)).astype(np.int64)


def make_x(seed: int, M: int, K: int, n_outliers: int = 0, factor: float = 20.0,
           row_offset: int = 0) -> np.ndarray:
    """Activations [M, K] as bfloat16 bit patterns (uint16): N(0,1), outlier channels scaled.

    ``row_offset`` selects a different sub-stream, so that disjoint row blocks (for example the
    shards of different ranks) can be drawn independently of one another.
    """
    x = _rng(seed, _T_X, K, row_offset).standard_normal((M, K), dtype=np.float32)
    ch = outlier_channels(seed, K, n_outliers)
    if ch.size:
        x[:, ch] *= np.float32(factor)
    return f32_to_bf16_bits(x)


def make_w(seed: int, N: int, K: int, sigma: float = 0.02) -> np.ndarray:
    """Weights [N, K] fp32 ~ N(0, sigma), laid out like ``nn.Linear.weight``."""
    w = _rng(seed, _T_W, N, K).standard_normal((N, K), dtype=np.float32)
    w *= np.float32(sigma)
    return w


def make_lorc(seed: int, N: int, K: int, r: int, sigma: float = 0.01) -> Tuple[np.ndarray, np.ndarray]:
    """LoRC factors U [N, r] and V [r, K] as fp16 (returned as float16 arrays)."""
    U = (_rng(seed, _T_U, N, r).standard_normal((N, r), dtype=np.float32) * np.float32(sigma)).astype(np.float16)
    V = (_rng(seed, _T_V, r, K).standard_normal((r, K), dtype=np.float32) * np.float32(sigma)).astype(np.float16)
    return U, V


@dataclass
class LayerInputs:
    M: int
    N: int
    K: int
    x_bits: np.ndarray                 # uint16 [M, K]  bf16 patterns
    W: np.ndarray                      # float32 [N, K]
    U: np.ndarray | None = None        # float16 [N, r]
    V: np.ndarray | None = None        # float16 [r, K]
    r: int = 0
    meta: dict = field(default_factory=dict)


def make_layer(wl: Workload, shape: LayerShape, M: int, with_lorc: bool | None = None) -> LayerInputs:
    r = wl.lorc_rank if (with_lorc is None or with_lorc) else 0
    x = make_x(wl.seed, M, shape.K, wl.n_outliers(shape.K), wl.outlier_factor)
    W = make_w(wl.seed, shape.N, shape.K, wl.sigma_w)
    U = V = None
    if r > 0:
        U, V = make_lorc(wl.seed, shape.N, shape.K, r)
    return LayerInputs(M, shape.N, shape.K, x, W, U, V, r,
                       {"workload": wl.name, "shape": shape.name, "group": wl.group})
