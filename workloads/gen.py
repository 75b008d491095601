"""Seeded synthetic tensors shaped like the paper's rollout linears.

The paper measures on Qwen2.5-3B (GSM8K) and Qwen2.5-Math-7B (DAPO-Math-17K)
rollouts (Section 5.1); neither weights nor data are available offline, so these
tensors stand in for them: same layer shapes, Gaussian bulk, and a few outlier
channels that dominate their quantization blocks (the structure Section 4.2 and
Figures 1-2 describe).  Everything is generated on the host with numpy's
``default_rng`` and rounded to bf16 (round-to-nearest-even); the same bit
patterns feed the CPU oracle and the CUDA library.

No arithmetic of the method lives here.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import numpy as np

# Pattern ids are part of the input description (which S the config asks for);
# they mirror the C enum in include/resq.h.
S_NONE, S_DENSE, S_2_4, S_ROW50, S_CHAN50, S_BLOCK = 0, 1, 2, 3, 4, 5


@dataclass(frozen=True)
class LayerSpec:
    name: str
    K: int  # input features (paper: d)
    N: int  # output features (paper: n)
    silu_mul_input: bool = False  # activation is SiLU(g)*u (input of down_proj)


@dataclass(frozen=True)
class WorkloadConfig:
    index: int
    name: str
    M: int  # tokens (paper: m)
    layers: Tuple[LayerSpec, ...]
    outlier_scale: float
    outlier_frac: float  # fraction of channels scaled; 0 => use outlier_count
    outlier_count: int
    w_std: float
    patterns: Tuple[int, ...]
    formats: Tuple[str, ...] = ("hif4",)


_Q3B = (
    LayerSpec("qkv", 2048, 2560),
    LayerSpec("o", 2048, 2048),
    LayerSpec("gate_up", 2048, 22016),
    LayerSpec("down", 11008, 2048, silu_mul_input=True),
)
_Q7B = (
    LayerSpec("qkv", 3584, 4608),
    LayerSpec("o", 3584, 3584),
    LayerSpec("gate_up", 3584, 37888),
    LayerSpec("down", 18944, 3584, silu_mul_input=True),
)

CONFIGS: Tuple[WorkloadConfig, ...] = (
    WorkloadConfig(0, "tiny", 64, (LayerSpec("lin", 2048, 2048),), 64.0, 0.0, 8, 0.02, (S_2_4,)),
    WorkloadConfig(1, "qwen2.5-3b-decode", 256, _Q3B, 50.0, 0.005, 0, 0.02, (S_2_4,)),
    WorkloadConfig(2, "qwen2.5-3b-prefill", 8192, _Q3B, 50.0, 0.005, 0, 0.02,
                   (S_ROW50, S_CHAN50), ("hif4", "mxfp4")),
    WorkloadConfig(3, "qwen2.5-math-7b-decode", 512, _Q7B, 100.0, 0.005, 0, 0.015, (S_BLOCK,)),
    WorkloadConfig(4, "qwen2.5-math-7b-prefill", 16384, _Q7B, 100.0, 0.005, 0, 0.015,
                   (S_DENSE, S_2_4, S_ROW50, S_CHAN50, S_BLOCK), ("hif4", "mxfp4")),
)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 bit patterns (uint16), round-to-nearest-even. Finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to float32 exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def tensor_seed(config: int, layer: int, which: int) -> int:
    """which: 0 = activation X, 1 = weight W."""
    return 1000 * config + 10 * layer + which


def _normal_f32(rng: np.random.Generator, shape, chunk_rows: int = 4096) -> np.ndarray:
    rows, cols = shape
    out = np.empty((rows, cols), dtype=np.float32)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        rng.standard_normal((r1 - r0, cols), dtype=np.float32, out=out[r0:r1])
    return out


def make_activation(cfg: WorkloadConfig, layer_idx: int, M: int | None = None) -> np.ndarray:
    """bf16 bit patterns [M, K] of the activation entering layer `layer_idx`."""
    spec = cfg.layers[layer_idx]
    M = cfg.M if M is None else M
    rng = np.random.default_rng(tensor_seed(cfg.index, layer_idx, 0))
    if spec.silu_mul_input:
        g = _normal_f32(rng, (M, spec.K))
        u = _normal_f32(rng, (M, spec.K))
        # SiLU(g) * u = g * u / (1 + exp(-g)), evaluated in float32
        den = np.exp(-g)
        den += np.float32(1.0)
        x = g
        x *= u
        x /= den
        del den, u
    else:
        x = _normal_f32(rng, (M, spec.K))
    n_out = cfg.outlier_count if cfg.outlier_count > 0 else int(math.ceil(cfg.outlier_frac * spec.K))
    ch = np.sort(rng.choice(spec.K, size=n_out, replace=False))
    x[:, ch] *= np.float32(cfg.outlier_scale)
    np.nan_to_num(x, copy=False, nan=0.0, posinf=0.0, neginf=0.0)
    return f32_to_bf16_bits(x)


def make_weight(cfg: WorkloadConfig, layer_idx: int) -> np.ndarray:
    """bf16 bit patterns [N, K] of the layer weight, N(0, w_std)."""
    spec = cfg.layers[layer_idx]
    rng = np.random.default_rng(tensor_seed(cfg.index, layer_idx, 1))
    w = _normal_f32(rng, (spec.N, spec.K))
    w *= np.float32(cfg.w_std)
    return f32_to_bf16_bits(w)


def make_layer(cfg: WorkloadConfig, layer_idx: int, M: int | None = None,
               N: int | None = None) -> Tuple[np.ndarray, np.ndarray]:
    """(X bits [M,K], W bits [N,K]).  `N` keeps only the first N weight rows (sampling)."""
    x = make_activation(cfg, layer_idx, M)
    w = make_weight(cfg, layer_idx)
    if N is not None:
        w = np.ascontiguousarray(w[:N])
    return x, w
