"""Seeded synthetic inputs for the VeLoRA linear-layer path.

Serves both the CPU oracle and the CUDA library (through the tests and the
benchmark) and holds none of the method's arithmetic: it only draws random
tensors with the shapes and value distributions of the workloads the paper
trains on (arxiv 2405.17991, Section 4: ViT-B/16, LLaMA pre-training and
fine-tuning), rounds them ONCE to the storage type, and hands out the very
same bit patterns to every consumer.

Recipe (one counter-based Philox stream per tensor, key = (1000*config + layer, stream)):
  X  = G * diag(c): G ~ N(0,1), c a per-channel scale drawn per config
       (config 3: c = 20 on a seeded 1 % of the channels, 1 elsewhere)
  W  ~ N(0, 1/D)   (config 1: N(0,1))
  dY ~ N(0, sigma_dy^2)
fp32 masters, then one round-to-nearest-even to bfloat16 for the bf16 configs.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

_STREAM_X, _STREAM_SCALE, _STREAM_W, _STREAM_DY, _STREAM_ROWS = 1, 2, 3, 4, 5


@dataclass(frozen=True)
class Layer:
    name: str
    D: int          # input width
    O: int          # output width


@dataclass(frozen=True)
class Config:
    index: int
    name: str
    dtype: str                      # "f32" or "bf16": storage type of X, W, dY
    N: int                          # tokens (batch x sequence, flattened)
    layers: Tuple[Layer, ...]
    Dsubs: Tuple[int, ...]          # sub-token lengths to run (first = default)
    scale: str                      # "none" | "lognormal" | "outlier"
    scale_sigma: float = 0.0
    sigma_dy: float = 1.0
    w_unit_variance: bool = False


def _llama(hidden: int, mlp: int) -> Tuple[Layer, ...]:
    return (
        Layer("q", hidden, hidden), Layer("k", hidden, hidden), Layer("v", hidden, hidden),
        Layer("o", hidden, hidden), Layer("up", hidden, mlp), Layer("gate", hidden, mlp),
        Layer("down", mlp, hidden),
    )


CONFIGS: Dict[int, Config] = {
    1: Config(1, "tiny-fp32", "f32", 256, (Layer("lin", 64, 64),), (16,), "none", sigma_dy=1.0,
              w_unit_variance=True),
    2: Config(2, "llama60m-block", "bf16", 32 * 256, _llama(512, 1376), (64,), "lognormal", 0.5),
    3: Config(3, "vit-b16-block", "bf16", 64 * 197,
              (Layer("qkv", 768, 2304), Layer("proj", 768, 768), Layer("fc1", 768, 3072),
               Layer("fc2", 3072, 768)), (32,), "outlier"),
    4: Config(4, "llama1b-block", "bf16", 16 * 256, _llama(2048, 5461), (128,), "lognormal", 0.5,
              sigma_dy=0.1),
    5: Config(5, "llama7b-block", "bf16", 4 * 2048, _llama(4096, 11008), (64, 256), "lognormal", 1.0),
}


def num_subtokens(D: int, Dsub: int) -> int:
    return -(-D // Dsub)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    u = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Array:
    """One stored tensor: ``bits`` is uint16 (bf16 patterns) or float32, row-major."""
    bits: np.ndarray
    dtype: str

    @property
    def shape(self):
        return self.bits.shape

    def f64(self) -> np.ndarray:
        """Exact widening of the stored values to float64."""
        if self.dtype == "bf16":
            return bf16_bits_to_f32(self.bits).astype(np.float64)
        return self.bits.astype(np.float64)

    def rows(self, idx) -> "Array":
        return Array(np.ascontiguousarray(self.bits[idx]), self.dtype)

    def cols(self, idx) -> "Array":
        return Array(np.ascontiguousarray(self.bits[:, idx]), self.dtype)

    def torch(self, device="cpu", ld: Optional[int] = None):
        """Torch tensor with the same bit patterns; ``ld`` pads the row pitch (returns a view)."""
        import torch
        if self.dtype == "bf16":
            t = torch.from_numpy(self.bits.view(np.int16).copy()).view(torch.bfloat16)
        else:
            t = torch.from_numpy(self.bits.copy())
        if ld is not None and t.ndim == 2 and ld != t.shape[1]:
            buf = torch.zeros((t.shape[0], ld), dtype=t.dtype)
            buf[:, : t.shape[1]] = t
            t = buf
            return t.to(device)[:, : self.bits.shape[1]]
        return t.to(device)


def from_values(a: np.ndarray, dtype: str) -> Array:
    """Store fp32 master values in ``dtype`` (one rounding for bf16)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "bf16":
        return Array(f32_to_bf16_bits(a), "bf16")
    if dtype == "f32":
        return Array(a, "f32")
    raise ValueError(dtype)


def _rng(cfg_index: int, layer_index: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[1000 * cfg_index + layer_index, stream]))


def _normal(rng, shape, sigma=1.0) -> np.ndarray:
    a = rng.standard_normal(shape, dtype=np.float32)
    if sigma != 1.0:
        a *= np.float32(sigma)
    return a


def channel_scale(cfg: Config, layer_index: int, D: int) -> np.ndarray:
    rng = _rng(cfg.index, layer_index, _STREAM_SCALE)
    if cfg.scale == "none":
        return np.ones(D, dtype=np.float32)
    if cfg.scale == "lognormal":
        return np.exp(cfg.scale_sigma * rng.standard_normal(D)).astype(np.float32)
    if cfg.scale == "outlier":
        c = np.ones(D, dtype=np.float32)
        k = max(1, int(round(0.01 * D)))
        c[rng.choice(D, size=k, replace=False)] = 20.0
        return c
    raise ValueError(cfg.scale)


def make_X(cfg: Config, layer_index: int, N: Optional[int] = None) -> Array:
    layer = cfg.layers[layer_index]
    n = cfg.N if N is None else N
    g = _normal(_rng(cfg.index, layer_index, _STREAM_X), (n, layer.D))
    g *= channel_scale(cfg, layer_index, layer.D)[None, :]
    return from_values(g, cfg.dtype)


def make_W(cfg: Config, layer_index: int) -> Array:
    layer = cfg.layers[layer_index]
    sigma = 1.0 if cfg.w_unit_variance else float(layer.D) ** -0.5
    return from_values(_normal(_rng(cfg.index, layer_index, _STREAM_W), (layer.O, layer.D), sigma), cfg.dtype)


def make_dY(cfg: Config, layer_index: int, N: Optional[int] = None) -> Array:
    layer = cfg.layers[layer_index]
    n = cfg.N if N is None else N
    return from_values(_normal(_rng(cfg.index, layer_index, _STREAM_DY), (n, layer.O), cfg.sigma_dy), cfg.dtype)


def sample_rows(cfg: Config, layer_index: int, total: int, count: int, salt: int = 0) -> np.ndarray:
    """Sorted seeded sample of ``count`` distinct indices in [0, total)."""
    rng = np.random.Generator(np.random.Philox(key=[1000 * cfg.index + layer_index, _STREAM_ROWS + salt]))
    count = min(count, total)
    return np.sort(rng.choice(total, size=count, replace=False))


def small_case(seed: int, N: int, D: int, O: int, dtype: str = "bf16", sigma_dy: float = 1.0,
               mean_offset: float = 0.0) -> Dict[str, Array]:
    """Free-form seeded case for edge-shape tests: X (lognormal channel scales), W, dY."""
    def rng(stream):
        return np.random.Generator(np.random.Philox(key=[seed, stream]))
    x = _normal(rng(_STREAM_X), (N, D))
    x *= np.exp(0.5 * rng(_STREAM_SCALE).standard_normal(D)).astype(np.float32)[None, :]
    if mean_offset:
        x += np.float32(mean_offset)
    w = _normal(rng(_STREAM_W), (O, D), float(D) ** -0.5)
    dy = _normal(rng(_STREAM_DY), (N, O), sigma_dy)
    return {"X": from_values(x, dtype), "W": from_values(w, dtype), "dY": from_values(dy, dtype)}
