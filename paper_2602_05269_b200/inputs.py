"""Seeded synthetic inputs for the HGF linear layer, shared by the tests and the benchmark.

This module holds none of the method's arithmetic: it only draws random tensors with the shapes
and value distributions of the workloads and encodes them in the storage types the layer takes
(raw bit patterns, numpy).  It imports neither the CUDA library nor the oracle.

Recipe (one layer, d_in = K, d_out = N, rank r, M tokens):
  W   fp32 [N][K]   ~ N(0, std 0.02)
  x   bf16 [M][K]   ~ N(0, 1) drawn in fp32; floor(0.02 K) channels (a seeded choice, the same
                    channels for every token) multiplied by 20; then rounded to bf16 (nearest even)
  At  fp16 [r][K]   ~ N(0, std 1/sqrt(K))     (A transposed: K contiguous)
  Bt  fp16 [N][r]   ~ N(0, std 1/sqrt(r))     (B transposed: r contiguous)
  gate fp32 [N]     ~ U(0, 1)
Each tensor has its own stream: numpy.random.default_rng([seed, config, layer, kind]).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

KIND_W, KIND_X, KIND_A, KIND_B, KIND_G, KIND_CH = 0, 1, 2, 3, 4, 5


@dataclass(frozen=True)
class LayerShape:
    name: str
    d_in: int
    d_out: int
    r: int


def _block(d: int, ffn: int, r: int):
    """The seven projections of one transformer block."""
    return [LayerShape("q", d, d, r), LayerShape("k", d, d, r), LayerShape("v", d, d, r),
            LayerShape("o", d, d, r), LayerShape("up", d, ffn, r), LayerShape("gate", d, ffn, r),
            LayerShape("down", ffn, d, r)]


# The five workload configurations: layer shapes and token counts.
CONFIGS = {
    0: {"layers": [LayerShape("l0", 512, 512, 16)], "M": [4]},
    1: {"layers": _block(2048, 5632, 32), "M": [1, 4, 16]},
    2: {"layers": _block(3200, 8640, 64), "M": [1, 8]},
    3: {"layers": _block(2048, 5632, 32), "M": [512, 2048, 8192]},
    4: {"layers": _block(4096, 11008, 64), "M": [1, 4096], "n_blocks": 32},
}


def distinct_shapes(config: int):
    seen, out = set(), []
    for s in CONFIGS[config]["layers"]:
        key = (s.d_in, s.d_out, s.r)
        if key not in seen:
            seen.add(key)
            out.append(s)
    return out


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (nearest, ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(a, np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def f32_to_fp16_bits(a: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(a, np.float32).astype(np.float16).view(np.uint16)


def fp16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(b, np.uint16).view(np.float16).astype(np.float32)


def _rng(seed, config, layer, kind):
    return np.random.default_rng([seed, config, layer, kind])


def make_weights(d_out: int, d_in: int, *, seed=0, config=0, layer=0) -> np.ndarray:
    return (_rng(seed, config, layer, KIND_W).standard_normal((d_out, d_in), np.float32)
            * np.float32(0.02))


def make_x(M: int, d_in: int, *, seed=0, config=0, layer=0) -> np.ndarray:
    """bf16 bit patterns [M][d_in] with 2 % outlier channels (x20)."""
    x = _rng(seed, config, layer, KIND_X).standard_normal((M, d_in), np.float32)
    n_out = int(0.02 * d_in)
    ch = _rng(seed, config, layer, KIND_CH).choice(d_in, size=n_out, replace=False)
    x[:, ch] *= np.float32(20.0)
    return f32_to_bf16_bits(x)


def make_lora(d_in: int, d_out: int, r: int, *, seed=0, config=0, layer=0):
    """(At fp16 bits [r][d_in], Bt fp16 bits [d_out][r], gate fp32 [d_out])."""
    At = _rng(seed, config, layer, KIND_A).standard_normal((r, d_in), np.float32) / np.float32(np.sqrt(d_in))
    Bt = _rng(seed, config, layer, KIND_B).standard_normal((d_out, r), np.float32) / np.float32(np.sqrt(r))
    g = _rng(seed, config, layer, KIND_G).random(d_out, np.float32)
    return f32_to_fp16_bits(At), f32_to_fp16_bits(Bt), g


def make_layer(shape: LayerShape, M: int, *, seed=0, config=0, layer=0):
    """All tensors of one layer problem as a dict of numpy arrays."""
    At, Bt, g = make_lora(shape.d_in, shape.d_out, shape.r, seed=seed, config=config, layer=layer)
    return {
        "W": make_weights(shape.d_out, shape.d_in, seed=seed, config=config, layer=layer),
        "x": make_x(M, shape.d_in, seed=seed, config=config, layer=layer),
        "At": At, "Bt": Bt, "gate": g,
        "d_in": shape.d_in, "d_out": shape.d_out, "r": shape.r, "M": M,
    }
