"""Seeded synthetic inputs shaped like the paper's SR workloads.

This module holds no ConvAttn arithmetic: it only draws random arrays, rounds
them to the storage dtype, and converts between logical ``[B,C,H,W]`` order and
the two memory layouts.  Both the CUDA path and the CPU oracle are fed from
here so that they see exactly the same stored values.

Shapes follow the paper's setting (feature width C=64, 16 attention channels,
13x13 large kernel, LR maps of 320x180 / 640x360 for HD output, 64x64 training
patches in batches of 64); values are white noise because the kernel's run time
does not depend on the data.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

F32 = "f32"
BF16 = "bf16"
NCHW = "nchw"
NHWC = "nhwc"


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    C: int
    C_a: int
    H: int
    W: int
    K: int
    dtype: str
    seed: int
    per_image_scale: bool = False

    @property
    def pixels(self) -> int:
        return self.B * self.H * self.W


# The five evaluation configurations (smallest first).
WORKLOADS = (
    Workload("cfg1_64x64_f32", 1, 64, 16, 64, 64, 13, F32, 0),
    Workload("cfg2_320x180_f32", 1, 64, 16, 180, 320, 13, F32, 1),
    Workload("cfg3_640x360_bf16", 1, 64, 16, 360, 640, 13, BF16, 2),
    Workload("cfg4_b64_64x64_bf16", 64, 64, 16, 64, 64, 13, BF16, 3, True),
    Workload("cfg5_1920x1080_ca32_bf16", 1, 64, 32, 1080, 1920, 13, BF16, 4),
)
WORKLOADS_BY_NAME = {w.name: w for w in WORKLOADS}


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even), returned as uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    r = ((u + bias) >> 16).astype(np.uint16)
    nan = np.isnan(a)
    if nan.any():
        r = np.where(nan, np.uint16(0x7FC0), r)
    return r


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to float32 exactly."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def round_to(a: np.ndarray, dtype: str) -> np.ndarray:
    """float32 array holding the values that survive storage in `dtype`."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == F32:
        return a
    if dtype == BF16:
        return bf16_bits_to_f32(f32_to_bf16_bits(a))
    raise ValueError(dtype)


def to_layout(a_nchw: np.ndarray, layout: str) -> np.ndarray:
    """Dense memory image of a logical [B,C,H,W] array in the given layout."""
    if layout == NCHW:
        return np.ascontiguousarray(a_nchw)
    if layout == NHWC:
        return np.ascontiguousarray(np.transpose(a_nchw, (0, 2, 3, 1)))
    raise ValueError(layout)


def from_layout(a_mem: np.ndarray, layout: str) -> np.ndarray:
    """Inverse of to_layout: back to logical [B,C,H,W]."""
    if layout == NCHW:
        return np.ascontiguousarray(a_mem)
    if layout == NHWC:
        return np.ascontiguousarray(np.transpose(a_mem, (0, 3, 1, 2)))
    raise ValueError(layout)


def _kaiming_uniform(rng, shape, fan_in):
    bound = 1.0 / np.sqrt(float(fan_in))
    return rng.uniform(-bound, bound, size=shape).astype(np.float32)


def make_inputs(B, C, C_a, H, W, K=13, dtype=F32, seed=0, per_image_scale=False, channel_means=False):
    """Draw one problem instance.

    Returns a dict of float32 arrays already rounded to `dtype`:
      x [B,C,H,W] ~ N(0,1) (times a per-image U(0.5,2) scale if asked; plus a
      per-(image,channel) mean ~ U(-2,2) if `channel_means`, which makes the GAP
      path matter), w_large [C_a,K,K], w_dyn [9*C_a,C_a], b_dyn [9*C_a], all three
      kaiming-uniform: U(-1/sqrt(fan_in), 1/sqrt(fan_in)) with fan_in K*K, C_a, C_a.
    """
    rng = np.random.default_rng(seed)
    x = rng.standard_normal(size=(B, C, H, W), dtype=np.float32)
    if per_image_scale:
        x *= rng.uniform(0.5, 2.0, size=(B, 1, 1, 1)).astype(np.float32)
    if channel_means:
        x += rng.uniform(-2.0, 2.0, size=(B, C, 1, 1)).astype(np.float32)
    w_large = _kaiming_uniform(rng, (C_a, K, K), K * K)
    w_dyn = _kaiming_uniform(rng, (9 * C_a, C_a), C_a)
    b_dyn = _kaiming_uniform(rng, (9 * C_a,), C_a)
    return {
        "x": round_to(x, dtype),
        "w_large": round_to(w_large, dtype),
        "w_dyn": round_to(w_dyn, dtype),
        "b_dyn": round_to(b_dyn, dtype),
    }


def make_estimator_mlp(C_a, h, dtype=F32, seed=0):
    """Weights of the two-layer kernel estimator (hidden width h), float32 arrays rounded to `dtype`:
    w_down [h,C_a], b_down [h] ~ U(-1,1)/sqrt(C_a) * 4 (so that the pre-activations of pooled
    features of order one fall across the curved part of the activation, not only its linear tails),
    w_up [9*C_a,h], b_up [9*C_a] kaiming-uniform with fan_in h."""
    rng = np.random.default_rng(1000003 * (seed + 1) + h)
    w_down = 4.0 * _kaiming_uniform(rng, (h, C_a), C_a)
    b_down = 4.0 * _kaiming_uniform(rng, (h,), C_a)
    w_up = _kaiming_uniform(rng, (9 * C_a, h), h)
    b_up = _kaiming_uniform(rng, (9 * C_a,), h)
    return {
        "w_down": round_to(w_down, dtype),
        "b_down": round_to(b_down, dtype),
        "w_up": round_to(w_up, dtype),
        "b_up": round_to(b_up, dtype),
    }


def make_pointwise(C_a, dtype=F32, seed=0):
    """w_point [C_a,C_a] (row = output channel): the 1x1 large-kernel filter of the decomposed form,
    kaiming-uniform with fan_in C_a plus the identity, float32 rounded to `dtype`."""
    rng = np.random.default_rng(7000003 * (seed + 1) + C_a)
    w = _kaiming_uniform(rng, (C_a, C_a), C_a) + np.eye(C_a, dtype=np.float32)
    return round_to(w, dtype)


def make_fuse(C, dtype=F32, seed=0):
    """w_fuse [C,C] (row = output channel) and b_fuse [C] of the module's closing 1x1 convolution, kaiming-uniform
    with fan_in C, float32 rounded to `dtype`."""
    rng = np.random.default_rng(11000027 * (seed + 1) + C)
    return {"w_fuse": round_to(_kaiming_uniform(rng, (C, C), C), dtype), "b_fuse": round_to(_kaiming_uniform(rng, (C,), C), dtype)}


def make_dense_kernel(C_a, K=13, dtype=F32, seed=0):
    """w_dense [C_a,C_a,K,K] (output channel, input channel, row, column): the dense large kernel of the main
    model, kaiming-uniform with fan_in C_a*K*K, float32 rounded to `dtype`."""
    rng = np.random.default_rng(9000011 * (seed + 1) + C_a * 31 + K)
    return round_to(_kaiming_uniform(rng, (C_a, C_a, K, K), C_a * K * K), dtype)


def make_workload(wl: Workload, channel_means=False):
    return make_inputs(wl.B, wl.C, wl.C_a, wl.H, wl.W, wl.K, wl.dtype, wl.seed, wl.per_image_scale,
                       channel_means)
