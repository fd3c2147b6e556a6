"""Seeded synthetic ViT-shaped inputs for the MXFP4 linear layer.

This module is shared by the tests, the benchmark and the CPU oracle's callers.  It holds only
the input recipe (shapes, distributions, seeds, bf16 rounding of the generated values) and none
of the method's arithmetic.

The tensors stand in for the DeiT activations / weights / gradients of the paper's ImageNet-1K
runs, which are not available: activations ~ N(0,1) with a few outlier channels, weights
truncated-normal(std 0.02), gradients heavy-tailed (Student-t, 3 degrees of freedom) and small.
"""
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Layer:
    name: str
    M: int  # tokens
    K: int  # in features
    N: int  # out features
    x_law: str = "normal"  # "normal" | "gelu"
    outlier_frac: float = 0.0  # fraction of channels scaled by outlier_gain (0 => use outlier_count)
    outlier_count: int = 0
    outlier_gain: float = 1.0
    dy_scale: float = 1e-3
    qema: bool = False
    osc: bool = False  # per-element oscillation counters (Sec. 6.1) kept with the weight quantizer


# The workloads.  Token counts of 1-5: 1024, 128*197, 256*197.
CONFIGS = {
    1: [Layer("deit_tiny_fc1", 1024, 192, 768, outlier_count=4, outlier_gain=20.0)],
    2: [Layer("deit_small_fc1", 25216, 384, 1536, outlier_count=4, outlier_gain=20.0, qema=True),
        Layer("deit_small_fc2", 25216, 1536, 384, outlier_count=4, outlier_gain=20.0, qema=True)],
    3: [Layer("deit_base_qkv", 50432, 768, 2304, outlier_frac=0.01, outlier_gain=50.0),
        Layer("deit_base_proj", 50432, 768, 768, outlier_frac=0.01, outlier_gain=50.0)],
    4: [Layer("vit_large_fc1", 50432, 1024, 4096, dy_scale=1e-4),
        Layer("vit_large_fc2", 50432, 4096, 1024, x_law="gelu", dy_scale=1e-4)],
    5: [Layer("deit_small_qkv", 25216, 384, 1152, qema=True, osc=True),
        Layer("deit_small_proj", 25216, 384, 384, qema=True, osc=True),
        Layer("deit_small_fc1", 25216, 384, 1536, qema=True, osc=True),
        Layer("deit_small_fc2", 25216, 1536, 384, x_law="gelu", qema=True, osc=True)],
    # Swin-T at batch 128: 56x56, 28x28 and 7x7 tokens per image with 96, 192 and 768 channels.  Feature counts that
    # are not multiples of 128 (96, 288) and token counts whose last 128-row tile is partial.
    6: [Layer("swin_t_s1_qkv", 401408, 96, 288, outlier_count=2, outlier_gain=20.0),
        Layer("swin_t_s1_fc1", 401408, 96, 384, outlier_count=2, outlier_gain=20.0),
        Layer("swin_t_s1_fc2", 401408, 384, 96, x_law="gelu"),
        Layer("swin_t_s2_proj", 100352, 192, 192, outlier_count=2, outlier_gain=20.0),
        Layer("swin_t_s4_qkv", 6272, 768, 2304, outlier_frac=0.01, outlier_gain=50.0)],
}


def tensor_seed(config: int, layer: int, which: str) -> int:
    """Seed of one tensor: 1000*config + 10*layer + {X:0, W:1, dY:2}."""
    return 1000 * config + 10 * layer + {"X": 0, "W": 1, "dY": 2}[which]


def sr_seed(config: int, layer: int) -> int:
    """Seed of the stochastic-rounding streams of one layer's backward pass."""
    return 0x5EED0000 + 1000 * config + 10 * layer


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); returned as float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """The 16-bit patterns of float32 values that are already bf16-representable."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return (u >> np.uint32(16)).astype(np.uint16)


def _normal(rng, shape):
    return rng.standard_normal(shape, dtype=np.float32)


def _student_t3(rng, shape):
    z = _normal(rng, shape)
    c = np.zeros(shape, dtype=np.float32)
    for _ in range(3):
        g = _normal(rng, shape)
        c += g * g
    return z / np.sqrt(c / 3.0)


def make_x(layer: Layer, seed: int, rows: int = None) -> np.ndarray:
    rows = layer.M if rows is None else rows
    rng = np.random.Generator(np.random.PCG64(seed))
    x = _normal(rng, (rows, layer.K))
    if layer.x_law == "gelu":
        from math import sqrt
        try:
            from scipy.special import erf
            x = (0.5 * x * (1.0 + erf(x / sqrt(2.0)))).astype(np.float32)
        except ImportError:  # tanh form
            x = (0.5 * x * (1.0 + np.tanh(0.7978845608 * (x + 0.044715 * x ** 3)))).astype(np.float32)
    n_out = layer.outlier_count or int(round(layer.outlier_frac * layer.K))
    if n_out:
        ch = rng.choice(layer.K, size=n_out, replace=False)
        x[:, ch] *= np.float32(layer.outlier_gain)
    return round_to_bf16(x)


def make_w(layer: Layer, seed: int, std: float = 0.02) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(seed))
    w = _normal(rng, (layer.N, layer.K))
    bad = np.abs(w) > 2.0
    while bad.any():
        w[bad] = _normal(rng, int(bad.sum()))
        bad = np.abs(w) > 2.0
    return round_to_bf16(w * np.float32(std))


def make_dy(layer: Layer, seed: int, rows: int = None) -> np.ndarray:
    rows = layer.M if rows is None else rows
    rng = np.random.Generator(np.random.PCG64(seed))
    return round_to_bf16(_student_t3(rng, (rows, layer.N)) * np.float32(layer.dy_scale))


def make_ema(layer: Layer, w: np.ndarray, seed: int, steps: int = 3):
    """EMA state that differs from the weight: start at ema = W, then perturb W ``steps`` times by
    N(0, (1e-3*0.02)^2) and return (w_perturbed_history, ema0).  No EMA arithmetic happens here:
    the caller runs the quantizer under test over the history."""
    rng = np.random.Generator(np.random.PCG64(seed + 7))
    hist = []
    cur = w.copy()
    for _ in range(steps):
        cur = round_to_bf16(cur + _normal(rng, w.shape) * np.float32(1e-3 * 0.02))
        hist.append(cur)
    return hist, w.astype(np.float32).copy()


def make_layer(config: int, layer_idx: int, rows: int = None):
    """All three tensors of one layer of one config, as float32 arrays of bf16-exact values."""
    layer = CONFIGS[config][layer_idx]
    x = make_x(layer, tensor_seed(config, layer_idx, "X"), rows)
    w = make_w(layer, tensor_seed(config, layer_idx, "W"))
    dy = make_dy(layer, tensor_seed(config, layer_idx, "dY"), rows)
    return layer, x, w, dy
