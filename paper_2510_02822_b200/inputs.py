"""Seeded synthetic inputs shaped like the paper's CNN / ViT workloads.

This module only draws numbers: a counter-based generator (splitmix64 -> uniform ->
Box-Muller) fills tensors whose shapes and per-channel range structure follow the layers
the paper evaluates (ViT / DeiT linears, ResNet-50 convolutions).  It holds none of the
method's arithmetic; the oracle and the CUDA library both receive its arrays as data.
Weights are drawn directly as int8 with fp32 per-output-channel scales (a random-init
8-bit model), activations as fp32 together with one per-tensor scale.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

_GOLD = np.uint64(0x9E3779B97F4A7C15)


def _mix(z):
    z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
    z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
    return z ^ (z >> np.uint64(31))


def uniform(seed: int, stream: int, n: int) -> np.ndarray:
    """n doubles in [0, 1): element i depends only on (seed, stream, i)."""
    with np.errstate(over="ignore"):
        base = _mix(np.uint64(seed) * _GOLD + np.uint64(stream) * np.uint64(0xD1B54A32D192ED03) + _GOLD)
        ctr = np.arange(1, n + 1, dtype=np.uint64) * _GOLD + base
        z = _mix(ctr)
    return (z >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def normal(seed: int, stream: int, n: int) -> np.ndarray:
    u1 = uniform(seed, 2 * stream, n)
    u2 = uniform(seed, 2 * stream + 1, n)
    return np.sqrt(-2.0 * np.log(1.0 - u1)) * np.cos(2.0 * np.pi * u2)


def log_uniform(seed, stream, n, lo, hi):
    return np.exp(np.log(lo) + uniform(seed, stream, n) * (np.log(hi) - np.log(lo)))


def _int8_weights(w_fp: np.ndarray, axis_out: int):
    """Random-init 8-bit model: per-output-channel scale = absmax / 127, integers by rounding."""
    red = tuple(i for i in range(w_fp.ndim) if i != axis_out)
    amax = np.abs(w_fp).max(axis=red, keepdims=True)
    scale = (amax / 127.0).astype(np.float32)
    wq = np.clip(np.rint(w_fp / scale.astype(np.float64)), -127, 127).astype(np.int8)
    return wq, scale.reshape(-1).astype(np.float32)


@dataclass
class LinearCase:
    name: str
    M: int
    K: int
    N: int
    G: int
    X: np.ndarray        # [M, K] fp32 activations of the timed / checked call
    Xcal: np.ndarray     # [256, K] fp32 separate calibration draw (static positions come from it)
    x_scale: float       # per-tensor activation scale
    Wq: np.ndarray       # [K, N] int8, original channel order
    w_scale: np.ndarray  # [N] fp32
    bias: np.ndarray     # [N] fp32
    y_scale: float       # output scale for the int8 re-quantization
    meta: dict = field(default_factory=dict)


@dataclass
class ConvCase:
    name: str
    Nb: int
    H: int
    W: int
    C: int
    Cout: int
    R: int
    S: int
    stride: int
    pad: int
    G: int
    X: np.ndarray        # [Nb, H, W, C] fp32
    Xcal: np.ndarray     # [4, H, W, C] fp32
    x_scale: float
    Wq: np.ndarray       # [Cout, R, S, C] int8
    w_scale: np.ndarray
    bias: np.ndarray
    y_scale: float


def _y_scale(Xrows, x_scale, Wq2d, w_scale, bias):
    """Output scale: 99.9th percentile of |y| over a few rows / 127 (a data choice, fp64)."""
    xq = np.clip(np.rint(Xrows.astype(np.float64) / x_scale), -128, 127)
    y = (xq @ Wq2d.astype(np.float64)) * (x_scale * w_scale.astype(np.float64))[None, :] + bias[None, :]
    return float(np.float32(max(np.percentile(np.abs(y), 99.9), 1e-6) / 127.0))


def ranged_linear(name, M, K, N, G=16, seed=0, group_structured=False) -> LinearCase:
    """Per-input-channel activation ranges log-uniform over [0.05, 8] (the single-GEMM and
    the DeiT-S small-batch configurations).  group_structured=True draws the range per
    channel group instead (x a per-channel factor in [0.5, 1]) so that groups differ in
    their extraction positions; used by extra parity cases."""
    if group_structured:
        r = np.repeat(log_uniform(seed, 1, K // G, 0.05, 8.0), G) * (0.5 + 0.5 * uniform(seed, 7, K))
    else:
        r = log_uniform(seed, 1, K, 0.05, 8.0)
    z = normal(seed, 2, M * K).reshape(M, K)
    X = (r[None, :] * np.clip(z, -3, 3) / 3.0).astype(np.float32)
    zc = normal(seed + 500, 2, 256 * K).reshape(256, K)
    Xcal = (r[None, :] * np.clip(zc, -3, 3) / 3.0).astype(np.float32)
    x_scale = float(np.float32(r.max() / 127.0))
    a = log_uniform(seed, 3, K, 0.25, 1.0)
    b = log_uniform(seed, 4, N, 0.5, 2.0)
    w = normal(seed, 5, K * N).reshape(K, N) * a[:, None] * b[None, :]
    Wq, w_scale = _int8_weights(w, 1)
    bias = (normal(seed, 6, N) * 0.1).astype(np.float32)
    ys = _y_scale(X[:256], x_scale, Wq, w_scale, bias)
    return LinearCase(name, M, K, N, G, X, Xcal, x_scale, Wq, w_scale, bias, ys)


def vit_linear(name, M, K, N, G=16, seed=0) -> LinearCase:
    """Gaussian activations with a fixed 5 % of outlier channels scaled x20 (ViT-shaped linears)."""
    outl = uniform(seed, 1, K) < 0.05
    ch = np.where(outl, 20.0, 1.0)
    X = (normal(seed, 2, M * K).reshape(M, K) * ch[None, :]).astype(np.float32)
    Xcal = (normal(seed + 500, 2, 256 * K).reshape(256, K) * ch[None, :]).astype(np.float32)
    x_scale = float(np.float32(np.abs(Xcal).max() / 127.0))
    w = normal(seed, 5, K * N).reshape(K, N) * 0.02
    Wq, w_scale = _int8_weights(w, 1)
    bias = (normal(seed, 6, N) * 0.02).astype(np.float32)
    ys = _y_scale(X[:256], x_scale, Wq, w_scale, bias)
    return LinearCase(name, M, K, N, G, X, Xcal, x_scale, Wq, w_scale, bias, ys, {"outlier_channels": int(outl.sum())})


def resnet_conv(name, Nb, H, C, Cout, R, G=16, seed=0, stride=1) -> ConvCase:
    """Post-ReLU half-normal NHWC activations with log-uniform per-channel ranges; He-normal
    weights scaled per input channel (ResNet-50-shaped convolutions)."""
    W = H
    pad = R // 2
    r = log_uniform(seed, 1, C, 0.05, 8.0)
    X = (np.abs(normal(seed, 2, Nb * H * W * C)).reshape(Nb, H, W, C) * r).astype(np.float32)
    Xcal = (np.abs(normal(seed + 500, 2, 4 * H * W * C)).reshape(4, H, W, C) * r).astype(np.float32)
    x_scale = float(np.float32(np.abs(Xcal).max() / 127.0))
    a = log_uniform(seed, 3, C, 0.25, 1.0)
    w = normal(seed, 5, Cout * R * R * C).reshape(Cout, R, R, C) * np.sqrt(2.0 / (R * R * C)) * a
    Wq, w_scale = _int8_weights(w, 0)
    bias = (normal(seed, 6, Cout) * 0.1).astype(np.float32)
    # output scale from the centre taps only (cheap): a data choice, not part of the method
    xc = X[:1].reshape(-1, C)[:256]
    ys = _y_scale(xc, x_scale, Wq[:, R // 2, R // 2, :].T.copy(), w_scale, bias) * float(R)
    return ConvCase(name, Nb, H, W, C, Cout, R, R, stride, pad, G, X, Xcal, x_scale, Wq, w_scale, bias, float(np.float32(ys)))


# ---- the benchmark configurations ---------------------------------------------------
VIT_B_LAYERS = [("qkv", 768, 2304), ("proj", 768, 768), ("fc1", 768, 3072), ("fc2", 3072, 768)]
DEIT_S_LAYERS = [("qkv", 384, 1152), ("proj", 384, 384), ("fc1", 384, 1536), ("fc2", 1536, 384)]
VIT_L_LAYERS = [("qkv", 1024, 3072), ("proj", 1024, 1024), ("fc1", 1024, 4096), ("fc2", 4096, 1024)]
RESNET50_CONVS = [("conv3x3_56", 56, 64, 64, 3), ("conv3x3_28", 28, 128, 128, 3), ("conv3x3_14", 14, 256, 256, 3),
                  ("conv3x3_7", 7, 512, 512, 3), ("conv1x1_56", 56, 64, 256, 1), ("conv1x1_28", 28, 128, 512, 1),
                  ("conv1x1_14", 14, 256, 1024, 1), ("conv1x1_7", 7, 512, 2048, 1)]
RATIOS = [0.0, 0.25, 0.5, 0.75, 1.0]


def config1() -> LinearCase:
    return ranged_linear("cfg1_single_gemm", 256, 384, 384, 16, seed=0)


def config2(batch=64):
    return [vit_linear(f"cfg2_vitb_{n}", batch * 197, K, N, 16, seed=2000 + i) for i, (n, K, N) in enumerate(VIT_B_LAYERS)]


def config3(batch=32):
    return [resnet_conv(f"cfg3_{n}", batch, H, C, Co, R, 16, seed=3000 + i) for i, (n, H, C, Co, R) in enumerate(RESNET50_CONVS)]


def config4(batch=1):
    return [ranged_linear(f"cfg4_deits_b{batch}_{n}", batch * 197, K, N, 16, seed=4000 + i) for i, (n, K, N) in enumerate(DEIT_S_LAYERS)]


# ------------------------------------------------------------------ request traces (serving experiment)
def poisson_arrivals(seed: int, rate: float, n: int) -> np.ndarray:
    """Arrival times (seconds, ascending) of n requests of a Poisson process with `rate` requests per
    second, the request pattern of the paper's serving experiment (100 to 3000 requests per second)."""
    gaps = -np.log(1.0 - uniform(seed, 900, n)) / float(rate)
    return np.cumsum(gaps)


def fluctuating_arrivals(seed: int, rate_min: float, rate_max: float, period_s: float, duration_s: float) -> np.ndarray:
    """Arrival times of a Poisson process whose rate swings between rate_min and rate_max (the paper
    sets the peak to three times the minimum) along a raised cosine of the given period: stands in for
    the public cloud traces the paper replays, which are not available here.  Drawn by thinning a
    process of rate rate_max."""
    n = int(rate_max * duration_s * 1.2) + 64
    t = poisson_arrivals(seed, rate_max, n)
    t = t[t < duration_s]
    rate_t = rate_min + (rate_max - rate_min) * 0.5 * (1.0 - np.cos(2.0 * np.pi * t / period_s))
    keep = uniform(seed, 901, t.size) * rate_max < rate_t
    return t[keep]
