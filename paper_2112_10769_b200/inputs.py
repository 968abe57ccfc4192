"""Seeded synthetic inputs for the five benchmark workloads.

This module holds input generation only: no quantizer, no random stream of the
method, no GEMM.  Both the CUDA tests/benchmark and the CPU checker draw their
tensors from here so that they see identical bytes.

Tensors follow the shapes of the paper's models (a ResNet-50 3x3 convolution as
an im2col GEMM at batch 256, a Transformer feed-forward layer) and the value
distributions the paper describes: weights and activations roughly normal,
neural gradients heavy-tailed and near-lognormal (Sec. 1, Sec. 2).

bf16 tensors are carried as uint16 bit patterns (numpy has no bf16).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class LayerConfig:
    name: str
    M: int
    K: int
    N: int
    dtype: str            # "f32" or "bf16"
    relu: bool            # activations = max(N(0,1), 0)
    w_var: float          # weight variance
    g_mu: float           # log-magnitude mean of the gradient
    g_sigma: float
    g_zero_frac: float
    seeds: tuple          # (A, W, G)
    luq_seed: int = 0
    n_samples: int = 1


CONFIGS = {
    # single linear layer, all three GEMMs, small enough for the CPU checker
    "cfg1": LayerConfig("cfg1", 256, 256, 256, "f32", True, 2.0 / 256, -10.0, 2.5, 0.30, (101, 102, 103)),
    # ResNet-50 3x3 conv 256->256 at 14x14, batch 256, as an im2col GEMM
    "cfg2": LayerConfig("cfg2", 50176, 2304, 256, "f32", True, 2.0 / 2304, -12.0, 3.0, 0.40, (201, 202, 203)),
    # Transformer FFN 1024 -> 4096 over 8192 tokens, bf16 inputs
    "cfg3": LayerConfig("cfg3", 8192, 1024, 4096, "bf16", False, 1.0 / 1024, -11.0, 2.5, 0.05, (301, 302, 303)),
    # cfg2 with two averaged gradient samples
    "cfg5": LayerConfig("cfg5", 50176, 2304, 256, "f32", True, 2.0 / 2304, -12.0, 3.0, 0.40, (201, 202, 203),
                        luq_seed=0, n_samples=2),
}

# quantizer sweep: 1-D fp32 gradient tensors of 2^e elements
SWEEP_EXPONENTS = (20, 22, 24, 26, 28, 30)
SWEEP_MU, SWEEP_SIGMA, SWEEP_ZERO_FRAC = -10.0, 3.0, 0.20


def to_bf16_bits(x32: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _chunks(n: int, step: int = 1 << 24):
    for lo in range(0, n, step):
        yield lo, min(n, lo + step)


def normal(shape, var: float, seed: int, relu: bool = False) -> np.ndarray:
    rng = np.random.default_rng(seed)
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float32)
    std = float(np.sqrt(var))
    for lo, hi in _chunks(n):
        v = rng.standard_normal(hi - lo) * std
        if relu:
            np.maximum(v, 0.0, out=v)
        out[lo:hi] = v
    return out.reshape(shape)


def lognormal_gradient(shape, mu: float, sigma: float, zero_frac: float, seed: int) -> np.ndarray:
    """sign * exp(N(mu, sigma)) with equiprobable sign; an independent mask sets
    `zero_frac` of the entries to +0.0."""
    rng = np.random.default_rng(seed)
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float32)
    for lo, hi in _chunks(n):
        m = hi - lo
        mag = np.exp(rng.standard_normal(m) * sigma + mu)
        sign = np.where(rng.random(m) < 0.5, -1.0, 1.0)
        keep = rng.random(m) >= zero_frac
        out[lo:hi] = np.where(keep, sign * mag, 0.0)
    return out.reshape(shape)


def layer_inputs(cfg: LayerConfig, rows: int | None = None):
    """(A, W, G) for a layer config.  `rows` truncates M (first rows of the same
    stream) for bounded CPU samples.  bf16 configs return uint16 bit patterns."""
    M = cfg.M if rows is None else min(rows, cfg.M)
    A = normal((M, cfg.K), 1.0, cfg.seeds[0], relu=cfg.relu)
    W = normal((cfg.N, cfg.K), cfg.w_var, cfg.seeds[1])
    G = lognormal_gradient((M, cfg.N), cfg.g_mu, cfg.g_sigma, cfg.g_zero_frac, cfg.seeds[2])
    if cfg.dtype == "bf16":
        return to_bf16_bits(A), to_bf16_bits(W), to_bf16_bits(G)
    return A, W, G


def sweep_tensor(exponent: int) -> np.ndarray:
    return lognormal_gradient((1 << exponent,), SWEEP_MU, SWEEP_SIGMA, SWEEP_ZERO_FRAC, 400 + exponent)


def small_layer(M: int, K: int, N: int, seed: int, dtype: str = "f32", g_mu: float = -3.0,
                g_sigma: float = 2.0, zero_frac: float = 0.2):
    """Small layers for parity tests: the gradient's log-magnitude spread is
    narrower than in the benchmark configs so that every LUQ bin is exercised."""
    A = normal((M, K), 1.0, seed, relu=True)
    W = normal((N, K), 2.0 / max(K, 1), seed + 1)
    G = lognormal_gradient((M, N), g_mu, g_sigma, zero_frac, seed + 2)
    if dtype == "bf16":
        return to_bf16_bits(A), to_bf16_bits(W), to_bf16_bits(G)
    return A, W, G


def log_uniform_magnitudes(n: int, lo_exp: float, hi_exp: float, seed: int) -> np.ndarray:
    """+-2^U(lo_exp, hi_exp): magnitudes spread evenly over many binades."""
    rng = np.random.default_rng(seed)
    mag = np.exp2(rng.uniform(lo_exp, hi_exp, n))
    sign = np.where(rng.random(n) < 0.5, -1.0, 1.0)
    return (sign * mag).astype(np.float32)
