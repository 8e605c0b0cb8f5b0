"""Seeded synthetic inputs for the QLLM quantized-linear hot path.

This module only draws random tensors with the shapes and outlier structure of
LLaMA projection inputs (a few channels whose magnitude is tens of times that of
the rest, fixed across tokens).  It contains none of the method's arithmetic and
is the one module that both the CUDA path's callers and the CPU oracle's callers
take their inputs from.  Everything is numpy; bfloat16 tensors are carried as
uint16 bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class LayerConfig:
    name: str
    M: int                 # tokens
    K: int                 # input channels (C)
    N: int                 # output channels
    a_bits: int
    w_bits: int
    x_dtype: str           # "f32" | "bf16"
    seed: int
    n_outlier: int         # outlier channels
    outlier_lo: float      # outlier factor range (lo == hi: fixed factor)
    outlier_hi: float
    n_massive: int = 0     # additional channels scaled by massive_factor
    massive_factor: float = 1000.0
    w_std: float = 0.02
    beta_std: float = 0.0  # LayerNorm beta ~ N(0, beta_std); 0 -> no beta
    calib_tokens: int = 128  # 0 -> calibrate on X itself
    theta_rule: str = "pct99"  # "pct99" | "extra8"
    lr_rank: int = 4       # rank of the synthetic low-rank correction (0 = none)
    ln_eps: float = 1e-5

    def scaled(self, **kw) -> "LayerConfig":
        return replace(self, **kw)


CONFIGS = {
    "c1": LayerConfig("c1", M=64, K=256, N=512, a_bits=4, w_bits=4, x_dtype="f32", seed=0,
                      n_outlier=4, outlier_lo=50.0, outlier_hi=50.0, beta_std=0.02,
                      calib_tokens=0, theta_rule="extra8"),
    "c2": LayerConfig("c2", M=2048, K=4096, N=12288, a_bits=4, w_bits=4, x_dtype="bf16", seed=2,
                      n_outlier=20, outlier_lo=20.0, outlier_hi=100.0),
    "c3": LayerConfig("c3", M=16, K=4096, N=22016, a_bits=4, w_bits=4, x_dtype="bf16", seed=3,
                      n_outlier=20, outlier_lo=20.0, outlier_hi=100.0),
    "c4": LayerConfig("c4", M=4096, K=5120, N=15360, a_bits=6, w_bits=6, x_dtype="bf16", seed=4,
                      n_outlier=25, outlier_lo=20.0, outlier_hi=100.0),
    "c5": LayerConfig("c5", M=4096, K=8192, N=10240, a_bits=4, w_bits=4, x_dtype="bf16", seed=5,
                      n_outlier=40, outlier_lo=20.0, outlier_hi=100.0, n_massive=2, w_std=0.015),
    # the W4A8 setting of the paper's tables on the c2 shape: 8-bit activations, 4-bit weights
    "c2_w4a8": LayerConfig("c2_w4a8", M=2048, K=4096, N=12288, a_bits=8, w_bits=4, x_dtype="bf16", seed=2,
                           n_outlier=20, outlier_lo=20.0, outlier_hi=100.0),
}


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns, round to nearest even."""
    u = np.ascontiguousarray(a, np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(cfg: LayerConfig, stream: int) -> np.random.Generator:
    return np.random.default_rng([cfg.seed, stream])


def channel_factors(cfg: LayerConfig) -> np.ndarray:
    """Per-channel multiplier: 1 everywhere except the seed-chosen outlier channels."""
    r = _rng(cfg, 0)
    f = np.ones(cfg.K, np.float32)
    idx = r.choice(cfg.K, size=cfg.n_outlier + cfg.n_massive, replace=False)
    f[idx[:cfg.n_outlier]] = r.uniform(cfg.outlier_lo, cfg.outlier_hi, cfg.n_outlier).astype(np.float32)
    if cfg.n_massive:
        f[idx[cfg.n_outlier:]] = cfg.massive_factor
    return f


def _tokens(cfg: LayerConfig, stream: int, rows: int, factors: np.ndarray) -> np.ndarray:
    x = _rng(cfg, stream).standard_normal((rows, cfg.K), dtype=np.float32) * factors[None, :]
    if cfg.x_dtype == "bf16":
        return f32_to_bf16_bits(x)
    return x


def activations(cfg: LayerConfig, M: int | None = None, stream: int = 1) -> np.ndarray:
    """X [M][K]: float32, or uint16 bfloat16 bits.  `stream` picks an independent draw."""
    return _tokens(cfg, stream, cfg.M if M is None else M, channel_factors(cfg))


def calibration_tokens(cfg: LayerConfig) -> np.ndarray:
    """Calibration tokens (same outlier channels and factors); X itself when calib_tokens == 0."""
    if cfg.calib_tokens == 0:
        return activations(cfg)
    return _tokens(cfg, 2, cfg.calib_tokens, channel_factors(cfg))


def layernorm_params(cfg: LayerConfig):
    r = _rng(cfg, 3)
    gamma = (1.0 + 0.1 * r.standard_normal(cfg.K)).astype(np.float32)
    beta = (cfg.beta_std * r.standard_normal(cfg.K)).astype(np.float32) if cfg.beta_std > 0 else None
    return gamma, beta


def weights(cfg: LayerConfig) -> np.ndarray:
    """W [N][K] float32 (output-channel major)."""
    return _rng(cfg, 4).standard_normal((cfg.N, cfg.K), dtype=np.float32) * np.float32(cfg.w_std)


def low_rank(cfg: LayerConfig):
    """(A [K][r], B [r][N]) or (None, None)."""
    if cfg.lr_rank <= 0:
        return None, None
    r = _rng(cfg, 5)
    A = (0.03 * r.standard_normal((cfg.K, cfg.lr_rank))).astype(np.float32)
    B = (0.03 * r.standard_normal((cfg.lr_rank, cfg.N))).astype(np.float32)
    return A, B


def random_codes(seed: int, rows: int, cols: int, bits: int) -> np.ndarray:
    """Uniform random codes in [0, 2^bits), one per byte."""
    return np.random.default_rng([seed, 99]).integers(0, 1 << bits, size=(rows, cols), dtype=np.uint8)


def pack_nibbles(codes: np.ndarray) -> np.ndarray:
    """Storage layout of 4-bit codes: byte k = code[2k] | code[2k+1] << 4 (a layout, not arithmetic)."""
    c = np.ascontiguousarray(codes, np.uint8)
    return (c[..., 0::2] | (c[..., 1::2] << np.uint8(4))).astype(np.uint8)


def unpack_nibbles(packed: np.ndarray) -> np.ndarray:
    p = np.ascontiguousarray(packed, np.uint8)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), np.uint8)
    out[..., 0::2] = p & np.uint8(0xF)
    out[..., 1::2] = p >> np.uint8(4)
    return out
