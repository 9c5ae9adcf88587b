"""Seeded synthetic inputs for the five benchmark configurations.

This module only *draws numbers*: it contains none of the method's arithmetic
(no FP8 coding, no scaling, no loss).  Both the CPU oracle's tests and the CUDA
path's tests feed on the arrays it returns, so the two sides always see the
same bits.  bf16 tensors are returned as numpy ``uint16`` bit patterns (numpy
has no bf16 type); values are drawn in float32 and rounded to bf16 with
round-to-nearest-even.

The distributions stand in for the activations, weights and gradients of the
transformer families the paper trains (GPT-2 on OpenWebText, ViT/Swin on
ImageNet-1K), whose data and weights are not available: shapes follow the model
family, magnitudes follow the regimes the paper reports ("normal" values around
10, "massive" outliers above 1000, peaks up to a few 10^4).

Seeds: ``1000 * config + tensor_index``; config 1 starts at seed 0.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bf16 (ties to even); returns uint16 bits."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    r = ((u >> 16) & 1) + 0x7FFF
    out = ((u + r) >> 16).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = 0x7FC0
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def normal_bf16(seed: int, shape, std: float = 1.0) -> np.ndarray:
    """N(0, std^2) (the second parameter of "N(0, s)" in the configs is the std)."""
    x = _rng(seed).standard_normal(size=shape, dtype=np.float32) * np.float32(std)
    return f32_to_bf16_bits(x)


def normal_with_extreme_outliers_bf16(seed: int, shape, frac: float = 1e-3,
                                      lo: float = 1000.0, hi: float = 3000.0) -> np.ndarray:
    """N(0,1) with ``round(frac * size)`` entries, chosen uniformly without
    replacement, overwritten by +-U(lo, hi) (fair sign): the extreme-outlier
    regime that breaks per-tensor FP8."""
    g = _rng(seed)
    x = g.standard_normal(size=shape, dtype=np.float32)
    n = x.size
    k = int(round(frac * n))
    pos = g.choice(n, size=k, replace=False)
    mag = g.uniform(lo, hi, size=k).astype(np.float32)
    sgn = np.where(g.integers(0, 2, size=k) == 0, np.float32(-1), np.float32(1))
    x.reshape(-1)[pos] = mag * sgn
    return f32_to_bf16_bits(x)


def normal_with_outlier_channels_bf16(seed: int, shape, frac_channels: float = 1e-4,
                                      factor: float = 500.0) -> np.ndarray:
    """N(0,1) with ``max(1, round(frac_channels * d))`` whole channels (columns)
    multiplied by ``factor``."""
    g = _rng(seed)
    x = g.standard_normal(size=shape, dtype=np.float32)
    d = shape[-1]
    k = max(1, int(round(frac_channels * d)))
    ch = g.choice(d, size=k, replace=False)
    x[..., ch] *= np.float32(factor)
    return f32_to_bf16_bits(x)


def normal_plus_student_t_bf16(seed: int, shape, df: float = 3.0, t_scale: float = 1.0) -> np.ndarray:
    """N(0,1) + t_scale * Student-t(df), independent draws (heavy tails)."""
    g = _rng(seed)
    x = g.standard_normal(size=shape, dtype=np.float32)
    t = g.standard_t(df, size=shape).astype(np.float32)
    return f32_to_bf16_bits(x + np.float32(t_scale) * t)


@dataclass(frozen=True)
class Linear:
    name: str
    K: int  # in-features  (contraction of the forward GEMM)
    N: int  # out-features


@dataclass(frozen=True)
class Config:
    idx: int
    name: str
    M: int            # tokens
    d: int            # width of the block output the penalty reads
    linears: tuple
    n_blocks: int     # block outputs entering one TWEO call
    x_kind: str       # "outlier_entries" | "outlier_channels" | "normal" | "student_t"
    grad_fmt: str     # "e5m2"


CONFIGS = {
    1: Config(1, "single_linear_penalty", 512, 256, (Linear("lin", 256, 1024),), 1, "outlier_entries", "e5m2"),
    2: Config(2, "gpt2_small_block", 8 * 1024, 768,
              (Linear("qkv", 768, 2304), Linear("proj", 768, 768), Linear("fc1", 768, 3072),
               Linear("fc2", 3072, 768)), 1, "outlier_channels", "e5m2"),
    3: Config(3, "vit_b16_step", 256 * 197, 768,
              (Linear("qkv", 768, 2304), Linear("proj", 768, 768), Linear("fc1", 768, 3072),
               Linear("fc2", 3072, 768)), 12, "normal", "e5m2"),
    4: Config(4, "llama_1b_block", 4 * 4096, 2048,
              (Linear("qkv", 2048, 6144), Linear("o", 2048, 2048), Linear("gate", 2048, 5632),
               Linear("up", 2048, 5632), Linear("down", 5632, 2048)), 1, "student_t", "e5m2"),
}

# config 5: static W8A8 inference GEMM sweep (LLaMA-7B linear shapes)
W8A8_KN = ((4096, 4096), (4096, 11008), (11008, 4096))
W8A8_M = (1, 16, 128, 1024, 8192)
W8A8_CALIB_BATCHES = 32
W8A8_CALIB_ROWS = 1024


def _seed(cfg: int, tensor_index: int) -> int:
    return (0 if cfg == 1 else 1000 * cfg) + tensor_index


def activation(cfg: Config, seed: int, shape) -> np.ndarray:
    if cfg.x_kind == "outlier_entries":
        return normal_with_extreme_outliers_bf16(seed, shape)
    if cfg.x_kind == "outlier_channels":
        return normal_with_outlier_channels_bf16(seed, shape)
    if cfg.x_kind == "student_t":
        return normal_plus_student_t_bf16(seed, shape)
    return normal_bf16(seed, shape, 1.0)


def linear_inputs(cfg_idx: int, lin_idx: int, M: int | None = None, block: int = 0):
    """(X [M,K], W [N,K], dY [M,N]) as bf16 bits for one linear of a config.
    W is stored one row per output feature (K contiguous)."""
    cfg = CONFIGS[cfg_idx]
    lin = cfg.linears[lin_idx]
    M = cfg.M if M is None else M
    base = 10 * lin_idx + 100 * block
    x = activation(cfg, _seed(cfg_idx, base + 0), (M, lin.K))
    w = normal_bf16(_seed(cfg_idx, base + 1), (lin.N, lin.K), 0.02)
    dy = normal_bf16(_seed(cfg_idx, base + 2), (M, lin.N), 1e-3)
    return x, w, dy


def block_output(cfg_idx: int, block: int = 0, M: int | None = None) -> np.ndarray:
    """The block-output activation A^(l) [M, d] the penalty is taken on."""
    cfg = CONFIGS[cfg_idx]
    M = cfg.M if M is None else M
    return activation(cfg, _seed(cfg_idx, 900 + block), (M, cfg.d))


def w8a8_weight(K: int, N: int) -> np.ndarray:
    return normal_bf16(_seed(5, (K * 7 + N) % 997), (N, K), 0.02)


def w8a8_calibration_batch(K: int, i: int, rows: int = W8A8_CALIB_ROWS) -> np.ndarray:
    return normal_bf16(5000 + i, (rows, K), 1.0)


def w8a8_activation(M: int, K: int) -> np.ndarray:
    return normal_bf16(_seed(5, 500 + (M * 13 + K) % 401), (M, K), 1.0)
