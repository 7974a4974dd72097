"""Seeded synthetic inputs shaped like the paper's LLaMA-2 linear layers.

This module only draws random numbers and rounds them to BF16.  It holds none of
the method's arithmetic and is the one piece of code that both the tests of the
CPU oracle and the CUDA path are fed from: the same BF16 bit patterns go to both.

Shapes follow LLaMA-2 1.3B / 7B / 13B linears (Section 4.1); the structure
(normal weights, heavy-tailed activations whose outliers sit in a few channels)
follows the distribution study of Appendix D.  They stand in for the paper's real
activations, which need its trained checkpoints.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


def to_bf16_bits(x32: np.ndarray) -> np.ndarray:
    """float32 -> BF16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


@dataclass(frozen=True)
class Linear:
    name: str
    K: int          # input channels  c_i
    N: int          # output channels c_o


@dataclass(frozen=True)
class Config:
    index: int
    name: str
    M: int                      # tokens
    linears: tuple
    act_dist: str               # "normal" | "student_t3" | "laplace"
    outlier_frac: float
    outlier_scale: float
    outlier_mode: str           # "channels" | "channels_count" | "elements"
    alphas: tuple
    w_std: float = 0.02
    dy_std: float = 1e-3


def _llama(h: int, ffn: int, attn=True, mlp=True):
    out = []
    if attn:
        out += [Linear(n, h, h) for n in ("q", "k", "v", "o")]
    if mlp:
        out += [Linear("gate", h, ffn), Linear("up", h, ffn), Linear("down", ffn, h)]
    return tuple(out)


CONFIGS = (
    Config(0, "single-1024", 256, (Linear("fc", 1024, 1024),), "normal", 8, 50.0,
           "channels_count", (0.99,)),
    Config(1, "llama-1.3b-layer", 4096, _llama(2048, 5504), "student_t3", 0.005, 30.0,
           "channels", (0.999,)),
    Config(2, "llama-7b-mlp", 8192, _llama(4096, 11008, attn=False), "normal", 0.01, 50.0,
           "channels", (0.99, 0.999)),
    Config(3, "llama-13b-attn", 8192, _llama(5120, 13824, mlp=False), "laplace", 0.002, 100.0,
           "elements", (0.9999,)),
    Config(4, "llama-13b-layer", 16384, _llama(5120, 13824), "student_t3", 0.01, 50.0,
           "channels", (0.99,)),
)


def _rng(seed: int, cfg: int, layer: int, tensor: int) -> np.random.Generator:
    return np.random.default_rng([seed, cfg, layer, tensor])


def activations(cfg: Config, K: int, seed: int = 0, layer: int = 0, M: int | None = None) -> np.ndarray:
    """A[M x K] as BF16 bits (uint16)."""
    M = cfg.M if M is None else M
    rng = _rng(seed, cfg.index, layer, 0)
    if cfg.act_dist == "normal":
        a = rng.standard_normal((M, K), dtype=np.float32)
    elif cfg.act_dist == "student_t3":
        a = rng.standard_t(3.0, size=(M, K)).astype(np.float32)
    elif cfg.act_dist == "laplace":
        a = rng.laplace(0.0, 1.0, size=(M, K)).astype(np.float32)
    else:
        raise ValueError(cfg.act_dist)
    if cfg.outlier_mode == "elements":
        mask = rng.random((M, K), dtype=np.float32) < np.float32(cfg.outlier_frac)
        a = np.where(mask, a * np.float32(cfg.outlier_scale), a)
    else:
        n_ch = int(cfg.outlier_frac) if cfg.outlier_mode == "channels_count" \
            else int(round(cfg.outlier_frac * K))
        ch = rng.choice(K, size=n_ch, replace=False)
        a[:, ch] *= np.float32(cfg.outlier_scale)
    return to_bf16_bits(a)


def weights(cfg: Config, K: int, N: int, seed: int = 0, layer: int = 0) -> np.ndarray:
    """W[K x N] (input channels x output channels) as BF16 bits."""
    rng = _rng(seed, cfg.index, layer, 1)
    w = rng.standard_normal((K, N), dtype=np.float32) * np.float32(cfg.w_std)
    return to_bf16_bits(w)


def output_grads(cfg: Config, N: int, seed: int = 0, layer: int = 0, M: int | None = None) -> np.ndarray:
    """dY[M x N] as BF16 bits."""
    M = cfg.M if M is None else M
    rng = _rng(seed, cfg.index, layer, 2)
    g = rng.standard_normal((M, N), dtype=np.float32) * np.float32(cfg.dy_std)
    return to_bf16_bits(g)


def small_case(M: int, K: int, N: int, seed: int = 0, alpha_outliers: int = 4,
               dist: str = "normal"):
    """A small three-tensor case for parity tests: (A, W, dY) BF16 bits."""
    cfg = Config(99, "small", M, (Linear("fc", K, N),), dist, alpha_outliers, 40.0,
                 "channels_count", (0.99,))
    return (activations(cfg, K, seed, M * 7 + K), weights(cfg, K, N, seed, M * 7 + K),
            output_grads(cfg, N, seed, M * 7 + K))
