"""Seeded generators for the synthetic tensors.

All randomness comes from numpy's counter-based Philox generator keyed by
(base seed, workload name, layer name, tensor name), so any tensor can be
regenerated alone and both the oracle and the CUDA library receive the very
same bytes.  Values are rounded to bfloat16 here (round to nearest even), the
storage type of weights and activations; the arrays returned hold the bf16 bit
patterns as uint16.  ``from_bf16_bits`` widens them exactly to float32.
"""
from __future__ import annotations

import hashlib

import numpy as np

BASE_SEED = 20240711


def tensor_seed(*names) -> int:
    h = hashlib.sha256(("/".join(str(n) for n in names)).encode()).digest()
    return BASE_SEED ^ int.from_bytes(h[:8], "little")


def _rng(*names) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=tensor_seed(*names) & ((1 << 64) - 1)))


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit pattern, round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(shape, std: float, *names) -> np.ndarray:
    g = _rng(*names)
    x = g.standard_normal(size=shape, dtype=np.float32) * np.float32(std)
    return to_bf16_bits(x)


def student_t_bf16(shape, scale: float, df: int, *names) -> np.ndarray:
    g = _rng(*names)
    x = g.standard_t(df, size=shape).astype(np.float32) * np.float32(scale)
    return to_bf16_bits(x)


def weight_for(cfg, lin) -> np.ndarray:
    """Synthetic stand-in for a trained weight matrix [out, in] (bf16 bits).

    normal: N(0, scale^2).  student_t4: scale * t(4), heavy tails like trained
    LLM weights.  With ``outlier_frac`` > 0 a seeded set of ceil(frac*in) input
    channels (columns) is multiplied by ``outlier_gain``.
    """
    shape = (lin.out_features, lin.in_features)
    if cfg.weight_dist == "normal":
        g = _rng(cfg.name, lin.name, "W")
        w = g.standard_normal(size=shape, dtype=np.float32) * np.float32(cfg.weight_scale)
    elif cfg.weight_dist == "student_t4":
        g = _rng(cfg.name, lin.name, "W")
        w = g.standard_t(4, size=shape).astype(np.float32) * np.float32(cfg.weight_scale)
    else:
        raise ValueError(cfg.weight_dist)
    if cfg.outlier_frac > 0.0:
        n_out = int(np.ceil(cfg.outlier_frac * lin.in_features))
        cols = _rng(cfg.name, lin.name, "outlier_cols").choice(lin.in_features, size=n_out, replace=False)
        w[:, cols] *= np.float32(cfg.outlier_gain)
    return to_bf16_bits(w)


def activations_for(cfg, lin, tokens=None):
    """(X[T, in], dY[T, out]) as bf16 bits: X ~ N(0, x_std^2), dY ~ N(0, dy_std^2)."""
    T = cfg.tokens if tokens is None else tokens
    X = normal_bf16((T, lin.in_features), cfg.x_std, cfg.name, lin.name, "X")
    dY = normal_bf16((T, lin.out_features), cfg.dy_std, cfg.name, lin.name, "dY")
    return X, dY
