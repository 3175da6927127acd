"""Seeded synthetic inputs shaped like the paper's decode workloads.

This module only draws random numbers and lays them out; it contains none of
the method's arithmetic (no scores, thresholds or attention), so both the CUDA
path and the CPU checker can be fed from it without sharing any computation.

bfloat16 tensors are produced as ``numpy.uint16`` bit patterns (rounded once,
round-to-nearest-even), so every consumer sees identical bits.

Workload recipe (stands in for the paper's evaluation prompts and trained
predictors, of which only shapes and densities are used):
  * Q, K, V ~ N(0, 1);
  * predictor input x_t ~ N(0, 1)^d_in, linear predictor rows w_h ~ N(0, 1/d_in);
  * a head with target keep rate r gets bias b_h = ||w_h|| * Phi^-1(r) + tau_logit,
    so that P(<w_h, x_t> + b_h >= tau_logit) = r;
  * per-(layer, KV head) keep rates r ~ Beta(a, b) (heads range from
    local-only to nearly full, like the paper's per-head density spread).
"""
from __future__ import annotations

import math

import numpy as np


def to_bf16_bits(a) -> np.ndarray:
    """float32 -> bfloat16 bit patterns, round to nearest even (finite inputs)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return u.astype(np.uint16)


def bf16_bits_to_f32(b) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32)


def normal_bf16(rng: np.random.Generator, shape, std: float = 1.0) -> np.ndarray:
    return to_bf16_bits(rng.standard_normal(shape, dtype=np.float32) * np.float32(std))


def linear_predictor(rng: np.random.Generator, n_kv_heads: int, d_in: int) -> np.ndarray:
    """Rows w_h ~ N(0, 1/d_in) as bf16 bits, shape [n_kv_heads, d_in]."""
    return normal_bf16(rng, (n_kv_heads, d_in), std=1.0 / math.sqrt(d_in))


def mlp_predictor(rng: np.random.Generator, n_kv_heads: int, d_in: int, hidden: int):
    """Two-layer predictor weights (bf16 bits) and float32 biases."""
    W1 = normal_bf16(rng, (hidden, d_in), std=1.0 / math.sqrt(d_in))
    b1 = (rng.standard_normal(hidden, dtype=np.float32) * np.float32(0.1))
    W2 = normal_bf16(rng, (n_kv_heads, hidden), std=1.0 / math.sqrt(hidden))
    b2 = (rng.standard_normal(n_kv_heads, dtype=np.float32) * np.float32(0.1))
    return W1, b1, W2, b2


def _ndtri(p: float) -> float:
    """Inverse standard-normal CDF; 0 and 1 map to -inf / +inf."""
    if p <= 0.0:
        return -math.inf
    if p >= 1.0:
        return math.inf
    from statistics import NormalDist
    return NormalDist().inv_cdf(p)


def bias_for_keep_rate(W_bits: np.ndarray, rates, tau_logit: float) -> np.ndarray:
    """b_h such that a N(0,1)^d_in input passes the threshold with probability rates[h]."""
    W = bf16_bits_to_f32(W_bits).astype(np.float64)
    norms = np.sqrt((W * W).sum(axis=1))
    rates = np.broadcast_to(np.asarray(rates, dtype=np.float64), norms.shape)
    b = np.array([n * _ndtri(float(r)) for n, r in zip(norms, rates)], dtype=np.float64)
    return (b + float(tau_logit)).astype(np.float32)


def keep_rates(rng: np.random.Generator, n_layers: int, n_kv_heads: int, a: float, b: float):
    """Per-(layer, KV head) keep rates ~ Beta(a, b), clipped to [0, 1]."""
    return np.clip(rng.beta(a, b, size=(n_layers, n_kv_heads)), 0.0, 1.0)


def logits_with_keep_rate(rng: np.random.Generator, shape, rate: float, tau_logit: float,
                          guard: float = 0.0) -> np.ndarray:
    """float32 logits of which a fraction ``rate`` lies at or above tau_logit.

    Values are tau_logit +/- (guard + |N(0,1)|), so none falls within ``guard`` of
    the threshold (used where a decision must not depend on rounding)."""
    mag = np.abs(rng.standard_normal(shape, dtype=np.float32)) + np.float32(guard)
    sign = np.where(rng.random(shape) < rate, 1.0, -1.0).astype(np.float32)
    base = np.float32(tau_logit) if math.isfinite(tau_logit) else np.float32(0.0)
    return (base + sign * mag).astype(np.float32)
