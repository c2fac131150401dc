"""Seeded synthetic inputs shaped like the paper's long-context workloads.

This module only draws random tensors; it holds none of the method's arithmetic and is
the one module that both the CUDA-side tests/bench and the CPU oracle's tests import.

Recipes (per (sequence, layer, KV head) stream; all values are rounded to the storage
dtype so that every consumer sees exactly the same numbers):

``outlier2``   keys N(0,1) with 2 channels (drawn once per stream set) scaled x8;
               values N(0,1); queries N(0,1).                       (tiny fp32 case)
``llama``      per head mean vector mu ~ N(0, 0.5^2); k = (mu + z) * s with z ~ N(0,1) and
               s = 10 on 4 channels fixed per head, 1 elsewhere; values N(0,1);
               queries N(0,1).                                      (8B / 32B shaped cases)
``student_t``  keys i.i.d. Student-t(nu=4) per element, values N(0,1), queries N(0,1).
                                                                    (14B shaped case)
"""
from __future__ import annotations

import numpy as np

RECIPES = ("outlier2", "llama", "student_t")


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round a float32 array to the storage dtype ('fp32' or 'bf16'); returns float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "fp32":
        return x
    if dtype == "bf16":
        return bf16_bits_to_f32(to_bf16_bits(x))
    raise ValueError(dtype)


def _rng(data_seed: int, *coords: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([int(data_seed), *map(int, coords)])))


def head_profile(recipe: str, data_seed: int, layer: int, head: int, d: int):
    """Per-head constants of a recipe: (mean vector, per-channel scale), both float32 [d]."""
    g = _rng(data_seed, 7001, layer, head)
    mu = np.zeros(d, np.float32)
    scale = np.ones(d, np.float32)
    if recipe == "outlier2":
        ch = _rng(data_seed, 7002).choice(d, size=2, replace=False)
        scale[ch] = 8.0
    elif recipe == "llama":
        mu = (0.5 * g.standard_normal(d)).astype(np.float32)
        ch = g.choice(d, size=4, replace=False)
        scale[ch] = 10.0
    elif recipe == "student_t":
        pass
    else:
        raise ValueError(recipe)
    return mu, scale


def stream_kv(recipe: str, data_seed: int, seq: int, layer: int, head: int, n: int, d: int,
              dtype: str = "bf16"):
    """Keys and values of one stream: two float32 arrays [n, d] rounded to ``dtype``."""
    g = _rng(data_seed, 1, seq, layer, head)
    mu, scale = head_profile(recipe, data_seed, layer, head, d)
    if recipe == "student_t":
        z = g.standard_normal((n, d), dtype=np.float32)
        chi = g.chisquare(4.0, size=(n, d)).astype(np.float32)
        k = z / np.sqrt(chi / 4.0)
    else:
        k = (mu[None, :] + g.standard_normal((n, d), dtype=np.float32)) * scale[None, :]
    v = g.standard_normal((n, d), dtype=np.float32)
    return round_to(k, dtype), round_to(v, dtype)


def layer_kv(recipe: str, data_seed: int, layer: int, n_seqs: int, n_kv_heads: int, n: int, d: int,
             dtype: str = "bf16"):
    """K, V of one layer: float32 [n_seqs, n_kv_heads, n, d] rounded to ``dtype``."""
    K = np.empty((n_seqs, n_kv_heads, n, d), np.float32)
    V = np.empty_like(K)
    for s in range(n_seqs):
        for h in range(n_kv_heads):
            K[s, h], V[s, h] = stream_kv(recipe, data_seed, s, layer, h, n, d, dtype)
    return K, V


def queries(data_seed: int, layer: int, step: int, n_seqs: int, n_q_heads: int, d: int,
            dtype: str = "bf16") -> np.ndarray:
    """Decode queries of one step: float32 [n_seqs, n_q_heads, d], N(0,1), rounded."""
    g = _rng(data_seed, 2, layer, step)
    return round_to(g.standard_normal((n_seqs, n_q_heads, d), dtype=np.float32), dtype)


def kept_positions(data_seed: int, seq: int, layer: int, head: int, length: int, T: int) -> np.ndarray:
    """Sorted uniform-random subset of [0, length * 2^T) of size ``length`` (int32)."""
    g = _rng(data_seed, 3, seq, layer, head)
    total = length << T
    return np.sort(g.choice(total, size=length, replace=False)).astype(np.int32)


def to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """Bytes as the library stores them: float32 array, or uint16 bf16 bit patterns."""
    if dtype == "fp32":
        return np.ascontiguousarray(x, dtype=np.float32)
    return to_bf16_bits(x)
