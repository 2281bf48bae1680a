"""Seeded synthetic inputs shaped like the paper's decoding workloads.

This module is the one thing the CPU oracle's tests and the CUDA path share.
It holds none of the method's arithmetic (no quantizer, no layout, no index
collection, no GEMV): it only draws weights and hidden states with the shapes
and value distributions of Llama-2/3 decode-time linear layers (the models the
paper evaluates, Sec. 6) and picks thresholds for a target sparsity level (the
paper calibrates one threshold per matrix or matrix group, Sec. 5).

Everything is numpy on the host, drawn in fp32 with ``Generator(PCG64(seed))``
and rounded once to fp16.
"""
from __future__ import annotations

import math

import numpy as np

# (name, m = out features, n = in features, distribution of the layer's input)
LLAMA3_8B_LINEARS = (
    ("q", 4096, 4096, "laplace"),
    ("k", 1024, 4096, "laplace"),
    ("v", 1024, 4096, "laplace"),
    ("o", 4096, 4096, "laplace"),
    ("gate", 14336, 4096, "laplace"),
    ("up", 14336, 4096, "laplace"),
    ("down", 4096, 14336, "gauss"),
)

# Llama-2-70B-shaped linears (attention 8192->8192, up 8192->28672, down 28672->8192)
LLAMA2_70B_LINEARS = (
    ("attn", 8192, 8192, "laplace"),
    ("up", 28672, 8192, "laplace"),
    ("down", 8192, 28672, "laplace"),
)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(int(seed)))


def weights(m: int, n: int, seed: int, std: float = 0.02) -> np.ndarray:
    """fp16 W[m][n] ~ N(0, std^2), row-major (m outputs, n inputs)."""
    g = _rng(seed)
    w = g.standard_normal((m, n), dtype=np.float32)
    w *= np.float32(std)
    return w.astype(np.float16)


def activations(n: int, seed: int, dist: str = "laplace",
                outlier_frac: float = 0.0, outlier_scale: float = 20.0) -> np.ndarray:
    """fp16 hidden state x[n]: Laplace(0,1) (attention / MLP inputs) or N(0,1)
    (down-projection input); optionally a seeded fraction of entries is
    multiplied by ``outlier_scale`` (heavy-tailed outlier channels)."""
    g = _rng(seed)
    if dist == "laplace":
        x = g.laplace(0.0, 1.0, size=n).astype(np.float32)
    elif dist == "gauss":
        x = g.standard_normal(n, dtype=np.float32)
    else:
        raise ValueError("unknown distribution %r" % (dist,))
    if outlier_frac > 0.0:
        k = max(1, int(round(outlier_frac * n)))
        pos = g.choice(n, size=k, replace=False)
        x[pos] *= np.float32(outlier_scale)
    return x.astype(np.float16)


def threshold_for_sparsity(x: np.ndarray, sparsity: float) -> float:
    """Nearest-rank threshold: the ceil(sparsity*n)-th smallest |x_k| (1-based),
    so that at least that many entries have |x_k| <= t and are dropped;
    ``sparsity <= 0`` returns -1 (nothing dropped).  The value is an fp16 value
    and is returned as a Python float (exact)."""
    n = x.size
    if sparsity <= 0.0 or n == 0:
        return -1.0
    rank = min(n, max(1, int(math.ceil(sparsity * n - 1e-9))))
    a = np.sort(np.abs(x.astype(np.float32)))
    return float(a[rank - 1])


def pooled_threshold(xs, sparsity: float) -> float:
    """One threshold calibrated once on several vectors of the same site (the
    paper's calibrate-once scheme): nearest-rank over the pooled magnitudes."""
    return threshold_for_sparsity(np.concatenate([np.asarray(v).ravel() for v in xs]), sparsity)


def realised_sparsity(x: np.ndarray, t: float) -> float:
    """Fraction of entries NOT strictly above the threshold (reporting only)."""
    a = np.abs(x.astype(np.float32))
    return float(np.count_nonzero(~(a > np.float32(t)))) / max(1, x.size)


def lossless_weights(m: int, n: int, a: int = 5, b: int = 3, levels: int = 16) -> np.ndarray:
    """W[j][k] = ((a*j + b*k) mod levels) / levels with a odd and levels a power of two (16 for
    4-bit codes, 8 for 3-bit ones): every run of >= levels consecutive rows of a column holds both 0
    and (levels-1)/levels, so a min/max quantizer with that many levels reproduces the matrix exactly
    (scale 1/levels, offset 0)."""
    assert a % 2 == 1 and levels in (8, 16)
    j = np.arange(m, dtype=np.int64)[:, None]
    k = np.arange(n, dtype=np.int64)[None, :]
    return (((a * j + b * k) % levels).astype(np.float32) / float(levels)).astype(np.float16)


def small_rational_activations(n: int, seed: int) -> np.ndarray:
    """x_k drawn from {+-1, +-2, +-0.5}: products with ``lossless_weights`` sum
    exactly in fp32."""
    g = _rng(seed)
    vals = np.array([1.0, -1.0, 2.0, -2.0, 0.5, -0.5], dtype=np.float32)
    return vals[g.integers(0, len(vals), size=n)].astype(np.float16)
