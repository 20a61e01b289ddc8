"""Seeded synthetic tensors shaped like the paper's workloads (LLaMA-style projection weights
and KV caches).  They stand in for the real model tensors, which are not available offline.

This module holds no codec arithmetic: it only draws random fp16 tensors.  It is the one
module shared by the tests of the CPU oracle and of the CUDA library.

Seeds: data 1000+cfg, calibration 2000+cfg, outlier channels 3000+cfg.
"""
from __future__ import annotations

import numpy as np

G = 128


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def weight_matrix(rows: int, cols: int, seed: int, sigma: float = 0.02, row_scale: bool = True) -> np.ndarray:
    """Student-t(df=5) * sigma, optionally times a per-row lognormal(0, 0.5) factor; fp16 [rows][cols]."""
    rng = _rng(seed)
    out = np.empty((rows, cols), dtype=np.float16)
    rs = np.exp(rng.normal(0.0, 0.5, size=rows)) if row_scale else np.ones(rows)
    step = max(1, (1 << 24) // cols)
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        w = rng.standard_t(5.0, size=(r1 - r0, cols)) * sigma * rs[r0:r1, None]
        out[r0:r1] = w.astype(np.float16)
    return out


def kv_cache(batch: int, heads: int, seq: int, seed: int, outlier_seed: int, head_dim: int = G) -> np.ndarray:
    """N(0,1) with 4 fixed channels of each head scaled by 10; fp16 [batch][heads][seq][head_dim]."""
    rng = _rng(seed)
    orng = _rng(outlier_seed)
    chan_scale = np.ones((heads, head_dim), dtype=np.float32)
    for h in range(heads):
        chan_scale[h, orng.choice(head_dim, size=4, replace=False)] = 10.0
    out = np.empty((batch, heads, seq, head_dim), dtype=np.float16)
    for b in range(batch):
        for h in range(heads):
            x = rng.standard_normal(size=(seq, head_dim), dtype=np.float32) * chan_scale[h]
            out[b, h] = x.astype(np.float16)
    return out


def activations(batch: int, k: int, seed: int) -> np.ndarray:
    """fp16 N(0,1) [batch][k]."""
    return _rng(seed).standard_normal(size=(batch, k), dtype=np.float32).astype(np.float16)


def queries(batch: int, n_q_heads: int, seed: int, head_dim: int = G) -> np.ndarray:
    """fp16 N(0,1) [batch][n_q_heads][head_dim]."""
    return _rng(seed).standard_normal(size=(batch, n_q_heads, head_dim), dtype=np.float32).astype(np.float16)


def random_blocks(n_groups: int, seed: int) -> np.ndarray:
    """Uniform random bytes, [n_groups][64]: corrupt-stream input for decoder totality tests."""
    return _rng(seed).integers(0, 256, size=(n_groups, 64), dtype=np.uint8)
