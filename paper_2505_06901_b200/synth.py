"""Seeded synthetic tensors shaped like the paper's workloads (LLaMA-style projection weights
and KV caches).  They stand in for the real model tensors, which are not available offline.

This module holds no codec arithmetic: it only draws random fp16 tensors.  It is the one
module shared by the tests of the CPU oracle and of the CUDA library.

Seeds: data 1000+cfg, calibration 2000+cfg, outlier channels 3000+cfg.  Every tensor is drawn
in independent chunks, chunk c from PCG64(SeedSequence([seed, c])), so the values do not depend
on how many threads draw them.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

G = 128
_ROWS_PER_CHUNK = 256


def _rng(seed: int, chunk: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, chunk])))


def _threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return os.cpu_count() or 1


def _parallel(fn, n: int) -> None:
    t = min(_threads(), n)
    if t <= 1:
        for i in range(n):
            fn(i)
    else:
        with ThreadPoolExecutor(t) as ex:
            list(ex.map(fn, range(n)))


def weight_matrix(rows: int, cols: int, seed: int, sigma: float = 0.02, row_scale: bool = True) -> np.ndarray:
    """Student-t(df=5) * sigma, optionally times a per-row lognormal(0, 0.5) factor; fp16 [rows][cols]."""
    out = np.empty((rows, cols), dtype=np.float16)
    rs = np.exp(_rng(seed, 1 << 30).normal(0.0, 0.5, size=rows)).astype(np.float32) if row_scale else np.ones(rows, np.float32)

    def chunk(c: int) -> None:
        r0, r1 = c * _ROWS_PER_CHUNK, min(rows, (c + 1) * _ROWS_PER_CHUNK)
        rng = _rng(seed, c)
        z = rng.standard_normal(size=(r1 - r0, cols), dtype=np.float32)
        chi2 = rng.standard_gamma(2.5, size=(r1 - r0, cols), dtype=np.float32) * np.float32(2.0)
        t = z / np.sqrt(chi2 / np.float32(5.0))           # Student-t with 5 degrees of freedom
        out[r0:r1] = (t * (np.float32(sigma) * rs[r0:r1, None])).astype(np.float16)

    _parallel(chunk, (rows + _ROWS_PER_CHUNK - 1) // _ROWS_PER_CHUNK)
    return out


def kv_cache(batch: int, heads: int, seq: int, seed: int, outlier_seed: int, head_dim: int = G) -> np.ndarray:
    """N(0,1) with 4 fixed channels of each head scaled by 10; fp16 [batch][heads][seq][head_dim]."""
    orng = _rng(outlier_seed)
    chan_scale = np.ones((heads, head_dim), dtype=np.float32)
    for h in range(heads):
        chan_scale[h, orng.choice(head_dim, size=4, replace=False)] = 10.0
    out = np.empty((batch, heads, seq, head_dim), dtype=np.float16)

    def chunk(i: int) -> None:
        b, h = divmod(i, heads)
        x = _rng(seed, i).standard_normal(size=(seq, head_dim), dtype=np.float32) * chan_scale[h]
        out[b, h] = x.astype(np.float16)

    _parallel(chunk, batch * heads)
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
