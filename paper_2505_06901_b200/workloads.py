"""The five benchmark configurations as compressed, ready-to-upload tensors.

Built from the seeded generators in synth.py with the library's own host calibrator and
encoder (ecco_calibrate_host / ecco_encode_host).  Used by the GPU tests and bench.py.

Metadata is per tensor (Sec. 4.2, "tensor-wise metadata"): the patterns and codebooks are
calibrated once per configuration on a separate seeded calibration tensor, and every tensor
gets its own copy whose exponent is fitted to that tensor.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import binding as B
from . import synth

G = 128


@dataclass
class Compressed:
    name: str
    shape: tuple            # logical fp16 shape
    blocks: np.ndarray      # uint8 [n_groups][64]
    meta: B.Meta
    stats: object
    source: np.ndarray | None = None   # the fp16 original (kept only on request)
    extra: dict = field(default_factory=dict)

    @property
    def n_groups(self) -> int:
        return self.blocks.shape[0]


def _clone_meta(meta: B.Meta) -> B.Meta:
    S, e, pat, cb, kp = meta.tables()
    return B.ecco_meta_create(S, e, pat, cb, kp)


def calibrate_weights(cfg: int, sigma: float, row_scale: bool, S: int = 64) -> B.Meta:
    cal = synth.weight_matrix(1024, 1024, 2000 + cfg, sigma=sigma, row_scale=row_scale)
    return B.ecco_calibrate_host(cal, S=S, H=4, seed=cfg, select=B.SELECT_MSE)


def calibrate_kv(cfg: int, heads: int, S: int = 64, select: int = B.SELECT_MINMAX) -> B.Meta:
    cal = synth.kv_cache(1, heads, max(256, 8192 // heads), 2000 + cfg, 3000 + cfg)
    return B.ecco_calibrate_host(cal, S=S, H=4, seed=cfg, select=select)


def weight_tensor(name: str, rows: int, cols: int, seed: int, base_meta: B.Meta, sigma: float, row_scale: bool,
                  keep_source: bool = False) -> Compressed:
    w = synth.weight_matrix(rows, cols, seed, sigma=sigma, row_scale=row_scale)
    meta = _clone_meta(base_meta)
    blocks, st = B.ecco_encode_host(meta, w, B.SELECT_MSE)
    return Compressed(name, (rows, cols), blocks, meta, st, w if keep_source else None)


def kv_tensor(name: str, batch: int, heads: int, seq: int, seed: int, outlier_seed: int, base_meta: B.Meta,
              select: int = B.SELECT_MINMAX, keep_source: bool = False) -> Compressed:
    x = synth.kv_cache(batch, heads, seq, seed, outlier_seed)
    meta = _clone_meta(base_meta)
    # the KV cache is encoded online in the paper (Sec. 3.2), so the exponent stays the calibrated one
    blocks, st = B.ecco_encode_host(meta, x, select | B.KEEP_EXPONENT)
    return Compressed(name, (batch, heads, seq, G), blocks, meta, st, x if keep_source else None)


LLAMA7B_LAYER = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
                 ("gate", 11008, 4096), ("up", 11008, 4096), ("down", 4096, 11008)]
LLAMA70B_MLP = [("gate", 28672, 8192), ("up", 28672, 8192), ("down", 8192, 28672)]


def config1(keep_source: bool = False) -> Compressed:
    """1024x1024 weight matrix, Student-t(5)*0.02 with per-row lognormal(0, 0.5) scale."""
    return weight_tensor("cfg1", 1024, 1024, 1001, calibrate_weights(1, 0.02, True), 0.02, True, keep_source)


def config2(names=None, keep_source: bool = False) -> list:
    """Llama-2-7B-shaped decoder layer: q/k/v/o 4096x4096, gate/up 11008x4096, down 4096x11008."""
    base = calibrate_weights(2, 0.02, True)
    return [weight_tensor(n, r, c, 1002 * 16 + i, base, 0.02, True, keep_source)
            for i, (n, r, c) in enumerate(LLAMA7B_LAYER) if names is None or n in names]


def config3(which=("K",), keep_source: bool = False) -> list:
    """KV cache of one Llama-2-7B-shaped layer: [8][32][4096][128], 4 outlier channels x10 per head."""
    base = calibrate_kv(3, 32)
    return [kv_tensor(w, 8, 32, 4096, 1003 * 16 + i, 3003, base, keep_source=keep_source)
            for i, w in enumerate(("K", "V")) if w in which]


def config4(names=None, keep_source: bool = False) -> list:
    """70B-shaped MLP weights, Student-t(5)*0.01, no row scale: gate/up 28672x8192, down 8192x28672."""
    base = calibrate_weights(4, 0.01, False)
    return [weight_tensor(n, r, c, 1004 * 16 + i, base, 0.01, False, keep_source)
            for i, (n, r, c) in enumerate(LLAMA70B_MLP) if names is None or n in names]


def config5(which=("K",), keep_source: bool = False) -> list:
    """Long-context GQA KV cache: [16][8][32768][128]."""
    base = calibrate_kv(5, 8)
    return [kv_tensor(w, 16, 8, 32768, 1005 * 16 + i, 3005, base, keep_source=keep_source)
            for i, w in enumerate(("K", "V")) if w in which]
