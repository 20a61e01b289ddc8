"""Pins of the oracle's number formats against library routines and closed forms."""
import numpy as np
import pytest
import torch


def test_fp16_decode_all_codes_matches_numpy(eo):
    codes = np.arange(65536, dtype=np.uint16)
    ref = codes.view(np.float16).astype(np.float32)
    for c in range(0, 65536):
        v = eo.fp16_to_f32(c)
        r = ref[c]
        if np.isnan(r):
            assert np.isnan(v)
        else:
            assert v == r and np.signbit(v) == np.signbit(r), c


def test_fp16_encode_matches_numpy_rounding(eo):
    rng = np.random.Generator(np.random.PCG64(7))
    # every fp16 value, every midpoint between neighbours, and values just off the midpoints
    h = np.arange(0, 0x7C00, dtype=np.uint16).view(np.float16).astype(np.float64)
    mids = (h[:-1] + h[1:]) / 2
    cand = np.concatenate([h, mids, mids * (1 + 1e-7), mids * (1 - 1e-7), [65504, 65519.9, 65520, 70000, 1e-9, 2.0 ** -25],
                           rng.standard_normal(20000) * 3, rng.standard_normal(5000) * 1e-5]).astype(np.float32)
    cand = np.concatenate([cand, -cand])
    with np.errstate(over="ignore"):
        ref = cand.astype(np.float16).view(np.uint16)
    for f, r in zip(cand.tolist(), ref.tolist()):
        assert eo.f32_to_fp16(f) == r, (f, r)


def test_e4m3_decode_matches_torch_on_all_non_nan_codes(eo):
    codes = torch.arange(256, dtype=torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).to(torch.float32).numpy()
    for c in range(256):
        v = eo.e4m3_to_f32(c)
        if (c & 0x7F) == 0x7F:
            assert abs(v) == 480.0  # the oracle's arithmetic reading of the NaN code
        else:
            assert v == ref[c] and np.signbit(v) == np.signbit(ref[c])
    assert eo.e4m3_to_f32(0x7E) == 448.0 and eo.e4m3_to_f32(0x01) == 2.0 ** -9


def test_e4m3_encode_matches_torch_in_range_and_saturates(eo):
    rng = np.random.Generator(np.random.PCG64(8))
    grid = np.array([eo.e4m3_to_f32(c) for c in range(0x7F)], dtype=np.float64)
    mids = (grid[:-1] + grid[1:]) / 2
    cand = np.concatenate([grid, mids, mids * (1 + 1e-6), mids * (1 - 1e-6), rng.uniform(0, 448, 20000),
                           rng.standard_normal(5000) * 0.01]).astype(np.float32)
    cand = np.concatenate([cand, -cand])
    cand = cand[np.abs(cand) <= 448]
    ref = torch.from_numpy(cand).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    for f, r in zip(cand.tolist(), ref.tolist()):
        assert eo.e4m3_from_f32(f) == r, (f, r)
    for f in (448.1, 463.9, 464.0, 480.0, 1e6, float("inf")):
        assert eo.e4m3_from_f32(f) == 0x7E and eo.e4m3_from_f32(-f) == 0xFE
    # nearest-value property straight from the definition, ties to the even code
    for f in cand[:4000].tolist():
        c = eo.e4m3_from_f32(abs(f))
        d = np.abs(grid - abs(f))
        assert d[c] == d.min()
        if (d == d.min()).sum() == 2:
            assert c % 2 == 0


def test_dequantisation_product_is_exact_in_fp32(eo):
    """fp16 centroid (11-bit significand) x E4M3 scale (4-bit) x 2^e has at most 15 significant
    bits, so the fp32 product is exact and 'one rounding to fp16' is well defined: the oracle's
    result must equal the correctly rounded exact product computed with integers/fp64."""
    rng = np.random.Generator(np.random.PCG64(9))
    cents = rng.integers(0, 0x3C01, size=40).astype(np.uint16)  # |c| <= 1
    for e in (-12, -9, -3, 0):
        T = 2.0 ** e
        for c16 in cents.tolist():
            c = float(np.uint16(c16).view(np.float16))
            for q in range(0, 0x7F):
                s = eo.e4m3_to_f32(q) * T
                exact = c * s  # exact in fp64 too
                assert float(np.float32(c) * np.float32(s)) == exact
                got = eo.f32_to_fp16(np.float32(c) * np.float32(s))
                with np.errstate(over="ignore"):
                    want = int(np.float64(exact).astype(np.float16).view(np.uint16))
                assert got == want
