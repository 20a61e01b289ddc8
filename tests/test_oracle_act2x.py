"""Pins of the oracle's 2x activation codec (7-bit values, bit-interleaved fp16 scale and zero point)."""
import numpy as np
import pytest


def test_hand_assembled_block(eo):
    """scale 0.5 (fp16 0x3800), zero point 2.0 (fp16 0x4000), q_i = i - 32 for i < 64: derived by hand.
    Metadata bits, lsb first: scale 0x3800 -> bits 11,12,13 set; zero 0x4000 -> bit 14 -> metadata bit 30."""
    blk = np.zeros(64, dtype=np.uint8)
    for i in range(64):
        blk[i] = (i - 32) & 0x7F
    for mbit in (11, 12, 13, 30):
        blk[mbit] |= 0x80
    out = eo.act_decode(blk)[0].astype(np.float64)
    assert np.array_equal(out, (np.arange(64) - 32) * 0.5 + 2.0)


def test_roundtrip_bounds_and_field_layout(eo, synth):
    x = synth.activations(64, 4096, 21).reshape(-1, 64)
    x[3] = np.float16(1.25)                       # constant group: zero scale
    x[4, :] = 0
    x[5] = (np.arange(64) * 3 - 50).astype(np.float16)   # exactly on a grid of step 3 * 63/127... not exact, just monotone
    blocks = eo.act_encode(x)
    assert blocks.shape == (x.shape[0], 64)
    assert np.all(blocks[:, 32:] < 0x80)          # metadata bits 32..63 are zero
    meta = np.zeros(x.shape[0], dtype=np.uint32)
    for i in range(32):
        meta |= (blocks[:, i].astype(np.uint32) >> 7) << i
    scale = (meta & 0xFFFF).astype(np.uint16).view(np.float16).astype(np.float64)
    zero = (meta >> 16).astype(np.uint16).view(np.float16).astype(np.float64)
    xf = x.astype(np.float64)
    lo, hi = xf.min(1), xf.max(1)
    assert np.array_equal(scale, ((hi - lo).astype(np.float32) / np.float32(127)).astype(np.float16).astype(np.float64))
    q = (blocks & 0x7F).astype(np.int32)
    q = np.where(q >= 64, q - 128, q)
    assert q.min() >= -64 and q.max() <= 63
    out = eo.act_decode(blocks).astype(np.float64)
    # closed-form error bound: half a step plus the roundings of zero point and result
    bound = scale[:, None] * 0.5 + np.abs(zero[:, None]) * 2.0 ** -10 + np.abs(xf) * 2.0 ** -10 + scale[:, None] * 1.01
    assert np.all(np.abs(out - xf) <= bound)
    rel = np.sqrt(((out - xf) ** 2).mean() / (xf ** 2).mean())
    assert rel < 0.02                             # 7-bit uniform quantisation of N(0,1) groups
    assert np.array_equal(out[3], xf[3]) and np.all(out[4] == 0)
    # minimum maps to q = -64, order is preserved
    assert np.all(q[np.arange(x.shape[0]), xf.argmin(1)][scale > 0] == -64)
    assert np.all(np.diff(q[5]) >= 0)
    # quantisation, recomputed exactly: q = rint((x - zero) * (1 / scale)) in fp32 (the compressor's multiply-and-round
    # circuit, Sec. 4.3), round half to even, clamped to the 7-bit range -- truncation or round-half-up would fail here
    x32, s32, z32 = x.astype(np.float32), scale.astype(np.float32)[:, None], zero.astype(np.float32)[:, None]
    live = (scale > 0)[:, None]
    with np.errstate(divide="ignore", invalid="ignore"):
        inv = (np.float32(1.0) / s32).astype(np.float32)
        want_q = np.clip(np.rint(((x32 - z32).astype(np.float32) * inv).astype(np.float32)), -64, 63)
    want_q = np.where(live, want_q, 0).astype(np.int32)
    assert np.array_equal(q, want_q)
    # dequantisation = one fused multiply-add in fp32, one rounding to fp16
    want = (q.astype(np.float64) * scale[:, None] + zero[:, None]).astype(np.float32).astype(np.float16)
    assert np.array_equal(out.astype(np.float16).view(np.uint16), want.view(np.uint16))


def test_non_finite_input_is_refused(eo):
    x = np.zeros(64, dtype=np.float16)
    x[7] = np.inf
    with pytest.raises(RuntimeError):
        eo.act_encode(x)
