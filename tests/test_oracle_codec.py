"""Pins of the oracle's encoder and decoder: a hand-assembled block, an independent bit-string
decoder, encode->decode round trips, brute-force pattern choice, clip/pad rules, totality."""
import ctypes
import json
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def pack_bits(bitstring):
    """'0101...' in stream order -> 64 bytes, stream bit k at bit k%8 of byte k//8."""
    assert len(bitstring) == 512
    out = np.zeros(64, dtype=np.uint8)
    for k, ch in enumerate(bitstring):
        if ch == "1":
            out[k >> 3] |= 1 << (k & 7)
    return out


def lsb_first(value, nbits):
    return "".join("1" if (value >> i) & 1 else "0" for i in range(nbits))


def codewords(eo, lens, maxlen):
    codes, _ = eo.canonical_codes(lens, maxlen)
    return [format(int(c), "b").zfill(int(l)) for c, l in zip(codes, lens)]


def bitstring_decode(eo, meta, blk):
    """Independent decoder working on a text bit string with dictionary prefix matching.
    Returns (kp, hf, qs, symbols, end_bit, pads[(loc, byte)])."""
    bits = "".join(lsb_first(int(b), 8) for b in blk) + "0" * 16
    qs = int(bits[0:8][::-1], 2)
    hf = int(bits[8:10][::-1], 2)
    kpw = {w: k for k, w in enumerate(codewords(eo, meta.kp_lengths(), 12))}
    pos, cur = 10, ""
    while cur not in kpw:
        cur += bits[pos + len(cur)]
    kp = kpw[cur]
    pos += len(cur)
    cw = {w: s for s, w in enumerate(codewords(eo, meta.cb_lengths()[kp, hf], 8))}
    syms = []
    while len(syms) < 128:
        cur = ""
        while cur not in cw:
            cur += bits[pos + len(cur)]
        if pos + len(cur) > 512:
            break
        syms.append(cw[cur])
        pos += len(cur)
    pads = []
    if len(syms) == 128:
        for j in range(min(16, (512 - pos) // 15)):
            f = bits[512 - 15 * (j + 1): 512 - 15 * j]
            pads.append((int(f[:7][::-1], 2), int(f[7:][::-1], 2)))
    return kp, hf, qs, syms, pos, pads


def test_hand_assembled_block(eo):
    g = json.load(open(os.path.join(GOLDEN, "worked_block.json")))
    meta = eo.Meta()
    meta.S, meta.H, meta.e = g["S"], 4, g["e"]
    for k in range(meta.S):
        meta.kp_len[k] = g["kp_len"][k]
        for h in range(4):
            for s in range(16):
                meta.cb_len[k][h][s] = 4
        for j in range(15):
            meta.pattern[k][j] = int(np.float16((j - 7) / 16).view(np.uint16))   # other patterns differ
    for s in range(16):
        meta.cb_len[3][2][s] = g["cb_len_kp3_hf2"][s]
    for j in range(15):
        meta.pattern[3][j] = int(np.float16(g["pattern_kp3_times_8"][j] / 8).view(np.uint16))
    assert eo.meta_check(meta) == 0

    cw = g["codewords"]
    stream = lsb_first(int(g["scale_byte"], 16), 8) + lsb_first(g["id_hf"], 2) + g["id_kp_codeword"]
    stream += cw["0"] + cw["4"] + cw["1"] * 126
    assert len(stream) == g["end_bit"]
    pads = "".join(lsb_first(100 + j, 7) + lsb_first(0x30 + j, 8) for j in reversed(range(16)))
    stream += "0" * (512 - len(stream) - len(pads)) + pads
    blk = pack_bits(stream)
    for idx, val in g["hand_bytes"].items():
        assert blk[int(idx)] == int(val, 16), idx

    out, sym, info = eo.decode_block(meta, blk)
    assert (info.kp, info.hf, info.qs, info.n_fit, info.n_pad, info.end_bit) == (3, 2, 0x3A, 128, 16, 270)
    assert sym[0] == 0 and sym[1] == 4 and np.all(sym[2:] == 1)
    want = np.full(128, -30 / 512, dtype=np.float64)
    want[0], want[1] = -35 / 512, -15 / 512
    for j in range(16):
        want[100 + j] = (8 + j) / 256 if j < 8 else j / 128
    assert np.array_equal(out.astype(np.float64), want)
    # the independent bit-string decoder reads the same fields
    kp, hf, qs, syms, end, pd = bitstring_decode(eo, meta, blk)
    assert (kp, hf, qs, end) == (3, 2, 0x3A, 270) and syms == [0, 4] + [1] * 126
    assert pd == [(100 + j, 0x30 + j) for j in range(16)]


def numpy_quantize(meta_pat, x16, e, select):
    """Independent restatement of Fig. 4 steps 2 and 5 with numpy (brute force over patterns)."""
    x = x16.astype(np.float32)
    T = np.float32(2.0 ** e)
    p = int(np.argmax(np.abs(x)))
    return x, T, p


def test_pattern_choice_is_the_brute_force_optimum(eo, cfg1_small, kv_small):
    for fx, key, select in ((cfg1_small, "w", 0), (kv_small, "k", 1)):
        meta = fx["meta"]
        pats = meta.patterns().astype(np.float32).astype(np.float64)     # [S][15]
        groups = fx[key].reshape(-1, 128)
        T = np.float32(2.0 ** meta.e)
        for g in range(0, groups.shape[0], 97):
            x = groups[g].astype(np.float32)
            q = eo.quantize_group(meta, groups[g], select)
            p = int(np.argmax(np.abs(x)))                                # first index of the max
            assert q["pstar"] == p
            assert q["qs"] == eo.e4m3_from_f32(float(x[p] / T))
            s = np.float32(abs(eo.e4m3_to_f32(q["qs"]))) * T
            u = np.delete(x / s, p).astype(np.float64)
            assert np.array_equal(np.delete(q["u"], p).astype(np.float64), u)
            d = (u[None, :, None] - pats[:, None, :]) ** 2              # [S][127][15]
            if select == 0:
                score = d.min(axis=2).sum(axis=1)
            else:
                score = (pats[:, 0] - u.min()) ** 2 + (pats[:, 14] - u.max()) ** 2
            # sequential fp64 sums in the oracle vs pairwise sums here: allow rounding noise on near-ties
            assert score[q["kp"]] <= score.min() * (1 + 1e-12) + 1e-300
            if np.sort(score)[1] > score.min() * (1 + 1e-9):
                assert q["kp"] == int(score.argmin())
            sym = np.delete(q["sym"], p)
            assert q["sym"][p] == 15 and sym.max() <= 14
            assert np.array_equal(sym, d[q["kp"]].argmin(axis=1))        # nearest centroid, ties low


def test_roundtrip_recovers_every_field(eo, cfg1_small, kv_small):
    seen_clip = seen_pad = 0
    for fx, key, select in ((cfg1_small, "w", 0), (kv_small, "k", 1)):
        meta, groups = fx["meta"], fx[key].reshape(-1, 128)
        cb = meta.cb_lengths()
        T = np.float32(2.0 ** meta.e)
        for g in range(0, groups.shape[0], 5):
            blk, sym, ei = eo.encode_group(meta, groups[g], select)
            assert np.array_equal(blk, fx["blocks"][g])
            out, dsym, di = eo.decode_block(meta, blk)
            assert (di.kp, di.hf, di.qs, di.n_fit, di.n_pad, di.end_bit) == (ei.kp, ei.hf, ei.qs, ei.n_fit, ei.n_pad, ei.end_bit)
            assert np.array_equal(dsym[: ei.n_fit], sym[: ei.n_fit])
            # step 8: the chosen codebook is the arg-min of the total length, ties low
            totals = cb[ei.kp][:, sym].astype(np.int64).sum(axis=1)
            assert ei.hf == int(totals.argmin())
            # step 9: clip = number of whole codewords that fit; pad count from the slack
            ends = 10 + int(meta.kp_lengths()[ei.kp]) + np.cumsum(cb[ei.kp, ei.hf][sym])
            n_fit = int((ends <= 512).sum())
            assert ei.n_fit == n_fit
            x = groups[g].astype(np.float32)
            if n_fit < 128:
                seen_clip += 1
                assert ei.n_pad == 0 and np.all(out[n_fit:].view(np.uint16) == 0)
            else:
                assert ei.end_bit == ends[-1] and ei.n_pad == min(16, (512 - ei.end_bit) // 15)
            # mapper: one fp32 product, one rounding
            s = np.float32(abs(eo.e4m3_to_f32(ei.qs))) * T
            pat = meta.patterns()[ei.kp].astype(np.float32)
            want = np.zeros(128, dtype=np.float16)
            for i in range(n_fit):
                want[i] = np.float16(np.float32(eo.e4m3_to_f32(ei.qs)) * T) if sym[i] == 15 else np.float16(pat[sym[i]] * s)
            if ei.n_pad:
                seen_pad += 1
                order = sorted((i for i in range(128) if i != ei.pstar), key=lambda i: (-abs(float(x[i])), i))
                for j in range(ei.n_pad):
                    loc = order[j]
                    want[loc] = np.float16(np.float32(eo.e4m3_to_f32(eo.e4m3_from_f32(float(x[loc] / T)))) * T)
            assert np.array_equal(out.view(np.uint16), want.view(np.uint16)), g
            # the abs-max element comes back as its FP8 rounding
            if ei.n_fit > ei.pstar:
                assert abs(float(out[ei.pstar]) - float(x[ei.pstar])) <= abs(float(x[ei.pstar])) * 2 ** -4 + 1e-7
            # the independent bit-string decoder agrees on the stream
            if g % 50 == 0:
                kp, hf, qs, syms, end, pd = bitstring_decode(eo, meta, blk)
                assert (kp, hf, qs, end) == (di.kp, di.hf, di.qs, di.end_bit)
                assert syms == list(dsym[: di.n_fit]) and len(pd) == di.n_pad
    assert seen_clip > 5 and seen_pad > 5       # both cases are exercised by the synthetic data


def test_literal_clip_never_decodes_a_spurious_symbol(eo, cfg1_small):
    """The slack after the last whole codeword holds a proper prefix of the next codeword; by
    prefix-freeness no codeword fits inside it, so the decoder's 'reject a codeword crossing bit
    512' rule recovers n_fit exactly."""
    meta, st = cfg1_small["meta"], cfg1_small["stats"]
    assert st.clipped_groups > 0
    groups = cfg1_small["w"].reshape(-1, 128)
    n = 0
    for g in range(groups.shape[0]):
        _, sym, ei = eo.encode_group(meta, groups[g], 0)
        if ei.n_fit < 128:
            _, dsym, di = eo.decode_block(meta, cfg1_small["blocks"][g])
            assert di.n_fit == ei.n_fit and np.all(dsym[ei.n_fit:] == 0xFF)
            n += 1
            if n > 40:
                break


def test_block_and_stats_consistency_numbers(eo, cfg1_small):
    blocks, st = cfg1_small["blocks"], cfg1_small["stats"]
    assert blocks.shape == (2048, 64) and blocks.dtype == np.uint8     # 4 bits x 128 = 512 bits = 64 B
    assert st.n_groups == 2048 and sum(st.kp_usage) == 2048 and sum(st.hf_usage) == 2048
    assert sum(st.sym_count) == 2048 * 128 and st.sym_count[15] == 2048  # one abs-max per group
    assert 15 == 7 + 8                                                  # pad = 7-bit location + FP8 value
    mean_bits = st.total_bits / st.n_groups
    assert 400 < mean_bits <= 512
    # average code length within one bit of the empirical entropy of the symbols
    p = np.array(st.sym_count[:], dtype=np.float64)
    p = p[p > 0] / p.sum()
    H = float(-(p * np.log2(p)).sum())
    assert (mean_bits - 10) / 128 < H + 1.0


def test_decoder_is_total_on_garbage(eo, cfg1_small, synth):
    meta = cfg1_small["meta"]
    rb = synth.random_blocks(4096, 99)
    out = eo.decode(meta, rb)
    assert out.shape == (4096, 128) and np.isfinite(out.astype(np.float32)).all()
    for pattern in (0x00, 0xFF, 0xAA, 0x55):
        eo.decode(meta, np.full((4, 64), pattern, dtype=np.uint8))


def test_degenerate_groups(eo, cfg1_small):
    meta = cfg1_small["meta"].copy()
    zero = np.zeros(128, dtype=np.float16)
    blk, sym, info = eo.encode_group(meta, zero, 0)
    out, _, _ = eo.decode_block(meta, blk)
    assert info.pstar == 0 and info.qs == 0 and np.all(out.astype(np.float32) == 0)
    const = np.full(128, 0.01, dtype=np.float16)
    blk, sym, info = eo.encode_group(meta, const, 0)
    out, _, di = eo.decode_block(meta, blk)
    assert info.pstar == 0 and sym[0] == 15 and len(set(sym[1:].tolist())) == 1
    # a scale that underflows FP8 (|x|/T below half the smallest subnormal) gives s = 0 and zeros
    tiny = np.full(128, 2.0 ** -24, dtype=np.float16)
    meta.e = 0
    blk, sym, info = eo.encode_group(meta, tiny, 0)
    out, _, _ = eo.decode_block(meta, blk)
    assert info.qs == 0 and np.all(out.astype(np.float32) == 0)
    bad = zero.copy(); bad[5] = np.inf
    with pytest.raises(RuntimeError):
        eo.encode_group(meta, bad, 0)
    bad[5] = np.nan
    with pytest.raises(RuntimeError):
        eo.encode(meta, bad, 0)


def test_exponent_is_the_smallest_power_of_two_that_avoids_saturation(eo, cfg1_small):
    meta = cfg1_small["meta"].copy()
    for mx in (0.0, 1e-6, 0.01, 0.4375, 0.43751, 448.0, 449.0, 65504.0):
        x = np.zeros(256, dtype=np.float16); x[3] = -mx
        eo.set_exponent(meta, x)
        v = float(np.float16(mx))
        assert v <= 448 * 2.0 ** meta.e
        assert meta.e == -32 or v > 448 * 2.0 ** (meta.e - 1)


def test_fused_consumers_reduce_to_textbook_products(eo, cfg1_small, kv_small, synth):
    meta, blocks = cfg1_small["meta"], cfg1_small["blocks"]
    W = eo.decode(meta, blocks).reshape(256, 1024).astype(np.float64)
    x = synth.activations(3, 1024, 5)
    y, ya = eo.gemv(meta, blocks, 256, 1024, x, 3)
    ref = x.astype(np.float64) @ W.T
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-12)
    assert np.allclose(ya, np.abs(x.astype(np.float64))[:, None, :].__mul__(np.abs(W)[None]).sum(-1), rtol=1e-12)
    # attention scores with 2 query heads per KV head
    km, kb = kv_small["meta"], kv_small["blocks"]
    K = eo.decode(km, kb).reshape(2, 4, 256, 128).astype(np.float64)
    q = synth.queries(2, 8, 6)
    s, sa = eo.attn_scores(km, kb, 2, 4, 256, 2, q, 128 ** -0.5)
    ref = np.einsum("bhrd,bhtd->bhrt", q.astype(np.float64).reshape(2, 4, 2, 128), K).reshape(2, 8, 256) * 128 ** -0.5
    assert np.allclose(s, ref, rtol=1e-12, atol=1e-12)
    assert np.all(sa >= np.abs(s) - 1e-12)


def test_compression_quality_on_the_synthetic_distributions(eo, cfg1_small, kv_small):
    """Sanity of the whole pipeline: 4-bit-class reconstruction error on both distributions."""
    w = cfg1_small["w"].astype(np.float32)
    out = eo.decode(cfg1_small["meta"], cfg1_small["blocks"]).reshape(w.shape).astype(np.float32)
    assert np.sqrt(((out - w) ** 2).mean() / (w ** 2).mean()) < 0.15
    k = kv_small["k"].astype(np.float32)
    out = eo.decode(kv_small["meta"], kv_small["blocks"]).reshape(k.shape).astype(np.float32)
    assert np.sqrt(((out - k) ** 2).mean() / (k ** 2).mean()) < 0.2
    # threaded driver gives the same bytes as the single-threaded loop
    a = eo.decode_threads(kv_small["meta"], kv_small["blocks"], 3)
    assert np.array_equal(a.view(np.uint16), eo.decode(kv_small["meta"], kv_small["blocks"]).view(np.uint16))


def test_attention_output_reduces_to_textbook_softmax_times_v(eo, kv_small, synth):
    km, kb = kv_small["meta"], kv_small["blocks"]
    V = eo.decode(km, kb).reshape(2, 4, 256, 128).astype(np.float64)
    rng = np.random.Generator(np.random.PCG64(31))
    scores = (rng.standard_normal((2, 8, 256)) * 3).astype(np.float32)
    out, oa = eo.attn_values(km, kb, 2, 4, 256, 2, scores)
    s = scores.astype(np.float64)
    p = np.exp(s - s.max(-1, keepdims=True))
    p /= p.sum(-1, keepdims=True)
    ref = np.einsum("bhrt,bhtd->bhrd", p.reshape(2, 4, 2, 256), V).reshape(2, 8, 128)
    assert np.allclose(out, ref, rtol=1e-12, atol=1e-14)
    assert np.all(oa >= np.abs(out) - 1e-12)
    # a one-hot softmax (one logit far above the rest) returns that token's decompressed vector
    scores[:] = -1e4
    scores[:, :, 17] = 0.0
    out, _ = eo.attn_values(km, kb, 2, 4, 256, 2, scores)
    assert np.allclose(out.reshape(2, 4, 2, 128), V[:, :, 17][:, :, None, :], rtol=1e-12)


def test_variable_length_container_round_trip(eo, cfg1_small):
    """No clipping, no padding: every group decodes to exactly the mapped values of its 128 symbols, the
    stream is the concatenation of the groups' bit strings, and groups that fit a block agree with it."""
    meta, w = cfg1_small["meta"], cfg1_small["w"]
    stream, off = eo.var_encode(meta, w[:64], eo.SELECT_MSE)
    n = 64 * 1024 // 128
    assert off.size == n + 1 and off[0] == 0 and np.all(np.diff(off.astype(np.int64)) >= 10 + 1 + 256)
    out = eo.var_decode(meta, stream, off)
    cb, kl, pats = meta.cb_lengths(), meta.kp_lengths(), meta.patterns().astype(np.float32)
    T = np.float32(2.0 ** meta.e)
    blocks = cfg1_small["blocks"]
    n_unclipped = 0
    for g in range(n):
        q = eo.quantize_group(meta, w.reshape(-1, 128)[g], eo.SELECT_MSE)
        totals = cb[q["kp"]][:, q["sym"]].astype(np.int64).sum(axis=1)
        hf = int(totals.argmin())
        assert int(off[g + 1] - off[g]) == 10 + int(kl[q["kp"]]) + int(totals[hf])          # bit-exact length
        s = np.float32(abs(eo.e4m3_to_f32(q["qs"]))) * T
        want = np.array([np.float16(np.float32(eo.e4m3_to_f32(q["qs"])) * T) if sy == 15 else np.float16(pats[q["kp"]][sy] * s)
                         for sy in q["sym"]], dtype=np.float16)
        assert np.array_equal(out[g].view(np.uint16), want.view(np.uint16))
        # the group's bits are the block's bits when the block was neither clipped nor padded past them
        _, _, info = eo.decode_block(meta, blocks[g])
        if info.n_fit == 128:
            n_unclipped += 1
            L = int(off[g + 1] - off[g])
            bits_blk = int.from_bytes(blocks[g].tobytes(), "little") & ((1 << L) - 1)
            big = int.from_bytes(stream[int(off[g]) // 8: int(off[g]) // 8 + 140].tobytes(), "little") >> (int(off[g]) % 8)
            assert big & ((1 << L) - 1) == bits_blk
    assert n_unclipped > n // 2
    # totality: garbage stream, arbitrary (even overlapping) offsets
    rng = np.random.Generator(np.random.PCG64(3))
    junk = rng.integers(0, 256, 4096, dtype=np.uint8)
    joff = np.sort(rng.integers(0, 4096 * 8, 33)).astype(np.uint64)
    joff[-1] = 4096 * 8
    assert np.isfinite(eo.var_decode(meta, junk, joff).astype(np.float32)).all()
