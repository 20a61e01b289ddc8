"""CPU tests of the library's host half: ABI surface, encoder parity with the oracle (byte for
byte, given the oracle's metadata), calibrator invariants, decode-table image."""
import ctypes
import re
import os

import numpy as np
import pytest

from helpers import lib_meta_from_oracle, oracle_meta_from_lib

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="session")
def binding():
    from paper_2505_06901_b200 import binding as b

    b.lib()
    return b


def test_library_exports_every_declared_symbol(binding):
    header = open(os.path.join(ROOT, "include", "ecco.h")).read()
    declared = set(re.findall(r"\b(ecco_[a-z0-9_]+)\s*\(", header))
    declared -= {"ecco_meta"}
    assert declared == set(binding.EXPORTS), declared ^ set(binding.EXPORTS)
    L = ctypes.CDLL(binding.lib_path())
    for name in declared:
        assert hasattr(L, name), name
    assert ctypes.sizeof(binding.Stats) == 8 * (6 + 64 + 4 + 16)
    assert binding.lib().ecco_error_string(-3) == b"non-finite input value"


def test_argument_errors_without_a_gpu(binding, cfg1_small, eo):
    L = binding.lib()
    lm = lib_meta_from_oracle(binding, cfg1_small["meta"])
    assert L.ecco_decompress(None, None, 0, None, None) == 0                    # empty input is a no-op
    assert L.ecco_decompress(None, None, 5, None, None) == binding.ERR_INVALID_ARG
    assert L.ecco_decompress(16, 32, 5, 48 + 1, None) == binding.ERR_ALIGNMENT  # checked before any CUDA call
    assert L.ecco_gemv(16, 32, 100, 100, 64, 1, 128, None, 0, None) == binding.ERR_INVALID_ARG   # k % 128
    assert L.ecco_gemv(16, 32, 100, 128, 64, 9, 128, None, 0, None) == binding.ERR_INVALID_ARG   # batch > 8
    assert L.ecco_attn_scores(16, 32, 1, 1, 8, 9, 64, ctypes.c_float(1.0), 128, None) == binding.ERR_INVALID_ARG
    assert L.ecco_gemv_workspace_bytes(4096, 4096, 1) >= 4096 * 4 * 32
    assert L.ecco_gemv_workspace_bytes(4096, 100, 1) == 0
    # bad metadata tables are refused
    pat, cb, kp = cfg1_small["meta"].patterns(), cfg1_small["meta"].cb_lengths(), cfg1_small["meta"].kp_lengths()
    bad_cb = cb.copy(); bad_cb[3, 1, 0] = 9
    with pytest.raises(binding.EccoError) as ei:
        binding.ecco_meta_create(64, -9, pat, bad_cb, kp)
    assert ei.value.code == binding.ERR_BAD_META
    bad_cb = cb.copy(); bad_cb[3, 1, 0] = 2 if cb[3, 1, 0] != 2 else 3          # breaks the Kraft equality
    with pytest.raises(binding.EccoError):
        binding.ecco_meta_create(64, -9, pat, bad_cb, kp)
    bad_pat = pat.copy(); bad_pat[5, 3], bad_pat[5, 4] = pat[5, 4] + np.float16(0.5), pat[5, 3]
    with pytest.raises(binding.EccoError):
        binding.ecco_meta_create(64, -9, bad_pat, cb, kp)
    x = cfg1_small["w"].copy().reshape(-1); x[77] = np.inf
    with pytest.raises(binding.EccoError) as ei:
        binding.ecco_encode_host(lm, x)
    assert ei.value.code == binding.ERR_NONFINITE_INPUT


@pytest.mark.parametrize("which", ["weights_mse", "kv_minmax", "kv_mse"])
def test_host_encoder_matches_oracle_byte_for_byte(binding, eo, cfg1_small, kv_small, which):
    if which == "weights_mse":
        ometa, x, flags, want = cfg1_small["meta"], cfg1_small["w"], binding.SELECT_MSE, cfg1_small["blocks"]
    elif which == "kv_minmax":
        ometa, x, flags, want = kv_small["meta"], kv_small["k"], binding.SELECT_MINMAX | binding.KEEP_EXPONENT, kv_small["blocks"]
    else:
        ometa, x, flags = kv_small["meta"], kv_small["k"], binding.SELECT_MSE | binding.KEEP_EXPONENT
        want, _ = eo.encode(ometa, x, eo.SELECT_MSE)
    lm = lib_meta_from_oracle(binding, ometa)
    got, st = binding.ecco_encode_host(lm, x, flags)
    assert lm.tables()[1] == ometa.e
    bad = np.nonzero((got != want).any(axis=1))[0]
    assert bad.size == 0, f"{bad.size} blocks differ, first {bad[:5]}"
    _, ost = eo.encode(ometa, x, flags & 1)
    for f in ("n_groups", "clipped_groups", "clipped_values", "padded_groups", "padded_values", "total_bits"):
        assert getattr(st, f) == getattr(ost, f), f
    assert list(st.kp_usage) == list(ost.kp_usage) and list(st.sym_count) == list(ost.sym_count)


def test_host_encoder_refits_the_exponent_like_the_oracle(binding, eo, cfg1_small):
    ometa = cfg1_small["meta"].copy()
    x = (cfg1_small["w"].astype(np.float32) * 37.0).astype(np.float16)
    eo.set_exponent(ometa, x)
    assert ometa.e != cfg1_small["meta"].e
    lm = lib_meta_from_oracle(binding, cfg1_small["meta"])
    got, _ = binding.ecco_encode_host(lm, x, binding.SELECT_MSE)
    want, _ = eo.encode(ometa, x, eo.SELECT_MSE)
    assert lm.tables()[1] == ometa.e and np.array_equal(got, want)


def test_host_encoder_on_adversarial_patterns_and_inputs(binding, eo):
    """Duplicate centroids, distance plateaus, exact midpoints, zero/constant/tiny groups."""
    rng = np.random.Generator(np.random.PCG64(42))
    m = eo.Meta()
    m.S, m.H, m.e = 8, 4, -6
    base = np.array([-1, -0.5, -0.5, -0.25, -0.25, -0.25, 0, 0, 0.125, 0.25, 0.25, 0.5, 0.5, 1, 1], dtype=np.float64)
    for k in range(8):
        pat = np.sort(base * (0.4 + 0.1 * k)) if k % 2 == 0 else np.sort(rng.uniform(-1, 1, 15).round(2))
        if k == 7:
            pat = np.zeros(15)
        for j in range(15):
            m.pattern[k][j] = int(np.float16(pat[j]).view(np.uint16))
        m.kp_len[k] = 3
        for h in range(4):
            ln = eo.huffman_2_8(rng.dirichlet(np.ones(16) * 0.5))
            for s in range(16):
                m.cb_len[k][h][s] = int(ln[s])
    assert eo.meta_check(m) == 0
    groups = []
    grid = np.array([-1, -0.75, -0.5, -0.375, -0.25, -0.125, 0, 0.0625, 0.125, 0.1875, 0.25, 0.375, 0.5, 0.75, 1.0])
    for t in range(300):
        g = rng.choice(grid, 128) * rng.choice([0.5, 1.0, 2.0, 0.01])
        g[rng.integers(128)] = rng.choice([-3.0, 3.0, 2.0])
        groups.append(g)
    groups.append(np.zeros(128)); groups.append(np.full(128, 0.25)); groups.append(np.full(128, 2.0 ** -24))
    groups.append(np.concatenate([np.full(64, 1.0), np.full(64, -1.0)]))
    x = np.array(groups, dtype=np.float16)
    for sel in (0, 1):
        want, _ = eo.encode(m, x, sel)
        lm = lib_meta_from_oracle(binding, m)
        got, _ = binding.ecco_encode_host(lm, x, sel | binding.KEEP_EXPONENT)
        assert np.array_equal(got, want), np.nonzero((got != want).any(axis=1))[0][:5]


def test_host_calibrator_yields_valid_and_useful_metadata(binding, eo, synth):
    cal = synth.weight_matrix(256, 1024, 2001)
    w = synth.weight_matrix(256, 1024, 1001)
    lm = binding.ecco_calibrate_host(cal, S=64, H=4, seed=5, select=binding.SELECT_MSE)
    lm2 = binding.ecco_calibrate_host(cal, S=64, H=4, seed=5, select=binding.SELECT_MSE)
    S, e, pat, cb, kp = lm.tables()
    t2 = lm2.tables()
    assert S == 64 and np.array_equal(pat.view(np.uint16), t2[2].view(np.uint16)) and np.array_equal(cb, t2[3])  # deterministic
    om = oracle_meta_from_lib(eo, lm)
    assert eo.meta_check(om) == 0                       # Kraft equality etc., checked by the oracle's validator
    assert np.all(np.diff(pat.astype(np.float32), axis=1) >= 0) and np.abs(pat.astype(np.float32)).max() <= 1.05
    blocks, st = binding.ecco_encode_host(lm, w, binding.SELECT_MSE)
    om.e = lm.tables()[1]
    out = eo.decode(om, blocks).reshape(w.shape).astype(np.float32)
    rel = np.sqrt(((out - w.astype(np.float32)) ** 2).mean() / (w.astype(np.float32) ** 2).mean())
    assert rel < 0.15                                   # same class as the oracle's own calibration (~0.10)
    assert st.clipped_values / (st.n_groups * 128) < 0.02
    # the oracle's encoder agrees with the library's on the library's metadata too
    want, _ = eo.encode(om, w, eo.SELECT_MSE)
    assert np.array_equal(blocks, want)
    # sub-sampled calibration and the KV rule run and validate
    km = binding.ecco_calibrate_host(synth.kv_cache(1, 4, 512, 2003, 3003), S=16, seed=2, select=binding.SELECT_MINMAX,
                                     max_groups=1024)
    assert eo.meta_check(oracle_meta_from_lib(eo, km)) == 0 and km.tables()[0] == 16
    with pytest.raises(binding.EccoError):
        binding.ecco_calibrate_host(cal[:1, :128 * 8].copy(), S=64)   # fewer groups than patterns


def test_device_image_tables_decode_like_the_oracle(binding, eo, cfg1_small):
    """The prebuilt lookup tables, read on the CPU: walking a block with them gives the oracle's
    symbols and end position (checks table layout and bit order without a GPU)."""
    ometa = cfg1_small["meta"]
    lm = lib_meta_from_oracle(binding, ometa)
    img = binding.ecco_meta_serialize_device(lm)
    assert img.size == binding.ecco_meta_device_bytes(lm) == 84160 + 65536 + 5120
    hdr = img[:64].view(np.uint32)
    assert hdr[0] == 0x4F434345 and hdr[2] == 64 and hdr[3] == 4 and hdr[4:5].view(np.int32)[0] == ometa.e
    assert img[20:24].view(np.float32)[0] == 2.0 ** ometa.e
    pat = img[64:64 + 2048].view(np.float16).reshape(64, 16)
    assert np.array_equal(pat[:, :15].view(np.uint16), ometa.patterns().view(np.uint16)) and np.all(pat[:, 15] == 0)
    kpl = img[64 + 2048:64 + 2048 + 8192].view(np.uint16)
    syml = img[64 + 2048 + 8192:64 + 2048 + 8192 + 65536].reshape(256, 256)
    enc = img[75840:75840 + 8192].view(np.uint16).reshape(64, 4, 16)
    assert np.array_equal(enc >> 8, ometa.cb_lengths())                  # encoder table: lengths per (pattern, codebook, symbol)
    assert np.array_equal(img[84032:84160].view(np.uint16) >> 12, ometa.kp_lengths())
    assert np.all((syml >> 4) >= 2) and np.all((syml >> 4) <= 8)
    for g in range(0, 2048, 41):
        blk = cfg1_small["blocks"][g]
        _, sym, info = eo.decode_block(ometa, blk)
        bits = int.from_bytes(blk.tobytes(), "little")
        e = int(kpl[(bits >> 10) & 0xFFF])
        assert e & 0xFF == info.kp
        pos = 10 + (e >> 8)
        cb = info.kp * 4 + info.hf
        lut = syml[cb]
        rot = ((cb * 11 + (cb >> 3)) & 31) << 2          # per-codebook index rotation of the image
        n = 0
        while n < 128:
            t = int(lut[((bits >> pos) & 0xFF) ^ rot])
            if pos + (t >> 4) > 512:
                break
            assert (t & 15) == sym[n]
            pos += t >> 4
            n += 1
        assert n == info.n_fit and pos == info.end_bit


def test_device_image_rank_tables_and_arithmetic_constants(binding, eo, cfg1_small):
    """The mixed decoder's tables against the oracle's canonical codes: for every codebook and every 8-bit
    window, the rank table has the oracle's codeword length and a rank that is a bijection of the symbol,
    and the arithmetic route (threshold compare, codeword + delta) lands on the same length and rank."""
    ometa = cfg1_small["meta"]
    lm = lib_meta_from_oracle(binding, ometa)
    img = binding.ecco_meta_serialize_device(lm)
    syml = img[64 + 2048 + 8192:64 + 2048 + 8192 + 65536].reshape(256, 256)
    rankl = img[84160:84160 + 65536].reshape(256, 256)
    ar = img[84160 + 65536:].view(np.uint32).reshape(5, 256)
    lengths = ometa.cb_lengths()                                   # [pattern][codebook][symbol]
    spread = 1 | 1 << 10 | 1 << 20
    guard = 0x100 | 0x100 << 10 | 0x100 << 20
    for cb in range(ometa.S * 4):
        lens = [int(x) for x in lengths[cb // 4, cb % 4]]
        codes, kraft = eo.canonical_codes(lens, 8)
        assert kraft == 256
        rot = ((cb * 11 + (cb >> 3)) & 31) << 2
        c1, c2, d, rlo, rhi = (int(ar[i, cb]) for i in range(5))
        rank_of = rlo | rhi << 32
        assert sorted((rank_of >> 4 * s) & 15 for s in range(16)) == list(range(16))
        delta = {L: (d >> 4 * (L - 2)) & 15 for L in range(2, 8)}
        delta[8] = 0
        for s in range(16):                                        # every window that starts with the codeword of s
            L, code = lens[s], int(codes[s])
            for rest in range(1 << (8 - L)):
                b = code << (8 - L) | rest                         # first stream bit on top
                i = int(f"{b:08b}"[::-1], 2)                       # the same window, first stream bit in bit 0
                assert int(syml[cb, i ^ rot]) == (L << 4 | s)
                assert int(rankl[cb, i ^ rot]) == (L << 4 | ((rank_of >> 4 * s) & 15))
                m = ((b * spread + c1) & 0xFFFFFFFF & (guard | 0xC0000000)) | ((b * 2 * spread + c2) & 0xFFFFFFFF & (2 * guard))
                assert bin(m).count("1") == L
                assert ((b >> (8 - L)) + delta[L]) & 15 == (rank_of >> 4 * s) & 15
    # rows of unused patterns decode as sixteen 4-bit codewords in every table
    for cb in range(ometa.S * 4, 256):
        assert np.all(rankl[cb] >> 4 == 4) and np.all(syml[cb] >> 4 == 4)


def _complete_length_multisets():
    """Every way to give 16 symbols code lengths in 2..8 with Kraft sum exactly 1, as counts per length."""
    out = []

    def rec(L, left, kraft, counts):
        if L == 9:
            if left == 0 and kraft == 0:
                out.append(tuple(counts))
            return
        worth = 1 << (8 - L)
        for c in range(min(left, kraft // worth) + 1):
            rec(L + 1, left - c, kraft - c * worth, counts + [c])

    rec(2, 16, 256, [])
    return out


def test_rank_tables_and_arithmetic_constants_for_every_code_shape(binding, eo):
    """The mixed decoder's tables over EVERY admissible shape of a 2..8-bit code on 16 symbols (all multisets of
    lengths with Kraft sum 1, lengths dealt to the symbols at random): for all 256 window bytes the arithmetic
    route gives the canonical code's length, and codeword + delta is a bijection onto the ranks that agrees with
    the rank table.  The expected lengths and codewords come from the oracle's canonical-code routine."""
    shapes = _complete_length_multisets()
    assert len(shapes) > 200 and (0, 0, 16, 0, 0, 0, 0) in shapes and (3, 0, 3, 0, 2, 0, 8) in shapes
    rng = np.random.Generator(np.random.PCG64(2024))
    spread = 1 | 1 << 10 | 1 << 20
    guard = 0x100 | 0x100 << 10 | 0x100 << 20
    per_meta = 64 * 4
    kp_len = eo.huffman_limited(np.ones(64), 12)
    pat = np.sort(rng.uniform(-1, 1, (64, 15)), axis=1).astype(np.float16)
    for base in range(0, len(shapes), per_meta):
        chunk = shapes[base:base + per_meta]
        cb = np.full((64, 4, 16), 4, dtype=np.uint8)
        for i, counts in enumerate(chunk):
            lens = np.repeat(np.arange(2, 9), counts)
            cb[i // 4, i % 4] = rng.permutation(lens)
        lm = binding.ecco_meta_create(64, -5, pat, cb, kp_len)
        img = binding.ecco_meta_serialize_device(lm)
        rankl = img[84160:84160 + 65536].reshape(256, 256)
        ar = img[84160 + 65536:].view(np.uint32).reshape(5, 256)
        for i in range(len(chunk)):
            lens = [int(x) for x in cb[i // 4, i % 4]]
            codes, kraft = eo.canonical_codes(lens, 8)
            assert kraft == 256
            rot = ((i * 11 + (i >> 3)) & 31) << 2
            c1, c2, d, rlo, rhi = (int(ar[j, i]) for j in range(5))
            rank_of = rlo | rhi << 32
            assert sorted((rank_of >> 4 * s) & 15 for s in range(16)) == list(range(16))
            delta = {L: (d >> 4 * (L - 2)) & 15 for L in range(2, 8)}
            delta[8] = 0
            expect_len = np.zeros(256, dtype=np.int64)
            expect_rank = np.zeros(256, dtype=np.int64)
            for s in range(16):
                L, code = lens[s], int(codes[s])
                lo = code << (8 - L)
                expect_len[lo:lo + (1 << (8 - L))] = L
                expect_rank[lo:lo + (1 << (8 - L))] = (rank_of >> 4 * s) & 15
            assert expect_len.min() >= 2                       # the code is complete: every window byte decodes
            for b in range(256):
                m = ((b * spread + c1) & 0xFFFFFFFF & (guard | 0xC0000000)) | ((b * 2 * spread + c2) & 0xFFFFFFFF & (2 * guard))
                L = bin(m).count("1")
                assert L == expect_len[b], (chunk[i], b)
                assert ((b >> (8 - L)) + delta[L]) & 15 == expect_rank[b], (chunk[i], b)
                rev = int(f"{b:08b}"[::-1], 2)
                assert int(rankl[i, rev ^ rot]) == (L << 4 | expect_rank[b])


def test_variable_length_host_encoder_matches_oracle(binding, eo, cfg1_small, kv_small):
    for fx, key, flags in ((cfg1_small, "w", binding.SELECT_MSE), (kv_small, "k", binding.SELECT_MINMAX | binding.KEEP_EXPONENT)):
        ometa, x = fx["meta"], fx[key]
        lm = lib_meta_from_oracle(binding, ometa)
        stream, index, total = binding.ecco_var_encode_host(lm, x, flags)
        want_stream, want_off = eo.var_encode(ometa, x, flags & 1)
        n = x.size // 128
        assert total == int(want_off[n]) and stream.size % 16 == 0
        assert np.array_equal(stream[: want_stream.size], want_stream) and not stream[want_stream.size:].any()
        idx64 = index[: 8 * (1 + (n + 4095) // 4096)].view(np.uint64)
        off32 = index[8 * (1 + (n + 4095) // 4096): 8 * (1 + (n + 4095) // 4096) + 4 * n].view(np.uint32)
        assert idx64[0] == total
        starts = idx64[1:][np.arange(n) >> 12] + off32
        assert np.array_equal(starts, want_off[:n])
        # no clipping: positions the fixed block had to drop (decoded as +0 there) carry their mapped value here
        out = eo.var_decode(ometa, want_stream, want_off)
        groups = x.reshape(-1, 128)
        seen = 0
        for g in range(0, n, 7):
            _, _, info = eo.decode_block(ometa, fx["blocks"][g])
            if info.n_fit < 128:
                q = eo.quantize_group(ometa, groups[g], flags & 1)
                tail = out[g, info.n_fit:].astype(np.float32)
                pat = ometa.patterns()[q["kp"]].astype(np.float32)
                s = np.float32(abs(eo.e4m3_to_f32(q["qs"]))) * np.float32(2.0 ** ometa.e)
                want = np.array([pat[sy] * s if sy < 15 else eo.e4m3_to_f32(q["qs"]) * 2.0 ** ometa.e for sy in q["sym"][info.n_fit:]])
                assert np.array_equal(tail, want.astype(np.float16).astype(np.float32))
                seen += 1
        assert seen > 3
