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
    # several matrices in one call: the same checks per item, at most eight items, all before any CUDA call
    good = (16, 32, 100, 128, 64, 128)
    items = lambda seq: binding.gemv_items(seq)
    assert L.ecco_gemv_batch(items([]), 0, 1, None, 0, None) == binding.ERR_INVALID_ARG
    assert L.ecco_gemv_batch(items([good] * 9), 9, 1, None, 0, None) == binding.ERR_INVALID_ARG
    assert L.ecco_gemv_batch(items([good, (16, 32, 100, 100, 64, 128)]), 2, 1, None, 0, None) == binding.ERR_INVALID_ARG     # k % 128
    assert L.ecco_gemv_batch(items([good, (16, 32 + 4, 100, 128, 64, 128)]), 2, 1, None, 0, None) == binding.ERR_ALIGNMENT   # blocks
    assert L.ecco_gemv_batch(items([good]), 1, 9, None, 0, None) == binding.ERR_INVALID_ARG                                   # batch > 8
    one = binding.ecco_gemv_batch_workspace_bytes([good], 3)
    assert one == binding.ecco_gemv_workspace_bytes(100, 128, 3) > 0
    assert binding.ecco_gemv_batch_workspace_bytes([good, (0, 0, 4096, 4096, 0, 0)], 3) > one
    assert binding.ecco_gemv_batch_workspace_bytes([good] * 9, 1) == 0
    assert binding.ecco_gemv_batch_workspace_bytes([(0, 0, 100, 100, 0, 0)], 1) == 0
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


OFF_PATTERN, OFF_KP, OFF_REC, OFF_ENC_CB, OFF_ENC_KP, OFF_SHAPE = 64, 2112, 10304, 14400, 22592, 22720


def _image_views(img):
    """The sections of a device image (layout: csrc/ecco_format.h), as numpy views."""
    hdr = img[:64].view(np.uint32)
    n_shapes, shape_bytes, pair_bytes, pair_align, off_pair = (int(v) for v in hdr[7:12])
    v = dict(hdr=hdr, n_shapes=n_shapes, pair_bytes=pair_bytes, pair_align=pair_align, off_pair=off_pair)
    assert shape_bytes == n_shapes * 256 and off_pair == (OFF_SHAPE + shape_bytes + 15) // 16 * 16
    assert img.size == hdr[6] == off_pair + pair_bytes
    v["pattern"] = img[OFF_PATTERN:OFF_KP].view(np.float16).reshape(64, 16)
    v["kp"] = img[OFF_KP:OFF_REC].view(np.uint16)
    v["rec"] = img[OFF_REC:OFF_ENC_CB].view(np.uint32).reshape(256, 4)
    v["enc_cb"] = img[OFF_ENC_CB:OFF_ENC_KP].view(np.uint16).reshape(64, 4, 16)
    v["enc_kp"] = img[OFF_ENC_KP:OFF_SHAPE].view(np.uint16)
    v["shape"] = img[OFF_SHAPE:OFF_SHAPE + shape_bytes].reshape(n_shapes, 256)
    v["pair"] = img[off_pair:off_pair + pair_bytes]
    return v


def _rotation(shape):
    """Byte-offset rotation of the tables of a shape (csrc/ecco_format.h: table_rotation)."""
    return ((shape * 11 + (shape >> 3)) & 31) << 2


def _walk_with_image_tables(v, blk):
    """A block decoded the way the kernels do it, in Python: four symbols per step from a window that starts one
    bit early, two pair-table lookups, escapes completed through the shape table, and the one-symbol-per-lookup
    walk with the clip test once a step could cross bit 512.  -> (kp, hf, symbols, end bit or 0)."""
    bits = int.from_bytes(blk.tobytes(), "little")         # stream bit k = bit k of this integer; bits past 511 are zero
    hf = (bits >> 8) & 3
    e = int(v["kp"][(bits >> 10) & 0xFFF])
    kp, pos = e & 0xFF, 10 + (e >> 8)
    rec = v["rec"][kp * 4 + hf]
    shape, width, pair_off = (int(rec[0]) >> 8) & 0xFF, int(rec[0]) >> 16, (int(rec[0]) & 0xFF) << 9
    rank_of = int(rec[2]) | int(rec[3]) << 32
    sym_of_rank = {(rank_of >> 4 * s) & 15: s for s in range(16)}
    assert len(sym_of_rank) == 16
    rot = _rotation(shape)                                 # tables are stored rotated: window i at byte offset (size * i) ^ rot
    blut = v["shape"][shape][np.arange(256) ^ rot]
    plut = v["pair"][pair_off:pair_off + (2 << width)].view(np.uint16) if width else None
    mask = ((1 << width) - 1) << 1
    ranks, alive = [], True

    def entry(off):                                        # signed 16-bit pair-table entry at byte offset off
        x = int(plut[(off ^ rot) >> 1])
        return x - 65536 if x & 0x8000 else x

    def resolve(e, p):
        b = int(blut[(bits >> (p + (e & 15))) & 0xFF])
        return (e & 0x078F) + (b >> 4) + ((b & 15) << 11)

    for step in range(32):
        single = plut is None
        if not single:
            win = (bits >> (pos - 1)) & 0xFFFFFFFF
            e0 = entry(win & mask)
            if e0 < 0:
                e0 = resolve(e0, pos)
            e1 = entry((win >> (e0 & 31)) & mask)
            if e1 < 0:
                e1 = resolve(e1, pos + (e0 & 31))
            acc = (e0 + e1) & 0x7F
            if pos + acc > 512:
                single = True
            else:
                ranks += [(e0 >> 7) & 15, (e0 >> 11) & 15, (e1 >> 7) & 15, (e1 >> 11) & 15]
                pos += acc
        if single:
            for _ in range(4):
                t = int(blut[(bits >> pos) & 0xFF]) if pos < 520 else int(blut[0])
                if alive and pos + (t >> 4) <= 512:
                    ranks.append(t & 15)
                else:
                    alive = False
                pos += t >> 4
    return kp, hf, [sym_of_rank[r] for r in ranks], pos if alive else 0


def test_device_image_tables_decode_like_the_oracle(binding, eo, cfg1_small, kv_small):
    """The prebuilt lookup tables, read on the CPU: walking a block with them, the way the kernels do, gives the
    oracle's symbols and end position (checks table layout, bit order, escapes and the clip rule without a GPU)."""
    for fx in (cfg1_small, kv_small):
        ometa = fx["meta"]
        lm = lib_meta_from_oracle(binding, ometa)
        img = binding.ecco_meta_serialize_device(lm)
        assert img.size == binding.ecco_meta_device_bytes(lm)
        v = _image_views(img)
        hdr = v["hdr"]
        assert hdr[0] == 0x4F434345 and hdr[1] == 4 and hdr[2] == 64 and hdr[3] == 4 and hdr[4:5].view(np.int32)[0] == ometa.e
        assert img[20:24].view(np.float32)[0] == 2.0 ** ometa.e
        assert np.array_equal(v["pattern"][:, :15].view(np.uint16), ometa.patterns().view(np.uint16)) and np.all(v["pattern"][:, 15] == 0)
        assert np.array_equal(v["enc_cb"] >> 8, ometa.cb_lengths())      # encoder table: lengths per (pattern, codebook, symbol)
        assert np.array_equal(v["enc_kp"] >> 12, ometa.kp_lengths())
        assert v["pair_bytes"] > 0 and v["n_shapes"] < 64
        assert np.all((v["shape"] >> 4) >= 2) and np.all((v["shape"] >> 4) <= 8)
        escapes = 0
        for g in range(0, 2048, 13):
            blk = fx["blocks"][g]
            _, sym, info = eo.decode_block(ometa, blk)
            kp, hf, got, end = _walk_with_image_tables(v, blk)
            assert (kp, hf) == (info.kp, info.hf)
            assert len(got) == info.n_fit and got == [int(x) for x in sym[:info.n_fit]]
            assert end == (info.end_bit if info.n_fit == 128 else 0)
        # random blocks too: whatever the header bits select must decode like the oracle says
        rb = np.random.Generator(np.random.PCG64(4)).integers(0, 256, size=(150, 64), dtype=np.uint8)
        for blk in rb:
            _, sym, info = eo.decode_block(ometa, blk)
            kp, hf, got, end = _walk_with_image_tables(v, blk)
            assert (kp, hf) == (info.kp, info.hf) and got == [int(x) for x in sym[:info.n_fit]]


def test_device_image_shape_and_pair_tables_against_canonical_codes(binding, eo, cfg1_small):
    """Every codebook's record, shape table and pair table against the oracle's canonical code: ranks are a
    bijection of the symbols in (length, id) order; for every 8-bit window the shape table has the codeword's
    length and rank; for every W-bit window the pair table has both symbols when the second codeword ends inside
    the window and an escape with the first symbol otherwise; tables are aligned to their size, widest first."""
    ometa = cfg1_small["meta"]
    lm = lib_meta_from_oracle(binding, ometa)
    v = _image_views(binding.ecco_meta_serialize_device(lm))
    lengths = ometa.cb_lengths()
    widths_by_offset = {}
    for cb in range(ometa.S * 4):
        lens = [int(x) for x in lengths[cb // 4, cb % 4]]
        codes, kraft = eo.canonical_codes(lens, 8)
        assert kraft == 256
        rec = v["rec"][cb]
        shape, width, pair_off = (int(rec[0]) >> 8) & 0xFF, int(rec[0]) >> 16, (int(rec[0]) & 0xFF) << 9
        rank_of = int(rec[2]) | int(rec[3]) << 32
        order = sorted(range(16), key=lambda s: (lens[s], s))
        assert [(rank_of >> 4 * s) & 15 for s in order] == list(range(16))
        want_len, want_rank = np.zeros(256, np.int64), np.zeros(256, np.int64)
        for s in range(16):
            L, code = lens[s], int(codes[s])
            for rest in range(1 << (8 - L)):
                i = int(f"{code << (8 - L) | rest:08b}"[::-1], 2)     # the window with the first stream bit in bit 0
                want_len[i], want_rank[i] = L, (rank_of >> 4 * s) & 15
        rot = _rotation(shape)
        table = v["shape"][shape][np.arange(256) ^ rot]
        assert np.array_equal(table >> 4, want_len) and np.array_equal(table & 15, want_rank)
        assert 8 <= width <= 12 and pair_off % (2 << width) == 0
        widths_by_offset[pair_off] = width
        idx = np.arange(1 << width)
        pt = v["pair"][pair_off:pair_off + (2 << width)].view(np.uint16).astype(np.int64)[idx ^ (rot >> 1)]
        l0, r0 = want_len[idx & 255], want_rank[idx & 255]
        rest = idx >> l0
        l1, r1 = want_len[rest & 255], want_rank[rest & 255]
        fits = l0 + l1 <= width
        assert np.array_equal(pt[fits], (l0 + l1 + (r0 << 7) + (r1 << 11))[fits])
        assert np.array_equal(pt[~fits], (l0 + (r0 << 7) + 0x8000)[~fits])
        assert fits.mean() > 0.5
    offs = sorted(widths_by_offset)
    assert offs[0] == 0 and all(widths_by_offset[a] >= widths_by_offset[b] for a, b in zip(offs, offs[1:]))
    assert v["pair_align"] == 2 << widths_by_offset[0]
    assert sum(2 << w for w in widths_by_offset.values()) == v["pair_bytes"] <= 80 * 1024


def test_device_image_tables_depend_on_the_metadata_only(binding, eo, cfg1_small):
    """Tensors encoded with the same patterns and codebooks must get the same decode tables and the same table hash
    (ecco_decompress_batch decodes consecutive tensors of equal hash as one run), whatever was encoded with the
    metadata before the image was made and whatever exponent the tensor got."""
    fresh = lib_meta_from_oracle(binding, cfg1_small["meta"])
    used = lib_meta_from_oracle(binding, cfg1_small["meta"])
    skewed = (cfg1_small["w"].astype(np.float32) ** 3 * 50.0).astype(np.float16)     # other codebook choices, other exponent
    binding.ecco_encode_host(used, skewed, binding.SELECT_MSE)
    assert used.tables()[1] != fresh.tables()[1]
    a, b = binding.ecco_meta_serialize_device(fresh), binding.ecco_meta_serialize_device(used)
    va, vb = _image_views(a), _image_views(b)
    assert a.size == b.size and np.array_equal(va["hdr"][12:14], vb["hdr"][12:14])
    assert np.array_equal(a[OFF_PATTERN:], b[OFF_PATTERN:])          # everything but the header (exponent, T)
    other = lib_meta_from_oracle(binding, cfg1_small["meta"])
    S, e, pat, cb, kp = other.tables()
    cb = cb.copy()
    cb[0, 0] = cb[0, 0][::-1]                                         # same lengths on other symbols: another code
    changed = binding.ecco_meta_create(S, e, pat, cb, kp)
    vc = _image_views(binding.ecco_meta_serialize_device(changed))
    assert not np.array_equal(va["hdr"][12:14], vc["hdr"][12:14])


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


def test_device_image_for_every_code_shape(binding, eo):
    """EVERY admissible shape of a 2..8-bit code on 16 symbols (all multisets of lengths with Kraft sum 1, lengths
    dealt to the symbols at random), 128 at a time (so that they fit pair tables of at least eight bits) and all
    255 in one image (which then has no pair tables): blocks of random bits walked with the image's tables decode
    like the oracle's."""
    shapes = _complete_length_multisets()
    assert len(shapes) == 255 and (0, 0, 16, 0, 0, 0, 0) in shapes and (3, 0, 3, 0, 2, 0, 8) in shapes
    rng = np.random.Generator(np.random.PCG64(2024))
    kp_len = eo.huffman_limited(np.ones(64), 12)
    pat = np.sort(rng.uniform(-1, 1, (64, 15)), axis=1).astype(np.float16)
    for chunk, want_pairs in ((shapes[:128], True), (shapes[127:], True), (shapes + shapes[:1], False)):
        cb = np.zeros((64, 4, 16), dtype=np.uint8)
        for i in range(256):
            cb[i // 4, i % 4] = rng.permutation(np.repeat(np.arange(2, 9), chunk[i % len(chunk)]))
        lm = binding.ecco_meta_create(64, -5, pat, cb, kp_len)
        v = _image_views(binding.ecco_meta_serialize_device(lm))
        assert v["n_shapes"] == min(len(chunk), 255) and (v["pair_bytes"] > 0) == want_pairs
        om = oracle_meta_from_lib(eo, lm)
        rb = rng.integers(0, 256, size=(300, 64), dtype=np.uint8)
        for blk in rb:
            _, sym, info = eo.decode_block(om, blk)
            kp, hf, got, end = _walk_with_image_tables(v, blk)
            assert (kp, hf) == (info.kp, info.hf) and got == [int(x) for x in sym[:info.n_fit]]
            assert end == (info.end_bit if info.n_fit == 128 else 0)


def _oracle_encode_threads(eo, om, x, select):
    """eo.encode over disjoint ranges of groups from one Python thread per core (ctypes drops the GIL)."""
    from concurrent.futures import ThreadPoolExecutor

    g = x.reshape(-1, 128)
    n = g.shape[0]
    threads = max(1, min(len(os.sched_getaffinity(0)), n // 256))
    bounds = [n * i // threads for i in range(threads + 1)]
    out = np.zeros((n, 64), dtype=np.uint8)

    def work(i):
        lo, hi = bounds[i], bounds[i + 1]
        if hi > lo:
            out[lo:hi] = eo.encode(om, g[lo:hi], select)[0]

    with ThreadPoolExecutor(threads) as ex:
        list(ex.map(work, range(threads)))
    return out


def test_host_encoder_matches_oracle_on_samples_of_the_large_configurations(binding, eo, synth):
    """65 536 groups with the shapes, seeds and distributions of each larger configuration (the first rows of the
    7B- and 70B-shaped matrices, the first tokens of the two KV caches), encoded with the library's own calibrated
    metadata: the threaded host encoder and the plain oracle must write the same bytes."""
    from paper_2505_06901_b200 import workloads as W

    n = 1 << 16
    cases = [("cfg2 gate", W.calibrate_weights(2, 0.02, True), synth.weight_matrix(n * 128 // 4096, 4096, 1002 * 16 + 4), binding.SELECT_MSE, 0),
             ("cfg2 down", W.calibrate_weights(2, 0.02, True), synth.weight_matrix(n * 128 // 11008 // 1 + 1, 11008, 1002 * 16 + 6)[:762], binding.SELECT_MSE, 0),
             ("cfg4 gate", W.calibrate_weights(4, 0.01, False), synth.weight_matrix(n * 128 // 8192, 8192, 1004 * 16, sigma=0.01, row_scale=False), binding.SELECT_MSE, 0),
             ("cfg3 K", W.calibrate_kv(3, 32), synth.kv_cache(1, 32, n // 32, 1003 * 16, 3003), binding.SELECT_MINMAX, binding.KEEP_EXPONENT),
             ("cfg5 K", W.calibrate_kv(5, 8), synth.kv_cache(1, 8, n // 8, 1005 * 16, 3005), binding.SELECT_MINMAX, binding.KEEP_EXPONENT)]
    for name, base, x, select, keep in cases:
        S, e, pat, cb, kp = base.tables()
        lm = binding.ecco_meta_create(S, e, pat, cb, kp)
        blocks, st = binding.ecco_encode_host(lm, x, select | keep)
        om = oracle_meta_from_lib(eo, lm)                   # carries the exponent the library fitted (weights) or kept (KV)
        want = _oracle_encode_threads(eo, om, x, select)
        bad = np.nonzero((blocks != want).any(axis=1))[0]
        assert bad.size == 0, (name, bad.size, bad[:5])
        assert blocks.shape[0] >= 60000 and st.n_groups == blocks.shape[0]


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
