"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle.

Decompression must match the oracle bit for bit.  The fused calls accumulate in fp32 and are held
to |y - y_ref| <= 1e-3 * sum_i |w_i x_i| per output (y_ref = the oracle's fp64 sum over the
decompressed fp16 values); the plain relative error is also checked where |y_ref| is not small.
"""
import numpy as np
import pytest

from helpers import lib_meta_from_oracle, oracle_meta_from_lib, record_fused

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 1e-3


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2505_06901_b200 import binding

    binding.lib()
    return binding


@pytest.fixture(scope="module")
def W():
    from paper_2505_06901_b200 import workloads

    return workloads


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def gpu_decompress(B, lmeta, blocks):
    n = blocks.shape[0]
    d_meta = B.meta_to_device(lmeta)
    d_blocks = dev(blocks)
    d_out = torch.empty(max(n, 1) * 128, dtype=torch.float16, device="cuda")
    before = B.ecco_kernel_launch_count()
    B.ecco_decompress(d_meta, d_blocks, n, d_out)
    torch.cuda.synchronize()
    assert B.ecco_device_status() == 0
    assert B.ecco_kernel_launch_count() == before + (1 if n else 0)
    return d_out[: n * 128].cpu().numpy().reshape(n, 128)


def assert_bit_exact(got, want):
    g, w = got.view(np.uint16), want.view(np.uint16)
    bad = np.nonzero((g != w).any(axis=1))[0]
    assert bad.size == 0, f"{bad.size} of {g.shape[0]} groups differ; first group {bad[:3]}, positions {np.nonzero(g[bad[0]] != w[bad[0]])[0][:8]}"


def gpu_gemv(B, lmeta, blocks, n_out, k, x, batch):
    d_meta, d_blocks, d_x = B.meta_to_device(lmeta), dev(blocks), dev(x)
    d_y = torch.full((batch, n_out), float("nan"), dtype=torch.float32, device="cuda")
    wsb = B.ecco_gemv_workspace_bytes(n_out, k, batch)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    ws.fill_(0xCD)                                   # stale contents must not matter
    B.ecco_gemv(d_meta, d_blocks, n_out, k, d_x, batch, d_y, ws, wsb)
    torch.cuda.synchronize()
    assert B.ecco_device_status() == 0
    return d_y.cpu().numpy().astype(np.float64), (d_meta, d_blocks, d_x, ws, wsb)


def check_fused(got, ref, refabs, label="fused"):
    """|y - ref| <= 1e-3 sum|w x| for every output, and the plain relative error <= 1e-3 wherever the reference is
    not small against its row (|ref| >= 0.1 rms); the largest values seen are kept for the session summary."""
    err = np.abs(got - ref)
    scaled = float((err / (refabs + 1e-30)).max())
    big = np.abs(ref) >= 0.1 * np.sqrt((ref ** 2).mean())
    plain = float((err[big] / np.abs(ref[big])).max()) if big.any() else 0.0
    record_fused(label, scaled, plain)
    assert np.all(err <= TOL * refabs + 1e-30), (label, scaled)
    assert plain <= TOL, (label, plain)


# ------------------------------------------------------------------ decompress
@pytest.mark.parametrize("n_groups", [0, 1, 31, 32, 33, 1000, 1023, 1025, 2048])
def test_decompress_matches_oracle_ragged_sizes(B, eo, cfg1_small, n_groups):
    lm = lib_meta_from_oracle(B, cfg1_small["meta"])
    blocks = cfg1_small["blocks"][:n_groups]
    got = gpu_decompress(B, lm, blocks)
    if n_groups:
        assert_bit_exact(got, eo.decode(cfg1_small["meta"], blocks))


def test_decompress_config1_full_with_library_metadata(B, eo, W):
    t = W.config1(keep_source=True)
    assert t.n_groups == 8192
    om = oracle_meta_from_lib(eo, t.meta)
    want_blocks, _ = eo.encode(om, t.source, eo.SELECT_MSE)
    assert np.array_equal(t.blocks, want_blocks)             # CPU encode: library == oracle
    got = gpu_decompress(B, t.meta, t.blocks)
    assert_bit_exact(got, eo.decode(om, t.blocks))
    src = t.source.astype(np.float32).reshape(-1, 128)
    rel = np.sqrt(((got.astype(np.float32) - src) ** 2).mean() / (src ** 2).mean())
    assert rel < 0.15


def test_decompress_kv_blocks_and_s16(B, eo, kv_small, synth):
    lm = lib_meta_from_oracle(B, kv_small["meta"])
    assert_bit_exact(gpu_decompress(B, lm, kv_small["blocks"]), eo.decode(kv_small["meta"], kv_small["blocks"]))
    # the paper's hardware compressor uses 16 patterns for the KV cache
    cal = synth.kv_cache(1, 4, 512, 2003, 3003)
    m16 = eo.calibrate(cal, S=16, H=4, seed=3, select=eo.SELECT_MINMAX)
    blocks, _ = eo.encode(m16, kv_small["k"], eo.SELECT_MINMAX)
    assert_bit_exact(gpu_decompress(B, lib_meta_from_oracle(B, m16), blocks), eo.decode(m16, blocks))


def test_decompress_is_total_on_garbage_and_edge_blocks(B, eo, cfg1_small, synth):
    meta = cfg1_small["meta"]
    lm = lib_meta_from_oracle(B, meta)
    rb = synth.random_blocks(4096, 99)
    assert_bit_exact(gpu_decompress(B, lm, rb), eo.decode(meta, rb))
    edge = np.stack([np.full(64, v, dtype=np.uint8) for v in (0x00, 0xFF, 0xAA, 0x55, 0x7F, 0x80)] * 8)
    assert_bit_exact(gpu_decompress(B, lm, edge), eo.decode(meta, edge))


def make_meta(eo, lens_fn, S=4, e=-5, seed=0):
    rng = np.random.Generator(np.random.PCG64(seed))
    m = eo.Meta()
    m.S, m.H, m.e = S, 4, e
    kl = eo.huffman_limited(np.ones(S), 12)
    for k in range(S):
        m.kp_len[k] = int(kl[k])
        pat = np.sort(rng.uniform(-1, 1, 15))
        for j in range(15):
            m.pattern[k][j] = int(np.float16(pat[j]).view(np.uint16))
        for h in range(4):
            ln = lens_fn(k, h, rng)
            for s in range(16):
                m.cb_len[k][h][s] = int(ln[s])
    assert eo.meta_check(m) == 0
    return m


def skew_lens(k, h, rng):
    """The most skewed admissible code (Kraft: 3/4 + 3/16 + 2/64 + 8/256 = 1).  Codebook 0 gives the
    2-bit codes to the middle centroids, where the values cluster (short streams, up to 16 pads); the
    other codebooks are random permutations (long streams, heavy clipping)."""
    lens = np.array([2, 2, 2, 4, 4, 4, 6, 6, 8, 8, 8, 8, 8, 8, 8, 8])
    out = np.zeros(16, dtype=np.int64)
    if h == 0:
        out[[7, 6, 8, 5, 9, 4, 10, 3, 11, 2, 12, 1, 13, 0, 14, 15]] = lens
    else:
        out[rng.permutation(16)] = lens
    return list(out)


def test_decompress_adversarial_codebooks(B, eo):
    """All-4-bit codes (10 + ID_KP + 128 x 4 > 512 bits: every group clips), the most skewed admissible
    code (2-bit symbols next to 8-bit ones: heavy clipping and up to 16 pads), long ID_KP codes,
    extreme exponents."""
    rng = np.random.Generator(np.random.PCG64(11))
    flat = make_meta(eo, lambda k, h, r: [4] * 16)
    skew = make_meta(eo, skew_lens, seed=3)
    for meta in (flat, skew):
        x = (rng.standard_t(3, size=(512, 128)) * 0.05).astype(np.float16)
        blocks, st = eo.encode(meta, x, eo.SELECT_MSE)
        got = gpu_decompress(B, lib_meta_from_oracle(B, meta), blocks)
        assert_bit_exact(got, eo.decode(meta, blocks))
        assert st.clipped_groups == st.n_groups if meta is flat else (st.padded_groups > 0 and st.clipped_groups > 0)
    # symbols forced to the longest codes -> every group clips; to the shortest -> 16 pads
    m = skew
    x = np.zeros((64, 128), dtype=np.float16)
    x[:, 0] = 1.0
    blocks, st = eo.encode(m, x, eo.SELECT_MSE)
    assert_bit_exact(gpu_decompress(B, lib_meta_from_oracle(B, m), blocks), eo.decode(m, blocks))
    for e in (-32, 16):
        m2 = make_meta(eo, lambda k, h, r: [4] * 16, e=e, seed=5)
        rb = np.random.Generator(np.random.PCG64(e + 100)).integers(0, 256, size=(256, 64), dtype=np.uint8)
        assert_bit_exact(gpu_decompress(B, lib_meta_from_oracle(B, m2), rb), eo.decode(m2, rb))
    # S = 64 with a deliberately unbalanced ID_KP code (lengths up to 12 bits)
    m3 = make_meta(eo, lambda k, h, r: [4] * 16, S=64, seed=7)
    kl = eo.huffman_limited(1.7 ** np.arange(64), 12)
    assert kl.max() == 12
    for k in range(64):
        m3.kp_len[k] = int(kl[k])
    assert eo.meta_check(m3) == 0
    rb = np.random.Generator(np.random.PCG64(8)).integers(0, 256, size=(2048, 64), dtype=np.uint8)
    assert_bit_exact(gpu_decompress(B, lib_meta_from_oracle(B, m3), rb), eo.decode(m3, rb))


def test_decompress_batch_matches_oracle_per_item(B, eo, cfg1_small, kv_small, synth):
    """One call over tensors with different metadata and sizes: every item as ecco_decompress alone would give it.
    Covers more than eight items (two launches), an empty item, tiny items (the small-tensor kernel in the middle
    of the batch) and a ragged tail; the items are independent of each other, as the call requires."""
    wm, km = cfg1_small["meta"], kv_small["meta"]
    d_wm, d_km = B.meta_to_device(lib_meta_from_oracle(B, wm)), B.meta_to_device(lib_meta_from_oracle(B, km))
    wb, kb = cfg1_small["blocks"], kv_small["blocks"]
    rb = synth.random_blocks(700, 5)
    plan = [(wm, d_wm, np.tile(wb, (3, 1))), (km, d_km, kb), (wm, d_wm, wb[:0]), (wm, d_wm, wb[:7]), (km, d_km, kb[:33]),
            (wm, d_wm, rb), (km, d_km, np.tile(kb, (2, 1))[:4095]), (wm, d_wm, wb[:1]), (km, d_km, kb[100:1124]),
            (wm, d_wm, wb[5:1030]), (km, d_km, kb[:31])]
    items, outs = [], []
    for meta, d_meta, blocks in plan:
        n = blocks.shape[0]
        d_b = dev(blocks) if n else torch.empty((1, 64), dtype=torch.uint8, device="cuda")
        d_o = torch.full((max(n, 1) * 128,), float("nan"), dtype=torch.float16, device="cuda")
        items.append((d_meta, d_b, n, d_o))
        outs.append(d_o)
    B.ecco_decompress_batch(items)
    torch.cuda.synchronize()
    assert B.ecco_device_status() == 0
    for (meta, _, blocks), d_o in zip(plan, outs):
        n = blocks.shape[0]
        if n:
            assert_bit_exact(d_o[: n * 128].cpu().numpy().reshape(n, 128), eo.decode(meta, blocks))
    B.ecco_decompress_batch([])                                                   # nothing to do is not an error
    # one bad item stops the whole call before anything runs
    canary = torch.full((2048 * 128,), 7.0, dtype=torch.float16, device="cuda")
    with pytest.raises(B.EccoError) as ei:
        B.ecco_decompress_batch([(d_wm, dev(wb), 2048, canary), (d_wm, dev(wb).data_ptr() + 8, 2048, canary)])
    assert ei.value.code == B.ERR_ALIGNMENT
    torch.cuda.synchronize()
    assert bool((canary == 7.0).all())


def test_decompress_every_code_shape_on_random_streams(B, eo, synth):
    """All 255 admissible shapes of a 2..8-bit code on 16 symbols (every multiset of lengths with Kraft sum 1,
    dealt to the symbols at random), one per codebook, decoded from random bit streams: whatever a block's header
    bits select, table lookups and arithmetic decoding must give the oracle's values, clips and outliers."""
    shapes = []

    def rec(L, left, kraft, counts):
        if L == 9:
            if left == 0 and kraft == 0:
                shapes.append(tuple(counts))
            return
        worth = 1 << (8 - L)
        for c in range(min(left, kraft // worth) + 1):
            rec(L + 1, left - c, kraft - c * worth, counts + [c])

    rec(2, 16, 256, [])
    assert len(shapes) == 255
    rng = np.random.Generator(np.random.PCG64(99))
    m = eo.Meta()
    m.S, m.H, m.e = 64, 4, -3
    kl = eo.huffman_limited(np.ones(64), 12)
    for k in range(64):
        m.kp_len[k] = int(kl[k])
        pat = np.sort(rng.uniform(-1, 1, 15))
        for j in range(15):
            m.pattern[k][j] = int(np.float16(pat[j]).view(np.uint16))
        for h in range(4):
            lens = rng.permutation(np.repeat(np.arange(2, 9), shapes[(k * 4 + h) % len(shapes)]))
            for s in range(16):
                m.cb_len[k][h][s] = int(lens[s])
    assert eo.meta_check(m) == 0
    rb = synth.random_blocks(32 * 1024, 31)
    lm = lib_meta_from_oracle(B, m)
    assert_bit_exact(gpu_decompress(B, lm, rb), eo.decode_threads(m, rb, 8))
    # the fused consumers over the same streams (their decoder is all-table; one and eight rows of x take the
    # scalar and the tensor-core kernel)
    for batch in (1, 8):
        x = synth.activations(batch, 2048, 40 + batch)
        got, _ = gpu_gemv(B, lm, rb, 2048, 2048, x, batch)
        ref, refabs = eo.gemv(m, rb, 2048, 2048, x, batch)
        check_fused(got, ref, refabs, f"gemv b{batch} code shapes")


def test_decompress_rejects_bad_arguments_on_device(B, cfg1_small):
    lm = lib_meta_from_oracle(B, cfg1_small["meta"])
    d_meta, d_blocks = B.meta_to_device(lm), dev(cfg1_small["blocks"])
    d_out = torch.empty(2048 * 128 + 8, dtype=torch.float16, device="cuda")
    L = B.lib()
    assert L.ecco_decompress(d_meta.data_ptr(), d_blocks.data_ptr(), 10, d_out.data_ptr() + 2, None) == B.ERR_ALIGNMENT
    assert L.ecco_decompress(d_meta.data_ptr(), d_blocks.data_ptr() + 8, 10, d_out.data_ptr(), None) == B.ERR_ALIGNMENT
    assert L.ecco_decompress(None, d_blocks.data_ptr(), 10, d_out.data_ptr(), None) == B.ERR_INVALID_ARG
    # a side stream works like the current one
    s = torch.cuda.Stream()
    B.ecco_decompress(d_meta, d_blocks, 2048, d_out, stream=s)
    s.synchronize()
    assert B.ecco_device_status() == 0


def test_bounded_wait_gives_up_and_reports(B, eo, cfg1_small):
    """The device-side wait on the table copy is bounded: when it runs out the kernel records
    ECCO_ERR_DEVICE_TIMEOUT and returns, ecco_device_status reports it once, and the context stays usable."""
    assert B.ecco_device_status() == 0
    B.ecco_test_wait_timeout()
    assert B.ecco_device_status() == B.ERR_DEVICE_TIMEOUT
    assert B.ecco_device_status() == 0                      # reading clears it
    lm = lib_meta_from_oracle(B, cfg1_small["meta"])
    assert_bit_exact(gpu_decompress(B, lm, cfg1_small["blocks"][:100]), eo.decode(cfg1_small["meta"], cfg1_small["blocks"][:100]))


# ------------------------------------------------------------------ fused GEMV
@pytest.mark.parametrize("n_out,k,batch", [(256, 1024, 1), (256, 1024, 3), (256, 1024, 8), (100, 1024, 2), (513, 512, 5),
                                           (2048, 128, 1), (64, 4096, 4), (1, 128, 1)])
def test_gemv_matches_oracle(B, eo, cfg1_small, synth, n_out, k, batch):
    meta = cfg1_small["meta"]
    n_groups = n_out * (k // 128)
    reps = -(-n_groups // 2048)
    blocks = np.tile(cfg1_small["blocks"], (reps, 1))[:n_groups]
    x = synth.activations(batch, k, 50 + n_out + batch)
    got, keep = gpu_gemv(B, lib_meta_from_oracle(B, meta), blocks, n_out, k, x, batch)
    ref, refabs = eo.gemv(meta, blocks, n_out, k, x, batch)
    check_fused(got, ref, refabs, f"gemv b{batch}")
    # a second call on the same (now dirty) workspace gives the same bits: fixed summation order
    d_meta, d_blocks, d_x, ws, wsb = keep
    d_y2 = torch.empty((batch, n_out), dtype=torch.float32, device="cuda")
    B.ecco_gemv(d_meta, d_blocks, n_out, k, d_x, batch, d_y2, ws, wsb)
    torch.cuda.synchronize()
    assert np.array_equal(d_y2.cpu().numpy().astype(np.float64), got)


def test_gemv_handles_pads_clips_and_garbage(B, eo, cfg1_small, synth):
    meta = cfg1_small["meta"]
    rb = synth.random_blocks(512 * 4, 123)                 # garbage streams: duplicate pad locations etc.
    x = synth.activations(8, 512, 9)
    got, _ = gpu_gemv(B, lib_meta_from_oracle(B, meta), rb, 512, 512, x, 8)
    ref, refabs = eo.gemv(meta, rb, 512, 512, x, 8)
    check_fused(got, ref, refabs, "gemv b8 garbage")
    skew = make_meta(eo, skew_lens, seed=3)   # many pads, many clips
    w = (np.random.Generator(np.random.PCG64(1)).standard_t(3, size=(256, 256)) * 0.05).astype(np.float16)
    blocks, st = eo.encode(skew, w, eo.SELECT_MSE)
    assert st.padded_values > st.n_groups and st.clipped_groups > 0
    x = synth.activations(2, 256, 10)
    got, _ = gpu_gemv(B, lib_meta_from_oracle(B, skew), blocks, 256, 256, x, 2)
    ref, refabs = eo.gemv(skew, blocks, 256, 256, x, 2)
    check_fused(got, ref, refabs, "gemv b2 skewed code")


@pytest.mark.parametrize("batch", [1, 2, 3, 8])
def test_gemv_batch_gives_every_item_what_gemv_gives(B, eo, cfg1_small, synth, batch):
    """Several matrices in one call (shapes that differ in rows and in k, a ragged row count, a one-row matrix, a shared
    x, per-tensor exponents that differ): every item within the fused tolerance of the oracle and, to rounding, what
    ecco_gemv gives on it alone (the k range of a row is cut into partial sums at other places, so the last bits may
    differ); the same call twice gives the same bits.  Eight items is the most one call takes."""
    meta = cfg1_small["meta"]
    shapes = [(256, 1024), (100, 1024), (513, 512), (64, 4096), (1, 128), (2048, 128), (31, 256), (96, 1024)]
    x_shared = synth.activations(batch, 1024, 77)
    items, keep, want = [], [], []
    for i, (n_out, k) in enumerate(shapes):
        n_groups = n_out * (k // 128)
        blocks = np.roll(np.tile(cfg1_small["blocks"], (-(-n_groups // 2048), 1)), 17 * i, axis=0)[:n_groups]
        om = meta.copy()
        om.e = meta.e + (i % 3) - 1                           # same tables, another exponent
        x = x_shared if k == 1024 else synth.activations(batch, k, 80 + i)
        d_meta, d_blocks, d_x = B.meta_to_device(lib_meta_from_oracle(B, om)), dev(blocks), dev(x)
        d_y = torch.full((batch, n_out), float("nan"), dtype=torch.float32, device="cuda")
        items.append((d_meta, d_blocks, n_out, k, d_x, d_y))
        keep.append((om, blocks, x))
        wsb = B.ecco_gemv_workspace_bytes(n_out, k, batch)
        ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
        d_alone = torch.empty((batch, n_out), dtype=torch.float32, device="cuda")
        B.ecco_gemv(d_meta, d_blocks, n_out, k, d_x, batch, d_alone, ws, wsb)
        want.append(d_alone)
    wsb = B.ecco_gemv_batch_workspace_bytes(items, batch)
    assert wsb > 0
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    first = None
    for _ in range(2):                                        # the second call starts from a used workspace
        B.ecco_gemv_batch(items, batch, ws, wsb)
        torch.cuda.synchronize()
        assert B.ecco_device_status() == 0
        outs = [it[5].cpu().numpy() for it in items]
        if first is not None:
            assert all(np.array_equal(a, b) for a, b in zip(first, outs))
        first = outs
    for (om, blocks, x), it, alone, got in zip(keep, items, want, first):
        ref, refabs = eo.gemv(om, blocks, it[2], it[3], x, batch)
        check_fused(got.astype(np.float64), ref, refabs, f"gemv batch-call b{batch}")
        assert np.all(np.abs(got - alone.cpu().numpy()) <= 1e-5 * refabs + 1e-30)
    # argument errors stop the call before anything runs; too small a workspace is refused
    with pytest.raises(B.EccoError) as ei:
        B.ecco_gemv_batch(items + items[:1], batch, ws, wsb)
    assert ei.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.EccoError) as ei:
        B.ecco_gemv_batch(items, batch, ws, wsb - 256)
    assert ei.value.code == B.ERR_WORKSPACE
    # an item with other decode tables is detected on the device: nothing is written, the status says so
    S, e, pat, cb, kp = lib_meta_from_oracle(B, meta).tables()
    cb = cb.copy()
    cb[0, 0] = cb[0, 0][::-1]
    other = B.meta_to_device(B.ecco_meta_create(S, e, pat, cb, kp))
    canary = torch.full((batch, shapes[0][0]), 7.0, dtype=torch.float32, device="cuda")
    bad = [(items[0][0], items[0][1], items[0][2], items[0][3], items[0][4], canary),
           (other, items[1][1], items[1][2], items[1][3], items[1][4], items[1][5])]
    B.ecco_gemv_batch(bad, batch, ws, wsb)
    torch.cuda.synchronize()
    assert B.ecco_device_status() == B.ERR_INVALID_ARG
    assert B.ecco_device_status() == 0                        # reported once
    assert bool((canary == 7.0).all())
    B.ecco_gemv_batch(items, batch, ws, wsb)                  # and the next good call is unaffected
    torch.cuda.synchronize()
    assert np.array_equal(items[0][5].cpu().numpy(), first[0])


def test_gemv_workspace_errors(B, cfg1_small, synth):
    lm = lib_meta_from_oracle(B, cfg1_small["meta"])
    d_meta, d_blocks = B.meta_to_device(lm), dev(cfg1_small["blocks"])
    d_x, d_y = dev(synth.activations(1, 1024, 1)), torch.empty((1, 256), dtype=torch.float32, device="cuda")
    with pytest.raises(B.EccoError) as ei:
        B.ecco_gemv(d_meta, d_blocks, 256, 1024, d_x, 1, d_y, None, 0)
    assert ei.value.code == B.ERR_WORKSPACE
    small = torch.empty(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.EccoError) as ei:
        B.ecco_gemv(d_meta, d_blocks, 256, 1024, d_x, 1, d_y, small, 64)
    assert ei.value.code == B.ERR_WORKSPACE


# ------------------------------------------------------------------ fused attention scores
@pytest.mark.parametrize("batch,heads,seq,qpk", [(2, 4, 256, 1), (2, 4, 256, 2), (2, 4, 256, 8), (1, 3, 77, 4), (1, 1, 1, 1),
                                                 (2, 2, 513, 3)])
def test_attn_scores_match_oracle(B, eo, kv_small, synth, batch, heads, seq, qpk):
    meta = kv_small["meta"]
    n = batch * heads * seq
    blocks = np.tile(kv_small["blocks"], (-(-n // 2048), 1))[:n]
    q = synth.queries(batch, heads * qpk, 60 + seq)
    scale = 128 ** -0.5
    d_meta, d_blocks, d_q = B.meta_to_device(lib_meta_from_oracle(B, meta)), dev(blocks), dev(q)
    d_s = torch.full((batch, heads * qpk, seq), float("nan"), dtype=torch.float32, device="cuda")
    B.ecco_attn_scores(d_meta, d_blocks, batch, heads, seq, qpk, d_q, scale, d_s)
    torch.cuda.synchronize()
    assert B.ecco_device_status() == 0
    ref, refabs = eo.attn_scores(meta, blocks, batch, heads, seq, qpk, q, scale)
    check_fused(d_s.cpu().numpy().astype(np.float64), ref, refabs, f"scores q{qpk}")


# ------------------------------------------------------------------ full-size configurations
def host_threads():
    import os

    return max(1, len(os.sched_getaffinity(0)))


def sample_groups(n, rng, k=6144):
    idx = np.unique(np.concatenate([np.arange(min(n, 1024)), np.arange(max(0, n - 1024), n), rng.integers(0, n, k)]))
    return idx


def assert_device_equals_oracle(eo, om, blocks, d_out):
    """Every group of the tensor: the oracle decodes all of them on the host cores, the comparison runs on the GPU."""
    n = blocks.shape[0]
    want = eo.decode_threads(om, blocks, host_threads()).view(np.int16)
    d_want = torch.from_numpy(want).cuda()
    got = d_out.view(torch.int16).view(n, 128)
    if not torch.equal(got, d_want):
        bad = torch.nonzero((got != d_want).any(dim=1)).flatten()
        g = int(bad[0])
        raise AssertionError(f"{bad.numel()} of {n} groups differ; first group {g}, positions "
                             f"{torch.nonzero(got[g] != d_want[g]).flatten()[:8].tolist()}")


def check_full_decompress(B, eo, t, d_out=None):
    d_meta, d_blocks = B.meta_to_device(t.meta), dev(t.blocks)
    d_out = torch.empty(t.n_groups * 128, dtype=torch.float16, device="cuda")
    B.ecco_decompress(d_meta, d_blocks, t.n_groups, d_out)
    torch.cuda.synchronize()
    assert B.ecco_device_status() == 0
    om = oracle_meta_from_lib(eo, t.meta)
    assert_device_equals_oracle(eo, om, t.blocks, d_out)
    return om, d_meta, d_blocks


def oracle_gemv_threads(eo, om, blocks, n_out, k, x, batch):
    """eo.gemv over disjoint row ranges from one Python thread per host core (ctypes drops the GIL)."""
    from concurrent.futures import ThreadPoolExecutor

    kb = k // 128
    threads = min(host_threads(), n_out)
    bounds = [n_out * i // threads for i in range(threads + 1)]
    ref, refabs = np.zeros((batch, n_out)), np.zeros((batch, n_out))

    def work(i):
        lo, hi = bounds[i], bounds[i + 1]
        if hi > lo:
            r, a = eo.gemv(om, blocks[lo * kb:hi * kb], hi - lo, k, x, batch)
            ref[:, lo:hi], refabs[:, lo:hi] = r, a

    with ThreadPoolExecutor(threads) as ex:
        list(ex.map(work, range(threads)))
    return ref, refabs


def check_full_gemv(B, eo, synth, t, om, d_meta, d_blocks, batch, all_rows=False):
    n_out, k = t.shape
    x = synth.activations(batch, k, 70 + batch)
    d_x = dev(x)
    d_y = torch.empty((batch, n_out), dtype=torch.float32, device="cuda")
    wsb = B.ecco_gemv_workspace_bytes(n_out, k, batch)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    B.ecco_gemv(d_meta, d_blocks, n_out, k, d_x, batch, d_y, ws, wsb)
    torch.cuda.synchronize()
    assert B.ecco_device_status() == 0
    y = d_y.cpu().numpy().astype(np.float64)
    if all_rows:
        ref, refabs = oracle_gemv_threads(eo, om, t.blocks, n_out, k, x, batch)
        check_fused(y, ref, refabs, f"gemv b{batch} full {n_out}x{k}")
        return
    rows = np.unique(np.concatenate([[0, n_out - 1], np.random.Generator(np.random.PCG64(n_out + batch)).integers(0, n_out, 48)]))
    kb = k // 128
    sub = np.concatenate([t.blocks[r * kb:(r + 1) * kb] for r in rows])
    ref, refabs = eo.gemv(om, sub, len(rows), k, x, batch)
    check_fused(y[:, rows], ref, refabs, f"gemv b{batch} full {n_out}x{k}")


def test_config2_llama7b_layer_full_size(B, eo, W, synth):
    items, metas = [], []
    for t in W.config2(names=("q", "gate", "down")):
        om, d_meta, d_blocks = check_full_decompress(B, eo, t)
        for batch in (1, 8):                               # every output row against the oracle's fp64 product
            check_full_gemv(B, eo, synth, t, om, d_meta, d_blocks, batch, all_rows=True)
        items.append((d_meta, d_blocks, t.n_groups, torch.empty(t.n_groups * 128, dtype=torch.float16, device="cuda")))
        metas.append((om, t))
    # the three tensors in the launch configuration bench.py times: one batched call (one run: the tensors share
    # their tables and differ in the exponent), every group against the oracle
    B.ecco_decompress_batch(items)
    torch.cuda.synchronize()
    assert B.ecco_device_status() == 0
    for (om, t), (_, _, n, d_out) in zip(metas, items):
        assert_device_equals_oracle(eo, om, t.blocks, d_out)
    # the fused GEMV in the launch configuration bench.py times: matrices that share x in one ecco_gemv_batch call
    # (here q with itself standing in for k and v, and gate twice for gate + up), every output row against the oracle
    (oq, tq), (og, tg) = metas[0], metas[1]
    for batch in (1, 8):
        for om, t, (d_meta, d_blocks, _, _), copies in ((oq, tq, items[0], 3), (og, tg, items[1], 2)):
            n_out, k = t.shape
            x = synth.activations(batch, k, 90 + batch)
            d_x = dev(x)
            ys = [torch.full((batch, n_out), float("nan"), dtype=torch.float32, device="cuda") for _ in range(copies)]
            call = [(d_meta, d_blocks, n_out, k, d_x, y) for y in ys]
            wsb = B.ecco_gemv_batch_workspace_bytes(call, batch)
            ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
            B.ecco_gemv_batch(call, batch, ws, wsb)
            torch.cuda.synchronize()
            assert B.ecco_device_status() == 0
            ref, refabs = oracle_gemv_threads(eo, om, t.blocks, n_out, k, x, batch)
            for y in ys:
                check_fused(y.cpu().numpy().astype(np.float64), ref, refabs, f"gemv batch-call b{batch} full {n_out}x{k}")


def check_full_attn(B, eo, synth, t, qpk):
    batch, heads, seq, _ = t.shape
    om = oracle_meta_from_lib(eo, t.meta)
    q = synth.queries(batch, heads * qpk, 80 + qpk)
    d_meta, d_blocks, d_q = B.meta_to_device(t.meta), dev(t.blocks), dev(q)
    d_s = torch.empty((batch, heads * qpk, seq), dtype=torch.float32, device="cuda")
    B.ecco_attn_scores(d_meta, d_blocks, batch, heads, seq, qpk, d_q, 128 ** -0.5, d_s)
    torch.cuda.synchronize()
    assert B.ecco_device_status() == 0
    s = d_s.cpu().numpy().astype(np.float64)
    rng = np.random.Generator(np.random.PCG64(seq + qpk))
    for _ in range(6):
        b, h = int(rng.integers(batch)), int(rng.integers(heads))
        t0 = int(rng.integers(0, seq - 256 + 1))
        g0 = (b * heads + h) * seq + t0
        ref, refabs = eo.attn_scores(om, t.blocks[g0:g0 + 256], 1, 1, 256, qpk, q[b, h * qpk:(h + 1) * qpk], 128 ** -0.5)
        check_fused(s[b, h * qpk:(h + 1) * qpk, t0:t0 + 256], ref[0], refabs[0], f"scores q{qpk} full")
    assert np.isfinite(s).all()


def check_full_attn_values(B, eo, t, qpk, n_heads_checked=3):
    batch, heads, seq, _ = t.shape
    om = oracle_meta_from_lib(eo, t.meta)
    rng = np.random.Generator(np.random.PCG64(seq * 3 + qpk))
    scores = (rng.standard_normal((batch, heads * qpk, seq)) * 2.0).astype(np.float32)
    got = gpu_attn_values(B, t.meta, t.blocks, batch, heads, seq, qpk, scores)
    assert np.isfinite(got).all()
    for _ in range(n_heads_checked):
        b, h = int(rng.integers(batch)), int(rng.integers(heads))
        g0 = (b * heads + h) * seq
        ref, refabs = eo.attn_values(om, t.blocks[g0:g0 + seq], 1, 1, seq, qpk, scores[b:b + 1, h * qpk:(h + 1) * qpk])
        check_fused(got[b, h * qpk:(h + 1) * qpk], ref[0], refabs[0], f"values q{qpk} full")


def test_config3_kv_cache_full_size(B, eo, W, synth):
    k, v = W.config3(which=("K", "V"))
    assert k.n_groups == 8 * 32 * 4096
    check_full_decompress(B, eo, k)
    check_full_attn(B, eo, synth, k, 1)
    check_full_decompress(B, eo, v)
    check_full_attn_values(B, eo, v, 1)


def test_config4_llama70b_mlp_full_size(B, eo, W, synth):
    for t in W.config4(names=("gate", "down")):
        assert t.n_groups == 1835008
        om, d_meta, d_blocks = check_full_decompress(B, eo, t)
        check_full_gemv(B, eo, synth, t, om, d_meta, d_blocks, 1)


def test_config5_long_context_gqa_full_size(B, eo, W, synth):
    k, v = W.config5(which=("K", "V"))
    assert k.n_groups == 16 * 8 * 32768
    check_full_decompress(B, eo, k)
    check_full_attn(B, eo, synth, k, 8)
    check_full_attn_values(B, eo, v, 8, n_heads_checked=2)


def test_config4_streams_past_4_gib_of_output(B, eo, W):
    """cfg-4 streams of 1 GiB and 4 GiB (2^24 and 2^26 groups: 4 GiB and 16 GiB of fp16, byte offsets beyond 2^32 and
    TMA row coordinates beyond 2^24), built as bench.py builds them by tiling the encoded gate matrix on the device.
    Compared bit for bit with the oracle: the first and last tile, both sides of every 2^32-byte boundary of the
    output, and 4096 random groups; in between, a hash of every copy of the matrix must equal the first copy's."""
    (t,) = W.config4(names=("gate",))
    om = oracle_meta_from_lib(eo, t.meta)
    d_meta, d_one = B.meta_to_device(t.meta), dev(t.blocks)
    n1 = t.n_groups
    want_one = None
    for log2n in (24, 26):
        n = 1 << log2n
        reps = -(-n // n1)
        d_blocks = d_one.repeat(reps, 1)[:n].contiguous()
        d_out = torch.empty(n * 128, dtype=torch.float16, device="cuda")
        B.ecco_decompress(d_meta, d_blocks, n, d_out)
        torch.cuda.synchronize()
        assert B.ecco_device_status() == 0
        out = d_out.view(n, 128)
        per_4gib = (1 << 32) // 256                         # groups per 2^32 bytes of output
        rng = np.random.Generator(np.random.PCG64(log2n))
        idx = [np.arange(64), np.arange(n - 64, n), rng.integers(0, n, 4096)]
        for b in range(per_4gib, n, per_4gib):
            idx.append(np.arange(b - 64, b + 64))
        idx = np.unique(np.concatenate(idx))
        got = out[torch.from_numpy(idx).cuda()].cpu().numpy()
        assert_bit_exact(got, eo.decode_threads(om, t.blocks[idx % n1], host_threads()))
        # every whole copy of the matrix decodes to the same bits as the first one, which is compared in full
        if want_one is None:
            assert_device_equals_oracle(eo, om, t.blocks, d_out[: n1 * 128])
            want_one = True
        first = out[:n1].view(torch.int16)
        for r in range(1, n // n1):
            assert torch.equal(out[r * n1:(r + 1) * n1].view(torch.int16), first), (log2n, r)
        tail = n - (n // n1) * n1
        if tail:
            assert torch.equal(out[n - tail:].view(torch.int16), first[:tail]), (log2n, "tail")
        del d_blocks, d_out, out, first


# ------------------------------------------------------------------ 2x activation codec
@pytest.mark.parametrize("n_groups", [0, 1, 7, 8, 9, 1000, 4097, 1 << 16])
def test_act2x_compress_and_decompress_match_oracle(B, eo, synth, n_groups):
    x = synth.activations(max(n_groups, 1), 64, 300 + n_groups % 97)[:n_groups]
    if n_groups > 8:
        x[3] = np.float16(-0.75)                     # constant group: zero scale
        x[5] = (x[5].astype(np.float32) * 1000).astype(np.float16)
        x[6] = (x[6].astype(np.float32) * 1e-4).astype(np.float16)   # subnormal-sized steps
    d_x = torch.from_numpy(np.ascontiguousarray(x)).cuda() if n_groups else torch.empty(64, dtype=torch.float16, device="cuda")
    d_blocks = torch.full((max(n_groups, 1), 64), 0xEE, dtype=torch.uint8, device="cuda")
    B.ecco_act_compress(d_x, n_groups, d_blocks)
    d_out = torch.empty((max(n_groups, 1), 64), dtype=torch.float16, device="cuda")
    B.ecco_act_decompress(d_blocks, n_groups, d_out)
    torch.cuda.synchronize()
    if n_groups == 0:
        return
    want_blocks = eo.act_encode(x)
    got_blocks = d_blocks.cpu().numpy()
    bad = np.nonzero((got_blocks != want_blocks).any(axis=1))[0]
    assert bad.size == 0, f"{bad.size} blocks differ, first {bad[:4]}"
    assert np.array_equal(d_out.cpu().numpy().view(np.uint16), eo.act_decode(want_blocks).view(np.uint16))
    # decompression is total: random bytes decode like the oracle says
    rb = synth.random_blocks(n_groups, 17)
    d_rb = torch.from_numpy(rb).cuda()
    B.ecco_act_decompress(d_rb, n_groups, d_out)
    torch.cuda.synchronize()
    got, want = d_out.cpu().numpy().view(np.uint16), eo.act_decode(rb).view(np.uint16)
    finite = np.isfinite(eo.act_decode(rb).astype(np.float32))       # NaN payloads may differ, everything else may not
    assert np.array_equal(got[finite], want[finite])


# ------------------------------------------------------------------ fused attention output (softmax . V)
def gpu_attn_values(B, lmeta, blocks, batch, heads, seq, qpk, scores):
    d_meta, d_blocks, d_s = B.meta_to_device(lmeta), dev(blocks), dev(scores)
    d_o = torch.full((batch, heads * qpk, 128), float("nan"), dtype=torch.float32, device="cuda")
    wsb = B.ecco_attn_values_workspace_bytes(batch, heads, seq, qpk)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    ws.fill_(0xCD)
    B.ecco_attn_values(d_meta, d_blocks, batch, heads, seq, qpk, d_s, d_o, ws, wsb)
    torch.cuda.synchronize()
    assert B.ecco_device_status() == 0
    return d_o.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("batch,heads,seq,qpk", [(2, 4, 256, 1), (2, 4, 256, 8), (1, 3, 77, 4), (1, 1, 1, 1), (2, 2, 1300, 3),
                                                 (1, 2, 5000, 2)])
def test_attn_values_match_oracle(B, eo, kv_small, synth, batch, heads, seq, qpk):
    meta = kv_small["meta"]
    n = batch * heads * seq
    blocks = np.tile(kv_small["blocks"], (-(-n // 2048), 1))[:n]
    rng = np.random.Generator(np.random.PCG64(seq * 7 + qpk))
    scores = (rng.standard_normal((batch, heads * qpk, seq)) * 2.5).astype(np.float32)
    got = gpu_attn_values(B, lib_meta_from_oracle(B, meta), blocks, batch, heads, seq, qpk, scores)
    ref, refabs = eo.attn_values(meta, blocks, batch, heads, seq, qpk, scores)
    check_fused(got, ref, refabs, f"values q{qpk}")


def test_attn_values_on_garbage_blocks_and_peaked_softmax(B, eo, kv_small, synth):
    meta = kv_small["meta"]
    rb = synth.random_blocks(2 * 2 * 700, 321)             # duplicate pad locations, clips, 16-pad groups
    rng = np.random.Generator(np.random.PCG64(5))
    scores = (rng.standard_normal((2, 4, 700)) * 2).astype(np.float32)
    scores[0, 1, :] = -50.0
    scores[0, 1, 333] = 10.0                               # one-hot softmax
    got = gpu_attn_values(B, lib_meta_from_oracle(B, meta), rb, 2, 2, 700, 2, scores)
    ref, refabs = eo.attn_values(meta, rb, 2, 2, 700, 2, scores)
    check_fused(got, ref, refabs, "values q2 garbage")


@pytest.mark.parametrize("qpk", [1, 8])
def test_attn_values_keeps_small_probabilities(B, eo, kv_small, synth, qpk):
    """One token takes almost all the weight and its vector is all zeros, so every output is the sum of the other
    tokens' contributions at p ~ 1e-9: probabilities must survive the trip through the fp16 operands of the tensor
    cores.  A second row spreads its weight evenly over 5000 tokens (p = 2e-4 each, below fp16's normal range).
    Bound: 1e-3 sum p|V| plus 2^-38 sum |V|, the floor of the scaled fp16 pair."""
    meta = kv_small["meta"]
    seq = 5000
    rng = np.random.Generator(np.random.PCG64(17))
    x = synth.kv_cache(1, 1, seq, 1003, 3003).reshape(seq, 128).copy()
    x[1234] = 0
    blocks, _ = eo.encode(meta, x.astype(np.float16), eo.SELECT_MINMAX)
    dec = eo.decode(meta, blocks).astype(np.float64)
    assert not dec[1234].any()
    scores = (rng.standard_normal((1, qpk, seq))).astype(np.float32)
    scores[0, 0, 1234] += 22.0                             # p of the others ~ e^-22 / 1: 3e-10
    if qpk > 1:
        scores[0, 1, :] = 0.25                             # uniform: p = 2e-4 for every token
    got = gpu_attn_values(B, lib_meta_from_oracle(B, meta), blocks, 1, 1, seq, qpk, scores)
    ref, refabs = eo.attn_values(meta, blocks, 1, 1, seq, qpk, scores)
    floor = np.abs(dec).sum(axis=0) * 2.0 ** -38
    err = np.abs(got - ref)
    assert np.all(err <= TOL * refabs + floor), float((err / (TOL * refabs + floor)).max())
    assert np.abs(ref[0, 0]).max() < 1e-6 and np.abs(got[0, 0]).max() > 0      # the small sums are really there
    if qpk > 1:
        assert np.all(err[0, 1] <= 2e-5 * refabs[0, 1])    # evenly spread weights: far inside the bound


@pytest.mark.parametrize("seq", [301, 4100])
def test_attn_values_with_masked_scores(B, eo, kv_small, synth, seq):
    """Scores of -inf (masked tokens) carry no weight: at the start of a row (before the row statistics have seen any
    finite score), in the middle, in whole 16-byte chunks and at a ragged end; rows of odd length start at addresses
    that are not 16-byte aligned."""
    meta = kv_small["meta"]
    heads, qpk = 2, 3
    n = heads * seq
    blocks = np.tile(kv_small["blocks"], (-(-n // 2048), 1))[:n]
    rng = np.random.Generator(np.random.PCG64(5 + seq))
    scores = (rng.standard_normal((1, heads * qpk, seq)) * 2.0).astype(np.float32)
    scores[0, :, :9] = -np.inf
    scores[0, 1, 100:164] = -np.inf
    scores[0, 2, -3:] = -np.inf
    scores[0, 3, rng.random(seq) < 0.5] = -np.inf
    scores[0, 4, 1:] = -np.inf
    scores[0, 4, 0] = 0.5                                  # a single live token, first in the row
    got = gpu_attn_values(B, lib_meta_from_oracle(B, meta), blocks, 1, heads, seq, qpk, scores)
    ref, refabs = eo.attn_values(meta, blocks, 1, heads, seq, qpk, scores)
    assert np.isfinite(ref).all()
    check_fused(got, ref, refabs, "values masked")


# ------------------------------------------------------------------ online KV compressor
def gpu_kv_compress(B, lmeta, x):
    n = x.size // 128
    d_meta = B.meta_to_device(lmeta)
    d_x = dev(x.reshape(-1)) if n else torch.empty(128, dtype=torch.float16, device="cuda")
    d_blocks = torch.full((max(n, 1), 64), 0xEE, dtype=torch.uint8, device="cuda")
    B.ecco_kv_compress(d_meta, d_x, n, d_blocks)
    torch.cuda.synchronize()
    assert B.ecco_device_status() == 0
    return d_blocks.cpu().numpy()[:n]


def assert_blocks_equal(got, want):
    bad = np.nonzero((got != want).any(axis=1))[0]
    assert bad.size == 0, f"{bad.size} of {got.shape[0]} blocks differ; first {bad[:5]}"


@pytest.mark.parametrize("n_groups", [0, 1, 7, 8, 9, 2048])
def test_kv_compress_matches_oracle_encoder(B, eo, kv_small, n_groups):
    meta = kv_small["meta"]
    x = kv_small["k"].reshape(-1, 128)[:n_groups]
    got = gpu_kv_compress(B, lib_meta_from_oracle(B, meta), x)
    if n_groups:
        assert_blocks_equal(got, kv_small["blocks"][:n_groups])


def test_kv_compress_edge_groups_and_s16(B, eo, kv_small, synth):
    meta = kv_small["meta"]
    rng = np.random.Generator(np.random.PCG64(77))
    groups = [np.zeros(128), np.full(128, 0.5), np.full(128, -3.0), np.concatenate([np.full(64, 1.0), np.full(64, -1.0)]),
              np.full(128, 2.0 ** -24), rng.standard_normal(128) * 1e-3, rng.standard_normal(128) * 300,   # saturating scales
              np.where(np.arange(128) % 2 == 0, 5.0, -5.0), np.arange(128) - 64.0, rng.choice([-2.0, 0.0, 2.0], 128)]
    for _ in range(200):
        g = rng.standard_normal(128) * rng.choice([0.1, 1.0, 10.0])
        g[rng.integers(128)] *= rng.choice([1.0, 20.0])
        if rng.random() < 0.3:
            g[rng.integers(128, size=5)] = g[rng.integers(128)]            # ties in |x|
        groups.append(g)
    x = np.array(groups, dtype=np.float16)
    want, st = eo.encode(meta, x, eo.SELECT_MINMAX)
    assert st.clipped_groups > 0 and st.padded_groups > 0
    assert_blocks_equal(gpu_kv_compress(B, lib_meta_from_oracle(B, meta), x), want)
    # the paper's hardware compressor works with 16 patterns
    cal = synth.kv_cache(1, 4, 512, 2003, 3003)
    m16 = eo.calibrate(cal, S=16, H=4, seed=3, select=eo.SELECT_MINMAX)
    want, _ = eo.encode(m16, kv_small["k"], eo.SELECT_MINMAX)
    assert_blocks_equal(gpu_kv_compress(B, lib_meta_from_oracle(B, m16), kv_small["k"]), want)
    # a skewed codebook: long streams (heavy clipping) and short ones (16 pads)
    skew = make_meta(eo, skew_lens, seed=3)
    xs = (rng.standard_t(3, size=(512, 128)) * 0.05).astype(np.float16)
    want, st = eo.encode(skew, xs, eo.SELECT_MINMAX)
    assert_blocks_equal(gpu_kv_compress(B, lib_meta_from_oracle(B, skew), xs), want)


def test_kv_compress_full_size_round_trip(B, eo, W, synth):
    """cfg 3 K cache: GPU-compressed blocks equal the host encoder's, and decompress to the same fp16."""
    (t,) = W.config3(which=("K",), keep_source=True)
    got = gpu_kv_compress(B, t.meta, t.source)
    assert_blocks_equal(got, t.blocks)


# ------------------------------------------------------------------ variable-length container
def oracle_offsets_from_index(index, n):
    nc = (n + 4095) // 4096
    idx64 = index[: 8 * (1 + nc)].view(np.uint64)
    off32 = index[8 * (1 + nc): 8 * (1 + nc) + 4 * n].view(np.uint32)
    return np.concatenate([idx64[1:][np.arange(n) >> 12] + off32, idx64[:1]]).astype(np.uint64)


def gpu_var_decompress(B, lmeta, stream, index, n):
    d_out = torch.full((n, 128), float("nan"), dtype=torch.float16, device="cuda")
    B.ecco_var_decompress(B.meta_to_device(lmeta), dev(stream), dev(index), n, d_out)
    torch.cuda.synchronize()
    assert B.ecco_device_status() == 0
    return d_out.cpu().numpy()


@pytest.mark.parametrize("n_groups", [1, 31, 33, 1000, 2048])
def test_var_decompress_matches_oracle(B, eo, cfg1_small, n_groups):
    meta = cfg1_small["meta"]
    lm = lib_meta_from_oracle(B, meta)
    x = cfg1_small["w"].reshape(-1, 128)[:n_groups]
    stream, index, total = B.ecco_var_encode_host(lm, x, B.SELECT_MSE | B.KEEP_EXPONENT)
    got = gpu_var_decompress(B, lm, stream, index, n_groups)
    assert_bit_exact(got, eo.var_decode(meta, stream, oracle_offsets_from_index(index, n_groups)))


def test_var_decompress_is_total_on_garbage(B, eo, cfg1_small, synth):
    """Random stream bytes with a valid-looking but arbitrary index: overlapping, empty and over-long groups."""
    meta = cfg1_small["meta"]
    lm = lib_meta_from_oracle(B, meta)
    n = 4096 + 100
    rng = np.random.Generator(np.random.PCG64(12))
    stream = synth.random_blocks(4096, 5).reshape(-1)                      # 256 KiB of noise, a multiple of 16
    total = stream.size * 8 - 37
    starts = np.sort(rng.integers(0, total, n)).astype(np.uint64)
    starts[5] = starts[4]                                                   # empty group
    nc = (n + 4095) // 4096
    index = np.zeros((8 * (1 + nc) + 4 * n + 15) // 16 * 16, dtype=np.uint8)
    idx64 = index[: 8 * (1 + nc)].view(np.uint64)
    idx64[0] = total
    for c in range(nc):
        idx64[1 + c] = starts[c * 4096]
    index[8 * (1 + nc): 8 * (1 + nc) + 4 * n].view(np.uint32)[:] = (starts - idx64[1:][np.arange(n) >> 12]).astype(np.uint32)
    got = gpu_var_decompress(B, lm, stream, index, n)
    assert_bit_exact(got, eo.var_decode(meta, stream, np.concatenate([starts, [np.uint64(total)]]).astype(np.uint64)))


def test_var_decompress_config2_gate_full_size(B, eo, W, synth):
    (t,) = W.config2(names=("gate",), keep_source=True)
    stream, index, total = B.ecco_var_encode_host(t.meta, t.source, B.SELECT_MSE | B.KEEP_EXPONENT)
    n = t.n_groups
    d_out = torch.empty((n, 128), dtype=torch.float16, device="cuda")
    B.ecco_var_decompress(B.meta_to_device(t.meta), dev(stream), dev(index), n, d_out)
    torch.cuda.synchronize()
    om = oracle_meta_from_lib(eo, t.meta)
    offs = oracle_offsets_from_index(index, n)
    # sampled runs of consecutive groups (the oracle needs each group's end = the next group's start)
    rng = np.random.Generator(np.random.PCG64(2))
    for g0 in [0, n - 512] + [int(v) for v in rng.integers(0, n - 512, 6)]:
        want = eo.var_decode(om, stream, np.concatenate([offs[g0:g0 + 512], offs[g0 + 512:g0 + 513]]))
        assert_bit_exact(d_out[g0:g0 + 512].cpu().numpy(), want)
    assert bool(torch.isfinite(d_out).all())
    assert total / n < 512                                                  # on average the stream is shorter than the blocks


# ------------------------------------------------------------------ capture into a CUDA graph
def test_calls_can_be_captured_into_a_cuda_graph(B, eo, kv_small, cfg1_small, synth):
    """The device calls neither synchronise nor allocate, so a chain of them can be captured into a CUDA graph
    (after one eager call of each, which sets the kernels' attributes) and replayed; the replay gives the eager
    results bit for bit, also after the inputs have changed in place."""
    wm, km = B.meta_to_device(lib_meta_from_oracle(B, cfg1_small["meta"])), B.meta_to_device(lib_meta_from_oracle(B, kv_small["meta"]))
    wb, kb = dev(cfg1_small["blocks"]), dev(kv_small["blocks"])                 # 256 x 1024 weights, K cache [2][4][256]
    n_out, k, heads, seq, qpk = 256, 1024, 8, 256, 2
    x = dev(synth.activations(8, k, 3))
    q = dev(synth.queries(1, heads * qpk, 4))
    out = torch.empty(2048 * 128, dtype=torch.float16, device="cuda")
    y1, y8 = torch.empty((1, n_out), dtype=torch.float32, device="cuda"), torch.empty((8, n_out), dtype=torch.float32, device="cuda")
    sc = torch.empty((1, heads * qpk, seq), dtype=torch.float32, device="cuda")
    av = torch.empty((1, heads * qpk, 128), dtype=torch.float32, device="cuda")
    items1, items8 = [(wm, wb, n_out, k, x, y1)], [(wm, wb, n_out, k, x, y8)]
    nb1, nb8 = B.ecco_gemv_batch_workspace_bytes(items1, 1), B.ecco_gemv_batch_workspace_bytes(items8, 8)
    ws1, ws8 = torch.empty(nb1, dtype=torch.uint8, device="cuda"), torch.empty(nb8, dtype=torch.uint8, device="cuda")
    nbv = B.ecco_attn_values_workspace_bytes(1, heads, seq, qpk)
    wsv = torch.empty(nbv, dtype=torch.uint8, device="cuda")
    a1, a8 = B.gemv_items(items1), B.gemv_items(items8)

    def chain(st):
        B.ecco_decompress(wm, wb, 2048, out, st)
        B.ecco_gemv_batch(a1, 1, ws1, nb1, st)
        B.ecco_gemv_batch(a8, 8, ws8, nb8, st)
        B.ecco_attn_scores(km, kb, 1, heads, seq, qpk, q, 0.0884, sc, st)
        B.ecco_attn_values(km, kb, 1, heads, seq, qpk, sc, av, wsv, nbv, st)

    results = lambda: [t.clone() for t in (out, y1, y8, sc, av)]
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        chain(st)                                          # eager: also the first call of every kernel
        st.synchronize()
        want = results()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            chain(st)
        for t in (out, y1, y8, sc, av):
            t.fill_(float("nan"))
        g.replay()
        st.synchronize()
        assert B.ecco_device_status() == 0
        assert all(torch.equal(a, b) for a, b in zip(want, results()))
        x.mul_(0.5)                                        # new inputs in the same buffers
        q.mul_(2.0)
        g.replay()
        st.synchronize()
        replayed = results()
        chain(st)
        st.synchronize()
        assert all(torch.equal(a, b) for a, b in zip(replayed, results()))
        assert not torch.equal(replayed[1], want[1])


# ------------------------------------------------------------------ stream order of back-to-back calls
def test_back_to_back_calls_keep_stream_order(B, eo, kv_small, cfg1_small, synth):
    """The kernels are launched so that one may start while its predecessor in the stream drains.  Calls that
    depend on each other through a buffer (write-after-write on an output, read-after-write on blocks, scores and
    a shared workspace), issued with no synchronisation in between, must give what they give one at a time."""
    meta, lm = kv_small["meta"], lib_meta_from_oracle(B, kv_small["meta"])
    d_meta = B.meta_to_device(lm)
    reps = 96                                              # 196 608 groups: every SM busy, tails overlap heads
    x = np.tile(kv_small["k"].reshape(-1, 128), (reps, 1))
    n = x.shape[0]
    want_blocks = np.tile(kv_small["blocks"], (reps, 1))
    want_a = np.tile(eo.decode(meta, kv_small["blocks"]), (reps, 1))
    other = np.ascontiguousarray(want_blocks[::-1])        # a second, different tensor of the same size
    want_b = np.ascontiguousarray(want_a[::-1])
    d_x, d_other = dev(x.reshape(-1)), dev(other)
    d_blocks = torch.full((n, 64), 0xEE, dtype=torch.uint8, device="cuda")
    d_out = torch.zeros(n * 128, dtype=torch.float16, device="cuda")
    d_out2 = torch.zeros(n * 128, dtype=torch.float16, device="cuda")
    for _ in range(6):
        B.ecco_kv_compress(d_meta, d_x, n, d_blocks)       # blocks written ...
        B.ecco_decompress(d_meta, d_blocks, n, d_out2)     # ... and read by the next kernel
        B.ecco_decompress(d_meta, d_other, n, d_out)       # the same output twice: the later call wins
        B.ecco_decompress(d_meta, d_blocks, n, d_out)
        B.ecco_decompress(d_meta, d_other, n, d_out)
        d_blocks_snapshot = d_blocks.clone()
        d_blocks.fill_(0xEE)                               # a non-library kernel in between
    torch.cuda.synchronize()
    assert B.ecco_device_status() == 0
    assert_blocks_equal(d_blocks_snapshot.cpu().numpy(), want_blocks)
    assert_bit_exact(d_out2.cpu().numpy().reshape(n, 128), want_a)
    assert_bit_exact(d_out.cpu().numpy().reshape(n, 128), want_b)

    # two products through ONE workspace, then scores -> softmax . V, all back to back
    wmeta, wlm = cfg1_small["meta"], lib_meta_from_oracle(B, cfg1_small["meta"])
    d_wmeta = B.meta_to_device(wlm)
    n_out, k = 4096, 2048
    blocks_a = np.tile(cfg1_small["blocks"], (32, 1))[: n_out * k // 128]
    blocks_b = np.ascontiguousarray(blocks_a[::-1])
    d_a, d_b = dev(blocks_a), dev(blocks_b)
    for batch in (1, 8):
        xs = synth.activations(batch, k, 400 + batch)
        d_xs = dev(xs)
        wsb = B.ecco_gemv_workspace_bytes(n_out, k, batch)
        ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
        ws.fill_(0xA5)
        one = []
        for blk in (d_a, d_b):                             # one at a time
            y = torch.empty((batch, n_out), dtype=torch.float32, device="cuda")
            B.ecco_gemv(d_wmeta, blk, n_out, k, d_xs, batch, y, ws, wsb)
            torch.cuda.synchronize()
            one.append(y.cpu().numpy())
        ys = [torch.empty((batch, n_out), dtype=torch.float32, device="cuda") for _ in range(8)]
        for i, y in enumerate(ys):                         # back to back through the same workspace
            B.ecco_gemv(d_wmeta, d_b if i & 1 else d_a, n_out, k, d_xs, batch, y, ws, wsb)
        torch.cuda.synchronize()
        assert B.ecco_device_status() == 0
        for i, y in enumerate(ys):
            assert np.array_equal(y.cpu().numpy(), one[i & 1]), (batch, i)

    batch, heads, seq, qpk = 2, 4, 256, 4
    kb, vb = kv_small["blocks"], np.ascontiguousarray(kv_small["blocks"][::-1])
    q = synth.queries(batch, heads * qpk, 77)
    d_k, d_v, d_q = dev(kb), dev(vb), dev(q)
    wsb = B.ecco_attn_values_workspace_bytes(batch, heads, seq, qpk)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    sc = torch.empty((batch, heads * qpk, seq), dtype=torch.float32, device="cuda")
    out = torch.empty((batch, heads * qpk, 128), dtype=torch.float32, device="cuda")
    B.ecco_attn_scores(d_meta, d_k, batch, heads, seq, qpk, d_q, 0.0884, sc)
    torch.cuda.synchronize()
    B.ecco_attn_values(d_meta, d_v, batch, heads, seq, qpk, sc, out, ws, wsb)
    torch.cuda.synchronize()
    want = out.cpu().numpy().copy()
    for _ in range(4):
        sc.zero_()
        out.zero_()
        B.ecco_attn_scores(d_meta, d_k, batch, heads, seq, qpk, d_q, 0.0884, sc)
        B.ecco_attn_values(d_meta, d_v, batch, heads, seq, qpk, sc, out, ws, wsb)
    torch.cuda.synchronize()
    assert B.ecco_device_status() == 0
    assert np.array_equal(out.cpu().numpy(), want)
