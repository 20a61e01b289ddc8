"""Randomised comparison of every device call with the CPU oracle, bounded and seeded.

Each configuration draws its own metadata (number of patterns, exponent, patterns with duplicate centroids, a random
admissible code shape per codebook, a skewed ID_KP code), its own data (random bit streams, or heavy-tailed values
encoded by the oracle) and ragged sizes, and runs decompress, the fused GEMV (batch 1..8), attention scores and
attention output, the online KV compressor, the variable-length container and the 2x activation codec against the
oracle.  A second test issues random sequences of dependent calls with no synchronisation and requires the results of
the same sequences run one call at a time (stream order under the overlapped launches).
"""
import numpy as np
import pytest

from helpers import lib_meta_from_oracle, record_fused

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 1e-3
N_CONFIGS = 300
N_SEQUENCES = 100


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2505_06901_b200 import binding

    binding.lib()
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def code_shapes():
    """Every multiset of 16 code lengths in 2..8 with Kraft sum 1, as counts per length."""
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


def random_meta(eo, rng, shapes, few_shapes):
    S = int(rng.choice([2, 3, 5, 16, 33, 64]))
    m = eo.Meta()
    m.S, m.H, m.e = S, 4, int(rng.integers(-20, 8))
    kl = eo.huffman_limited(rng.random(S) ** 3 + 1e-3, 12)
    # few_shapes: a handful of code shapes, so that the image gets pair tables (two symbols per lookup); otherwise one
    # random shape per codebook, up to 256 different ones (no pair tables: one symbol per lookup)
    pool = [shapes[int(i)] for i in rng.integers(len(shapes), size=int(rng.integers(1, 12)))] if few_shapes else shapes
    for k in range(S):
        m.kp_len[k] = int(kl[k])
        pat = np.sort(rng.uniform(-1, 1, 15) * rng.choice([1.0, 0.3, 1e-3]))
        if rng.random() < 0.2:
            pat[3:6] = pat[3]                                # duplicate centroids
        for j in range(15):
            m.pattern[k][j] = int(np.float16(pat[j]).view(np.uint16))
        for h in range(4):
            lens = rng.permutation(np.repeat(np.arange(2, 9), pool[int(rng.integers(len(pool)))]))
            for s in range(16):
                m.cb_len[k][h][s] = int(lens[s])
    assert eo.meta_check(m) == 0
    return m


def fused_ok(got, ref, refabs, label):
    err = np.abs(got - ref)
    scaled = float((err / (refabs + 1e-30)).max())
    record_fused(label, scaled, 0.0)
    return bool(np.all(err <= TOL * refabs + 1e-30)), scaled


def test_random_configurations_match_the_oracle(B, eo, synth):
    shapes = code_shapes()
    failures = []
    for it in range(N_CONFIGS):
        rng = np.random.Generator(np.random.PCG64(10_000 + it))
        m = random_meta(eo, rng, shapes, few_shapes=it % 3 != 0)
        lm = lib_meta_from_oracle(B, m)
        d_meta = B.meta_to_device(lm)
        n = int(rng.choice([1, 31, 33, 500, 1024, 3000]))
        x = None
        if rng.random() < 0.4:
            blocks = synth.random_blocks(n, 77 + it)
        else:
            scale = 2.0 ** m.e * rng.choice([1, 30, 400])
            x = (rng.standard_t(3, size=(n, 128)) * scale * 0.05).astype(np.float16)
            x = np.nan_to_num(x, posinf=6e4, neginf=-6e4)
            blocks, _ = eo.encode(m, x, int(rng.integers(2)))
        d_b = dev(blocks)
        # decompress: bit for bit
        d_o = torch.full((n * 128,), float("nan"), dtype=torch.float16, device="cuda")
        B.ecco_decompress(d_meta, d_b, n, d_o)
        want = eo.decode_threads(m, blocks, 8)
        if not np.array_equal(d_o.cpu().numpy().view(np.uint16).reshape(n, 128), want.view(np.uint16)):
            failures.append((it, "decompress"))
        # fused GEMV on a [rows][k] view of the same blocks
        kb = int(rng.choice([1, 2, 8]))
        rows = n // kb
        if rows >= 1:
            batch, k = int(rng.integers(1, 9)), kb * 128
            xx = synth.activations(batch, k, 5 + it)
            y = torch.full((batch, rows), float("nan"), dtype=torch.float32, device="cuda")
            wsb = B.ecco_gemv_workspace_bytes(rows, k, batch)
            ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
            B.ecco_gemv(d_meta, d_b, rows, k, dev(xx), batch, y, ws, wsb)
            ref, refabs = eo.gemv(m, blocks[: rows * kb], rows, k, xx, batch)
            ok, worst = fused_ok(y.cpu().numpy().astype(np.float64), ref, refabs, "random gemv")
            if not ok:
                failures.append((it, "gemv", batch, worst))
        # several matrices in one ecco_gemv_batch call: the same blocks cut into up to four matrices of random shapes
        if n >= 33 and it % 2 == 0:
            batch = int(rng.integers(1, 9))
            parts, at = [], 0
            while at < n and len(parts) < 4:
                kbp = int(rng.choice([1, 2, 4]))
                rows_p = int(rng.integers(1, max(2, (n - at) // kbp // 2 + 2)))
                if rows_p * kbp > n - at or (at * 64) % 16:
                    break
                parts.append((at, rows_p, kbp))
                at += rows_p * kbp
            items, checks = [], []
            for (g0, rows_p, kbp) in parts:
                xx = synth.activations(batch, kbp * 128, 31 + it + g0)
                yb = torch.full((batch, rows_p), float("nan"), dtype=torch.float32, device="cuda")
                items.append((d_meta, d_b[g0:], rows_p, kbp * 128, dev(xx), yb))
                checks.append((blocks[g0: g0 + rows_p * kbp], rows_p, kbp * 128, xx, yb))
            if items:
                wsb = B.ecco_gemv_batch_workspace_bytes(items, batch)
                ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
                B.ecco_gemv_batch(items, batch, ws, wsb)
                for blk, rows_p, kk, xx, yb in checks:
                    ref, refabs = eo.gemv(m, blk, rows_p, kk, xx, batch)
                    ok, worst = fused_ok(yb.cpu().numpy().astype(np.float64), ref, refabs, "random gemv batch")
                    if not ok:
                        failures.append((it, "gemv_batch", batch, rows_p, kk, worst))
        # attention scores and attention output on a [batch][heads][seq] view
        heads = int(rng.choice([1, 2, 3]))
        seq = n // heads
        if seq >= 1:
            qpk = int(rng.integers(1, 9))
            q = synth.queries(1, heads * qpk, 9 + it)
            sc = torch.full((1, heads * qpk, seq), float("nan"), dtype=torch.float32, device="cuda")
            B.ecco_attn_scores(d_meta, d_b, 1, heads, seq, qpk, dev(q), 0.0884, sc)
            ref, refabs = eo.attn_scores(m, blocks[: heads * seq], 1, heads, seq, qpk, q, 0.0884)
            ok, worst = fused_ok(sc.cpu().numpy().astype(np.float64), ref, refabs, "random scores")
            if not ok:
                failures.append((it, "scores", qpk, worst))
            logits = (rng.standard_normal((1, heads * qpk, seq)) * 2.0).astype(np.float32)
            out = torch.full((1, heads * qpk, 128), float("nan"), dtype=torch.float32, device="cuda")
            avb = B.ecco_attn_values_workspace_bytes(1, heads, seq, qpk)
            avws = torch.empty(avb, dtype=torch.uint8, device="cuda")
            B.ecco_attn_values(d_meta, d_b, 1, heads, seq, qpk, dev(logits), out, avws, avb)
            ref, refabs = eo.attn_values(m, blocks[: heads * seq], 1, heads, seq, qpk, logits)
            floor = np.abs(eo.decode(m, blocks[: heads * seq]).astype(np.float64)).reshape(heads, seq, 128).sum(axis=1) * 2.0 ** -38
            err = np.abs(out.cpu().numpy().astype(np.float64) - ref)
            bound = TOL * refabs + np.repeat(floor, qpk, axis=0)[None]
            if not np.all(err <= bound + 1e-30):
                failures.append((it, "values", qpk, float((err / (bound + 1e-30)).max())))
        # online KV compressor and the variable-length container, on encoded data
        if x is not None:
            d_c = torch.zeros((n, 64), dtype=torch.uint8, device="cuda")
            B.ecco_kv_compress(d_meta, dev(x.view(np.uint16).reshape(-1)), n, d_c)
            want_c, _ = eo.encode(m, x, eo.SELECT_MINMAX)
            if not np.array_equal(d_c.cpu().numpy(), want_c):
                failures.append((it, "kv_compress"))
            stream, index, total = B.ecco_var_encode_host(lm, x, B.SELECT_MSE | B.KEEP_EXPONENT)
            want_stream, want_off = eo.var_encode(m, x, eo.SELECT_MSE)
            d_v = torch.full((n, 128), float("nan"), dtype=torch.float16, device="cuda")
            B.ecco_var_decompress(d_meta, dev(stream), dev(index), n, d_v)
            if not np.array_equal(d_v.cpu().numpy().view(np.uint16), eo.var_decode(m, want_stream, want_off).view(np.uint16)):
                failures.append((it, "var_decompress"))
        # 2x activation codec: compress real values, decompress arbitrary bytes
        ng = int(rng.choice([1, 9, 700]))
        a = (rng.standard_normal((ng, 64)) * rng.choice([1e-4, 1.0, 1e3])).astype(np.float16)
        d_ab = torch.zeros((ng, 64), dtype=torch.uint8, device="cuda")
        B.ecco_act_compress(dev(a), ng, d_ab)
        if not np.array_equal(d_ab.cpu().numpy(), eo.act_encode(a)):
            failures.append((it, "act_compress"))
        rb = synth.random_blocks(ng, 300 + it)
        d_ao = torch.zeros((ng, 64), dtype=torch.float16, device="cuda")
        B.ecco_act_decompress(dev(rb), ng, d_ao)
        want_a = eo.act_decode(rb)
        finite = np.isfinite(want_a.astype(np.float32))
        if not np.array_equal(d_ao.cpu().numpy().view(np.uint16)[finite], want_a.view(np.uint16)[finite]):
            failures.append((it, "act_decompress"))
        torch.cuda.synchronize()
        assert B.ecco_device_status() == 0
    assert not failures, failures[:10]


def test_random_call_sequences_keep_stream_order(B, eo, kv_small, cfg1_small, synth):
    """10 to 30 dependent calls issued back to back against the same calls with a synchronisation after each one."""
    km, wm = B.meta_to_device(lib_meta_from_oracle(B, kv_small["meta"])), B.meta_to_device(lib_meta_from_oracle(B, cfg1_small["meta"]))
    reps = 16
    N = 2048 * reps
    kblocks, wblocks = np.tile(kv_small["blocks"], (reps, 1)), np.tile(cfg1_small["blocks"], (reps, 1))
    src = [dev(kblocks), dev(wblocks), dev(np.ascontiguousarray(wblocks[::-1]))]
    metas = [km, wm, wm]
    xk = dev(np.tile(kv_small["k"].reshape(-1, 128), (reps, 1)).reshape(-1))
    n_out, k = 1024, 4096                                   # 32768 groups as a matrix
    heads, seq = 8, 4096
    x1, x8, q = dev(synth.activations(1, k, 3)), dev(synth.activations(8, k, 4)), dev(synth.queries(1, heads, 5))
    wsb = max(B.ecco_gemv_workspace_bytes(n_out, k, 8), B.ecco_gemv_workspace_bytes(n_out, k, 1))
    avb = B.ecco_attn_values_workspace_bytes(1, heads, seq, 1)

    def fresh():
        return dict(out=[torch.zeros(N * 128, dtype=torch.float16, device="cuda") for _ in range(3)],
                    blk=[torch.zeros((N, 64), dtype=torch.uint8, device="cuda") for _ in range(2)],
                    y=[torch.zeros((8, n_out), dtype=torch.float32, device="cuda") for _ in range(3)],
                    sc=torch.zeros((1, heads, seq), dtype=torch.float32, device="cuda"),
                    av=torch.zeros((1, heads, 128), dtype=torch.float32, device="cuda"),
                    ws=torch.zeros(wsb, dtype=torch.uint8, device="cuda"), avws=torch.zeros(avb, dtype=torch.uint8, device="cuda"))

    def run(prog, st, sync):
        for op in prog:
            kind = op[0]
            if kind == "dec":
                B.ecco_decompress(metas[op[1]], src[op[1]], N, st["out"][op[2]])
            elif kind == "decblk":                           # reads what the compressor wrote
                B.ecco_decompress(km, st["blk"][op[1]], N, st["out"][op[2]])
            elif kind == "kvc":
                B.ecco_kv_compress(km, xk, N, st["blk"][op[1]])
            elif kind == "batch":
                B.ecco_decompress_batch([(metas[i], src[i], N, st["out"][j]) for i, j in op[1]])
            elif kind == "gemv":
                B.ecco_gemv(wm, src[1 + op[1]], n_out, k, x1 if op[2] == 1 else x8, op[2], st["y"][op[3]][: op[2]], st["ws"], wsb)
            elif kind == "attn":
                B.ecco_attn_scores(km, src[0], 1, heads, seq, 1, q, 0.0884, st["sc"])
            elif kind == "attnv":
                B.ecco_attn_values(km, src[0], 1, heads, seq, 1, st["sc"], st["av"], st["avws"], avb)
            elif kind == "fill":                             # a kernel of someone else in between
                st["out"][op[1]].fill_(1.0)
            if sync:
                torch.cuda.synchronize()
        torch.cuda.synchronize()

    bad = []
    for it in range(N_SEQUENCES):
        rng = np.random.Generator(np.random.PCG64(123_000 + it))
        prog = []
        for _ in range(int(rng.integers(10, 30))):
            kind = rng.choice(["dec", "decblk", "kvc", "batch", "gemv", "attn", "attnv", "fill"], p=[.25, .1, .1, .1, .2, .08, .1, .07])
            if kind == "dec":
                prog.append(("dec", int(rng.integers(3)), int(rng.integers(3))))
            elif kind == "decblk":
                prog.append(("decblk", int(rng.integers(2)), int(rng.integers(3))))
            elif kind == "kvc":
                prog.append(("kvc", int(rng.integers(2))))
            elif kind == "batch":                            # independent items: distinct outputs
                outs = rng.permutation(3)[: int(rng.integers(1, 4))]
                prog.append(("batch", [(int(rng.integers(3)), int(j)) for j in outs]))
            elif kind == "gemv":
                prog.append(("gemv", int(rng.integers(2)), int(rng.choice([1, 8])), int(rng.integers(3))))
            elif kind == "fill":
                prog.append(("fill", int(rng.integers(3))))
            else:
                prog.append((str(kind),))
        a, b = fresh(), fresh()
        run(prog, a, True)
        run(prog, b, False)
        assert B.ecco_device_status() == 0
        for name in ("out", "blk", "y"):
            for i, (u, v) in enumerate(zip(a[name], b[name])):
                if not torch.equal(u.view(torch.uint8), v.view(torch.uint8)):
                    bad.append((it, name, i))
        for name in ("sc", "av"):
            if not torch.equal(a[name], b[name]):
                bad.append((it, name))
    assert not bad, bad[:10]
