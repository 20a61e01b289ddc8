"""Pins of the oracle's prefix codes: Kraft equality, prefix-freeness, optimality against a
textbook Huffman construction and against brute force, the entropy bound."""
import heapq
import itertools

import numpy as np
import pytest


def textbook_huffman_lengths(freq):
    """Unconstrained Huffman (heap of subtrees); returns the multiset-optimal lengths."""
    heap = [(f, i, [i]) for i, f in enumerate(freq)]
    heapq.heapify(heap)
    ln = [0] * len(freq)
    tick = len(freq)
    while len(heap) > 1:
        a = heapq.heappop(heap)
        b = heapq.heappop(heap)
        for s in a[2] + b[2]:
            ln[s] += 1
        heapq.heappush(heap, (a[0] + b[0], tick, a[2] + b[2]))
        tick += 1
    return ln


def is_prefix_free(codes, lens):
    words = [format(int(c), "b").zfill(int(l)) for c, l in zip(codes, lens)]
    for i, a in enumerate(words):
        for j, b in enumerate(words):
            if i != j and b.startswith(a):
                return False
    return True


def test_canonical_code_order_and_worked_example(eo):
    # the code used by the worked block example: lengths 2,2,3,3,3,4,6,7,7,7,8x6
    lens = [2, 2, 3, 3, 3, 4, 6, 7, 7, 7, 8, 8, 8, 8, 8, 8]
    codes, kraft = eo.canonical_codes(lens, 8)
    assert kraft == 256
    words = [format(int(c), "b").zfill(l) for c, l in zip(codes, lens)]
    assert words[:10] == ["00", "01", "100", "101", "110", "1110", "111100", "1111010", "1111011", "1111100"]
    assert words[10:] == ["11111010", "11111011", "11111100", "11111101", "11111110", "11111111"]
    assert is_prefix_free(codes, lens)
    # the ID_KP code of the example
    kcodes, kk = eo.canonical_codes([2, 2, 3, 3, 3, 3], 12)
    assert kk == 4096
    assert [format(int(c), "b").zfill(l) for c, l in zip(kcodes, [2, 2, 3, 3, 3, 3])] == ["00", "01", "100", "101", "110", "111"]


@pytest.mark.parametrize("seed", range(12))
def test_huffman_2_8_kraft_prefix_and_optimality(eo, seed):
    rng = np.random.Generator(np.random.PCG64(100 + seed))
    kind = seed % 4
    if kind == 0:
        f = rng.dirichlet(np.ones(16))
    elif kind == 1:
        f = rng.dirichlet(np.ones(16) * 0.2)          # skewed, some near-zero symbols
    elif kind == 2:
        f = np.exp(-0.5 * ((np.arange(16) - 7) / 2.0) ** 2); f[15] = 1 / 128; f /= f.sum()  # bell-shaped indices
    else:
        f = rng.integers(0, 5, 16).astype(float); f[0] += 1; f /= f.sum()   # ties and zeros
    ln = eo.huffman_2_8(f)
    assert ln.min() >= 2 and ln.max() <= 8
    codes, kraft = eo.canonical_codes(ln, 8)
    assert kraft == 256                                 # Kraft equality
    assert is_prefix_free(codes, ln)
    cost = float(np.dot(f, ln))
    tb = textbook_huffman_lengths(f.tolist())
    tb_cost = float(np.dot(f, tb))
    assert cost >= tb_cost - 1e-12                      # nothing beats unconstrained Huffman
    if min(tb) >= 2 and max(tb) <= 8:
        assert abs(cost - tb_cost) < 1e-12              # and it is reached when it is admissible
    # more frequent symbols never get longer codes
    for a in range(16):
        for b in range(16):
            if f[a] > f[b]:
                assert ln[a] <= ln[b]
    # entropy bound: mean length < H + 1 (the floor of 2 bits lifts it to max(2, .) + ...)
    p = f[f > 0]
    H = float(-(p * np.log2(p)).sum())
    if min(tb) >= 2 and max(tb) <= 8:
        assert cost < H + 1
    assert cost >= H - 1e-12


def test_huffman_2_8_is_optimal_among_all_admissible_length_vectors(eo):
    """Brute force over every multiset of lengths in [2,8] with Kraft sum 1 (the search space the
    oracle claims to cover), re-enumerated independently with itertools."""
    vectors = []
    for n in itertools.product(range(5), range(9), range(17), range(17), range(17)):
        if sum(n) > 16:
            continue
        rest = 16 - sum(n)
        k = n[0] * 64 + n[1] * 32 + n[2] * 16 + n[3] * 8 + n[4] * 4
        # n7 codes worth 2, n8 worth 1: n7 + n8 = rest, 2 n7 + n8 = 256 - k
        n7 = 256 - k - rest
        n8 = rest - n7
        if n7 < 0 or n8 < 0:
            continue
        vectors.append(sum(([L] * c for L, c in zip(range(2, 9), list(n) + [n7, n8])), []))
    assert len(vectors) > 100
    rng = np.random.Generator(np.random.PCG64(5))
    V = np.array(vectors, dtype=np.float64)             # each row ascending lengths
    for trial in range(20):
        f = rng.dirichlet(np.ones(16) * (0.15 if trial % 2 else 1.0))
        fs = np.sort(f)[::-1]
        best = (V @ fs).min()
        got = float(np.dot(f, eo.huffman_2_8(f)))
        assert abs(got - best) < 1e-12


def brute_force_limited(freq, maxlen):
    n = len(freq)
    best = None
    for ln in itertools.product(range(1, maxlen + 1), repeat=n):
        if sum(2.0 ** -l for l in ln) <= 1.0 + 1e-12:
            c = sum(f * l for f, l in zip(freq, ln))
            if best is None or c < best - 1e-12:
                best = c
    return best


@pytest.mark.parametrize("n,maxlen", [(2, 1), (3, 2), (4, 2), (4, 3), (5, 3), (5, 4), (6, 3), (6, 4), (7, 3)])
def test_package_merge_against_brute_force(eo, n, maxlen):
    rng = np.random.Generator(np.random.PCG64(n * 10 + maxlen))
    for trial in range(6):
        f = rng.dirichlet(np.ones(n) * (0.3 if trial % 2 else 1.0)) if trial < 5 else np.ones(n)
        ln = eo.huffman_limited(f, maxlen)
        assert ln.min() >= 1 and ln.max() <= maxlen
        _, kraft = eo.canonical_codes(ln, maxlen)
        assert kraft == (1 << maxlen)                   # complete
        assert abs(float(np.dot(f, ln)) - brute_force_limited(f.tolist(), maxlen)) < 1e-12


def test_package_merge_equals_textbook_huffman_when_the_limit_is_slack(eo):
    rng = np.random.Generator(np.random.PCG64(77))
    for trial in range(20):
        n = int(rng.integers(2, 65))
        f = rng.dirichlet(np.ones(n)) + 1e-3
        tb = textbook_huffman_lengths(f.tolist())
        ln = eo.huffman_limited(f, 12)
        _, kraft = eo.canonical_codes(ln, 12)
        assert kraft == 4096 and ln.max() <= 12
        if max(tb) <= 12:
            assert abs(float(np.dot(f, ln)) - float(np.dot(f, tb))) < 1e-9
    # a Fibonacci-like distribution forces the limit to bind
    f = np.array([1.6 ** i for i in range(20)])
    tb = textbook_huffman_lengths(f.tolist())
    assert max(tb) > 12
    ln = eo.huffman_limited(f, 12)
    _, kraft = eo.canonical_codes(ln, 12)
    assert ln.max() == 12 and kraft == 4096
    assert float(np.dot(f, ln)) >= float(np.dot(f, tb))


def test_every_code_of_a_calibrated_metadata_is_complete_and_in_range(eo, cfg1_small):
    meta = cfg1_small["meta"]
    assert eo.meta_check(meta) == 0
    cb = meta.cb_lengths()
    assert cb.shape == (64, 4, 16) and cb.min() >= 2 and cb.max() <= 8
    for k in range(meta.S):
        for h in range(4):
            codes, kraft = eo.canonical_codes(cb[k, h], 8)
            assert kraft == 256 and is_prefix_free(codes, cb[k, h])
    kl = meta.kp_lengths()
    codes, kraft = eo.canonical_codes(kl, 12)
    assert kraft == 4096 and kl.min() >= 1 and kl.max() <= 12 and is_prefix_free(codes, kl)
    # paper's consistency numbers: lengths 2..8 -> 1..4 symbols per 8 stream bits, 7-bit overlap
    assert 8 // cb.max() == 1 and 8 // cb.min() == 4 and cb.max() - 1 == 7
