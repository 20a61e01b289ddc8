"""ctypes front end of the plain C oracle in ``ecco_oracle.c``.

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's cpu_baseline /
reference arm import this; the library under ``paper_2505_06901_b200`` never does, and this
module imports nothing from the library.  All arithmetic lives in the C file; this module
only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ecco_oracle.c")
_LIB = os.path.join(_HERE, "libecco_oracle.so")

G = 128
BLOCK = 64
MAXS = 64
SELECT_MSE = 0
SELECT_MINMAX = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C99, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-Wall", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


class Meta(C.Structure):
    _fields_ = [
        ("S", C.c_int32),
        ("H", C.c_int32),
        ("e", C.c_int32),
        ("reserved", C.c_int32),
        ("pattern", (C.c_uint16 * 16) * MAXS),
        ("cb_len", ((C.c_uint8 * 16) * 4) * MAXS),
        ("kp_len", C.c_uint8 * MAXS),
    ]

    def patterns(self) -> np.ndarray:
        """[S][15] fp16 patterns."""
        a = np.ctypeslib.as_array(self.pattern).view(np.float16)
        return a[: self.S, :15].copy()

    def cb_lengths(self) -> np.ndarray:
        return np.ctypeslib.as_array(self.cb_len)[: self.S].copy()

    def kp_lengths(self) -> np.ndarray:
        return np.ctypeslib.as_array(self.kp_len)[: self.S].copy()

    def copy(self) -> "Meta":
        m = Meta()
        C.memmove(C.byref(m), C.byref(self), C.sizeof(Meta))
        return m


class Stats(C.Structure):
    _fields_ = [
        ("n_groups", C.c_uint64),
        ("clipped_groups", C.c_uint64),
        ("clipped_values", C.c_uint64),
        ("padded_groups", C.c_uint64),
        ("padded_values", C.c_uint64),
        ("total_bits", C.c_uint64),
        ("kp_usage", C.c_uint64 * MAXS),
        ("hf_usage", C.c_uint64 * 4),
        ("sym_count", C.c_uint64 * 16),
    ]


class GroupInfo(C.Structure):
    _fields_ = [
        ("pstar", C.c_int32),
        ("kp", C.c_int32),
        ("hf", C.c_int32),
        ("n_fit", C.c_int32),
        ("n_pad", C.c_int32),
        ("end_bit", C.c_int32),
        ("qs", C.c_uint8),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        L.eo_fp16_to_f32.restype = C.c_float
        L.eo_fp16_to_f32.argtypes = [C.c_uint16]
        L.eo_f32_to_fp16.restype = C.c_uint16
        L.eo_f32_to_fp16.argtypes = [C.c_float]
        L.eo_e4m3_to_f32.restype = C.c_float
        L.eo_e4m3_to_f32.argtypes = [C.c_uint8]
        L.eo_e4m3_from_f32.restype = C.c_uint8
        L.eo_e4m3_from_f32.argtypes = [C.c_float]
        L.eo_kmeans1d.restype = C.c_double
        assert L.eo_sizeof_meta() == C.sizeof(Meta)
        assert L.eo_sizeof_stats() == C.sizeof(Stats)
        assert L.eo_sizeof_info() == C.sizeof(GroupInfo)
    return _lib


def _p(a: np.ndarray, t):
    return a.ctypes.data_as(C.POINTER(t))


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def _u16(x) -> np.ndarray:
    x = np.ascontiguousarray(x)
    if x.dtype == np.float16:
        x = x.view(np.uint16)
    assert x.dtype == np.uint16
    return x


# ---------------------------------------------------------------- number formats
def fp16_to_f32(h: int) -> float:
    return float(lib().eo_fp16_to_f32(int(h)))


def f32_to_fp16(f: float) -> int:
    return int(lib().eo_f32_to_fp16(C.c_float(f)))


def e4m3_to_f32(b: int) -> float:
    return float(lib().eo_e4m3_to_f32(int(b)))


def e4m3_from_f32(f: float) -> int:
    return int(lib().eo_e4m3_from_f32(C.c_float(f)))


# ---------------------------------------------------------------- codes
def canonical_codes(lengths, maxlen: int):
    ln = np.ascontiguousarray(lengths, dtype=np.uint8)
    code = np.zeros(len(ln), dtype=np.uint16)
    kraft = C.c_uint32(0)
    lib().eo_canonical_codes(_p(ln, C.c_uint8), len(ln), maxlen, _p(code, C.c_uint16), C.byref(kraft))
    return code, kraft.value


def huffman_2_8(freq) -> np.ndarray:
    f = np.ascontiguousarray(freq, dtype=np.float64)
    assert f.shape == (16,)
    ln = np.zeros(16, dtype=np.uint8)
    _check(lib().eo_huffman_2_8(_p(f, C.c_double), _p(ln, C.c_uint8)), "huffman_2_8")
    return ln


def huffman_limited(freq, maxlen: int) -> np.ndarray:
    f = np.ascontiguousarray(freq, dtype=np.float64)
    ln = np.zeros(len(f), dtype=np.uint8)
    _check(lib().eo_huffman_limited(_p(f, C.c_double), len(f), maxlen, _p(ln, C.c_uint8)), "huffman_limited")
    return ln


# ---------------------------------------------------------------- clustering
def kmeans1d(v, k: int, w=None):
    v = np.ascontiguousarray(v, dtype=np.float64)
    assert np.all(np.diff(v) >= 0)
    cen = np.zeros(k, dtype=np.float64)
    wp = None
    if w is not None:
        w = np.ascontiguousarray(w, dtype=np.float64)
        wp = _p(w, C.c_double)
    cost = lib().eo_kmeans1d(_p(v, C.c_double), wp, len(v), k, _p(cen, C.c_double))
    return cen, float(cost)


def lloyd(x, k: int, seed: int, max_iter: int):
    x = np.ascontiguousarray(x, dtype=np.float64)
    n, d = x.shape
    cen = np.zeros((k, d), dtype=np.float64)
    assign = np.zeros(n, dtype=np.int32)
    trace = np.zeros(max_iter + 1, dtype=np.float64)
    it = lib().eo_lloyd(_p(x, C.c_double), n, d, k, C.c_uint64(seed), max_iter, _p(cen, C.c_double),
                        _p(assign, C.c_int32), _p(trace, C.c_double))
    return cen, assign, trace, it


def group_pattern(x16, e: int, weights=None) -> np.ndarray:
    x = _u16(x16)
    pat = np.zeros(15, dtype=np.float64)
    wp = None
    if weights is not None:
        weights = np.ascontiguousarray(weights, dtype=np.float32)
        wp = _p(weights, C.c_float)
    _check(lib().eo_group_pattern(_p(x, C.c_uint16), e, wp, _p(pat, C.c_double)), "group_pattern")
    return pat


# ---------------------------------------------------------------- codec
def calibrate(calib16, S: int = 64, H: int = 4, seed: int = 1, select: int = SELECT_MSE, weights=None,
              lloyd_iters: int = 30) -> Meta:
    x = _u16(calib16).reshape(-1)
    assert x.size % G == 0
    m = Meta()
    wp = None
    if weights is not None:
        weights = np.ascontiguousarray(weights, dtype=np.float32)
        assert weights.shape == (G,)
        wp = _p(weights, C.c_float)
    _check(lib().eo_calibrate(_p(x, C.c_uint16), C.c_uint64(x.size // G), wp, S, H, C.c_uint64(seed), select,
                              lloyd_iters, C.byref(m)), "calibrate")
    return m


def set_exponent(meta: Meta, x16) -> None:
    x = _u16(x16).reshape(-1)
    _check(lib().eo_set_exponent(C.byref(meta), _p(x, C.c_uint16), C.c_uint64(x.size)), "set_exponent")


def meta_check(meta: Meta) -> int:
    return int(lib().eo_meta_check(C.byref(meta)))


def quantize_group(meta: Meta, x16, select: int = SELECT_MSE):
    x = _u16(x16).reshape(-1)
    assert x.size == G
    u = np.zeros(G, dtype=np.float32)
    sym = np.zeros(G, dtype=np.uint8)
    p = C.c_int32()
    kp = C.c_int32()
    qs = C.c_uint8()
    err = C.c_double()
    _check(lib().eo_quantize_group(C.byref(meta), _p(x, C.c_uint16), select, C.byref(p), C.byref(qs),
                                   _p(u, C.c_float), C.byref(kp), _p(sym, C.c_uint8), C.byref(err)), "quantize_group")
    return dict(pstar=p.value, qs=qs.value, u=u, kp=kp.value, sym=sym, err=err.value)


def encode(meta: Meta, x16, select: int = SELECT_MSE):
    """-> (blocks uint8 [n_groups][64], Stats)."""
    x = _u16(x16).reshape(-1)
    assert x.size % G == 0
    n = x.size // G
    blocks = np.zeros((n, BLOCK), dtype=np.uint8)
    st = Stats()
    _check(lib().eo_encode(C.byref(meta), _p(x, C.c_uint16), C.c_uint64(n), select, _p(blocks, C.c_uint8),
                           C.byref(st)), "encode")
    return blocks, st


def encode_group(meta: Meta, x16, select: int = SELECT_MSE):
    x = _u16(x16).reshape(-1)
    assert x.size == G
    blk = np.zeros(BLOCK, dtype=np.uint8)
    sym = np.zeros(G, dtype=np.uint8)
    info = GroupInfo()
    _check(lib().eo_encode_group(C.byref(meta), _p(x, C.c_uint16), select, _p(blk, C.c_uint8), _p(sym, C.c_uint8),
                                 C.byref(info)), "encode_group")
    return blk, sym, info


def decode_block(meta: Meta, blk):
    blk = np.ascontiguousarray(blk, dtype=np.uint8).reshape(-1)
    assert blk.size == BLOCK
    out = np.zeros(G, dtype=np.uint16)
    sym = np.zeros(G, dtype=np.uint8)
    info = GroupInfo()
    _check(lib().eo_decode_block(C.byref(meta), _p(blk, C.c_uint8), _p(out, C.c_uint16), _p(sym, C.c_uint8),
                                 C.byref(info)), "decode_block")
    return out.view(np.float16), sym, info


def decode(meta: Meta, blocks, out=None) -> np.ndarray:
    """-> fp16 [n_groups][128].  Single-threaded, block by block."""
    b = np.ascontiguousarray(blocks, dtype=np.uint8).reshape(-1, BLOCK)
    n = b.shape[0]
    if out is None:
        out = np.zeros((n, G), dtype=np.uint16)
    _check(lib().eo_decode(C.byref(meta), _p(b, C.c_uint8), C.c_uint64(n), _p(out, C.c_uint16)), "decode")
    return out.view(np.float16)


def decode_threads(meta: Meta, blocks, threads: int) -> np.ndarray:
    """The same decoder called on disjoint ranges of groups from `threads` Python threads
    (ctypes drops the GIL during the call).  Used to keep large parity checks and the timed
    CPU baseline short; the arithmetic is unchanged."""
    from concurrent.futures import ThreadPoolExecutor

    b = np.ascontiguousarray(blocks, dtype=np.uint8).reshape(-1, BLOCK)
    n = b.shape[0]
    out = np.zeros((n, G), dtype=np.uint16)
    threads = max(1, min(threads, n))
    bounds = [n * i // threads for i in range(threads + 1)]

    def work(i):
        lo, hi = bounds[i], bounds[i + 1]
        if hi > lo:
            _check(lib().eo_decode(C.byref(meta), _p(b[lo:hi], C.c_uint8), C.c_uint64(hi - lo),
                                   _p(out[lo:hi], C.c_uint16)), "decode")

    with ThreadPoolExecutor(threads) as ex:
        list(ex.map(work, range(threads)))
    return out.view(np.float16)


def gemv(meta: Meta, blocks, n_out: int, k: int, x16, batch: int):
    """-> (y fp64 [batch][n_out], sum|w x| fp64 [batch][n_out])."""
    b = np.ascontiguousarray(blocks, dtype=np.uint8).reshape(-1)
    assert b.size == n_out * (k // G) * BLOCK
    x = _u16(x16).reshape(-1)
    assert x.size == batch * k
    y = np.zeros((batch, n_out), dtype=np.float64)
    ya = np.zeros((batch, n_out), dtype=np.float64)
    _check(lib().eo_gemv(C.byref(meta), _p(b, C.c_uint8), n_out, k, _p(x, C.c_uint16), batch, _p(y, C.c_double),
                         _p(ya, C.c_double)), "gemv")
    return y, ya


def attn_scores(meta: Meta, kblocks, batch: int, n_kv_heads: int, seq: int, q_per_kv: int, q16, scale: float):
    """-> (scores fp64 [batch][n_kv_heads*q_per_kv][seq], scale*sum|q k| of the same shape)."""
    b = np.ascontiguousarray(kblocks, dtype=np.uint8).reshape(-1)
    assert b.size == batch * n_kv_heads * seq * BLOCK
    q = _u16(q16).reshape(-1)
    nq = n_kv_heads * q_per_kv
    assert q.size == batch * nq * G
    s = np.zeros((batch, nq, seq), dtype=np.float64)
    sa = np.zeros((batch, nq, seq), dtype=np.float64)
    _check(lib().eo_attn_scores(C.byref(meta), _p(b, C.c_uint8), batch, n_kv_heads, seq, q_per_kv, _p(q, C.c_uint16),
                                C.c_double(scale), _p(s, C.c_double), _p(sa, C.c_double)), "attn_scores")
    return s, sa


# ---------------------------------------------------------------- 2x activation format
ACT_G = 64


def act_encode(x16) -> np.ndarray:
    """fp16 [n_groups*64] -> uint8 [n_groups][64]."""
    x = _u16(x16).reshape(-1)
    assert x.size % ACT_G == 0
    n = x.size // ACT_G
    blocks = np.zeros((n, 64), dtype=np.uint8)
    _check(lib().eo_act_encode(_p(x, C.c_uint16), C.c_uint64(n), _p(blocks, C.c_uint8)), "act_encode")
    return blocks


def act_decode(blocks) -> np.ndarray:
    """uint8 [n_groups][64] -> fp16 [n_groups][64]."""
    b = np.ascontiguousarray(blocks, dtype=np.uint8).reshape(-1, 64)
    out = np.zeros((b.shape[0], ACT_G), dtype=np.uint16)
    lib().eo_act_decode(_p(b, C.c_uint8), C.c_uint64(b.shape[0]), _p(out, C.c_uint16))
    return out.view(np.float16)


def attn_values(meta: Meta, vblocks, batch: int, n_kv_heads: int, seq: int, q_per_kv: int, scores):
    """softmax(scores) . V~ -> (out fp64 [batch][n_kv_heads*q_per_kv][128], sum_t p_t |V~| of the same shape)."""
    b = np.ascontiguousarray(vblocks, dtype=np.uint8).reshape(-1)
    assert b.size == batch * n_kv_heads * seq * BLOCK
    s = np.ascontiguousarray(scores, dtype=np.float32)
    nq = n_kv_heads * q_per_kv
    assert s.shape == (batch, nq, seq)
    out = np.zeros((batch, nq, G), dtype=np.float64)
    oa = np.zeros((batch, nq, G), dtype=np.float64)
    _check(lib().eo_attn_values(C.byref(meta), _p(b, C.c_uint8), batch, n_kv_heads, seq, q_per_kv, _p(s, C.c_float),
                                _p(out, C.c_double), _p(oa, C.c_double)), "attn_values")
    return out, oa


# ---------------------------------------------------------------- variable-length container
VAR_MAX_BITS = 10 + 12 + 128 * 8


def var_encode(meta: Meta, x16, select: int = SELECT_MSE):
    """-> (stream uint8, offsets uint64 [n_groups + 1]) : the groups' fields back to back, nothing clipped or padded."""
    x = _u16(x16).reshape(-1)
    assert x.size % G == 0
    n = x.size // G
    stream = np.zeros((n * VAR_MAX_BITS + 7) // 8 + 8, dtype=np.uint8)
    offsets = np.zeros(n + 1, dtype=np.uint64)
    _check(lib().eo_var_encode(C.byref(meta), _p(x, C.c_uint16), C.c_uint64(n), select, _p(stream, C.c_uint8),
                               _p(offsets, C.c_uint64)), "var_encode")
    return stream[: (int(offsets[n]) + 7) // 8].copy(), offsets


def var_decode(meta: Meta, stream, offsets) -> np.ndarray:
    s = np.ascontiguousarray(stream, dtype=np.uint8)
    o = np.ascontiguousarray(offsets, dtype=np.uint64)
    n = o.size - 1
    assert (int(o[n]) + 7) // 8 <= s.size
    out = np.zeros((n, G), dtype=np.uint16)
    _check(lib().eo_var_decode(C.byref(meta), _p(s, C.c_uint8), _p(o, C.c_uint64), C.c_uint64(n), _p(out, C.c_uint16)), "var_decode")
    return out.view(np.float16)
