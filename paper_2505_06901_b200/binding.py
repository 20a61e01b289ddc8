"""Thin ctypes binding of the C ABI declared in include/ecco.h: argument marshalling only.

Every step of the hot path runs inside libecco_b200.so; there is no Python or CPU fallback.
Device buffers are torch tensors (torch is used for device memory and streams only) and travel
as raw pointers; host buffers are numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

GROUP = 128
BLOCK_BYTES = 64
MAX_PATTERNS = 64
SELECT_MSE = 0
SELECT_MINMAX = 1
KEEP_EXPONENT = 2

ECCO_OK = 0
ERR_INVALID_ARG = -1
ERR_ALIGNMENT = -2
ERR_NONFINITE_INPUT = -3
ERR_BAD_META = -4
ERR_UNSUPPORTED_ARCH = -5
ERR_CUDA = -6
ERR_WORKSPACE = -7
ERR_DEVICE_TIMEOUT = -8

EXPORTS = [
    "ecco_calibrate_host", "ecco_meta_create", "ecco_meta_get", "ecco_meta_free", "ecco_encode_host",
    "ecco_meta_device_bytes", "ecco_meta_serialize_device", "ecco_decompress", "ecco_decompress_batch", "ecco_gemv_workspace_bytes",
    "ecco_gemv", "ecco_gemv_batch_workspace_bytes", "ecco_gemv_batch", "ecco_gemv_static_ws", "ecco_attn_scores", "ecco_act_compress", "ecco_act_decompress",
    "ecco_attn_values_workspace_bytes", "ecco_attn_values", "ecco_kv_compress",
    "ecco_var_stream_bytes_bound", "ecco_var_index_bytes", "ecco_var_encode_host", "ecco_var_decompress", "ecco_error_string", "ecco_last_cuda_error", "ecco_device_status",
    "ecco_kernel_launch_count", "ecco_test_wait_timeout",
]


class DecompressItem(C.Structure):
    """ecco_decompress_item of include/ecco.h."""
    _fields_ = [("d_meta", C.c_void_p), ("d_blocks", C.c_void_p), ("n_groups", C.c_uint64), ("d_out_fp16", C.c_void_p)]


class GemvItem(C.Structure):
    """ecco_gemv_item of include/ecco.h."""
    _fields_ = [("d_meta", C.c_void_p), ("d_blocks", C.c_void_p), ("n_out", C.c_int32), ("k", C.c_int32),
                ("d_x_fp16", C.c_void_p), ("d_y", C.c_void_p)]


class EccoError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        msg = lib().ecco_error_string(code).decode()
        if code == ERR_CUDA:
            msg += f" [cudaError {lib().ecco_last_cuda_error()}]"
        super().__init__(f"{what}: {msg} ({code})")


class Params(C.Structure):
    _fields_ = [("S", C.c_int32), ("H", C.c_int32), ("seed", C.c_uint64), ("select", C.c_uint32),
                ("kmeans_iters", C.c_int32), ("max_groups", C.c_uint64), ("threads", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("n_groups", C.c_uint64), ("clipped_groups", C.c_uint64), ("clipped_values", C.c_uint64),
                ("padded_groups", C.c_uint64), ("padded_values", C.c_uint64), ("total_bits", C.c_uint64),
                ("kp_usage", C.c_uint64 * MAX_PATTERNS), ("hf_usage", C.c_uint64 * 4), ("sym_count", C.c_uint64 * 16)]


_lib = None


def lib_path() -> str:
    return _build.LIB


def lib():
    """Loads libecco_b200.so (building it in-tree if the sources are newer).  Raises if it cannot be
    had: nothing in this package works without it."""
    global _lib
    if _lib is None:
        if not os.path.exists(_build.LIB) or _build.is_stale():
            _build.build_library()
        L = C.CDLL(_build.LIB)
        vp, u64, i32, sz = C.c_void_p, C.c_uint64, C.c_int32, C.c_size_t
        L.ecco_calibrate_host.argtypes = [vp, u64, vp, C.POINTER(Params), C.POINTER(vp)]
        L.ecco_meta_create.argtypes = [i32, i32, vp, vp, vp, C.POINTER(vp)]
        L.ecco_meta_get.argtypes = [vp, C.POINTER(i32), C.POINTER(i32), vp, vp, vp]
        L.ecco_meta_free.argtypes = [vp]
        L.ecco_meta_free.restype = None
        L.ecco_encode_host.argtypes = [vp, vp, u64, C.c_uint32, vp, C.POINTER(Stats)]
        L.ecco_meta_device_bytes.argtypes = [vp]
        L.ecco_meta_device_bytes.restype = sz
        L.ecco_meta_serialize_device.argtypes = [vp, vp, sz]
        L.ecco_decompress.argtypes = [vp, vp, u64, vp, vp]
        L.ecco_decompress_batch.argtypes = [C.POINTER(DecompressItem), i32, vp]
        L.ecco_gemv_workspace_bytes.argtypes = [i32, i32, i32]
        L.ecco_gemv_workspace_bytes.restype = sz
        L.ecco_gemv.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp, sz, vp]
        L.ecco_gemv_static_ws.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp]
        L.ecco_gemv_batch_workspace_bytes.argtypes = [C.POINTER(GemvItem), i32, i32]
        L.ecco_gemv_batch_workspace_bytes.restype = sz
        L.ecco_gemv_batch.argtypes = [C.POINTER(GemvItem), i32, i32, vp, sz, vp]
        L.ecco_attn_scores.argtypes = [vp, vp, i32, i32, i32, i32, vp, C.c_float, vp, vp]
        L.ecco_attn_values_workspace_bytes.argtypes = [i32, i32, i32, i32]
        L.ecco_attn_values_workspace_bytes.restype = sz
        L.ecco_attn_values.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp, sz, vp]
        L.ecco_kv_compress.argtypes = [vp, vp, u64, vp, vp]
        L.ecco_var_stream_bytes_bound.argtypes = [u64]
        L.ecco_var_stream_bytes_bound.restype = sz
        L.ecco_var_index_bytes.argtypes = [u64]
        L.ecco_var_index_bytes.restype = sz
        L.ecco_var_encode_host.argtypes = [vp, vp, u64, C.c_uint32, vp, sz, vp, sz, C.POINTER(u64)]
        L.ecco_var_decompress.argtypes = [vp, vp, vp, u64, vp, vp]
        L.ecco_act_compress.argtypes = [vp, u64, vp, vp]
        L.ecco_act_decompress.argtypes = [vp, u64, vp, vp]
        L.ecco_error_string.argtypes = [C.c_int]
        L.ecco_error_string.restype = C.c_char_p
        L.ecco_last_cuda_error.restype = C.c_int
        L.ecco_device_status.restype = C.c_int
        L.ecco_kernel_launch_count.restype = u64
        L.ecco_test_wait_timeout.argtypes = [vp]
        _lib = L
    return _lib


def _check(rc: int, what: str):
    if rc != ECCO_OK:
        raise EccoError(rc, what)


def _host_u16(x) -> np.ndarray:
    x = np.ascontiguousarray(x)
    if x.dtype == np.float16:
        x = x.view(np.uint16)
    if x.dtype != np.uint16:
        raise TypeError("expected fp16 (or raw uint16) host data")
    return x


class Meta:
    """Owner of an ecco_meta handle."""

    def __init__(self, handle: int):
        self._h = C.c_void_p(handle)

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h and _lib is not None:
            _lib.ecco_meta_free(h)

    @property
    def handle(self):
        return self._h

    def tables(self):
        """-> (S, e, patterns fp16 [S][15], cb_len u8 [S][4][16], kp_len u8 [S])."""
        S, e = C.c_int32(), C.c_int32()
        _check(lib().ecco_meta_get(self._h, C.byref(S), C.byref(e), None, None, None), "ecco_meta_get")
        pat = np.zeros((S.value, 15), dtype=np.uint16)
        cb = np.zeros((S.value, 4, 16), dtype=np.uint8)
        kp = np.zeros(S.value, dtype=np.uint8)
        _check(lib().ecco_meta_get(self._h, None, None, pat.ctypes.data, cb.ctypes.data, kp.ctypes.data), "ecco_meta_get")
        return S.value, e.value, pat.view(np.float16), cb, kp


# ------------------------------------------------------------------ host calls
def ecco_calibrate_host(calib_fp16, S: int = 64, H: int = 4, seed: int = 1, select: int = SELECT_MSE,
                        elem_weights=None, kmeans_iters: int = 0, max_groups: int = 0, threads: int = 0) -> Meta:
    x = _host_u16(calib_fp16).reshape(-1)
    if x.size % GROUP:
        raise ValueError("calibration tensor is not a whole number of 128-value groups")
    p = Params(S, H, seed, select, kmeans_iters, max_groups, threads)
    w = None
    if elem_weights is not None:
        w = np.ascontiguousarray(elem_weights, dtype=np.float32)
        if w.shape != (GROUP,):
            raise ValueError("elem_weights must hold 128 floats")
    out = C.c_void_p()
    _check(lib().ecco_calibrate_host(x.ctypes.data, x.size // GROUP, w.ctypes.data if w is not None else None,
                                     C.byref(p), C.byref(out)), "ecco_calibrate_host")
    return Meta(out.value)


def ecco_meta_create(S: int, e: int, patterns_fp16, cb_len, kp_len) -> Meta:
    pat = _host_u16(patterns_fp16)
    cb = np.ascontiguousarray(cb_len, dtype=np.uint8)
    kp = np.ascontiguousarray(kp_len, dtype=np.uint8)
    if pat.shape != (S, 15) or cb.shape != (S, 4, 16) or kp.shape != (S,):
        raise ValueError("table shapes must be [S][15], [S][4][16], [S]")
    out = C.c_void_p()
    _check(lib().ecco_meta_create(S, e, pat.ctypes.data, cb.ctypes.data, kp.ctypes.data, C.byref(out)), "ecco_meta_create")
    return Meta(out.value)


def ecco_encode_host(meta: Meta, src_fp16, flags: int = SELECT_MSE, out_blocks=None, want_stats: bool = True):
    """-> (blocks uint8 [n_groups][64], Stats or None)."""
    x = _host_u16(src_fp16).reshape(-1)
    if x.size % GROUP:
        raise ValueError("tensor is not a whole number of 128-value groups")
    n = x.size // GROUP
    if out_blocks is None:
        out_blocks = np.empty((n, BLOCK_BYTES), dtype=np.uint8)
    assert out_blocks.dtype == np.uint8 and out_blocks.size == n * BLOCK_BYTES and out_blocks.flags.c_contiguous
    st = Stats() if want_stats else None
    _check(lib().ecco_encode_host(meta.handle, x.ctypes.data, n, flags, out_blocks.ctypes.data,
                                  C.byref(st) if st is not None else None), "ecco_encode_host")
    return out_blocks, st


def ecco_meta_device_bytes(meta: Meta) -> int:
    return int(lib().ecco_meta_device_bytes(meta.handle))


def ecco_meta_serialize_device(meta: Meta) -> np.ndarray:
    """-> uint8 host image; copy it to 16-byte aligned device memory and pass that as d_meta."""
    n = ecco_meta_device_bytes(meta)
    buf = np.zeros(n, dtype=np.uint8)
    _check(lib().ecco_meta_serialize_device(meta.handle, buf.ctypes.data, n), "ecco_meta_serialize_device")
    return buf


def ecco_var_encode_host(meta: Meta, src_fp16, flags: int = SELECT_MSE):
    """Variable-length container: -> (stream uint8, a multiple of 16 bytes; index uint8; total_bits)."""
    x = _host_u16(src_fp16).reshape(-1)
    if x.size % GROUP:
        raise ValueError("tensor is not a whole number of 128-value groups")
    n = x.size // GROUP
    stream = np.empty(int(lib().ecco_var_stream_bytes_bound(n)), dtype=np.uint8)
    index = np.zeros(int(lib().ecco_var_index_bytes(n)), dtype=np.uint8)
    total = C.c_uint64(0)
    _check(lib().ecco_var_encode_host(meta.handle, x.ctypes.data, n, flags, stream.ctypes.data, stream.size, index.ctypes.data,
                                      index.size, C.byref(total)), "ecco_var_encode_host")
    used = (total.value + 127) // 128 * 16
    return stream[:used].copy(), index, total.value


# ------------------------------------------------------------------ device calls
def _ptr(t) -> int:
    """Raw device pointer of a CUDA torch tensor (or an int that already is one)."""
    if isinstance(t, int):
        return t
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("device arguments must be contiguous CUDA tensors")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def meta_to_device(meta: Meta, device="cuda"):
    """Convenience: serialise and upload; returns a uint8 CUDA tensor to pass as d_meta."""
    import torch

    return torch.from_numpy(ecco_meta_serialize_device(meta)).to(device)


def ecco_decompress(d_meta, d_blocks, n_groups: int, d_out_fp16, stream=None) -> None:
    _check(lib().ecco_decompress(_ptr(d_meta), _ptr(d_blocks), n_groups, _ptr(d_out_fp16), _stream(stream)),
           "ecco_decompress")


def decompress_items(items):
    """The host array ecco_decompress_batch reads, from a sequence of (d_meta, d_blocks, n_groups, d_out_fp16).  A
    caller that issues the same batch again and again builds it once and passes it instead of the sequence."""
    arr = (DecompressItem * max(len(items), 1))()
    for i, (d_meta, d_blocks, n_groups, d_out) in enumerate(items):
        arr[i].d_meta, arr[i].d_blocks, arr[i].n_groups, arr[i].d_out_fp16 = _ptr(d_meta), _ptr(d_blocks), n_groups, _ptr(d_out)
    arr.n_items = len(items)
    return arr


def ecco_decompress_batch(items, stream=None) -> None:
    """items: sequence of (d_meta, d_blocks, n_groups, d_out_fp16), or what decompress_items made of one; one call
    for all of them (see include/ecco.h)."""
    arr = items if isinstance(items, C.Array) else decompress_items(items)
    _check(lib().ecco_decompress_batch(arr, arr.n_items, _stream(stream)), "ecco_decompress_batch")


def ecco_gemv_workspace_bytes(n_out: int, k: int, batch: int) -> int:
    return int(lib().ecco_gemv_workspace_bytes(n_out, k, batch))


def ecco_gemv(d_meta, d_blocks, n_out: int, k: int, d_x_fp16, batch: int, d_y, d_workspace, workspace_bytes: int,
              stream=None) -> None:
    _check(lib().ecco_gemv(_ptr(d_meta), _ptr(d_blocks), n_out, k, _ptr(d_x_fp16), batch, _ptr(d_y),
                           _ptr(d_workspace) if d_workspace is not None else None, workspace_bytes, _stream(stream)),
           "ecco_gemv")


def gemv_items(items):
    """The host array ecco_gemv_batch reads, from a sequence of (d_meta, d_blocks, n_out, k, d_x_fp16, d_y).  A caller
    that issues the same group again and again builds it once and passes it instead of the sequence."""
    arr = (GemvItem * max(len(items), 1))()
    for i, (d_meta, d_blocks, n_out, k, d_x, d_y) in enumerate(items):
        arr[i].d_meta, arr[i].d_blocks, arr[i].n_out, arr[i].k = _ptr(d_meta), _ptr(d_blocks), n_out, k
        arr[i].d_x_fp16, arr[i].d_y = _ptr(d_x), _ptr(d_y)
    arr.n_items = len(items)
    return arr


def ecco_gemv_batch_workspace_bytes(items, batch: int) -> int:
    """items: sequence of (d_meta, d_blocks, n_out, k, d_x_fp16, d_y) (pointers may be None here)."""
    arr = (GemvItem * max(len(items), 1))()
    for i, it in enumerate(items):
        arr[i].n_out, arr[i].k = it[2], it[3]
    return int(lib().ecco_gemv_batch_workspace_bytes(arr, len(items), batch))


def ecco_gemv_batch(items, batch: int, d_workspace, workspace_bytes: int, stream=None) -> None:
    """items: sequence of (d_meta, d_blocks, n_out, k, d_x_fp16, d_y), or what gemv_items made of one; one call for
    all of them (see include/ecco.h)."""
    arr = items if isinstance(items, C.Array) else gemv_items(items)
    _check(lib().ecco_gemv_batch(arr, arr.n_items, batch, _ptr(d_workspace) if d_workspace is not None else None,
                                 workspace_bytes, _stream(stream)), "ecco_gemv_batch")


STATIC_WORKSPACE_BYTES = 4 << 20


def ecco_gemv_static_ws(d_meta, d_blocks, n_out: int, k: int, d_x_fp16, batch: int, d_y, stream=None) -> None:
    """ecco_gemv without a caller workspace and without any allocation: the scratch is a fixed
    STATIC_WORKSPACE_BYTES array inside the library, shared by all calls on the device (so calls that
    overlap on the GPU race).  For callers that may not allocate device memory when they run, such
    as engine plug-ins with a fixed memory plan.  Make the first call on a device outside stream
    capture.  Raises EccoError(ERR_WORKSPACE) for shapes that need more scratch than the array."""
    _check(lib().ecco_gemv_static_ws(_ptr(d_meta), _ptr(d_blocks), n_out, k, _ptr(d_x_fp16), batch, _ptr(d_y),
                                     _stream(stream)), "ecco_gemv_static_ws")


def ecco_attn_scores(d_meta, d_kblocks, batch: int, n_kv_heads: int, seq: int, q_per_kv: int, d_q_fp16, scale: float,
                     d_scores, stream=None) -> None:
    _check(lib().ecco_attn_scores(_ptr(d_meta), _ptr(d_kblocks), batch, n_kv_heads, seq, q_per_kv, _ptr(d_q_fp16),
                                  C.c_float(scale), _ptr(d_scores), _stream(stream)), "ecco_attn_scores")


def ecco_attn_values_workspace_bytes(batch: int, n_kv_heads: int, seq: int, q_per_kv: int) -> int:
    return int(lib().ecco_attn_values_workspace_bytes(batch, n_kv_heads, seq, q_per_kv))


def ecco_attn_values(d_meta, d_vblocks, batch: int, n_kv_heads: int, seq: int, q_per_kv: int, d_scores, d_out, d_workspace,
                     workspace_bytes: int, stream=None) -> None:
    """softmax(scores) . V~ over a compressed V cache -> fp32 [batch][n_kv_heads*q_per_kv][128]."""
    _check(lib().ecco_attn_values(_ptr(d_meta), _ptr(d_vblocks), batch, n_kv_heads, seq, q_per_kv, _ptr(d_scores), _ptr(d_out),
                                  _ptr(d_workspace) if d_workspace is not None else None, workspace_bytes, _stream(stream)),
           "ecco_attn_values")


def ecco_kv_compress(d_meta, d_x_fp16, n_groups: int, d_blocks, stream=None) -> None:
    """Online 4x compressor (min/max pattern selection, calibrated exponent): fp16 device tensor -> 64-byte blocks."""
    _check(lib().ecco_kv_compress(_ptr(d_meta), _ptr(d_x_fp16), n_groups, _ptr(d_blocks), _stream(stream)), "ecco_kv_compress")


def ecco_var_decompress(d_meta, d_stream, d_index, n_groups: int, d_out_fp16, stream=None) -> None:
    """Decompress the variable-length container (see ecco_var_encode_host) to fp16 [n_groups][128]."""
    _check(lib().ecco_var_decompress(_ptr(d_meta), _ptr(d_stream), _ptr(d_index), n_groups, _ptr(d_out_fp16), _stream(stream)),
           "ecco_var_decompress")


def ecco_act_compress(d_x_fp16, n_groups: int, d_blocks, stream=None) -> None:
    """2x activation format: 64 fp16 values -> 64 bytes per group (device to device)."""
    _check(lib().ecco_act_compress(_ptr(d_x_fp16), n_groups, _ptr(d_blocks), _stream(stream)), "ecco_act_compress")


def ecco_act_decompress(d_blocks, n_groups: int, d_out_fp16, stream=None) -> None:
    _check(lib().ecco_act_decompress(_ptr(d_blocks), n_groups, _ptr(d_out_fp16), _stream(stream)), "ecco_act_decompress")


def ecco_device_status() -> int:
    return int(lib().ecco_device_status())


def ecco_kernel_launch_count() -> int:
    return int(lib().ecco_kernel_launch_count())


def ecco_test_wait_timeout(stream=None) -> None:
    """Test aid: one small kernel whose bounded wait runs out (see include/ecco.h)."""
    _check(lib().ecco_test_wait_timeout(_stream(stream)), "ecco_test_wait_timeout")
