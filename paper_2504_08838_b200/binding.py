"""ctypes binding of ``libsd2.so`` -- argument marshalling only.

Function names mirror the C ABI in ``include/sd2.h``.  Device buffers are torch CUDA
tensors (torch is used for device memory and streams, nothing else); host buffers are
numpy arrays.  A missing shared library or a failing call raises: there is no fallback.
"""

from __future__ import annotations

import ctypes
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libsd2.so")

SD2_OK = 0
SD2_ERR_INVALID_ARG, SD2_ERR_SHAPE, SD2_ERR_ALLOC, SD2_ERR_CUDA = -1, -2, -3, -4
SD2_ERR_UNSUPPORTED, SD2_ERR_CORRUPT, SD2_ERR_TIMEOUT = -5, -6, -7
SD2_FORMAT_AUTO, SD2_FORMAT_BITMASK, SD2_FORMAT_GAP4, SD2_FORMAT_GAP4_PAIRED, SD2_FORMAT_GAP4_MMA = 0, 1, 2, 3, 4
SD2_DTYPE_BF16, SD2_DTYPE_F32 = 0, 1

EXPORTS = [
    "sd2_pack_host", "sd2_unpack_host", "sd2_blob_free", "sd2_compress", "sd2_load_blob",
    "sd2_decompress", "sd2_info", "sd2_free", "sd2_spmm", "sd2_spmm_fused", "sd2_block_step",
    "sd2_block_workspace_bytes", "sd2_block_workspace_layout", "sd2_status_string", "sd2_stream_check",
    "sd2_drafter_create", "sd2_drafter_step", "sd2_drafter_buffers", "sd2_drafter_free",
    "sd2_block_step_static", "sd2_selftest_timeout", "sd2_drafter_query",
    "sd2_rmsnorm", "sd2_add_rmsnorm", "sd2_rope_cache", "sd2_attention_decode", "sd2_rope_attention", "sd2_add", "sd2_embedding", "sd2_lm_head",
    "sd2_decoder_workspace_bytes", "sd2_decoder_block_step", "sd2_debug_fail_allocations",
]


class Sd2Options(ctypes.Structure):
    _fields_ = [("format", ctypes.c_int32), ("y_dtype", ctypes.c_int32)]


class Sd2Error(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__("%s: %s (%d)" % (what, status_string(status), status))


_lib = None


def lib():
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libsd2.so is missing (%s): run `python -m paper_2504_08838_b200.build`; "
                               "there is no CPU fallback" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        p, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32
        pp = ctypes.POINTER(ctypes.c_void_p)
        pi64 = ctypes.POINTER(ctypes.c_int64)
        pi32 = ctypes.POINTER(ctypes.c_int32)
        opt = ctypes.POINTER(Sd2Options)
        sig = {
            "sd2_pack_host": [p, p, i64, i64, opt, pp, pi64],
            "sd2_unpack_host": [p, i64, p, pi64, pi64, pi64, pi64, pi32],
            "sd2_blob_free": [p],
            "sd2_compress": [p, p, i64, i64, opt, pp],
            "sd2_load_blob": [p, i64, pp],
            "sd2_decompress": [p, p],
            "sd2_info": [p, pi64, pi64, pi64, pi64, pi32],
            "sd2_free": [p],
            "sd2_spmm": [p, p, p, i64, p],
            "sd2_spmm_fused": [pp, i32, p, pp, i64, p],
            "sd2_block_step": [pp, p, p, i64, p, p],
            "sd2_block_workspace_bytes": [pp, i64, pi64],
            "sd2_block_workspace_layout": [pp, i64, pi64],
            "sd2_stream_check": [p],
            "sd2_drafter_create": [pp, i32, i64, pp],
            "sd2_drafter_step": [p, p, p, i64, p],
            "sd2_drafter_buffers": [p, i32, pp],
            "sd2_drafter_query": [p, i64, pi64],
            "sd2_drafter_free": [p],
            "sd2_block_step_static": [pp, p, p, i64, p],
            "sd2_selftest_timeout": [p],
            "sd2_rmsnorm": [p, p, p, i64, i64, ctypes.c_float, p],
            "sd2_add_rmsnorm": [p, p, p, p, p, i64, i64, ctypes.c_float, p],
            "sd2_rope_cache": [p, p, p, p, p, i64, i64, i64, i64, i64, i64, ctypes.c_double, p],
            "sd2_attention_decode": [p, p, p, p, i64, i64, i64, i64, i64, i64, p],
            "sd2_rope_attention": [p, p, p, p, p, p, i64, i64, i64, i64, i64, i64, ctypes.c_double, p],
            "sd2_add": [p, p, p, i64, p],
            "sd2_embedding": [p, p, p, i64, i64, i64, p],
            "sd2_lm_head": [p, p, p, p, i64, i64, i64, p],
            "sd2_debug_fail_allocations": [i64, i64],
            "sd2_decoder_workspace_bytes": [pp, i64, pi64],
            "sd2_decoder_block_step": [pp, p, p, p, p, p, p, i64, i64, i64, i64, i64, ctypes.c_float, ctypes.c_double, p, p],
        }
        for name, argtypes in sig.items():
            fn = getattr(L, name)
            fn.argtypes = argtypes
            fn.restype = ctypes.c_int
        L.sd2_status_string.argtypes = [ctypes.c_int]
        L.sd2_status_string.restype = ctypes.c_char_p
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().sd2_status_string(int(status)).decode()


def _check(status: int, what: str):
    if status != SD2_OK:
        raise Sd2Error(status, what)


def _opt(fmt, y_dtype):
    return ctypes.byref(Sd2Options(int(fmt), int(y_dtype)))


def _host_ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _ptr(t):
    """Address of a numpy array (host) or a torch tensor (host or device)."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data_as(ctypes.c_void_p)
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    return ctypes.c_void_p(int(stream))


# ---- host format builder ---------------------------------------------------------------

def sd2_pack_host(weight: np.ndarray, mask, fmt=SD2_FORMAT_AUTO, y_dtype=SD2_DTYPE_BF16) -> bytes:
    """Encode ``weight`` (uint16 bf16 patterns ``[M, K]``) under ``mask`` into a blob."""
    weight = np.ascontiguousarray(weight, dtype=np.uint16)
    M, K = weight.shape
    if mask is not None:
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
        assert mask.shape == (M, K)
    blob = ctypes.c_void_p()
    n = ctypes.c_int64()
    _check(lib().sd2_pack_host(_host_ptr(weight), _host_ptr(mask), M, K, _opt(fmt, y_dtype),
                               ctypes.byref(blob), ctypes.byref(n)), "sd2_pack_host")
    try:
        return ctypes.string_at(blob, n.value)
    finally:
        lib().sd2_blob_free(blob)


def sd2_unpack_host(blob: bytes, want_dense: bool = True):
    """``(dense uint16 [M,K] or None, info dict)``; raises Sd2Error(CORRUPT) on a bad blob."""
    M, K, nnz, cb = (ctypes.c_int64() for _ in range(4))
    fmt = ctypes.c_int32()
    buf = ctypes.create_string_buffer(blob, len(blob))
    _check(lib().sd2_unpack_host(buf, len(blob), None, ctypes.byref(M), ctypes.byref(K), ctypes.byref(nnz),
                                 ctypes.byref(cb), ctypes.byref(fmt)), "sd2_unpack_host")
    info = dict(M=M.value, K=K.value, nnz=nnz.value, compressed_bytes=cb.value, format=fmt.value)
    dense = None
    if want_dense:
        dense = np.empty((M.value, K.value), dtype=np.uint16)
        _check(lib().sd2_unpack_host(buf, len(blob), _host_ptr(dense), None, None, None, None, None), "sd2_unpack_host")
    return dense, info


# ---- handles ---------------------------------------------------------------------------

class Handle:
    """Owns one ``sd2_handle``; freed on ``close()`` or garbage collection."""

    def __init__(self, raw: int):
        self.raw = ctypes.c_void_p(raw)
        M, K, nnz, cb = (ctypes.c_int64() for _ in range(4))
        fmt = ctypes.c_int32()
        _check(lib().sd2_info(self.raw, ctypes.byref(M), ctypes.byref(K), ctypes.byref(nnz), ctypes.byref(cb),
                              ctypes.byref(fmt)), "sd2_info")
        self.M, self.K, self.nnz, self.compressed_bytes, self.format = M.value, K.value, nnz.value, cb.value, fmt.value
        self.y_dtype = SD2_DTYPE_BF16

    def close(self):
        if self.raw is not None and self.raw.value:
            lib().sd2_free(self.raw)
            self.raw = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def sd2_compress(weight, mask, fmt=SD2_FORMAT_AUTO, y_dtype=SD2_DTYPE_BF16) -> Handle:
    """``weight``: uint16 numpy ``[M,K]`` or a torch bf16/int16 tensor (host or device)."""
    if isinstance(weight, np.ndarray):
        weight = np.ascontiguousarray(weight, dtype=np.uint16)
    if isinstance(mask, np.ndarray):
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
    M, K = weight.shape
    out = ctypes.c_void_p()
    _check(lib().sd2_compress(_ptr(weight), _ptr(mask), M, K, _opt(fmt, y_dtype), ctypes.byref(out)), "sd2_compress")
    h = Handle(out.value)
    h.y_dtype = y_dtype
    return h


def sd2_load_blob(blob: bytes, y_dtype=None) -> Handle:
    out = ctypes.c_void_p()
    buf = ctypes.create_string_buffer(blob, len(blob))
    _check(lib().sd2_load_blob(buf, len(blob), ctypes.byref(out)), "sd2_load_blob")
    h = Handle(out.value)
    if y_dtype is not None:
        h.y_dtype = y_dtype
    return h


def sd2_decompress(h: Handle) -> np.ndarray:
    dense = np.empty((h.M, h.K), dtype=np.uint16)
    _check(lib().sd2_decompress(h.raw, _host_ptr(dense)), "sd2_decompress")
    return dense


def sd2_info(h: Handle) -> dict:
    return dict(M=h.M, K=h.K, nnz=h.nnz, compressed_bytes=h.compressed_bytes, format=h.format)


def sd2_free(h: Handle):
    h.close()


# ---- hot path --------------------------------------------------------------------------

def sd2_spmm(h: Handle, X, Y, stream=None):
    """``X``: device bf16 ``[N, K]``; ``Y``: device ``[N, M]`` (bf16 or fp32 per the handle)."""
    N = X.shape[0] if X.dim() == 2 else 1
    _check(lib().sd2_spmm(h.raw, _ptr(X), _ptr(Y), N, _stream(stream)), "sd2_spmm")


def _handle_array(hs):
    arr = (ctypes.c_void_p * len(hs))(*[h.raw.value for h in hs])
    return arr


def sd2_spmm_fused(hs, X, Ys, stream=None):
    N = X.shape[0] if X.dim() == 2 else 1
    ys = (ctypes.c_void_p * len(Ys))(*[y.data_ptr() for y in Ys])
    _check(lib().sd2_spmm_fused(_handle_array(hs), len(hs), _ptr(X), ys, N, _stream(stream)), "sd2_spmm_fused")


def sd2_block_workspace_bytes(hs, N: int) -> int:
    n = ctypes.c_int64()
    _check(lib().sd2_block_workspace_bytes(_handle_array(hs), N, ctypes.byref(n)), "sd2_block_workspace_bytes")
    return n.value


def sd2_block_workspace_layout(hs, N: int):
    off = (ctypes.c_int64 * 7)()
    _check(lib().sd2_block_workspace_layout(_handle_array(hs), N, off), "sd2_block_workspace_layout")
    return list(off)


def sd2_stream_check(stream=None):
    """Synchronise the stream; raises Sd2Error(TIMEOUT) if a device-side wait ran out."""
    _check(lib().sd2_stream_check(_stream(stream)), "sd2_stream_check")


def sd2_block_step(hs, x, y, workspace, stream=None, handle_array=None):
    N = x.shape[0] if x.dim() == 2 else 1
    arr = handle_array if handle_array is not None else _handle_array(hs)
    _check(lib().sd2_block_step(arr, _ptr(x), _ptr(y), N, _ptr(workspace), _stream(stream)), "sd2_block_step")


# ---- whole drafter ---------------------------------------------------------------------

class Drafter:
    """Owns one ``sd2_drafter`` (and keeps its handles alive)."""

    def __init__(self, raw: int, blocks):
        self.raw = ctypes.c_void_p(raw)
        self.blocks = blocks

    def close(self):
        if self.raw is not None and self.raw.value:
            lib().sd2_drafter_free(self.raw)
            self.raw = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def sd2_drafter_create(blocks, n_max: int = 1) -> Drafter:
    """``blocks``: list of 7-handle lists (q, k, v, o, gate, up, down), one per drafter block."""
    flat = [h for hs in blocks for h in hs]
    out = ctypes.c_void_p()
    _check(lib().sd2_drafter_create(_handle_array(flat), len(blocks), n_max, ctypes.byref(out)), "sd2_drafter_create")
    return Drafter(out.value, blocks)


def sd2_drafter_step(d: Drafter, x, y, stream=None):
    N = x.shape[0] if x.dim() == 2 else 1
    _check(lib().sd2_drafter_step(d.raw, _ptr(x), _ptr(y), N, _stream(stream)), "sd2_drafter_step")


def sd2_drafter_buffers(d: Drafter, block: int):
    """Device addresses of q, k, v, hdn, g, u, t and the block output of one block."""
    ptrs = (ctypes.c_void_p * 8)()
    _check(lib().sd2_drafter_buffers(d.raw, block, ptrs), "sd2_drafter_buffers")
    return [int(p or 0) for p in ptrs]


def sd2_drafter_query(d: Drafter, N: int) -> dict:
    """Launches per step of N rows, widest panel, device bytes owned, bytes streamed per launch, stages, kept weights."""
    out = (ctypes.c_int64 * 6)()
    _check(lib().sd2_drafter_query(d.raw, N, out), "sd2_drafter_query")
    keys = ("launches", "panel_rows", "owned_bytes", "streamed_bytes", "stages", "kept_weights")
    return dict(zip(keys, (int(v) for v in out)))


def sd2_drafter_free(d: Drafter):
    d.close()


def sd2_block_step_static(hs, x, y, stream=None):
    """``sd2_block_step`` with the intermediates in the library's built-in scratch array: for callers
    that may not allocate device memory.  Calls must not overlap on the GPU (they share the array)."""
    N = x.shape[0] if x.dim() == 2 else 1
    _check(lib().sd2_block_step_static(_handle_array(hs), _ptr(x), _ptr(y), N, _stream(stream)), "sd2_block_step_static")


def sd2_selftest_timeout(stream=None):
    """Launch the diagnostic whose device-side wait must run out (see ``sd2_stream_check``)."""
    _check(lib().sd2_selftest_timeout(_stream(stream)), "sd2_selftest_timeout")


# ---- glue of a whole decode step -----------------------------------------------------------

def sd2_rmsnorm(x, w, y, eps: float, stream=None):
    N, H = x.shape
    _check(lib().sd2_rmsnorm(_ptr(x), _ptr(w), _ptr(y), N, H, eps, _stream(stream)), "sd2_rmsnorm")


def sd2_add_rmsnorm(a, b, total, w, y, eps: float, stream=None):
    N, H = a.shape
    _check(lib().sd2_add_rmsnorm(_ptr(a), _ptr(b), _ptr(total), _ptr(w), _ptr(y), N, H, eps, _stream(stream)), "sd2_add_rmsnorm")


def sd2_rope_cache(q, k, v, k_cache, v_cache, heads_q: int, heads_kv: int, pos: int, theta: float, stream=None):
    """q [N, heads_q*d] rotated in place; rope(k), v appended at ``pos`` of the caches [N, T_max, heads_kv*d]."""
    N = q.shape[0]
    d = q.shape[1] // heads_q
    _check(lib().sd2_rope_cache(_ptr(q), _ptr(k), _ptr(v), _ptr(k_cache), _ptr(v_cache), N, heads_q, heads_kv, d, pos,
                                k_cache.shape[1], theta, _stream(stream)), "sd2_rope_cache")


def sd2_attention_decode(q, k_cache, v_cache, out, heads_q: int, heads_kv: int, T: int, stream=None):
    N = q.shape[0]
    d = q.shape[1] // heads_q
    _check(lib().sd2_attention_decode(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(out), N, heads_q, heads_kv, d, T,
                                      k_cache.shape[1], _stream(stream)), "sd2_attention_decode")


def sd2_rope_attention(q, k, v, k_cache, v_cache, out, heads_q: int, heads_kv: int, pos: int, theta: float, stream=None):
    N = q.shape[0]
    d = q.shape[1] // heads_q
    _check(lib().sd2_rope_attention(_ptr(q), _ptr(k), _ptr(v), _ptr(k_cache), _ptr(v_cache), _ptr(out), N, heads_q, heads_kv, d,
                                    pos, k_cache.shape[1], theta, _stream(stream)), "sd2_rope_attention")


def sd2_add(a, b, y, stream=None):
    _check(lib().sd2_add(_ptr(a), _ptr(b), _ptr(y), a.numel(), _stream(stream)), "sd2_add")


def sd2_embedding(tokens, table, x, stream=None):
    V, H = table.shape
    _check(lib().sd2_embedding(_ptr(tokens), _ptr(table), _ptr(x), tokens.numel(), V, H, _stream(stream)), "sd2_embedding")


def sd2_lm_head(x, w_out, logits, tokens=None, stream=None):
    N, H = x.shape
    V = w_out.shape[0]
    _check(lib().sd2_lm_head(_ptr(x), _ptr(w_out), _ptr(logits), _ptr(tokens) if tokens is not None else None, N, V, H,
                             _stream(stream)), "sd2_lm_head")


def sd2_decoder_workspace_bytes(hs, N: int) -> int:
    out = ctypes.c_int64()
    _check(lib().sd2_decoder_workspace_bytes(_handle_array(hs), N, ctypes.byref(out)), "sd2_decoder_workspace_bytes")
    return out.value


def sd2_decoder_block_step(hs, norm_attn, norm_ffn, x, y, k_cache, v_cache, heads_q: int, heads_kv: int, pos: int,
                           eps: float, theta: float, workspace, stream=None, handle_array=None):
    N = x.shape[0]
    arr = handle_array if handle_array is not None else _handle_array(hs)
    _check(lib().sd2_decoder_block_step(arr, _ptr(norm_attn), _ptr(norm_ffn), _ptr(x), _ptr(y), _ptr(k_cache), _ptr(v_cache), N,
                                        heads_q, heads_kv, pos, k_cache.shape[1], eps, theta, _ptr(workspace), _stream(stream)),
           "sd2_decoder_block_step")


def sd2_debug_fail_allocations(skip: int, fail: int):
    """Let the library's next ``skip`` allocations through and fail the ``fail`` after them; (0, 0) = off."""
    _check(lib().sd2_debug_fail_allocations(skip, fail), "sd2_debug_fail_allocations")
