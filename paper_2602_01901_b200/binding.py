"""ctypes binding of the C ABI in ``include/qc.h``: argument marshalling only.

Every function here has the name and argument order of its C counterpart; tensors are
passed as raw device (or host) pointers.  ``load()`` raises if the compiled library is
missing -- there is no fallback path.
"""

from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqcache.so")

QC_OK = 0
QC_ERR_INVALID_ARG = 1
QC_ERR_UNSUPPORTED = 2
QC_ERR_OOM_PAGES = 3
QC_ERR_STATE = 4
QC_ERR_CUDA = 5
QC_ERR_TIMEOUT = 6
QC_ERR_BAD_PAGE = 7
QC_ERR_PLAN = 8

QC_LAYER_FULL, QC_LAYER_LAZY = 0, 1
QC_MODE_VLA_QC, QC_MODE_VLA_EQ8, QC_MODE_GLA = 0, 1, 2
QC_STREAM_K_TEXT, QC_STREAM_K_VISUAL, QC_STREAM_V_TEXT, QC_STREAM_V_VISUAL = 0, 1, 2, 3
QC_KIND_TEXT, QC_KIND_VISUAL = 0, 1

EXPORTS = (
    "qc_init", "qc_cache_bytes_required", "qc_alloc_cache", "qc_prefill_append", "qc_prefill_attend", "qc_decode_step",
    "qc_decode_step_host", "qc_layer_similarity", "qc_lazy_blocks", "qc_free_seq", "qc_free", "qc_get_stats", "qc_debug_page_table",
    "qc_debug_read_qcache", "qc_debug_read_row", "qc_set_option", "qc_get_profile", "qc_status_string",
    "qc_attend_static", "qc_decode_begin", "qc_decode_layer",
)


class qc_config(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("page_size", C.c_int32), ("max_seqs", C.c_int32), ("max_tokens_per_seq", C.c_int32),
        ("n_pages", C.c_int64), ("softmax_scale", C.c_float), ("lazy_mode", C.c_int32),
        ("split_tokens", C.c_int32), ("layer_kind", C.POINTER(C.c_uint8)),
    ]


class qc_stats(C.Structure):
    _fields_ = [
        ("pages_total", C.c_int64), ("pages_in_use", C.c_int64), ("page_bytes", C.c_int64),
        ("kv_bytes_stored", C.c_int64), ("kv_bytes_all_full", C.c_int64),
        ("kv_bytes_stored_paged", C.c_int64), ("kv_bytes_all_full_paged", C.c_int64),
        ("qcache_bytes", C.c_int64), ("decode_steps", C.c_int64), ("attend_launches", C.c_int64),
        ("device_error", C.c_int32), ("n_active_seqs", C.c_int32),
        ("kernel_launches", C.c_int64), ("kv_bytes_swept", C.c_int64),
    ]


class qc_profile(C.Structure):
    _fields_ = [
        ("steps", C.c_int64), ("attend_ms", C.c_double), ("step_ms", C.c_double),
        ("kv_bytes_read", C.c_int64), ("items", C.c_int64),
        ("prefill_calls", C.c_int64), ("prefill_attend_ms", C.c_double), ("prefill_flops", C.c_double),
        ("attend_kernel_ms", C.c_double), ("attend_kernel_launches", C.c_int64),
    ]


class QcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib: Optional[C.CDLL] = None


def load() -> C.CDLL:
    """Load the compiled library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2602_01901_b200.build` "
            "(there is no CPU or PyTorch fallback)"
        )
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    pi32, pu8 = C.POINTER(C.c_int32), C.POINTER(C.c_uint8)
    sig = {
        "qc_init": [i32, vp, C.POINTER(vp)],
        "qc_cache_bytes_required": [C.POINTER(qc_config), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)],
        "qc_alloc_cache": [vp, C.POINTER(qc_config), vp, C.c_size_t, vp, C.c_size_t, C.POINTER(vp)],
        "qc_prefill_append": [vp, i32, pi32, pi32, pu8, vp, vp],
        "qc_prefill_attend": [vp, i32, i32, pu8, vp, vp, vp, vp],
        "qc_decode_step": [vp, i32, pi32, vp, vp, vp, vp, vp],
        "qc_layer_similarity": [vp, i32, pi32, vp, vp, i32, C.POINTER(C.c_float)],
        "qc_lazy_blocks": [C.POINTER(C.c_float), i32, C.c_float, i32, pu8],
        "qc_decode_step_host": [vp, i32, pi32, vp, vp, vp, vp, vp],
        "qc_decode_begin": [vp, i32, pi32],
        "qc_decode_layer": [vp, i32, vp, vp, vp, vp, vp],
        "qc_free_seq": [vp, i32],
        "qc_free": [vp, vp],
        "qc_get_stats": [vp, C.POINTER(qc_stats)],
        "qc_debug_page_table": [vp, i32, i32, i32, pi32, i32, pi32, pi32, pi32],
        "qc_debug_read_qcache": [vp, i32, vp],
        "qc_debug_read_row": [vp, i32, i32, i32, i32, i32, vp],
        "qc_set_option": [vp, C.c_char_p, i64],
        "qc_get_profile": [vp, C.POINTER(qc_profile)],
        "qc_attend_static": [i32, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, C.c_float],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = i32
    lib.qc_status_string.argtypes = [i32]
    lib.qc_status_string.restype = C.c_char_p
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().qc_status_string(status).decode()


def _check(status: int, where: str) -> None:
    if status != QC_OK:
        raise QcError(status, where)


def _i32_array(values: Sequence[int]):
    return (C.c_int32 * len(values))(*values)


def make_config(n_layers, n_q_heads, n_kv_heads, head_dim, page_size, max_seqs, max_tokens_per_seq, n_pages,
                layer_kind: Sequence[int], lazy_mode=QC_MODE_VLA_QC, split_tokens=0, softmax_scale=0.0):
    kinds = (C.c_uint8 * len(layer_kind))(*[int(k) for k in layer_kind])
    cfg = qc_config(n_layers, n_q_heads, n_kv_heads, head_dim, page_size, max_seqs, max_tokens_per_seq,
                    n_pages, softmax_scale, lazy_mode, split_tokens, C.cast(kinds, C.POINTER(C.c_uint8)))
    cfg._keepalive = kinds
    return cfg


# ---- the calls, one to one ----------------------------------------------------------------

def qc_init(device: int, cuda_stream: int = 0) -> C.c_void_p:
    ctx = C.c_void_p()
    _check(load().qc_init(device, C.c_void_p(cuda_stream), C.byref(ctx)), "qc_init")
    return ctx


def qc_cache_bytes_required(cfg: qc_config):
    pool, ws = C.c_size_t(), C.c_size_t()
    _check(load().qc_cache_bytes_required(C.byref(cfg), C.byref(pool), C.byref(ws)), "qc_cache_bytes_required")
    return pool.value, ws.value


def qc_alloc_cache(ctx, cfg: qc_config, pool_ptr: int, pool_bytes: int, ws_ptr: int, ws_bytes: int) -> C.c_void_p:
    cache = C.c_void_p()
    _check(load().qc_alloc_cache(ctx, C.byref(cfg), C.c_void_p(pool_ptr), pool_bytes, C.c_void_p(ws_ptr), ws_bytes,
                                 C.byref(cache)), "qc_alloc_cache")
    return cache


def qc_prefill_append(cache, seq_ids: Sequence[int], n_tokens: Sequence[int], kind, k_ptr: int, v_ptr: int) -> None:
    kind_bytes = bytes(bytearray(int(x) for x in kind)) if not isinstance(kind, (bytes, bytearray)) else bytes(kind)
    kbuf = (C.c_uint8 * max(1, len(kind_bytes))).from_buffer_copy(kind_bytes or b"\0")
    _check(load().qc_prefill_append(cache, len(seq_ids), _i32_array(seq_ids), _i32_array(n_tokens),
                                    C.cast(kbuf, C.POINTER(C.c_uint8)), C.c_void_p(k_ptr), C.c_void_p(v_ptr)),
           "qc_prefill_append")


def qc_prefill_attend(cache, seq_id: int, kind, q_ptr: int, k_ptr: int, v_ptr: int, out_ptr: int) -> None:
    kind_bytes = bytes(bytearray(int(x) for x in kind)) if not isinstance(kind, (bytes, bytearray)) else bytes(kind)
    kbuf = (C.c_uint8 * max(1, len(kind_bytes))).from_buffer_copy(kind_bytes or b"\0")
    _check(load().qc_prefill_attend(cache, seq_id, len(kind_bytes), C.cast(kbuf, C.POINTER(C.c_uint8)),
                                    C.c_void_p(q_ptr), C.c_void_p(k_ptr), C.c_void_p(v_ptr), C.c_void_p(out_ptr)),
           "qc_prefill_attend")


def qc_layer_similarity(cache, seq_ids: Sequence[int], q_ptr: int, rows_ptr: int, max_len: int, n_layers: int):
    sim = (C.c_float * max(1, n_layers - 1))()
    _check(load().qc_layer_similarity(cache, len(seq_ids), _i32_array(seq_ids), C.c_void_p(q_ptr), C.c_void_p(rows_ptr),
                                      max_len, sim), "qc_layer_similarity")
    return [float(x) for x in sim[: n_layers - 1]]


def qc_lazy_blocks(similarity: Sequence[float], eps: float, max_block: int = 0):
    n_layers = len(similarity) + 1
    sim = (C.c_float * max(1, len(similarity)))(*similarity)
    kind = (C.c_uint8 * n_layers)()
    _check(load().qc_lazy_blocks(sim, n_layers, eps, max_block, kind), "qc_lazy_blocks")
    return list(kind)


def qc_decode_step(cache, seq_ids, q_ptr: int, k_ptr: int, v_ptr: int, out_ptr: int, lse_ptr: int = 0) -> None:
    ids = seq_ids if isinstance(seq_ids, C.Array) else _i32_array(seq_ids)
    _check(load().qc_decode_step(cache, len(ids), ids, C.c_void_p(q_ptr), C.c_void_p(k_ptr), C.c_void_p(v_ptr),
                                 C.c_void_p(out_ptr), C.c_void_p(lse_ptr or None)), "qc_decode_step")


def qc_decode_begin(cache, seq_ids) -> None:
    ids = seq_ids if isinstance(seq_ids, C.Array) else _i32_array(seq_ids)
    _check(load().qc_decode_begin(cache, len(ids), ids), "qc_decode_begin")


def qc_decode_layer(cache, layer: int, q_ptr: int, k_ptr: int, v_ptr: int, out_ptr: int, lse_ptr: int = 0) -> None:
    _check(load().qc_decode_layer(cache, layer, C.c_void_p(q_ptr), C.c_void_p(k_ptr), C.c_void_p(v_ptr),
                                  C.c_void_p(out_ptr), C.c_void_p(lse_ptr or None)), "qc_decode_layer")


def qc_decode_step_host(cache, seq_ids, q_ptr: int, k_ptr: int, v_ptr: int, out_ptr: int, lse_ptr: int = 0) -> None:
    ids = seq_ids if isinstance(seq_ids, C.Array) else _i32_array(seq_ids)
    _check(load().qc_decode_step_host(cache, len(ids), ids, C.c_void_p(q_ptr), C.c_void_p(k_ptr),
                                      C.c_void_p(v_ptr), C.c_void_p(out_ptr), C.c_void_p(lse_ptr or None)),
           "qc_decode_step_host")


def qc_free_seq(cache, seq_id: int) -> None:
    _check(load().qc_free_seq(cache, seq_id), "qc_free_seq")


def qc_free(ctx=None, cache=None) -> None:
    _check(load().qc_free(ctx, cache), "qc_free")


def qc_get_stats(cache) -> qc_stats:
    st = qc_stats()
    _check(load().qc_get_stats(cache, C.byref(st)), "qc_get_stats")
    return st


def qc_debug_page_table(cache, layer: int, stream: int, seq_id: int, cap: int = 1 << 16):
    ids = (C.c_int32 * cap)()
    n_pages, n_tokens, owner = C.c_int32(), C.c_int32(), C.c_int32()
    _check(load().qc_debug_page_table(cache, layer, stream, seq_id, ids, cap, C.byref(n_pages), C.byref(n_tokens),
                                      C.byref(owner)), "qc_debug_page_table")
    return list(ids[: min(cap, n_pages.value)]), n_tokens.value, owner.value


def qc_debug_read_qcache(cache, layer: int, host_ptr: int) -> None:
    _check(load().qc_debug_read_qcache(cache, layer, C.c_void_p(host_ptr)), "qc_debug_read_qcache")


def qc_debug_read_row(cache, layer: int, stream: int, seq_id: int, token: int, kv_head: int, host_ptr: int) -> None:
    _check(load().qc_debug_read_row(cache, layer, stream, seq_id, token, kv_head, C.c_void_p(host_ptr)),
           "qc_debug_read_row")


def qc_set_option(cache, key: str, value: int) -> None:
    _check(load().qc_set_option(cache, key.encode(), value), "qc_set_option")


def qc_get_profile(cache) -> qc_profile:
    pr = qc_profile()
    _check(load().qc_get_profile(cache, C.byref(pr)), "qc_get_profile")
    return pr


QC_STATIC_MAX_ROWS = 512
QC_STATIC_SPLITS = 8
QC_STATIC_MAX_TOKENS = 65536


def qc_attend_static(device: int, cuda_stream: int, q_ptr: int, k_ptr: int, v_ptr: int, out_ptr: int, n_seqs: int,
                     n_tokens: int, n_q_heads: int, n_kv_heads: int, head_dim: int, softmax_scale: float = 0.0) -> None:
    """Decode attention with the library's built-in scratch array: for callers that cannot
    allocate device memory (see include/qc.h).  Raises QcError for sizes beyond the fixed limits."""
    _check(load().qc_attend_static(device, C.c_void_p(cuda_stream), C.c_void_p(q_ptr), C.c_void_p(k_ptr),
                                   C.c_void_p(v_ptr), C.c_void_p(out_ptr), n_seqs, n_tokens, n_q_heads, n_kv_heads,
                                   head_dim, softmax_scale), "qc_attend_static")
