"""ctypes binding of libquoka.so: argument marshalling only.

Every function has the name and the argument order of its C entry point
(include/quoka.h) and takes torch tensors where the C call takes pointers.  All
computation happens in the library's CUDA kernels; there is no Python or CPU
fallback.  If the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libquoka.so")
_lib = None

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_STATIC_LIMIT, ERR_BAD_INDEX = range(8)
STATIC_SCRATCH_BYTES = 8 << 20
BF16, F32 = 0, 1
IMPL_AUTO, IMPL_SIMT, IMPL_TENSOR = 0, 1, 2
SCORE_COSINE, SCORE_DOT = 0, 1
AGG_MAX, AGG_MEAN = 0, 1

EXPORTS = [
    "quoka_kv_budget_cap", "quoka_workspace_size", "quoka_select_queries", "quoka_score_keys",
    "quoka_update_key_norms", "quoka_select_keys", "quoka_sparse_attn", "quoka_dense_chunk_attn", "quoka_prefill_chunk",
    "quoka_prefill_chunk_host", "quoka_prefill_chunk_static", "quoka_last_device_status", "quoka_status_string", "quoka_launch_count",
    "quoka_append_kv", "quoka_check_block_table", "quoka_selftest_wait_timeout",
]


class QuokaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


class QuokaParams(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("chunk_len", C.c_int32), ("n_retain", C.c_int32), ("kv_budget", C.c_int32), ("budget_frac", C.c_float),
        ("dtype", C.c_int32), ("impl", C.c_int32), ("softmax_scale", C.c_float), ("max_ctx_len", C.c_int32),
        ("ctx_len", C.c_void_p),
        ("q_stride_b", C.c_int64), ("q_stride_h", C.c_int64), ("q_stride_t", C.c_int64),
        ("o_stride_b", C.c_int64), ("o_stride_h", C.c_int64), ("o_stride_t", C.c_int64),
        ("page_size", C.c_int32), ("max_pages_per_seq", C.c_int32), ("block_table", C.c_void_p),
        ("kv_stride_b", C.c_int64), ("kv_stride_h", C.c_int64), ("kv_stride_t", C.c_int64),
        ("kv_rows", C.c_int64),
        ("score_mode", C.c_int32), ("query_agg", C.c_int32),
        ("k_inv_norm", C.c_void_p),
    ]


def load():
    """Load libquoka.so (once).  A missing library is an error: build it with
    ``python -m paper_2602_08722_b200.build``."""
    global _lib
    if _lib is not None:
        return _lib
    _lib = _open(_LIB_PATH)
    return _lib


def open_debug_library():
    """A second, independent handle: libquoka_debug.so (built with -DQUOKA_DEBUG).  Its functions are called
    through ctypes directly (same argument types as load()'s); the functions of this module keep using libquoka.so."""
    path = os.path.join(os.path.dirname(_LIB_PATH), "libquoka_debug.so")
    return _open(path)


def _open(path):
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: the CUDA library has not been built "
                           "(python -m paper_2602_08722_b200.build); there is no fallback path")
    lib = C.CDLL(path)
    lib.quoka_status_string.restype = C.c_char_p
    lib.quoka_status_string.argtypes = [C.c_int]
    lib.quoka_launch_count.restype = C.c_int64
    vp, sz = C.c_void_p, C.c_size_t
    pp = C.POINTER(QuokaParams)
    lib.quoka_kv_budget_cap.argtypes = [pp, C.POINTER(C.c_int32)]
    lib.quoka_workspace_size.argtypes = [pp, C.POINTER(C.c_size_t)]
    lib.quoka_select_queries.argtypes = [pp, vp, vp, vp, vp, sz, vp]
    lib.quoka_score_keys.argtypes = [pp, vp, vp, vp, vp, sz, vp]
    lib.quoka_select_keys.argtypes = [pp, vp, vp, vp, vp, sz, vp]
    lib.quoka_update_key_norms.argtypes = [pp, vp, vp, C.c_int32, vp, sz, vp]
    lib.quoka_sparse_attn.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.quoka_dense_chunk_attn.argtypes = [pp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.quoka_prefill_chunk.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.quoka_prefill_chunk_host.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.quoka_prefill_chunk_static.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp]
    lib.quoka_last_device_status.argtypes = [vp, vp, C.POINTER(C.c_int32)]
    lib.quoka_append_kv.argtypes = [pp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.quoka_check_block_table.argtypes = [pp, vp, vp]
    lib.quoka_selftest_wait_timeout.argtypes = [vp, C.c_int64, vp, vp]
    for name in EXPORTS:
        if name not in ("quoka_status_string", "quoka_launch_count"):
            getattr(lib, name).restype = C.c_int
    return lib


def status_string(status: int) -> str:
    return load().quoka_status_string(int(status)).decode()


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(status: int, where: str):
    if status != OK:
        raise QuokaError(status, where)


def make_params(q, k_cache, out, ctx_len, *, n_retain, kv_budget=0, budget_frac=0.0, max_ctx_len,
                block_table=None, impl=IMPL_AUTO, softmax_scale=0.0, score_mode=SCORE_COSINE,
                query_agg=AGG_MAX) -> QuokaParams:
    """Fill quoka_params from tensors: q/out (b, n_Q, C, d); k_cache (b, n_KV, rows, d)
    contiguous or (pages, n_KV, 64, d) with a block table (b, max_pages)."""
    b, n_q, c, d = q.shape
    p = QuokaParams()
    p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim = b, n_q, k_cache.shape[1], d
    p.chunk_len, p.n_retain = c, int(n_retain)
    p.kv_budget, p.budget_frac = int(kv_budget), float(budget_frac)
    p.dtype = BF16 if q.dtype == torch.bfloat16 else F32
    p.impl, p.softmax_scale, p.max_ctx_len = int(impl), float(softmax_scale), int(max_ctx_len)
    p.score_mode, p.query_agg = int(score_mode), int(query_agg)
    p.ctx_len = ctx_len.data_ptr()
    p.q_stride_b, p.q_stride_h, p.q_stride_t = q.stride(0), q.stride(1), q.stride(2)
    p.o_stride_b, p.o_stride_h, p.o_stride_t = out.stride(0), out.stride(1), out.stride(2)
    p.kv_stride_b, p.kv_stride_h, p.kv_stride_t = k_cache.stride(0), k_cache.stride(1), k_cache.stride(2)
    if block_table is None:
        p.page_size, p.max_pages_per_seq, p.block_table = 0, 0, None
        p.kv_rows = k_cache.shape[2]
    else:
        p.page_size, p.max_pages_per_seq, p.block_table = 64, block_table.shape[1], block_table.data_ptr()
        p.kv_rows = k_cache.shape[0]
    return p


def quoka_kv_budget_cap(p: QuokaParams) -> int:
    cap = C.c_int32(0)
    _check(load().quoka_kv_budget_cap(C.byref(p), C.byref(cap)), "quoka_kv_budget_cap")
    return cap.value


def quoka_workspace_size(p: QuokaParams) -> int:
    n = C.c_size_t(0)
    _check(load().quoka_workspace_size(C.byref(p), C.byref(n)), "quoka_workspace_size")
    return n.value


def alloc_workspace(p: QuokaParams, device="cuda") -> torch.Tensor:
    """A zeroed uint8 tensor of quoka_workspace_size bytes (torch's allocator is 512-byte aligned)."""
    return torch.zeros(quoka_workspace_size(p), dtype=torch.uint8, device=device)


def quoka_select_queries(p, q, q_idx, qbar, ws, stream=None):
    _check(load().quoka_select_queries(C.byref(p), _ptr(q), _ptr(q_idx), _ptr(qbar), _ptr(ws), ws.numel(),
                                       _stream(stream)), "quoka_select_queries")


def quoka_score_keys(p, qbar, k_cache, scores, ws, stream=None):
    _check(load().quoka_score_keys(C.byref(p), _ptr(qbar), _ptr(k_cache), _ptr(scores), _ptr(ws), ws.numel(),
                                   _stream(stream)), "quoka_score_keys")


def quoka_update_key_norms(p, k_cache, k_inv_norm, all_rows, ws, stream=None):
    _check(load().quoka_update_key_norms(C.byref(p), _ptr(k_cache), _ptr(k_inv_norm), int(bool(all_rows)), _ptr(ws),
                                         ws.numel(), _stream(stream)), "quoka_update_key_norms")


def quoka_select_keys(p, scores, k_idx, k_cnt, ws, stream=None):
    _check(load().quoka_select_keys(C.byref(p), _ptr(scores), _ptr(k_idx), _ptr(k_cnt), _ptr(ws), ws.numel(),
                                    _stream(stream)), "quoka_select_keys")


def quoka_sparse_attn(p, q, k_cache, v_cache, k_idx, k_cnt, out, lse, ws, stream=None):
    _check(load().quoka_sparse_attn(C.byref(p), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(k_idx), _ptr(k_cnt),
                                    _ptr(out), _ptr(lse), _ptr(ws), ws.numel(), _stream(stream)),
           "quoka_sparse_attn")


def quoka_dense_chunk_attn(p, q, k_cache, v_cache, out, lse, ws, stream=None):
    _check(load().quoka_dense_chunk_attn(C.byref(p), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(out), _ptr(lse),
                                         _ptr(ws), ws.numel(), _stream(stream)), "quoka_dense_chunk_attn")


def quoka_prefill_chunk(p, q, k_cache, v_cache, out, k_idx_out, k_cnt_out, ws, stream=None):
    _check(load().quoka_prefill_chunk(C.byref(p), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(out),
                                      _ptr(k_idx_out), _ptr(k_cnt_out), _ptr(ws), ws.numel(), _stream(stream)),
           "quoka_prefill_chunk")


def quoka_prefill_chunk_host(p, ctx_len_host, q_host, k_new_host, v_new_host, out_host, q_dev, k_cache, v_cache,
                             out_dev, ws, stream=None):
    _check(load().quoka_prefill_chunk_host(C.byref(p), _ptr(ctx_len_host), _ptr(q_host), _ptr(k_new_host),
                                           _ptr(v_new_host), _ptr(out_host), _ptr(q_dev), _ptr(k_cache),
                                           _ptr(v_cache), _ptr(out_dev), _ptr(ws), ws.numel(), _stream(stream)),
           "quoka_prefill_chunk_host")


def quoka_prefill_chunk_static(p, q, k_cache, v_cache, out, k_idx_out, k_cnt_out, stream=None):
    """The fused call on the library's built-in scratch array: for callers that cannot allocate a
    workspace.  Raises QuokaError(ERR_STATIC_LIMIT) when the problem does not fit the array."""
    _check(load().quoka_prefill_chunk_static(C.byref(p), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(out),
                                             _ptr(k_idx_out), _ptr(k_cnt_out), _stream(stream)),
           "quoka_prefill_chunk_static")


def quoka_last_device_status(ws, stream=None) -> int:
    st = C.c_int32(0)
    _check(load().quoka_last_device_status(_ptr(ws), _stream(stream), C.byref(st)), "quoka_last_device_status")
    return st.value


def quoka_append_kv(p, k_new, v_new, k_cache, v_cache, k_inv_norm, ws, stream=None):
    _check(load().quoka_append_kv(C.byref(p), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache),
                                  _ptr(k_inv_norm), _ptr(ws), ws.numel(), _stream(stream)), "quoka_append_kv")


def quoka_check_block_table(p, ctx_len_host, block_table_host) -> int:
    """Status of the host-side block-table check (OK or ERR_INVALID_ARG); both arguments are CPU int32 tensors."""
    return int(load().quoka_check_block_table(C.byref(p), _ptr(ctx_len_host), _ptr(block_table_host)))


def quoka_selftest_wait_timeout(ws, limit_cycles, gave_up, stream=None):
    _check(load().quoka_selftest_wait_timeout(_ptr(ws), int(limit_cycles), _ptr(gave_up), _stream(stream)),
           "quoka_selftest_wait_timeout")


def quoka_launch_count() -> int:
    return int(load().quoka_launch_count())
