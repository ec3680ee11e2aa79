"""ctypes binding of libxkv.so -- argument marshalling only; every step runs in the CUDA library.

The functions carry the names and argument order of include/xkv.h.  Device buffers may be passed
as torch tensors (their data_ptr is taken) or as integer addresses.  A negative status raises
XkvError.  There is no fallback: if libxkv.so has not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libxkv.so")

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_BUDGET = -1, -2, -3, -4
ERR_CUDA, ERR_TIMEOUT, ERR_CAPACITY = -5, -6, -7
POOL_MAX, POOL_AVG = 0, 1
OP_SCORE, OP_SELECT_COMPACT, OP_DECODE_ATTN, OP_PREFILL_ATTN = 0, 1, 2, 3
BUDGET_PER_LAYER, BUDGET_PER_SEQUENCE, BUDGET_PER_HEAD = 0, 1, 2
KV_BF16, KV_INT8 = 0, 1

STATIC_SCRATCH_BYTES = 16 << 20

EXPORTS = ("xkv_score", "xkv_score_lse", "xkv_prefill_attn", "xkv_batch_curves", "xkv_head_curves", "xkv_build_block_table", "xkv_alloc_budgets", "xkv_average_budgets", "xkv_select_compact", "xkv_decode_attn", "xkv_decode_attn_static",
           "xkv_workspace_bytes",
           "xkv_read_device_status", "xkv_profile_events", "xkv_test_hooks", "xkv_launch_count", "xkv_status_string",
           "xkv_version")


class XkvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class Dims(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("window", ctypes.c_int32), ("pool_kernel", ctypes.c_int32),
                ("pool_mode", ctypes.c_int32), ("scale", ctypes.c_float),
                ("kv_stride_token", ctypes.c_int64), ("kv_stride_head", ctypes.c_int64)]


class Cache(ctypes.Structure):
    _fields_ = [("k_pages", ctypes.c_void_p), ("v_pages", ctypes.c_void_p),
                ("block_table", ctypes.c_void_p), ("seq_lens", ctypes.c_void_p),
                ("n_layers", ctypes.c_int32), ("page_size", ctypes.c_int32),
                ("max_pages_per_seq", ctypes.c_int32), ("n_pages", ctypes.c_int32),
                ("k_scales", ctypes.c_void_p), ("v_scales", ctypes.c_void_p),
                ("kv_format", ctypes.c_int32), ("reserved", ctypes.c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2412_05896_b200.build` "
                           "(there is no CPU fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    L.xkv_score.restype = i32
    L.xkv_score.argtypes = [ctypes.POINTER(Dims), vp, vp, vp, i64, i32, vp, vp, vp, vp, i32, vp, sz, vp]
    L.xkv_score_lse.restype = i32
    L.xkv_score_lse.argtypes = [ctypes.POINTER(Dims), vp, vp, vp, i64, i32, vp, vp, vp, vp, vp, i32, vp, sz, vp]
    L.xkv_prefill_attn.restype = i32
    L.xkv_prefill_attn.argtypes = [ctypes.POINTER(Dims), vp, vp, vp, vp, i64, i32, vp, vp, vp, sz, vp]
    L.xkv_batch_curves.restype = i32
    L.xkv_batch_curves.argtypes = [vp, i32, i32, i32, i32, vp, vp]
    L.xkv_head_curves.restype = i32
    L.xkv_head_curves.argtypes = [ctypes.POINTER(Dims), vp, vp, vp, i64, i32, vp, i32, vp]
    L.xkv_build_block_table.restype = i32
    L.xkv_build_block_table.argtypes = [vp, vp, ctypes.POINTER(Cache), i32, vp]
    L.xkv_alloc_budgets.restype = i32
    L.xkv_alloc_budgets.argtypes = [vp, i32, i32, i32, vp, i32, i64, ctypes.c_double, i32, i32, vp, vp]
    L.xkv_average_budgets.restype = i32
    L.xkv_average_budgets.argtypes = [vp, i32, i32, vp]
    L.xkv_select_compact.restype = i32
    L.xkv_select_compact.argtypes = [ctypes.POINTER(Dims), i32, vp, i32, vp, vp, vp, vp, vp, i64, i32,
                                     ctypes.POINTER(Cache), vp, i32, vp, sz, vp]
    L.xkv_decode_attn.restype = i32
    L.xkv_decode_attn.argtypes = [ctypes.POINTER(Dims), ctypes.POINTER(Cache), i32, i32, vp, vp, vp, vp, vp,
                                  i32, vp, sz, vp]
    L.xkv_decode_attn_static.restype = i32
    L.xkv_decode_attn_static.argtypes = [ctypes.POINTER(Dims), ctypes.POINTER(Cache), i32, i32, vp, vp, vp, vp,
                                         vp, i32, vp, vp]
    L.xkv_workspace_bytes.restype = sz
    L.xkv_workspace_bytes.argtypes = [i32, ctypes.POINTER(Dims), i32, i64, i32, i32, i32]
    L.xkv_read_device_status.restype = i32
    L.xkv_read_device_status.argtypes = [vp, vp]
    L.xkv_profile_events.restype = None
    L.xkv_profile_events.argtypes = [vp, vp]
    L.xkv_test_hooks.restype = None
    L.xkv_test_hooks.argtypes = [i64, i32]
    L.xkv_launch_count.restype = i64
    L.xkv_launch_count.argtypes = []
    L.xkv_status_string.restype = ctypes.c_char_p
    L.xkv_status_string.argtypes = [i32]
    L.xkv_version.restype = i32
    L.xkv_version.argtypes = []
    _lib = L
    return L


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()       # torch tensor


def _nbytes(x) -> int:
    if isinstance(x, np.ndarray):
        return x.nbytes
    return x.numel() * x.element_size()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(status: int, where: str) -> int:
    if status < 0:
        raise XkvError(status, where)
    return status


def status_string(status: int) -> str:
    return lib().xkv_status_string(status).decode()


def version() -> int:
    return lib().xkv_version()


def launch_count() -> int:
    return lib().xkv_launch_count()


def workspace_bytes(op: int, dims: Dims, max_seqlen: int = 0, total_tokens: int = 0, n_layers: int = 0,
                    max_cache_len: int = 0, chunk_rows: int = 0) -> int:
    n = lib().xkv_workspace_bytes(op, ctypes.byref(dims), max_seqlen, total_tokens, n_layers, max_cache_len,
                                  chunk_rows)
    if n == 0:
        raise XkvError(ERR_INVALID_ARG, "xkv_workspace_bytes")
    return n


def score(dims: Dims, q_win, k, cu_seqlens, total_tokens: int, max_seqlen: int, scores, sorted_scores, gains,
          mass, curve_len: int, workspace, stream=None) -> None:
    _check(lib().xkv_score(ctypes.byref(dims), _ptr(q_win), _ptr(k), _ptr(cu_seqlens), total_tokens, max_seqlen,
                           _ptr(scores), _ptr(sorted_scores), _ptr(gains), _ptr(mass), curve_len,
                           _ptr(workspace), _nbytes(workspace), _stream(stream)), "xkv_score")


def score_lse(dims: Dims, q_win, k, cu_seqlens, total_tokens: int, max_seqlen: int, lse, scores, sorted_scores,
              gains, mass, curve_len: int, workspace, stream=None) -> None:
    """xkv_score with the window rows' normalisers given (lse dev fp32 [Hq, T] from prefill_attn)."""
    _check(lib().xkv_score_lse(ctypes.byref(dims), _ptr(q_win), _ptr(k), _ptr(cu_seqlens), total_tokens, max_seqlen,
                               _ptr(lse), _ptr(scores), _ptr(sorted_scores), _ptr(gains), _ptr(mass), curve_len,
                               _ptr(workspace), _nbytes(workspace), _stream(stream)), "xkv_score_lse")


def prefill_attn(dims: Dims, q, k, v, cu_seqlens, total_tokens: int, max_seqlen: int, out, lse, workspace,
                 stream=None) -> None:
    """q dev bf16 [T, Hq, d], k/v dev bf16 [T, Hkv, d] -> out dev bf16 [T, Hq, d], lse dev fp32 [Hq, T]."""
    _check(lib().xkv_prefill_attn(ctypes.byref(dims), _ptr(q), _ptr(k), _ptr(v), _ptr(cu_seqlens), total_tokens,
                                  max_seqlen, _ptr(out), _ptr(lse), _ptr(workspace), _nbytes(workspace),
                                  _stream(stream)), "xkv_prefill_attn")


def batch_curves(gains, n_layers: int, batch: int, curve_len: int, divisor: int, out, stream=None) -> None:
    """gains dev [L, B, curve_len] -> out dev [L, curve_len] = sum over b / divisor."""
    _check(lib().xkv_batch_curves(_ptr(gains), n_layers, batch, curve_len, divisor, _ptr(out), _stream(stream)),
           "xkv_batch_curves")


def head_curves(dims: Dims, scores, sorted_scores, cu_seqlens, total_tokens: int, max_seqlen: int, head_gains,
                curve_len: int, stream=None) -> None:
    """scores, sorted dev [Hkv, T] of one layer -> head_gains dev [Hkv, B, curve_len]."""
    _check(lib().xkv_head_curves(ctypes.byref(dims), _ptr(scores), _ptr(sorted_scores), _ptr(cu_seqlens), total_tokens,
                                 max_seqlen, _ptr(head_gains), curve_len, _stream(stream)), "xkv_head_curves")


def build_block_table(first_page, n_pages_lb, cache: Cache, batch: int, stream=None) -> None:
    _check(lib().xkv_build_block_table(_ptr(first_page), _ptr(n_pages_lb), ctypes.byref(cache), batch,
                                       _stream(stream)), "xkv_build_block_table")


def alloc_budgets(gains: np.ndarray, prefix_len, per_sequence: bool = False, total: int = -1,
                  r_target: float = 0.0, n_min: int = 0, n_max: int = 0):
    """gains: host float32 [L, B, curve_len].  Returns (budgets int32 [L] or [B, L], r_avg)."""
    gains = np.ascontiguousarray(gains, dtype=np.float32)
    L, B, curve_len = gains.shape
    prefix = np.ascontiguousarray(prefix_len, dtype=np.int32)
    assert prefix.shape == (B,)
    budgets = np.zeros((B, L) if per_sequence else (L,), dtype=np.int32)
    r_avg = np.zeros(B if per_sequence else 1, dtype=np.float64)
    _check(lib().xkv_alloc_budgets(gains.ctypes.data, L, B, curve_len, prefix.ctypes.data, int(per_sequence),
                                   int(total), float(r_target), n_min, n_max, budgets.ctypes.data,
                                   r_avg.ctypes.data), "xkv_alloc_budgets")
    return budgets, (r_avg if per_sequence else float(r_avg[0]))


def average_budgets(lists) -> np.ndarray:
    """lists: int [n_tasks, n_layers] recorded by alloc_budgets for sampled tasks -> the averaged list [n_layers]."""
    lists = np.ascontiguousarray(lists, dtype=np.int32)
    n_tasks, L = lists.shape
    out = np.zeros(L, dtype=np.int32)
    _check(lib().xkv_average_budgets(lists.ctypes.data, n_tasks, L, out.ctypes.data), "xkv_average_budgets")
    return out


def select_compact(dims: Dims, layer: int, budget, per_sequence, scores, sorted_scores, k, v, cu_seqlens,
                   total_tokens: int, max_seqlen: int, cache: Cache, sel, sel_stride: int, workspace,
                   stream=None) -> None:
    budget = np.ascontiguousarray(np.atleast_1d(budget), dtype=np.int32)
    _check(lib().xkv_select_compact(ctypes.byref(dims), layer, budget.ctypes.data, int(per_sequence),
                                    _ptr(scores), _ptr(sorted_scores), _ptr(k), _ptr(v), _ptr(cu_seqlens),
                                    total_tokens, max_seqlen, ctypes.byref(cache), _ptr(sel), sel_stride,
                                    _ptr(workspace), _nbytes(workspace), _stream(stream)), "xkv_select_compact")


def decode_attn(dims: Dims, cache: Cache, layer_begin: int, layer_end: int, q, k_new, v_new, out, lse,
                chunk_rows: int, workspace, stream=None) -> None:
    _check(lib().xkv_decode_attn(ctypes.byref(dims), ctypes.byref(cache), layer_begin, layer_end, _ptr(q),
                                 _ptr(k_new), _ptr(v_new), _ptr(out), _ptr(lse), chunk_rows, _ptr(workspace),
                                 _nbytes(workspace), _stream(stream)), "xkv_decode_attn")


def decode_attn_static(dims: Dims, cache: Cache, layer_begin: int, layer_end: int, q, k_new, v_new, out, lse,
                       chunk_rows: int, status_out=None, stream=None) -> None:
    """xkv_decode_attn without a caller workspace: the scratch is a fixed array inside the library
    (STATIC_SCRATCH_BYTES), for callers that must not allocate.  Raises XkvError(ERR_WORKSPACE) when the
    problem needs more scratch than that.  Keep calls on one stream: they share the array."""
    _check(lib().xkv_decode_attn_static(ctypes.byref(dims), ctypes.byref(cache), layer_begin, layer_end, _ptr(q),
                                        _ptr(k_new), _ptr(v_new), _ptr(out), _ptr(lse), chunk_rows,
                                        _ptr(status_out), _stream(stream)), "xkv_decode_attn_static")


def profile_events(start, stop) -> None:
    """start/stop: torch.cuda.Event(enable_timing=True) that have been recorded once, or None, None."""
    lib().xkv_profile_events(None if start is None else start.cuda_event,
                             None if stop is None else stop.cuda_event)


def test_hooks(wait_limit_ns: int = 0, withhold_decode_item: int = -1) -> None:
    """Shortens every bounded device wait and/or withholds one decode merge ticket (tests of the expiry path);
    test_hooks() restores the defaults."""
    lib().xkv_test_hooks(wait_limit_ns, withhold_decode_item)


def read_device_status(workspace, stream=None) -> int:
    """The workspace's sticky status word (first error since the last read); reading resets it."""
    return lib().xkv_read_device_status(_ptr(workspace), _stream(stream))
