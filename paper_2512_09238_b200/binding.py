"""ctypes binding of the C-ABI library declared in ``include/tca.h``.

Argument marshalling only: every function below has the name and the argument order of
its C counterpart, takes torch CUDA tensors (device buffers) or numpy arrays (host
buffers), passes raw pointers and sizes, and raises :class:`TcaError` on a non-zero
status.  Nothing is computed in Python and nothing falls back to the CPU: if
``libtca.so`` has not been built, importing the library handle raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libtca.so")

TCA_OK, TCA_ERR_INVALID_ARG, TCA_ERR_UNSUPPORTED, TCA_ERR_WORKSPACE = 0, -1, -2, -3
TCA_ERR_CUDA, TCA_ERR_TIMEOUT, TCA_ERR_CAPACITY, TCA_ERR_SCRATCH_LIMIT, TCA_ERR_BOUNDS = -4, -5, -6, -7, -8
TCA_DECODE_STATIC_SCRATCH_BYTES = 16 << 20
TCA_F32, TCA_BF16 = 0, 1
TCA_FLAG_PREFILL_SIMT, TCA_FLAG_ENTROPY_INDEX, TCA_FLAG_RANDOM_ORDER, TCA_FLAG_FLAT_TOPB = 1, 2, 4, 8
TCA_FLAG_PREFILL_BAND_FIRST = 16
TCA_BUILD_DEBUG_BOUNDS = 1
(TCA_OP_SCORE, TCA_OP_SELECT, TCA_OP_COMPACT, TCA_OP_PREFILL, TCA_OP_DECODE, TCA_OP_APPEND, TCA_OP_CALIB,
 TCA_OP_SCORE_SELECT) = range(8)
TCA_STATE_WORDS = 8

EXPORTS = (
    "tca_strerror", "tca_version", "tca_budget_resolve", "tca_workspace_bytes", "tca_score",
    "tca_select", "tca_cache_init", "tca_compact_kv", "tca_attn_prefill", "tca_attn_decode",
    "tca_cache_append", "tca_ws_status", "tca_attn_decode_static", "tca_attn_prefill_rows",
    "tca_calib_colmean", "tca_calib_score", "tca_calib_choose", "tca_calib_candidates",
    "tca_decode_static_status", "tca_selftest_wait_expiry", "tca_score_select", "tca_build_info",
    "tca_cache_status", "tca_attn_prefill_gather", "tca_compact_kv_range",
)


class TcaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().tca_strerror(status).decode()} ({status})")


class tca_params(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("block", C.c_int32), ("window", C.c_int32),
                ("alpha", C.c_float), ("sm_scale", C.c_float), ("dtype", C.c_int32),
                ("flags", C.c_int32), ("seed", C.c_int32)]


class tca_cache_desc(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("pos", C.c_void_p), ("state", C.c_void_p),
                ("rows_total", C.c_int64), ("n_units", C.c_int64), ("tail_cap", C.c_int64),
                ("seg_start", C.c_void_p), ("global_cap", C.c_void_p), ("n_global", C.c_void_p),
                ("tail_head", C.c_void_p), ("n_tail", C.c_void_p), ("seq_len", C.c_void_p),
                ("t_keep", C.c_void_p)]


_lib = None


def load_library(path: str) -> C.CDLL:
    """Load a build of the library from `path` and declare the argument types of its entry points."""
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with "
                           "`python -m paper_2512_09238_b200._build` (needs nvcc)")
    L = C.CDLL(path)
    L.tca_strerror.restype = C.c_char_p
    L.tca_strerror.argtypes = [C.c_int]
    L.tca_version.restype = C.c_int
    L.tca_workspace_bytes.restype = C.c_size_t
    L.tca_workspace_bytes.argtypes = [C.POINTER(tca_params), C.c_int64, C.c_int]
    L.tca_budget_resolve.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int64, C.c_void_p,
                                     C.c_void_p, C.c_void_p]
    P = C.POINTER(tca_params)
    D = C.POINTER(tca_cache_desc)
    vp, i64, sz = C.c_void_p, C.c_int64, C.c_size_t
    L.tca_score.argtypes = [P, vp, vp, i64, vp, vp, sz, vp]
    L.tca_select.argtypes = [P, vp, i64, vp, C.c_int32, vp, vp, vp, vp, vp, sz, vp]
    L.tca_score_select.argtypes = [P, vp, vp, i64, vp, C.c_int32, vp, vp, vp, vp, vp, vp, sz, vp]
    L.tca_cache_init.argtypes = [P, D, vp]
    L.tca_compact_kv.argtypes = [P, vp, vp, i64, vp, vp, vp, D, vp]
    L.tca_compact_kv_range.argtypes = [P, vp, vp, i64, i64, i64, vp, vp, vp, D, vp]
    L.tca_attn_prefill.argtypes = [P, vp, vp, vp, i64, D, vp, vp, sz, vp]
    L.tca_attn_prefill_rows.argtypes = [P, vp, vp, vp, i64, i64, i64, D, vp, vp, sz, vp]
    L.tca_attn_prefill_gather.argtypes = [P, vp, vp, vp, i64, i64, i64, vp, vp, vp, vp, sz, vp]
    L.tca_calib_colmean.argtypes = [P, vp, vp, i64, vp, vp, sz, vp]
    L.tca_calib_score.argtypes = [P, vp, i64, vp, vp, vp, vp]
    L.tca_calib_choose.argtypes = [vp, vp, C.c_int, C.c_double]
    L.tca_calib_candidates.argtypes = [C.c_int, C.c_int, C.c_double, vp]
    L.tca_attn_decode.argtypes = [P, vp, D, vp, vp, sz, vp]
    L.tca_cache_append.argtypes = [P, D, vp, vp, vp, vp]
    L.tca_ws_status.argtypes = [vp, vp]
    L.tca_cache_status.argtypes = [D, vp, vp]
    L.tca_attn_decode_static.argtypes = [P, vp, D, vp, vp]
    L.tca_decode_static_status.argtypes = [vp]
    L.tca_selftest_wait_expiry.argtypes = [vp, C.c_uint64, vp, vp]
    L.tca_build_info.argtypes = []
    for name in EXPORTS:
        if name not in ("tca_strerror", "tca_workspace_bytes"):
            getattr(L, name).restype = C.c_int
    return L


def lib() -> C.CDLL:
    """The loaded library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        # TCA_LIBRARY names another build of the same library, e.g. the range-checked libtca_dbg.so
        _lib = load_library(os.environ.get("TCA_LIBRARY") or LIB_PATH)
    return _lib


# ----------------------------------------------------------------------------- helpers
def make_params(batch, n_q_heads, n_kv_heads, head_dim, block, window, alpha=0.5, sm_scale=None,
                dtype=TCA_BF16, flags=0, seed=0) -> tca_params:
    if sm_scale is None:
        sm_scale = 1.0 / float(np.sqrt(head_dim))
    return tca_params(batch, n_q_heads, n_kv_heads, head_dim, block, window, alpha, sm_scale, dtype, flags, seed)


def _dev(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("device buffers must be contiguous CUDA tensors")
    return t.data_ptr()


def _host(a: Optional[np.ndarray], dtype) -> Optional[int]:
    if a is None:
        return None
    if a.dtype != dtype or not a.flags["C_CONTIGUOUS"]:
        raise ValueError(f"host buffer must be a C-contiguous {np.dtype(dtype).name} array")
    return a.ctypes.data


def _stream(stream=None) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def _check(status: int, where: str) -> None:
    if status != TCA_OK:
        raise TcaError(status, where)


def _ws_args(ws: Optional[torch.Tensor]):
    return (_dev(ws), 0 if ws is None else ws.numel() * ws.element_size())


def alloc_workspace(prm: tca_params, L: int, op: int, device="cuda") -> torch.Tensor:
    """A zero-filled device buffer of tca_workspace_bytes(prm, L, op) bytes (torch owns the
    memory).  Zero-filled because the first word of the prefill and decode workspaces is a
    sticky error flag that tca_ws_status reads."""
    n = tca_workspace_bytes(prm, L, op)
    if n == 0:
        raise TcaError(TCA_ERR_INVALID_ARG, "tca_workspace_bytes")
    return torch.zeros(n, dtype=torch.uint8, device=device)


# ----------------------------------------------------------------------------- the C entry points
def tca_version() -> int:
    return lib().tca_version()


def tca_strerror(status: int) -> str:
    return lib().tca_strerror(status).decode()


def tca_workspace_bytes(prm: tca_params, L: int, op: int) -> int:
    return int(lib().tca_workspace_bytes(C.byref(prm), L, op))


def tca_budget_resolve(p: np.ndarray, m: int):
    """p [Hkv, nK] float64 -> (n_k [Hkv, nK] int32, n_sel [Hkv] int64, tbar [Hkv] int32)."""
    p = np.ascontiguousarray(p, dtype=np.float64)
    H, nK = p.shape
    n_k = np.zeros((H, nK), dtype=np.int32)
    n_sel = np.zeros(H, dtype=np.int64)
    tbar = np.zeros(H, dtype=np.int32)
    _check(lib().tca_budget_resolve(p.ctypes.data, H, nK, m, n_k.ctypes.data, n_sel.ctypes.data,
                                    tbar.ctypes.data), "tca_budget_resolve")
    return n_k, n_sel, tbar


def tca_score(prm, q_last, K, L, logscore, ws, stream=None) -> None:
    _check(lib().tca_score(C.byref(prm), _dev(q_last), _dev(K), L, _dev(logscore), *_ws_args(ws),
                           _stream(stream)), "tca_score")


def tca_select(prm, logscore, L, n_k, idx, offsets_dev, h_out, t_out, ws, stream=None) -> None:
    n_k = np.ascontiguousarray(n_k, dtype=np.int32)
    _check(lib().tca_select(C.byref(prm), _dev(logscore), L, _host(n_k, np.int32), n_k.shape[1], _dev(idx),
                            _dev(offsets_dev), _dev(h_out), _dev(t_out), *_ws_args(ws), _stream(stream)),
           "tca_select")


def tca_score_select(prm, q_last, K, L, n_k, logscore, idx, offsets_dev, h_out, t_out, ws, stream=None) -> None:
    n_k = np.ascontiguousarray(n_k, dtype=np.int32)
    _check(lib().tca_score_select(C.byref(prm), _dev(q_last), _dev(K), L, _host(n_k, np.int32), n_k.shape[1],
                                  _dev(logscore), _dev(idx), _dev(offsets_dev), _dev(h_out), _dev(t_out),
                                  *_ws_args(ws), _stream(stream)), "tca_score_select")


def tca_build_info() -> int:
    return lib().tca_build_info()


def tca_cache_status(cache: "Cache", stream=None):
    """(status, detail) with detail = [unit, which check, offending value] when status is TCA_ERR_BOUNDS."""
    detail = np.zeros(3, dtype=np.int64)
    st = lib().tca_cache_status(C.byref(cache.desc), _stream(stream), detail.ctypes.data)
    return st, detail


def tca_cache_init(prm, cache: "Cache", stream=None) -> None:
    _check(lib().tca_cache_init(C.byref(prm), C.byref(cache.desc), _stream(stream)), "tca_cache_init")


def tca_compact_kv(prm, K, V, L, idx, offsets_dev, offsets_host, cache: "Cache", stream=None) -> None:
    _check(lib().tca_compact_kv(C.byref(prm), _dev(K), _dev(V), L, _dev(idx), _dev(offsets_dev),
                                _host(offsets_host, np.int64), C.byref(cache.desc), _stream(stream)),
           "tca_compact_kv")


def tca_compact_kv_range(prm, K, V, L, pos_begin, pos_end, idx, offsets_dev, offsets_host, cache: "Cache",
                         stream=None) -> None:
    _check(lib().tca_compact_kv_range(C.byref(prm), _dev(K), _dev(V), L, pos_begin, pos_end, _dev(idx),
                                      _dev(offsets_dev), _host(offsets_host, np.int64), C.byref(cache.desc),
                                      _stream(stream)), "tca_compact_kv_range")


def tca_attn_prefill(prm, Q, K, V, L, cache: "Cache", O, ws, stream=None) -> None:
    _check(lib().tca_attn_prefill(C.byref(prm), _dev(Q), _dev(K), _dev(V), L, C.byref(cache.desc), _dev(O),
                                  *_ws_args(ws), _stream(stream)), "tca_attn_prefill")


def tca_attn_prefill_rows(prm, Q, K, V, L, row_begin, row_end, cache: "Cache", O, ws, stream=None) -> None:
    _check(lib().tca_attn_prefill_rows(C.byref(prm), _dev(Q), _dev(K), _dev(V), L, row_begin, row_end,
                                       C.byref(cache.desc), _dev(O), *_ws_args(ws), _stream(stream)),
           "tca_attn_prefill_rows")


def tca_attn_prefill_gather(prm, Q, K, V, L, row_begin, row_end, idx, offsets_dev, O, ws, stream=None) -> None:
    _check(lib().tca_attn_prefill_gather(C.byref(prm), _dev(Q), _dev(K), _dev(V), L, row_begin, row_end,
                                         _dev(idx), _dev(offsets_dev), _dev(O), *_ws_args(ws), _stream(stream)),
           "tca_attn_prefill_gather")


def tca_attn_decode(prm, q, cache: "Cache", O, ws, stream=None) -> None:
    _check(lib().tca_attn_decode(C.byref(prm), _dev(q), C.byref(cache.desc), _dev(O), *_ws_args(ws),
                                 _stream(stream)), "tca_attn_decode")


def tca_attn_decode_static(prm, q, cache: "Cache", O, stream=None) -> None:
    """tca_attn_decode without a workspace: the partials live in a 16 MiB array inside the
    library, so the call allocates nothing.  For callers that cannot allocate device memory
    (all of it owned by a host engine's pool, or no allocator available in a latency-critical
    loop).  Calls share that array: do not let two of them overlap on the GPU."""
    _check(lib().tca_attn_decode_static(C.byref(prm), _dev(q), C.byref(cache.desc), _dev(O), _stream(stream)),
           "tca_attn_decode_static")


def tca_decode_static_status(stream=None) -> int:
    """TCA_OK, or TCA_ERR_TIMEOUT if a bounded wait gave up inside a tca_attn_decode_static call on
    this device since the last query (the array's status word and counters are then cleared)."""
    return lib().tca_decode_static_status(_stream(stream))


def tca_selftest_wait_expiry(ws, limit_ns: int, waited_ns=None, stream=None) -> None:
    """Makes one bounded device-side wait run out after limit_ns and leave through the kernels'
    abort path; afterwards tca_ws_status(ws) is TCA_ERR_TIMEOUT."""
    _check(lib().tca_selftest_wait_expiry(_dev(ws), int(limit_ns), _dev(waited_ns), _stream(stream)),
           "tca_selftest_wait_expiry")


def tca_cache_append(prm, cache: "Cache", k_new, v_new, q_cur, stream=None) -> None:
    _check(lib().tca_cache_append(C.byref(prm), C.byref(cache.desc), _dev(k_new), _dev(v_new), _dev(q_cur),
                                  _stream(stream)), "tca_cache_append")


def tca_ws_status(ws, stream=None) -> int:
    return lib().tca_ws_status(_dev(ws), _stream(stream))


# ----------------------------------------------------------------------------- cache descriptor holder
class Cache:
    """Owns the buffers a ``tca_cache_desc`` points at (torch device tensors, numpy host
    arrays) and keeps them alive.  Layout per unit: ``global_cap[u]`` rows for the global
    subset followed by ``tail_cap`` ring rows; segments are laid out back to back."""

    def __init__(self, prm: tca_params, global_cap: Sequence[int], tail_cap: int, t_keep: Sequence[int],
                 device="cuda", init: bool = True):
        U = prm.batch * prm.n_kv_heads
        gcap = np.ascontiguousarray(global_cap, dtype=np.int64)
        if gcap.shape != (U,):
            raise ValueError("global_cap must have one entry per (sequence, KV head)")
        self.prm = prm
        self.global_cap = gcap
        self.tail_cap = int(tail_cap)
        seg = np.zeros(U, dtype=np.int64)
        seg[1:] = np.cumsum(gcap[:-1] + self.tail_cap)
        self.seg_start = seg
        self.rows_total = int(seg[-1] + gcap[-1] + self.tail_cap)
        self.n_global = np.zeros(U, dtype=np.int64)
        self.tail_head = np.zeros(U, dtype=np.int64)
        self.n_tail = np.zeros(U, dtype=np.int64)
        self.seq_len = np.zeros(U, dtype=np.int64)
        self.t_keep = np.ascontiguousarray(t_keep, dtype=np.int64)
        tdt = torch.bfloat16 if prm.dtype == TCA_BF16 else torch.float32
        self.k = torch.zeros(self.rows_total, prm.head_dim, dtype=tdt, device=device)
        self.v = torch.zeros(self.rows_total, prm.head_dim, dtype=tdt, device=device)
        self.pos = torch.full((self.rows_total,), -1, dtype=torch.int32, device=device)
        self.state = torch.zeros(U * TCA_STATE_WORDS, dtype=torch.int64, device=device)
        self.desc = tca_cache_desc(
            self.k.data_ptr(), self.v.data_ptr(), self.pos.data_ptr(), self.state.data_ptr(),
            self.rows_total, U, self.tail_cap, self.seg_start.ctypes.data, self.global_cap.ctypes.data,
            self.n_global.ctypes.data, self.tail_head.ctypes.data, self.n_tail.ctypes.data,
            self.seq_len.ctypes.data, self.t_keep.ctypes.data)
        if init:
            tca_cache_init(prm, self)

    def unit_rows(self, u: int) -> np.ndarray:
        """Physical cache rows of unit u in logical order (global rows, then tail oldest first)."""
        g = self.seg_start[u] + np.arange(self.n_global[u])
        ring = self.seg_start[u] + self.global_cap[u]
        t = ring + (self.tail_head[u] + np.arange(self.n_tail[u])) % self.tail_cap
        return np.concatenate([g, t]).astype(np.int64)


def tca_calib_colmean(prm, Q, K, L, colmean, ws, stream=None) -> None:
    _check(lib().tca_calib_colmean(C.byref(prm), _dev(Q), _dev(K), L, _dev(colmean), *_ws_args(ws), _stream(stream)),
           "tca_calib_colmean")


def tca_calib_score(prm, colmean, L, idx, offsets_dev, a_out, stream=None) -> None:
    _check(lib().tca_calib_score(C.byref(prm), _dev(colmean), L, _dev(idx), _dev(offsets_dev), _dev(a_out),
                                 _stream(stream)), "tca_calib_score")


def tca_calib_choose(a: np.ndarray, sizes: np.ndarray, tau: float) -> int:
    a = np.ascontiguousarray(a, dtype=np.float64)
    sizes = np.ascontiguousarray(sizes, dtype=np.int64)
    r = lib().tca_calib_choose(a.ctypes.data, sizes.ctypes.data, len(a), float(tau))
    if r < 0:
        raise TcaError(r, "tca_calib_choose")
    return int(r)


def tca_calib_candidates(block: int, n_candidates: int = 14, sigma: float = 1.0) -> np.ndarray:
    nK = int(block).bit_length()
    p = np.zeros((n_candidates, nK), dtype=np.float64)
    _check(lib().tca_calib_candidates(block, n_candidates, float(sigma), p.ctypes.data), "tca_calib_candidates")
    return p
