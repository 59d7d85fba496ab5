"""ctypes front end of the C oracle (``pafu_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Each function takes numpy arrays (bf16 tensors as ``uint16`` bit patterns) and returns
numpy arrays; the arithmetic itself is in the C file, in fp64.  ``build()`` compiles the
C file with gcc into ``libpafu_oracle.so`` beside it when it is missing or stale.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pafu_oracle.c")
_LIB = os.path.join(_HERE, "libpafu_oracle.so")
_lib = None

_c_u16p = ctypes.POINTER(ctypes.c_uint16)
_c_f32p = ctypes.POINTER(ctypes.c_float)
_c_f64p = ctypes.POINTER(ctypes.c_double)
_c_i32p = ctypes.POINTER(ctypes.c_int32)
_c_i64p = ctypes.POINTER(ctypes.c_int64)
_c_u8p = ctypes.POINTER(ctypes.c_uint8)


def build(force: bool = False) -> str:
    """Compile the oracle (gcc -O2 -fopenmp); returns the library path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.pafu_oracle_score.restype = None
        lib.pafu_oracle_score.argtypes = [_c_u16p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int32,
                                          ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                          ctypes.c_int32, _c_u16p, _c_u16p, _c_u16p, _c_u16p,
                                          _c_f32p]
        lib.pafu_oracle_select.restype = ctypes.c_int64
        lib.pafu_oracle_select.argtypes = [_c_f32p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                           ctypes.c_int64, _c_i32p]
        lib.pafu_oracle_gather_rows.restype = None
        lib.pafu_oracle_gather_rows.argtypes = [_c_u8p, _c_i32p, ctypes.c_int64, ctypes.c_int64,
                                                _c_u8p]
        lib.pafu_oracle_attn.restype = None
        lib.pafu_oracle_attn.argtypes = [_c_u16p, ctypes.c_int64, _c_u16p, _c_u16p, ctypes.c_int64,
                                         _c_u16p, _c_u16p, ctypes.c_int64, ctypes.c_int32,
                                         ctypes.c_int32, ctypes.c_double, _c_i64p, ctypes.c_int64,
                                         _c_f64p, _c_f64p]
        lib.pafu_oracle_sse.restype = None
        lib.pafu_oracle_sse.argtypes = [_c_u16p, _c_u16p, ctypes.c_int64, ctypes.c_int32,
                                        ctypes.c_int32, ctypes.c_int64, ctypes.c_double, _c_f64p,
                                        _c_f64p]
        lib.pafu_oracle_sse_meanfirst.restype = None
        lib.pafu_oracle_sse_meanfirst.argtypes = lib.pafu_oracle_sse.argtypes
        lib.pafu_oracle_sse_gmax.restype = None
        lib.pafu_oracle_sse_gmax.argtypes = [_c_u16p, _c_u16p, ctypes.c_int64, ctypes.c_int32,
                                             ctypes.c_int32, ctypes.c_double, _c_f64p, _c_f64p]
        lib.pafu_oracle_sse_cols.restype = None
        lib.pafu_oracle_sse_cols.argtypes = [_c_u16p, _c_u16p, ctypes.c_int64, ctypes.c_int32,
                                             ctypes.c_int32, ctypes.c_int64, ctypes.c_double, _c_i64p,
                                             ctypes.c_int64, _c_f64p, _c_f64p]
        _lib = lib
    return _lib


def n_threads() -> int:
    """Threads the OpenMP loops will use (OMP_NUM_THREADS or the visible cores)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def _u16(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _p(a: Optional[np.ndarray], ty):
    if a is None:
        return ctypes.cast(None, ty)
    return a.ctypes.data_as(ty)


def score(X: np.ndarray, w1: np.ndarray, b1: Optional[np.ndarray], w2: np.ndarray,
          b2: Optional[np.ndarray], act: int = 0, final: int = 0) -> np.ndarray:
    """Salience head on every row of X [n_tokens, d_in] (bf16 bits) -> fp32 [n_tokens]."""
    X = _u16(X).reshape(X.shape[0], -1)
    w1 = _u16(w1); w2 = _u16(w2)
    d_hidden, d_in = w1.shape
    d_out = w2.shape[0]
    assert X.shape[1] == d_in and w2.shape[1] == d_hidden
    b1 = None if b1 is None else _u16(b1)
    b2 = None if b2 is None else _u16(b2)
    out = np.empty(X.shape[0], dtype=np.float32)
    _load().pafu_oracle_score(_p(X, _c_u16p), X.shape[0], d_in, d_in, d_hidden, d_out, act, final,
                              _p(w1, _c_u16p), _p(b1, _c_u16p), _p(w2, _c_u16p), _p(b2, _c_u16p),
                              _p(out, _c_f32p))
    return out


def select(scores: np.ndarray, n_sink: int, n_recent: int, budget: int) -> np.ndarray:
    """Indices (ascending, int32) of the retained tokens of one stream."""
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    T = scores.shape[0]
    idx = np.empty(max(T, 1), dtype=np.int32)
    n = _load().pafu_oracle_select(_p(scores, _c_f32p), T, n_sink, n_recent, budget,
                                   _p(idx, _c_i32p))
    if n < 0:
        raise ValueError("negative argument")
    return idx[:n].copy()


def compact(x: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """out[i] = x[idx[i]] along the first axis, as raw byte copies."""
    x = np.ascontiguousarray(x)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    row_bytes = x.dtype.itemsize * int(np.prod(x.shape[1:], dtype=np.int64))
    out = np.empty((idx.shape[0],) + x.shape[1:], dtype=x.dtype)
    _load().pafu_oracle_gather_rows(x.view(np.uint8).ctypes.data_as(_c_u8p), _p(idx, _c_i32p),
                                    idx.shape[0], row_bytes,
                                    out.view(np.uint8).ctypes.data_as(_c_u8p))
    return out


def cache_update(K, V, SL: np.ndarray, newK, newV, s_new: np.ndarray, capacity: int, n_sink: int):
    """One chunk of the rolling-cache update of Algorithm 2, for every layer at once.

    ``K``, ``V``: lists (one entry per layer) of arrays ``[T, ...]``; ``SL``: the salience list
    ``[T]`` carried with the cache; ``newK``, ``newV``: the chunk's rows per layer ``[C, ...]``;
    ``s_new``: the chunk's salience scores ``[C]``.  When the chunk no longer fits
    (``T + C > capacity``) the cache is first pruned to ``capacity - C`` tokens: the sink prefix
    and the highest entries of ``SL`` (ties to the lower index), ONE index list applied to
    every layer's K and V and to ``SL`` itself; then the chunk and its scores are appended.
    Returns ``(K, V, SL, ids)`` with ``ids`` the index list of the pruning, or None."""
    SL = np.ascontiguousarray(SL, dtype=np.float32)
    s_new = np.ascontiguousarray(s_new, dtype=np.float32)
    T, C = SL.shape[0], s_new.shape[0]
    if C > capacity:
        raise ValueError("chunk longer than the cache")
    ids = None
    if T + C > capacity:
        ids = select(SL, n_sink, 0, capacity - C)
        K = [compact(k, ids) for k in K]
        V = [compact(v, ids) for v in V]
        SL = compact(SL, ids)
    K = [np.concatenate([k, np.ascontiguousarray(n)]) for k, n in zip(K, newK)]
    V = [np.concatenate([v, np.ascontiguousarray(n)]) for v, n in zip(V, newV)]
    SL = np.concatenate([SL, s_new])
    return K, V, SL, ids


def attention(Q: np.ndarray, Kc: np.ndarray, Vc: np.ndarray, Kq: Optional[np.ndarray],
              Vq: Optional[np.ndarray], scale: Optional[float] = None,
              rows: Optional[Sequence[int]] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Softmax attention of one stream's queries Q [Lq, N, D] over the keys Kc [B, N, D]
    followed by Kq [Lkq, N, D].  Returns (O [n_rows, N, D] fp64, LSE [N, n_rows] fp64)."""
    Q = _u16(Q)
    Lq, N, D = Q.shape
    Kc = _u16(Kc).reshape(-1, N, D); Vc = _u16(Vc).reshape(-1, N, D)
    B = Kc.shape[0]
    if Kq is None:
        Kq = np.zeros((0, N, D), np.uint16); Vq = np.zeros((0, N, D), np.uint16)
    Kq = _u16(Kq).reshape(-1, N, D); Vq = _u16(Vq).reshape(-1, N, D)
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n_rows = Lq if r is None else r.shape[0]
    O = np.empty((n_rows, N, D), dtype=np.float64)
    LSE = np.empty((N, n_rows), dtype=np.float64)
    _load().pafu_oracle_attn(_p(Q, _c_u16p), Lq, _p(Kc, _c_u16p), _p(Vc, _c_u16p), B,
                             _p(Kq, _c_u16p), _p(Vq, _c_u16p), Kq.shape[0], N, D, float(scale),
                             _p(r, _c_i64p), n_rows, _p(O, _c_f64p), _p(LSE, _c_f64p))
    return O, LSE


def sse(Q: np.ndarray, K: np.ndarray, block_len: int, scale: Optional[float] = None
        ) -> Tuple[np.ndarray, np.ndarray]:
    """Teacher salience target s [L] (Eq. 5) and its components [3, L] = low, diag, up (Eq. 4)."""
    Q = _u16(Q); K = _u16(K)
    L, N, D = Q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    s = np.empty(L, dtype=np.float64)
    comp = np.empty((3, L), dtype=np.float64)
    _load().pafu_oracle_sse(_p(Q, _c_u16p), _p(K, _c_u16p), L, N, D, block_len, float(scale),
                            _p(s, _c_f64p), _p(comp, _c_f64p))
    return s, comp


def sse_mean_first(Q: np.ndarray, K: np.ndarray, block_len: int, scale: Optional[float] = None
                   ) -> Tuple[np.ndarray, np.ndarray]:
    """The salience target in Algorithm 3's order (mean over heads, then the maximum over the
    queries of each block class): s [L] and components [3, L] = low, diag, up."""
    Q = _u16(Q); K = _u16(K)
    L, N, D = Q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    s = np.empty(L, dtype=np.float64)
    comp = np.empty((3, L), dtype=np.float64)
    _load().pafu_oracle_sse_meanfirst(_p(Q, _c_u16p), _p(K, _c_u16p), L, N, D, block_len, float(scale),
                                      _p(s, _c_f64p), _p(comp, _c_f64p))
    return s, comp


def sse_cols(Q: np.ndarray, K: np.ndarray, block_len: int, cols: Sequence[int],
             scale: Optional[float] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 4 / Eq. 5 for the listed key positions only (no L x L matrix is held): returns
    (s [n_cols], comp [3, n_cols])."""
    Q = _u16(Q); K = _u16(K)
    L, N, D = Q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    c = np.ascontiguousarray(cols, dtype=np.int64)
    s = np.empty(c.shape[0], dtype=np.float64)
    comp = np.empty((3, c.shape[0]), dtype=np.float64)
    _load().pafu_oracle_sse_cols(_p(Q, _c_u16p), _p(K, _c_u16p), L, N, D, block_len, float(scale),
                                 _p(c, _c_i64p), c.shape[0], _p(s, _c_f64p), _p(comp, _c_f64p))
    return s, comp


def sse_global_max(Q: np.ndarray, K: np.ndarray, scale: Optional[float] = None) -> np.ndarray:
    """Global max pooling of the attention weights (the "Max" ablation, Sec. 4.3): [L]."""
    Q = _u16(Q); K = _u16(K)
    L, N, D = Q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    g = np.empty(L, dtype=np.float64)
    _load().pafu_oracle_sse_gmax(_p(Q, _c_u16p), _p(K, _c_u16p), L, N, D, float(scale), _p(g, _c_f64p),
                                 _p(None, _c_f64p))
    return g


def sse_global_avg(Q: np.ndarray, K: np.ndarray, scale: Optional[float] = None) -> np.ndarray:
    """Global average pooling of the attention weights (the "Avg" ablation, Sec. 4.3): [L]."""
    Q = _u16(Q); K = _u16(K)
    L, N, D = Q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    g = np.empty(L, dtype=np.float64); a = np.empty(L, dtype=np.float64)
    _load().pafu_oracle_sse_gmax(_p(Q, _c_u16p), _p(K, _c_u16p), L, N, D, float(scale), _p(g, _c_f64p),
                                 _p(a, _c_f64p))
    return a
