"""Thin ctypes binding of ``libpafu.so``: argument marshalling only.

Functions carry the C names (``pafu_score`` ...).  Device tensors are torch CUDA tensors
(bf16 for token tensors and weights, fp32 scores, int32 indices); the binding passes their
``data_ptr()`` and the current CUDA stream.  There is no CPU path: loading fails loudly when
the library has not been built, and every call raises ``PafuError`` on a non-zero status.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libpafu.so")

PAFU_MAX_STREAMS = 32
ACT_GELU, ACT_SILU = 0, 1
FINAL_NONE, FINAL_SIGMOID = 0, 1

STATUS_NAMES = {0: "PAFU_OK", 1: "PAFU_ERR_INVALID_ARG", 2: "PAFU_ERR_BAD_BUDGET",
                3: "PAFU_ERR_UNSUPPORTED_SHAPE", 4: "PAFU_ERR_WORKSPACE_TOO_SMALL",
                5: "PAFU_ERR_MISALIGNED", 6: "PAFU_ERR_CUDA", 7: "PAFU_ERR_TIMEOUT",
                8: "PAFU_ERR_TOO_LARGE"}

EXPORTS = ["pafu_version", "pafu_status_string", "pafu_kept_counts", "pafu_workspace_bytes",
           "pafu_workspace_status", "pafu_workspace_counters", "pafu_score", "pafu_score_qkv", "pafu_select", "pafu_compact",
           "pafu_chunk_attn", "pafu_chunk_attn_indexed", "pafu_chunk_attn_noalloc", "pafu_step", "pafu_step_indexed", "pafu_step_timed", "pafu_step_host_arena_bytes", "pafu_step_host", "pafu_step_host_async",
           "pafu_sse_workspace_bytes", "pafu_sse", "pafu_sse_mean_first", "pafu_compact_layers", "pafu_cache_update"]


class PafuError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = STATUS_NAMES.get(status, str(status))
        try:
            msg += " (%s)" % lib().pafu_status_string(status).decode()
        except Exception:
            pass
        super().__init__("%s failed: %s" % (where, msg))


class CShape(ctypes.Structure):
    _fields_ = [("n_heads", ctypes.c_int32), ("d_head", ctypes.c_int32),
                ("n_streams", ctypes.c_int32), ("cu_T", ctypes.c_void_p),
                ("cu_Lq", ctypes.c_void_p)]


class CHead(ctypes.Structure):
    _fields_ = [("d_in", ctypes.c_int32), ("d_hidden", ctypes.c_int32), ("d_out", ctypes.c_int32),
                ("act", ctypes.c_int32), ("final", ctypes.c_int32),
                ("w1", ctypes.c_void_p), ("b1", ctypes.c_void_p),
                ("w2", ctypes.c_void_p), ("b2", ctypes.c_void_p)]


class CPolicy(ctypes.Structure):
    _fields_ = [("n_sink", ctypes.c_int64), ("n_recent", ctypes.c_int64),
                ("budget", ctypes.c_int64)]


class CCache(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("n_heads", ctypes.c_int32), ("d_head", ctypes.c_int32),
                ("cur", ctypes.c_int32), ("capacity", ctypes.c_int64), ("n_sink", ctypes.c_int64),
                ("T", ctypes.c_int64), ("K", ctypes.c_void_p * 2), ("V", ctypes.c_void_p * 2),
                ("SL", ctypes.c_void_p * 2), ("idx", ctypes.c_void_p)]


class CStepArgs(ctypes.Structure):
    _fields_ = [("shape", CShape), ("head", ctypes.POINTER(CHead)),
                ("policy", ctypes.POINTER(CPolicy)),
                ("K", ctypes.c_void_p), ("V", ctypes.c_void_p), ("Q", ctypes.c_void_p),
                ("Kq", ctypes.c_void_p), ("Vq", ctypes.c_void_p), ("scale", ctypes.c_float),
                ("scores", ctypes.c_void_p), ("idx", ctypes.c_void_p), ("Kc", ctypes.c_void_p),
                ("Vc", ctypes.c_void_p), ("SLc", ctypes.c_void_p), ("O", ctypes.c_void_p),
                ("LSE", ctypes.c_void_p), ("ws", ctypes.c_void_p), ("ws_bytes", ctypes.c_size_t)]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libpafu.so is missing at %s - build it with "
                "`python -m paper_2601_21896_b200.build` (needs nvcc); there is no CPU path" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_size_t
        L.pafu_version.restype = i32
        L.pafu_version.argtypes = []
        L.pafu_status_string.restype = ctypes.c_char_p
        L.pafu_status_string.argtypes = [i32]
        L.pafu_kept_counts.restype = i32
        L.pafu_kept_counts.argtypes = [ctypes.POINTER(CShape), ctypes.POINTER(CPolicy), vp]
        L.pafu_workspace_bytes.restype = sz
        L.pafu_workspace_bytes.argtypes = [ctypes.POINTER(CShape), ctypes.POINTER(CPolicy),
                                           ctypes.POINTER(CHead)]
        L.pafu_workspace_status.restype = i32
        L.pafu_workspace_status.argtypes = [vp, vp]
        L.pafu_workspace_counters.restype = i32
        L.pafu_workspace_counters.argtypes = [vp, vp, vp]
        L.pafu_score.restype = i32
        L.pafu_score.argtypes = [ctypes.POINTER(CHead), vp, i64, i64, vp, vp, sz, vp]
        L.pafu_score_qkv.restype = i32
        L.pafu_score_qkv.argtypes = [ctypes.POINTER(CHead), vp, vp, vp, i64, i64, vp, vp, sz, vp]
        L.pafu_select.restype = i32
        L.pafu_select.argtypes = [vp, ctypes.POINTER(CShape), ctypes.POINTER(CPolicy), vp, vp, sz, vp]
        L.pafu_compact.restype = i32
        L.pafu_compact.argtypes = [vp, vp, vp, vp, ctypes.POINTER(CShape), ctypes.POINTER(CPolicy),
                                   vp, vp, vp, vp]
        L.pafu_chunk_attn.restype = i32
        L.pafu_chunk_attn.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.POINTER(CShape),
                                      ctypes.c_float, vp, vp, vp, sz, vp]
        L.pafu_chunk_attn_indexed.restype = i32
        L.pafu_chunk_attn_indexed.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.POINTER(CShape),
                                              ctypes.c_float, vp, vp, vp, sz, vp]
        L.pafu_step_indexed.restype = i32
        L.pafu_step_indexed.argtypes = [ctypes.POINTER(CStepArgs), vp]
        L.pafu_cache_update.restype = i32
        L.pafu_cache_update.argtypes = [ctypes.POINTER(CCache), ctypes.POINTER(CHead), vp, vp, vp, vp, vp, i64,
                                        ctypes.POINTER(i32), vp, sz, vp]
        L.pafu_compact_layers.restype = i32
        L.pafu_compact_layers.argtypes = [vp, vp, i32, vp, vp, ctypes.POINTER(CShape), ctypes.POINTER(CPolicy),
                                          vp, vp, vp, vp]
        L.pafu_sse_workspace_bytes.restype = sz
        L.pafu_sse_workspace_bytes.argtypes = [i64, i32, i32, i64]
        L.pafu_sse.restype = i32
        L.pafu_sse.argtypes = [vp, vp, vp, i64, i32, i32, i64, ctypes.c_float, vp, vp, vp, vp, vp, sz, vp]
        L.pafu_sse_mean_first.restype = i32
        L.pafu_sse_mean_first.argtypes = [vp, vp, vp, i64, i32, i32, i64, ctypes.c_float, vp, vp, vp, sz, vp]
        L.pafu_chunk_attn_noalloc.restype = i32
        L.pafu_chunk_attn_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.POINTER(CShape),
                                              ctypes.c_float, vp, vp, vp]
        L.pafu_step.restype = i32
        L.pafu_step.argtypes = [ctypes.POINTER(CStepArgs), vp]
        L.pafu_step_timed.restype = i32
        L.pafu_step_timed.argtypes = [ctypes.POINTER(CStepArgs), ctypes.POINTER(vp), vp]
        L.pafu_step_host_arena_bytes.restype = sz
        L.pafu_step_host_arena_bytes.argtypes = [ctypes.POINTER(CShape), ctypes.POINTER(CPolicy),
                                                 ctypes.POINTER(CHead)]
        L.pafu_step_host.restype = i32
        L.pafu_step_host.argtypes = [ctypes.POINTER(CStepArgs), vp, sz, vp]
        L.pafu_step_host_async.restype = i32
        L.pafu_step_host_async.argtypes = [ctypes.POINTER(CStepArgs), vp, sz, vp, vp]
        _lib = L
    return _lib


# ------------------------------------------------------------------------- marshalling
def _ptr(t) -> Optional[int]:
    """Address of a torch tensor (device or host) / numpy array, or None."""
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous(), "tensor must be contiguous"
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    raise TypeError(type(t))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, where: str) -> None:
    if status != 0:
        raise PafuError(status, where)


class Shape:
    """Host-side geometry: keeps the prefix arrays alive for the duration of a call."""

    def __init__(self, n_heads: int, d_head: int, cu_T: Optional[Sequence[int]] = None,
                 cu_Lq: Optional[Sequence[int]] = None, n_streams: Optional[int] = None):
        self.cu_T = None if cu_T is None else np.ascontiguousarray(cu_T, dtype=np.int64)
        self.cu_Lq = None if cu_Lq is None else np.ascontiguousarray(cu_Lq, dtype=np.int64)
        if n_streams is None:
            ref = self.cu_T if self.cu_T is not None else self.cu_Lq
            n_streams = len(ref) - 1
        self.n_heads, self.d_head, self.n_streams = n_heads, d_head, n_streams
        self.c = CShape(n_heads, d_head, n_streams, _ptr(self.cu_T), _ptr(self.cu_Lq))


class Head:
    """Salience head: device bf16 weights in torch.nn.Linear layout."""

    def __init__(self, w1, b1, w2, b2, act: int = ACT_GELU, final: int = FINAL_NONE,
                 dims: Optional[Sequence[int]] = None):
        self.tensors = (w1, b1, w2, b2)
        if dims is None:
            dims = (w1.shape[1], w1.shape[0], w2.shape[0])
        self.c = CHead(int(dims[0]), int(dims[1]), int(dims[2]), act, final,
                       _ptr(w1), _ptr(b1), _ptr(w2), _ptr(b2))


def make_policy(n_sink, n_recent, budget, n_streams: int):
    """ctypes array of per-stream policies; scalars are broadcast."""
    def seq(v):
        return list(v) if isinstance(v, (list, tuple, np.ndarray)) else [v] * n_streams
    arr = (CPolicy * n_streams)()
    for s, (a, b, c) in enumerate(zip(seq(n_sink), seq(n_recent), seq(budget))):
        arr[s] = CPolicy(int(a), int(b), int(c))
    return arr


# ------------------------------------------------------------------------------ entry points
def pafu_version() -> int:
    return lib().pafu_version()


def pafu_kept_counts(shape: Shape, policy) -> np.ndarray:
    cu_B = np.zeros(shape.n_streams + 1, dtype=np.int64)
    _check(lib().pafu_kept_counts(ctypes.byref(shape.c), policy, _ptr(cu_B)), "pafu_kept_counts")
    return cu_B


def pafu_workspace_bytes(shape: Shape, policy=None, head: Optional[Head] = None) -> int:
    return lib().pafu_workspace_bytes(ctypes.byref(shape.c), policy,
                                      ctypes.byref(head.c) if head is not None else None)


def pafu_workspace_status(ws: torch.Tensor) -> int:
    return lib().pafu_workspace_status(_ptr(ws), _stream())


def pafu_workspace_counters(ws: torch.Tensor) -> np.ndarray:
    """(exact passes on first/ragged tiles, exact passes forced by a row sum, rescales)."""
    out = np.zeros(3, dtype=np.int64)
    _check(lib().pafu_workspace_counters(_ptr(ws), _ptr(out), _stream()), "pafu_workspace_counters")
    return out


def pafu_score(head: Head, X: torch.Tensor, scores: torch.Tensor, ws: Optional[torch.Tensor] = None,
               n_tokens: Optional[int] = None, ldx: Optional[int] = None) -> None:
    n = X.shape[0] if n_tokens is None else n_tokens
    ld = (X.numel() // max(X.shape[0], 1)) if ldx is None else ldx
    _check(lib().pafu_score(ctypes.byref(head.c), _ptr(X), n, ld, _ptr(scores), _ptr(ws),
                            0 if ws is None else ws.numel() * ws.element_size(), _stream()),
           "pafu_score")


def pafu_score_qkv(head: Head, Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, scores: torch.Tensor,
                   ws: Optional[torch.Tensor] = None, n_tokens: Optional[int] = None,
                   ld: Optional[int] = None) -> None:
    n = K.shape[0] if n_tokens is None else n_tokens
    stride = (K.numel() // max(K.shape[0], 1)) if ld is None else ld
    _check(lib().pafu_score_qkv(ctypes.byref(head.c), _ptr(Q), _ptr(K), _ptr(V), n, stride, _ptr(scores), _ptr(ws),
                                0 if ws is None else ws.numel() * ws.element_size(), _stream()),
           "pafu_score_qkv")


def pafu_select(scores: torch.Tensor, shape: Shape, policy, idx: torch.Tensor,
                ws: Optional[torch.Tensor] = None) -> None:
    _check(lib().pafu_select(_ptr(scores), ctypes.byref(shape.c), policy, _ptr(idx), _ptr(ws),
                             0 if ws is None else ws.numel() * ws.element_size(), _stream()),
           "pafu_select")


def pafu_compact(K, V, SL, idx, shape: Shape, policy, Kc, Vc, SLc) -> None:
    _check(lib().pafu_compact(_ptr(K), _ptr(V), _ptr(SL), _ptr(idx), ctypes.byref(shape.c), policy,
                              _ptr(Kc), _ptr(Vc), _ptr(SLc), _stream()), "pafu_compact")


def pafu_compact_layers(Ks, Vs, SL, idx, shape: Shape, policy, Kcs, Vcs, SLc) -> None:
    """One index list applied to every layer's cache (lists of per-layer tensors)."""
    n = len(Ks)
    arr = lambda ts: (ctypes.c_void_p * max(n, 1))(*[_ptr(t) for t in ts])
    _check(lib().pafu_compact_layers(arr(Ks), arr(Vs), n, _ptr(SL), _ptr(idx), ctypes.byref(shape.c), policy,
                                     arr(Kcs), arr(Vcs), _ptr(SLc), _stream()), "pafu_compact_layers")


class Cache:
    """The rolling KV cache of Algorithm 2 for one stream: two sets of per-layer K / V buffers
    and salience lists of `capacity` tokens on the current CUDA device, and the host-side counters
    (`T` tokens in the cache, `cur` the buffer set that holds them)."""

    def __init__(self, n_layers: int, n_heads: int, d_head: int, capacity: int, n_sink: int, device="cuda"):
        mk = lambda: [torch.zeros((capacity, n_heads, d_head), dtype=torch.bfloat16, device=device) for _ in range(n_layers)]
        self.Kb, self.Vb = [mk(), mk()], [mk(), mk()]
        self.SLb = [torch.zeros(capacity, dtype=torch.float32, device=device) for _ in range(2)]
        self.idx = torch.zeros(capacity, dtype=torch.int32, device=device)
        arr = lambda ts: (ctypes.c_void_p * n_layers)(*[_ptr(t) for t in ts])
        self._arrs = [arr(self.Kb[0]), arr(self.Kb[1]), arr(self.Vb[0]), arr(self.Vb[1])]   # kept alive with the struct
        c = CCache()
        c.n_layers, c.n_heads, c.d_head, c.cur = n_layers, n_heads, d_head, 0
        c.capacity, c.n_sink, c.T = capacity, n_sink, 0
        for b in range(2):
            c.K[b] = ctypes.cast(self._arrs[b], ctypes.c_void_p)
            c.V[b] = ctypes.cast(self._arrs[2 + b], ctypes.c_void_p)
            c.SL[b] = _ptr(self.SLb[b])
        c.idx = _ptr(self.idx)
        self.c = c

    T = property(lambda self: int(self.c.T))
    cur = property(lambda self: int(self.c.cur))
    K = property(lambda self: [k[: self.T] for k in self.Kb[self.cur]])     # the cache as it stands, per layer
    V = property(lambda self: [v[: self.T] for v in self.Vb[self.cur]])
    SL = property(lambda self: self.SLb[self.cur][: self.T])


def pafu_cache_update(cache: Cache, head: "Head", Qs, Ks, Vs, Knew, Vnew, ws: torch.Tensor) -> bool:
    """Algorithm 2's update for one generated chunk; returns True if the cache was pruned first."""
    n = len(Knew)
    arr = lambda ts: (ctypes.c_void_p * max(n, 1))(*[_ptr(t) for t in ts])
    pruned = ctypes.c_int32(0)
    _check(lib().pafu_cache_update(ctypes.byref(cache.c), ctypes.byref(head.c), _ptr(Qs), _ptr(Ks), _ptr(Vs),
                                   arr(Knew), arr(Vnew), int(Knew[0].shape[0]) if n else 0, ctypes.byref(pruned),
                                   _ptr(ws), ws.numel() * ws.element_size(), _stream()), "pafu_cache_update")
    return bool(pruned.value)


def pafu_chunk_attn(Q, Kc, Vc, cu_B, Kq, Vq, shape: Shape, scale: float, O, LSE=None,
                    ws: Optional[torch.Tensor] = None) -> None:
    cu_B = np.ascontiguousarray(cu_B, dtype=np.int64)
    _check(lib().pafu_chunk_attn(_ptr(Q), _ptr(Kc), _ptr(Vc), _ptr(cu_B), _ptr(Kq), _ptr(Vq),
                                 ctypes.byref(shape.c), float(scale), _ptr(O), _ptr(LSE), _ptr(ws),
                                 0 if ws is None else ws.numel() * ws.element_size(), _stream()),
           "pafu_chunk_attn")


def pafu_chunk_attn_indexed(Q, K, V, idx, cu_B, Kq, Vq, shape: Shape, scale: float, O, LSE=None,
                            ws: Optional[torch.Tensor] = None) -> None:
    """Chunk attention over rows idx[.] of the uncompacted cache K, V (no compacted copy)."""
    cu_B = np.ascontiguousarray(cu_B, dtype=np.int64)
    _check(lib().pafu_chunk_attn_indexed(_ptr(Q), _ptr(K), _ptr(V), _ptr(idx), _ptr(cu_B), _ptr(Kq), _ptr(Vq),
                                         ctypes.byref(shape.c), float(scale), _ptr(O), _ptr(LSE), _ptr(ws),
                                         0 if ws is None else ws.numel() * ws.element_size(), _stream()),
           "pafu_chunk_attn_indexed")


def pafu_chunk_attn_noalloc(Q, Kc, Vc, cu_B, Kq, Vq, shape: Shape, scale: float, O, LSE=None) -> None:
    """Chunk attention that takes no workspace: its scratch is a fixed array inside the library
    (see include/pafu.h for the size limit and the rule that calls must not overlap)."""
    cu_B = np.ascontiguousarray(cu_B, dtype=np.int64)
    _check(lib().pafu_chunk_attn_noalloc(_ptr(Q), _ptr(Kc), _ptr(Vc), _ptr(cu_B), _ptr(Kq), _ptr(Vq),
                                         ctypes.byref(shape.c), float(scale), _ptr(O), _ptr(LSE),
                                         _stream()), "pafu_chunk_attn_noalloc")


def step_args(shape: Shape, head: Head, policy, K, V, Q, Kq, Vq, scale, scores, idx, Kc, Vc, SLc,
              O, LSE, ws) -> CStepArgs:
    args = CStepArgs(shape.c, ctypes.pointer(head.c), ctypes.cast(policy, ctypes.POINTER(CPolicy)),
                     _ptr(K), _ptr(V), _ptr(Q), _ptr(Kq), _ptr(Vq), float(scale), _ptr(scores),
                     _ptr(idx), _ptr(Kc), _ptr(Vc), _ptr(SLc), _ptr(O), _ptr(LSE), _ptr(ws),
                     0 if ws is None else ws.numel() * ws.element_size())
    args._keep = (shape, head, policy)   # the struct only holds raw pointers into these
    return args


def pafu_step(args: CStepArgs) -> None:
    _check(lib().pafu_step(ctypes.byref(args), _stream()), "pafu_step")


def pafu_sse_workspace_bytes(L: int, n_heads: int, d_head: int, block_len: int) -> int:
    return lib().pafu_sse_workspace_bytes(L, n_heads, d_head, block_len)


def pafu_sse(Q, K, LSE, block_len: int, scale: float, s, comp, ws, gmax=None, gavg=None) -> None:
    """Teacher salience target (Eq. 4, Eq. 5) of Q, K [L, N, D]; LSE [N, L] or None; gmax [L]
    (global max pooling) and gavg [L] (global average pooling) or None."""
    L, N, D = Q.shape
    _check(lib().pafu_sse(_ptr(Q), _ptr(K), _ptr(LSE), L, N, D, block_len, float(scale), _ptr(s), _ptr(comp),
                          _ptr(gmax), _ptr(gavg), _ptr(ws), ws.numel() * ws.element_size(), _stream()), "pafu_sse")


def pafu_sse_mean_first(Q, K, LSE, block_len: int, scale: float, s, comp, ws) -> None:
    """The salience target with the mean over heads taken before the maximum over queries
    (Algorithm 3's order); arguments as pafu_sse."""
    L, N, D = Q.shape
    _check(lib().pafu_sse_mean_first(_ptr(Q), _ptr(K), _ptr(LSE), L, N, D, block_len, float(scale), _ptr(s), _ptr(comp),
                                     _ptr(ws), ws.numel() * ws.element_size(), _stream()), "pafu_sse_mean_first")


def pafu_step_indexed(args: CStepArgs) -> None:
    _check(lib().pafu_step_indexed(ctypes.byref(args), _stream()), "pafu_step_indexed")


def event_handles(events: Sequence["torch.cuda.Event"]):
    """ctypes array of the cudaEvent_t handles of five torch timing events (each must have
    been recorded once so that torch has created it)."""
    arr = (ctypes.c_void_p * 5)()
    for i, e in enumerate(events):
        arr[i] = e.cuda_event
    return arr


def pafu_step_timed(args: CStepArgs, handles) -> None:
    _check(lib().pafu_step_timed(ctypes.byref(args), handles, _stream()), "pafu_step_timed")


def pafu_step_host_arena_bytes(shape: Shape, policy, head: Head) -> int:
    return lib().pafu_step_host_arena_bytes(ctypes.byref(shape.c), policy, ctypes.byref(head.c))


def pafu_step_host(args: CStepArgs, arena: torch.Tensor) -> None:
    _check(lib().pafu_step_host(ctypes.byref(args), _ptr(arena),
                                arena.numel() * arena.element_size(), _stream()), "pafu_step_host")


def pafu_step_host_async(args: CStepArgs, arena: torch.Tensor, timeout_word: torch.Tensor, stream=None) -> None:
    """pafu_step_host without the final synchronisation; timeout_word is a pinned int32 tensor of
    one element, valid (like the host outputs) after the stream has been synchronised."""
    st = _stream() if stream is None else stream.cuda_stream
    _check(lib().pafu_step_host_async(ctypes.byref(args), _ptr(arena), arena.numel() * arena.element_size(), st,
                                      _ptr(timeout_word)), "pafu_step_host_async")
