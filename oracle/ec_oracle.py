"""numpy front end of the C oracle (test infrastructure only).

Every function here only marshals arrays into ``libec_oracle.so``; the arithmetic is in
``ec_oracle.c``. Nothing in this package imports or calls the CUDA library.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional, Tuple

import numpy as np

from .build import build as _build

_lib = C.CDLL(_build())

_u16p = C.POINTER(C.c_uint16)
_f64p = C.POINTER(C.c_double)
_i32p = C.POINTER(C.c_int32)
_i64p = C.POINTER(C.c_int64)


def _p(a: np.ndarray, t):
    return a.ctypes.data_as(t)


_lib.eco_keep_count.restype = C.c_int
_lib.eco_keep_count.argtypes = [C.c_int, C.c_double]
_lib.eco_importance.restype = None
_lib.eco_importance.argtypes = [_u16p, _u16p, C.c_int, C.c_int, C.c_int, C.c_double, _f64p, _f64p]
_lib.eco_importance_statistic.restype = C.c_int
_lib.eco_importance_statistic.argtypes = [_u16p, _u16p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double, C.c_int,
                                          C.c_double, _f64p]
_lib.eco_importance_prefix.restype = None
_lib.eco_importance_prefix.argtypes = [_u16p, _u16p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double, _f64p, _f64p]
_lib.eco_attention_prefix.restype = None
_lib.eco_attention_prefix.argtypes = [_u16p, _u16p, _u16p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double, _f64p, _f64p]
_lib.eco_layer_mean.restype = None
_lib.eco_layer_mean.argtypes = [_f64p, C.c_int, C.c_int, C.c_int, _f64p]
_lib.eco_group_mean.restype = None
_lib.eco_group_mean.argtypes = [_f64p, C.c_int, C.c_int, C.c_int, _f64p]
_lib.eco_gather.restype = None
_lib.eco_gather.argtypes = [_u16p, C.c_int, C.c_int, C.c_int, _i32p, C.c_int, _f64p]
_lib.eco_select.restype = None
_lib.eco_select.argtypes = [_f64p, C.c_int, C.c_int, C.c_int, C.c_int, _i32p]
_lib.eco_buckets.restype = None
_lib.eco_buckets.argtypes = [_i32p, C.c_int, C.c_int, C.c_int, _i32p, _i32p]
_lib.eco_merge.restype = None
_lib.eco_merge.argtypes = [_u16p, C.c_int, C.c_int, C.c_int, _i32p, _i32p, C.c_int, _f64p]
_lib.eco_round_bf16.restype = None
_lib.eco_round_bf16.argtypes = [_f64p, C.c_int64, _u16p]
_lib.eco_widen_bf16.restype = None
_lib.eco_widen_bf16.argtypes = [_u16p, C.c_int64, _f64p]
_lib.eco_decode_step.restype = C.c_int
_lib.eco_decode_step.argtypes = [_f64p, _f64p, _i64p, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int),
                                 _u16p, _u16p, _u16p, C.c_double, C.c_int64, C.c_int, C.c_int,
                                 C.c_int, C.c_double, C.c_int64, _f64p, _i64p]
_lib.eco_num_threads.restype = C.c_int

POLICY_FIXED = 0
POLICY_RATIO = 1


def num_threads() -> int:
    return int(_lib.eco_num_threads())


def keep_count(T: int, ratio: float) -> int:
    return int(_lib.eco_keep_count(int(T), float(ratio)))


def _bits(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("bf16 tensors are passed as uint16 bit patterns")
    return a


def importance(Q: np.ndarray, K: np.ndarray, scale: float) -> Tuple[np.ndarray, np.ndarray]:
    """Q, K: uint16 [..., T, D]. Returns (scores, lse), float64 [..., T]."""
    Q, K = _bits(Q), _bits(K)
    assert Q.shape == K.shape
    T, D = Q.shape[-2:]
    U = int(np.prod(Q.shape[:-2], dtype=np.int64))
    scores = np.empty(Q.shape[:-1], np.float64)
    lse = np.empty(Q.shape[:-1], np.float64)
    _lib.eco_importance(_p(Q, _u16p), _p(K, _u16p), U, T, D, float(scale), _p(scores, _f64p), _p(lse, _f64p))
    return scores, lse


def importance_prefix(Q: np.ndarray, K: np.ndarray, scale: float) -> Tuple[np.ndarray, np.ndarray]:
    """Q uint16 [..., Tq, D], K uint16 [..., P+Tq, D] (P >= 0 earlier keys every query sees).
    Returns (scores [..., P+Tq], lse [..., Tq]) in float64."""
    Q, K = _bits(Q), _bits(K)
    assert Q.shape[:-2] == K.shape[:-2] and Q.shape[-1] == K.shape[-1] and K.shape[-2] >= Q.shape[-2]
    Tq, D = Q.shape[-2:]
    P = K.shape[-2] - Tq
    U = int(np.prod(Q.shape[:-2], dtype=np.int64))
    scores = np.empty(K.shape[:-1], np.float64)
    lse = np.empty(Q.shape[:-1], np.float64)
    _lib.eco_importance_prefix(_p(Q, _u16p), _p(K, _u16p), U, Tq, P, D, float(scale), _p(scores, _f64p), _p(lse, _f64p))
    return scores, lse


def attention_prefix(Q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float) -> Tuple[np.ndarray, np.ndarray]:
    """Causal attention output of the prompt tokens (the forward pass Algorithm 1 takes its attention
    from). Q uint16 [..., Tq, D]; K, V uint16 [..., P+Tq, D]. Returns (out [..., Tq, D], lse [..., Tq])."""
    Q, K, V = _bits(Q), _bits(K), _bits(V)
    assert Q.shape[:-2] == K.shape[:-2] and Q.shape[-1] == K.shape[-1] and K.shape == V.shape
    assert K.shape[-2] >= Q.shape[-2]
    Tq, D = Q.shape[-2:]
    P = K.shape[-2] - Tq
    U = int(np.prod(Q.shape[:-2], dtype=np.int64))
    out = np.empty(Q.shape, np.float64)
    lse = np.empty(Q.shape[:-1], np.float64)
    _lib.eco_attention_prefix(_p(Q, _u16p), _p(K, _u16p), _p(V, _u16p), U, Tq, P, D, float(scale),
                              _p(out, _f64p), _p(lse, _f64p))
    return out, lse


STAT_SUM, STAT_MEAN, STAT_MAX, STAT_MOVING_AVERAGE = 0, 1, 2, 3


def importance_statistic(Q: np.ndarray, K: np.ndarray, scale: float, stat: int, beta: float = 0.0) -> np.ndarray:
    """Sum, mean, maximum or moving average (factor beta) of the attention each key receives
    (Sec. 3.2 "Importance Metrics"). Q uint16 [..., Tq, D], K uint16 [..., P+Tq, D].
    Returns scores [..., P+Tq] in float64."""
    Q, K = _bits(Q), _bits(K)
    assert Q.shape[:-2] == K.shape[:-2] and Q.shape[-1] == K.shape[-1] and K.shape[-2] >= Q.shape[-2]
    Tq, D = Q.shape[-2:]
    P = K.shape[-2] - Tq
    U = int(np.prod(Q.shape[:-2], dtype=np.int64))
    scores = np.empty(K.shape[:-1], np.float64)
    rc = _lib.eco_importance_statistic(_p(Q, _u16p), _p(K, _u16p), U, Tq, P, D, float(scale), int(stat), float(beta),
                                       _p(scores, _f64p))
    if rc != 0:
        raise ValueError("unknown statistic")
    return scores


def layer_mean(scores: np.ndarray) -> np.ndarray:
    """scores float64 [N, H, T] -> [N, T]."""
    s = np.ascontiguousarray(scores, np.float64)
    N, H, T = s.shape
    out = np.empty((N, T), np.float64)
    _lib.eco_layer_mean(_p(s, _f64p), N, H, T, _p(out, _f64p))
    return out


def group_mean(scores: np.ndarray, share: int) -> np.ndarray:
    """scores float64 [U, T] with U a multiple of share -> [U // share, T]."""
    s = np.ascontiguousarray(scores, np.float64)
    U, T = s.shape
    assert U % share == 0
    out = np.empty((U // share, T), np.float64)
    _lib.eco_group_mean(_p(s, _f64p), U // share, int(share), T, _p(out, _f64p))
    return out


def gather(X: np.ndarray, anchors: np.ndarray) -> np.ndarray:
    """X uint16 [..., T, D]; anchors int32 [..., C] -> float64 [..., C, D] (the anchors' own rows)."""
    X = _bits(X)
    a = np.ascontiguousarray(anchors, np.int32)
    T, D = X.shape[-2:]
    Ck = a.shape[-1]
    U = int(np.prod(X.shape[:-2], dtype=np.int64))
    out = np.empty(X.shape[:-2] + (Ck, D), np.float64)
    _lib.eco_gather(_p(X, _u16p), U, T, D, _p(a, _i32p), Ck, _p(out, _f64p))
    return out


def select(scores: np.ndarray, C_keep: int, protect_ends: bool) -> np.ndarray:
    """scores float64 [..., T] -> anchors int32 [..., C_keep], ascending."""
    s = np.ascontiguousarray(scores, np.float64)
    T = s.shape[-1]
    U = int(np.prod(s.shape[:-1], dtype=np.int64))
    out = np.empty(s.shape[:-1] + (C_keep,), np.int32)
    _lib.eco_select(_p(s, _f64p), U, T, int(C_keep), int(bool(protect_ends)), _p(out, _i32p))
    return out


def buckets(anchors: np.ndarray, T: int) -> Tuple[np.ndarray, np.ndarray]:
    """anchors int32 [..., C] -> (lo, hi), inclusive bucket bounds."""
    a = np.ascontiguousarray(anchors, np.int32)
    Ck = a.shape[-1]
    U = int(np.prod(a.shape[:-1], dtype=np.int64))
    lo = np.empty_like(a)
    hi = np.empty_like(a)
    _lib.eco_buckets(_p(a, _i32p), U, int(T), Ck, _p(lo, _i32p), _p(hi, _i32p))
    return lo, hi


def merge(X: np.ndarray, lo: np.ndarray, hi: np.ndarray) -> np.ndarray:
    """X uint16 [..., T, D]; lo, hi int32 [..., C] -> float64 [..., C, D]."""
    X = _bits(X)
    lo = np.ascontiguousarray(lo, np.int32)
    hi = np.ascontiguousarray(hi, np.int32)
    T, D = X.shape[-2:]
    Ck = lo.shape[-1]
    U = int(np.prod(X.shape[:-2], dtype=np.int64))
    assert lo.shape == X.shape[:-2] + (Ck,) and hi.shape == lo.shape
    out = np.empty(X.shape[:-2] + (Ck, D), np.float64)
    _lib.eco_merge(_p(X, _u16p), U, T, D, _p(lo, _i32p), _p(hi, _i32p), Ck, _p(out, _f64p))
    return out


def round_bf16(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, np.float64)
    out = np.empty(x.shape, np.uint16)
    _lib.eco_round_bf16(_p(x, _f64p), x.size, _p(out, _u16p))
    return out


def widen_bf16(b: np.ndarray) -> np.ndarray:
    b = _bits(b)
    out = np.empty(b.shape, np.float64)
    _lib.eco_widen_bf16(_p(b, _u16p), b.size, _p(out, _f64p))
    return out


class DecodeQueue:
    """The cache as the paper's queue: rows in order, delete-by-position, fp64 contents.

    K0, V0: float64 [..., len, D] initial rows (identities 0..len-1). ``cap`` rows are
    reserved so appended rows fit. ``n_seen``: tokens processed so far (the prompt length
    right after the prompt call); the retention-ratio policy reads it, every step adds one.
    """

    def __init__(self, K0: np.ndarray, V0: np.ndarray, cap: Optional[int] = None, n_seen: int = 0):
        K0 = np.ascontiguousarray(K0, np.float64)
        V0 = np.ascontiguousarray(V0, np.float64)
        assert K0.shape == V0.shape
        self.lead = K0.shape[:-2]
        self.len, self.D = K0.shape[-2:]
        self.U = int(np.prod(self.lead, dtype=np.int64))
        self.cap = int(cap) if cap is not None else self.len + 1
        assert self.cap >= self.len + 1
        self.K = np.zeros((self.U, self.cap, self.D), np.float64)
        self.V = np.zeros((self.U, self.cap, self.D), np.float64)
        self.K[:, :self.len] = K0.reshape(self.U, self.len, self.D)
        self.V[:, :self.len] = V0.reshape(self.U, self.len, self.D)
        self.ids = np.full(self.cap, -1, np.int64)
        self.ids[:self.len] = np.arange(self.len)
        self.next_id = self.len
        self.n_seen = int(n_seen)

    def step(self, q, k_new, v_new, scale: float, *, policy: int, budget: int = 0, offset: int,
             ratio: float = 0.0):
        """One generation step. Returns (out float64 [..., D], evicted queue position or -1,
        evicted identity or -1)."""
        q, k_new, v_new = _bits(q), _bits(k_new), _bits(v_new)
        out = np.empty((self.U, self.D), np.float64)
        ln = C.c_int(self.len)
        ev = np.zeros(1, np.int64)
        rc = _lib.eco_decode_step(_p(self.K, _f64p), _p(self.V, _f64p), _p(self.ids, _i64p), self.U,
                                  self.cap, self.D, C.byref(ln), _p(q, _u16p), _p(k_new, _u16p),
                                  _p(v_new, _u16p), float(scale), self.next_id, int(policy),
                                  int(budget), int(offset), float(ratio), self.n_seen,
                                  _p(out, _f64p), _p(ev, _i64p))
        if rc == -2:
            raise RuntimeError("decode queue capacity exceeded")
        self.next_id += 1
        self.n_seen += 1
        self.len = ln.value
        return out.reshape(self.lead + (self.D,)), rc, int(ev[0])

    def identities(self) -> np.ndarray:
        return self.ids[:self.len].copy()
