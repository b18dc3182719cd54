"""ctypes binding of libec.so: one Python function per C entry point, same names.

Only argument marshalling happens here (tensor -> device pointer, shape -> ints, the
current torch stream -> cudaStream_t). All arithmetic runs in the CUDA kernels. Tensors
must live on the current CUDA device and be contiguous. There is no CPU fallback: if the
library cannot be loaded, the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libec.so")

EC_OK, EC_ERR_NULL, EC_ERR_SHAPE, EC_ERR_ALIGN, EC_ERR_ARG = 0, 1, 2, 3, 4
EC_ERR_WORKSPACE, EC_ERR_CUDA, EC_ERR_TIMEOUT, EC_ERR_TOO_LARGE = 5, 6, 7, 8
EC_PER_HEAD = 0
EC_STAT_SUM, EC_STAT_MEAN, EC_STAT_MAX, EC_STAT_MOVING_AVERAGE = 0, 1, 2, 3
EC_LAYER_SHARED = 1

EXPORTS = (
    "ec_status_string", "ec_keep_count",
    "ec_importance_workspace", "ec_importance", "ec_importance_prefix", "ec_importance_statistic", "ec_importance_from_lse", "ec_prefill_attention", "ec_device_status", "ec_selftest_wait_timeout",
    "ec_select_merge_workspace", "ec_select_merge", "ec_select_compact_workspace", "ec_select_compact",
    "ec_cache_init", "ec_cache_init_ratio", "ec_cache_track_order", "ec_cache_concat", "ec_decode_workspace", "ec_decode_step", "ec_decode_steps",
    "ec_decode_noalloc_capacity", "ec_decode_step_noalloc", "ec_compress_host", "ec_decode_steps_host",
    "ec_probe_read_stream", "ec_probe_mixed_stream", "ec_decode_splits",
)


class EcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (ec_status {status})")


class ec_cache(C.Structure):
    """Mirror of the C struct ec_cache (host-side plain data)."""
    _fields_ = [("Kc", C.c_void_p), ("Vc", C.c_void_p),
                ("N", C.c_int), ("H", C.c_int), ("D", C.c_int), ("cap", C.c_int),
                ("len", C.c_int), ("budget", C.c_int), ("offset", C.c_int),
                ("ring_head", C.c_int), ("step", C.c_int64),
                ("policy", C.c_int), ("recent_head", C.c_int), ("keep_ratio", C.c_double),
                ("n_tot", C.c_int64), ("recent_slots_host", C.POINTER(C.c_int)),
                ("queue_slots_host", C.POINTER(C.c_int))]


_lib = None


def lib() -> C.CDLL:
    """Load libec.so (once). Raises if it has not been built: there is no fallback path."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2407_18121_b200.build` "
                          "(the CUDA library is the only implementation)")
    L = C.CDLL(LIB_PATH)
    vp, i, f, sz = C.c_void_p, C.c_int, C.c_float, C.c_size_t
    L.ec_status_string.restype = C.c_char_p
    L.ec_status_string.argtypes = [i]
    L.ec_keep_count.restype = i
    L.ec_keep_count.argtypes = [i, C.c_double]
    L.ec_importance_workspace.restype = sz
    L.ec_importance_workspace.argtypes = [i, i, i, i]
    L.ec_importance.restype = i
    L.ec_importance.argtypes = [vp, vp, vp, vp, i, i, i, i, f, vp, sz, vp]
    L.ec_importance_prefix.restype = i
    L.ec_importance_prefix.argtypes = [vp, vp, vp, vp, i, i, i, i, i, f, vp, sz, vp]
    L.ec_importance_statistic.restype = i
    L.ec_importance_statistic.argtypes = [vp, vp, vp, vp, i, i, i, i, i, f, i, C.c_double, vp, sz, vp]
    L.ec_importance_from_lse.restype = i
    L.ec_importance_from_lse.argtypes = [vp, vp, vp, vp, i, i, i, i, f, vp, sz, vp]
    L.ec_prefill_attention.restype = i
    L.ec_prefill_attention.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, f, vp, sz, vp]
    L.ec_device_status.restype = i
    L.ec_device_status.argtypes = [vp, vp]
    L.ec_selftest_wait_timeout.restype = i
    L.ec_selftest_wait_timeout.argtypes = [vp, C.c_uint, vp]
    L.ec_select_merge_workspace.restype = sz
    L.ec_select_merge_workspace.argtypes = [i, i, i, i, i, i]
    L.ec_select_merge.restype = i
    L.ec_select_merge.argtypes = [vp, vp, vp, i, i, i, i, i, i, i, vp, vp, i, vp, vp, vp, sz, vp]
    L.ec_select_compact_workspace.restype = sz
    L.ec_select_compact_workspace.argtypes = [i, i, i, i, i, i]
    L.ec_select_compact.restype = i
    L.ec_select_compact.argtypes = [vp, vp, vp, i, i, i, i, i, i, i, i, vp, vp, i, vp, vp, vp, sz, vp]
    L.ec_cache_init.restype = i
    L.ec_cache_init.argtypes = [C.POINTER(ec_cache), vp, vp, i, i, i, i, i, i, i]
    L.ec_cache_init_ratio.restype = i
    L.ec_cache_init_ratio.argtypes = [C.POINTER(ec_cache), vp, vp, i, i, i, i, i, i, C.c_double, C.c_int64,
                                      C.POINTER(C.c_int)]
    L.ec_cache_track_order.restype = i
    L.ec_cache_track_order.argtypes = [C.POINTER(ec_cache), C.POINTER(C.c_int)]
    L.ec_cache_concat.restype = i
    L.ec_cache_concat.argtypes = [C.POINTER(ec_cache), vp, vp, i, vp, vp, vp]
    L.ec_decode_workspace.restype = sz
    L.ec_decode_workspace.argtypes = [C.POINTER(ec_cache)]
    L.ec_decode_step.restype = i
    L.ec_decode_step.argtypes = [vp, vp, vp, C.POINTER(ec_cache), f, vp, C.POINTER(i), C.POINTER(i), vp, sz, vp]
    L.ec_decode_steps.restype = i
    L.ec_decode_steps.argtypes = [vp, vp, vp, i, C.POINTER(ec_cache), f, vp, C.POINTER(i), vp, sz, vp]
    L.ec_compress_host.restype = i
    L.ec_compress_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, i, i, i, i, f, i, i, i, vp, vp, i, vp, vp, vp, sz, vp, sz, vp]
    L.ec_decode_steps_host.restype = i
    L.ec_decode_steps_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i, i, C.POINTER(ec_cache), f, vp, sz, vp, vp, vp]
    L.ec_decode_noalloc_capacity.restype = sz
    L.ec_decode_noalloc_capacity.argtypes = []
    L.ec_decode_step_noalloc.restype = i
    L.ec_decode_step_noalloc.argtypes = [vp, vp, vp, C.POINTER(ec_cache), f, vp, C.POINTER(i), C.POINTER(i), vp]
    L.ec_probe_read_stream.restype = i
    L.ec_probe_read_stream.argtypes = [vp, sz, vp, vp]
    L.ec_probe_mixed_stream.restype = i
    L.ec_probe_mixed_stream.argtypes = [vp, sz, vp, i, vp, vp]
    L.ec_decode_splits.restype = i
    L.ec_decode_splits.argtypes = [C.POINTER(ec_cache)]
    _lib = L
    return L


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("device tensors are required (the library has no host path)")
    if not t.is_contiguous():
        raise ValueError("tensors must be contiguous")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, where: str) -> None:
    if status != EC_OK:
        raise EcError(status, where)


def status_string(status: int) -> str:
    return lib().ec_status_string(int(status)).decode()


def ec_keep_count(T: int, keep_ratio: float) -> int:
    return int(lib().ec_keep_count(int(T), float(keep_ratio)))


def ec_importance_workspace(N: int, H: int, T: int, D: int) -> int:
    return int(lib().ec_importance_workspace(N, H, T, D))


def ec_importance(Q: torch.Tensor, K: torch.Tensor, scores: torch.Tensor, lse: Optional[torch.Tensor],
                  scale: float, ws: torch.Tensor) -> None:
    """Q, K: bf16 [N,H,T,D]; scores (out), lse (out, optional): fp32 [N,H,T]; ws: uint8 scratch."""
    N, H, T, D = Q.shape
    st = lib().ec_importance(_ptr(Q), _ptr(K), _ptr(scores), _ptr(lse), N, H, T, D, float(scale),
                             _ptr(ws), ws.numel() * ws.element_size(), _stream())
    _check(st, "ec_importance")


def ec_importance_prefix(Q: torch.Tensor, K: torch.Tensor, scores: torch.Tensor, lse: Optional[torch.Tensor],
                         scale: float, ws: torch.Tensor) -> None:
    """Q: bf16 [N,H,Tq,D]; K: bf16 [N,H,P+Tq,D] (P earlier rows every query sees); scores (out): fp32
    [N,H,P+Tq]; lse (out, optional): fp32 [N,H,Tq]; ws sized by ec_importance_workspace(N,H,Tq,D)."""
    N, H, Tq, D = Q.shape
    P = K.shape[2] - Tq
    st = lib().ec_importance_prefix(_ptr(Q), _ptr(K), _ptr(scores), _ptr(lse), N, H, Tq, P, D, float(scale),
                                    _ptr(ws), ws.numel() * ws.element_size(), _stream())
    _check(st, "ec_importance_prefix")


def ec_importance_statistic(Q: torch.Tensor, K: torch.Tensor, scores: torch.Tensor, lse: Optional[torch.Tensor],
                            scale: float, statistic: int, beta: float, ws: torch.Tensor) -> None:
    """ec_importance_prefix with the statistic chosen: EC_STAT_SUM, EC_STAT_MEAN, EC_STAT_MAX or
    EC_STAT_MOVING_AVERAGE (factor 0 < beta < 1). Shapes as ec_importance_prefix."""
    N, H, Tq, D = Q.shape
    P = K.shape[2] - Tq
    st = lib().ec_importance_statistic(_ptr(Q), _ptr(K), _ptr(scores), _ptr(lse), N, H, Tq, P, D, float(scale),
                                       int(statistic), float(beta), _ptr(ws), ws.numel() * ws.element_size(), _stream())
    _check(st, "ec_importance_statistic")


def ec_importance_from_lse(Q: torch.Tensor, K: torch.Tensor, lse: torch.Tensor, scores: torch.Tensor,
                           scale: float, ws: torch.Tensor) -> None:
    """Importance from a known per-row log-sum-exp (fp32 [N,H,T], natural log): column-sum pass only."""
    N, H, T, D = Q.shape
    st = lib().ec_importance_from_lse(_ptr(Q), _ptr(K), _ptr(lse), _ptr(scores), N, H, T, D, float(scale),
                                      _ptr(ws), ws.numel() * ws.element_size(), _stream())
    _check(st, "ec_importance_from_lse")


def ec_prefill_attention(Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, out: torch.Tensor,
                         lse: Optional[torch.Tensor], scores: Optional[torch.Tensor], scale: float,
                         ws: torch.Tensor) -> None:
    """Causal attention of the prompt tokens. Q: bf16 [N,H,Tq,D]; K, V: bf16 [N,H,P+Tq,D]; out (out): bf16
    [N,H,Tq,D]; lse (out, optional): fp32 [N,H,Tq]; scores (out, optional): fp32 [N,H,P+Tq], the importance
    from the column-sum pass alone; ws sized by ec_importance_workspace(N,H,Tq,D)."""
    N, H, Tq, D = Q.shape
    P = K.shape[2] - Tq
    if K.shape != V.shape or tuple(out.shape) != tuple(Q.shape):
        raise ValueError("K and V must have one shape, out the shape of Q")
    st = lib().ec_prefill_attention(_ptr(Q), _ptr(K), _ptr(V), _ptr(out), _ptr(lse), _ptr(scores), N, H, Tq, P, D,
                                    float(scale), _ptr(ws), ws.numel() * ws.element_size(), _stream())
    _check(st, "ec_prefill_attention")


def ec_device_status(ws: torch.Tensor) -> int:
    return int(lib().ec_device_status(_ptr(ws), _stream()))


def ec_selftest_wait_timeout(ws: torch.Tensor, limit_us: int) -> None:
    """Enqueue the bounded-wait self-test: afterwards ec_device_status(ws) reports EC_ERR_TIMEOUT."""
    _check(lib().ec_selftest_wait_timeout(_ptr(ws), int(limit_us), _stream()), "ec_selftest_wait_timeout")


def ec_select_merge_workspace(N: int, H: int, T: int, D: int, n_keep: int, population: int) -> int:
    return int(lib().ec_select_merge_workspace(N, H, T, D, n_keep, population))


def ec_select_merge(K: torch.Tensor, V: torch.Tensor, scores: torch.Tensor, n_keep: int, population: int,
                    protect_ends: bool, Kc: torch.Tensor, Vc: torch.Tensor, anchor_pos: torch.Tensor,
                    bucket_len: Optional[torch.Tensor], ws: torch.Tensor) -> None:
    """K, V: bf16 [N,H,T,D]; scores fp32 [N,H,T]; Kc, Vc (out): bf16 [N,H,cap,D];
    anchor_pos (out), bucket_len (out, optional): int32 [N,H,n_keep]."""
    N, H, T, D = K.shape
    cap = Kc.shape[2]
    st = lib().ec_select_merge(_ptr(K), _ptr(V), _ptr(scores), N, H, T, D, int(n_keep), int(population),
                               int(bool(protect_ends)), _ptr(Kc), _ptr(Vc), cap, _ptr(anchor_pos),
                               _ptr(bucket_len), _ptr(ws), ws.numel() * ws.element_size(), _stream())
    _check(st, "ec_select_merge")


EC_COMPACT_MERGE = 0
EC_COMPACT_EVICT = 1


def ec_select_compact_workspace(N: int, H: int, T: int, D: int, n_keep: int, share: int) -> int:
    return int(lib().ec_select_compact_workspace(N, H, T, D, n_keep, share))


def ec_select_compact(K: torch.Tensor, V: torch.Tensor, scores: torch.Tensor, n_keep: int, share: int,
                      protect_ends: bool, compaction: int, Kc: torch.Tensor, Vc: torch.Tensor,
                      anchor_pos: torch.Tensor, bucket_len: Optional[torch.Tensor], ws: torch.Tensor) -> None:
    """ec_select_merge with an explicit sharing width (`share` consecutive units rank one averaged score
    vector) and a choice between bucket means (EC_COMPACT_MERGE) and plain eviction (EC_COMPACT_EVICT)."""
    N, H, T, D = K.shape
    cap = Kc.shape[2]
    st = lib().ec_select_compact(_ptr(K), _ptr(V), _ptr(scores), N, H, T, D, int(n_keep), int(share),
                                 int(bool(protect_ends)), int(compaction), _ptr(Kc), _ptr(Vc), cap,
                                 _ptr(anchor_pos), _ptr(bucket_len), _ptr(ws), ws.numel() * ws.element_size(),
                                 _stream())
    _check(st, "ec_select_compact")


def ec_cache_init(Kc: torch.Tensor, Vc: torch.Tensor, length: int, budget: int, offset: int) -> ec_cache:
    """Describe a compacted cache held in Kc, Vc: bf16 [N,H,cap,D] with `length` valid rows."""
    N, H, cap, D = Kc.shape
    c = ec_cache()
    st = lib().ec_cache_init(C.byref(c), _ptr(Kc), _ptr(Vc), N, H, D, cap, int(length), int(budget), int(offset))
    _check(st, "ec_cache_init")
    return c


def ec_cache_init_ratio(Kc: torch.Tensor, Vc: torch.Tensor, length: int, offset: int, keep_ratio: float,
                        n_tot: int, track_order: bool = True) -> ec_cache:
    """Cache under the retention-ratio policy: it grows while length < keep_ratio * tokens seen and
    evicts at the fixed truncation location otherwise. The host ring of recent slots is owned by
    the returned object, and so is the queue-order list that ec_cache_track_order maintains (needed
    by ec_cache_concat; `track_order=False` leaves it out)."""
    N, H, cap, D = Kc.shape
    c = ec_cache()
    c._recent = (C.c_int * int(offset))()          # kept alive with the struct
    st = lib().ec_cache_init_ratio(C.byref(c), _ptr(Kc), _ptr(Vc), N, H, D, cap, int(length), int(offset),
                                   float(keep_ratio), int(n_tot), c._recent)
    _check(st, "ec_cache_init_ratio")
    if track_order:
        c._order = (C.c_int * int(cap))()          # queue order of the rows, kept alive with the struct
        _check(lib().ec_cache_track_order(C.byref(c), c._order), "ec_cache_track_order")
    return c


def ec_decode_workspace(cache: ec_cache) -> int:
    return int(lib().ec_decode_workspace(C.byref(cache)))


def ec_decode_step(q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, cache: ec_cache, scale: float,
                   out: torch.Tensor, ws: torch.Tensor):
    """q, k_new, v_new: bf16 [N,H,D]; out (out): bf16 [N,H,D].
    Returns (evicted physical slot or -1, slot that now holds the new row)."""
    ev, sl = C.c_int(-1), C.c_int(-1)
    st = lib().ec_decode_step(_ptr(q), _ptr(k_new), _ptr(v_new), C.byref(cache), float(scale), _ptr(out),
                              C.byref(ev), C.byref(sl), _ptr(ws), ws.numel() * ws.element_size(), _stream())
    _check(st, "ec_decode_step")
    return ev.value, sl.value


def ec_decode_steps(q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, cache: ec_cache, scale: float,
                    out: torch.Tensor, ws: torch.Tensor, want_slots: bool = False):
    """q, k_new, v_new, out: bf16 [steps,N,H,D]. Issues all steps from native code."""
    steps = q.shape[0]
    slots = (C.c_int * steps)() if want_slots else None
    st = lib().ec_decode_steps(_ptr(q), _ptr(k_new), _ptr(v_new), steps, C.byref(cache), float(scale), _ptr(out),
                               slots, _ptr(ws), ws.numel() * ws.element_size(), _stream())
    _check(st, "ec_decode_steps")
    return list(slots) if want_slots else None


def ec_cache_concat(cache: ec_cache, K_new: torch.Tensor, V_new: torch.Tensor, K_all: torch.Tensor,
                    V_all: torch.Tensor) -> None:
    """K_all, V_all [N,H,len+Tq,D] <- the cache's rows in queue order, then K_new, V_new [N,H,Tq,D]."""
    Tq = K_new.shape[2]
    if tuple(K_all.shape) != (cache.N, cache.H, cache.len + Tq, cache.D) or K_all.shape != V_all.shape:
        raise ValueError("K_all, V_all must be [N, H, len + Tq, D]")
    if tuple(K_new.shape) != (cache.N, cache.H, Tq, cache.D) or K_new.shape != V_new.shape:
        raise ValueError("K_new, V_new must be [N, H, Tq, D]")
    st = lib().ec_cache_concat(C.byref(cache), _ptr(K_new), _ptr(V_new), Tq, _ptr(K_all), _ptr(V_all), _stream())
    _check(st, "ec_cache_concat")


def ec_decode_noalloc_capacity() -> int:
    return int(lib().ec_decode_noalloc_capacity())


def ec_decode_step_noalloc(q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, cache: ec_cache,
                           scale: float, out: torch.Tensor):
    """ec_decode_step without a workspace argument, for callers that may not allocate device
    memory: the scratch is a fixed 2 MiB array inside the library. Raises EcError with status
    EC_ERR_TOO_LARGE when the cache is too big for it. Calls that could overlap on the GPU must
    be serialised by the caller, since they share that array."""
    ev, sl = C.c_int(-1), C.c_int(-1)
    st = lib().ec_decode_step_noalloc(_ptr(q), _ptr(k_new), _ptr(v_new), C.byref(cache), float(scale), _ptr(out),
                                      C.byref(ev), C.byref(sl), _stream())
    _check(st, "ec_decode_step_noalloc")
    return ev.value, sl.value


def _host_ptr(t: torch.Tensor) -> int:
    if t.is_cuda or not t.is_contiguous():
        raise ValueError("a contiguous host tensor is required")
    return t.data_ptr()


def ec_compress_host(Q_host, K_host, V_host, Q, K, V, scores, scale: float, n_keep: int, population: int,
                     protect_ends: bool, Kc, Vc, anchor_pos, anchor_pos_host, ws_imp, ws_sel) -> None:
    """Prompt call from host tensors (bf16 [N,H,T,D], pinned for asynchronous copies): upload into the
    device staging tensors Q, K, V, importance, selection + merge, optional download of the index map."""
    N, H, T, D = Q.shape
    st = lib().ec_compress_host(_host_ptr(Q_host), _host_ptr(K_host), _host_ptr(V_host), _ptr(Q), _ptr(K), _ptr(V),
                                _ptr(scores), N, H, T, D, float(scale), int(n_keep), int(population),
                                int(bool(protect_ends)), _ptr(Kc), _ptr(Vc), Kc.shape[2], _ptr(anchor_pos),
                                None if anchor_pos_host is None else _host_ptr(anchor_pos_host),
                                _ptr(ws_imp), ws_imp.numel(), _ptr(ws_sel), ws_sel.numel(), _stream())
    _check(st, "ec_compress_host")


def ec_decode_steps_host(q_host, k_host, v_host, out_host, q, k, v, out, cache: ec_cache, scale: float, ws,
                         upload_stream: torch.cuda.Stream, download_stream: torch.cuda.Stream, chunk: int = 64) -> None:
    """Decode loop from host tensors [steps,N,H,D]: chunked uploads and downloads on two side streams overlap
    the decoding on the current stream; q, k, v, out are device staging tensors of the same shape."""
    steps = q_host.shape[0]
    st = lib().ec_decode_steps_host(_host_ptr(q_host), _host_ptr(k_host), _host_ptr(v_host), _host_ptr(out_host),
                                    _ptr(q), _ptr(k), _ptr(v), _ptr(out), steps, int(chunk), C.byref(cache),
                                    float(scale), _ptr(ws), ws.numel() * ws.element_size(), _stream(),
                                    upload_stream.cuda_stream, download_stream.cuda_stream)
    _check(st, "ec_decode_steps_host")


def ec_probe_read_stream(buf: torch.Tensor, sink: torch.Tensor) -> None:
    """Enqueue one read-only pass over `buf` (any dtype, byte size a multiple of 16); `sink`: uint32/int32 [1]."""
    _check(lib().ec_probe_read_stream(_ptr(buf), buf.numel() * buf.element_size(), _ptr(sink), _stream()),
           "ec_probe_read_stream")


def ec_probe_mixed_stream(buf: torch.Tensor, dst: torch.Tensor, write_every: int, sink: torch.Tensor) -> None:
    """ec_probe_read_stream that also writes one 256-byte row in `write_every` to `dst` (densely)."""
    need = -(-(buf.numel() * buf.element_size() // 256) // max(1, write_every)) * 256
    if write_every > 0 and dst.numel() * dst.element_size() < need:
        raise ValueError("dst is too small for this write ratio")
    _check(lib().ec_probe_mixed_stream(_ptr(buf), buf.numel() * buf.element_size(), _ptr(dst), int(write_every),
                                       _ptr(sink), _stream()), "ec_probe_mixed_stream")


def ec_decode_splits(cache: ec_cache) -> int:
    return int(lib().ec_decode_splits(C.byref(cache)))
