"""ctypes binding of libprefixkv.so: same entry-point names as include/prefixkv.h.

Argument marshalling only.  Tensors are torch CUDA tensors (torch is used for
device memory and streams); every step of the path runs in the library's
kernels.  There is no CPU fallback: a missing library raises at import.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

from . import build as _build

(PKV_OK, PKV_ERR_INVALID_ARG, PKV_ERR_UNSUPPORTED, PKV_ERR_WORKSPACE, PKV_ERR_CUDA,
 PKV_ERR_STATIC_LIMIT) = range(6)
(DEV_OK, DEV_BAD_SCORE, DEV_RANGE, DEV_BUDGET_TOO_SMALL, DEV_BAD_LENGTH, DEV_CAPACITY,
 DEV_TIMEOUT) = range(7)
WS_SCORE, WS_SEARCH, WS_COMPACT, WS_DECODE = range(4)
MERGE_POSITION, MERGE_FEATURE = 1, 2
F32, BF16 = 0, 1

EXPORTS = ["prefixkv_workspace_bytes", "prefixkv_last_cuda_error", "prefixkv_score",
           "prefixkv_search", "prefixkv_apply_lengths", "prefixkv_compact",
           "prefixkv_decode_attn", "prefixkv_gini", "prefixkv_rescale",
           "prefixkv_estimate_config", "prefixkv_decode_attn_static",
           "prefixkv_selftest_bounded_wait", "prefixkv_compact_merge", "prefixkv_decode_static_limit_bytes"]


class Shape(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("layers", ctypes.c_int32), ("heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("prompt_len", ctypes.c_int32),
                ("dtype", ctypes.c_int32)]


class Strides(ctypes.Structure):
    _fields_ = [("b", ctypes.c_int64), ("l", ctypes.c_int64), ("h", ctypes.c_int64),
                ("n", ctypes.c_int64)]


class CacheStruct(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("row_offset", ctypes.c_void_p),
                ("len", ctypes.c_void_p), ("cap", ctypes.c_void_p),
                ("total_cap_rows", ctypes.c_int64), ("decode_cap", ctypes.c_int32),
                ("evict_distance", ctypes.c_int32), ("len0", ctypes.c_void_p),
                ("gen", ctypes.c_void_p), ("slot_ring", ctypes.c_void_p)]


class PrefixKVError(RuntimeError):
    pass


def _load():
    path = _build.LIB_PATH
    if not os.path.exists(path):
        raise ImportError(
            "libprefixkv.so is not built; run `python -m paper_2412_03409_b200.build` "
            "(needs nvcc). There is no fallback path.")
    lib = ctypes.CDLL(path)
    lib.prefixkv_workspace_bytes.restype = ctypes.c_size_t
    lib.prefixkv_workspace_bytes.argtypes = [ctypes.POINTER(Shape), ctypes.c_int]
    lib.prefixkv_last_cuda_error.restype = ctypes.c_char_p
    vp, i32, i64, f64, sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_double,
                             ctypes.c_size_t)
    sp = ctypes.POINTER(Shape)
    lib.prefixkv_score.argtypes = [sp, vp, Strides, vp, Strides, vp, vp, vp, vp, sz, vp]
    lib.prefixkv_search.argtypes = [sp, vp, vp, f64, i32, i64, i64, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.prefixkv_apply_lengths.argtypes = [sp, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp]
    lib.prefixkv_compact.argtypes = [sp, vp, Strides, vp, Strides, vp, vp,
                                     ctypes.POINTER(CacheStruct), vp, vp, vp, sz, vp]
    lib.prefixkv_decode_attn.argtypes = [sp, ctypes.POINTER(CacheStruct), vp, vp, vp, vp, i32, i32,
                                         vp, vp, vp, sz, vp]
    lib.prefixkv_gini.argtypes = [sp, vp, vp, vp]
    lib.prefixkv_rescale.argtypes = [sp, vp, vp, vp, vp]
    lib.prefixkv_estimate_config.argtypes = [sp, vp, i64, vp, vp, vp]
    lib.prefixkv_decode_attn_static.argtypes = [sp, ctypes.POINTER(CacheStruct), vp, vp, vp, vp,
                                                i32, i32, vp, vp, vp]
    lib.prefixkv_selftest_bounded_wait.argtypes = [i32, vp, vp]
    lib.prefixkv_compact_merge.argtypes = [sp, vp, Strides, vp, Strides, vp, vp, ctypes.POINTER(CacheStruct), i32,
                                           vp, vp, vp, vp, sz, vp]
    for name in EXPORTS[2:-1]:
        getattr(lib, name).restype = ctypes.c_int
    lib.prefixkv_decode_static_limit_bytes.restype = ctypes.c_size_t
    lib.prefixkv_decode_static_limit_bytes.argtypes = []
    return lib


_lib = _load()


def lib():
    return _lib


def _check(rc, what):
    if rc != PKV_OK:
        names = ["OK", "INVALID_ARG", "UNSUPPORTED", "WORKSPACE", "CUDA", "STATIC_LIMIT"]
        extra = _lib.prefixkv_last_cuda_error().decode() if rc >= PKV_ERR_CUDA else ""
        raise PrefixKVError("%s failed: PKV_ERR_%s %s" % (what, names[rc] if rc < 6 else rc, extra))


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_shape(B, L, H, D, N, dtype) -> Shape:
    return Shape(B, L, H, D, N, F32 if dtype == torch.float32 else BF16)


def strides_of(t: torch.Tensor) -> Strides:
    """Element strides of a [B, L, H, N, D] view (D must be contiguous)."""
    assert t.dim() == 5 and t.stride(4) == 1
    return Strides(t.stride(0), t.stride(1), t.stride(2), t.stride(3))


def prefixkv_workspace_bytes(shape: Shape, which: int) -> int:
    return int(_lib.prefixkv_workspace_bytes(ctypes.byref(shape), which))


def alloc_workspace(shape: Shape, which: int, device) -> torch.Tensor:
    n = max(256, prefixkv_workspace_bytes(shape, which))
    return torch.empty(n, dtype=torch.uint8, device=device)


def _ws(ws):
    return (_ptr(ws), ws.numel()) if ws is not None else (None, 0)


def prefixkv_score(shape, q, k, layer_scale, scores, ws, lse=None):
    p, n = _ws(ws)
    _check(_lib.prefixkv_score(ctypes.byref(shape), _ptr(q), strides_of(q), _ptr(k), strides_of(k),
                               _ptr(layer_scale), _ptr(lse), _ptr(scores), p, n, _stream()),
           "prefixkv_score")


def prefixkv_search(shape, scores, budget_rows, tol, max_iters, slack_rows, order, cum, length,
                    p_out, iters_out, dev_status, ws=None, slack_over_rows=0):
    p, n = _ws(ws)
    _check(_lib.prefixkv_search(ctypes.byref(shape), _ptr(scores), _ptr(budget_rows), float(tol),
                                int(max_iters), int(slack_rows), int(slack_over_rows), _ptr(order), _ptr(cum),
                                _ptr(length), _ptr(p_out), _ptr(iters_out), _ptr(dev_status), p, n,
                                _stream()), "prefixkv_search")


def prefixkv_apply_lengths(shape, scores, len_in, per_sample, order, cum, length, dev_status,
                           ws=None):
    p, n = _ws(ws)
    _check(_lib.prefixkv_apply_lengths(ctypes.byref(shape), _ptr(scores), _ptr(len_in),
                                       int(per_sample), _ptr(order), _ptr(cum), _ptr(length),
                                       _ptr(dev_status), p, n, _stream()), "prefixkv_apply_lengths")


@dataclass
class Cache:
    """Device buffers of one ragged cache plus the C struct that points at them."""
    k: torch.Tensor
    v: torch.Tensor
    row_offset: torch.Tensor
    len: torch.Tensor
    cap: torch.Tensor
    total_cap_rows: int
    decode_cap: int
    evict_distance: int = 0
    len0: torch.Tensor = None
    gen: torch.Tensor = None
    slot_ring: torch.Tensor = None
    c: CacheStruct = None

    def __post_init__(self):
        self.c = CacheStruct(self.k.data_ptr(), self.v.data_ptr(), self.row_offset.data_ptr(),
                             self.len.data_ptr(), self.cap.data_ptr(), self.total_cap_rows,
                             self.decode_cap, self.evict_distance,
                             self.len0.data_ptr() if self.len0 is not None else None,
                             self.gen.data_ptr() if self.gen is not None else None,
                             self.slot_ring.data_ptr() if self.slot_ring is not None else None)


def alloc_cache(shape: Shape, total_rows: int, decode_cap: int, device, fill=None,
                evict_distance: int = 0) -> Cache:
    """total_rows: host-known upper bound on the retained rows of all samples."""
    nseg = shape.batch * shape.layers
    dt = torch.float32 if shape.dtype == F32 else torch.bfloat16
    cap_rows = int(total_rows) + nseg * int(decode_cap)
    if fill is None:
        mk = lambda *s: torch.empty(*s, dtype=dt, device=device)
    else:
        mk = lambda *s: torch.full(s, fill, dtype=dt, device=device)
    return Cache(mk(cap_rows, shape.heads, shape.head_dim), mk(cap_rows, shape.heads, shape.head_dim),
                 torch.zeros(nseg + 1, dtype=torch.int64, device=device),
                 torch.zeros(nseg, dtype=torch.int32, device=device),
                 torch.zeros(nseg, dtype=torch.int32, device=device), cap_rows, int(decode_cap),
                 int(evict_distance),
                 torch.zeros(nseg, dtype=torch.int32, device=device) if evict_distance > 0 else None,
                 torch.zeros(nseg, dtype=torch.int32, device=device) if evict_distance > 0 else None,
                 torch.full((nseg, evict_distance + 1), -1, dtype=torch.int32, device=device)
                 if evict_distance > 0 else None)


def prefixkv_compact(shape, k, v, order, length, cache: Cache, dev_status, ws, kept=None):
    p, n = _ws(ws)
    _check(_lib.prefixkv_compact(ctypes.byref(shape), _ptr(k), strides_of(k), _ptr(v), strides_of(v),
                                 _ptr(order), _ptr(length), ctypes.byref(cache.c), _ptr(kept),
                                 _ptr(dev_status), p, n, _stream()), "prefixkv_compact")


def prefixkv_decode_attn(shape, cache: Cache, q, k_new, v_new, layer_scale, out, dev_status, ws,
                         layer_begin=0, layer_end=None):
    p, n = _ws(ws)
    le = shape.layers if layer_end is None else layer_end
    _check(_lib.prefixkv_decode_attn(ctypes.byref(shape), ctypes.byref(cache.c), _ptr(q), _ptr(k_new),
                                     _ptr(v_new), _ptr(layer_scale), int(layer_begin), int(le),
                                     _ptr(out), _ptr(dev_status), p, n, _stream()),
           "prefixkv_decode_attn")


def prefixkv_gini(shape, cum, gini):
    _check(_lib.prefixkv_gini(ctypes.byref(shape), _ptr(cum), _ptr(gini), _stream()), "prefixkv_gini")


def prefixkv_decode_static_limit_bytes() -> int:
    return int(_lib.prefixkv_decode_static_limit_bytes())


def prefixkv_decode_attn_static(shape, cache: Cache, q, k_new, v_new, layer_scale, out, dev_status,
                                layer_begin=0, layer_end=None):
    """Decode step that takes no workspace: for callers that cannot allocate device
    memory by the time they decode (all of it already sits in their own pool, or an
    allocation's device-wide synchronisation is not acceptable between tokens).  The
    split-K scratch is a fixed 16 MiB array inside the library; larger shapes raise.
    Calls share that array, so do not let two of them overlap on one GPU."""
    le = shape.layers if layer_end is None else layer_end
    _check(_lib.prefixkv_decode_attn_static(ctypes.byref(shape), ctypes.byref(cache.c), _ptr(q),
                                            _ptr(k_new), _ptr(v_new), _ptr(layer_scale),
                                            int(layer_begin), int(le), _ptr(out), _ptr(dev_status),
                                            _stream()), "prefixkv_decode_attn_static")


def prefixkv_rescale(shape, length, budget_rows, dev_status):
    _check(_lib.prefixkv_rescale(ctypes.byref(shape), _ptr(length), _ptr(budget_rows), _ptr(dev_status),
                                 _stream()), "prefixkv_rescale")


def prefixkv_estimate_config(shape, length, budget_rows, len_out, dev_status):
    _check(_lib.prefixkv_estimate_config(ctypes.byref(shape), _ptr(length), int(budget_rows),
                                         _ptr(len_out), _ptr(dev_status), _stream()),
           "prefixkv_estimate_config")


def prefixkv_selftest_bounded_wait(which, dev_status):
    _check(_lib.prefixkv_selftest_bounded_wait(int(which), _ptr(dev_status), _stream()),
           "prefixkv_selftest_bounded_wait")


def prefixkv_compact_merge(shape, k, v, order, length, cache: Cache, mode, dev_status, ws, kept=None, match=None):
    p, n = _ws(ws)
    _check(_lib.prefixkv_compact_merge(ctypes.byref(shape), _ptr(k), strides_of(k), _ptr(v), strides_of(v),
                                       _ptr(order), _ptr(length), ctypes.byref(cache.c), int(mode), _ptr(kept),
                                       _ptr(match), _ptr(dev_status), p, n, _stream()), "prefixkv_compact_merge")
