"""PrefixKV CPU oracle (test infrastructure only).

Thin ctypes access to ``prefixkv_oracle.c``: a plain single-threaded fp64
restatement of the paper's definitions (Sec. 3.1-3.3, Eq. 1, Algorithm 1).
Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
import this package.  It shares nothing with the CUDA library and never
imports it.

All array arguments are numpy arrays on the host.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "prefixkv_oracle.c")
_LIB = os.path.join(_HERE, "libprefixkv_oracle.so")

OK, BAD_SCORE, RANGE, BUDGET_TOO_SMALL, BAD_LENGTH = 0, 1, 2, 3, 4


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fused multiply-add contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared",
             "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_length_for_p.restype = ctypes.c_int32
        _lib.orc_gini.restype = ctypes.c_double
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def score_layer(q, k, scale, want_f64=False):
    """I_l^n for one layer of one sample.  q, k: [H, N, D] fp32 -> [N] fp32."""
    q, k = _f32(q), _f32(k)
    H, N, D = q.shape
    assert k.shape == q.shape
    out = np.empty(N, np.float32)
    out64 = np.empty(N, np.float64)
    _L().orc_score_layer(_p(q, ctypes.c_float), _p(k, ctypes.c_float), H, N, D,
                         ctypes.c_double(float(scale)), _p(out, ctypes.c_float),
                         _p(out64, ctypes.c_double))
    return (out, out64) if want_f64 else out


def lse_layer(q, k, scale):
    """Natural-log normaliser of every query's causal softmax.  q, k: [H, N, D] -> [H, N] fp64."""
    q, k = _f32(q), _f32(k)
    H, N, D = q.shape
    assert k.shape == q.shape
    out = np.empty((H, N), np.float64)
    _L().orc_lse_layer(_p(q, ctypes.c_float), _p(k, ctypes.c_float), H, N, D,
                       ctypes.c_double(float(scale)), _p(out, ctypes.c_double))
    return out


def sort_desc(scores):
    """Priority sequence s_l^1..s_l^N: positions by (importance desc, position asc)."""
    scores = _f32(scores)
    N = scores.shape[0]
    order = np.empty(N, np.int32)
    _L().orc_sort_desc(_p(scores, ctypes.c_float), N, _p(order, ctypes.c_int32))
    return order


def cumulative(scores, order):
    """Fixed-point (2^-32) inclusive prefix sums along the priority sequence."""
    scores = _f32(scores)
    order = np.ascontiguousarray(order, np.int32)
    N = scores.shape[0]
    cum = np.zeros(N, np.uint64)
    st = _L().orc_cumulative(_p(scores, ctypes.c_float), _p(order, ctypes.c_int32), N,
                             _p(cum, ctypes.c_uint64))
    return cum, int(st)


def length_for_p(cum, p):
    cum = np.ascontiguousarray(cum, np.uint64)
    return int(_L().orc_length_for_p(_p(cum, ctypes.c_uint64), cum.shape[0],
                                     ctypes.c_double(float(p))))


@dataclass
class SearchResult:
    len: np.ndarray
    p: float
    iters: int
    status: int


def search(cum, budget, tol=1e-6, max_iters=64, slack=0, slack_over=0):
    """Algorithm 1 over cum[L, N] with an integer row budget.  A midpoint whose total misses the
    budget by at most `slack` rows from below, or `slack_over` rows from above, ends the search."""
    cum = np.ascontiguousarray(cum, np.uint64)
    L, N = cum.shape
    ln = np.zeros(L, np.int32)
    p = ctypes.c_double(0.0)
    it = ctypes.c_int32(0)
    st = _L().orc_search(_p(cum, ctypes.c_uint64), L, N, ctypes.c_int64(int(budget)),
                         ctypes.c_double(float(tol)), ctypes.c_int32(int(max_iters)),
                         ctypes.c_int64(int(slack)), ctypes.c_int64(int(slack_over)),
                         _p(ln, ctypes.c_int32), ctypes.byref(p), ctypes.byref(it))
    return SearchResult(ln, p.value, it.value, int(st))


def check_lengths(len_in, N):
    len_in = np.ascontiguousarray(len_in, np.int32)
    return int(_L().orc_check_lengths(_p(len_in, ctypes.c_int32), len_in.shape[0], int(N)))


def retained_positions(order, length):
    order = np.ascontiguousarray(order, np.int32)
    kept = np.empty(int(length), np.int32)
    _L().orc_retained_positions(_p(order, ctypes.c_int32), order.shape[0], int(length),
                                _p(kept, ctypes.c_int32))
    return kept


def gather_rows(src, kept):
    """src [H, N, D] fp32 -> [len, H, D] rows in ascending position."""
    src = _f32(src)
    kept = np.ascontiguousarray(kept, np.int32)
    H, N, D = src.shape
    dst = np.empty((kept.shape[0], H, D), np.float32)
    _L().orc_gather_rows(_p(src, ctypes.c_float), H, N, D, _p(kept, ctypes.c_int32),
                         kept.shape[0], _p(dst, ctypes.c_float))
    return dst


MERGE_POSITION, MERGE_FEATURE = 1, 2


def merge_match(k, kept, mode, want_gap=False):
    """Which retained vector every position merges into (Sec. 4.3).  k [H, N, D]; kept ascending.
    Returns match[H, N] (indices into kept) and, on request, the best-minus-second metric."""
    k = _f32(k)
    kept = np.ascontiguousarray(kept, np.int32)
    H, N, D = k.shape
    match = np.empty((H, N), np.int32)
    gap = np.empty((H, N), np.float64)
    _L().orc_merge_match(_p(k, ctypes.c_float), H, N, D, _p(kept, ctypes.c_int32), kept.shape[0], int(mode),
                         _p(match, ctypes.c_int32), _p(gap, ctypes.c_double))
    return (match, gap) if want_gap else match


def merge_rows(src, kept, match):
    """Merged cache rows [len, H, D] (fp64) of src [H, N, D] under the assignment match[H, N]."""
    src = _f32(src)
    kept = np.ascontiguousarray(kept, np.int32)
    match = np.ascontiguousarray(match, np.int32)
    H, N, D = src.shape
    dst = np.empty((kept.shape[0], H, D), np.float64)
    _L().orc_merge_rows(_p(src, ctypes.c_float), H, N, D, _p(kept, ctypes.c_int32), kept.shape[0],
                        _p(match, ctypes.c_int32), _p(dst, ctypes.c_double))
    return dst


def decode_attn(q, kc, vc, scale):
    """q [H, D]; kc, vc [rows, H, D] (new row already appended) -> [H, D] fp64."""
    q, kc, vc = _f32(q), _f32(kc), _f32(vc)
    rows, H, D = kc.shape
    out = np.empty((H, D), np.float64)
    _L().orc_decode_attn(_p(q, ctypes.c_float), _p(kc, ctypes.c_float),
                         _p(vc, ctypes.c_float), rows, H, D,
                         ctypes.c_double(float(scale)), _p(out, ctypes.c_double))
    return out


def gini(scores, order):
    scores = _f32(scores)
    order = np.ascontiguousarray(order, np.int32)
    return float(_L().orc_gini(_p(scores, ctypes.c_float), _p(order, ctypes.c_int32),
                               scores.shape[0]))


def budget_rows(r, L, N):
    """Integer budget r * L * N (Sec. 3.2), rounded down."""
    return int(np.floor(r * L * N + 1e-9))


def select_sample(scores, budget, tol=1e-6, max_iters=64, slack=0, slack_over=0):
    """Sort + cumulative + search for one sample.  scores: [L, N] fp32."""
    scores = _f32(scores)
    L, N = scores.shape
    order = np.stack([sort_desc(scores[l]) for l in range(L)])
    cums, status = [], OK
    for l in range(L):
        c, st = cumulative(scores[l], order[l])
        cums.append(c)
        if st != OK and status == OK:
            status = st
    cum = np.stack(cums)
    if status != OK:
        return order, cum, SearchResult(np.zeros(L, np.int32), 0.0, 0, status)
    return order, cum, search(cum, budget, tol, max_iters, slack, slack_over)


def apportion(weight, budget, N):
    """Split `budget` rows over layers: one each, the rest in proportion to weight[l]."""
    weight = np.ascontiguousarray(weight, np.int64)
    out = np.zeros(weight.shape[0], np.int32)
    st = _L().orc_apportion(_p(weight, ctypes.c_int64), weight.shape[0], ctypes.c_int64(int(budget)),
                            int(N), _p(out, ctypes.c_int32))
    return out, int(st)


def rescale(length, budget, N):
    """Scale a searched configuration to meet the budget exactly (grows one below it, shrinks
    one above it, never below one row per layer)."""
    return apportion(np.asarray(length, np.int64) - 1, budget, N)


def estimate_config(lengths, budget, N):
    """One configuration for all inputs from the per-sample lengths[K, L] of K sample prompts."""
    return apportion((np.asarray(lengths, np.int64) - 1).sum(axis=0), budget, N)


def decode_slot(len0, N, g, n, d, ring):
    """Where generated token g goes in a layer's cache (see orc_decode_slot).
    ring: int32 array of d + 1 entries, updated in place.  Returns (dst, evicted, rows_after)."""
    assert ring.dtype == np.int32 and ring.flags["C_CONTIGUOUS"] and ring.shape[0] == d + 1
    dst, ev = ctypes.c_int32(0), ctypes.c_int32(0)
    _L().orc_decode_slot.restype = ctypes.c_int32
    rows = _L().orc_decode_slot(int(len0), int(N), int(g), int(n), int(d), _p(ring, ctypes.c_int32),
                                ctypes.byref(dst), ctypes.byref(ev))
    return dst.value, bool(ev.value), int(rows)
