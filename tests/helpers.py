"""Oracle-side drivers shared by the GPU parity tests (host numpy only)."""
from __future__ import annotations

import multiprocessing
from concurrent.futures import ProcessPoolExecutor

import numpy as np
import torch

import oracle


def to_np32(t: torch.Tensor) -> np.ndarray:
    """Exact fp32 copy on the host (bf16 -> fp32 is exact)."""
    return t.detach().to("cpu", torch.float32).numpy()


def _score_job(args):
    q, k, scale = args
    return oracle.score_layer(q, k, scale)


def oracle_scores(q, k, layer_scale, segs=None, workers=8):
    """q, k: [B, L, H, N, D] torch (any device).  Returns {(b, l): scores[N]}."""
    B, L = q.shape[:2]
    segs = [(b, l) for b in range(B) for l in range(L)] if segs is None else list(segs)
    jobs = [(to_np32(q[b, l]), to_np32(k[b, l]), float(layer_scale[l])) for b, l in segs]
    work = q.shape[2] * q.shape[3] ** 2 * q.shape[4] * len(jobs)
    if work < 5e8 or workers <= 1 or len(jobs) == 1:
        res = [_score_job(j) for j in jobs]
    else:
        oracle.build()
        ctx = multiprocessing.get_context("spawn")     # never fork a process that holds a CUDA context
        with ProcessPoolExecutor(max_workers=workers, mp_context=ctx) as ex:
            res = list(ex.map(_score_job, jobs))
    return dict(zip(segs, res))


def oracle_select(scores_np, budgets, tol=1e-6, max_iters=64, slack=0):
    """scores_np [B, L, N] fp32 -> per-sample (order, cum, SearchResult)."""
    out = []
    for b in range(scores_np.shape[0]):
        out.append(oracle.select_sample(scores_np[b], int(budgets[b]), tol, max_iters, slack))
    return out


def check_scores(got: np.ndarray, ref: np.ndarray, tol: float):
    """|g - o| <= tol * max(|o|, 1e-3): relative, with a floor for near-zero scores
    (the scores of a layer have mean exactly 1)."""
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    bound = tol * np.maximum(np.abs(ref.astype(np.float64)), 1e-3)
    worst = float((err / bound).max())
    assert worst <= 1.0, "score error %.3g x bound (max abs err %.3g)" % (worst, err.max())
    return worst
