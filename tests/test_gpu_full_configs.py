"""The five full-size workloads, in the launch configuration bench.py times, against the
oracle: sampled outputs where the oracle can compute them one by one, properties that hold at
any size elsewhere.  Selection is compared bit for bit on the library's own fp32 scores."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_scores, oracle_scores, oracle_select, to_np32
from paper_2412_03409_b200 import workloads as wl

pytestmark = pytest.mark.gpu

SCORE_TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-3}
DECODE_TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}


def _session(w, budget_rows, decode_cap):
    from paper_2412_03409_b200.session import Session
    return Session(w.B, w.L, w.H, w.D, w.N, w.dtype, wl.layer_scale(w), decode_cap=decode_cap,
                   max_budget_rows=budget_rows)


def _check_selection(s, scores_np, budgets, tol, samples):
    for b in samples:
        order, cum, res = oracle.select_sample(scores_np[b], int(budgets[b]), tol)
        np.testing.assert_array_equal(s.order[b].cpu().numpy(), order)
        np.testing.assert_array_equal(s.cum[b].cpu().numpy().view(np.uint64), cum)
        np.testing.assert_array_equal(s.len[b].cpu().numpy(), res.len)
        assert s.p[b].item() == res.p and s.iters[b].item() == res.iters
        assert int(s.len[b].sum()) <= budgets[b]
    return


def _score_properties(scores, N):
    assert torch.isfinite(scores).all() and (scores >= 0).all()
    sums = scores.double().sum(dim=-1)
    assert (sums - N).abs().max().item() <= 2e-3 * N            # every softmax row sums to one
    assert (scores[..., 0] >= 1.0 - 2e-3).all()                 # the first key is seen by all queries


def _check_steps(T):
    return sorted({t for t in (0, 1, 2, 7, 63, T - 1) if t < T})


def _decode_check(w, s, k, v, segs, steps, scale, check=None):
    """Decode `steps` tokens; compare the sampled segments with the oracle at the steps in
    `check` (all of them when None).  Only the sampled segments' appended rows are kept on the
    host, so every step of the full-size run can be decoded."""
    check = set(range(steps)) if check is None else set(check)
    caches = {}
    for b, l in segs:
        n = int(s.len[b, l])
        kept = oracle.retained_positions(s.order[b, l].cpu().numpy(), n)
        np.testing.assert_array_equal(s.kept[b, l, :n].cpu().numpy(), kept)
        off = int(s.cache.row_offset[b * w.L + l])
        rk = oracle.gather_rows(to_np32(k[b, l]), kept)
        assert np.array_equal(to_np32(s.cache.k[off:off + n]), rk)      # compaction is byte-exact
        caches[(b, l)] = [[rk], [oracle.gather_rows(to_np32(v[b, l]), kept)]]
    worst = 0.0
    for t in range(steps):
        qd, kn, vn = wl.make_decode_inputs(w, t, "cuda")
        out = s.decode(qd, kn, vn)
        for (b, l), (ck, cv) in caches.items():
            ck.append(to_np32(kn[b, l])[None])
            cv.append(to_np32(vn[b, l])[None])
        if t not in check:
            continue
        got = {seg: to_np32(out[seg[0], seg[1]]) for seg in caches}
        for (b, l), (ck, cv) in caches.items():
            ref = oracle.decode_attn(to_np32(qd[b, l]), np.concatenate(ck), np.concatenate(cv),
                                     float(scale[l]))
            assert np.isfinite(got[(b, l)]).all()
            worst = max(worst, float(np.abs(got[(b, l)] - ref).max()))
    assert worst <= DECODE_TOL[w.dtype], worst
    assert s.status.cpu().tolist() == [0] * w.B
    lens0 = s.len.flatten().cpu()
    assert torch.equal(s.cache.len.cpu(), lens0 + steps)               # every segment grew by one row per step


def test_llava7b_b1_full():
    w = wl.WORKLOADS["llava7b_b1"]
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    s = _session(w, w.budget_rows(), w.T)
    s.compress(q, k, v, w.budget_rows(), tol=w.tol)
    torch.cuda.synchronize()
    assert s.status.cpu().tolist() == [0]
    _score_properties(s.scores, w.N)
    got = s.scores.cpu().numpy()
    for (b, l), r in oracle_scores(q, k, scale, segs=[(0, 0), (0, 13), (0, 31)]).items():
        check_scores(got[b, l], r, SCORE_TOL[w.dtype])
    _check_selection(s, got, [w.budget_rows()], w.tol, [0])
    assert int(s.len.min()) < int(s.len.max())      # the per-layer lengths are ragged
    _decode_check(w, s, k, v, [(0, 0), (0, 13), (0, 31)], w.T, scale)


def test_llava7b_b16_budget_sweep():
    w = wl.WORKLOADS["llava7b_b16"]
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    s = _session(w, w.budget_rows(max(w.budget_ratios)), w.T)
    s.score(q, k)                       # scores do not depend on the budget: computed once
    _score_properties(s.scores, w.N)
    got = s.scores.cpu().numpy()
    for (b, l), r in oracle_scores(q, k, scale, segs=[(3, 5), (15, 31)]).items():
        check_scores(got[b, l], r, SCORE_TOL[w.dtype])
    prev = None
    for ratio in w.budget_ratios:
        budgets = [w.budget_rows(ratio)] * w.B
        s.search(budgets[0], tol=w.tol)
        s.compact(k, v)
        torch.cuda.synchronize()
        _check_selection(s, got, budgets, w.tol, range(w.B))
        lens = s.len.cpu().clone()
        if prev is not None:
            assert (lens >= prev).all()              # lengths grow with the budget
        prev = lens
        # per-sample ragged lengths packed in one cache
        offs = s.cache.row_offset.cpu().numpy()
        np.testing.assert_array_equal(np.diff(offs), s.cache.cap.cpu().numpy())
        _decode_check(w, s, k, v, [(0, 0), (7, 16), (15, 31)], w.T, scale, _check_steps(w.T))


def test_llava13b_b8_sampled():
    w = wl.WORKLOADS["llava13b_b8"]
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    s = _session(w, w.budget_rows(), w.T)
    s.compress(q, k, v, w.budget_rows(), tol=w.tol)
    torch.cuda.synchronize()
    assert s.status.cpu().tolist() == [0] * w.B
    _score_properties(s.scores, w.N)
    got = s.scores.cpu().numpy()
    for (b, l), r in oracle_scores(q, k, scale, segs=[(5, 20)]).items():
        check_scores(got[b, l], r, SCORE_TOL[w.dtype])
    _check_selection(s, got, [w.budget_rows()] * w.B, w.tol, [0, 7])
    _decode_check(w, s, k, v, [(0, 0), (7, 39)], w.T, scale, _check_steps(w.T))


def test_longctx_b4_properties_and_selection():
    w = wl.WORKLOADS["longctx_b4"]
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    s = _session(w, w.budget_rows(), w.T)
    s.compress(q, k, v, w.budget_rows(), tol=w.tol)
    torch.cuda.synchronize()
    assert s.status.cpu().tolist() == [0] * w.B
    _score_properties(s.scores, w.N)
    first = s.scores.clone()
    s.score(q, k)
    assert torch.equal(first, s.scores)              # deterministic at full size
    got = s.scores.cpu().numpy()
    _check_selection(s, got, [w.budget_rows()] * w.B, w.tol, [0])
    assert int(s.len.sum(dim=1).max()) <= w.budget_rows() == 26214
    _decode_check(w, s, k, v, [(0, 3), (3, 31)], w.T, scale, _check_steps(w.T))


def test_score_longest_prompt_against_oracle():
    """N = 16384 (the longest supported prompt) with one head so that the oracle finishes."""
    w = wl.scaled(wl.WORKLOADS["longctx_b4"], B=1, L=1, H=1)
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    s = _session(w, w.budget_rows(), 1)
    got = s.score(q, k).cpu().numpy()
    ref = oracle_scores(q, k, scale)[(0, 0)]
    check_scores(got[0, 0], ref, SCORE_TOL[w.dtype])
    s.search(w.budget_rows(), tol=w.tol)
    _check_selection(s, got, [w.budget_rows()], w.tol, [0])
