"""Pins for the CPU oracle: closed forms, library routines, exact arithmetic,
brute force and a hand-worked example.  None of these re-type the oracle's own
loops; each is chosen so that a plausible slip (sign, index, transposed operand,
missing term, wrong tie-break or rounding) fails."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------
# Importance score (Sec. 3.2)
# --------------------------------------------------------------------------
def _softmax_colsum_library(q, k, scale):
    """Column sums of the causal softmax via torch.softmax on a masked matrix."""
    H, N, D = q.shape
    qt = torch.from_numpy(q).double()
    kt = torch.from_numpy(k).double()
    logits = scale * qt @ kt.transpose(1, 2)                      # [H, m, n]
    mask = torch.ones(N, N, dtype=torch.bool).tril()              # n <= m
    logits = logits.masked_fill(~mask, float("-inf"))
    a = torch.softmax(logits, dim=-1)
    return a.sum(dim=1).mean(dim=0).numpy()                       # sum over m, mean over heads


@pytest.mark.parametrize("H,N,D,scale", [(3, 37, 8, 0.7), (2, 64, 16, 1.0), (1, 5, 4, 2.5)])
def test_score_matches_library_softmax(H, N, D, scale):
    rng = np.random.default_rng(H * 100 + N)
    q = rng.standard_normal((H, N, D)).astype(np.float32)
    k = rng.standard_normal((H, N, D)).astype(np.float32)
    f32, f64 = oracle.score_layer(q, k, scale, want_f64=True)
    ref = _softmax_colsum_library(q, k, scale)
    np.testing.assert_allclose(f64, ref, rtol=1e-12, atol=1e-14)
    np.testing.assert_array_equal(f32, ref.astype(np.float32))
    # swapping the operands must not give the same answer (transposition check)
    swapped = oracle.score_layer(k, q, scale)
    assert np.abs(swapped - f32).max() > 1e-3


def test_score_zero_query_is_harmonic():
    """Q = 0 makes every causal row uniform: a^{m,n} = 1/m, so
    I^n = H_N - H_{n-1} (1-based n), for any head count."""
    H, N, D = 3, 50, 4
    rng = np.random.default_rng(1)
    q = np.zeros((H, N, D), np.float32)
    k = rng.standard_normal((H, N, D)).astype(np.float32)
    _, f64 = oracle.score_layer(q, k, 1.0, want_f64=True)
    harm = [Fraction(0)]
    for i in range(1, N + 1):
        harm.append(harm[-1] + Fraction(1, i))
    ref = np.array([float(harm[N] - harm[n]) for n in range(N)])
    np.testing.assert_allclose(f64, ref, rtol=1e-13)
    # same with scale = 0 and arbitrary Q
    q2 = rng.standard_normal((H, N, D)).astype(np.float32)
    _, g64 = oracle.score_layer(q2, k, 0.0, want_f64=True)
    np.testing.assert_allclose(g64, ref, rtol=1e-13)


def test_score_invariants():
    H, N, D = 4, 48, 8
    rng = np.random.default_rng(2)
    q = rng.standard_normal((H, N, D)).astype(np.float32)
    k = rng.standard_normal((H, N, D)).astype(np.float32)
    _, I = oracle.score_layer(q, k, 0.9, want_f64=True)
    # every causal softmax row sums to one, so the scores sum to N
    assert abs(I.sum() - N) < 1e-9 * N
    # first key is seen by every query and alone by the first: I^1 >= 1
    assert I[0] >= 1.0
    # last key is seen only by the last query: I^N = mean_h a^{N,N}
    ref = _softmax_colsum_library(q, k, 0.9)
    assert abs(I[-1] - ref[-1]) < 1e-14
    # the head mean does not depend on head order
    perm = np.array([2, 0, 3, 1])
    _, Ip = oracle.score_layer(q[perm], k[perm], 0.9, want_f64=True)
    np.testing.assert_allclose(Ip, I, rtol=1e-13)
    # adding one vector to every key shifts each row's logits by a constant
    kq = np.round(k * 1024) / np.float32(1024)          # so that k + 0.5 is exact in fp32
    c = np.full((1, 1, D), 0.5, np.float32)
    _, I0 = oracle.score_layer(q, kq, 0.9, want_f64=True)
    _, Is = oracle.score_layer(q, kq + c, 0.9, want_f64=True)
    np.testing.assert_allclose(Is, I0, rtol=1e-11)
    # head mean, not head sum: duplicating the heads changes nothing
    _, Id = oracle.score_layer(np.concatenate([q, q]), np.concatenate([k, k]), 0.9, want_f64=True)
    np.testing.assert_allclose(Id, I, rtol=1e-13)


def test_lse_matches_library_and_closed_form():
    """The per-query normaliser: torch.logsumexp over the masked logits; log(m) when every
    logit of query m (1-based) is zero; and exp(logit - lse) column-summed reproduces the score."""
    H, N, D, scale = 3, 41, 8, 0.8
    rng = np.random.default_rng(77)
    q = rng.standard_normal((H, N, D)).astype(np.float32)
    k = rng.standard_normal((H, N, D)).astype(np.float32)
    lse = oracle.lse_layer(q, k, scale)
    logits = scale * torch.from_numpy(q).double() @ torch.from_numpy(k).double().transpose(1, 2)
    mask = torch.ones(N, N, dtype=torch.bool).tril()
    ref = torch.logsumexp(logits.masked_fill(~mask, float("-inf")), dim=-1).numpy()
    np.testing.assert_allclose(lse, ref, rtol=1e-13, atol=1e-13)
    zero = oracle.lse_layer(np.zeros_like(q), k, 1.0)
    np.testing.assert_allclose(zero, np.log(np.arange(1, N + 1))[None].repeat(H, 0), rtol=1e-14, atol=1e-15)
    # operand order matters (q^m . k^j with j <= m, not the transpose)
    assert np.abs(oracle.lse_layer(k, q, scale) - lse).max() > 1e-3
    probs = torch.exp(logits - torch.from_numpy(lse)[..., None]).masked_fill(~mask, 0.0)
    _, I = oracle.score_layer(q, k, scale, want_f64=True)
    np.testing.assert_allclose(probs.sum(dim=1).mean(dim=0).numpy(), I, rtol=1e-12)


def test_score_single_token():
    q = np.full((2, 1, 4), 3.0, np.float32)
    assert oracle.score_layer(q, q, 1.0)[0] == 1.0


# --------------------------------------------------------------------------
# Priority sequence (Sec. 3.2)
# --------------------------------------------------------------------------
def test_sort_matches_library_and_tie_break():
    rng = np.random.default_rng(3)
    for N in (1, 2, 17, 300):
        s = rng.random(N).astype(np.float32)
        s[rng.integers(0, N, N // 3 + 1)] = s[rng.integers(0, N, N // 3 + 1)]   # ties
        ref = sorted(range(N), key=lambda n: (-float(s[n]), n))
        np.testing.assert_array_equal(oracle.sort_desc(s), ref)
    np.testing.assert_array_equal(oracle.sort_desc(np.ones(9, np.float32)), np.arange(9))
    np.testing.assert_array_equal(oracle.sort_desc(np.arange(9, dtype=np.float32)), np.arange(9)[::-1])
    # -0.0 and +0.0 are one value: position decides
    z = np.array([0.0, -0.0, 1.0, -0.0, 0.0], np.float32)
    np.testing.assert_array_equal(oracle.sort_desc(z), [2, 0, 1, 3, 4])


# --------------------------------------------------------------------------
# Cumulative priority in 2^-32 fixed point (Sec. 3.2)
# --------------------------------------------------------------------------
def _round_half_even(fr: Fraction) -> int:
    fl = fr.numerator // fr.denominator
    rem = fr - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        return fl + 1
    return fl


def test_cumulative_exact_arithmetic():
    rng = np.random.default_rng(4)
    N = 200
    s = np.exp(rng.standard_normal(N) * 3 - 8).astype(np.float32)
    s[:4] = [2.0 ** -33, 3 * 2.0 ** -33, 5 * 2.0 ** -33, 2.0 ** -34]      # halves: 0, 2, 2, 0
    order = oracle.sort_desc(s)
    cum, st = oracle.cumulative(s, order)
    assert st == oracle.OK
    run, ref = 0, []
    for j in order:
        run += _round_half_even(Fraction(float(s[j])) * 2 ** 32)
        ref.append(run)
    assert [int(c) for c in cum] == ref
    assert all(int(cum[i]) <= int(cum[i + 1]) for i in range(N - 1))
    # the total does not depend on the order of summation
    rev, _ = oracle.cumulative(s, order[::-1].copy())
    assert int(rev[-1]) == int(cum[-1])
    w = {float(s[i]): _round_half_even(Fraction(float(s[i])) * 2 ** 32) for i in range(4)}
    assert [w[float(s[i])] for i in range(4)] == [0, 2, 2, 0]


def test_cumulative_rejects_bad_scores():
    for bad in (float("nan"), float("inf"), -1.0):
        s = np.array([1.0, bad, 0.5], np.float32)
        _, st = oracle.cumulative(s, np.array([0, 1, 2], np.int32))
        assert st == oracle.BAD_SCORE
    s = np.array([2.0 ** 22, 1.0], np.float32)            # 2^54 in fixed point
    _, st = oracle.cumulative(s, np.array([0, 1], np.int32))
    assert st == oracle.RANGE


# --------------------------------------------------------------------------
# Retained length for a given p (Sec. 3.3)
# --------------------------------------------------------------------------
def test_length_rule_special_cases():
    N = 64
    ones = np.ones(N, np.float32)
    cum, _ = oracle.cumulative(ones, np.arange(N, dtype=np.int32))
    for p in (0.0, 1e-9, 0.1, 0.25, 0.3, 0.5, 0.77, 0.999):
        assert oracle.length_for_p(cum, p) == max(1, math.ceil(p * N)), p
    assert oracle.length_for_p(cum, 1.0) == N and oracle.length_for_p(cum, 1.5) == N
    onehot = np.zeros(N, np.float32); onehot[7] = 3.0
    order = oracle.sort_desc(onehot)
    cum, _ = oracle.cumulative(onehot, order)
    assert order[0] == 7
    for p in (0.0, 0.3, 0.999999):
        assert oracle.length_for_p(cum, p) == 1
    assert oracle.length_for_p(cum, 1.0) == N
    # equality at the threshold counts as reached ("larger than or equal to")
    s = np.array([0.5, 0.25, 0.25], np.float32)
    cum, _ = oracle.cumulative(s, np.arange(3, dtype=np.int32))
    assert oracle.length_for_p(cum, 0.5) == 1
    assert oracle.length_for_p(cum, np.nextafter(0.5, 1.0)) == 2
    assert oracle.length_for_p(cum, 0.75) == 2
    # monotone in p
    rng = np.random.default_rng(5)
    s = rng.random(100).astype(np.float32)
    cum, _ = oracle.cumulative(s, oracle.sort_desc(s))
    lens = [oracle.length_for_p(cum, p) for p in np.linspace(0, 1, 501)]
    assert lens == sorted(lens) and lens[0] == 1 and lens[-1] == 100


# --------------------------------------------------------------------------
# Binary search (Algorithm 1, Eq. 1)
# --------------------------------------------------------------------------
def _length_exact(cum_row, p: float) -> int:
    """The length rule re-derived with Python integers (no oracle code)."""
    N = len(cum_row)
    if p >= 1.0:
        return N
    theta = math.ceil(p * float(int(cum_row[-1])))
    return min(N, 1 + sum(1 for c in cum_row if int(c) < theta))


def _brute_force_config(cum, budget):
    """Largest feasible configuration by trying every breakpoint of S(p).

    S only changes where p * total crosses a cumulative value, so the fp64
    numbers around each cum/total are the only places the answer can change."""
    L, N = cum.shape
    cands = {0.0}
    for l in range(L):
        T = int(cum[l, -1])
        for c in cum[l]:
            x = float(Fraction(int(c), T))
            for _ in range(3):
                x = np.nextafter(x, 0.0)
            for _ in range(7):
                if 0.0 <= x < 1.0:
                    cands.add(float(x))
                x = np.nextafter(x, 2.0)
    best = None
    for p in sorted(cands):
        lens = [_length_exact(cum[l], p) for l in range(L)]
        if sum(lens) <= budget:
            best = (p, lens)
        else:
            break
    return best


@pytest.mark.parametrize("seed", range(6))
def test_search_equals_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    L, N = int(rng.integers(2, 6)), int(rng.integers(3, 24))
    scores = (rng.random((L, N)) ** rng.integers(1, 5)).astype(np.float32) + np.float32(1e-3)
    for budget in sorted({L, L + 1, (L * N) // 3, (L * N) // 2, L * N - 1}):
        if budget < L:
            continue
        order, cum, res = oracle.select_sample(scores, budget, tol=0.0, max_iters=4000)
        assert res.status == oracle.OK
        p_bf, len_bf = _brute_force_config(cum, budget)
        assert list(res.len) == len_bf, (budget, res, p_bf)
        assert res.len.sum() <= budget
        # with a tolerance the answer is feasible and never better than the optimum
        _, _, r6 = oracle.select_sample(scores, budget, tol=1e-6)
        assert r6.len.sum() <= sum(len_bf) <= budget
        assert r6.iters <= 20
        assert all(a <= b for a, b in zip(r6.len, len_bf))


def test_search_hand_example():
    A = np.array([11, 3, 2], np.float32) / 16
    B = np.array([6, 5, 5], np.float32) / 16
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "search_hand_example.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 4
    for budget, p, la, lb, steps in rows:
        _, cum, res = oracle.select_sample(np.stack([A, B]), int(budget), tol=0.0, max_iters=4000)
        assert [int(c) for c in cum[0]] == [11 << 28, 14 << 28, 16 << 28]
        assert res.p == float(p), (budget, res)
        assert list(res.len) == [int(la), int(lb)]
        if int(steps) >= 0:
            assert res.iters == int(steps)


def test_search_invariants():
    rng = np.random.default_rng(7)
    L, N = 6, 40
    scores = np.exp(rng.standard_normal((L, N)) * np.linspace(0.2, 2.5, L)[:, None]).astype(np.float32)
    prev = None
    for budget in range(L, L * N + 3, 7):
        _, cum, res = oracle.select_sample(scores, budget, tol=0.0, max_iters=4000)
        assert res.len.sum() <= budget
        assert (res.len >= 1).all() and (res.len <= N).all()
        if prev is not None:
            assert (res.len >= prev).all()          # lengths grow with the budget
        prev = res.len.copy()
    # full budget keeps everything at p = 1 without a single step
    _, _, res = oracle.select_sample(scores, L * N)
    assert res.p == 1.0 and (res.len == N).all() and res.iters == 0
    # below one row per layer is an error
    _, _, res = oracle.select_sample(scores, L - 1)
    assert res.status == oracle.BUDGET_TOO_SMALL
    # identical layers get identical lengths, floor(budget / L) when nothing ties
    same = np.tile(scores[3], (L, 1))
    for budget in (L * 5, L * 5 + 3, L * 17 + 5):
        _, _, res = oracle.select_sample(same, budget, tol=0.0, max_iters=4000)
        assert (res.len == budget // L).all(), (budget, res.len)
    # concentrated layers keep fewer rows than dispersed ones (Sec. 4.3, Fig. 5)
    _, _, res = oracle.select_sample(scores, L * N // 2, tol=0.0, max_iters=4000)
    assert res.len[0] > res.len[-1]
    # tol = 1e-6 stops after exactly 20 halvings unless delta hits zero first
    _, _, r6 = oracle.select_sample(scores, L * N // 2, tol=1e-6)
    assert r6.iters <= 20
    # iteration cap
    _, _, r3 = oracle.select_sample(scores, L * N // 2, tol=0.0, max_iters=3)
    assert r3.iters <= 3 and r3.len.sum() <= L * N // 2
    # one-sided slack: may stop early, never exceeds the budget
    _, _, rs = oracle.select_sample(scores, L * N // 2, tol=0.0, max_iters=4000, slack=5)
    assert 0 <= L * N // 2 - rs.len.sum() <= 5
    assert rs.iters <= res.iters


def test_given_lengths_validation():
    assert oracle.check_lengths([1, 5, 10], 10) == oracle.OK
    assert oracle.check_lengths([0, 5], 10) == oracle.BAD_LENGTH
    assert oracle.check_lengths([3, 11], 10) == oracle.BAD_LENGTH


# --------------------------------------------------------------------------
# Compaction (Sec. 3.1, Fig. 2a)
# --------------------------------------------------------------------------
def test_compact_keeps_top_ranked_rows_in_position_order():
    rng = np.random.default_rng(8)
    H, N, D = 3, 29, 4
    s = rng.random(N).astype(np.float32)
    order = oracle.sort_desc(s)
    src = rng.standard_normal((H, N, D)).astype(np.float32)
    for ln in (1, 7, N):
        kept = oracle.retained_positions(order, ln)
        assert list(kept) == sorted(int(x) for x in order[:ln])
        # the kept set is exactly the ln largest scores
        thresh = np.sort(s)[::-1][ln - 1]
        assert all(s[i] >= thresh for i in kept)
        rows = oracle.gather_rows(src, kept)
        np.testing.assert_array_equal(rows, src[:, kept, :].transpose(1, 0, 2))


# --------------------------------------------------------------------------
# Decode attention (Sec. 3.1)
# --------------------------------------------------------------------------
def test_decode_matches_library_attention():
    rng = np.random.default_rng(9)
    R, H, D = 33, 5, 16
    q = rng.standard_normal((H, D)).astype(np.float32)
    kc = rng.standard_normal((R, H, D)).astype(np.float32)
    vc = rng.standard_normal((R, H, D)).astype(np.float32)
    scale = 0.31
    out = oracle.decode_attn(q, kc, vc, scale)
    qt = torch.from_numpy(q).double()[:, None, :]                     # [H, 1, D]
    kt = torch.from_numpy(kc).double().permute(1, 0, 2)               # [H, R, D]
    vt = torch.from_numpy(vc).double().permute(1, 0, 2)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, scale=scale)[:, 0, :]
    np.testing.assert_allclose(out, ref.numpy(), rtol=1e-12, atol=1e-14)


def test_decode_special_cases():
    rng = np.random.default_rng(10)
    R, H, D = 12, 2, 8
    q = rng.standard_normal((H, D)).astype(np.float32)
    kc = rng.standard_normal((R, H, D)).astype(np.float32)
    vc = rng.standard_normal((R, H, D)).astype(np.float32)
    # a single row returns its value
    np.testing.assert_allclose(oracle.decode_attn(q, kc[:1], vc[:1], 1.0), vc[0], rtol=0, atol=0)
    # constant V comes back unchanged
    const = np.broadcast_to(np.float32(1.5), vc.shape).copy()
    np.testing.assert_allclose(oracle.decode_attn(q, kc, const, 1.0), 1.5, rtol=1e-14)
    # scale 0 gives the mean of the value rows
    np.testing.assert_allclose(oracle.decode_attn(q, kc, vc, 0.0), vc.mean(axis=0, dtype=np.float64),
                               rtol=1e-12, atol=1e-15)
    # the order of cached rows does not matter
    perm = rng.permutation(R)
    np.testing.assert_allclose(oracle.decode_attn(q, kc[perm], vc[perm], 0.7),
                               oracle.decode_attn(q, kc, vc, 0.7), rtol=1e-12, atol=1e-14)


def test_full_budget_decode_equals_dense_attention():
    """p = 1 keeps every prompt row, so decoding over the compacted cache plus
    the appended row is dense attention over the original K, V."""
    rng = np.random.default_rng(11)
    L, H, N, D = 2, 3, 20, 8
    q = rng.standard_normal((L, H, N, D)).astype(np.float32)
    k = rng.standard_normal((L, H, N, D)).astype(np.float32)
    v = rng.standard_normal((L, H, N, D)).astype(np.float32)
    scores = np.stack([oracle.score_layer(q[l], k[l], 0.35) for l in range(L)])
    order, cum, res = oracle.select_sample(scores, L * N)
    assert res.p == 1.0
    qn, kn, vn = (rng.standard_normal((L, H, D)).astype(np.float32) for _ in range(3))
    for l in range(L):
        kept = oracle.retained_positions(order[l], res.len[l])
        kc = np.concatenate([oracle.gather_rows(k[l], kept), kn[l][None]])
        vc = np.concatenate([oracle.gather_rows(v[l], kept), vn[l][None]])
        out = oracle.decode_attn(qn[l], kc, vc, 0.35)
        kt = torch.from_numpy(np.concatenate([k[l], kn[l][:, None]], axis=1)).double()
        vt = torch.from_numpy(np.concatenate([v[l], vn[l][:, None]], axis=1)).double()
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(qn[l]).double()[:, None], kt, vt, scale=0.35)[:, 0]
        np.testing.assert_allclose(out, ref.numpy(), rtol=1e-12, atol=1e-14)


# --------------------------------------------------------------------------
# Lorenz / Gini diagnostic (Sec. 3.2, Fig. 3)
# --------------------------------------------------------------------------
def test_gini_closed_forms():
    N = 50
    ones = np.ones(N, np.float32)
    assert abs(oracle.gini(ones, oracle.sort_desc(ones))) < 1e-12
    onehot = np.zeros(N, np.float32); onehot[3] = 2.0
    assert abs(oracle.gini(onehot, oracle.sort_desc(onehot)) - (1 - 1 / N)) < 1e-12
    # linear ramp 1..N: G = (N - 1) / (3 N)  (textbook value for the discrete uniform ramp, trapezoid rule)
    ramp = np.arange(1, N + 1, dtype=np.float32)
    g = oracle.gini(ramp, oracle.sort_desc(ramp))
    x = np.sort(ramp.astype(np.float64))
    ref = (2 * np.sum(np.arange(1, N + 1) * x) / (N * x.sum())) - (N + 1) / N
    assert abs(g - ref) < 1e-12


# --------------------------------------------------------------------------
# Meeting the budget exactly / offline configuration (Sec. 3.3)
# --------------------------------------------------------------------------
def _hamilton(weight, budget, N):
    """Hamilton's largest-remainder apportionment in closed form with exact rationals: every layer
    gets the floor of its quota, and the layers with the `rem` largest fractional parts (ties to
    the lower layer) one more -- one round, because fewer than L rows are left after the floors.
    Returns None when a layer would pass N rows (the cap is outside this textbook form)."""
    L = len(weight)
    extra = budget - L
    w = [int(x) for x in weight]
    if sum(w) == 0:
        w = [1] * L
    W = sum(w)
    quota = [Fraction(x * extra, W) for x in w]
    floors = [q.numerator // q.denominator for q in quota]
    rem = extra - sum(floors)
    assert 0 <= rem < L
    lucky = sorted(range(L), key=lambda l: (-(quota[l] - floors[l]), l))[:rem]
    out = [1 + floors[l] + (1 if l in lucky else 0) for l in range(L)]
    return out if max(out) <= N else None


def test_rescale_meets_budget_and_keeps_proportions():
    rng = np.random.default_rng(21)
    uncapped = capped = shrunk = 0
    for _ in range(120):
        L, N = int(rng.integers(1, 12)), int(rng.integers(2, 60))
        length = rng.integers(1, N + 1, L)
        budget = int(rng.integers(L, L * N + 5))
        out, st = oracle.rescale(length, budget, N)
        assert st == oracle.OK
        assert out.sum() == min(budget, L * N)
        assert (out <= N).all() and (out >= 1).all()
        if budget >= length.sum():
            assert (out >= length).all()                   # a configuration below the budget only grows
        else:
            assert (out <= length).all()                   # one above it only shrinks, never below one row
            shrunk += 1
        ref = _hamilton(length - 1, budget, N)
        if ref is not None:
            assert list(out) == ref
            uncapped += 1
        else:
            # the cap binds: whoever is not full got at least its floor quota, and a layer with a
            # larger weight never ends up with fewer rows
            capped += 1
            w = length - 1
            for a in range(L):
                for b in range(L):
                    if w[a] > w[b]:
                        assert out[a] >= out[b]
        same, _ = oracle.rescale(length, int(length.sum()), N)      # nothing to do: unchanged
        np.testing.assert_array_equal(same, length)
    assert uncapped > 20 and capped > 5 and shrunk > 20
    # the hand-worked search example: budget 4 was missed by one row (len = (1, 2)); the row
    # goes to the layer with the larger share beyond its mandatory row
    out, _ = oracle.rescale([1, 2], 4, 3)
    assert list(out) == [1, 3]
    assert oracle.rescale([1, 2], 1, 3)[1] == oracle.BUDGET_TOO_SMALL


def _bisect_model(cum, budget, under, over, max_iters=4000):
    """Algorithm 1 retold with Python integers and the independent length rule above: the
    midpoints are k / 2^j, the first one whose total lies within the thresholds is the answer."""
    L = cum.shape[0]
    lo, hi, it = Fraction(0), Fraction(1), 0
    while it < max_iters:
        mid = (lo + hi) / 2
        if float(mid) in (float(lo), float(hi)):
            break
        S = sum(_length_exact(cum[l], float(mid)) for l in range(L))
        it += 1
        if -under <= S - budget <= over:
            return float(mid), it, S
        if S < budget:
            lo = mid
        else:
            hi = mid
    return float(lo), it, sum(_length_exact(cum[l], float(lo)) for l in range(L))


@pytest.mark.parametrize("seed", range(5))
def test_search_two_sided_threshold(seed):
    """Sec. 3.3 / Tab. robustness-delta: the search may end once |delta| is within a threshold;
    the configuration is then scaled to the budget."""
    rng = np.random.default_rng(300 + seed)
    L, N = int(rng.integers(3, 8)), int(rng.integers(20, 60))
    scores = np.exp(rng.standard_normal((L, N)) * rng.uniform(0.3, 2.0, (L, 1))).astype(np.float32)
    budget = L * N // 3
    prev_iters = None
    for delta in (0, 1, 2, 4, 8, 16, 40):
        _, cum, res = oracle.select_sample(scores, budget, tol=0.0, max_iters=4000, slack=delta, slack_over=delta)
        p_ref, it_ref, S_ref = _bisect_model(cum, budget, delta, delta)
        assert (res.p, res.iters, int(res.len.sum())) == (p_ref, it_ref, S_ref)
        if prev_iters is not None:
            assert res.iters <= prev_iters                 # a wider threshold never needs more steps
        prev_iters = res.iters
        fixed, st = oracle.rescale(res.len, budget, N)     # "scale ... to meet the target budget"
        assert st == oracle.OK and fixed.sum() == budget and (fixed >= 1).all() and (fixed <= N).all()
        if res.len.sum() > budget:
            assert (fixed <= res.len).all()
        # over-side only: never accepted below the budget unless exact
        _, _, ro = oracle.select_sample(scores, budget, tol=0.0, max_iters=4000, slack=0, slack_over=delta)
        assert (ro.p, ro.iters) == _bisect_model(cum, budget, 0, delta)[:2]
    # a threshold as wide as the whole range accepts the very first midpoint
    _, _, r1 = oracle.select_sample(scores, budget, slack=L * N, slack_over=L * N)
    assert r1.iters == 1 and r1.p == 0.5


def test_search_delta_hand_example():
    A = np.array([11, 3, 2], np.float32) / 16
    B = np.array([6, 5, 5], np.float32) / 16
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "search_delta_hand_example.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 5
    for budget, under, over, p, la, lb, steps, ra, rb in rows:
        _, _, res = oracle.select_sample(np.stack([A, B]), int(budget), tol=0.0, max_iters=4000,
                                         slack=int(under), slack_over=int(over))
        assert (res.p, list(res.len), res.iters) == (float(p), [int(la), int(lb)], int(steps))
        fixed, _ = oracle.rescale(res.len, int(budget), 3)
        assert list(fixed) == [int(ra), int(rb)] and fixed.sum() == int(budget)


def test_offline_configuration_from_samples():
    rng = np.random.default_rng(22)
    K, L, N = 10, 6, 50
    base = rng.integers(2, N, L)
    lens = np.clip(base[None] + rng.integers(-2, 3, (K, L)), 1, N)
    budget = L * N // 3
    cfg, st = oracle.estimate_config(lens, budget, N)
    assert st == oracle.OK and cfg.sum() == budget and (cfg >= 1).all() and (cfg <= N).all()
    assert list(cfg) == _hamilton((lens - 1).sum(axis=0), budget, N)
    # identical samples: the configuration is the rescaled single-sample one
    one, _ = oracle.rescale(lens[0], budget, N) if lens[0].sum() <= budget else (None, None)
    rep, _ = oracle.estimate_config(np.tile(lens[0], (K, 1)), budget, N)
    assert list(rep) == _hamilton(lens[0] - 1, budget, N)
    # layers that keep more rows in the samples keep more rows in the configuration
    order = np.argsort((lens - 1).sum(axis=0))
    assert (np.diff(cfg[order]) >= 0).all()
    # all samples at one row per layer: the budget is spread evenly
    flat, _ = oracle.estimate_config(np.ones((3, 4), np.int64), 10, 20)
    assert sorted(flat.tolist()) == [2, 2, 3, 3] and flat.sum() == 10


# --------------------------------------------------------------------------
# Keeping the proportions while decoding (Sec. 3.1, Fig. 2a)
# --------------------------------------------------------------------------
def _token_list_model(len0, N, d, steps):
    """Independent model: the cache as a list of tokens ('p', i) / ('g', i)."""
    cache = [("p", i) for i in range(len0)]
    sizes = []
    for g in range(steps):
        target = (len0 * (N + g + 1)) // N
        victim = ("g", g - d)
        if d > 0 and len(cache) + 1 > target and g >= d and victim in cache:
            cache[cache.index(victim)] = ("g", g)          # the new row takes the dropped row's slot
        else:
            cache.append(("g", g))
        sizes.append(len(cache))
    return cache, sizes


@pytest.mark.parametrize("len0,N,d", [(13, 64, 4), (50, 64, 3), (1, 40, 1), (64, 64, 5), (20, 100, 8), (7, 64, 0)])
def test_decode_time_pruning_rule(len0, N, d):
    steps = 120
    ring = np.full(d + 1, -1, np.int32)
    rows = [("p", i) for i in range(len0)]
    n = len0
    for g in range(steps):
        dst, ev, n_after = oracle.decode_slot(len0, N, g, n, d, ring)
        if ev:
            assert rows[dst] == ("g", g - d) and n_after == n
            rows[dst] = ("g", g)
        else:
            assert dst == n and n_after == n + 1
            rows.append(("g", g))
        n = n_after
        # proportion kept: never more than the layer's share plus the d tokens not yet prunable
        assert d == 0 or n <= (len0 * (N + g + 1)) // N + d
        assert all(("g", i) in rows for i in range(max(0, g - d + 1), g + 1)) or d == 0   # recent window
        assert all(("p", i) in rows for i in range(len0))                                  # prompt rows stay
    ref_rows, ref_sizes = _token_list_model(len0, N, d, steps)
    assert rows == ref_rows and n == ref_sizes[-1]
    if d == 0 or len0 == N:
        assert n == len0 + steps                                                            # nothing dropped
    else:
        assert n < len0 + steps


# --------------------------------------------------------------------------
# Cache merging (Sec. 4.3, "Eviction or merging")
# --------------------------------------------------------------------------
def test_merge_position_hand_example():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "merge_position_hand_example.txt"))
            if ln.strip() and not ln.startswith("#")]
    N = int(rows[0][0])
    kept = np.array([int(x) for x in rows[1]], np.int32)
    want_match = [int(x) for x in rows[2]]
    want_rows = [float(x) for x in rows[3]]
    src = np.arange(N, dtype=np.float32)[None, :, None] * np.ones((2, 1, 3), np.float32)   # k[h, p, :] = p
    match = oracle.merge_match(src, kept, oracle.MERGE_POSITION)
    assert match[0].tolist() == want_match and match[1].tolist() == want_match
    merged = oracle.merge_rows(src, kept, match)
    np.testing.assert_allclose(merged[:, 0, 0], want_rows, rtol=0, atol=1e-12)
    np.testing.assert_allclose(merged[:, 1, 2], want_rows, rtol=0, atol=1e-12)


def test_merge_feature_special_cases_and_library():
    rng = np.random.default_rng(31)
    H, N, D = 3, 40, 8
    # one-hot keys: a pruned key merges into the retained key with the same hot index
    hot = rng.integers(0, D, (H, N))
    k = np.zeros((H, N, D), np.float32)
    for h in range(H):
        k[h, np.arange(N), hot[h]] = rng.uniform(0.5, 2.0, N).astype(np.float32)
    kept = np.sort(rng.choice(N, 14, replace=False)).astype(np.int32)
    match = oracle.merge_match(k, kept, oracle.MERGE_FEATURE)
    for h in range(H):
        for m in range(N):
            same = [r for r, n in enumerate(kept) if hot[h, n] == hot[h, m]]
            if m in kept:
                assert kept[match[h, m]] == m
            elif same:
                assert match[h, m] == same[0]              # the lowest position among equal cosines (all 1)
            else:
                assert match[h, m] == 0                    # every cosine is 0: the lowest retained position
    # random keys: a normalised matrix product and argmax from the library
    k = rng.standard_normal((H, N, D)).astype(np.float32)
    v = rng.standard_normal((H, N, D)).astype(np.float32)
    match, gap = oracle.merge_match(k, kept, oracle.MERGE_FEATURE, want_gap=True)
    kn = k.astype(np.float64) / np.linalg.norm(k.astype(np.float64), axis=-1, keepdims=True)
    cos = np.einsum("hmd,hnd->hmn", kn, kn[:, kept])
    pruned = np.setdiff1d(np.arange(N), kept)
    np.testing.assert_array_equal(match[:, pruned], cos.argmax(axis=-1)[:, pruned])
    top2 = np.sort(cos, axis=-1)[:, :, -2:]
    np.testing.assert_allclose(gap[:, pruned], (top2[..., 1] - top2[..., 0])[:, pruned], atol=1e-12)
    # merged rows: scatter-add with numpy, and the total is preserved
    merged = oracle.merge_rows(v, kept, match)
    acc = np.zeros((len(kept), H, D))
    cnt = np.zeros((len(kept), H))
    for h in range(H):
        np.add.at(acc[:, h], match[h], v[h].astype(np.float64))
        np.add.at(cnt[:, h], match[h], 1.0)
    np.testing.assert_allclose(merged, acc / cnt[..., None], rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose((merged * cnt[..., None]).sum(axis=0), v.astype(np.float64).sum(axis=1), rtol=1e-12)
    # nothing pruned: merging is plain compaction
    full = np.arange(N, dtype=np.int32)
    for mode in (oracle.MERGE_POSITION, oracle.MERGE_FEATURE):
        m_all = oracle.merge_match(k, full, mode)
        assert (m_all == np.arange(N)[None]).all()
        np.testing.assert_array_equal(oracle.merge_rows(v, full, m_all), oracle.gather_rows(v, full).astype(np.float64))
    # Position: nearest retained position, the lower one at equal distance, the same in every head
    mp = oracle.merge_match(k, kept, oracle.MERGE_POSITION)
    for m in range(N):
        d = np.abs(kept.astype(np.int64) - m)
        assert (mp[:, m] == int(np.argmin(d))).all()       # argmin takes the first (lowest) of equals
