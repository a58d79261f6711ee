"""CUDA library vs CPU oracle, stage by stage, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_scores, oracle_scores, oracle_select, to_np32
from paper_2412_03409_b200 import workloads as wl

pytestmark = pytest.mark.gpu

SCORE_TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-3}     # relative
DECODE_TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}    # max abs


@pytest.fixture(scope="module")
def api():
    from paper_2412_03409_b200 import api as _api
    return _api


def _session(*a, **kw):
    from paper_2412_03409_b200.session import Session
    return Session(*a, **kw)


def _u64(t):
    return t.cpu().numpy().view(np.uint64)


# --------------------------------------------------------------------------
# selection: bit-exact on the oracle's own fp32 scores
# --------------------------------------------------------------------------
@pytest.mark.parametrize("B,L,N,ratio,tol", [
    (1, 4, 128, 0.5, 1e-6), (2, 5, 1, 1.0, 1e-6), (3, 7, 33, 0.3, 0.0), (2, 32, 640, 0.2, 1e-6),
    (1, 40, 2048, 0.2, 1e-6), (2, 3, 1000, 0.1, 0.0), (1, 6, 16384, 0.05, 1e-6), (1, 2, 5000, 0.7, 1e-9),
])
def test_selection_bit_exact(api, B, L, N, ratio, tol):
    scores = np.stack([wl.synthetic_scores(L, N, seed=17 * b + N) for b in range(B)])
    budgets = [max(L, int(ratio * L * N) + 3 * b) for b in range(B)]
    iters = 64 if tol > 0 else 2000
    s = _session(B, L, 4, 64, N, torch.float32, np.ones(L), decode_cap=1)
    s.search(torch.tensor(budgets), tol=tol, max_iters=iters, scores=torch.from_numpy(scores).cuda())
    torch.cuda.synchronize()
    ref = oracle_select(scores, budgets, tol, iters)
    assert s.status.cpu().tolist() == [0] * B
    for b, (order, cum, res) in enumerate(ref):
        np.testing.assert_array_equal(s.order[b].cpu().numpy(), order)
        np.testing.assert_array_equal(_u64(s.cum[b]), cum)
        np.testing.assert_array_equal(s.len[b].cpu().numpy(), res.len)
        assert s.p[b].item() == res.p
        assert s.iters[b].item() == res.iters
        assert int(s.len[b].sum()) <= budgets[b]


def test_selection_slack_and_iteration_cap(api):
    L, N = 8, 300
    scores = wl.synthetic_scores(L, N, seed=5)[None]
    for tol, iters, slack in [(0.0, 5, 0), (0.0, 2000, 7), (1e-3, 64, 0), (0.0, 0, 0)]:
        s = _session(1, L, 4, 64, N, torch.float32, np.ones(L), decode_cap=1)
        s.search(L * N // 3, tol=tol, max_iters=iters, slack_rows=slack,
                 scores=torch.from_numpy(scores).cuda())
        _, _, res = oracle_select(scores, [L * N // 3], tol, iters, slack)[0]
        np.testing.assert_array_equal(s.len[0].cpu().numpy(), res.len)
        assert s.p[0].item() == res.p and s.iters[0].item() == res.iters


@pytest.mark.parametrize("B,L,N", [(3, 8, 300), (2, 32, 640)])
def test_selection_two_sided_threshold_then_rescale(api, B, L, N):
    """Sec. 3.3: the search ends once |delta| is within a threshold (per side here), possibly above
    the budget; prefixkv_rescale then meets the budget exactly.  Both bit for bit against the oracle."""
    scores = np.stack([wl.synthetic_scores(L, N, seed=b + 40) for b in range(B)])
    budgets = [L * N // 3 + 11 * b for b in range(B)]
    over_seen = False
    for under, over in [(0, 3), (5, 5), (0, 25), (40, 40), (L * N, L * N)]:
        s = _session(B, L, 4, 64, N, torch.float32, np.ones(L), decode_cap=1)
        s.search(torch.tensor(budgets), tol=0.0, max_iters=2000, slack_rows=under, slack_over_rows=over,
                 scores=torch.from_numpy(scores).cuda())
        searched = s.len.cpu().numpy().copy()
        api.prefixkv_rescale(s.shape, s.len, s.budget, s.status)
        fixed = s.len.cpu().numpy()
        for b in range(B):
            _, _, res = oracle.select_sample(scores[b], budgets[b], 0.0, 2000, under, over)
            np.testing.assert_array_equal(searched[b], res.len)
            assert s.p[b].item() == res.p and s.iters[b].item() == res.iters
            assert -under <= int(res.len.sum()) - budgets[b] <= over or res.iters > 30
            ref, st = oracle.rescale(res.len, budgets[b], N)
            assert st == oracle.OK
            np.testing.assert_array_equal(fixed[b], ref)
            assert fixed[b].sum() == budgets[b] and (fixed[b] >= 1).all()
            if res.len.sum() > budgets[b]:
                over_seen = True
                assert (fixed[b] <= res.len).all()
        assert s.status.cpu().tolist() == [0] * B
    assert over_seen                                  # some search did end above its budget


def test_rescale_with_full_layers(api):
    """Budgets close to L * N: layers reach all N rows and what they cannot take goes round to the
    others (many rounds for the kernel's bulk hand-out to reproduce)."""
    rng = np.random.default_rng(8)
    B, L, N = 8, 40, 64
    lens = rng.integers(1, N + 1, (B, L)).astype(np.int32)
    lens[0] = 1                                          # all weights zero
    lens[1, :35] = N                                     # most layers already full
    budgets = np.array([L * N - 3, L * N - 40, L * N, L * N + 9, L * N // 2, L, L + 1, L * N - 700])
    s = _session(B, L, 4, 64, N, torch.float32, np.ones(L), decode_cap=1)
    s.len.copy_(torch.from_numpy(lens))
    s.budget.copy_(torch.from_numpy(budgets))
    s.status.zero_()
    api.prefixkv_rescale(s.shape, s.len, s.budget, s.status)
    got = s.len.cpu().numpy()
    for b in range(B):
        ref, st = oracle.rescale(lens[b], int(budgets[b]), N)
        assert st == oracle.OK
        np.testing.assert_array_equal(got[b], ref)
        assert got[b].sum() == min(int(budgets[b]), L * N)
    assert s.status.cpu().tolist() == [0] * B


def test_selection_degenerate_cases(api):
    L, N = 4, 64
    scores = wl.synthetic_scores(L, N, seed=9)
    batch = np.stack([scores, scores, scores, scores])
    bad = batch.copy()
    bad[2, 1, 5] = np.nan
    bad[3, 0, 0] = -1.0
    s = _session(4, L, 4, 64, N, torch.float32, np.ones(L), decode_cap=1)
    # full budget, minimal budget, NaN, negative
    s.search(torch.tensor([L * N, L, L * N // 2, L * N // 2]), scores=torch.from_numpy(bad).cuda())
    st = s.status.cpu().tolist()
    assert st == [api.DEV_OK, api.DEV_OK, api.DEV_BAD_SCORE, api.DEV_BAD_SCORE]
    assert s.p[0].item() == 1.0 and bool((s.len[0] == N).all()) and s.iters[0].item() == 0
    ref = oracle_select(batch[:2], [L * N, L])
    np.testing.assert_array_equal(s.len[1].cpu().numpy(), ref[1][2].len)
    assert bool((s.len[1] == 1).all())
    # below one row per layer
    s.search(torch.tensor([L - 1, L * 3, L * 3, L * 3]), scores=torch.from_numpy(batch).cuda())
    assert s.status.cpu().tolist() == [api.DEV_BUDGET_TOO_SMALL, 0, 0, 0]
    # ties and signed zeros: position decides
    z = np.zeros((1, 1, 40), np.float32)
    z[0, 0, ::3] = -0.0
    z[0, 0, 7] = 2.0
    z[0, 0, 30] = 2.0
    s1 = _session(1, 1, 4, 64, 40, torch.float32, np.ones(1), decode_cap=1)
    s1.search(10, scores=torch.from_numpy(z).cuda())
    np.testing.assert_array_equal(s1.order[0, 0].cpu().numpy(), oracle.sort_desc(z[0, 0]))
    # fixed-point range
    big = np.full((1, 1, 40), 2.0 ** 21, np.float32)
    s1.search(10, scores=torch.from_numpy(big).cuda())
    assert s1.status.item() == api.DEV_RANGE
    _, st_ref = oracle.cumulative(big[0, 0], oracle.sort_desc(big[0, 0]))
    assert st_ref == oracle.RANGE


def test_apply_given_lengths(api):
    B, L, N = 2, 6, 200
    scores = np.stack([wl.synthetic_scores(L, N, seed=b) for b in range(B)])
    s = _session(B, L, 4, 64, N, torch.float32, np.ones(L), decode_cap=1)
    dev_scores = torch.from_numpy(scores).cuda()
    uniform = torch.full((L,), int(0.25 * N), dtype=torch.int32)          # R_l = r for every layer
    s.apply_lengths(uniform, scores=dev_scores)
    assert s.status.cpu().tolist() == [0, 0]
    assert bool((s.len.cpu() == int(0.25 * N)).all())
    for b in range(B):
        for l in range(L):
            np.testing.assert_array_equal(s.order[b, l].cpu().numpy(), oracle.sort_desc(scores[b, l]))
    per = torch.randint(1, N + 1, (B, L), dtype=torch.int32)
    s.apply_lengths(per, scores=dev_scores)
    np.testing.assert_array_equal(s.len.cpu().numpy(), per.numpy())
    assert oracle.check_lengths(per[0].numpy(), N) == oracle.OK
    per[1, 2] = N + 1
    s.apply_lengths(per, scores=dev_scores)
    assert s.status.cpu().tolist() == [0, api.DEV_BAD_LENGTH]
    assert oracle.check_lengths(per[1].numpy(), N) == oracle.BAD_LENGTH


# --------------------------------------------------------------------------
# compaction: byte-exact rows, untouched head-room
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,H,D,N", [(torch.float32, 4, 64, 128), (torch.bfloat16, 8, 128, 333),
                                         (torch.bfloat16, 3, 64, 70), (torch.float32, 2, 128, 50)])
def test_compact_rows_and_offsets(api, dtype, H, D, N):
    B, L, cap = 2, 3, 4
    w = wl.scaled(wl.WORKLOADS["tiny"], B=B, L=L, H=H, D=D, N=N, dtype=dtype, seed=31)
    q, k, v = wl.make_prompt(w, "cuda")
    scores = np.stack([wl.synthetic_scores(L, N, seed=b + 50) for b in range(B)])
    budgets = [L * N // 3, L * N // 2]
    s = _session(B, L, H, D, N, dtype, np.ones(L), decode_cap=cap, poison=True)
    s.search(torch.tensor(budgets), scores=torch.from_numpy(scores).cuda())
    s.compact(k, v)
    torch.cuda.synchronize()
    assert s.status.cpu().tolist() == [0, 0]
    ref = oracle_select(scores, budgets)
    lens = np.concatenate([r[2].len for r in ref])
    np.testing.assert_array_equal(s.cache.len.cpu().numpy(), lens)
    np.testing.assert_array_equal(s.cache.cap.cpu().numpy(), lens + cap)
    offs = np.concatenate([[0], np.cumsum(lens + cap)])
    np.testing.assert_array_equal(s.cache.row_offset.cpu().numpy(), offs)
    ck, cv = to_np32(s.cache.k), to_np32(s.cache.v)
    for b in range(B):
        for l in range(L):
            seg = b * L + l
            kept = oracle.retained_positions(ref[b][0][l], lens[seg])
            np.testing.assert_array_equal(s.kept[b, l, :lens[seg]].cpu().numpy(), kept)
            rk = oracle.gather_rows(to_np32(k[b, l]), kept)
            rv = oracle.gather_rows(to_np32(v[b, l]), kept)
            np.testing.assert_array_equal(ck[offs[seg]:offs[seg] + lens[seg]], rk)
            np.testing.assert_array_equal(cv[offs[seg]:offs[seg] + lens[seg]], rv)
            assert np.isnan(ck[offs[seg] + lens[seg]:offs[seg + 1]]).all()     # head-room untouched
    assert np.isnan(ck[offs[-1]:]).all()


def test_compact_strided_source_and_capacity(api):
    B, L, H, D, N = 1, 2, 4, 64, 96
    w = wl.scaled(wl.WORKLOADS["tiny"], B=B, L=L, H=H, D=D, N=N, dtype=torch.bfloat16, seed=3)
    q, k, v = wl.make_prompt(w, "cuda")
    # token-major storage [B, L, N, H, D] viewed as [B, L, H, N, D]
    k_tm = k.permute(0, 1, 3, 2, 4).contiguous().permute(0, 1, 3, 2, 4)
    v_tm = v.permute(0, 1, 3, 2, 4).contiguous().permute(0, 1, 3, 2, 4)
    scores = wl.synthetic_scores(L, N, seed=8)[None]
    s = _session(B, L, H, D, N, torch.bfloat16, np.ones(L), decode_cap=2)
    s.search(N, scores=torch.from_numpy(scores).cuda())
    s.compact(k_tm, v_tm)
    a_k, a_len = s.cache.k.clone(), s.cache.len.clone()
    s.compact(k, v)
    assert torch.equal(a_len, s.cache.len)
    for seg in range(L):
        o, n = int(s.cache.row_offset[seg]), int(s.cache.len[seg])
        assert torch.equal(a_k[o:o + n].view(torch.int16), s.cache.k[o:o + n].view(torch.int16))
    # a cache too small for the request is reported, not overrun
    small = _session(B, L, H, D, N, torch.bfloat16, np.ones(L), decode_cap=2, max_budget_rows=10,
                     poison=True)
    small.search(N, scores=torch.from_numpy(scores).cuda())
    small.compact(k, v)
    assert small.status.item() == api.DEV_CAPACITY


# --------------------------------------------------------------------------
# decode attention
# --------------------------------------------------------------------------
def _decode_reference(w, s, k, v, ref_sel, steps, layer_scale):
    """Oracle caches per segment, grown step by step; returns the worst |error|."""
    caches = {}
    for b in range(w.B):
        order, _, res = ref_sel[b]
        for l in range(w.L):
            kept = oracle.retained_positions(order[l], res.len[l])
            caches[(b, l)] = [oracle.gather_rows(to_np32(k[b, l]), kept),
                              oracle.gather_rows(to_np32(v[b, l]), kept)]
    worst = 0.0
    for t in range(steps):
        qd, kn, vn = wl.make_decode_inputs(w, t, "cuda")
        out = s.decode(qd, kn, vn)
        torch.cuda.synchronize()
        got = to_np32(out)
        for (b, l), (ck, cv) in caches.items():
            ck = np.concatenate([ck, to_np32(kn[b, l])[None]])
            cv = np.concatenate([cv, to_np32(vn[b, l])[None]])
            caches[(b, l)] = [ck, cv]
            ref = oracle.decode_attn(to_np32(qd[b, l]), ck, cv, float(layer_scale[l]))
            assert np.isfinite(got[b, l]).all()
            worst = max(worst, float(np.abs(got[b, l] - ref).max()))
    return worst


@pytest.mark.parametrize("name,kw", [
    ("tiny", {}),
    ("llava7b_b1", dict(L=3, H=8, N=200, T=5)),
    ("llava7b_b16", dict(B=3, L=2, H=4, N=97, T=4)),
    ("tiny", dict(D=128, H=2, T=3)),
    ("llava7b_b1", dict(L=2, H=5, D=64, N=130, T=3)),
    ("tiny", dict(D=128, H=32, L=2, N=100, T=3)),           # fp32 rows of 16 KiB: four-row units
    ("llava7b_b1", dict(L=2, H=64, N=90, T=2)),              # 64 heads: four heads per consumer warp
    ("llava7b_b1", dict(L=2, H=72, D=64, N=90, T=2)),        # more heads than the streaming kernel takes: two-kernel path
    ("llava7b_b16", dict(B=40, L=32, H=2, D=64, N=24, T=2)),  # 1280 segments: two layer chunks through the streaming kernel
    # few segments, many (segment, head) items: the per-head kernel (whole softmax rows per CTA)
    ("llava7b_b1", dict(L=20, H=32, N=100, T=3)),            # bf16, 256-byte head slices
    ("tiny", dict(L=16, H=40, N=70, T=3)),                   # fp32, D = 64
    ("tiny", dict(B=2, L=10, H=32, D=128, N=50, T=2)),       # fp32, D = 128: 512-byte slices, one row per warp step
    ("llava7b_b1", dict(L=10, H=64, D=64, N=150, T=2)),      # bf16, D = 64: 128-byte slices, four rows per warp step
    ("llava7b_b1", dict(L=20, H=32, N=700, T=2, budget_ratios=(1.0,))),   # 22 tiles per item: more than consumer warps
    ("llava7b_b1", dict(L=24, H=27, N=100, T=2)),            # odd head count
    ("llava7b_b1", dict(L=24, H=40, D=64, N=100, T=2)),      # bf16, D = 64, 40 heads
    ("llava7b_b1", dict(L=37, H=18, N=100, T=2)),            # 666 items over 148 CTAs: four or five each
    ("llava7b_b1", dict(B=4, L=32, H=8, N=60, T=2)),         # 128 segments (several samples) on the per-head kernel
])
def test_decode_matches_oracle(api, name, kw):
    w = wl.scaled(wl.WORKLOADS[name], **kw)
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    scores = np.stack([wl.synthetic_scores(w.L, w.N, seed=b + 7) for b in range(w.B)])
    budgets = [w.budget_rows()] * w.B
    s = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=w.T)
    s.search(torch.tensor(budgets), scores=torch.from_numpy(scores).cuda())
    s.compact(k, v)
    ref_sel = oracle_select(scores, budgets)
    len0 = s.cache.len.clone()
    worst = _decode_reference(w, s, k, v, ref_sel, w.T, scale)
    assert worst <= DECODE_TOL[w.dtype], worst
    assert torch.equal(s.cache.len, len0 + w.T)
    assert s.status.cpu().tolist() == [0] * w.B
    # one more step than the head-room allows: reported, length unchanged
    qd, kn, vn = wl.make_decode_inputs(w, w.T, "cuda")
    s.decode(qd, kn, vn)
    assert s.status.cpu().tolist() == [api.DEV_CAPACITY] * w.B
    assert torch.equal(s.cache.len, len0 + w.T)


def test_decode_full_budget_is_dense_attention(api):
    """p = 1 keeps every row, so the ragged path must equal dense attention over
    the original K, V plus the appended row (library reference on the host)."""
    w = wl.scaled(wl.WORKLOADS["llava7b_b1"], L=2, H=4, N=150, T=1)
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    s = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=1)
    s.search(w.L * w.N, scores=torch.from_numpy(wl.synthetic_scores(w.L, w.N, 1)[None]).cuda())
    s.compact(k, v)
    assert s.p.item() == 1.0
    qd, kn, vn = wl.make_decode_inputs(w, 0, "cuda")
    out = s.decode(qd, kn, vn).double().cpu()
    for l in range(w.L):
        kk = torch.cat([k[0, l], kn[0, l][:, None]], dim=1).double().cpu()
        vv = torch.cat([v[0, l], vn[0, l][:, None]], dim=1).double().cpu()
        ref = torch.nn.functional.scaled_dot_product_attention(
            qd[0, l].double().cpu()[:, None], kk, vv, scale=float(scale[l]))[:, 0]
        assert (out[0, l] - ref).abs().max() <= DECODE_TOL[w.dtype]


@pytest.mark.parametrize("kw,step", [
    (dict(L=4, H=4, N=80, T=2), 1),                 # a model calls one layer at a time (streaming kernel)
    (dict(B=2, L=20, H=32, N=70, T=2), 10),         # two samples, ten layers per call: the per-head kernel on a sub-range
])
def test_decode_layer_range(api, kw, step):
    w = wl.scaled(wl.WORKLOADS["llava7b_b1"], **kw)
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    scores = torch.from_numpy(np.stack([wl.synthetic_scores(w.L, w.N, 4 + b) for b in range(w.B)])).cuda()
    a = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=2)
    b = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=2)
    for s in (a, b):
        s.search(w.budget_rows(), scores=scores)
        s.compact(k, v)
    qd, kn, vn = wl.make_decode_inputs(w, 0, "cuda")
    full = a.decode(qd, kn, vn).float().clone()
    b.out.zero_()
    for l in range(0, w.L, step):
        b.decode(qd, kn, vn, layer_begin=l, layer_end=l + step)
    assert (full - b.out.float()).abs().max() <= DECODE_TOL[w.dtype]
    assert torch.equal(a.cache.len, b.cache.len)


@pytest.mark.parametrize("kw", [dict(L=6, H=8, N=300, T=5),        # streaming kernel + merge kernel
                                dict(L=20, H=32, N=100, T=5)])     # per-head kernel
def test_decode_replayed_from_a_cuda_graph(api, kw):
    """One decode call captured in a CUDA graph and replayed token after token gives, bit for bit,
    what separate calls give: nothing a call leaves behind (lengths, workspace flags) may depend
    on its being launched afresh."""
    w = wl.scaled(wl.WORKLOADS["llava7b_b1"], **kw)
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    scores = torch.from_numpy(wl.synthetic_scores(w.L, w.N, 9)[None]).cuda()
    a, b, warm = (_session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=w.T) for _ in range(3))
    for s in (a, b, warm):
        s.search(w.budget_rows(), scores=scores)
        s.compact(k, v)
    sq, sk, sv = (t.clone() for t in wl.make_decode_inputs(w, 0, "cuda"))
    warm.decode(sq, sk, sv)                   # one-off set-up of the kernels happens outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        b.decode(sq, sk, sv)
    for t in range(w.T):
        qd, kn, vn = wl.make_decode_inputs(w, t, "cuda")
        sq.copy_(qd); sk.copy_(kn); sv.copy_(vn)
        graph.replay()
        ref = a.decode(qd, kn, vn)
        torch.cuda.synchronize()
        assert torch.equal(b.out, ref), t
        assert torch.equal(a.cache.len, b.cache.len), t
    assert int(b.status.max()) == 0


@pytest.mark.parametrize("kw", [dict(L=6, H=8, N=300, T=2),        # streaming kernel + merge kernel
                                dict(L=20, H=32, N=120, T=2)])     # per-head kernel (its flags live in the workspace)
@pytest.mark.parametrize("byte", [0x7f, 0xff, 0x00])
def test_decode_with_stale_workspace(api, byte, kw):
    """The decode workspace may hold anything (another shape's partials, an earlier call's plan):
    results do not depend on it.  (The merge kernel looks at its plan record early, before the record
    is final, and must bound what it does with that copy.)"""
    w = wl.scaled(wl.WORKLOADS["llava7b_b1"], **kw)
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    scores = torch.from_numpy(wl.synthetic_scores(w.L, w.N, 5)[None]).cuda()
    a = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=2)
    b = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=2)
    for s in (a, b):
        s.search(w.budget_rows(), scores=scores)
        s.compact(k, v)
    b.ws_decode.fill_(byte)
    for t in range(w.T):
        qd, kn, vn = wl.make_decode_inputs(w, t, "cuda")
        ref = a.decode(qd, kn, vn).clone()
        got = b.decode(qd, kn, vn)
        torch.cuda.synchronize()
        assert torch.equal(got, ref)
        b.ws_decode[: 4096].fill_(byte)            # and again over the plan records of the call just made
    assert torch.equal(a.cache.len, b.cache.len)
    assert a.status.cpu().tolist() == b.status.cpu().tolist() == [0]


@pytest.mark.parametrize("kw", [dict(H=4), dict(H=72, D=64),       # streaming kernel; two-kernel path (H > 64)
                                dict(H=32, L=10)])                 # per-head kernel
def test_decode_empty_segment_is_reported(api, kw):
    """A segment with no rows (never compacted) cannot be attended over: the sample's status says
    so, its output is zero, its length stays, and the other segments are unaffected."""
    w = wl.scaled(wl.WORKLOADS["llava7b_b16"], **{**dict(B=2, L=3, N=80, T=2), **kw})
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    scores = np.stack([wl.synthetic_scores(w.L, w.N, seed=b + 11) for b in range(w.B)])
    a = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=2)
    b = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=2)
    for s in (a, b):
        s.search(w.budget_rows(), scores=torch.from_numpy(scores).cuda())
        s.compact(k, v)
    empty = 1 * w.L + 2                              # sample 1, layer 2
    b.cache.len[empty] = 0
    qd, kn, vn = wl.make_decode_inputs(w, 0, "cuda")
    ref = a.decode(qd, kn, vn).float().clone()
    got = b.decode(qd, kn, vn).float()
    torch.cuda.synchronize()
    assert b.status.cpu().tolist() == [0, api.DEV_CAPACITY]
    assert int(b.cache.len[empty]) == 0
    assert (got[1, 2] == 0).all()
    mask = torch.ones(w.B, w.L, dtype=torch.bool)
    mask[1, 2] = False
    assert torch.equal(got[mask.cuda()], ref[mask.cuda()])
    assert torch.equal(b.cache.len[mask.flatten().cuda()], a.cache.len[mask.flatten().cuda()])


@pytest.mark.parametrize("name,kw", [
    ("tiny", {}),
    ("llava7b_b1", dict(L=3, H=8, N=200, T=3)),
    ("llava7b_b1", dict(L=20, H=32, N=90, T=3)),            # per-head kernel
])
def test_decode_without_append(api, name, kw):
    """k_new = v_new = NULL: the query attends over the rows already cached and nothing changes."""
    w = wl.scaled(wl.WORKLOADS[name], **kw)
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    scores = np.stack([wl.synthetic_scores(w.L, w.N, seed=b + 3) for b in range(w.B)])
    budgets = [w.budget_rows()] * w.B
    s = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=2)
    s.search(torch.tensor(budgets), scores=torch.from_numpy(scores).cuda())
    s.compact(k, v)
    qd, kn, vn = wl.make_decode_inputs(w, 0, "cuda")
    s.decode(qd, kn, vn)                           # one ordinary step first: the cache now ends in a decoded row
    len1 = s.cache.len.clone()
    ck, cv = s.cache.k.clone(), s.cache.v.clone()
    q2, _, _ = wl.make_decode_inputs(w, 1, "cuda")
    got = to_np32(s.decode(q2, None, None))
    torch.cuda.synchronize()
    bits = lambda t: t.view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32)   # unused rows may hold NaN patterns
    assert torch.equal(s.cache.len, len1)
    assert torch.equal(bits(s.cache.k), bits(ck)) and torch.equal(bits(s.cache.v), bits(cv))
    assert s.status.cpu().tolist() == [0] * w.B
    offs = s.cache.row_offset.cpu().numpy()
    worst = 0.0
    for b in range(w.B):
        for l in range(w.L):
            seg = b * w.L + l
            n, off = int(len1[seg]), int(offs[seg])
            ref = oracle.decode_attn(to_np32(q2[b, l]), to_np32(ck[off:off + n]), to_np32(cv[off:off + n]),
                                     float(scale[l]))
            assert np.isfinite(got[b, l]).all()
            worst = max(worst, float(np.abs(got[b, l] - ref).max()))
    assert worst <= DECODE_TOL[w.dtype], worst
    with pytest.raises(RuntimeError):              # one of the two alone is an argument error
        s.decode(q2, kn, None)


# --------------------------------------------------------------------------
# importance score
# --------------------------------------------------------------------------
@pytest.mark.parametrize("name,kw", [
    ("tiny", {}),
    ("tiny", dict(N=1)),
    ("tiny", dict(N=77, H=3, L=2, D=128)),
    ("llava7b_b1", dict(L=2, H=4, N=200)),
    ("llava7b_b1", dict(L=1, H=2, N=640)),
    ("llava7b_b16", dict(B=2, L=2, H=3, N=129, D=64)),
    ("longctx_b4", dict(B=1, L=2, H=2, N=1000)),
])
def test_score_matches_oracle(api, name, kw):
    w = wl.scaled(wl.WORKLOADS[name], **kw)
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    s = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=1)
    got = s.score(q, k).cpu().numpy()
    ref = oracle_scores(q, k, scale)
    for (b, l), r in ref.items():
        check_scores(got[b, l], r, SCORE_TOL[w.dtype])
        assert abs(got[b, l].astype(np.float64).sum() - w.N) <= 2e-3 * w.N
    # determinism: a second run gives the same bits
    again = s.score(q, k).cpu().numpy()
    np.testing.assert_array_equal(got, again)


@pytest.mark.parametrize("name,kw", [
    ("llava7b_b1", dict(L=2, H=4, N=200)),           # bf16: tensor maps built from the strides
    ("tiny", dict(N=90, H=3, L=2)),                  # fp32: strided loads
])
def test_score_token_major_layout(api, name, kw):
    """Q and K stored [B, L, N, H, D] (one token's heads together, as a model's projections leave
    them) and handed over through element strides: same scores, bit for bit, as the head-major copy."""
    w = wl.scaled(wl.WORKLOADS[name], **kw)
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    s = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=1)
    base = s.score(q, k).clone()
    qt = q.permute(0, 1, 3, 2, 4).contiguous().permute(0, 1, 3, 2, 4)     # same values, token-major storage
    kt = k.permute(0, 1, 3, 2, 4).contiguous().permute(0, 1, 3, 2, 4)
    assert qt.stride(3) == w.H * w.D and qt.stride(2) == w.D and torch.equal(qt, q)
    got = s.score(qt, kt)
    assert torch.equal(got, base)
    ref = oracle_scores(q, k, scale)
    for (b, l), r in ref.items():
        check_scores(got[b, l].cpu().numpy(), r, SCORE_TOL[w.dtype])


@pytest.mark.parametrize("name,kw", [
    ("llava7b_b1", dict(L=2, H=4, N=300)),           # bf16: tensor-core pass 2 on a converted lse
    ("llava7b_b16", dict(B=2, L=1, H=3, N=129, D=64)),
    ("tiny", dict(N=150, H=3, L=2)),                 # fp32: FMA pass 2 with the natural-log lse
    ("tiny", dict(N=70, H=2, L=1, D=128)),
])
def test_score_with_caller_lse(api, name, kw):
    """The log-sum-exp a prefill kernel would have kept is taken from the oracle (fp64, rounded
    once to fp32); the scores computed from it must meet the same bar against the oracle."""
    w = wl.scaled(wl.WORKLOADS[name], **kw)
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    s = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=1)
    lse = np.stack([np.stack([oracle.lse_layer(to_np32(q[b, l]), to_np32(k[b, l]), float(scale[l]))
                              for l in range(w.L)]) for b in range(w.B)])
    lse_dev = torch.from_numpy(lse.astype(np.float32)).cuda()
    s.scores.fill_(float("nan"))
    got = s.score(q, k, lse=lse_dev).cpu().numpy()
    for (b, l), r in oracle_scores(q, k, scale).items():
        check_scores(got[b, l], r, SCORE_TOL[w.dtype])


def test_score_bf16_layout_without_tensor_map(api):
    """A bf16 K that is one prompt shared by both samples (batch stride 0) cannot be described by
    a tensor map, so the call takes the FMA kernels with strided loads: same bar."""
    w = wl.scaled(wl.WORKLOADS["llava7b_b16"], B=2, L=2, H=3, N=100)
    q, k, v = wl.make_prompt(w, "cuda")
    kb = k[:1].expand(2, -1, -1, -1, -1)
    assert kb.stride(0) == 0
    scale = wl.layer_scale(w)
    s = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=1)
    got = s.score(q, kb).cpu().numpy()
    for (b, l), r in oracle_scores(q, kb, scale).items():
        check_scores(got[b, l], r, SCORE_TOL[w.dtype])


# --------------------------------------------------------------------------
# whole path on the tiny configuration, every output against the oracle
# --------------------------------------------------------------------------
def test_whole_path_tiny(api):
    w = wl.WORKLOADS["tiny"]
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    s = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=w.T, poison=True)
    s.compress(q, k, v, w.budget_rows(), tol=w.tol)
    torch.cuda.synchronize()
    ref_scores = oracle_scores(q, k, scale)
    got_scores = s.scores.cpu().numpy()
    for (b, l), r in ref_scores.items():
        check_scores(got_scores[b, l], r, SCORE_TOL[w.dtype])
    # selection is compared on identical fp32 scores: the library's own
    ref_sel = oracle_select(got_scores, [w.budget_rows()], w.tol)
    order, cum, res = ref_sel[0]
    np.testing.assert_array_equal(s.order[0].cpu().numpy(), order)
    np.testing.assert_array_equal(s.len[0].cpu().numpy(), res.len)
    assert s.p.item() == res.p and s.iters.item() == res.iters
    assert int(s.len.sum()) <= w.budget_rows()
    # concentrated layers (larger logit scale) keep fewer rows
    assert s.len[0, 0] > s.len[0, 3]
    worst = _decode_reference(w, s, k, v, ref_sel, w.T, scale)
    assert worst <= DECODE_TOL[w.dtype]


def test_gini_matches_oracle(api):
    B, L, N = 2, 5, 300
    scores = np.stack([wl.synthetic_scores(L, N, seed=b + 70) for b in range(B)])
    s = _session(B, L, 4, 64, N, torch.float32, np.ones(L), decode_cap=1)
    s.search(L * N // 2, scores=torch.from_numpy(scores).cuda())
    g = torch.empty((B, L), dtype=torch.float64, device="cuda")
    api.prefixkv_gini(s.shape, s.cum, g)
    for b in range(B):
        for l in range(L):
            ref = oracle.gini(scores[b, l], oracle.sort_desc(scores[b, l]))
            assert abs(g[b, l].item() - ref) < 1e-6


def test_argument_validation_fails_on_the_host(api):
    s = _session(1, 2, 4, 64, 32, torch.float32, np.ones(2), decode_cap=1)
    bad = api.make_shape(1, 2, 4, 48, 32, torch.float32)       # unsupported head_dim
    # (real buffers of the session, sized for the same B, L, N: a refusal that ever moved behind
    # a launch would fail the assertions below, not touch made-up addresses)
    s.len.fill_(-5)
    s.status.fill_(0)
    p = lambda t: t.data_ptr()
    rc = api.lib().prefixkv_search(bad, p(s.scores), p(s.budget), 0.0, 1, 0, 0, p(s.order), p(s.cum), p(s.len),
                                   p(s.p), p(s.iters), p(s.status), None, 0, None)
    torch.cuda.synchronize()
    assert rc == api.PKV_ERR_UNSUPPORTED
    assert bool((s.len == -5).all()) and int(s.status.abs().sum()) == 0
    long = api.make_shape(1, 2, 4, 64, 16385, torch.float32)
    assert api.prefixkv_workspace_bytes(long, api.WS_SCORE) == 0
    with pytest.raises(api.PrefixKVError):
        api.prefixkv_search(s.shape, None, s.budget, 1e-6, 64, 0, s.order, s.cum, s.len, s.p,
                            s.iters, s.status)
    with pytest.raises(api.PrefixKVError):                      # workspace too small
        api.prefixkv_decode_attn(s.shape, s.cache, s.out, s.out, s.out, s.layer_scale, s.out,
                                 s.status, torch.empty(256, dtype=torch.uint8, device="cuda"))


# --------------------------------------------------------------------------
# exact budget after an inexact search; offline configuration from sample prompts
# --------------------------------------------------------------------------
def test_rescale_and_offline_configuration(api):
    B, L, N = 6, 32, 640
    scores = np.stack([wl.synthetic_scores(L, N, seed=b + 300) for b in range(B)])
    budgets = [L * N // 5 + 7 * b for b in range(B)]
    s = _session(B, L, 4, 64, N, torch.float32, np.ones(L), decode_cap=1)
    # a coarse search (5 midpoints) leaves part of the budget unused
    s.search(torch.tensor(budgets), tol=0.0, max_iters=5, scores=torch.from_numpy(scores).cuda())
    searched = s.len.cpu().numpy().copy()
    assert (searched.sum(axis=1) < np.array(budgets)).any()
    api.prefixkv_rescale(s.shape, s.len, s.budget, s.status)
    got = s.len.cpu().numpy()
    for b in range(B):
        ref, st = oracle.rescale(searched[b], budgets[b], N)
        assert st == oracle.OK
        np.testing.assert_array_equal(got[b], ref)
        assert got[b].sum() == budgets[b] and (got[b] >= searched[b]).all()
    assert s.status.cpu().tolist() == [0] * B
    # one configuration for all inputs from the B sample prompts
    s.search(torch.tensor(budgets), scores=torch.from_numpy(scores).cuda())
    per_sample = s.len.cpu().numpy().copy()
    cfg = torch.zeros(L, dtype=torch.int32, device="cuda")
    api.prefixkv_estimate_config(s.shape, s.len, budgets[0], cfg, s.status)
    ref, st = oracle.estimate_config(per_sample, budgets[0], N)
    assert st == oracle.OK
    np.testing.assert_array_equal(cfg.cpu().numpy(), ref)
    assert int(cfg.sum()) == budgets[0]
    # and it feeds the given-lengths entry point
    s.apply_lengths(cfg.cpu(), scores=torch.from_numpy(scores).cuda())
    assert (s.len.cpu().numpy() == ref[None]).all() and s.status.cpu().tolist() == [0] * B
    # too small a budget is reported
    api.prefixkv_estimate_config(s.shape, s.len, L - 1, cfg, s.status)
    assert s.status[0].item() == api.DEV_BUDGET_TOO_SMALL


# --------------------------------------------------------------------------
# decode-time pruning at a fixed distance (keeps each layer's proportion)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("name,kw,d", [
    ("llava7b_b1", dict(B=2, L=3, H=4, N=96, T=40), 4),
    ("tiny", dict(T=30), 2),
    ("llava7b_b1", dict(L=2, H=8, N=200, T=24), 9),
])
def test_decode_time_pruning_matches_oracle(api, name, kw, d):
    w = wl.scaled(wl.WORKLOADS[name], **kw)
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    scores = np.stack([wl.synthetic_scores(w.L, w.N, seed=b + 40) for b in range(w.B)])
    budgets = [w.budget_rows()] * w.B
    s = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=w.T, evict_distance=d)
    s.search(torch.tensor(budgets), scores=torch.from_numpy(scores).cuda())
    s.compact(k, v)
    ref_sel = oracle_select(scores, budgets)
    state = {}
    for b in range(w.B):
        order, _, res = ref_sel[b]
        for l in range(w.L):
            kept = oracle.retained_positions(order[l], res.len[l])
            state[(b, l)] = dict(k=list(oracle.gather_rows(to_np32(k[b, l]), kept)),
                                 v=list(oracle.gather_rows(to_np32(v[b, l]), kept)),
                                 len0=int(res.len[l]), ring=np.full(d + 1, -1, np.int32))
    dropped = 0
    for g in range(w.T):
        qd, kn, vn = wl.make_decode_inputs(w, g, "cuda")
        got = to_np32(s.decode(qd, kn, vn))
        lens = s.cache.len.cpu().numpy()
        for (b, l), st in state.items():
            dst, ev, n_after = oracle.decode_slot(st["len0"], w.N, g, len(st["k"]), d, st["ring"])
            if ev:
                st["k"][dst], st["v"][dst] = to_np32(kn[b, l]), to_np32(vn[b, l])
                dropped += 1
            else:
                st["k"].append(to_np32(kn[b, l])); st["v"].append(to_np32(vn[b, l]))
            assert lens[b * w.L + l] == n_after == len(st["k"])
            ref = oracle.decode_attn(to_np32(qd[b, l]), np.stack(st["k"]), np.stack(st["v"]), float(scale[l]))
            assert np.isfinite(got[b, l]).all()
            assert np.abs(got[b, l] - ref).max() <= DECODE_TOL[w.dtype]
    assert dropped > 0 and s.status.cpu().tolist() == [0] * w.B
    # the cache holds exactly the oracle's rows, slot for slot
    offs = s.cache.row_offset.cpu().numpy()
    for (b, l), st in state.items():
        o = int(offs[b * w.L + l])
        np.testing.assert_array_equal(to_np32(s.cache.k[o:o + len(st["k"])]), np.stack(st["k"]))
        np.testing.assert_array_equal(to_np32(s.cache.v[o:o + len(st["v"])]), np.stack(st["v"]))
        assert int(s.cache.gen[b * w.L + l]) == w.T


# --------------------------------------------------------------------------
# bounded waits give up and report, without faulting or hanging anything
# --------------------------------------------------------------------------
@pytest.mark.parametrize("which", [0, 1])
def test_bounded_wait_reports_timeout(api, which):
    """A warp waits on a barrier that nothing completes, with a limit of a few thousand tries:
    the wait returns, the status word reads PKV_DEV_TIMEOUT and the context stays usable."""
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    api.prefixkv_selftest_bounded_wait(which, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [api.DEV_TIMEOUT, 0]
    assert int((torch.arange(8, device="cuda") + 1).sum()) == 36      # later work runs normally


# --------------------------------------------------------------------------
# cache merging (Sec. 4.3): pruned vectors averaged into the matched retained ones
# --------------------------------------------------------------------------
@pytest.mark.parametrize("name,kw", [
    ("tiny", dict(N=90, H=3, L=2)),                        # fp32, D = 64
    ("llava7b_b1", dict(L=2, H=4, N=333)),                 # bf16, D = 128, several 32-key tiles and a ragged one
    ("llava7b_b16", dict(B=2, L=2, H=2, N=160, D=64)),
])
@pytest.mark.parametrize("mode", ["position", "feature"])
def test_compact_with_merging_matches_oracle(api, name, kw, mode):
    w = wl.scaled(wl.WORKLOADS[name], **kw)
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    scores = np.stack([wl.synthetic_scores(w.L, w.N, seed=b + 60) for b in range(w.B)])
    s = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=2, poison=True)
    s.search(w.budget_rows(), scores=torch.from_numpy(scores).cuda())
    code = api.MERGE_POSITION if mode == "position" else api.MERGE_FEATURE
    match = torch.full((w.B, w.L, w.H, w.N), -7, dtype=torch.int32, device="cuda")
    s.compact_merge(k, v, code, match=match)
    torch.cuda.synchronize()
    assert s.status.cpu().tolist() == [0] * w.B
    tol = DECODE_TOL[w.dtype]
    # merged rows are averages formed in fp32 and rounded once to the cache type: the error is the
    # rounding of the result (half an ulp: 2^-9 relative for bf16, 2^-24 for fp32) plus the fp32
    # summation of at most N terms; bound with a factor two of margin, relative with a floor of 1
    rel = 2.0 ** -8 if w.dtype == torch.bfloat16 else 1e-5
    for b in range(w.B):
        for l in range(w.L):
            n = int(s.len[b, l])
            kept = oracle.retained_positions(s.order[b, l].cpu().numpy(), n)
            np.testing.assert_array_equal(s.kept[b, l, :n].cpu().numpy(), kept)
            got_match = match[b, l].cpu().numpy()
            ref_match, gap = oracle.merge_match(to_np32(k[b, l]), kept, code, want_gap=True)
            if mode == "position":
                np.testing.assert_array_equal(got_match, ref_match)      # integer decisions: bit-exact
            else:
                # the argmax is decided in fp32 on the GPU and in fp64 by the oracle: they must agree
                # wherever the best and second-best cosine differ by more than fp32 can blur; elsewhere
                # the GPU's choice is one of the near-equal best and the rows are checked under it
                differ = got_match != ref_match
                assert not (differ & (gap > 1e-5)).any()
                assert (got_match >= 0).all() and (got_match < n).all()
            off = int(s.cache.row_offset[b * w.L + l])
            for src, dst in ((k, s.cache.k), (v, s.cache.v)):
                ref = oracle.merge_rows(to_np32(src[b, l]), kept, got_match)
                got = to_np32(dst[off:off + n])
                assert (np.abs(got - ref) <= rel * np.maximum(np.abs(ref), 1.0)).all()
            # the head-room rows are untouched
            assert torch.isnan(s.cache.k[off + n:off + n + 2].float()).all()
    # decoding over the merged cache works like over any other
    qd, kn, vn = wl.make_decode_inputs(w, 0, "cuda")
    out = to_np32(s.decode(qd, kn, vn))
    b, l = w.B - 1, w.L - 1
    off, n = int(s.cache.row_offset[b * w.L + l]), int(s.cache.len[b * w.L + l])
    ref = oracle.decode_attn(to_np32(qd[b, l]), to_np32(s.cache.k[off:off + n]), to_np32(s.cache.v[off:off + n]),
                             float(scale[l]))
    assert np.abs(out[b, l] - ref).max() <= tol


def test_merging_with_nothing_pruned_is_plain_compaction(api):
    w = wl.scaled(wl.WORKLOADS["llava7b_b1"], L=2, H=4, N=100)
    q, k, v = wl.make_prompt(w, "cuda")
    scores = wl.synthetic_scores(w.L, w.N, seed=3)[None]
    a = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, wl.layer_scale(w), decode_cap=1)
    b = _session(w.B, w.L, w.H, w.D, w.N, w.dtype, wl.layer_scale(w), decode_cap=1)
    for s in (a, b):
        s.search(w.L * w.N, scores=torch.from_numpy(scores).cuda())      # full budget: every row kept
    a.compact(k, v)
    b.compact_merge(k, v, api.MERGE_FEATURE)
    torch.cuda.synchronize()
    # (equal as values: an average of one vector is that vector, except that -0.0 comes out as +0.0)
    for seg in range(w.L):
        o = int(a.cache.row_offset[seg])
        assert int(a.cache.len[seg]) == w.N
        assert torch.equal(a.cache.k[o:o + w.N].float(), b.cache.k[o:o + w.N].float())
        assert torch.equal(a.cache.v[o:o + w.N].float(), b.cache.v[o:o + w.N].float())
    assert torch.equal(a.cache.len, b.cache.len) and torch.equal(a.cache.row_offset, b.cache.row_offset)
