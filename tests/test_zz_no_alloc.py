"""The decode entry point that takes no workspace, for callers that cannot
allocate device memory when they decode (their framework already owns all of it,
or an allocation's device-wide synchronisation between tokens is unacceptable).

It must give the same answers as the workspace entry point.  Collected last on
purpose: if it fails under `-x`, every other test has already run.  It builds
its own inputs, so it also passes alone in a fresh process.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_03409_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DECODE_TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}    # max abs, as in test_gpu_parity


def _pair(w):
    """Two sessions with identical caches: one per entry point."""
    from paper_2412_03409_b200.session import Session
    q, k, v = wl.make_prompt(w, "cuda")
    scale = wl.layer_scale(w)
    scores = torch.from_numpy(np.stack([wl.synthetic_scores(w.L, w.N, seed=b + 11)
                                        for b in range(w.B)])).cuda()
    out = []
    for _ in range(2):
        s = Session(w.B, w.L, w.H, w.D, w.N, w.dtype, scale, decode_cap=w.T)
        s.search(w.budget_rows(), scores=scores)
        s.compact(k, v)
        out.append(s)
    return out


@pytest.mark.parametrize("name,kw", [("llava7b_b1", dict(L=3, H=8, N=200, T=3)),
                                     ("tiny", dict(T=3))])
def test_static_scratch_decode_matches_workspace_decode(name, kw):
    from paper_2412_03409_b200 import api
    w = wl.scaled(wl.WORKLOADS[name], **kw)
    assert api.prefixkv_workspace_bytes(api.make_shape(w.B, w.L, w.H, w.D, w.N, w.dtype),
                                        api.WS_DECODE) <= api.prefixkv_decode_static_limit_bytes()
    ref, sta = _pair(w)
    f32 = lambda t: t.detach().float().cpu().numpy()
    scale = wl.layer_scale(w)
    for t in range(2):                                   # two calls in a row share the array
        qd, kn, vn = wl.make_decode_inputs(w, t, "cuda")
        want = ref.decode(qd, kn, vn).float().clone()
        api.prefixkv_decode_attn_static(sta.shape, sta.cache, qd, kn, vn, sta.layer_scale, sta.out,
                                        sta.status)
        torch.cuda.synchronize()
        got = sta.out.float()
        assert torch.isfinite(got).all()
        assert (got - want).abs().max().item() <= DECODE_TOL[w.dtype]
        assert torch.equal(sta.cache.len, ref.cache.len)
        # and against the oracle, over the rows the cache now holds (the new one included)
        for seg in (0, w.B * w.L - 1):
            b, l = divmod(seg, w.L)
            o, n = int(sta.cache.row_offset[seg]), int(sta.cache.len[seg])
            want64 = oracle.decode_attn(f32(qd[b, l]), f32(sta.cache.k[o:o + n]), f32(sta.cache.v[o:o + n]),
                                        float(scale[l]))
            assert np.abs(f32(got[b, l]) - want64).max() <= DECODE_TOL[w.dtype]
    assert sta.status.cpu().tolist() == [0] * w.B
    # the appended rows landed in the cache exactly as with the workspace call
    for seg in range(w.B * w.L):
        o, n = int(ref.cache.row_offset[seg]), int(ref.cache.len[seg])
        a = sta.cache.k[o:o + n].contiguous().view(torch.uint8)
        b = ref.cache.k[o:o + n].contiguous().view(torch.uint8)
        assert torch.equal(a, b)


def test_static_scratch_decode_refuses_large_shapes():
    """A shape whose scratch need is above the built-in array is refused on the host, before any
    launch.  Every pointer handed over is a real (small) device buffer and the cache describes
    exactly those buffers, so that if the refusal ever moved behind a launch this test would fail
    an assertion below instead of sending a kernel to made-up addresses."""
    from paper_2412_03409_b200 import api
    big = api.make_shape(16, 32, 32, 128, 640, torch.bfloat16)
    assert api.prefixkv_workspace_bytes(big, api.WS_DECODE) > api.prefixkv_decode_static_limit_bytes()
    nseg = 16 * 32
    cache = api.alloc_cache(big, total_rows=0, decode_cap=1, device="cuda", fill=0.0)
    assert cache.k.shape[0] == nseg                          # one row of head-room per segment, nothing else
    cache.cap.fill_(1)
    cache.row_offset.copy_(torch.arange(nseg + 1, dtype=torch.int64, device="cuda"))
    x = torch.zeros((16, 32, 32, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.full_like(x, 7.0)
    scale = torch.ones(32, dtype=torch.float32, device="cuda")
    status = torch.zeros(16, dtype=torch.int32, device="cuda")
    p = lambda t: t.data_ptr()
    rc = api.lib().prefixkv_decode_attn_static(big, cache.c, p(x), p(x), p(x), p(scale), 0, 32, p(out),
                                               p(status), None)
    torch.cuda.synchronize()
    assert rc == api.PKV_ERR_STATIC_LIMIT
    assert b"16 MiB" in api.lib().prefixkv_last_cuda_error()
    assert int(cache.len.abs().sum()) == 0 and bool((out == 7.0).all()) and int(status.abs().sum()) == 0
