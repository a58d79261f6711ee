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
    assert sta.status.cpu().tolist() == [0] * w.B
    # the appended rows landed in the cache exactly as with the workspace call
    for seg in range(w.B * w.L):
        o, n = int(ref.cache.row_offset[seg]), int(ref.cache.len[seg])
        a = sta.cache.k[o:o + n].contiguous().view(torch.uint8)
        b = ref.cache.k[o:o + n].contiguous().view(torch.uint8)
        assert torch.equal(a, b)


def test_static_scratch_decode_refuses_large_shapes():
    from paper_2412_03409_b200 import api
    big = api.make_shape(16, 32, 32, 128, 640, torch.bfloat16)
    assert api.prefixkv_workspace_bytes(big, api.WS_DECODE) > api.prefixkv_decode_static_limit_bytes()
    cache = api.CacheStruct(16, 16, 16, 16, 16, 10, 1, 0, None, None, None)
    rc = api.lib().prefixkv_decode_attn_static(big, cache, 16, 16, 16, 16, 0, 32, 16, 16, None)
    assert rc == api.PKV_ERR_STATIC_LIMIT
    assert b"16 MiB" in api.lib().prefixkv_last_cuda_error()
