"""Host-only checks of the C ABI: the library loads without a GPU, exports every
function the header declares, sizes workspaces, and rejects bad arguments
before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def api():
    from paper_2412_03409_b200 import build
    build.build_library()
    from paper_2412_03409_b200 import api as _api
    return _api


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "prefixkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(prefixkv_\w+)\s*\(", text)))


def test_header_functions_are_exported(api):
    names = _declared_functions()
    assert len(names) >= 8
    for n in names:
        assert hasattr(api.lib(), n), n
    assert set(api.EXPORTS) <= set(names)
    # the Python binding mirrors every compute entry point by name
    for n in names:
        if n != "prefixkv_last_cuda_error":
            assert hasattr(api, n), n


def test_workspace_sizes(api):
    import torch
    sh = api.make_shape(1, 32, 32, 128, 640, torch.bfloat16)
    per = 32 * 32 * 640 * 4
    assert api.prefixkv_workspace_bytes(sh, api.WS_SCORE) >= 2 * per
    assert api.prefixkv_workspace_bytes(sh, api.WS_COMPACT) >= 32 * 640 * 4
    assert api.prefixkv_workspace_bytes(sh, api.WS_DECODE) > 0
    assert api.prefixkv_workspace_bytes(sh, 99) == 0
    for bad in (api.make_shape(1, 2, 4, 48, 32, torch.float32),       # head_dim
                api.make_shape(1, 2, 4, 64, 16385, torch.float32),    # prompt too long
                api.make_shape(0, 2, 4, 64, 32, torch.float32)):      # empty batch
        assert api.prefixkv_workspace_bytes(bad, api.WS_SCORE) == 0


def test_null_and_range_arguments_rejected_on_host(api):
    import torch
    lib = api.lib()
    sh = api.make_shape(1, 2, 4, 64, 32, torch.float32)
    z = api.Strides(0, 0, 0, 0)
    assert lib.prefixkv_score(sh, None, z, None, z, None, None, None, None, 0, None) == api.PKV_ERR_INVALID_ARG
    assert lib.prefixkv_search(sh, None, None, 1e-6, 64, 0, 0, None, None, None, None, None, None,
                               None, 0, None) == api.PKV_ERR_INVALID_ARG
    if torch.cuda.is_available():
        return      # the cases below pass made-up non-null addresses: only where no launch can reach a GPU
    assert lib.prefixkv_search(sh, 16, 16, -1.0, 64, 0, 0, 16, 16, 16, 16, 16, 16, None, 0, None) == \
        api.PKV_ERR_INVALID_ARG                                    # negative tolerance
    assert lib.prefixkv_apply_lengths(sh, None, None, 0, None, None, None, None, None, 0, None) == \
        api.PKV_ERR_INVALID_ARG
    assert lib.prefixkv_compact(sh, None, z, None, z, None, None, None, None, None, None, 0, None) == \
        api.PKV_ERR_INVALID_ARG
    cache = api.CacheStruct(16, 16, 16, 16, 16, 10, 1, 0, None, None, None)
    assert lib.prefixkv_decode_attn(sh, ctypes.byref(cache), 16, 16, 16, 16, 1, 1, 16, 16, None, 0,
                                    None) == api.PKV_ERR_INVALID_ARG   # empty layer range
    assert lib.prefixkv_decode_attn(sh, ctypes.byref(cache), 16, 16, 16, 16, 0, 2, 16, 16, None, 0,
                                    None) == api.PKV_ERR_WORKSPACE     # no workspace
    odd = api.Strides(7, 7, 7, 7)                                      # rows not on 16 bytes
    assert lib.prefixkv_score(sh, 16, odd, 16, odd, 16, None, 16, 256, 1 << 30, None) == \
        api.PKV_ERR_INVALID_ARG
    assert lib.prefixkv_gini(sh, None, None, None) == api.PKV_ERR_INVALID_ARG
