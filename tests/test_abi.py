"""The C-ABI library loads, exports every symbol the header declares, and its host-side logic
(argument checks, workspace sizing) works without a GPU."""
import ctypes
import os
import re

import pytest

from paper_2505_20776_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "specext.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(specext_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"specext_verify_attn", "specext_select_chunks", "specext_gather_kv",
            "specext_verify_attn_workspace"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in specext.h but not exported"
    # test hooks and the cross-check kernel's switch live in the test library only
    for n in ("specext_test_set_tuning", "specext_test_wait_timeout", "specext_set_tuning"):
        assert not hasattr(lib, n)


def test_test_library_builds_and_exports_its_hooks():
    from tests.testing_lib import load_testing_lib
    L = load_testing_lib()
    assert hasattr(L, "specext_test_set_tuning") and hasattr(L, "specext_test_wait_timeout")
    assert L.specext_test_set_tuning(7, 0) == 1
    assert L.specext_test_wait_timeout(0, None, None) == 1


def _desc(**kw):
    d = api.AttnDesc()
    d.n_q_heads, d.n_kv_heads, d.head_dim = 32, 8, 128
    d.prefix_len, d.n_tree, d.chunk_size = 16384, 60, 32
    d.softmax_scale, d.want_chunk_score = 0.0, 1
    d.q_stride_t, d.q_stride_h = 32 * 128, 128
    d.kv_stride_l, d.kv_stride_h = 8 * 128, 128
    d.tkv_stride_t, d.tkv_stride_h = 8 * 128, 128
    d.o_stride_t, d.o_stride_h = 32 * 128, 128
    for k, v in kw.items():
        setattr(d, k, v)
    return d


def test_workspace_size_and_descriptor_checks(lib):
    full = api.specext_verify_attn_workspace(_desc())
    assert full > 0 and full % 4 == 0
    without = api.specext_verify_attn_workspace(_desc(want_chunk_score=0))
    assert 0 < without < full
    # the per-chunk sums for [Hq*T rows padded to 256 per KV head][NC] plus one reference maximum per
    # (row, 128-key tile) make up the difference
    assert full - without == 4 * (8 * 128 * 256 * 4 + 8 * 128 * 256)
    for bad in (dict(head_dim=96), dict(n_tree=0), dict(n_tree=129), dict(chunk_size=3), dict(chunk_size=256),
                dict(n_kv_heads=5), dict(prefix_len=-4), dict(q_stride_h=100), dict(kv_stride_l=12),
                dict(softmax_scale=float("nan"))):
        assert api.specext_verify_attn_workspace(_desc(**bad)) == 0
    assert api.specext_verify_attn_workspace(_desc(prefix_len=0)) > 0


def test_host_side_rejection_needs_no_gpu(lib):
    d = _desc(head_dim=96)
    rc = lib.specext_verify_attn(ctypes.byref(d), *([None] * 9), None, 0, None, None)
    assert rc == 2
    d = _desc()
    rc = lib.specext_verify_attn(ctypes.byref(d), *([None] * 9), None, 0, None, None)
    assert rc == 1                                            # null pointers
    assert lib.specext_select_chunks(None, 4, 8, 0, 256, 32, 4, 0, 0, None, None, None, None) == 1
    assert lib.specext_select_gather(None, 4, 8, 0, 256, 32, 4, 0, 0, *([None] * 2), 1, 8, 128, 0, 1024, 128, *([None] * 7)) == 1
    assert lib.specext_status_string(4).decode().startswith("parent")
    assert lib.specext_launch_count() >= 0
