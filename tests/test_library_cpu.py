"""CPU-side checks of the C-ABI library: it builds, loads, exports every symbol the header
declares, and rejects bad arguments on the host before touching a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2506_08373_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def header_functions():
    text = open(os.path.join(ROOT, "include", "spec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spec\w*)\s*\(", text)))


def test_library_exports_every_declared_symbol(B):
    names = header_functions()
    assert set(names) == set(B.EXPORTS)
    for n in names:
        assert getattr(B.lib(), n) is not None


def test_struct_layout_matches_header(B):
    # 10 int32 + pointer + float + 6 int64, natural alignment
    assert ctypes.sizeof(B.spec_problem) == 104
    assert B.spec_problem.cu_seqlens.offset == 8 and B.spec_problem.k_stride_layer.offset == 56


def good_problem(B, **kw):
    args = dict(n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64, n_lookahead=8, n_window=8,
                softmax_scale=0.125, total_tokens=1024, n_in=1024)
    args.update(kw)
    return B.make_problem(**args)


def test_workspace_size_is_positive_and_zero_on_bad_problem(B):
    assert B.spec_workspace_bytes(good_problem(B)) > 0
    assert B.spec_workspace_bytes(good_problem(B, n_q_heads=7)) == 0
    assert "multiple" in B.spec_last_error()


@pytest.mark.parametrize("kw,code", [
    (dict(n_q_heads=7), -1), (dict(head_dim=96), -3), (dict(n_lookahead=0, n_window=0), -1),
    (dict(n_in=2048), -1), (dict(n_seq=2), -1), (dict(n_layers=0), -1),
])
def test_bad_geometry_is_rejected_on_the_host(B, kw, code):
    pr = good_problem(B, **kw)
    one = ctypes.c_void_p(256)      # non-NULL, aligned, never dereferenced: the call must fail first
    rc = B.lib().spec_score(ctypes.byref(pr), one, one, None, 0, 0, one, one, 1 << 30, None, None)
    assert rc == code and len(B.spec_last_error()) > 0


def test_bad_call_arguments_are_rejected_on_the_host(B):
    pr = good_problem(B)
    L = B.lib()
    one, odd = ctypes.c_void_p(256), ctypes.c_void_p(260)
    assert L.spec_score(ctypes.byref(pr), None, one, None, 0, 0, one, one, 1 << 30, None, None) == B.ERR_BAD_ARG
    assert L.spec_score(ctypes.byref(pr), odd, one, None, 0, 0, one, one, 1 << 30, None, None) == B.ERR_ALIGNMENT
    assert L.spec_score(ctypes.byref(pr), one, one, None, 5, 0, one, one, 1 << 30, None, None) == B.ERR_BAD_ARG
    assert L.spec_score(ctypes.byref(pr), one, one, None, 0, 0, one, one, 8, None, None) == B.ERR_WORKSPACE
    assert L.spec_pool_topk(ctypes.byref(pr), one, 0, 0, 16, 0, one, None, None, 0, None, None) == B.ERR_BAD_ARG
    assert L.spec_pool_topk(ctypes.byref(pr), one, 0, 7, 16, 17, one, None, None, 0, None, None) == B.ERR_BAD_ARG
    assert L.spec_pool_topk(ctypes.byref(pr), one, 3, 7, 16, 0, one, None, None, 0, None, None) == B.ERR_BAD_ARG
    assert L.spec_compact_kv(ctypes.byref(pr), one, None, one, 16, one, one, None, 0, 0, None, None) == B.ERR_BAD_ARG
    assert L.spec_compact_kv(ctypes.byref(pr), odd, None, one, 16, one, None, None, 0, 0, None, None) == B.ERR_ALIGNMENT
    assert L.spec_compact_kv(ctypes.byref(pr), one, None, one, 16, one, None, one, 0, 4, None, None) == B.ERR_BAD_ARG
    # keep_capacity below the worst case min(n, c_max*(2*n_neighbor+1))
    assert L.specpc_token_select(ctypes.byref(pr), one, 0, 0, 7, 16, 8, 0, one, 100, one, one, 1 << 30,
                                 None, None) == B.ERR_BAD_ARG
    assert "keep_capacity" in B.spec_last_error()
    # the two-stage pool of Algorithm 2 is a SpecPC option only, and its keep list is exactly c_max + window
    assert L.spec_pool_topk(ctypes.byref(pr), one, 2, 7, 16, 0, one, None, None, 0, None, None) == B.ERR_BAD_ARG
    assert L.specpc_token_select(ctypes.byref(pr), one, 1, 2, 7, 16, 8, 4, one, 19, one, one, 1 << 30,
                                 None, None) == B.ERR_BAD_ARG
    # ... and the workspace-free variant has no room for its second vector: refused by name, before any launch
    assert L.specpc_token_select_static(ctypes.byref(pr), one, 1, 2, 7, 16, 8, 4, one, 1024, one, None, None) == B.ERR_UNSUPPORTED
    assert "SPEC_POOL_AVG_THEN_MAX" in B.spec_last_error()
    assert L.spec_pool_topk_vert(ctypes.byref(pr), one, 0, 7, 16, 0, one, None, 0, one, None, None, 0, None, None) == B.ERR_BAD_ARG
    assert L.spec_pool_topk_vert(ctypes.byref(pr), one, 0, 7, 16, 0, one, None, 8, None, None, None, 0, None, None) == B.ERR_BAD_ARG
    assert L.spec_score(ctypes.byref(pr), one, one, None, 0, 2, one, one, 1 << 30, None, None) == B.ERR_BAD_ARG
    # prompt compression
    assert L.spec_gather_tokens(ctypes.byref(pr), one, None, None, 16, one, one, None, 64, one, None, None) == B.ERR_BAD_ARG
    assert L.spec_gather_tokens(ctypes.byref(pr), one, one, one, 16, one, one, None, 64, one, None, None) == B.ERR_BAD_ARG
    assert L.spec_gather_tokens(ctypes.byref(pr), one, None, one, 0, one, one, None, 64, one, None, None) == B.ERR_BAD_ARG
    assert L.spec_gather_tokens(ctypes.byref(pr), one, None, one, 16, one, odd, None, 64, one, None, None) == B.ERR_ALIGNMENT


def test_missing_library_fails_loudly(B, monkeypatch):
    from paper_2506_08373_b200 import binding, build
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(build, "LIB_PATH", "/nonexistent/libspec.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()
