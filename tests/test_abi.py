"""The C-ABI library builds, loads without a GPU and exports every symbol the
header declares; host-visible argument errors are reported before any launch."""
import ctypes
import os
import re

import pytest

import paper_2603_08088_b200 as tv
from paper_2603_08088_b200 import build as tv_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    tv_build.build()
    return tv.load()


def _declared_symbols(header="treeverify.h"):
    text = open(os.path.join(ROOT, "include", header)).read()
    return re.findall(r"^TV_API\s+[\w\s\*]+?\b(\w+)\(", text, flags=re.M)


def test_header_symbols_are_exported(lib):
    names = _declared_symbols()
    assert set(names) >= {"tree_build_mask", "tree_verify_attn", "tree_accept", "kv_commit",
                          "tv_verify_step_host", "tv_last_error"}
    for n in names:
        assert hasattr(lib, n), f"{n} declared in treeverify.h but not exported"
    assert set(names) == set(tv.EXPORTS)
    debug = _declared_symbols("treeverify_debug.h")            # test and tuning aids: declared apart, exported too
    assert set(debug) == {"tv_debug_attn_simt", "tv_debug_attn_expire", "tv_debug_attn_stream_only",
                          "tv_debug_set_attn_trace"}
    for n in debug:
        assert hasattr(lib, n), f"{n} declared in treeverify_debug.h but not exported"
    assert not set(debug) & set(names)


def test_version_and_size_queries(lib):
    assert tv.tv_version() >= 100
    assert tv.tv_accept_workspace_bytes(16, 60, 153600) >= 16 * 60 * 8
    assert tv.tv_attn_workspace_bytes(16, 60, 32, 8, 128, 4224) >= 256
    assert tv.tv_step_staging_bytes(2, 2, 15, 4, 2, 64, 256, 1024, 8, 5) > 0


def test_null_and_bad_dims_are_rejected_without_a_launch(lib):
    rc = lib.tree_build_mask(None, None, 1, 8, 3, 4, None, None, None, None, None, None, None, None)
    assert rc == 1 and b"NULL" in lib.tv_last_error()
    one = ctypes.c_void_p(0x1000)
    rc = lib.tree_build_mask(one, one, 1, 4096, 3, 4, one, None, None, None, None, None, one, None)
    assert rc == 1 and b"Nmax" in lib.tv_last_error()
    rc = lib.kv_commit(one, one, one, one, one, one, one, 1, 1, 8, 2, 12, 64, 4, 0, 0, one, None)
    assert rc == 1
    rc = lib.tree_accept(one, one, one, one, 1, 8, 100, 2, 3, one, None, None, one, one, one, one, one, 0, one, None)
    assert rc == 3     # workspace too small
    rc = lib.tree_verify_attn(one, one, one, one, one, one, one, one, 1, 300, 4, 2, 64, 64, 1.0, one, None,
                              one, 1 << 30, one, None)
    assert rc == 1     # Nmax > 256


def test_host_step_rejects_bad_dimensions_before_any_copy(lib):
    """tv_verify_step_host checks everything its four calls would refuse before it queues a copy, so an error
    return means the host buffers were never touched (no device is needed to see it: nothing is launched)."""
    from paper_2603_08088_b200.binding import StepHostArgs
    a = StepHostArgs()
    for name, _ in StepHostArgs._fields_:
        if name not in ("staging_bytes", "L", "B", "Nmax", "Hq", "Hkv", "d", "Scap", "V", "P", "Dp1", "scale", "stream"):
            setattr(a, name, 0x1000)
    a.staging_bytes = 1 << 40
    a.L, a.B, a.Nmax, a.Hq, a.Hkv, a.d, a.Scap, a.V, a.P, a.Dp1, a.scale = 2, 2, 15, 4, 2, 32, 256, 1024, 8, 5, 0.125
    assert lib.tv_verify_step_host(ctypes.byref(a)) == 1 and b"d must be 64 or 128" in lib.tv_last_error()
    a.d, a.Hq = 64, 5
    assert lib.tv_verify_step_host(ctypes.byref(a)) == 1 and b"Hq" in lib.tv_last_error()
    a.Hq, a.Nmax = 4, 300
    assert lib.tv_verify_step_host(ctypes.byref(a)) == 1 and b"Nmax" in lib.tv_last_error()


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2603_08088_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libtreeverify.so")
    with pytest.raises(ImportError):
        binding.load()
