"""The C-ABI library loads without a GPU and exports every symbol that include/kda.h declares;
argument errors that are detected before any CUDA call are reported with the right status."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2510_26692_b200 import build, api
    build.build()
    return api.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "kda.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(kda_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_header_symbols_exported(lib):
    names = declared_functions()
    assert "kda_chunk_fwd" in names and "kda_decode_step" in names and len(names) >= 10
    for n in names:
        assert hasattr(lib, n), "symbol %s declared in kda.h is not exported" % n


def test_unsupported_and_invalid_arguments(lib):
    import paper_2510_26692_b200 as K
    one = ctypes.c_void_p(256)
    # unsupported head size / chunk / dtype: rejected before any launch, no fallback
    rc = lib.kda_chunk_fwd(one, one, one, one, one, None, one, one, None, None, 1, 64, 2, 64, 64,
                           64, 1.0, K.KDA_BF16, one, 1 << 30, None)
    assert rc == 2 and "supported" in K.kda_last_error()
    rc = lib.kda_chunk_fwd(one, one, one, one, one, None, one, one, None, None, 1, 64, 2, 128, 128,
                           32, 1.0, K.KDA_BF16, one, 1 << 30, None)
    assert rc == 2
    rc = lib.kda_decode_step(one, one, one, one, one, one, None, one, 4, 2, 128, 64, 1.0,
                             K.KDA_BF16, None)
    assert rc == 2
    # misaligned pointer
    rc = lib.kda_chunk_fwd(ctypes.c_void_p(260), one, one, one, one, None, one, one, None, None, 1,
                           64, 2, 128, 128, 64, 1.0, K.KDA_BF16, one, 1 << 30, None)
    assert rc == 1 and "aligned" in K.kda_last_error()
    # cu_seqlens given on one side only
    rc = lib.kda_chunk_fwd(one, one, one, one, one, None, one, one, one, None, 1, 64, 2, 128, 128,
                           64, 1.0, K.KDA_BF16, one, 1 << 30, None)
    assert rc == 1
    # non-monotone / wrong-ended cu_seqlens (host copy is validated before any launch)
    bad = (ctypes.c_int32 * 3)(0, 80, 64)
    rc = lib.kda_chunk_fwd(one, one, one, one, one, None, one, one, one,
                           ctypes.cast(bad, ctypes.c_void_p), 2, 64, 2, 128, 128, 64, 1.0,
                           K.KDA_BF16, one, 1 << 30, None)
    assert rc == 1 and "decreases" in K.kda_last_error()
    bad2 = (ctypes.c_int32 * 3)(0, 10, 60)
    rc = lib.kda_chunk_fwd(one, one, one, one, one, None, one, one, one,
                           ctypes.cast(bad2, ctypes.c_void_p), 2, 64, 2, 128, 128, 64, 1.0,
                           K.KDA_BF16, one, 1 << 30, None)
    assert rc == 1
    # workspace too small / missing
    rc = lib.kda_chunk_fwd(one, one, one, one, one, None, one, one, None, None, 1, 64, 2, 128, 128,
                           64, 1.0, K.KDA_BF16, one, 1024, None)
    assert rc == 3 and "workspace" in K.kda_last_error()
    rc = lib.kda_chunk_fwd(one, one, one, one, one, None, one, one, None, None, 1, 64, 2, 128, 128,
                           64, 1.0, K.KDA_BF16, None, 0, None)
    assert rc == 3
    # q missing although o is requested
    rc = lib.kda_chunk_fwd(None, one, one, one, one, None, one, one, None, None, 1, 64, 2, 128, 128,
                           64, 1.0, K.KDA_BF16, one, 1 << 30, None)
    assert rc == 1


def test_workspace_queries(lib):
    import paper_2510_26692_b200 as K
    lo = K.kda_chunk_fwd_min_workspace_bytes(4096, 1, 32)
    hi = K.kda_chunk_fwd_workspace_bytes(4096, 1, 32)
    assert 0 < lo <= hi
    assert K.kda_chunk_fwd_workspace_bytes(1 << 20, 1, 32) <= (8 << 30)
    assert K.kda_chunk_fwd_workspace_bytes(4096, 1, 32, dk=64) == 0
    assert K.kda_chunk_fwd_host_workspace_bytes(4096, 1, 32) > hi
    assert K.kda_decode_step_host_workspace_bytes(256, 32) > 0


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2510_26692_b200 import api
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "_LIB_PATH", "/nonexistent/libkda_b200.so")
    with pytest.raises(ImportError):
        api.kda_version()


def test_per_device_table(lib):
    """What the library caches per device lives in one slot per device ordinal behind a mutex; the
    self-test exercises the table without any CUDA call.  Also from several threads at once."""
    import threading
    lib.kda_selftest_device_table.restype = ctypes.c_int
    assert lib.kda_selftest_device_table() == 0
    out = []
    ts = [threading.Thread(target=lambda: out.append(lib.kda_selftest_device_table())) for _ in range(8)]
    for t in ts:
        t.start()
    for t in ts:
        t.join()
    # (the lock probe may find the mutex taken by a sibling thread: code 5 is not a table fault)
    assert all(c in (0, 5) for c in out) and 0 in out


def test_chunk_path_switch(lib):
    import paper_2510_26692_b200 as K
    for mode in (2, 1, 0):
        K.kda_set_chunk_path(mode)
    assert lib.kda_set_chunk_path(3) == 1 and lib.kda_set_chunk_path(-1) == 1
