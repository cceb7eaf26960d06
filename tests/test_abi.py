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


def _plan(lib, chunks, H, avail, n_sm):
    arr = (ctypes.c_int32 * len(chunks))(*chunks)
    out = (ctypes.c_int64 * 4)()
    lib.kda_selftest_fused_plan.restype = ctypes.c_int
    lib.kda_selftest_fused_plan.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                            ctypes.c_int64, ctypes.c_int, ctypes.c_void_p]
    rc = lib.kda_selftest_fused_plan(ctypes.cast(arr, ctypes.c_void_p), len(chunks), H, avail, n_sm,
                                     ctypes.cast(out, ctypes.c_void_p))
    assert rc == 0
    return tuple(out)


def test_fused_schedule_plan(lib):
    """Host side of the fused prefill kernel: how many (sequence, head) chains run side by side, how
    deep their tile rings are, and how many production indices the call hands out.  Checked against
    the constraints the kernel relies on and against a count by enumeration."""
    import random
    rng = random.Random(7)
    cases = [([64], 32, 1024, 148), ([3, 11, 1, 5, 0, 14, 4, 3, 2, 0, 7], 5, 40, 148),
             ([5, 4], 40, 1024, 148), ([1], 1, 2, 148), ([9] * 7, 3, 7, 148), ([2, 2], 2, 1000, 8)]
    for _ in range(200):
        n = rng.randint(1, 12)
        cases.append(([rng.randint(0, 20) for _ in range(n)], rng.randint(1, 70),
                      rng.randint(2, 1200), rng.choice([4, 16, 132, 148, 160, 400])))
    for chunks, H, avail, n_sm in cases:
        Q, R, n_rounds, n_prod = _plan(lib, chunks, H, avail, n_sm)
        J = len(chunks) * H
        q_max = min(n_sm // 4, 64)          # two CTAs per chain, as many CTAs again for the tiles
        assert 1 <= Q <= min(J, q_max), (chunks, H, avail, n_sm, Q)
        assert 2 <= R <= 16 and Q * R <= avail          # the rings fit the workspace
        assert n_rounds == -(-J // Q)
        if H <= q_max and Q * 2 <= avail and Q < J and (H * (q_max // H)) * 2 <= avail:
            assert Q % H == 0                           # whole sequences per round
        # enumeration: every round takes (its longest chain) x (its chains) indices, and each
        # (chain, chunk) pair of the batch gets exactly one of them
        total, tiles = 0, 0
        for r in range(n_rounds):
            js = range(r * Q, min((r + 1) * Q, J))
            longest = max(chunks[j // H] for j in js)
            for c in range(longest):
                for j in js:
                    total += 1
                    tiles += c < chunks[j // H]
        assert total == n_prod and tiles == sum(chunks) * H
    # no schedule: fewer than two tiles of room, or a device with fewer than four SMs
    assert _plan(lib, [4], 2, 1, 148)[0] == 0
    assert _plan(lib, [4], 2, 64, 3)[0] == 0


def test_side_entry_points_reject_bad_arguments(lib):
    """Layer wrap, backward pass and DPLR comparison: argument errors found before any CUDA call."""
    import paper_2510_26692_b200 as K
    one = ctypes.c_void_p(256)
    f32, sz, i64, i32 = ctypes.c_float, ctypes.c_size_t, ctypes.c_int64, ctypes.c_int
    # kda_dplr_chunk_fwd: head size, misaligned pointer, cu_seqlens on one side only
    rc = lib.kda_dplr_chunk_fwd(one, one, one, one, one, one, None, one, one, None, None, 1, 64, 2, 64, 128, 64,
                                1.0, one, 1 << 30, None)
    assert rc == 2
    rc = lib.kda_dplr_chunk_fwd(one, one, one, ctypes.c_void_p(260), one, one, None, one, one, None, None, 1, 64, 2,
                                128, 128, 64, 1.0, one, 1 << 30, None)
    assert rc == 1 and "aligned" in K.kda_last_error()
    rc = lib.kda_dplr_chunk_fwd(one, one, one, one, one, one, None, one, one, one, None, 1, 64, 2, 128, 128, 64, 1.0,
                                one, 1 << 30, None)
    assert rc == 1
    assert lib.kda_dplr_chunk_fwd_workspace_bytes(4096, 1, 2, 128, 128, 64) >= \
        lib.kda_dplr_chunk_fwd_min_workspace_bytes(4096, 1, 2, 128, 128, 64) > 0
    assert lib.kda_dplr_chunk_fwd_workspace_bytes(4096, 1, 2, 64, 128, 64) == 0
    # kda_chunk_bwd: chunk length, missing gradient output, workspace too small
    args = [one] * 6 + [one, one] + [one] * 5 + [one, None, None]
    rc = lib.kda_chunk_bwd(*args, 1, 64, 2, 128, 128, 32, 1.0, K.KDA_BF16, one, 1 << 30, None)
    assert rc == 2
    bad = list(args)
    bad[9] = None      # dk
    rc = lib.kda_chunk_bwd(*bad, 1, 64, 2, 128, 128, 64, 1.0, K.KDA_BF16, one, 1 << 30, None)
    assert rc == 1 and "NULL" in K.kda_last_error()
    rc = lib.kda_chunk_bwd(*args, 1, 64, 2, 128, 128, 64, 1.0, K.KDA_BF16, one, 4096, None)
    assert rc == 3
    assert lib.kda_chunk_bwd_workspace_bytes(4096, 1, 32, 128, 128, 64) > 4096 * 32 * 128 * 4 * 12
    # kda_layer_fwd: decay-function parameters are required; y needs its gate and weight
    largs = [one] * 6 + [None, one, one]
    rc = lib.kda_layer_fwd(*largs, 1e-6, 1e-5, None, one, one, None, None, 1, 64, 2, 128, 128, 64, 1.0, one,
                           1 << 30, None)
    assert rc == 1 and "A_log" in K.kda_last_error()
    largs = [one] * 5 + [None, one, one, one]
    rc = lib.kda_layer_fwd(*largs, 1e-6, 1e-5, None, one, one, None, None, 1, 64, 2, 128, 128, 64, 1.0, one,
                           1 << 30, None)
    assert rc == 1 and "g_o" in K.kda_last_error()
    assert lib.kda_layer_fwd_workspace_bytes(4096, 1, 32, 128, 128, 64) >= \
        lib.kda_layer_fwd_min_workspace_bytes(4096, 1, 32, 128, 128, 64) > 0


def test_wait_limit_from_environment(lib):
    """KDA_WAIT_LIMIT_MS bounds every device-side wait; read once per process, so checked in children."""
    import subprocess
    import sys
    lib.kda_wait_limit_ns.restype = ctypes.c_uint64
    assert lib.kda_wait_limit_ns() == 1_000_000_000      # (this process: variable not set)
    code = ("import ctypes; from paper_2510_26692_b200 import api; l = api.load(); "
            "l.kda_wait_limit_ns.restype = ctypes.c_uint64; print(l.kda_wait_limit_ns())")
    for val, want in (("250", 250_000_000), ("0", 1_000_000_000), ("junk", 1_000_000_000), ("9999999", 1_000_000_000)):
        env = dict(os.environ, KDA_WAIT_LIMIT_MS=val)
        out = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True)
        assert out.returncode == 0, out.stderr
        assert int(out.stdout.strip().splitlines()[-1]) == want, (val, out.stdout)
