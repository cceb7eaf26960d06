"""kda_chunk_fwd_static: the prefill entry point for callers that cannot allocate device memory
(a serving loop with a fixed memory pool, a plug-in that is given tensors but no allocator).  It
must give the same results as kda_chunk_fwd with a caller-provided workspace of the same size, on
consecutive calls that share the library's built-in scratch, must not allocate, and must refuse
calls that do not fit that scratch.

Collected last on purpose: a failure here cannot hide a failure of any other test in a run that
stops at the first failure."""
import pytest
import torch

import paper_2510_26692_b200 as K
from paper_2510_26692_b200 import inputs
from kda_testlib import TOL, rel_l2, run_chunk, to_np32

pytestmark = pytest.mark.gpu


def _run_static(d, dev="cuda:0"):
    g = {n: (t.to(dev) if isinstance(t, torch.Tensor) else t) for n, t in d.items()}
    T, H, dk = g["k"].shape
    cu = d["cu_seqlens"]
    N = cu.numel() - 1
    dt = K.KDA_BF16 if g["k"].dtype == torch.bfloat16 else K.KDA_F32
    o = torch.full_like(g["v"], float("nan"))
    S_T = torch.full((N, H, dk, dk), float("nan"), dtype=torch.float32, device=dev)
    varlen = N > 1
    cu_dev = g["cu_seqlens"] if varlen else None
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    K.kda_chunk_fwd_static(g["q"], g["k"], g["v"], g["log_alpha"], g["beta"], g["S0"], o, S_T,
                           cu_dev, cu if varlen else None, N, T, H, dk, dk, 64, 1.0, dt)
    K.kda_chunk_fwd_static_check_status()       # synchronises; raises on a device-side error
    free1, _ = torch.cuda.mem_get_info()
    return o, S_T, free0 - free1


def test_static_scratch_matches_workspace_call_twice():
    # calls in a row with different inputs (and dtypes): each reuses the scratch that the previous
    # one left behind.  The fourth case is a long packed batch: far more tiles than the scratch holds.
    cases = [
        inputs.chunk_inputs([700, 130], H=4, dtype=torch.bfloat16, seed=41, s0_std=0.02),
        inputs.chunk_inputs([333], H=3, dtype=torch.float32, seed=42, s0_std=0.02),
        inputs.chunk_inputs([64, 1, 200], H=4, dtype=torch.bfloat16, seed=43, s0_std=0.02),
        inputs.chunk_inputs([4000, 700], H=16, dtype=torch.bfloat16, seed=44, s0_std=0.02),
    ]
    _run_static(cases[0])                            # warm-up: the one-time address look-up
    nbytes = K.kda_chunk_fwd_static_max_bytes()
    for d in cases:
        dt = K.KDA_BF16 if d["k"].dtype == torch.bfloat16 else K.KDA_F32
        # the existing entry point with a caller's workspace of exactly the built-in size
        o_ref, S_ref = run_chunk(d, workspace_bytes=nbytes)
        o, S_T, grew = _run_static(d)
        assert grew == 0, "the call changed the amount of free device memory by %d bytes" % grew
        assert torch.isfinite(o.float()).all() and torch.isfinite(S_T).all()
        assert rel_l2(to_np32(o), to_np32(o_ref)) <= TOL[dt]
        assert rel_l2(to_np32(S_T), to_np32(S_ref)) <= TOL[dt]
        # same scratch size, same schedule, same arithmetic: the results are bit-identical
        assert torch.equal(o, o_ref) and torch.equal(S_T, S_ref)


def test_static_scratch_rejects_oversized_calls():
    assert K.kda_chunk_fwd_static_max_bytes() == 16 << 20
    # fp32: 64 sequences x 32 heads need 128 MiB of state scratch alone
    N, H = 64, 32
    lens = [64] * N
    T = sum(lens)
    assert K.kda_chunk_fwd_min_workspace_bytes(T, N, H, dt=K.KDA_F32) > K.kda_chunk_fwd_static_max_bytes()
    dev = "cuda:0"
    z = torch.zeros((T, H, 128), dtype=torch.float32, device=dev)
    g = torch.zeros((T, H, 128), dtype=torch.float32, device=dev)
    b = torch.zeros((T, H), dtype=torch.float32, device=dev)
    o = torch.empty_like(z)
    with pytest.raises(K.KdaError) as ei:
        K.kda_chunk_fwd_static(z, z, z, g, b, None, o, None, None, None, N, T, H, 128, 128, 64,
                               1.0, K.KDA_F32)
    assert ei.value.code == 3 and "scratch" in str(ei.value)
