"""kda_chunk_fwd_static: the prefill entry point for callers that cannot allocate device memory
(a serving loop with a fixed memory pool, a plug-in that is given tensors but no allocator).  It
must give the same results as kda_chunk_fwd with a caller-provided workspace, on consecutive calls
that share the library's built-in scratch, and must refuse calls that do not fit that scratch.

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
    K.kda_chunk_fwd_static(g["q"], g["k"], g["v"], g["log_alpha"], g["beta"], g["S0"], o, S_T,
                           g["cu_seqlens"] if varlen else None, cu if varlen else None, N, T, H,
                           dk, dk, 64, 1.0, dt)
    torch.cuda.synchronize()
    return o, S_T


def test_static_scratch_matches_workspace_call_twice():
    # two calls in a row with different inputs (and dtypes): the second reuses the scratch that the
    # first one left behind
    cases = [
        inputs.chunk_inputs([700, 130], H=4, dtype=torch.bfloat16, seed=41, s0_std=0.02),
        inputs.chunk_inputs([333], H=3, dtype=torch.float32, seed=42, s0_std=0.02),
        inputs.chunk_inputs([64, 1, 200], H=4, dtype=torch.bfloat16, seed=43, s0_std=0.02),
    ]
    for d in cases:
        dt = K.KDA_BF16 if d["k"].dtype == torch.bfloat16 else K.KDA_F32
        o_ref, S_ref = run_chunk(d)                 # existing entry point, caller's workspace
        o, S_T = _run_static(d)
        assert torch.isfinite(o.float()).all() and torch.isfinite(S_T).all()
        assert rel_l2(to_np32(o), to_np32(o_ref)) <= TOL[dt]
        assert rel_l2(to_np32(S_T), to_np32(S_ref)) <= TOL[dt]


def test_static_scratch_rejects_oversized_calls():
    assert K.kda_chunk_fwd_static_max_bytes() == 16 << 20
    # 64 sequences x 32 heads need 128 MiB of state scratch alone
    N, H = 64, 32
    lens = [64] * N
    T = sum(lens)
    assert K.kda_chunk_fwd_min_workspace_bytes(T, N, H) > K.kda_chunk_fwd_static_max_bytes()
    dev = "cuda:0"
    z = torch.zeros((T, H, 128), dtype=torch.bfloat16, device=dev)
    g = torch.zeros((T, H, 128), dtype=torch.float32, device=dev)
    b = torch.zeros((T, H), dtype=torch.float32, device=dev)
    o = torch.empty_like(z)
    with pytest.raises(K.KdaError) as ei:
        K.kda_chunk_fwd_static(z, z, z, g, b, None, o, None, None, None, N, T, H, 128, 128, 64,
                               1.0, K.KDA_BF16)
    assert ei.value.code == 3 and "scratch" in str(ei.value)
