"""Parity of the diagonal-plus-low-rank comparison workload (kda_dplr_chunk_fwd, fp32) with its fp64
oracle, through the C ABI.  Tolerance: relative L2 error 1e-4 on o and on the final state, the same
as for the fp32 KDA path (fp32 FMA sums of length <= 128 and 64, no reduced-precision product)."""
import numpy as np
import pytest
import torch

import paper_2510_26692_b200 as K
from paper_2510_26692_b200 import inputs
from kda_testlib import GUARD, Guarded, rel_l2, to_np32

pytestmark = pytest.mark.gpu
TOL = 1e-4


def run_dplr(d, scale=1.0, want_o=True, workspace_bytes=None, dev="cuda:0"):
    g = {n: (t.to(dev) if isinstance(t, torch.Tensor) else t) for n, t in d.items()}
    T, H, dk = g["k"].shape
    cu = d["cu_seqlens"]
    N = cu.numel() - 1
    nb = workspace_bytes or K.kda_dplr_chunk_fwd_workspace_bytes(T, N, H)
    ws = Guarded(nb, dev)
    ob = Guarded(T * H * 128 * 4, dev)
    sb = Guarded(N * H * 128 * 128 * 4, dev)
    o = ob.view(torch.float32, (T, H, 128))
    S_T = sb.view(torch.float32, (N, H, 128, 128))
    o.fill_(float("nan"))
    S_T.fill_(float("nan"))
    varlen = N > 1
    K.kda_dplr_chunk_fwd(g["q"] if want_o else None, g["k"], g["v"], g["a"], g["b"], g["g"], g["S0"],
                         o if want_o else None, S_T, g["cu_seqlens"] if varlen else None,
                         cu if varlen else None, N, T, H, 128, 128, 64, scale, ws.body, nb)
    torch.cuda.synchronize()
    K.kda_check_status(ws.body)
    for b_, name in ((ws, "the workspace"), (ob, "o"), (sb, "S_T")):
        b_.check(name)
    return (o if want_o else None), S_T


def oracle_dplr(oracle_mod, d, scale=1.0):
    cu = d["cu_seqlens"].numpy().astype(np.int64)
    return oracle_mod.dplr_recurrence(*(d[n].numpy() for n in ("q", "k", "v", "a", "b", "g")),
                                      S0=None if d["S0"] is None else d["S0"].double().numpy(),
                                      cu_seqlens=cu, scale=scale)


@pytest.mark.parametrize("lens,H,s0", [([256], 2, 0.0), ([1000], 3, 0.05), ([64, 1, 200, 0, 130], 4, 0.05),
                                       ([2048], 16, 0.02), ([1], 1, 0.05), ([63, 65, 0], 1, 0.0)])
def test_dplr_matches_oracle(oracle_mod, lens, H, s0):
    d = inputs.dplr_inputs(lens, H=H, seed=21, s0_std=s0)
    o, S_T = run_dplr(d, scale=0.9)
    o_ref, S_ref = oracle_dplr(oracle_mod, d, scale=0.9)
    assert torch.isfinite(o).all() and torch.isfinite(S_T).all()
    eo, es = rel_l2(to_np32(o), o_ref), rel_l2(to_np32(S_T), S_ref)
    print("dplr", lens, H, eo, es)
    assert eo <= TOL and es <= TOL


def test_dplr_small_workspace_passes(oracle_mod):
    """With the minimum workspace the call walks the chunks one at a time; the result is the same
    to rounding (same arithmetic per chunk) and state-only calls work."""
    d = inputs.dplr_inputs([700, 130], H=2, seed=22, s0_std=0.05)
    nb = K.kda_dplr_chunk_fwd_min_workspace_bytes(830, 2, 2)
    o1, S1 = run_dplr(d, workspace_bytes=nb)
    o2, S2 = run_dplr(d)
    assert torch.equal(o1, o2) and torch.equal(S1, S2)
    _, S3 = run_dplr(d, want_o=False)
    assert torch.equal(S3, S2)
    o_ref, S_ref = oracle_dplr(oracle_mod, d)
    assert rel_l2(to_np32(o1), o_ref) <= TOL and rel_l2(to_np32(S1), S_ref) <= TOL


def test_dplr_bound_to_k_equals_kda(oracle_mod):
    """Section 6.1: with a = alpha . k, b = -beta k and the key beta k the general kernel computes
    Eq. 1.  Checked against the KDA oracle and against the library's own fp32 KDA path."""
    d = inputs.chunk_inputs([500], H=2, dtype=torch.float32, seed=23, s0_std=0.05)
    k, la, beta = d["k"], d["log_alpha"], d["beta"]
    dd = {"q": d["q"], "k": beta[..., None] * k, "v": d["v"], "a": torch.exp(la) * k, "b": -beta[..., None] * k,
          "g": la, "S0": d["S0"], "cu_seqlens": d["cu_seqlens"]}
    o, S_T = run_dplr(dd)
    o_ref, S_ref = oracle_mod.recurrence(*(d[n].numpy() for n in ("q", "k", "v", "log_alpha", "beta")),
                                         S0=d["S0"].double().numpy())
    assert rel_l2(to_np32(o), o_ref) <= TOL and rel_l2(to_np32(S_T), S_ref) <= TOL


def test_dplr_argument_errors():
    z = torch.zeros((64, 1, 128), device="cuda:0")
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda:0")
    with pytest.raises(K.KdaError) as ei:   # workspace too small for one tile per head
        K.kda_dplr_chunk_fwd(z, z, z, z, z, z, None, z.clone(), None, None, None, 1, 64, 1, 128, 128, 64, 1.0,
                             ws[:4096], 4096)
    assert ei.value.code == 3
    with pytest.raises(K.KdaError) as ei:
        K.kda_dplr_chunk_fwd(z, z, z, z, z, z, None, z.clone(), None, None, None, 1, 64, 1, 64, 128, 64, 1.0, ws)
    assert ei.value.code == 2
