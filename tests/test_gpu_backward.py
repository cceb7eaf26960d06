"""Parity of kda_chunk_bwd (gradients of the prefill operator) with the fp64 backward oracle, through
the C ABI.  Tolerance: relative L2 error 1e-4 per gradient tensor (fp32 FMA arithmetic over at most
a few thousand sequential tokens; stored inputs are exact in both)."""
import numpy as np
import pytest
import torch

import paper_2510_26692_b200 as K
from paper_2510_26692_b200 import inputs
from kda_testlib import Guarded, rel_l2, to_np32

pytestmark = pytest.mark.gpu
TOL = 1e-4
NAMES = ("dq", "dk", "dv", "dlog_alpha", "dbeta", "dS0")


def cotangents(d, seed, dtype):
    T, H, dv = d["v"].shape
    N = d["cu_seqlens"].numel() - 1
    g = torch.Generator().manual_seed(1000 + seed)
    d_o = torch.randn((T, H, dv), generator=g).to(dtype)
    dS_T = torch.randn((N, H, 128, dv), generator=g) * 0.1
    return d_o, dS_T


def run_bwd(d, d_o, dS_T, scale=1.0, dev="cuda:0", want_dS0=True):
    g = {n: (t.to(dev) if isinstance(t, torch.Tensor) else t) for n, t in d.items()}
    T, H, dk = g["k"].shape
    cu = d["cu_seqlens"]
    N = cu.numel() - 1
    dt = K.KDA_BF16 if g["k"].dtype == torch.bfloat16 else K.KDA_F32
    nb = K.kda_chunk_bwd_workspace_bytes(T, N, H)
    ws = Guarded(nb, dev)
    bufs = {"dq": Guarded(T * H * 128 * 4, dev), "dk": Guarded(T * H * 128 * 4, dev),
            "dv": Guarded(T * H * 128 * 4, dev), "dlog_alpha": Guarded(T * H * 128 * 4, dev),
            "dbeta": Guarded(max(T * H * 4, 16), dev), "dS0": Guarded(N * H * 128 * 128 * 4, dev)}
    out = {n: bufs[n].view(torch.float32, (T, H, 128)) for n in ("dq", "dk", "dv", "dlog_alpha")}
    out["dbeta"] = bufs["dbeta"].body[:T * H * 4].view(torch.float32).view(T, H)
    out["dS0"] = bufs["dS0"].view(torch.float32, (N, H, 128, 128))
    for x in out.values():
        x.fill_(float("nan"))
    varlen = N > 1
    K.kda_chunk_bwd(g["q"], g["k"], g["v"], g["log_alpha"], g["beta"], g["S0"],
                    None if d_o is None else d_o.to(dev), None if dS_T is None else dS_T.to(dev),
                    out["dq"], out["dk"], out["dv"], out["dlog_alpha"], out["dbeta"],
                    out["dS0"] if want_dS0 else None, g["cu_seqlens"] if varlen else None,
                    cu if varlen else None, N, T, H, 128, 128, 64, scale, dt, ws.body, nb)
    torch.cuda.synchronize()
    K.kda_check_status(ws.body)
    ws.check("the workspace")
    for n, b_ in bufs.items():
        b_.check(n)
    return out


def oracle_bwd(oracle_mod, d, d_o, dS_T, scale=1.0):
    cu = d["cu_seqlens"].numpy().astype(np.int64)
    return oracle_mod.backward(*(d[n].float().numpy() for n in ("q", "k", "v", "log_alpha", "beta")),
                               d_o=None if d_o is None else d_o.double().numpy(),
                               dS_T=None if dS_T is None else dS_T.double().numpy(),
                               S0=None if d["S0"] is None else d["S0"].double().numpy(),
                               cu_seqlens=cu, scale=scale)


@pytest.mark.parametrize("lens,H,dtype,s0", [([100], 2, torch.float32, 0.0),
                                             ([300], 3, torch.bfloat16, 0.05),
                                             ([64, 1, 200, 0, 130], 2, torch.bfloat16, 0.05),
                                             ([1024], 4, torch.float32, 0.02),
                                             ([3, 0, 9, 64, 65, 1], 1, torch.float32, 0.05),
                                             ([7, 8], 3, torch.bfloat16, 0.0)])
def test_backward_matches_oracle(oracle_mod, lens, H, dtype, s0):
    d = inputs.chunk_inputs(lens, H=H, dtype=dtype, seed=31, s0_std=s0)
    d_o, dS_T = cotangents(d, 31, dtype)
    out = run_bwd(d, d_o, dS_T, scale=0.8)
    ref = oracle_bwd(oracle_mod, d, d_o, dS_T, scale=0.8)
    errs = {n: rel_l2(to_np32(out[n]), ref[n]) for n in NAMES}
    print("bwd", lens, H, dtype, errs)
    for n in NAMES:
        assert torch.isfinite(out[n]).all(), n
        assert errs[n] <= TOL, (n, errs[n])


def test_backward_optional_cotangents_and_determinism(oracle_mod):
    d = inputs.chunk_inputs([200, 70], H=2, dtype=torch.bfloat16, seed=32, s0_std=0.05)
    d_o, dS_T = cotangents(d, 32, torch.bfloat16)
    a = run_bwd(d, d_o, None)
    ref = oracle_bwd(oracle_mod, d, d_o, None)
    for n in NAMES:
        assert rel_l2(to_np32(a[n]), ref[n]) <= TOL, n
    b = run_bwd(d, None, dS_T, want_dS0=False)
    ref = oracle_bwd(oracle_mod, d, None, dS_T)
    for n in NAMES[:-1]:
        assert rel_l2(to_np32(b[n]), ref[n]) <= TOL, n
    a2 = run_bwd(d, d_o, None)
    for n in NAMES:
        assert torch.equal(a[n], a2[n]), n       # fixed summation order: bit-identical runs


def test_backward_argument_errors():
    z = torch.zeros((64, 1, 128), device="cuda:0")
    b = torch.zeros((64, 1), device="cuda:0")
    ws = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda:0")
    with pytest.raises(K.KdaError) as ei:
        K.kda_chunk_bwd(z, z, z, z, b, None, z, None, z.clone(), z.clone(), z.clone(), z.clone(), b.clone(), None,
                        None, None, 1, 64, 1, 128, 128, 64, 1.0, K.KDA_F32, ws)
    assert ei.value.code == 3
