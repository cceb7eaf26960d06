"""Shared helpers of the GPU parity tests: run the CUDA library through its binding, run the oracle
on the same tensors, compare with the relative L2 norm the tolerances are stated in."""
from __future__ import annotations

import numpy as np
import torch

import paper_2510_26692_b200 as K

TOL = {K.KDA_BF16: 2e-2, K.KDA_F32: 1e-4}   # max relative L2 error on o and S_T


def rel_l2(x, ref) -> float:
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref)
    num = np.linalg.norm(x - ref)
    return float(num / den) if den > 0 else float(num)


def dt_of(t: torch.Tensor) -> int:
    return K.KDA_BF16 if t.dtype == torch.bfloat16 else K.KDA_F32


def to_np32(t):
    return None if t is None else t.detach().to("cpu", torch.float32).numpy()


def run_chunk(d, scale=1.0, want_o=True, want_state=True, workspace_bytes=None, dev="cuda:0",
              poison=True):
    """d: dict from inputs.chunk_inputs (CPU or CUDA tensors).  Returns (o, S_T) as CUDA tensors."""
    g = {n: (t.to(dev) if isinstance(t, torch.Tensor) else t) for n, t in d.items()}
    k = g["k"]
    T, H, dk = k.shape
    dv = g["v"].shape[-1]
    dt = dt_of(k)
    cu = d.get("cu_seqlens")
    N = int(cu.numel()) - 1 if cu is not None else 1
    if workspace_bytes is None:
        workspace_bytes = K.kda_chunk_fwd_workspace_bytes(T, N, H, dk, dv, 64, dt)
    ws = torch.empty(workspace_bytes, dtype=torch.uint8, device=dev)
    o = S_T = None
    if want_o:
        o = torch.empty_like(g["v"])
        if poison:
            o.fill_(float("nan"))
    if want_state:
        S_T = torch.empty((N, H, dk, dv), dtype=torch.float32, device=dev)
        if poison:
            S_T.fill_(float("nan"))
    varlen = cu is not None and N > 1 or (cu is not None and d.get("force_varlen", False))
    K.kda_chunk_fwd(g["q"] if want_o else g.get("q"), k, g["v"], g["log_alpha"], g["beta"],
                    g["S0"], o, S_T, g["cu_seqlens"] if varlen else None,
                    cu.cpu() if varlen else None, N, T, H, dk, dv, 64, scale, dt, ws,
                    workspace_bytes)
    torch.cuda.synchronize()
    return o, S_T


def oracle_chunk(oracle, d, scale=1.0, want_o=True):
    cu = d.get("cu_seqlens")
    S0 = d.get("S0")
    o, S_T = oracle.recurrence(
        to_np32(d["q"]) if want_o else None, to_np32(d["k"]), to_np32(d["v"]),
        to_np32(d["log_alpha"]), to_np32(d["beta"]),
        S0=None if S0 is None else S0.detach().cpu().double().numpy(),
        cu_seqlens=None if cu is None else cu.cpu().numpy().astype(np.int64), scale=scale,
        want_o=want_o)
    return o, S_T


def check_chunk(oracle, d, tol, scale=1.0, per_seq=True, **kw):
    """Runs both sides and asserts rel-L2 <= tol on o and S_T (per sequence for packed batches)."""
    o, S_T = run_chunk(d, scale=scale, **kw)
    o_ref, S_ref = oracle_chunk(oracle, d, scale=scale)
    o = to_np32(o)
    S_T = to_np32(S_T)
    assert np.isfinite(o).all() and np.isfinite(S_T).all()
    errs = {"o": rel_l2(o, o_ref), "S_T": rel_l2(S_T, S_ref)}
    cu = d.get("cu_seqlens")
    if per_seq and cu is not None:
        cu = cu.tolist()
        for n in range(len(cu) - 1):
            if cu[n + 1] > cu[n]:
                errs["o[%d]" % n] = rel_l2(o[cu[n]:cu[n + 1]], o_ref[cu[n]:cu[n + 1]])
            errs["S_T[%d]" % n] = rel_l2(S_T[n], S_ref[n])
    bad = {n: e for n, e in errs.items() if not e <= tol}
    assert not bad, "rel-L2 above %g: %s" % (tol, bad)
    return errs
