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


GUARD = 4096          # sentinel bytes on each side of every output / scratch buffer
SENTINEL = 0xA5


class Guarded:
    """A device buffer of `nbytes` usable bytes between two sentinel-filled margins (the only
    out-of-bounds evidence available where compute-sanitizer is closed)."""

    def __init__(self, nbytes: int, dev, fill_nan_as=None):
        self.raw = torch.full((nbytes + 2 * GUARD,), SENTINEL, dtype=torch.uint8, device=dev)
        self.body = self.raw[GUARD:GUARD + nbytes]

    def view(self, dtype, shape):
        return self.body.view(dtype).view(shape)

    def check(self, what: str):
        lo, hi = self.raw[:GUARD], self.raw[-GUARD:]
        assert bool((lo == SENTINEL).all()) and bool((hi == SENTINEL).all()), \
            "bytes outside %s were written" % what


def run_chunk(d, scale=1.0, want_o=True, want_state=True, workspace_bytes=None, dev="cuda:0",
              poison=True, expect_status=None, static=False):
    """d: dict from inputs.chunk_inputs (CPU or CUDA tensors).  Returns (o, S_T) as CUDA tensors.
    o, S_T and the workspace sit between sentinel margins that must come back untouched; o and
    S_T start NaN-filled; the status word must be clean afterwards (or equal `expect_status`)."""
    g = {n: (t.to(dev) if isinstance(t, torch.Tensor) else t) for n, t in d.items()}
    k = g["k"]
    T, H, dk = k.shape
    dv = g["v"].shape[-1]
    dt = dt_of(k)
    es = 2 if dt == K.KDA_BF16 else 4
    cu = d.get("cu_seqlens")
    N = int(cu.numel()) - 1 if cu is not None else 1
    if workspace_bytes is None:
        workspace_bytes = K.kda_chunk_fwd_workspace_bytes(T, N, H, dk, dv, 64, dt)
    wsg = Guarded(workspace_bytes, dev)
    ws = wsg.body
    assert ws.data_ptr() % 256 == 0
    o = S_T = og = sg = None
    if want_o:
        og = Guarded(T * H * dv * es, dev)
        o = og.view(k.dtype, (T, H, dv))
        if poison:
            o.fill_(float("nan"))
    if want_state:
        sg = Guarded(N * H * dk * dv * 4, dev)
        S_T = sg.view(torch.float32, (N, H, dk, dv))
        if poison:
            S_T.fill_(float("nan"))
    varlen = cu is not None and N > 1 or (cu is not None and d.get("force_varlen", False))
    args = (g["q"] if want_o else g.get("q"), k, g["v"], g["log_alpha"], g["beta"],
            g["S0"], o, S_T, g["cu_seqlens"] if varlen else None,
            cu.cpu() if varlen else None, N, T, H, dk, dv, 64, scale, dt)
    if static:
        K.kda_chunk_fwd_static(*args)
        torch.cuda.synchronize()
    else:
        K.kda_chunk_fwd(*args, ws, workspace_bytes)
        torch.cuda.synchronize()
        try:
            K.kda_check_status(ws)
            code = 0
        except K.KdaError as e:
            code = e.code
        assert code == (expect_status or 0), "status after the call: %d" % code
    wsg.check("the workspace")
    if og is not None:
        og.check("o")
    if sg is not None:
        sg.check("S_T")
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


def row_errors(x, ref):
    """Worst per-row (last axis) relative L2 error, rows weighed against max(their own norm, the
    tensor's RMS row norm) so that a near-zero row cannot dominate; and the largest absolute error
    relative to the largest reference magnitude."""
    x = np.asarray(x, dtype=np.float64).reshape(-1, x.shape[-1])
    ref = np.asarray(ref, dtype=np.float64).reshape(-1, ref.shape[-1])
    if ref.size == 0:
        return 0.0, 0.0
    rn = np.linalg.norm(ref, axis=1)
    floor = np.sqrt(np.mean(rn ** 2))
    den = np.maximum(rn, floor if floor > 0 else 1.0)
    row = float(np.max(np.linalg.norm(x - ref, axis=1) / den))
    mx = float(np.max(np.abs(x - ref)) / max(float(np.max(np.abs(ref))), 1e-30))
    return row, mx


ROW_FACTOR = 4.0      # a single (token, head) row may be this much worse than the tensor-level bound


def check_chunk(oracle, d, tol, scale=1.0, per_seq=True, verbose=False, **kw):
    """Runs both sides and asserts rel-L2 <= tol on o and S_T (per sequence for packed batches),
    and that no single row of o (token, head) or of S_T (sequence, head, dk row) is off by more
    than ROW_FACTOR * tol, nor any element by more than ROW_FACTOR * tol of the largest magnitude."""
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
    ro, mo = row_errors(o, o_ref)
    rs, msx = row_errors(S_T, S_ref)
    errs.update({"o_row_max": ro, "o_max_abs": mo, "S_row_max": rs, "S_max_abs": msx})
    if verbose:
        print("errors:", {n: float("%.3g" % e) for n, e in errs.items()
                          if n in ("o", "S_T", "o_row_max", "o_max_abs", "S_row_max", "S_max_abs")})
    lim = ROW_FACTOR * tol
    assert ro <= lim and rs <= lim, "a row is off by more than %g: o %.3g, S_T %.3g" % (lim, ro, rs)
    assert mo <= lim and msx <= lim, "an element is off by more than %g of the largest magnitude: " \
                                     "o %.3g, S_T %.3g" % (lim, mo, msx)
    return errs
