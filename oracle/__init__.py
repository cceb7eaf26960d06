"""KDA oracle package: TEST INFRASTRUCTURE ONLY.

A plain, slow CPU statement of what the KDA hot path computes, in fp64:

* ``recurrence`` / ``decode_step`` call ``kda_oracle.c``, the token-by-token recurrence of
  Section 3, Eq. 1 of the Kimi Linear paper.  This is the oracle.
* ``dplr_recurrence`` is the general diagonal-plus-low-rank recurrence of Section 6.1 ("Relation
  to DPLR"), the paper's comparison workload, in the same plain form (``kda_oracle.c``).
* ``backward`` is the adjoint of that recurrence (gradients of Eq. 1), also in ``kda_oracle.c``.
* ``chunkwise.chunk_kda_np`` is a second, independent numpy statement of the chunkwise algorithm of
  Section 3.1 (WY representation + UT transform + chunk state update + output equation).  It is a
  cross-check of the oracle, not the oracle.

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may import this package.
It shares nothing with the CUDA path and never imports it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kda_oracle.c")
_SO = os.path.join(_HERE, "libkda_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile ``kda_oracle.c`` with gcc (fp64, OpenMP over (sequence, head)); returns the .so path."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            f32p = ctypes.POINTER(ctypes.c_float)
            f64p = ctypes.POINTER(ctypes.c_double)
            lib.kda_oracle_recurrence.restype = ctypes.c_int
            lib.kda_oracle_recurrence.argtypes = [
                f32p, f32p, f32p, f32p, f32p, f64p, f64p, f64p,
                ctypes.POINTER(ctypes.c_int64), ctypes.c_int, ctypes.c_int, ctypes.c_int,
                ctypes.c_int, ctypes.c_double, ctypes.c_int]
            lib.kda_oracle_decode_step.restype = ctypes.c_int
            lib.kda_oracle_decode_step.argtypes = [
                f32p, f32p, f32p, f32p, f32p, f64p, ctypes.POINTER(ctypes.c_int32), f64p,
                ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double,
                ctypes.c_int]
            lib.kda_oracle_dplr_recurrence.restype = ctypes.c_int
            lib.kda_oracle_dplr_recurrence.argtypes = [
                f32p, f32p, f32p, f32p, f32p, f32p, f64p, f64p, f64p,
                ctypes.POINTER(ctypes.c_int64), ctypes.c_int, ctypes.c_int, ctypes.c_int,
                ctypes.c_int, ctypes.c_double, ctypes.c_int]
            lib.kda_oracle_backward.restype = ctypes.c_int
            lib.kda_oracle_backward.argtypes = [
                f32p, f32p, f32p, f32p, f32p, f64p, f64p, f64p, f64p, f64p, f64p, f64p, f64p, f64p,
                ctypes.POINTER(ctypes.c_int64), ctypes.c_int, ctypes.c_int, ctypes.c_int,
                ctypes.c_int, ctypes.c_double, ctypes.c_int]
            lib.kda_oracle_max_threads.restype = ctypes.c_int
            _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().kda_oracle_max_threads())


def _f32(x, shape=None):
    if x is None:
        return None
    a = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    if shape is not None:
        assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _ptr(a, ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def recurrence(q, k, v, log_alpha, beta, S0=None, cu_seqlens=None, scale=1.0,
               want_o=True, want_state=True, n_threads=0):
    """Eq. 1 applied token by token in fp64.

    q, k, log_alpha: [T,H,dk]; v: [T,H,dv]; beta: [T,H]; S0: [N,H,dk,dv] or None (zeros);
    cu_seqlens: [N+1] token offsets or None (one sequence).  Values are taken as float32 (bf16
    inputs must be widened by the caller, which is exact).  Returns (o [T,H,dv] fp64 or None,
    S_T [N,H,dk,dv] fp64 or None).
    """
    k = _f32(k)
    T, H, dk = k.shape
    v = _f32(v)
    dv = v.shape[-1]
    assert v.shape == (T, H, dv)
    q = _f32(q, (T, H, dk)) if q is not None else None
    log_alpha = _f32(log_alpha, (T, H, dk))
    beta = _f32(beta, (T, H))
    if cu_seqlens is None:
        cu = np.array([0, T], dtype=np.int64)
    else:
        cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int64))
        assert cu[0] == 0 and cu[-1] == T and np.all(np.diff(cu) >= 0)
    N = cu.shape[0] - 1
    S0a = None
    if S0 is not None:
        S0a = np.ascontiguousarray(np.asarray(S0, dtype=np.float64))
        assert S0a.shape == (N, H, dk, dv)
    if want_o:
        assert q is not None
    o = np.empty((T, H, dv), dtype=np.float64) if want_o else None
    S_T = np.empty((N, H, dk, dv), dtype=np.float64) if want_state else None
    rc = _load().kda_oracle_recurrence(
        _ptr(q, ctypes.c_float), _ptr(k, ctypes.c_float), _ptr(v, ctypes.c_float),
        _ptr(log_alpha, ctypes.c_float), _ptr(beta, ctypes.c_float),
        _ptr(S0a, ctypes.c_double), _ptr(o, ctypes.c_double), _ptr(S_T, ctypes.c_double),
        _ptr(cu, ctypes.c_int64), N, H, dk, dv, float(scale), int(n_threads))
    if rc != 0:
        raise RuntimeError("kda_oracle_recurrence failed")
    return o, S_T


def dplr_recurrence(q, k, v, a, b, g, S0=None, cu_seqlens=None, scale=1.0, want_o=True,
                    want_state=True, n_threads=0):
    """The general diagonal-plus-low-rank recurrence (Section 6.1, "Relation to DPLR") token by
    token in fp64:  S_t = (Diag(exp(g_t)) + b_t a_t^T) S_{t-1} + k_t v_t^T,  o_t = scale S_t^T q_t.

    q, k, a, b, g: [T,H,dk]; v: [T,H,dv]; S0: [N,H,dk,dv] or None; cu_seqlens as in
    ``recurrence``.  Returns (o or None, S_T or None) in fp64.
    """
    k = _f32(k)
    T, H, dk = k.shape
    v = _f32(v)
    dv = v.shape[-1]
    q = _f32(q, (T, H, dk)) if q is not None else None
    a = _f32(a, (T, H, dk))
    b = _f32(b, (T, H, dk))
    g = _f32(g, (T, H, dk))
    if cu_seqlens is None:
        cu = np.array([0, T], dtype=np.int64)
    else:
        cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int64))
        assert cu[0] == 0 and cu[-1] == T and np.all(np.diff(cu) >= 0)
    N = cu.shape[0] - 1
    S0a = None
    if S0 is not None:
        S0a = np.ascontiguousarray(np.asarray(S0, dtype=np.float64))
        assert S0a.shape == (N, H, dk, dv)
    if want_o:
        assert q is not None
    o = np.empty((T, H, dv), dtype=np.float64) if want_o else None
    S_T = np.empty((N, H, dk, dv), dtype=np.float64) if want_state else None
    rc = _load().kda_oracle_dplr_recurrence(
        _ptr(q, ctypes.c_float), _ptr(k, ctypes.c_float), _ptr(v, ctypes.c_float),
        _ptr(a, ctypes.c_float), _ptr(b, ctypes.c_float), _ptr(g, ctypes.c_float),
        _ptr(S0a, ctypes.c_double), _ptr(o, ctypes.c_double), _ptr(S_T, ctypes.c_double),
        _ptr(cu, ctypes.c_int64), N, H, dk, dv, float(scale), int(n_threads))
    if rc != 0:
        raise RuntimeError("kda_oracle_dplr_recurrence failed")
    return o, S_T


def backward(q, k, v, log_alpha, beta, d_o=None, dS_T=None, S0=None, cu_seqlens=None, scale=1.0,
             n_threads=0):
    """Gradients of Eq. 1 for L = sum_t <d_o_t, o_t> + <dS_T, S_T>, by the adjoint of the
    token-by-token recurrence in fp64 (``kda_oracle_backward``).  Shapes as in ``recurrence``; d_o
    [T,H,dv] and dS_T [N,H,dk,dv] may be None (zeros).  Returns a dict with dq, dk, dlog_alpha
    [T,H,dk], dv [T,H,dv], dbeta [T,H], dS0 [N,H,dk,dv], all fp64."""
    k = _f32(k)
    T, H, dk = k.shape
    v = _f32(v)
    dv = v.shape[-1]
    q = _f32(q, (T, H, dk))
    log_alpha = _f32(log_alpha, (T, H, dk))
    beta = _f32(beta, (T, H))
    if cu_seqlens is None:
        cu = np.array([0, T], dtype=np.int64)
    else:
        cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int64))
        assert cu[0] == 0 and cu[-1] == T and np.all(np.diff(cu) >= 0)
    N = cu.shape[0] - 1

    def f64(x, shape):
        if x is None:
            return None
        a = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
        assert a.shape == tuple(shape), (a.shape, shape)
        return a
    S0a, doa, dSa = f64(S0, (N, H, dk, dv)), f64(d_o, (T, H, dv)), f64(dS_T, (N, H, dk, dv))
    out = {"dq": np.empty((T, H, dk)), "dk": np.empty((T, H, dk)), "dv": np.empty((T, H, dv)),
           "dlog_alpha": np.empty((T, H, dk)), "dbeta": np.empty((T, H)), "dS0": np.empty((N, H, dk, dv))}
    rc = _load().kda_oracle_backward(
        _ptr(q, ctypes.c_float), _ptr(k, ctypes.c_float), _ptr(v, ctypes.c_float),
        _ptr(log_alpha, ctypes.c_float), _ptr(beta, ctypes.c_float), _ptr(S0a, ctypes.c_double),
        _ptr(doa, ctypes.c_double), _ptr(dSa, ctypes.c_double),
        _ptr(out["dq"], ctypes.c_double), _ptr(out["dk"], ctypes.c_double), _ptr(out["dv"], ctypes.c_double),
        _ptr(out["dlog_alpha"], ctypes.c_double), _ptr(out["dbeta"], ctypes.c_double),
        _ptr(out["dS0"], ctypes.c_double), _ptr(cu, ctypes.c_int64), N, H, dk, dv, float(scale),
        int(n_threads))
    if rc != 0:
        raise RuntimeError("kda_oracle_backward failed")
    return out


def decode_step(q, k, v, log_alpha, beta, S, state_slot=None, scale=1.0, n_threads=0):
    """One token of Eq. 1 per (sequence, head); ``S`` ([n_slots,H,dk,dv] float64, C-contiguous)
    is updated in place.  Returns o [N,H,dv] fp64."""
    k = _f32(k)
    N, H, dk = k.shape
    v = _f32(v)
    dv = v.shape[-1]
    q = _f32(q, (N, H, dk))
    log_alpha = _f32(log_alpha, (N, H, dk))
    beta = _f32(beta, (N, H))
    assert isinstance(S, np.ndarray) and S.dtype == np.float64 and S.flags.c_contiguous
    assert S.shape[1:] == (H, dk, dv)
    slot = None
    if state_slot is not None:
        slot = np.ascontiguousarray(np.asarray(state_slot, dtype=np.int32))
        assert slot.shape == (N,) and slot.min() >= 0 and slot.max() < S.shape[0]
    else:
        assert S.shape[0] >= N
    o = np.empty((N, H, dv), dtype=np.float64)
    rc = _load().kda_oracle_decode_step(
        _ptr(q, ctypes.c_float), _ptr(k, ctypes.c_float), _ptr(v, ctypes.c_float),
        _ptr(log_alpha, ctypes.c_float), _ptr(beta, ctypes.c_float), _ptr(S, ctypes.c_double),
        _ptr(slot, ctypes.c_int32), _ptr(o, ctypes.c_double), N, H, dk, dv, float(scale),
        int(n_threads))
    if rc != 0:
        raise RuntimeError("kda_oracle_decode_step failed")
    return o
