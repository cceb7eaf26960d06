"""ctypes binding of ``include/kda.h``: argument marshalling only.

Every function has the name and argument order of its C entry point; tensors are ``torch`` tensors
(used for device memory and streams only) whose ``data_ptr()`` is passed through.  Nothing is
computed here, and there is no fallback: if ``libkda_b200.so`` is missing or does not load, the
first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

KDA_F32 = 0
KDA_BF16 = 1
_STATUS = {0: "KDA_OK", 1: "KDA_ERR_INVALID_ARG", 2: "KDA_ERR_UNSUPPORTED", 3: "KDA_ERR_WORKSPACE",
           4: "KDA_ERR_CUDA", 5: "KDA_ERR_TIMEOUT", 6: "KDA_ERR_GATE_RANGE"}

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libkda_b200.so")
_lib = None


class KdaError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__("%s: %s" % (_STATUS.get(code, str(code)), msg))
        self.code = code


def library_path() -> str:
    return _LIB_PATH


def load():
    """Loads the CUDA library (built by ``paper_2510_26692_b200.build``); raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError("libkda_b200.so not found at %s: run `python -m "
                          "paper_2510_26692_b200.build` (needs nvcc); there is no fallback path"
                          % _LIB_PATH)
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, i64, f32, sz = (ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float,
                             ctypes.c_size_t)
    lib.kda_chunk_fwd_workspace_bytes.restype = sz
    lib.kda_chunk_fwd_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, i32, i32]
    lib.kda_chunk_fwd_min_workspace_bytes.restype = sz
    lib.kda_chunk_fwd_min_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, i32, i32]
    lib.kda_chunk_fwd.restype = i32
    lib.kda_chunk_fwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i64, i32, i32, i32,
                                  i32, f32, i32, vp, sz, vp]
    lib.kda_chunk_fwd_static_max_bytes.restype = sz
    lib.kda_chunk_fwd_static_max_bytes.argtypes = []
    lib.kda_chunk_fwd_static_check_status.restype = i32
    lib.kda_chunk_fwd_static_check_status.argtypes = [vp]
    lib.kda_chunk_fwd_static.restype = i32
    lib.kda_chunk_fwd_static.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i64, i32, i32,
                                         i32, i32, f32, i32, vp]
    lib.kda_dplr_chunk_fwd_workspace_bytes.restype = sz
    lib.kda_dplr_chunk_fwd_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, i32]
    lib.kda_dplr_chunk_fwd_min_workspace_bytes.restype = sz
    lib.kda_dplr_chunk_fwd_min_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, i32]
    lib.kda_dplr_chunk_fwd.restype = i32
    lib.kda_dplr_chunk_fwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i64, i32, i32,
                                       i32, i32, f32, vp, sz, vp]
    lib.kda_chunk_bwd_workspace_bytes.restype = sz
    lib.kda_chunk_bwd_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, i32]
    lib.kda_chunk_bwd.restype = i32
    lib.kda_chunk_bwd.argtypes = [vp] * 16 + [i32, i64, i32, i32, i32, i32, f32, i32, vp, sz, vp]
    lib.kda_layer_fwd_workspace_bytes.restype = sz
    lib.kda_layer_fwd_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, i32]
    lib.kda_layer_fwd_min_workspace_bytes.restype = sz
    lib.kda_layer_fwd_min_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, i32]
    lib.kda_layer_set_fused_output.restype = i32
    lib.kda_layer_set_fused_output.argtypes = [i32]
    lib.kda_layer_fwd.restype = i32
    lib.kda_layer_fwd.argtypes = [vp] * 9 + [f32, f32, vp, vp, vp, vp, vp, i32, i64, i32, i32, i32, i32, f32,
                                             vp, sz, vp]
    lib.kda_layer_decode_step.restype = i32
    lib.kda_layer_decode_step.argtypes = [vp] * 9 + [f32, f32, vp, vp, vp, i32, i32, i32, i32, f32, vp]
    lib.kda_decode_step.restype = i32
    lib.kda_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, f32, i32, vp]
    lib.kda_decode_multi.restype = i32
    lib.kda_decode_multi.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, f32, i32, vp]
    lib.kda_chunk_fwd_host_workspace_bytes.restype = sz
    lib.kda_chunk_fwd_host_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, i32, i32]
    lib.kda_chunk_fwd_host.restype = i32
    lib.kda_chunk_fwd_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i64, i32, i32, i32,
                                       i32, f32, i32, vp, sz, vp]
    lib.kda_decode_step_host_workspace_bytes.restype = sz
    lib.kda_decode_step_host_workspace_bytes.argtypes = [i32, i32, i32, i32, i32]
    lib.kda_decode_step_host.restype = i32
    lib.kda_decode_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, f32,
                                         i32, vp, sz, vp]
    lib.kda_check_status.restype = i32
    lib.kda_check_status.argtypes = [vp, vp]
    lib.kda_selftest_wait_timeout.restype = i32
    lib.kda_selftest_wait_timeout.argtypes = [vp, i32, vp]
    lib.kda_profile_enable.restype = None
    lib.kda_profile_enable.argtypes = [i32]
    lib.kda_profile_read.restype = i32
    lib.kda_profile_read.argtypes = [i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i32)]
    lib.kda_last_error.restype = ctypes.c_char_p
    lib.kda_launch_count.restype = ctypes.c_uint64
    lib.kda_version.restype = ctypes.c_char_p
    lib.kda_set_chunk_path.restype = i32
    lib.kda_set_chunk_path.argtypes = [i32]
    _lib = lib
    return lib


def kda_last_error() -> str:
    return load().kda_last_error().decode()


def kda_launch_count() -> int:
    return int(load().kda_launch_count())


def kda_version() -> str:
    return load().kda_version().decode()


def kda_set_chunk_path(mode: int) -> None:
    """0 = automatic, 1 = always the two kernels, 2 = always the fused kernel (see kda.h)."""
    _check(load().kda_set_chunk_path(int(mode)))


def _check(rc: int):
    if rc != 0:
        raise KdaError(rc, kda_last_error())


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return KDA_BF16
    if t.dtype == torch.float32:
        return KDA_F32
    raise TypeError("q/k/v/o must be float32 or bfloat16, got %s" % t.dtype)


def _ptr(t: Optional[torch.Tensor], cuda: bool, dtype=None, name="tensor"):
    if t is None:
        return None
    if not isinstance(t, torch.Tensor):
        raise TypeError("%s must be a torch.Tensor" % name)
    if t.is_cuda != cuda:
        raise ValueError("%s must live on %s" % (name, "the GPU" if cuda else "the host"))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    if dtype is not None and t.dtype != dtype:
        raise TypeError("%s must be %s, got %s" % (name, dtype, t.dtype))
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def kda_chunk_fwd_workspace_bytes(total_tokens, n_seqs, H, dk=128, dv=128, chunk=64, dt=KDA_BF16):
    return int(load().kda_chunk_fwd_workspace_bytes(total_tokens, n_seqs, H, dk, dv, chunk, dt))


def kda_chunk_fwd_min_workspace_bytes(total_tokens, n_seqs, H, dk=128, dv=128, chunk=64,
                                      dt=KDA_BF16):
    return int(load().kda_chunk_fwd_min_workspace_bytes(total_tokens, n_seqs, H, dk, dv, chunk, dt))


def kda_chunk_fwd_host_workspace_bytes(total_tokens, n_seqs, H, dk=128, dv=128, chunk=64,
                                       dt=KDA_BF16):
    return int(load().kda_chunk_fwd_host_workspace_bytes(total_tokens, n_seqs, H, dk, dv, chunk, dt))


def kda_decode_step_host_workspace_bytes(n_seqs, H, dk=128, dv=128, dt=KDA_BF16):
    return int(load().kda_decode_step_host_workspace_bytes(n_seqs, H, dk, dv, dt))


def kda_chunk_fwd(q, k, v, log_alpha, beta, S0, o, S_T, cu_seqlens_dev, cu_seqlens_host, n_seqs,
                  total_tokens, H, dk, dv, chunk, scale, dt, workspace, workspace_bytes=None,
                  stream=None):
    """``kda_chunk_fwd`` of ``include/kda.h``; device tensors, ``cu_seqlens_host`` a CPU int32
    tensor.  Asynchronous on ``stream`` (default: torch's current stream)."""
    f32 = torch.float32
    et = torch.bfloat16 if dt == KDA_BF16 else torch.float32
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    rc = load().kda_chunk_fwd(
        _ptr(q, True, et, "q"), _ptr(k, True, et, "k"), _ptr(v, True, et, "v"),
        _ptr(log_alpha, True, f32, "log_alpha"), _ptr(beta, True, f32, "beta"),
        _ptr(S0, True, f32, "S0"), _ptr(o, True, et, "o"), _ptr(S_T, True, f32, "S_T"),
        _ptr(cu_seqlens_dev, True, torch.int32, "cu_seqlens_dev"),
        _ptr(cu_seqlens_host, False, torch.int32, "cu_seqlens_host"),
        int(n_seqs), int(total_tokens), int(H), int(dk), int(dv), int(chunk), float(scale), int(dt),
        _ptr(workspace, True, None, "workspace"), int(workspace_bytes), _stream(stream))
    _check(rc)


def kda_dplr_chunk_fwd_workspace_bytes(total_tokens, n_seqs, H, dk=128, dv=128, chunk=64) -> int:
    return int(load().kda_dplr_chunk_fwd_workspace_bytes(int(total_tokens), int(n_seqs), int(H), dk, dv, chunk))


def kda_dplr_chunk_fwd_min_workspace_bytes(total_tokens, n_seqs, H, dk=128, dv=128, chunk=64) -> int:
    return int(load().kda_dplr_chunk_fwd_min_workspace_bytes(int(total_tokens), int(n_seqs), int(H), dk, dv,
                                                             chunk))


def kda_dplr_chunk_fwd(q, k, v, a, b, g, S0, o, S_T, cu_seqlens_dev, cu_seqlens_host, n_seqs,
                       total_tokens, H, dk, dv, chunk, scale, workspace, workspace_bytes=None, stream=None):
    """``kda_dplr_chunk_fwd`` of ``include/kda.h`` (the general diagonal-plus-low-rank comparison
    workload, fp32 device tensors).  Asynchronous on ``stream``."""
    f32 = torch.float32
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    rc = load().kda_dplr_chunk_fwd(
        _ptr(q, True, f32, "q"), _ptr(k, True, f32, "k"), _ptr(v, True, f32, "v"),
        _ptr(a, True, f32, "a"), _ptr(b, True, f32, "b"), _ptr(g, True, f32, "g"),
        _ptr(S0, True, f32, "S0"), _ptr(o, True, f32, "o"), _ptr(S_T, True, f32, "S_T"),
        _ptr(cu_seqlens_dev, True, torch.int32, "cu_seqlens_dev"),
        _ptr(cu_seqlens_host, False, torch.int32, "cu_seqlens_host"),
        int(n_seqs), int(total_tokens), int(H), int(dk), int(dv), int(chunk), float(scale),
        _ptr(workspace, True, None, "workspace"), int(workspace_bytes), _stream(stream))
    _check(rc)


def kda_chunk_bwd_workspace_bytes(total_tokens, n_seqs, H, dk=128, dv=128, chunk=64) -> int:
    return int(load().kda_chunk_bwd_workspace_bytes(int(total_tokens), int(n_seqs), int(H), dk, dv, chunk))


def kda_chunk_bwd(q, k, v, log_alpha, beta, S0, d_o, dS_T, dq, dk_out, dv_out, dlog_alpha, dbeta, dS0,
                  cu_seqlens_dev, cu_seqlens_host, n_seqs, total_tokens, H, dk, dv, chunk, scale, dt,
                  workspace, workspace_bytes=None, stream=None):
    """``kda_chunk_bwd`` of ``include/kda.h``: gradients of the prefill operator (fp32 outputs).
    Asynchronous on ``stream``."""
    f32 = torch.float32
    et = torch.bfloat16 if dt == KDA_BF16 else torch.float32
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    rc = load().kda_chunk_bwd(
        _ptr(q, True, et, "q"), _ptr(k, True, et, "k"), _ptr(v, True, et, "v"),
        _ptr(log_alpha, True, f32, "log_alpha"), _ptr(beta, True, f32, "beta"), _ptr(S0, True, f32, "S0"),
        _ptr(d_o, True, et, "d_o"), _ptr(dS_T, True, f32, "dS_T"),
        _ptr(dq, True, f32, "dq"), _ptr(dk_out, True, f32, "dk"), _ptr(dv_out, True, f32, "dv"),
        _ptr(dlog_alpha, True, f32, "dlog_alpha"), _ptr(dbeta, True, f32, "dbeta"), _ptr(dS0, True, f32, "dS0"),
        _ptr(cu_seqlens_dev, True, torch.int32, "cu_seqlens_dev"),
        _ptr(cu_seqlens_host, False, torch.int32, "cu_seqlens_host"),
        int(n_seqs), int(total_tokens), int(H), int(dk), int(dv), int(chunk), float(scale), int(dt),
        _ptr(workspace, True, None, "workspace"), int(workspace_bytes), _stream(stream))
    _check(rc)


def kda_layer_set_fused_output(on: bool) -> None:
    """False: ``kda_layer_fwd`` runs its output stage as a separate pass (default: inside the
    inter-chunk kernel when the device can hold the clusters this needs)."""
    _check(load().kda_layer_set_fused_output(1 if on else 0))


def kda_layer_fwd_workspace_bytes(total_tokens, n_seqs, H, dk=128, dv=128, chunk=64) -> int:
    return int(load().kda_layer_fwd_workspace_bytes(int(total_tokens), int(n_seqs), int(H), dk, dv, chunk))


def kda_layer_fwd_min_workspace_bytes(total_tokens, n_seqs, H, dk=128, dv=128, chunk=64) -> int:
    return int(load().kda_layer_fwd_min_workspace_bytes(int(total_tokens), int(n_seqs), int(H), dk, dv, chunk))


def kda_layer_fwd(q_c, k_c, v, g_a, b_pre, g_o, A_log, dt_bias, rms_weight, l2_eps, rms_eps, S0, y, S_T,
                  cu_seqlens_dev, cu_seqlens_host, n_seqs, total_tokens, H, dk, dv, chunk, scale, workspace,
                  workspace_bytes=None, stream=None):
    """``kda_layer_fwd`` of ``include/kda.h``: the operator with L2Norm, decay function, beta
    sigmoid, head-wise RMSNorm and output gate, from bf16 pre-activations.  Asynchronous."""
    f32, bf = torch.float32, torch.bfloat16
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    rc = load().kda_layer_fwd(
        _ptr(q_c, True, bf, "q_c"), _ptr(k_c, True, bf, "k_c"), _ptr(v, True, bf, "v"), _ptr(g_a, True, bf, "g_a"),
        _ptr(b_pre, True, f32, "b_pre"), _ptr(g_o, True, bf, "g_o"), _ptr(A_log, True, f32, "A_log"),
        _ptr(dt_bias, True, f32, "dt_bias"), _ptr(rms_weight, True, f32, "rms_weight"), float(l2_eps),
        float(rms_eps), _ptr(S0, True, f32, "S0"), _ptr(y, True, bf, "y"), _ptr(S_T, True, f32, "S_T"),
        _ptr(cu_seqlens_dev, True, torch.int32, "cu_seqlens_dev"),
        _ptr(cu_seqlens_host, False, torch.int32, "cu_seqlens_host"),
        int(n_seqs), int(total_tokens), int(H), int(dk), int(dv), int(chunk), float(scale),
        _ptr(workspace, True, None, "workspace"), int(workspace_bytes), _stream(stream))
    _check(rc)


def kda_layer_decode_step(q_c, k_c, v, g_a, b_pre, g_o, A_log, dt_bias, rms_weight, l2_eps, rms_eps, S,
                          state_slot, y, n_seqs, H, dk, dv, scale, stream=None):
    """``kda_layer_decode_step`` of ``include/kda.h``: one decode token per sequence with the layer's
    element-wise stages inside the kernel (bf16 activations, fp32 state in place)."""
    f32, bf = torch.float32, torch.bfloat16
    rc = load().kda_layer_decode_step(
        _ptr(q_c, True, bf, "q_c"), _ptr(k_c, True, bf, "k_c"), _ptr(v, True, bf, "v"), _ptr(g_a, True, bf, "g_a"),
        _ptr(b_pre, True, f32, "b_pre"), _ptr(g_o, True, bf, "g_o"), _ptr(A_log, True, f32, "A_log"),
        _ptr(dt_bias, True, f32, "dt_bias"), _ptr(rms_weight, True, f32, "rms_weight"), float(l2_eps),
        float(rms_eps), _ptr(S, True, f32, "S"), _ptr(state_slot, True, torch.int32, "state_slot"),
        _ptr(y, True, bf, "y"), int(n_seqs), int(H), int(dk), int(dv), float(scale), _stream(stream))
    _check(rc)


def kda_chunk_fwd_static_max_bytes() -> int:
    return int(load().kda_chunk_fwd_static_max_bytes())


def kda_chunk_fwd_static(q, k, v, log_alpha, beta, S0, o, S_T, cu_seqlens_dev, cu_seqlens_host,
                         n_seqs, total_tokens, H, dk, dv, chunk, scale, dt, stream=None):
    """``kda_chunk_fwd_static``: the prefill for callers that may not allocate device memory (a
    fixed-pool serving loop, a plug-in without an allocator).  Takes no workspace: the scratch is a
    16 MiB array inside the library, shared by all calls on the device, so calls that overlap on
    the GPU must be serialised; calls that need more scratch raise ``KdaError``
    (KDA_ERR_WORKSPACE).  The first call on a device does a one-time address look-up and should
    come before any stream capture."""
    f32 = torch.float32
    et = torch.bfloat16 if dt == KDA_BF16 else torch.float32
    rc = load().kda_chunk_fwd_static(
        _ptr(q, True, et, "q"), _ptr(k, True, et, "k"), _ptr(v, True, et, "v"),
        _ptr(log_alpha, True, f32, "log_alpha"), _ptr(beta, True, f32, "beta"),
        _ptr(S0, True, f32, "S0"), _ptr(o, True, et, "o"), _ptr(S_T, True, f32, "S_T"),
        _ptr(cu_seqlens_dev, True, torch.int32, "cu_seqlens_dev"),
        _ptr(cu_seqlens_host, False, torch.int32, "cu_seqlens_host"),
        int(n_seqs), int(total_tokens), int(H), int(dk), int(dv), int(chunk), float(scale), int(dt),
        _stream(stream))
    _check(rc)


def kda_decode_step(q, k, v, log_alpha, beta, S, state_slot, o, n_seqs, H, dk, dv, scale, dt,
                    stream=None):
    """``kda_decode_step`` of ``include/kda.h``; ``S`` is updated in place."""
    f32 = torch.float32
    et = torch.bfloat16 if dt == KDA_BF16 else torch.float32
    rc = load().kda_decode_step(
        _ptr(q, True, et, "q"), _ptr(k, True, et, "k"), _ptr(v, True, et, "v"),
        _ptr(log_alpha, True, f32, "log_alpha"), _ptr(beta, True, f32, "beta"),
        _ptr(S, True, f32, "S"), _ptr(state_slot, True, torch.int32, "state_slot"),
        _ptr(o, True, et, "o"), int(n_seqs), int(H), int(dk), int(dv), float(scale), int(dt),
        _stream(stream))
    _check(rc)


def kda_decode_multi(q, k, v, log_alpha, beta, S, state_slot, o, n_seqs, n_tokens, H, dk, dv, scale,
                     dt, stream=None):
    """``kda_decode_multi`` of ``include/kda.h``: ``n_tokens`` tokens per sequence, ``S`` in place."""
    f32 = torch.float32
    et = torch.bfloat16 if dt == KDA_BF16 else torch.float32
    rc = load().kda_decode_multi(
        _ptr(q, True, et, "q"), _ptr(k, True, et, "k"), _ptr(v, True, et, "v"),
        _ptr(log_alpha, True, f32, "log_alpha"), _ptr(beta, True, f32, "beta"),
        _ptr(S, True, f32, "S"), _ptr(state_slot, True, torch.int32, "state_slot"),
        _ptr(o, True, et, "o"), int(n_seqs), int(n_tokens), int(H), int(dk), int(dv), float(scale),
        int(dt), _stream(stream))
    _check(rc)


def kda_chunk_fwd_host(q, k, v, log_alpha, beta, S0, o, S_T, cu_seqlens_host, n_seqs, total_tokens,
                       H, dk, dv, chunk, scale, dt, workspace, workspace_bytes=None, stream=None):
    """``kda_chunk_fwd_host``: q..S_T are HOST tensors (pinned for asynchronous copies),
    ``workspace`` a device tensor."""
    f32 = torch.float32
    et = torch.bfloat16 if dt == KDA_BF16 else torch.float32
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    rc = load().kda_chunk_fwd_host(
        _ptr(q, False, et, "q"), _ptr(k, False, et, "k"), _ptr(v, False, et, "v"),
        _ptr(log_alpha, False, f32, "log_alpha"), _ptr(beta, False, f32, "beta"),
        _ptr(S0, False, f32, "S0"), _ptr(o, False, et, "o"), _ptr(S_T, False, f32, "S_T"),
        _ptr(cu_seqlens_host, False, torch.int32, "cu_seqlens_host"),
        int(n_seqs), int(total_tokens), int(H), int(dk), int(dv), int(chunk), float(scale), int(dt),
        _ptr(workspace, True, None, "workspace"), int(workspace_bytes), _stream(stream))
    _check(rc)


def kda_decode_step_host(q, k, v, log_alpha, beta, S_dev, state_slot_host, o, n_seqs, H, dk, dv,
                         scale, dt, workspace, workspace_bytes=None, stream=None):
    """``kda_decode_step_host``: per-token inputs and ``o`` on the host, states on the device."""
    f32 = torch.float32
    et = torch.bfloat16 if dt == KDA_BF16 else torch.float32
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    rc = load().kda_decode_step_host(
        _ptr(q, False, et, "q"), _ptr(k, False, et, "k"), _ptr(v, False, et, "v"),
        _ptr(log_alpha, False, f32, "log_alpha"), _ptr(beta, False, f32, "beta"),
        _ptr(S_dev, True, f32, "S"), _ptr(state_slot_host, False, torch.int32, "state_slot"),
        _ptr(o, False, et, "o"), int(n_seqs), int(H), int(dk), int(dv), float(scale), int(dt),
        _ptr(workspace, True, None, "workspace"), int(workspace_bytes), _stream(stream))
    _check(rc)


def kda_selftest_wait_timeout(workspace, limit_ms: int = 20, stream=None):
    """``kda_selftest_wait_timeout``: makes one bounded device-side wait run out; afterwards
    ``kda_check_status(workspace)`` raises ``KdaError`` with KDA_ERR_TIMEOUT."""
    _check(load().kda_selftest_wait_timeout(_ptr(workspace, True, None, "workspace"), int(limit_ms),
                                            _stream(stream)))


def kda_profile_enable(on: bool):
    load().kda_profile_enable(1 if on else 0)


def kda_profile_read(kind: int):
    """Returns (total_ms, launches) of one kernel kind (0 prologue, 1 intra, 2 inter, 3 decode)."""
    ms = ctypes.c_double(0.0)
    n = ctypes.c_int(0)
    _check(load().kda_profile_read(int(kind), ctypes.byref(ms), ctypes.byref(n)))
    return ms.value, n.value


def kda_check_status(workspace, stream=None):
    _check(load().kda_check_status(_ptr(workspace, True, None, "workspace"), _stream(stream)))


def kda_chunk_fwd_static_check_status(stream=None):
    """Reads and clears the status word of the library's built-in scratch (the counterpart of
    ``kda_check_status`` for ``kda_chunk_fwd_static`` calls); synchronises the stream."""
    _check(load().kda_chunk_fwd_static_check_status(_stream(stream)))
