#!/usr/bin/env python
"""Benchmark of the KDA hot path on B200.

One "step" is one pass of the prefill hot path, ``kda_chunk_fwd`` on the bf16 prefill workload
(B=1, T=4096, H=32, dk=dv=128, chunk 64, S0 ~ N(0,0.02)); the decode workload (256 sequences x 32
heads, 64 consecutive in-place steps) is timed in the same run and reported under ``"decode"``.

    python bench.py [--gpus N] [--steps K] [--warmup W]            # this library
    python bench.py --impl reference ...                             # the fp64 CPU oracle, timed

For N > 1 the script is launched by torchrun, one rank per GPU; every rank runs its own batch of
the same shape (sequences and heads are independent, so there is no collective on the data path)
and the reported value is the sum over ranks divided by the slowest rank's time.  Prints one JSON
line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

T_PREFILL, H, D, CHUNK = 4096, 32, 128, 64
DEC_SEQS, DEC_STEPS = 256, 64
METRIC = "KDA prefill tokens/s (H=32,d=128)"
# algorithmic HBM bytes per token and head of the bf16 prefill path: q,k,v 3x256 + gates 512 +
# beta 4 + o 256; plus S0 and S_T (2 x 64 KiB) per (sequence, head)
BYTES_PER_TOKEN_HEAD = 1540
STATE_BYTES = 2 * D * D * 4
# decode: state read + written, q,k,v,o bf16, gates fp32, beta
DEC_BYTES_PER_STATE = 2 * D * D * 4 + 4 * D * 2 + D * 4 + 4
FLOPS_PER_TOKEN_HEAD = 6 * D * D + 3 * CHUNK * D + CHUNK * CHUNK   # the paper's FLOPs model
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (prefill: intra 168.4 + 98.7 MB, inter 156.3 + 20.0 MB, fused kernel 170.8 + 33.6 MB;
# decode: 547.4 + 484.7 MB)
PREFILL_DRAM_TRAFFIC = {"intra_chunk": 267.1e6, "inter_chunk": 176.3e6}
DECODE_DRAM_TRAFFIC = 1032.1e6
FUSED_DRAM_TRAFFIC = 204.4e6
TRAFFIC_SOURCE = "ncu dram__bytes_read.sum + dram__bytes_write.sum per launch, copied from the summaries under profiles/ (not measured in this run)"
MIN_TIMED_S = 0.5      # the timed region is extended (whole blocks of `steps` calls) to at least this
MAX_BLOCKS = 2000


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            m = json.load(f)
        return {"hbm_gbs": float(m["hbm_gbs"]), "bf16_tflops": float(m["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def _sample(self):
        nv = self.nv
        self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
        try:
            r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
        except Exception:
            r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
                 0x4: "sw_power_cap", 0x80: "hw_power_brake"}
        for bit, name in names.items():
            if r & bit:
                self.reasons.add(name)

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            try:
                self._sample()
            except Exception:
                break
            time.sleep(self.period)

    def finish(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join()
        if self.ok and not self.samples:
            try:
                self._sample()
            except Exception:
                pass
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def reduce_max(x: float, world: int, device=None) -> float:
    """Max of a per-rank scalar over all ranks (the slowest rank defines the step time)."""
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms_per_step: float) -> float:
    """Units per second of the whole job: every rank processes `units_per_rank` per step."""
    return world * units_per_rank / (ms_per_step * 1e-3)


def oracle_arm(args, rank):
    """--impl reference: the fp64 oracle as it stands on the host cores, on the prefill workload."""
    if rank != 0:
        return 0
    import torch
    import oracle
    from paper_2510_26692_b200 import inputs
    oracle.build()
    d = inputs.chunk_inputs([T_PREFILL], H=H, dtype=torch.bfloat16, seed=1, s0_std=0.02)
    a = {n: (None if t is None else t.float().numpy()) for n, t in d.items()
         if n not in ("cu_seqlens",)}
    S0 = d["S0"].double().numpy()
    cores = oracle.max_threads()

    def step():
        oracle.recurrence(a["q"], a["k"], a["v"], a["log_alpha"], a["beta"], S0=S0)

    for _ in range(min(args.warmup, 2)):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    val = T_PREFILL / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": min(args.warmup, 2), "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": "prefill B=1 T=4096 H=32 dk=dv=128 chunk=64 bf16 q/k/v, S0~N(0,0.02)",
                   "sample": "whole workload each step"},
        "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                         "sample": "whole prefill workload (4096 tokens x 32 heads) per step"},
        "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def extra_workloads(K, inputs, torch, dev, peaks):
    """Device-resident timing of the packed varlen batch (the packed-batch workload) and of the 1 Mi-token
    state-only prefill; inputs are far larger than L2, so no rotation is needed."""
    out = {}
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, reps):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(reps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    # varlen: 16 sequences, lengths uniform on [512, 16384]
    lens = inputs.varlen_lengths(16, 512, 16384, seed=2)
    d = inputs.chunk_inputs(lens, H=H, dtype=torch.bfloat16, seed=2, s0_std=0.02, device=dev)
    T = sum(lens)
    cu_host = d["cu_seqlens"]
    cu_dev = cu_host.to(dev)
    nb = K.kda_chunk_fwd_workspace_bytes(T, 16, H, D, D, CHUNK, K.KDA_BF16)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    o = torch.empty((T, H, D), dtype=torch.bfloat16, device=dev)
    S_T = torch.empty((16, H, D, D), dtype=torch.float32, device=dev)
    ms = timed(lambda: K.kda_chunk_fwd(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["S0"], o,
                                       S_T, cu_dev, cu_host, 16, T, H, D, D, CHUNK, 1.0, K.KDA_BF16,
                                       ws, nb, stream), 10)
    nbytes = T * H * BYTES_PER_TOKEN_HEAD + 16 * H * STATE_BYTES
    out["varlen_16seq"] = {"workload": "16 packed sequences, lengths uniform on [512, 16384], H=32, bf16, per-sequence S0",
                           "total_tokens": T, "lengths": lens, "ms": ms, "tokens_per_s": T / (ms * 1e-3),
                           "algorithmic_bytes": nbytes, "achieved_gbs": nbytes / (ms * 1e-3) / 1e9,
                           "frac": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None,
                           "traffic_note": "not captured: the workload is above the size an ncu capture is kept to"}
    del d, ws, o, S_T
    torch.cuda.empty_cache()

    # long context: 1 Mi tokens, final state only (o = NULL, q unused)
    T = 1 << 20
    d = inputs.chunk_inputs_slabbed(T, H, seed=3, gate_mean=6.0, s0_std=0.02, device=dev, want_q=False)
    nb = K.kda_chunk_fwd_workspace_bytes(T, 1, H, D, D, CHUNK, K.KDA_BF16)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    S_T = torch.empty((1, H, D, D), dtype=torch.float32, device=dev)
    ms = timed(lambda: K.kda_chunk_fwd(None, d["k"], d["v"], d["log_alpha"], d["beta"], d["S0"], None,
                                       S_T, None, None, 1, T, H, D, D, CHUNK, 1.0, K.KDA_BF16, ws, nb,
                                       stream), 3)
    nbytes = T * H * 1028 + H * STATE_BYTES     # k, v, gates, beta; no q, no o
    out["long_context_1Mi_state_only"] = {"workload": "B=1, T=1048576, H=32, bf16, gates logsigmoid(N(6,1)), final state only (o = NULL)",
                                          "total_tokens": T, "ms": ms, "tokens_per_s": T / (ms * 1e-3),
                                          "algorithmic_bytes": nbytes, "achieved_gbs": nbytes / (ms * 1e-3) / 1e9,
                                          "frac": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None,
                                          "traffic_note": "not captured: the workload is above the size an ncu capture is kept to"}
    del d, ws, S_T
    torch.cuda.empty_cache()
    return out


def dplr_comparison(K, inputs, torch, dev, peaks):
    """The paper's one kernel-level experiment (Section 3.2 kernel-time figure; Section 6.1): the
    general diagonal-plus-low-rank chunk forward against KDA at batch 1, 16 heads.  Both in the
    library's fp32 FMA style (same chunk length, same two-kernel structure), so the ratio shows what
    binding a and b to k saves; the tensor-core bf16 KDA path is listed beside them."""
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, reps=5):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(reps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    T, Hh = 16384, 16
    out = {"workload": "B=1, T=16384, H=16, dk=dv=128, chunk=64 (inputs 134 MB per tensor > L2); paper figure: "
                       "DPLR 14.89 ms / KDA 7.60 ms = 1.96 at this length (other hardware)"}
    d = inputs.dplr_inputs([T], H=Hh, seed=5, s0_std=0.02, device=dev)
    nb = K.kda_dplr_chunk_fwd_workspace_bytes(T, 1, Hh)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    o = torch.empty((T, Hh, D), dtype=torch.float32, device=dev)
    S_T = torch.empty((1, Hh, D, D), dtype=torch.float32, device=dev)
    ms_dplr = timed(lambda: K.kda_dplr_chunk_fwd(d["q"], d["k"], d["v"], d["a"], d["b"], d["g"], d["S0"], o, S_T,
                                                 None, None, 1, T, Hh, D, D, CHUNK, 1.0, ws, nb, stream))
    K.kda_check_status(ws)
    nbytes = T * Hh * 7 * 512 + Hh * STATE_BYTES
    out["dplr_fp32"] = {"ms": ms_dplr, "algorithmic_bytes": nbytes,
                        "frac": nbytes / (ms_dplr * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    del d, ws
    torch.cuda.empty_cache()
    d = inputs.chunk_inputs([T], H=Hh, dtype=torch.float32, seed=5, s0_std=0.02, device=dev)
    nb = K.kda_chunk_fwd_workspace_bytes(T, 1, Hh, D, D, CHUNK, K.KDA_F32)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    ms_kda = timed(lambda: K.kda_chunk_fwd(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["S0"], o, S_T,
                                           None, None, 1, T, Hh, D, D, CHUNK, 1.0, K.KDA_F32, ws, nb, stream))
    K.kda_check_status(ws)
    nbytes = T * Hh * (5 * 512 + 4) + Hh * STATE_BYTES
    out["kda_fp32"] = {"ms": ms_kda, "algorithmic_bytes": nbytes,
                       "frac": nbytes / (ms_kda * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    out["dplr_over_kda_fp32"] = ms_dplr / ms_kda
    del d, ws, o
    torch.cuda.empty_cache()
    d = inputs.chunk_inputs([T], H=Hh, dtype=torch.bfloat16, seed=5, s0_std=0.02, device=dev)
    nb = K.kda_chunk_fwd_workspace_bytes(T, 1, Hh, D, D, CHUNK, K.KDA_BF16)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    o = torch.empty((T, Hh, D), dtype=torch.bfloat16, device=dev)
    ms_tc = timed(lambda: K.kda_chunk_fwd(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["S0"], o, S_T,
                                          None, None, 1, T, Hh, D, D, CHUNK, 1.0, K.KDA_BF16, ws, nb, stream), 20)
    K.kda_check_status(ws)
    out["kda_bf16_tensor_core"] = {"ms": ms_tc}
    del d, ws, o, S_T
    torch.cuda.empty_cache()
    return out


def backward_figure(K, inputs, torch, dev, peaks):
    """Gradients of the prefill operator (kda_chunk_bwd) on the headline prefill workload: d_o and
    dS_T random, forward recomputed inside the call."""
    stream = torch.cuda.current_stream()
    T = T_PREFILL
    d = inputs.chunk_inputs([T], H=H, dtype=torch.bfloat16, seed=1, s0_std=0.02, device=dev)
    g = torch.Generator(device=dev).manual_seed(77)
    d_o = torch.randn((T, H, D), generator=g, device=dev).to(torch.bfloat16)
    dS_T = torch.randn((1, H, D, D), generator=g, device=dev)
    nb = K.kda_chunk_bwd_workspace_bytes(T, 1, H)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    outs = [torch.empty((T, H, D), dtype=torch.float32, device=dev) for _ in range(4)]
    db = torch.empty((T, H), dtype=torch.float32, device=dev)
    dS0 = torch.empty_like(dS_T)

    def call():
        K.kda_chunk_bwd(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["S0"], d_o, dS_T, outs[0], outs[1],
                        outs[2], outs[3], db, dS0, None, None, 1, T, H, D, D, CHUNK, 1.0, K.KDA_BF16, ws, nb,
                        stream)
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(5):
        call()
    e1.record(stream)
    torch.cuda.synchronize()
    K.kda_check_status(ws)
    ms = e0.elapsed_time(e1) / 5
    # q, k, v, d_o bf16 + log alpha, beta fp32 read; dq, dk, dv, dlog_alpha, dbeta fp32 written; states
    nbytes = T * H * (4 * 256 + 512 + 4 + 4 * 512 + 4) + 4 * H * D * D * 4
    return {"workload": "gradients of the prefill workload (B=1 T=4096 H=32, bf16 q/k/v/d_o, fp32 gradients)",
            "ms": ms, "tokens_per_s": T / (ms * 1e-3), "algorithmic_bytes": nbytes,
            "achieved_gbs": nbytes / (ms * 1e-3) / 1e9, "frac": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "note": "token-sequential adjoint in fp32 FMA (one CTA per sequence, head and 32-column slice): "
                    "bound by the 4096 dependent steps, not by memory"}


def layer_figure(K, inputs, torch, dev, peaks):
    """kda_layer_fwd on the headline prefill shape: L2Norm, decay function and beta sigmoid inside the
    intra-chunk kernel, RMSNorm and output gate as a pass over the bf16 output."""
    stream = torch.cuda.current_stream()
    T = T_PREFILL
    sets = [inputs.layer_inputs([T], H=H, seed=60 + i, s0_std=0.02, device=dev) for i in range(3)]   # > L2 in total
    nb = K.kda_layer_fwd_workspace_bytes(T, 1, H)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    y = torch.empty((T, H, D), dtype=torch.bfloat16, device=dev)
    S_T = torch.empty((1, H, D, D), dtype=torch.float32, device=dev)

    def call(d):
        K.kda_layer_fwd(d["q_c"], d["k_c"], d["v"], d["g_a"], d["b_pre"], d["g_o"], d["A_log"], d["dt_bias"], d["w"],
                        1e-6, 1e-5, d["S0"], y, S_T, None, None, 1, T, H, D, D, CHUNK, D ** -0.5, ws, nb, stream)
    for i in range(5):
        call(sets[i % 3])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 60
    e0.record(stream)
    for i in range(reps):
        call(sets[i % 3])
    e1.record(stream)
    torch.cuda.synchronize()
    K.kda_check_status(ws)
    ms = e0.elapsed_time(e1) / reps
    # q_c, k_c, v, g_a, g_o read and y written in bf16, b_pre fp32; the states in and out
    nbytes = T * H * (6 * 256 + 4) + H * STATE_BYTES
    return {"workload": "B=1 T=4096 H=32, bf16 pre-activations (q_c, k_c, v, g_a, g_o), fp32 b_pre; inputs rotate over 3 copies",
            "ms": ms, "tokens_per_s": T / (ms * 1e-3), "algorithmic_bytes": nbytes,
            "achieved_gbs": nbytes / (ms * 1e-3) / 1e9, "frac": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "note": "two kernels per call: intra-chunk with the prologue inside, inter-chunk with the output stage inside (clusters of the four slice CTAs)"}


def decode_only(args, K, inputs, torch, dev, peaks):
    """Short decode-only run (used under a profiler): one block of 64 in-place steps, timed."""
    dd = inputs.decode_inputs(DEC_SEQS, H, DEC_STEPS, seed=4)
    gd = {n: t.to(dev) for n, t in dd.items()}
    S = gd["S"].clone()
    od = torch.empty((DEC_STEPS, DEC_SEQS, H, D), dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for rep in range(2):
        if rep == 1:
            e0.record(stream)
        for s in range(DEC_STEPS):
            K.kda_decode_step(gd["q"][s], gd["k"][s], gd["v"][s], gd["log_alpha"][s], gd["beta"][s],
                              S, None, od[s], DEC_SEQS, H, D, D, 1.0, K.KDA_BF16, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / DEC_STEPS
    gbs = DEC_SEQS * H * DEC_BYTES_PER_STATE / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "KDA decode tokens/s", "value": DEC_SEQS / (ms * 1e-3),
                      "ms_per_step": ms, "achieved_gbs": gbs, "frac": gbs / peaks["hbm_gbs"],
                      "partial": "decode-only"}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--decode-reps", type=int, default=5)
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the packed-batch and 1 Mi-token workloads (they run by default)")
    ap.add_argument("--all-workloads", action="store_true",
                    help="also time the packed varlen batch (16 sequences) and the 1 Mi-token "
                         "state-only prefill; needs ~70 GB of device memory")
    ap.add_argument("--min-timed-s", type=float, default=MIN_TIMED_S,
                    help="repeat the block of --steps calls until this much device time is measured "
                         "(0: one block, for runs under a profiler)")
    ap.add_argument("--chunk-path", type=int, default=0, choices=[0, 1, 2],
                    help="kda_set_chunk_path mode for the timed prefill: 0 automatic, 1 two kernels, 2 fused kernel")
    ap.add_argument("--prefill-only", action="store_true",
                    help="time only the device-resident prefill loop (short runs under a profiler)")
    ap.add_argument("--only", default=None, choices=["layer", "backward", "dplr"],
                    help="run one of the side figures alone (layer wrap, backward pass, DPLR comparison) and "
                         "print it as a partial JSON line; for profiling")
    ap.add_argument("--decode-only", action="store_true",
                    help="time only the decode loop (short runs under a profiler)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        if args.steps > 20:
            args.steps = 20
        return oracle_arm(args, rank)
    args.warmup = max(args.warmup, 3)

    import torch
    import torch.distributed as dist
    import paper_2510_26692_b200 as K
    from paper_2510_26692_b200 import inputs

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the KDA library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        return reduce_max(x, world, dev)

    if args.decode_only:
        return decode_only(args, K, inputs, torch, dev, peaks)
    if args.only:
        fn = {"layer": layer_figure, "backward": backward_figure, "dplr": dplr_comparison}[args.only]
        out = fn(K, inputs, torch, dev, peaks)
        if rank == 0:
            print(json.dumps({"partial": args.only, "gpu_launches": K.kda_launch_count(), args.only: out}))
        return 0
    K.kda_set_chunk_path(args.chunk_path)

    # ---- prefill workload: 3 input copies (each 206 MB > L2) rotated between steps ---------------
    n_copies = 3
    copies = []
    for c in range(n_copies):
        d = inputs.chunk_inputs([T_PREFILL], H=H, dtype=torch.bfloat16, seed=1 + 100 * c + 1000 * rank,
                                s0_std=0.02)
        copies.append({n: (t.to(dev) if isinstance(t, torch.Tensor) else t) for n, t in d.items()})
    dt = K.KDA_BF16
    ws_bytes = K.kda_chunk_fwd_workspace_bytes(T_PREFILL, 1, H, D, D, CHUNK, dt)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    o = torch.empty((T_PREFILL, H, D), dtype=torch.bfloat16, device=dev)
    S_T = torch.empty((1, H, D, D), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()

    def prefill_step(i):
        g = copies[i % n_copies]
        K.kda_chunk_fwd(g["q"], g["k"], g["v"], g["log_alpha"], g["beta"], g["S0"], o, S_T, None,
                        None, 1, T_PREFILL, H, D, D, CHUNK, 1.0, dt, ws, ws_bytes, stream)

    for i in range(args.warmup):
        prefill_step(i)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    l0 = K.kda_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # The timed unit is a block of exactly `steps` calls between two events (barrier and
    # synchronize on both sides, max over ranks).  Blocks are repeated until at least
    # MIN_TIMED_S of device time has been measured, so that the clock sampler sees the load, and
    # the median block is reported (min and max beside it).
    block_ms = []
    while True:
        barrier()
        e0.record(stream)
        for i in range(args.steps):
            prefill_step(i)
        e1.record(stream)
        barrier()
        block_ms.append(max_over_ranks(e0.elapsed_time(e1)))
        if sum(block_ms) >= args.min_timed_s * 1e3 or len(block_ms) >= MAX_BLOCKS:
            break
    launches = K.kda_launch_count() - l0
    clocks = sampler.finish()
    srt = sorted(block_ms)
    ms_total = srt[len(srt) // 2]
    ms_step = ms_total / args.steps
    tokens_per_s = whole_job_rate(T_PREFILL, world, ms_step)
    timing = {"blocks": len(block_ms), "steps_per_block": args.steps, "reported": "median block",
              "ms_per_step_min": srt[0] / args.steps, "ms_per_step_max": srt[-1] / args.steps,
              "timed_region_ms": sum(block_ms)}

    # per-kernel durations (separate pass: the event pairs perturb back-to-back launches slightly)
    K.kda_profile_enable(True)
    nprof = min(args.steps, 20)
    for i in range(nprof):
        prefill_step(i)
    kern = {}
    for kind, name in ((0, "prologue"), (1, "intra_chunk"), (2, "inter_chunk")):
        ms, n = K.kda_profile_read(kind)
        if n:
            kern[name] = {"launches_per_step": n / nprof, "ms_per_step": ms / nprof}
    K.kda_profile_enable(False)
    # The call's kernels overlap at their boundary (programmatic dependent launch), so the duration
    # that the whole path's algorithmic bytes are divided by is the device time of one call in the
    # timed region; the per-kernel event pairs below serialise the kernels and are kept as shares.
    step_bytes = T_PREFILL * H * BYTES_PER_TOKEN_HEAD + H * STATE_BYTES
    achieved = step_bytes / (ms_step * 1e-3) / 1e9
    roofline = {
        "bound": "hbm", "kernel": "kda_chunk_fwd (all kernels of one call: %s)" % "+".join(kern),
        "duration_ms": ms_step,
        "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
        "frac": (achieved / peaks["hbm_gbs"]) if achieved else None, "peak_source": peaks["source"],
        "frac_of_8TBs_nominal": (achieved / 8000.0) if achieved else None,
        "algorithmic_bytes_per_step": step_bytes, "traffic": sum(PREFILL_DRAM_TRAFFIC.values()),
        "traffic_per_kernel": PREFILL_DRAM_TRAFFIC, "traffic_source": TRAFFIC_SOURCE, "kernels": kern,
        "tensor_bound_tokens_per_s": peaks["bf16_tflops"] * 1e12 / (H * FLOPS_PER_TOKEN_HEAD),
        "hbm_bound_tokens_per_s": peaks["hbm_gbs"] * 1e9 / (step_bytes / T_PREFILL),
        "note": "HBM is the slower bound at d=128, C=64; the tensor-pipe bound is above it",
    }

    if args.prefill_only:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": tokens_per_s, "unit": "tokens/s",
                              "ms_per_step": ms_step, "steps": args.steps, "warmup": args.warmup,
                              "gpu_launches": launches, "kernels": kern, "timing": timing,
                              "partial": "prefill-only"}))
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- end to end through the host-buffer entry point -------------------------------------------
    g0 = copies[0]
    pin = {n: (t.cpu().pin_memory() if isinstance(t, torch.Tensor) else t) for n, t in g0.items()}
    o_h = torch.empty((T_PREFILL, H, D), dtype=torch.bfloat16).pin_memory()
    S_h = torch.empty((1, H, D, D), dtype=torch.float32).pin_memory()
    hws_bytes = K.kda_chunk_fwd_host_workspace_bytes(T_PREFILL, 1, H, D, D, CHUNK, dt)
    hws = torch.empty(hws_bytes, dtype=torch.uint8, device=dev)
    h2d = sum(pin[n].numel() * pin[n].element_size() for n in ("q", "k", "v", "log_alpha", "beta", "S0"))
    d2h = o_h.numel() * 2 + S_h.numel() * 4

    def e2e_step():
        K.kda_chunk_fwd_host(pin["q"], pin["k"], pin["v"], pin["log_alpha"], pin["beta"], pin["S0"],
                             o_h, S_h, None, 1, T_PREFILL, H, D, D, CHUNK, 1.0, dt, hws, hws_bytes,
                             stream)
        stream.synchronize()   # the caller reads o / S_T on the host after every step

    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(3):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = max_over_ranks(max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3)) / e2e_steps
    e2e = {"value": world * T_PREFILL / (e2e_ms * 1e-3), "unit": "tokens/s",
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms}
    del hws, pin

    # ---- decode workload ----------------------------------------------------------------------------
    dd = inputs.decode_inputs(DEC_SEQS, H, DEC_STEPS, seed=4 + 1000 * rank)
    gd = {n: t.to(dev) for n, t in dd.items()}
    S = gd["S"].clone()
    od = torch.empty((DEC_STEPS, DEC_SEQS, H, D), dtype=torch.bfloat16, device=dev)

    def decode_block():
        for s in range(DEC_STEPS):
            K.kda_decode_step(gd["q"][s], gd["k"][s], gd["v"][s], gd["log_alpha"][s], gd["beta"][s],
                              S, None, od[s], DEC_SEQS, H, D, D, 1.0, dt, stream)

    decode_block()
    barrier()
    e0.record(stream)
    for _ in range(args.decode_reps):
        decode_block()
    e1.record(stream)
    barrier()
    dec_ms = max_over_ranks(e0.elapsed_time(e1)) / (args.decode_reps * DEC_STEPS)
    dec_bytes = DEC_SEQS * H * DEC_BYTES_PER_STATE
    dec_gbs = dec_bytes / (dec_ms * 1e-3) / 1e9
    # multi-token decode (4 tokens per sequence and call): the state crosses HBM once per call
    MT = 4
    mq, mk, mv, mg, mb = (gd[n][:MT].transpose(0, 1).contiguous() for n in ("q", "k", "v", "log_alpha", "beta"))
    mo = torch.empty((DEC_SEQS, MT, H, D), dtype=torch.bfloat16, device=dev)

    def multi_block():
        for _ in range(16):
            K.kda_decode_multi(mq, mk, mv, mg, mb, S, None, mo, DEC_SEQS, MT, H, D, D, 1.0, dt, stream)

    multi_block()
    barrier()
    e0.record(stream)
    for _ in range(args.decode_reps):
        multi_block()
    e1.record(stream)
    barrier()
    mt_ms = max_over_ranks(e0.elapsed_time(e1)) / (args.decode_reps * 16)
    mt_bytes = DEC_SEQS * H * (2 * D * D * 4 + MT * (4 * D * 2 + D * 4 + 4))
    multi = {"tokens_per_call_and_sequence": MT, "ms_per_call": mt_ms,
             "value": world * DEC_SEQS * MT / (mt_ms * 1e-3), "unit": "tokens/s",
             "achieved_gbs": mt_bytes / (mt_ms * 1e-3) / 1e9,
             "frac": mt_bytes / (mt_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    decode = {
        "multi_token": multi,
        "metric": "KDA decode tokens/s (256 seqs x 32 heads, 64 in-place steps)",
        "value": world * DEC_SEQS / (dec_ms * 1e-3), "unit": "tokens/s", "ms_per_step": dec_ms,
        "roofline": {"bound": "hbm", "kernel": "kda_decode_kernel", "achieved": dec_gbs,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": dec_gbs / peaks["hbm_gbs"],
                     "peak_source": peaks["source"], "frac_of_8TBs_nominal": dec_gbs / 8000.0,
                     "algorithmic_bytes_per_step": dec_bytes, "traffic": DECODE_DRAM_TRAFFIC},
    }

    # ---- the same prefill through the fused cooperative kernel (the path of small workspaces) --------
    fused = None
    if world == 1:
        K.kda_set_chunk_path(2)
        try:
            for i in range(3):
                prefill_step(i)
            barrier()
            e0.record(stream)
            for i in range(20):
                prefill_step(i)
            e1.record(stream)
            barrier()
            fms = e0.elapsed_time(e1) / 20
            fused = {"kernel": "kda_fused_tc (one cooperative launch: intra-chunk engines and inter-chunk "
                               "chains, tiles through a ring in L2)", "ms_per_step": fms,
                     "tokens_per_s": T_PREFILL / (fms * 1e-3),
                     "frac": step_bytes / (fms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                     "traffic": FUSED_DRAM_TRAFFIC, "traffic_source": TRAFFIC_SOURCE}
        finally:
            K.kda_set_chunk_path(0)

    # ---- the other prefill workloads (packed batch, 1 Mi tokens) -------------------------------------
    other = None
    free_b, _ = torch.cuda.mem_get_info()
    if world == 1 and not args.no_other_workloads:
        if free_b >= 80 * (1 << 30):
            other = extra_workloads(K, inputs, torch, dev, peaks)
            other["dplr_comparison"] = dplr_comparison(K, inputs, torch, dev, peaks)
            other["backward"] = backward_figure(K, inputs, torch, dev, peaks)
            other["layer_fwd"] = layer_figure(K, inputs, torch, dev, peaks)
        else:
            other = {"skipped": "needs about 70 GB of free device memory, %.0f GB free" % (free_b / 2 ** 30)}

    # ---- CPU oracle beside it (rank 0, single-GPU runs only) --------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        d = inputs.chunk_inputs([T_PREFILL], H=H, dtype=torch.bfloat16, seed=1, s0_std=0.02)
        a = {n: t.float().numpy() for n, t in d.items() if n in ("q", "k", "v", "log_alpha", "beta")}
        S0 = d["S0"].double().numpy()
        best = None
        reps = 0
        t_all = time.perf_counter()
        while reps < 3 or (time.perf_counter() - t_all < 5.0 and reps < 20):
            t0 = time.perf_counter()
            oracle.recurrence(a["q"], a["k"], a["v"], a["log_alpha"], a["beta"], S0=S0)
            el = time.perf_counter() - t0
            best = el if best is None else min(best, el)
            reps += 1
        cpu = {"value": T_PREFILL / best, "unit": "tokens/s", "cores": oracle.max_threads(),
               "kind": "oracle",
               "sample": "whole prefill workload (4096 tokens x 32 heads), best of %d runs" % reps}

    if rank == 0:
        line = {
            "metric": METRIC, "value": tokens_per_s, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": "prefill B=1 T=4096 H=32 dk=dv=128 chunk=64, bf16 q/k/v, fp32 "
                                   "gates/beta/state, S0~N(0,0.02); one batch "
                                   "per GPU",
                       "l2": "inputs rotate over 3 copies of 206 MB each (> 126 MB L2)",
                       "decode_workload": "256 seqs x 32 heads, 64 in-place steps"},
            "clocks": clocks, "timing": timing, "e2e": e2e, "gpu_launches": launches,
            "roofline": roofline, "decode": decode, "cpu_baseline": cpu,
        }
        if fused is not None:
            line["fused_path"] = fused
        if other is not None:
            line["other_workloads"] = other
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
