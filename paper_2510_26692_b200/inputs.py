"""Seeded synthetic inputs shaped like the KDA workloads of the Kimi Linear paper.

This module only draws random tensors; it holds none of the method's arithmetic and is the one
module that both the CUDA-path tests/benchmark and the oracle-side tests may use.

Recipe (the paper's parameterisation, Section 4 "Neural Parameterization"): q and k are
L2-normalised per (token, head); q additionally carries the dk^-0.5 factor that the paper's
chunkwise pseudo-code applies (Appendix C); v ~ N(0,1); the per-channel log-decay is
logsigmoid(x) with x ~ N(gate_mean, 1); beta = sigmoid(N(0,1)); initial states ~ N(0, s0_std).
Each tensor has its own generator (seed*16 + index, in the order q,k,v,x,beta,S0) so that a
tensor's values do not depend on which other tensors are requested.
"""
from __future__ import annotations

from typing import Dict, Optional, Sequence

import torch

_ORDER = {"q": 0, "k": 1, "v": 2, "x": 3, "beta": 4, "S0": 5, "S": 6, "lens": 7, "a": 8, "b": 9, "eta": 10,
          "do": 11, "dS": 12, "go": 13, "w": 14, "bias": 15}


def _gen(seed: int, name: str, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) * 16 + _ORDER[name])
    return g


def _randn(shape, seed, name, device):
    return torch.randn(*shape, generator=_gen(seed, name, device), device=device,
                       dtype=torch.float32)


def _l2norm(x: torch.Tensor) -> torch.Tensor:
    return x * torch.rsqrt((x * x).sum(-1, keepdim=True) + 1e-6)


def varlen_lengths(n_seqs: int, lo: int, hi: int, seed: int) -> list:
    """Integer-uniform sequence lengths on [lo, hi] (inclusive), seeded."""
    g = _gen(seed, "lens", "cpu")
    return [int(x) for x in torch.randint(lo, hi + 1, (n_seqs,), generator=g)]


def cu_seqlens_of(lengths: Sequence[int]) -> torch.Tensor:
    cu = [0]
    for n in lengths:
        cu.append(cu[-1] + int(n))
    return torch.tensor(cu, dtype=torch.int32)


def chunk_inputs(lengths: Sequence[int], H: int, dk: int = 128, dv: int = 128,
                 dtype: torch.dtype = torch.bfloat16, seed: int = 0, gate_mean: float = 4.0,
                 s0_std: float = 0.0, scale_q: bool = True, device="cpu",
                 want_q: bool = True) -> Dict[str, Optional[torch.Tensor]]:
    """Inputs of one prefill call over ``len(lengths)`` packed sequences.

    Returns q,k [T,H,dk] and v [T,H,dv] in ``dtype`` (rounded after scaling), log_alpha [T,H,dk]
    and beta [T,H] in fp32, S0 [N,H,dk,dv] fp32 (None when s0_std == 0), cu_seqlens int32 [N+1].
    """
    T = int(sum(lengths))
    N = len(lengths)
    out: Dict[str, Optional[torch.Tensor]] = {}
    if want_q:
        q = _l2norm(_randn((T, H, dk), seed, "q", device))
        if scale_q:
            q = q * (dk ** -0.5)
        out["q"] = q.to(dtype)
        del q
    else:
        out["q"] = None
    out["k"] = _l2norm(_randn((T, H, dk), seed, "k", device)).to(dtype)
    out["v"] = _randn((T, H, dv), seed, "v", device).to(dtype)
    x = _randn((T, H, dk), seed, "x", device)
    x += gate_mean
    out["log_alpha"] = torch.nn.functional.logsigmoid(x)
    del x
    out["beta"] = torch.sigmoid(_randn((T, H), seed, "beta", device))
    out["S0"] = (_randn((N, H, dk, dv), seed, "S0", device) * s0_std) if s0_std > 0 else None
    out["cu_seqlens"] = cu_seqlens_of(lengths)
    return out


def chunk_inputs_slabbed(T: int, H: int, dk: int = 128, dv: int = 128, seed: int = 3,
                         gate_mean: float = 6.0, s0_std: float = 0.02, device="cuda",
                         slab: int = 65536, want_q: bool = True) -> Dict[str, Optional[torch.Tensor]]:
    """One long sequence (bf16 q/k/v) drawn slab by slab on ``device`` so that the fp32
    temporaries stay small; slab s of a tensor uses the generator seed (seed*4096 + s)*16 + index.
    Same distributions as :func:`chunk_inputs`."""
    bf = torch.bfloat16
    out: Dict[str, Optional[torch.Tensor]] = {
        "q": torch.empty((T, H, dk), dtype=bf, device=device) if want_q else None,
        "k": torch.empty((T, H, dk), dtype=bf, device=device),
        "v": torch.empty((T, H, dv), dtype=bf, device=device),
        "log_alpha": torch.empty((T, H, dk), dtype=torch.float32, device=device),
        "beta": torch.empty((T, H), dtype=torch.float32, device=device),
    }
    for s, t0 in enumerate(range(0, T, slab)):
        n = min(slab, T - t0)
        sd = seed * 4096 + s
        if want_q:
            out["q"][t0:t0 + n] = (_l2norm(_randn((n, H, dk), sd, "q", device)) * (dk ** -0.5)).to(bf)
        out["k"][t0:t0 + n] = _l2norm(_randn((n, H, dk), sd, "k", device)).to(bf)
        out["v"][t0:t0 + n] = _randn((n, H, dv), sd, "v", device).to(bf)
        out["log_alpha"][t0:t0 + n] = torch.nn.functional.logsigmoid(
            _randn((n, H, dk), sd, "x", device) + gate_mean)
        out["beta"][t0:t0 + n] = torch.sigmoid(_randn((n, H), sd, "beta", device))
    out["S0"] = (_randn((1, H, dk, dv), seed, "S0", device) * s0_std) if s0_std > 0 else None
    out["cu_seqlens"] = cu_seqlens_of([T])
    return out


def decode_inputs(n_seqs: int, H: int, steps: int, dk: int = 128, dv: int = 128,
                  dtype: torch.dtype = torch.bfloat16, seed: int = 4, gate_mean: float = 4.0,
                  s_std: float = 0.05, device="cpu") -> Dict[str, torch.Tensor]:
    """Inputs of ``steps`` consecutive decode steps: q,k,log_alpha [steps,N,H,dk], v [steps,N,H,dv],
    beta [steps,N,H], and the starting states S [N,H,dk,dv] fp32.  q and k are L2-normalised and q
    carries no dk^-0.5 factor (the decode workload states none)."""
    out = {}
    out["q"] = _l2norm(_randn((steps, n_seqs, H, dk), seed, "q", device)).to(dtype)
    out["k"] = _l2norm(_randn((steps, n_seqs, H, dk), seed, "k", device)).to(dtype)
    out["v"] = _randn((steps, n_seqs, H, dv), seed, "v", device).to(dtype)
    x = _randn((steps, n_seqs, H, dk), seed, "x", device) + gate_mean
    out["log_alpha"] = torch.nn.functional.logsigmoid(x)
    out["beta"] = torch.sigmoid(_randn((steps, n_seqs, H), seed, "beta", device))
    out["S"] = _randn((n_seqs, H, dk, dv), seed, "S", device) * s_std
    return out


def dplr_inputs(lengths: Sequence[int], H: int, dk: int = 128, dv: int = 128, seed: int = 0,
                gate_mean: float = 4.0, s0_std: float = 0.0, device="cpu") -> Dict[str, Optional[torch.Tensor]]:
    """Inputs of one call of the general diagonal-plus-low-rank workload (the paper's comparison
    kernel): q, k, v, the decay g = logsigmoid(N(gate_mean, 1)) as in ``chunk_inputs``, and two
    independent low-rank vectors: a = a unit vector times a factor in (0.5, 1), b = minus another
    unit vector (correlated with a's) times a factor in (0, 1), so that the transition
    Diag(exp(g)) + b a^T stays close to a contraction and long sequences neither blow up nor die
    out.  Everything fp32.
    """
    T = int(sum(lengths))
    N = len(lengths)
    out: Dict[str, Optional[torch.Tensor]] = {}
    out["q"] = _l2norm(_randn((T, H, dk), seed, "q", device)) * (dk ** -0.5)
    out["k"] = _l2norm(_randn((T, H, dk), seed, "k", device))
    out["v"] = _randn((T, H, dv), seed, "v", device)
    x = _randn((T, H, dk), seed, "x", device)
    x += gate_mean
    out["g"] = torch.nn.functional.logsigmoid(x)
    del x
    ra = _randn((T, H, dk), seed, "a", device)
    rb = _randn((T, H, dk), seed, "b", device)
    eta = torch.sigmoid(_randn((T, H, 2), seed, "eta", device))
    out["a"] = _l2norm(ra) * (0.5 + 0.5 * eta[..., 0:1])
    out["b"] = -_l2norm(ra + 0.5 * rb) * eta[..., 1:2]
    out["S0"] = (_randn((N, H, dk, dv), seed, "S0", device) * s0_std) if s0_std > 0 else None
    out["cu_seqlens"] = cu_seqlens_of(lengths)
    return out


def layer_inputs(lengths: Sequence[int], H: int, dk: int = 128, dv: int = 128, seed: int = 0,
                 gate_mean: float = 4.0, s0_std: float = 0.0, device="cpu") -> Dict[str, Optional[torch.Tensor]]:
    """Pre-activations of one KDA layer call (Section 4, "Neural Parameterization"): q_c, k_c (what
    leaves the short convolution and Swish, before L2Norm; N(0,1) times a per-token factor so that
    the norms vary), v, the decay pre-activation g_a (N(-gate_mean, 1): after the softplus and a
    per-head rate exp(A_log) of about one this gives the same decay range as ``chunk_inputs``), the
    beta pre-activation b_pre ~ N(0,1) (fp32), the output-gate pre-activation g_o ~ N(0,1), and the
    layer's parameters A_log [H] ~ N(0, 0.3), dt_bias [H,dk] ~ N(0, 0.3), RMSNorm weight w [dv] ~
    1 + N(0, 0.1).  Activations bf16, parameters fp32.
    """
    T = int(sum(lengths))
    N = len(lengths)
    bf = torch.bfloat16
    out: Dict[str, Optional[torch.Tensor]] = {}
    fac = 0.5 + torch.rand((T, H, 2), generator=_gen(seed, "eta", device), device=device) * 3.0
    out["q_c"] = (_randn((T, H, dk), seed, "q", device) * fac[..., 0:1]).to(bf)
    out["k_c"] = (_randn((T, H, dk), seed, "k", device) * fac[..., 1:2]).to(bf)
    out["v"] = _randn((T, H, dv), seed, "v", device).to(bf)
    out["g_a"] = (_randn((T, H, dk), seed, "x", device) - gate_mean).to(bf)
    out["b_pre"] = _randn((T, H), seed, "beta", device)
    out["g_o"] = _randn((T, H, dv), seed, "go", device).to(bf)
    out["A_log"] = _randn((H,), seed, "a", device) * 0.3
    out["dt_bias"] = _randn((H, dk), seed, "bias", device) * 0.3
    out["w"] = 1.0 + _randn((dv,), seed, "w", device) * 0.1
    out["S0"] = (_randn((N, H, dk, dv), seed, "S0", device) * s0_std) if s0_std > 0 else None
    out["cu_seqlens"] = cu_seqlens_of(lengths)
    return out
