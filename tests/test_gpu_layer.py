"""Parity of kda_layer_fwd (the operator with L2Norm, decay function, beta sigmoid, head-wise RMSNorm
and output gate computed from bf16 pre-activations) with the layer oracle, through the C ABI.
Tolerance: relative L2 error 2e-2 on y and on the final state, the bf16 tolerance of the prefill
(bf16 operands of the tensor-core products and a bf16 output)."""
import numpy as np
import pytest
import torch

import paper_2510_26692_b200 as K
from paper_2510_26692_b200 import inputs
from oracle import layer as layer_oracle
from kda_testlib import Guarded, rel_l2, to_np32

pytestmark = pytest.mark.gpu
TOL = 2e-2


def run_layer(d, scale, want_y=True, workspace_bytes=None, dev="cuda:0", l2_eps=1e-6, rms_eps=1e-5):
    g = {n: (t.to(dev) if isinstance(t, torch.Tensor) else t) for n, t in d.items()}
    T, H, dk = g["k_c"].shape
    cu = d["cu_seqlens"]
    N = cu.numel() - 1
    nb = workspace_bytes or K.kda_layer_fwd_workspace_bytes(T, N, H)
    ws = Guarded(nb, dev)
    yb = Guarded(T * H * 128 * 2, dev)
    sb = Guarded(N * H * 128 * 128 * 4, dev)
    y = yb.view(torch.bfloat16, (T, H, 128))
    S_T = sb.view(torch.float32, (N, H, 128, 128))
    y.fill_(float("nan"))
    S_T.fill_(float("nan"))
    varlen = N > 1
    K.kda_layer_fwd(g["q_c"] if want_y else None, g["k_c"], g["v"], g["g_a"], g["b_pre"], g["g_o"], g["A_log"],
                    g["dt_bias"], g["w"], l2_eps, rms_eps, g["S0"], y if want_y else None, S_T,
                    g["cu_seqlens"] if varlen else None, cu if varlen else None, N, T, H, 128, 128, 64, scale,
                    ws.body, nb)
    torch.cuda.synchronize()
    K.kda_check_status(ws.body)
    for b_, name in ((ws, "the workspace"), (yb, "y"), (sb, "S_T")):
        b_.check(name)
    return (y if want_y else None), S_T


def oracle_layer(oracle_mod, d, scale, l2_eps=1e-6, rms_eps=1e-5):
    f = {n: (t.float().numpy() if isinstance(t, torch.Tensor) else t) for n, t in d.items()}
    cu = d["cu_seqlens"].numpy().astype(np.int64)
    return layer_oracle.layer_forward(oracle_mod.recurrence, f["q_c"], f["k_c"], f["v"], f["g_a"], f["b_pre"],
                                      f["g_o"], f["A_log"], f["dt_bias"], f["w"],
                                      S0=None if d["S0"] is None else d["S0"].double().numpy(), cu_seqlens=cu,
                                      scale=scale, l2_eps=l2_eps, rms_eps=rms_eps)


@pytest.mark.parametrize("lens,H,s0", [([256], 2, 0.0), ([1000], 3, 0.02), ([64, 1, 200, 0, 130], 4, 0.02),
                                       ([4096], 8, 0.02), ([1, 63, 65], 1, 0.02), ([5], 3, 0.0)])
def test_layer_matches_oracle(oracle_mod, lens, H, s0):
    d = inputs.layer_inputs(lens, H=H, seed=41, s0_std=s0)
    scale = 128 ** -0.5
    y, S_T = run_layer(d, scale)
    y_ref, S_ref, _ = oracle_layer(oracle_mod, d, scale)
    assert torch.isfinite(y.float()).all() and torch.isfinite(S_T).all()
    ey, es = rel_l2(to_np32(y), y_ref), rel_l2(to_np32(S_T), S_ref)
    print("layer", lens, H, ey, es)
    assert ey <= TOL and es <= TOL


def test_layer_state_only_and_small_workspace(oracle_mod):
    d = inputs.layer_inputs([700, 130], H=2, seed=42, s0_std=0.02)
    scale = 128 ** -0.5
    y1, S1 = run_layer(d, scale, workspace_bytes=K.kda_layer_fwd_min_workspace_bytes(830, 2, 2))
    y2, S2 = run_layer(d, scale)
    assert torch.equal(y1, y2) and torch.equal(S1, S2)          # several passes: same arithmetic per chunk
    _, S3 = run_layer(d, scale, want_y=False)
    y_ref, S_ref, _ = oracle_layer(oracle_mod, d, scale)
    assert rel_l2(to_np32(S3), S_ref) <= TOL and rel_l2(to_np32(y1), y_ref) <= TOL


def test_layer_equals_plain_call_on_precomputed_inputs(oracle_mod):
    """The in-kernel prologue against the same quantities computed on the host in fp32 and handed to
    kda_chunk_fwd: the only difference is where q, k are rounded to bf16, so the two agree far inside
    the bf16 tolerance."""
    from kda_testlib import run_chunk
    d = inputs.layer_inputs([512], H=2, seed=43, s0_std=0.02)
    scale = 128 ** -0.5
    _, S_layer = run_layer(d, scale)
    q, k, la, beta = layer_oracle.layer_inputs(*(d[n].float().numpy() for n in ("q_c", "k_c", "g_a", "b_pre", "A_log", "dt_bias")))
    plain = {"q": torch.tensor(q * scale).to(torch.bfloat16), "k": torch.tensor(k).to(torch.bfloat16), "v": d["v"],
             "log_alpha": torch.tensor(la, dtype=torch.float32), "beta": torch.tensor(beta, dtype=torch.float32),
             "S0": d["S0"], "cu_seqlens": d["cu_seqlens"]}
    _, S_plain = run_chunk(plain)
    assert rel_l2(to_np32(S_layer), to_np32(S_plain)) <= 5e-3


def test_layer_output_stage_fused_and_separate_agree(oracle_mod):
    """The output stage inside the inter-chunk kernel (clusters exchanging the rows' sums of squares)
    against the same stage as a separate pass: both within tolerance of the oracle, and close to each
    other (the separate pass normalises the bf16-rounded output)."""
    scale = 128 ** -0.5
    for lens, H in (([700, 130, 64], 4), ([2048], 40)):      # 40 heads: more chains than 32-column slices fit
        d = inputs.layer_inputs(lens, H=H, seed=44, s0_std=0.02)
        try:
            K.kda_layer_set_fused_output(False)
            y_sep, S_sep = run_layer(d, scale)
        finally:
            K.kda_layer_set_fused_output(True)
        y_fus, S_fus = run_layer(d, scale)
        y_ref, S_ref, _ = oracle_layer(oracle_mod, d, scale)
        assert torch.equal(S_sep, S_fus)
        e_sep, e_fus = rel_l2(to_np32(y_sep), y_ref), rel_l2(to_np32(y_fus), y_ref)
        print("output stage", lens, H, "separate", e_sep, "fused", e_fus)
        assert e_sep <= TOL and e_fus <= TOL
        assert rel_l2(to_np32(y_fus), to_np32(y_sep)) <= 1e-2


def test_layer_decode_step_matches_oracle(oracle_mod):
    """One decode token per sequence with the layer's element-wise stages inside the kernel: against the
    layer oracle's inputs -> oracle.decode_step -> output gate, two steps in place, with slot
    indirection.  Tolerance 2e-2 on the bf16 output row, 1e-4 on the fp32 state (fp32 arithmetic on
    bf16 inputs; the only reduced precision is the stored output)."""
    N, H = 5, 3
    dev = "cuda:0"
    g = torch.Generator().manual_seed(77)
    A_log = torch.randn((H,), generator=g) * 0.3
    dt_bias = torch.randn((H, 128), generator=g) * 0.3
    w = 1 + 0.1 * torch.randn((128,), generator=g)
    n_slots = 9
    slot = torch.tensor([7, 0, 3, 8, 2], dtype=torch.int32)
    S = (torch.randn((n_slots, H, 128, 128), generator=g) * 0.05)
    S_dev = S.clone().to(dev)
    S_ref = S.double().numpy().copy()
    for step in range(2):
        bf = torch.bfloat16
        q_c = (torch.randn((N, H, 128), generator=g) * 2).to(bf)
        k_c = (torch.randn((N, H, 128), generator=g) * 0.7).to(bf)
        v = torch.randn((N, H, 128), generator=g).to(bf)
        g_a = (torch.randn((N, H, 128), generator=g) - 3).to(bf)
        b_pre = torch.randn((N, H), generator=g)
        g_o = torch.randn((N, H, 128), generator=g).to(bf)
        y = torch.full((N, H, 128), float("nan"), dtype=bf, device=dev)
        K.kda_layer_decode_step(q_c.to(dev), k_c.to(dev), v.to(dev), g_a.to(dev), b_pre.to(dev), g_o.to(dev),
                                A_log.to(dev), dt_bias.to(dev), w.to(dev), 1e-6, 1e-5, S_dev, slot.to(dev), y, N, H,
                                128, 128, 128 ** -0.5)
        torch.cuda.synchronize()
        q, k, la, beta = layer_oracle.layer_inputs(q_c.float().numpy(), k_c.float().numpy(), g_a.float().numpy(),
                                                   b_pre.numpy(), A_log.numpy(), dt_bias.numpy(), 1e-6)
        o_ref = oracle_mod.decode_step(q.astype(np.float32), k.astype(np.float32), v.float().numpy(),
                                       la.astype(np.float32), beta.astype(np.float32), S_ref,
                                       state_slot=slot.numpy(), scale=128 ** -0.5)
        y_ref = layer_oracle.output_gate(o_ref, g_o.float().numpy(), w.numpy(), 1e-5)
        ey = rel_l2(to_np32(y), y_ref)
        es = rel_l2(to_np32(S_dev), S_ref)
        print("layer decode step", step, ey, es)
        assert torch.isfinite(y.float()).all()
        assert ey <= TOL and es <= 1e-4
