"""Pins of the fp64 oracle against what the paper and the mathematics fix (no GPU needed).

Each test states the fact it uses in its own formula, different from the oracle's loop, so that a
dropped term, a wrong sign, a swapped decay/update order or a transposed operand fails at least one.
"""
import os

import numpy as np
import pytest

from oracle.chunkwise import chunk_kda_np

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(T, H, dk, dv, seed, gate_lo=0.3, gate_hi=1.0, unit_k=True):
    r = np.random.default_rng(seed)
    q = r.standard_normal((T, H, dk)).astype(np.float32)
    k = r.standard_normal((T, H, dk)).astype(np.float32)
    if unit_k:
        k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = r.standard_normal((T, H, dv)).astype(np.float32)
    la = np.log(r.uniform(gate_lo, gate_hi, (T, H, dk))).astype(np.float32)
    beta = r.uniform(0.05, 1.0, (T, H)).astype(np.float32)
    return q, k, v, la, beta


def _read_golden(name):
    rec = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, vals = line.split(":")
            rec[key.strip()] = np.array([float(x) for x in vals.split()])
    return rec


def test_hand_worked_example(oracle_mod):
    """Eq. 1 on the two-token example worked by hand in tests/golden/eq1_worked_example.txt."""
    g = _read_golden("eq1_worked_example.txt")
    S0 = g["S0"].reshape(1, 1, 2, 2)
    q = np.stack([g["q1"], g["q2"]]).reshape(2, 1, 2)
    k = np.stack([g["k1"], g["k2"]]).reshape(2, 1, 2)
    v = np.stack([g["v1"], g["v2"]]).reshape(2, 1, 2)
    la = np.log(np.stack([g["alpha1"], g["alpha2"]])).reshape(2, 1, 2)
    beta = np.array([g["beta1"][0], g["beta2"][0]]).reshape(2, 1)
    o, S_T = oracle_mod.recurrence(q, k, v, la, beta, S0=S0)
    np.testing.assert_allclose(o[0, 0], g["o1"], rtol=0, atol=1e-6)
    np.testing.assert_allclose(o[1, 0], g["o2"], rtol=0, atol=1e-6)
    np.testing.assert_allclose(S_T[0, 0].ravel(), g["S2"], rtol=0, atol=1e-6)
    # state after the first token alone
    _, S1 = oracle_mod.recurrence(q[:1], k[:1], v[:1], la[:1], beta[:1], S0=S0)
    np.testing.assert_allclose(S1[0, 0].ravel(), g["S1"], rtol=0, atol=1e-6)
    # the decode entry point is the same body: two steps in place
    S = S0.copy()
    o1 = oracle_mod.decode_step(q[0:1], k[0:1], v[0:1], la[0:1], beta[0:1], S)
    np.testing.assert_allclose(S[0, 0].ravel(), g["S1"], atol=1e-6)
    o2 = oracle_mod.decode_step(q[1:2], k[1:2], v[1:2], la[1:2], beta[1:2], S)
    np.testing.assert_allclose(o1[0, 0], g["o1"], atol=1e-6)
    np.testing.assert_allclose(o2[0, 0], g["o2"], atol=1e-6)
    np.testing.assert_allclose(S[0, 0].ravel(), g["S2"], atol=1e-6)


def test_single_token_closed_form(oracle_mod):
    """S0 = 0, one token: S1 = beta k v^T and o1 = scale beta (k.q) v  (Eq. 1)."""
    q, k, v, la, beta = _rand(1, 3, 5, 7, seed=1)
    o, S = oracle_mod.recurrence(q, k, v, la, beta, scale=0.7)
    for h in range(3):
        kk, vv, qq, b = (x[0, h].astype(np.float64) for x in (k, v, q, beta[..., None]))
        np.testing.assert_allclose(S[0, h], b * np.outer(kk, vv), rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(o[0, h], 0.7 * b * (kk @ qq) * vv, rtol=1e-12, atol=1e-14)


def test_alpha_one_is_delta_rule_and_scalar_alpha_is_gdn(oracle_mod):
    """alpha = 1 gives DeltaNet, S = (I - b k k^T) S + b k v^T; a scalar gate gives Gated
    DeltaNet, S = a (I - b k k^T) S + b k v^T  (Section 2.2)."""
    T, H, dk, dv = 12, 2, 6, 4
    q, k, v, la, beta = _rand(T, H, dk, dv, seed=2)
    r = np.random.default_rng(3)
    S0 = r.standard_normal((1, H, dk, dv))
    for mode in ("delta", "gdn"):
        if mode == "delta":
            a_t = np.ones((T, H))
        else:
            a_t = r.uniform(0.4, 1.0, (T, H))
        la_m = np.broadcast_to(np.log(a_t)[..., None], (T, H, dk)).astype(np.float32)
        a_eff = np.exp(la_m[..., 0].astype(np.float64))
        o, S_T = oracle_mod.recurrence(q, k, v, la_m, beta, S0=S0)
        for h in range(H):
            S = S0[0, h].copy()
            for t in range(T):
                kk = k[t, h].astype(np.float64)
                b = float(beta[t, h])
                S = a_eff[t, h] * ((np.eye(dk) - b * np.outer(kk, kk)) @ S) \
                    + b * np.outer(kk, v[t, h].astype(np.float64))
                np.testing.assert_allclose(o[t, h], S.T @ q[t, h].astype(np.float64),
                                           rtol=1e-11, atol=1e-12)
            np.testing.assert_allclose(S_T[0, h], S, rtol=1e-11, atol=1e-12)


def test_beta_zero_is_pure_decay(oracle_mod):
    """beta = 0: no erase, no write.  S_T = Diag(prod alpha) S0 and
    o_t = scale (gamma_{1..t} . q_t)^T S0."""
    T, H, dk, dv = 9, 2, 5, 3
    q, k, v, la, _ = _rand(T, H, dk, dv, seed=4)
    beta = np.zeros((T, H), np.float32)
    S0 = np.random.default_rng(5).standard_normal((1, H, dk, dv))
    o, S_T = oracle_mod.recurrence(q, k, v, la, beta, S0=S0, scale=1.3)
    G = np.cumsum(la.astype(np.float64), axis=0)
    for h in range(H):
        np.testing.assert_allclose(S_T[0, h], np.exp(G[-1, h])[:, None] * S0[0, h], rtol=1e-12)
        for t in range(T):
            np.testing.assert_allclose(o[t, h], 1.3 * (np.exp(G[t, h]) * q[t, h]) @ S0[0, h],
                                       rtol=1e-11, atol=1e-13)


def test_gla_on_pseudo_values(oracle_mod):
    """With vt_i = beta_i (v_i - (Diag(alpha_i) S_{i-1})^T k_i) the state is a gated-linear-
    attention sum: o_t = (gamma_t . q_t)^T S0 + sum_{i<=t} ((q_t . gamma_t/gamma_i) . k_i) vt_i
    (the 'pseudo-value' reading of the output equation in Section 3.1)."""
    T, H, dk, dv = 10, 1, 4, 3
    q, k, v, la, beta = _rand(T, H, dk, dv, seed=6)
    S0 = np.random.default_rng(7).standard_normal((1, H, dk, dv))
    o, _ = oracle_mod.recurrence(q, k, v, la, beta, S0=S0)
    # states after each prefix, from the oracle itself, to form the pseudo-values
    G = np.cumsum(la[:, 0].astype(np.float64), axis=0)
    vt = np.zeros((T, dv))
    for t in range(T):
        if t == 0:
            Sprev = S0[0, 0]
        else:
            _, Sp = oracle_mod.recurrence(q[:t], k[:t], v[:t], la[:t], beta[:t], S0=S0)
            Sprev = Sp[0, 0]
        Sd = np.exp(la[t, 0].astype(np.float64))[:, None] * Sprev
        vt[t] = beta[t, 0] * (v[t, 0] - Sd.T @ k[t, 0].astype(np.float64))
    for t in range(T):
        acc = (np.exp(G[t]) * q[t, 0]) @ S0[0, 0]
        for i in range(t + 1):
            acc = acc + np.sum(q[t, 0] * np.exp(G[t] - G[i]) * k[i, 0]) * vt[i]
        np.testing.assert_allclose(o[t, 0], acc, rtol=1e-10, atol=1e-12)


def test_exact_recall_invariant(oracle_mod):
    """beta_t = 1 and |k_t| = 1: the updated state returns v_t for k_t, i.e. q_t = k_t gives
    o_t = scale v_t whatever the gates and the earlier state (reconstruction objective,
    Section 2.2)."""
    T, H, dk, dv = 7, 2, 8, 5
    _, k, v, la, _ = _rand(T, H, dk, dv, seed=8)
    k64 = k.astype(np.float64)
    k = (k64 / np.linalg.norm(k64, axis=-1, keepdims=True)).astype(np.float32)
    beta = np.ones((T, H), np.float32)
    S0 = np.random.default_rng(9).standard_normal((1, H, dk, dv))
    o, _ = oracle_mod.recurrence(k, k, v, la, beta, S0=S0, scale=2.0)
    # float32 keys are unit only to ~1e-7, so the identity holds to that order
    np.testing.assert_allclose(o, 2.0 * v, rtol=0, atol=5e-6)


def test_brute_force_products(oracle_mod):
    """T <= 8: S_t = P_t S0 + H_t with explicit dk x dk products
    P_t = prod_{j=t..1} (I - b_j k_j k_j^T) Diag(a_j),
    H_t = sum_i (prod_{j=t..i+1} (I - b_j k_j k_j^T) Diag(a_j)) b_i k_i v_i^T  (Section 3.1,
    chunk expansion of Eq. 1)."""
    T, H, dk, dv = 8, 2, 6, 7
    q, k, v, la, beta = _rand(T, H, dk, dv, seed=10, unit_k=False)
    k *= 0.4
    S0 = np.random.default_rng(11).standard_normal((1, H, dk, dv))
    o, S_T = oracle_mod.recurrence(q, k, v, la, beta, S0=S0, scale=0.5)
    for h in range(H):
        A = [(np.eye(dk) - float(beta[t, h]) * np.outer(k[t, h].astype(np.float64), k[t, h]))
             @ np.diag(np.exp(la[t, h].astype(np.float64))) for t in range(T)]
        for t in range(T):
            P = np.eye(dk)
            for j in range(t + 1):
                P = A[j] @ P
            Hm = np.zeros((dk, dv))
            for i in range(t + 1):
                Pi = np.eye(dk)
                for j in range(i + 1, t + 1):
                    Pi = A[j] @ Pi
                Hm += Pi @ (float(beta[i, h]) * np.outer(k[i, h].astype(np.float64), v[i, h]))
            St = P @ S0[0, h] + Hm
            np.testing.assert_allclose(o[t, h], 0.5 * St.T @ q[t, h], rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(S_T[0, h], St, rtol=1e-10, atol=1e-12)


def test_whole_sequence_parallel_form(oracle_mod):
    """S0 = 0, the sequence as one block:
    O = Tril((Gamma.Q)(K/Gamma)^T) solve(I + StrictTril(Diag(b)(Gamma.K)(K/Gamma)^T), Diag(b) V)
    with LAPACK's solve (parallel form of KDA, Table 'parallel forms', with beta restored as in the
    UT transform of Section 3.1)."""
    T, H, dk, dv = 96, 2, 16, 12
    q, k, v, la, beta = _rand(T, H, dk, dv, seed=12, gate_lo=0.8, gate_hi=1.0)
    o, _ = oracle_mod.recurrence(q, k, v, la, beta)
    for h in range(H):
        G = np.cumsum(la[:, h].astype(np.float64), axis=0)
        Gam = np.exp(G)
        Kd, Ki, Qd = Gam * k[:, h], k[:, h] / Gam, Gam * q[:, h]
        b = beta[:, h].astype(np.float64)
        A = np.tril(b[:, None] * (Kd @ Ki.T), -1)
        X = np.linalg.solve(np.eye(T) + A, b[:, None] * v[:, h].astype(np.float64))
        O = np.tril(Qd @ Ki.T) @ X
        np.testing.assert_allclose(o[:, h], O, rtol=1e-8, atol=1e-9)


@pytest.mark.parametrize("C", [16, 32, 64])
@pytest.mark.parametrize("T", [64, 100, 193])
def test_chunkwise_form_equals_recurrence(oracle_mod, C, T):
    """The chunkwise algorithm (Section 3.1, Appendix C) regroups Eq. 1 exactly, for any chunk
    size and with a short last chunk."""
    H, dk, dv = 2, 16, 24
    q, k, v, la, beta = _rand(T, H, dk, dv, seed=13 + C + T)
    S0 = np.random.default_rng(14).standard_normal((1, H, dk, dv))
    o, S_T = oracle_mod.recurrence(q, k, v, la, beta, S0=S0, scale=0.25)
    o2, S2 = chunk_kda_np(q, k, v, la, beta, S0=S0[0], chunk=C, scale=0.25)
    np.testing.assert_allclose(o, o2, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(S_T[0], S2, rtol=1e-9, atol=1e-11)


def test_chunkwise_form_paper_shapes(oracle_mod):
    """Same agreement at the paper's head size (dk = dv = 128, C = 64) with the benchmark gates."""
    import torch
    from paper_2510_26692_b200 import inputs
    d = inputs.chunk_inputs([200], H=1, dtype=torch.float32, seed=0, s0_std=0.02)
    a = {n: (None if t is None else t.numpy()) for n, t in d.items()}
    o, S_T = oracle_mod.recurrence(a["q"], a["k"], a["v"], a["log_alpha"], a["beta"], S0=a["S0"])
    o2, S2 = chunk_kda_np(a["q"], a["k"], a["v"], a["log_alpha"], a["beta"], S0=a["S0"][0])
    assert np.linalg.norm(o - o2) / np.linalg.norm(o) < 1e-12
    assert np.linalg.norm(S_T[0] - S2) / np.linalg.norm(S2) < 1e-12


def test_composition_and_affine_form(oracle_mod):
    """Resume: run(T1) then run(T2, S0 = S_T1) equals run(T1+T2).  The map S_in -> S_out is
    affine, S_out = P S_in + H with P = run(v = 0, S0 = I) and H = run(S0 = 0)
    (Section 3.1, chunk expansion)."""
    T1, T2, H, dk, dv = 11, 9, 2, 6, 6
    q, k, v, la, beta = _rand(T1 + T2, H, dk, dv, seed=15)
    S0 = np.random.default_rng(16).standard_normal((1, H, dk, dv))
    o, S_T = oracle_mod.recurrence(q, k, v, la, beta, S0=S0)
    oa, Sa = oracle_mod.recurrence(q[:T1], k[:T1], v[:T1], la[:T1], beta[:T1], S0=S0)
    ob, Sb = oracle_mod.recurrence(q[T1:], k[T1:], v[T1:], la[T1:], beta[T1:], S0=Sa)
    np.testing.assert_allclose(np.concatenate([oa, ob]), o, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(Sb, S_T, rtol=1e-12, atol=1e-14)
    eye = np.broadcast_to(np.eye(dk), (1, H, dk, dk)).copy()
    _, P = oracle_mod.recurrence(q, k, np.zeros((T1 + T2, H, dk), np.float32), la, beta, S0=eye)
    _, Hm = oracle_mod.recurrence(q, k, v, la, beta)
    for h in range(H):
        np.testing.assert_allclose(P[0, h] @ S0[0, h] + Hm[0, h], S_T[0, h], rtol=1e-11,
                                   atol=1e-13)


def test_decode_one_pass_identity_and_slots(oracle_mod):
    """Decode: o = scale (Sd^T q + beta (q.k) r), Sd = Diag(alpha) S, r = v - Sd^T k (algebra on
    Eq. 1); sequence n uses state slot state_slot[n]; one decode step equals a one-token
    recurrence."""
    N, H, dk, dv = 5, 3, 8, 6
    r = np.random.default_rng(17)
    q, k, v, la, beta = (x.reshape((N, H) + x.shape[2:]) for x in _rand(N, H, dk, dv, seed=18))
    S = r.standard_normal((7, H, dk, dv))
    slot = np.array([6, 0, 3, 2, 5], np.int32)
    S_in = S.copy()
    o = oracle_mod.decode_step(q, k, v, la, beta, S, state_slot=slot, scale=0.9)
    for n in range(N):
        for h in range(H):
            Sd = np.exp(la[n, h].astype(np.float64))[:, None] * S_in[slot[n], h]
            kk, qq = k[n, h].astype(np.float64), q[n, h].astype(np.float64)
            rr = v[n, h] - Sd.T @ kk
            np.testing.assert_allclose(o[n, h], 0.9 * (Sd.T @ qq + beta[n, h] * (qq @ kk) * rr),
                                       rtol=1e-11, atol=1e-13)
            np.testing.assert_allclose(S[slot[n], h], Sd + beta[n, h] * np.outer(kk, rr),
                                       rtol=1e-12, atol=1e-14)
            o1, S1 = oracle_mod.recurrence(q[n:n + 1, h:h + 1], k[n:n + 1, h:h + 1],
                                           v[n:n + 1, h:h + 1], la[n:n + 1, h:h + 1],
                                           beta[n:n + 1, h:h + 1],
                                           S0=S_in[slot[n]:slot[n] + 1, h:h + 1], scale=0.9)
            np.testing.assert_allclose(o1[0, 0], o[n, h], rtol=1e-13, atol=1e-15)
            np.testing.assert_allclose(S1[0, 0], S[slot[n], h], rtol=1e-13, atol=1e-15)
    untouched = [s for s in range(7) if s not in set(slot.tolist())]
    np.testing.assert_array_equal(S[untouched], S_in[untouched])


def test_varlen_packing(oracle_mod):
    """Packed sequences are independent; a zero-length sequence leaves S_T = S0."""
    lens = [5, 0, 9, 1]
    T, H, dk, dv = sum(lens), 2, 4, 5
    q, k, v, la, beta = _rand(T, H, dk, dv, seed=19)
    S0 = np.random.default_rng(20).standard_normal((len(lens), H, dk, dv))
    cu = np.concatenate([[0], np.cumsum(lens)])
    o, S_T = oracle_mod.recurrence(q, k, v, la, beta, S0=S0, cu_seqlens=cu)
    for n, L in enumerate(lens):
        a, b = cu[n], cu[n + 1]
        if L == 0:
            np.testing.assert_array_equal(S_T[n], S0[n])
            continue
        on, Sn = oracle_mod.recurrence(q[a:b], k[a:b], v[a:b], la[a:b], beta[a:b],
                                       S0=S0[n:n + 1])
        np.testing.assert_array_equal(o[a:b], on)
        np.testing.assert_array_equal(S_T[n], Sn[0])
