"""Pins of the fp64 oracle of the general diagonal-plus-low-rank recurrence (the paper's comparison
workload, Section 6.1 "Relation to DPLR") against facts that do not come from its own loop."""
import numpy as np

from oracle.chunkwise import chunk_dplr_np


def _rand(T, H, dk, dv, seed):
    r = np.random.default_rng(seed)
    q = r.standard_normal((T, H, dk)).astype(np.float32)
    k = r.standard_normal((T, H, dk)).astype(np.float32)
    k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = r.standard_normal((T, H, dv)).astype(np.float32)
    a = r.standard_normal((T, H, dk)).astype(np.float32)
    a /= np.linalg.norm(a, axis=-1, keepdims=True)
    b = (-r.uniform(0.1, 0.9, (T, H, 1)) * (a + 0.3 * r.standard_normal((T, H, dk)))).astype(np.float32)
    g = np.log(r.uniform(0.4, 1.0, (T, H, dk))).astype(np.float32)
    return q, k, v, a, b, g


def test_kda_is_the_bound_special_case(oracle_mod):
    """Section 6.1: Eq. 1 is the DPLR recurrence with D = Diag(alpha), the contracted vector
    alpha . k, the added vector -beta k and the key beta k.  Two different loops of the oracle file
    must then agree to rounding."""
    r = np.random.default_rng(3)
    T, H, dk, dv = 37, 2, 8, 5
    q = r.standard_normal((T, H, dk)).astype(np.float32)
    k = r.standard_normal((T, H, dk)).astype(np.float32)
    k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = r.standard_normal((T, H, dv)).astype(np.float32)
    la = np.log(r.uniform(0.3, 1.0, (T, H, dk))).astype(np.float32)
    beta = r.uniform(0.05, 1.0, (T, H)).astype(np.float32)
    S0 = r.standard_normal((1, H, dk, dv))
    o_ref, S_ref = oracle_mod.recurrence(q, k, v, la, beta, S0=S0, scale=0.7)
    # the three bound vectors are formed in fp64 and handed over as fp32: allow for that rounding
    a = (np.exp(la.astype(np.float64)) * k).astype(np.float32)
    b = (-beta[..., None].astype(np.float64) * k).astype(np.float32)
    kb = (beta[..., None].astype(np.float64) * k).astype(np.float32)
    o, S_T = oracle_mod.dplr_recurrence(q, kb, v, a, b, la, S0=S0, scale=0.7)
    np.testing.assert_allclose(o, o_ref, rtol=0, atol=2e-6 * np.abs(o_ref).max())
    np.testing.assert_allclose(S_T, S_ref, rtol=0, atol=2e-6 * np.abs(S_ref).max())


def test_explicit_transition_matrices(oracle_mod):
    """Brute force on a tiny case: build every transition matrix Diag(exp g_t) + b_t a_t^T with numpy
    and multiply them out."""
    T, H, dk, dv = 6, 1, 4, 3
    q, k, v, a, b, g = _rand(T, H, dk, dv, 5)
    S0 = np.random.default_rng(6).standard_normal((1, H, dk, dv))
    o, S_T = oracle_mod.dplr_recurrence(q, k, v, a, b, g, S0=S0, scale=1.3)
    S = S0[0, 0].copy()
    for t in range(T):
        M = np.diag(np.exp(g[t, 0].astype(np.float64))) + np.outer(b[t, 0].astype(np.float64), a[t, 0].astype(np.float64))
        S = M @ S + np.outer(k[t, 0].astype(np.float64), v[t, 0].astype(np.float64))
        np.testing.assert_allclose(o[t, 0], 1.3 * S.T @ q[t, 0].astype(np.float64), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(S_T[0, 0], S, rtol=1e-12, atol=1e-12)


def test_without_low_rank_term_it_is_gated_linear_attention(oracle_mod):
    """a = 0 removes the low-rank term: S_T = sum_t Diag(prod_{s>t} exp g_s) k_t v_t^T in closed form,
    o_t = sum_{s<=t} (q_t . exp(G_t - G_s) . k_s) v_s."""
    T, H, dk, dv = 19, 2, 6, 4
    q, k, v, a, b, g = _rand(T, H, dk, dv, 8)
    o, S_T = oracle_mod.dplr_recurrence(q, k, v, np.zeros_like(a), b, g)
    G = np.cumsum(g.astype(np.float64), axis=0)
    for h in range(H):
        dec = np.exp(G[-1, h][None, :] - G[:, h])                     # [T,dk]
        np.testing.assert_allclose(S_T[0, h], (k[:, h] * dec).T @ v[:, h].astype(np.float64), rtol=1e-11, atol=1e-12)
        for t in (0, 7, T - 1):
            w = np.einsum("d,sd,sd->s", q[t, h].astype(np.float64), k[:t + 1, h].astype(np.float64),
                          np.exp(G[t, h][None, :] - G[:t + 1, h]))
            np.testing.assert_allclose(o[t, h], w @ v[:t + 1, h].astype(np.float64), rtol=1e-11, atol=1e-12)


def test_chunkwise_form_agrees(oracle_mod):
    """The chunkwise regrouping (four Gram matrices, one triangular solve, three output terms, two
    state terms) reproduces the recurrence, also with a ragged last chunk and packed sequences."""
    T, H, dk, dv = 150, 2, 16, 8
    q, k, v, a, b, g = _rand(T, H, dk, dv, 11)
    S0 = np.random.default_rng(12).standard_normal((2, H, dk, dv)) * 0.1
    cu = np.array([0, 70, 150])
    o, S_T = oracle_mod.dplr_recurrence(q, k, v, a, b, g, S0=S0, cu_seqlens=cu, scale=0.5)
    for n in range(2):
        s, e = cu[n], cu[n + 1]
        oc, Sc = chunk_dplr_np(q[s:e], k[s:e], v[s:e], a[s:e], b[s:e], g[s:e], S0=S0[n], chunk=64, scale=0.5)
        np.testing.assert_allclose(oc, o[s:e], rtol=0, atol=1e-9 * max(1.0, np.abs(o).max()))
        np.testing.assert_allclose(Sc, S_T[n], rtol=0, atol=1e-9 * max(1.0, np.abs(S_T).max()))


def test_workload_recipe_stays_bounded(oracle_mod):
    """The synthetic DPLR workload (see inputs.dplr_inputs) neither blows up nor dies out."""
    from paper_2510_26692_b200 import inputs
    d = inputs.dplr_inputs([1500], H=2, dk=32, dv=16, seed=2)
    o, S_T = oracle_mod.dplr_recurrence(*(d[n].numpy() for n in ("q", "k", "v", "a", "b", "g")))
    assert np.isfinite(o).all() and 1e-3 < np.abs(o[-200:]).mean() < 1e2
