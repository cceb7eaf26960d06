"""Pins of the fp64 backward oracle (adjoint of Eq. 1) against facts that do not come from its own
loop: central finite differences of the forward oracle, a one-token closed form, the zero-beta
special case, linearity, and independence of packed sequences."""
import numpy as np


def _rand(T, H, dk, dv, seed):
    r = np.random.default_rng(seed)
    q = r.standard_normal((T, H, dk)).astype(np.float32)
    k = r.standard_normal((T, H, dk)).astype(np.float32)
    k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = r.standard_normal((T, H, dv)).astype(np.float32)
    la = np.log(r.uniform(0.3, 1.0, (T, H, dk))).astype(np.float32)
    beta = r.uniform(0.05, 1.0, (T, H)).astype(np.float32)
    return q, k, v, la, beta


def _loss(oracle_mod, q, k, v, la, beta, S0, d_o, dS_T, cu, scale):
    o, S_T = oracle_mod.recurrence(q, k, v, la, beta, S0=S0, cu_seqlens=cu, scale=scale)
    return float((o * d_o).sum() + (S_T * dS_T).sum())


def test_finite_differences(oracle_mod):
    """Every gradient against central differences of the forward oracle along random directions,
    two packed sequences, non-zero S0 and dS_T.  The inputs are float32 arrays, so the probe points
    are chosen exactly representable (step 2^-7 on values rounded to 2^-10)."""
    T, H, dk, dv = 11, 2, 5, 4
    q, k, v, la, beta = (np.round(x * 1024) / 1024 for x in _rand(T, H, dk, dv, 1))
    r = np.random.default_rng(2)
    cu = np.array([0, 4, 11])
    S0 = r.standard_normal((2, H, dk, dv))
    d_o = r.standard_normal((T, H, dv))
    dS_T = r.standard_normal((2, H, dk, dv))
    scale = 0.75
    g = oracle_mod.backward(q, k, v, la, beta, d_o=d_o, dS_T=dS_T, S0=S0, cu_seqlens=cu, scale=scale)
    base = dict(q=q, k=k, v=v, la=la, beta=beta)
    names = {"q": "dq", "k": "dk", "v": "dv", "la": "dlog_alpha", "beta": "dbeta"}
    eps = 2.0 ** -7
    for name, gname in names.items():
        for trial in range(3):
            # direction with entries in {-1, 0, 1}: the perturbed inputs stay exact in float32
            d = r.integers(-1, 2, base[name].shape).astype(np.float64)
            args_p = {n: (x + eps * d).astype(np.float32) if n == name else x for n, x in base.items()}
            args_m = {n: (x - eps * d).astype(np.float32) if n == name else x for n, x in base.items()}
            assert np.array_equal(args_p[name].astype(np.float64), base[name] + eps * d)
            lp = _loss(oracle_mod, args_p["q"], args_p["k"], args_p["v"], args_p["la"], args_p["beta"], S0, d_o, dS_T, cu, scale)
            lm = _loss(oracle_mod, args_m["q"], args_m["k"], args_m["v"], args_m["la"], args_m["beta"], S0, d_o, dS_T, cu, scale)
            fd = (lp - lm) / (2 * eps)
            an = float((g[gname] * d).sum())
            # central differences: error O(eps^2 * third derivative)
            assert abs(fd - an) <= 2e-3 * max(1.0, abs(an)), (name, trial, fd, an)
    # dS0 exactly (the loss is linear in S0)
    d = r.standard_normal(S0.shape)
    l1 = _loss(oracle_mod, q, k, v, la, beta, S0 + d, d_o, dS_T, cu, scale)
    l0 = _loss(oracle_mod, q, k, v, la, beta, S0, d_o, dS_T, cu, scale)
    np.testing.assert_allclose(l1 - l0, (g["dS0"] * d).sum(), rtol=1e-9, atol=1e-9)


def test_one_token_closed_form(oracle_mod):
    """T = 1: S_1 = (I - beta k k^T) Diag(alpha) S_0 + beta k v^T and o = scale S_1^T q, differentiated
    by matrix calculus written out with numpy."""
    H, dk, dv = 1, 4, 3
    q, k, v, la, beta = _rand(1, H, dk, dv, 5)
    r = np.random.default_rng(6)
    S0 = r.standard_normal((1, H, dk, dv))
    d_o = r.standard_normal((1, H, dv))
    dS_T = r.standard_normal((1, H, dk, dv))
    sc = 1.25
    g = oracle_mod.backward(q, k, v, la, beta, d_o=d_o, dS_T=dS_T, S0=S0, scale=sc)
    qq, kk, vv = (x[0, 0].astype(np.float64) for x in (q, k, v))
    al = np.exp(la[0, 0].astype(np.float64))
    b = float(beta[0, 0])
    Sd = al[:, None] * S0[0, 0]
    Lam = dS_T[0, 0] + sc * np.outer(qq, d_o[0, 0])          # dL/dS_1
    Pm = np.eye(dk) - b * np.outer(kk, kk)
    S1 = Pm @ Sd + b * np.outer(kk, vv)
    np.testing.assert_allclose(g["dq"][0, 0], sc * S1 @ d_o[0, 0], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g["dv"][0, 0], b * Lam.T @ kk, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g["dS0"][0, 0], al[:, None] * (Pm.T @ Lam), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g["dlog_alpha"][0, 0], ((Pm.T @ Lam) * Sd).sum(1), rtol=1e-12, atol=1e-12)
    rr = vv - Sd.T @ kk
    np.testing.assert_allclose(g["dbeta"][0, 0], kk @ Lam @ rr, rtol=1e-12, atol=1e-12)
    # d/dk of <Lam, -b k k^T Sd + b k v^T>
    np.testing.assert_allclose(g["dk"][0, 0], b * (Lam @ rr) - b * Sd @ (Lam.T @ kk), rtol=1e-12, atol=1e-12)


def test_zero_beta_is_pure_decay(oracle_mod):
    """beta = 0: S_t = Diag(prod alpha) S_0, o_t = scale (Gamma_t . q_t)^T S_0; dk = dv = 0 and the
    other gradients have closed forms with cumulative decays."""
    T, H, dk, dv = 9, 1, 3, 2
    q, k, v, la, beta = _rand(T, H, dk, dv, 7)
    beta[:] = 0
    r = np.random.default_rng(8)
    S0 = r.standard_normal((1, H, dk, dv))
    d_o = r.standard_normal((T, H, dv))
    g = oracle_mod.backward(q, k, v, la, beta, d_o=d_o, S0=S0, scale=1.0)
    assert np.abs(g["dk"]).max() == 0 and np.abs(g["dv"]).max() == 0
    G = np.exp(np.cumsum(la[:, 0].astype(np.float64), axis=0))          # [T,dk]
    np.testing.assert_allclose(g["dq"][:, 0], G * (d_o[:, 0] @ S0[0, 0].T), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g["dS0"][0, 0], np.einsum("td,tj->dj", G * q[:, 0], d_o[:, 0]), rtol=1e-12, atol=1e-12)
    # dL/dlog_alpha_s = sum_{t>=s} (Gamma_t . q_t) . (S_0 d_o_t)
    contrib = G * q[:, 0] * (d_o[:, 0] @ S0[0, 0].T)
    np.testing.assert_allclose(g["dlog_alpha"][:, 0], np.cumsum(contrib[::-1], axis=0)[::-1], rtol=1e-12, atol=1e-12)


def test_linear_in_cotangents_and_sequences_independent(oracle_mod):
    T, H, dk, dv = 14, 2, 4, 4
    q, k, v, la, beta = _rand(T, H, dk, dv, 9)
    r = np.random.default_rng(10)
    cu = np.array([0, 6, 6, 14])      # the middle sequence is empty
    S0 = r.standard_normal((3, H, dk, dv))
    d1, d2 = r.standard_normal((T, H, dv)), r.standard_normal((T, H, dv))
    e1, e2 = r.standard_normal((3, H, dk, dv)), r.standard_normal((3, H, dk, dv))
    ga = oracle_mod.backward(q, k, v, la, beta, d_o=d1, dS_T=e1, S0=S0, cu_seqlens=cu)
    gb = oracle_mod.backward(q, k, v, la, beta, d_o=d2, dS_T=e2, S0=S0, cu_seqlens=cu)
    gc = oracle_mod.backward(q, k, v, la, beta, d_o=2 * d1 - d2, dS_T=2 * e1 - e2, S0=S0, cu_seqlens=cu)
    for n in ga:
        np.testing.assert_allclose(gc[n], 2 * ga[n] - gb[n], rtol=1e-10, atol=1e-10)
    # an empty sequence passes its cotangent straight through; the others do not see each other
    np.testing.assert_allclose(ga["dS0"][1], e1[1], rtol=0, atol=0)
    alone = oracle_mod.backward(q[6:], k[6:], v[6:], la[6:], beta[6:], d_o=d1[6:], dS_T=e1[2:], S0=S0[2:])
    for n in ("dq", "dk", "dv", "dlog_alpha", "dbeta"):
        np.testing.assert_allclose(ga[n][6:], alone[n], rtol=0, atol=0)
