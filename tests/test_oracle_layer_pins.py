"""Pins of the layer-wrap oracle (oracle/layer.py: L2Norm, decay function, beta, head-wise RMSNorm and
output gate around Eq. 1; paper Section 4) against facts its formulas do not state."""
import numpy as np

from oracle import layer


def _case(seed, T=23, H=2, d=8):
    r = np.random.default_rng(seed)
    return dict(q_c=r.standard_normal((T, H, d)) * 3, k_c=r.standard_normal((T, H, d)) * 0.2,
                v=r.standard_normal((T, H, d)), g_a=r.standard_normal((T, H, d)) - 2,
                b_pre=r.standard_normal((T, H)), g_o=r.standard_normal((T, H, d)),
                A_log=r.standard_normal(H) * 0.3, dt_bias=r.standard_normal((H, d)) * 0.3,
                w=1 + 0.1 * r.standard_normal(d))


def test_scalar_functions():
    np.testing.assert_allclose(layer.softplus(0.0), np.log(2.0), rtol=1e-15)
    x = np.linspace(-30, 30, 13)
    np.testing.assert_allclose(layer.softplus(x) - layer.softplus(-x), x, rtol=0, atol=1e-13)   # log(1+e^x) - log(1+e^-x) = x
    np.testing.assert_allclose(layer.softplus(50.0), 50.0, rtol=1e-15)
    np.testing.assert_allclose(layer.sigmoid(x) + layer.sigmoid(-x), 1.0, rtol=0, atol=1e-15)
    np.testing.assert_allclose(np.exp(-layer.softplus(x)), layer.sigmoid(-x), rtol=1e-12)      # e^-softplus(x) = sigmoid(-x)


def test_decay_lies_in_unit_interval_and_matches_sigmoid_power():
    """alpha = exp(-A softplus(z)) = sigmoid(-z)^A: in (0, 1], monotone in z."""
    c = _case(1)
    _, _, la, beta = layer.layer_inputs(c["q_c"], c["k_c"], c["g_a"], c["b_pre"], c["A_log"], c["dt_bias"])
    assert (la <= 0).all() and (beta > 0).all() and (beta < 1).all()
    z = c["g_a"] + c["dt_bias"][None]
    A = np.exp(c["A_log"])[None, :, None]
    np.testing.assert_allclose(np.exp(la), layer.sigmoid(-z) ** A, rtol=1e-12)


def test_l2norm_makes_the_wrap_scale_invariant(oracle_mod):
    """q_c and k_c only enter through their directions: any positive per-token factor drops out."""
    c = _case(2)
    y0, S0_, _ = layer.layer_forward(oracle_mod.recurrence, **c, l2_eps=0.0)
    c2 = dict(c)
    r = np.random.default_rng(3)
    c2["q_c"] = c["q_c"] * r.uniform(0.1, 9, (23, 2, 1))
    c2["k_c"] = c["k_c"] * r.uniform(0.1, 9, (23, 2, 1))
    y1, S1_, _ = layer.layer_forward(oracle_mod.recurrence, **c2, l2_eps=0.0)
    np.testing.assert_allclose(y1, y0, rtol=0, atol=1e-5 * np.abs(y0).max())
    np.testing.assert_allclose(S1_, S0_, rtol=0, atol=1e-5 * np.abs(S0_).max())
    q, k, _, _ = layer.layer_inputs(c["q_c"], c["k_c"], c["g_a"], c["b_pre"], c["A_log"], c["dt_bias"], l2_eps=0.0)
    np.testing.assert_allclose((q * q).sum(-1), 1.0, rtol=1e-12)
    np.testing.assert_allclose((k * k).sum(-1), 1.0, rtol=1e-12)


def test_output_gate_properties():
    """RMSNorm: with unit weight and an open gate every row has mean square 1 (eps = 0); the result
    does not depend on the scale of o; a closed gate (g_o = 0) halves it; the weight multiplies
    column-wise."""
    r = np.random.default_rng(4)
    o = r.standard_normal((7, 3, 16)) * 5
    big = np.full_like(o, 40.0)
    y = layer.output_gate(o, big, np.ones(16), rms_eps=0.0)
    np.testing.assert_allclose((y * y).mean(-1), 1.0, rtol=1e-12)
    np.testing.assert_allclose(layer.output_gate(3.7 * o, big, np.ones(16), rms_eps=0.0), y, rtol=1e-12)
    np.testing.assert_allclose(layer.output_gate(o, np.zeros_like(o), np.ones(16), rms_eps=0.0), 0.5 * y, rtol=1e-12)
    w = r.standard_normal(16)
    np.testing.assert_allclose(layer.output_gate(o, big, w, rms_eps=0.0), y * w, rtol=1e-12)


def test_wrap_is_the_recurrence_on_the_transformed_inputs(oracle_mod):
    """Closed gates in the limit: g_a -> -inf gives alpha = 1 (no decay), b_pre -> +inf gives beta = 1:
    the wrap then is the plain delta rule on the unit vectors, which numpy can run directly."""
    c = _case(5, T=9, H=1, d=4)
    c["g_a"] = np.full_like(c["g_a"], -80.0)
    c["b_pre"] = np.full_like(c["b_pre"], 40.0)
    y, S_T, o = layer.layer_forward(oracle_mod.recurrence, **c, l2_eps=0.0)
    q = c["q_c"] / np.linalg.norm(c["q_c"], axis=-1, keepdims=True)
    k = c["k_c"] / np.linalg.norm(c["k_c"], axis=-1, keepdims=True)
    S = np.zeros((4, 4))
    for t in range(9):
        kk = k[t, 0]
        S = S - np.outer(kk, kk @ S) + np.outer(kk, c["v"][t, 0])
        np.testing.assert_allclose(o[t, 0], S.T @ q[t, 0], rtol=0, atol=1e-6)
    np.testing.assert_allclose(S_T[0, 0], S, rtol=0, atol=1e-6)
