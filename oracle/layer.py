"""KDA layer wrap in numpy fp64: TEST INFRASTRUCTURE ONLY.

What surrounds the recurrence inside one KDA layer (paper Section 4, "Neural Parameterization"),
between the activations that leave the short convolutions and the input of the output projection:

  * q, k = L2Norm(q_c), L2Norm(k_c) over the head dimension (q then carries the caller's `scale`
    inside the recurrence);
  * log alpha = -exp(A_log[h]) * softplus(g_a + dt_bias[h, :]).  The paper only says that the decay
    function f is "similar to those used in GDN and Mamba"; this is that family's form (a negative
    per-head rate times a softplus of the biased pre-activation), the reading taken here;
  * beta = sigmoid(b_pre);
  * o = KDA(q, k, v, alpha, beta): Eq. 1 through ``oracle.recurrence``;
  * y = sigmoid(g_o) . RMSNorm(o) . w, the head-wise RMSNorm over the dv values of one token and
    head, with a learned weight w[dv] (the last equation of that section, before W_o).
"""
from __future__ import annotations

import numpy as np


def l2norm(x, eps):
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt((x * x).sum(-1, keepdims=True) + eps)


def softplus(x):
    x = np.asarray(x, dtype=np.float64)
    return np.maximum(x, 0.0) + np.log1p(np.exp(-np.abs(x)))


def sigmoid(x):
    x = np.asarray(x, dtype=np.float64)
    return 1.0 / (1.0 + np.exp(-x))


def layer_inputs(q_c, k_c, g_a, b_pre, A_log, dt_bias, l2_eps=1e-6):
    """The recurrence's inputs from the layer's pre-activations: (q, k, log_alpha, beta) in fp64."""
    q = l2norm(q_c, l2_eps)
    k = l2norm(k_c, l2_eps)
    A = np.exp(np.asarray(A_log, dtype=np.float64))[None, :, None]
    log_alpha = -A * softplus(np.asarray(g_a, dtype=np.float64) + np.asarray(dt_bias, dtype=np.float64)[None])
    return q, k, log_alpha, sigmoid(b_pre)


def output_gate(o, g_o, w, rms_eps=1e-5):
    o = np.asarray(o, dtype=np.float64)
    rstd = 1.0 / np.sqrt((o * o).mean(-1, keepdims=True) + rms_eps)
    return sigmoid(g_o) * (o * rstd) * np.asarray(w, dtype=np.float64)


def layer_forward(recurrence, q_c, k_c, v, g_a, b_pre, g_o, A_log, dt_bias, w, S0=None, cu_seqlens=None,
                  scale=1.0, l2_eps=1e-6, rms_eps=1e-5):
    """Whole wrap.  ``recurrence`` is ``oracle.recurrence`` (passed in: this module imports nothing
    of the package).  The recurrence takes float32 inputs, so q, k, log_alpha and beta are rounded to
    float32 on the way in (2^-24 relative, far below every tolerance that uses this).  Returns
    (y [T,H,dv], S_T [N,H,dk,dv], o [T,H,dv]) in fp64."""
    q, k, la, beta = layer_inputs(q_c, k_c, g_a, b_pre, A_log, dt_bias, l2_eps)
    o, S_T = recurrence(q.astype(np.float32), k.astype(np.float32), np.asarray(v, dtype=np.float32),
                        la.astype(np.float32), beta.astype(np.float32), S0=S0, cu_seqlens=cu_seqlens, scale=scale)
    return output_gate(o, g_o, w, rms_eps), S_T, o
