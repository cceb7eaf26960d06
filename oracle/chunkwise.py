"""Chunkwise KDA in numpy fp64: TEST INFRASTRUCTURE ONLY (a cross-check of the oracle).

An independent statement of the chunkwise algorithm of Section 3.1 of the Kimi Linear paper, taken
in the paper's order and notation with library routines for the linear algebra:

  * cumulative log-decay inside a chunk,  G_r = sum_{s<=r} log alpha_s,  Gamma = exp(G)
    ("Decay Formulation", Section 2.1);
  * UT transform:  M = (I + StrictTril(Diag(beta) (Gamma.K) (K/Gamma)^T))^{-1} Diag(beta),
    W = M (Gamma.K),  U = M V   (Section 3.1, "UT transform");
  * pseudo-values  V_new = U - W S,  output  O = (Gamma.Q) S + Tril((Gamma.Q)(K/Gamma)^T) V_new
    (Section 3.1, output equation);
  * state hand-over  S <- Diag(gamma^C) S + ((gamma^C / Gamma) . K)^T V_new
    (Section 3.1, chunk state update; gamma^C/gamma^i is the decay from token i, exclusive, to the
    chunk end).

A short last chunk is handled by running the same formulas on the rows that exist.  The decay
ratios are evaluated as exp(G_i - G_j) entry by entry, so no 1/Gamma is ever formed.
"""
from __future__ import annotations

import numpy as np


def chunk_kda_np(q, k, v, log_alpha, beta, S0=None, chunk=64, scale=1.0):
    """One sequence.  q,k,log_alpha [T,H,dk]; v [T,H,dv]; beta [T,H]; S0 [H,dk,dv] or None.
    Returns (o [T,H,dv], S_T [H,dk,dv]) in float64."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    g = np.asarray(log_alpha, dtype=np.float64)
    beta = np.asarray(beta, dtype=np.float64)
    T, H, dk = k.shape
    dv = v.shape[-1]
    o = np.zeros((T, H, dv))
    S_T = np.zeros((H, dk, dv))
    for h in range(H):
        S = np.zeros((dk, dv)) if S0 is None else np.array(S0[h], dtype=np.float64)
        for c0 in range(0, T, chunk):
            c1 = min(T, c0 + chunk)
            L = c1 - c0
            Q, K, V = q[c0:c1, h] * scale, k[c0:c1, h], v[c0:c1, h]
            b = beta[c0:c1, h]
            G = np.cumsum(g[c0:c1, h], axis=0)                      # [L,dk]
            # D[i,j,:] = exp(G_i - G_j): decay from token j (exclusive) to token i (inclusive)
            D = np.exp(np.clip(G[:, None, :] - G[None, :, :], None, 0.0))
            KK = np.einsum("id,jd,ijd->ij", K, K, D)
            QK = np.einsum("id,jd,ijd->ij", Q, K, D)
            A = np.tril(b[:, None] * KK, -1)                        # StrictTril(Diag(beta) ...)
            M = np.linalg.solve(np.eye(L) + A, np.diag(b))
            W = M @ (np.exp(G) * K)
            U = M @ V
            Vn = U - W @ S
            o[c0:c1, h] = (np.exp(G) * Q) @ S + np.tril(QK) @ Vn
            S = np.exp(G[-1])[:, None] * S + (np.exp(G[-1][None, :] - G) * K).T @ Vn
        S_T[h] = S
    return o, S_T


def chunk_dplr_np(q, k, v, a, b, g, S0=None, chunk=64, scale=1.0):
    """Chunkwise form of the general diagonal-plus-low-rank recurrence (Section 6.1, "Relation to
    DPLR"; the structure of the paper's chunkwise DPLR pseudo-code), one sequence, numpy fp64.  A
    cross-check of ``dplr_recurrence``, not the oracle.

    With G the cumulative log-decay inside the chunk, x_i = S_{i-1}^T a_i the contraction of a with
    the state before token i, and S the state entering the chunk:

      * four gated Gram matrices, the row factor of a stopping one token early:
        Aab[i,j] = sum_d a_i exp(G_{i-1} - G_j) b_j,  Aak likewise with k_j      (j < i)
        Aqb[i,j] = sum_d q_i exp(G_i - G_j) b_j,      Aqk likewise with k_j      (j <= i);
      * X = (I - Aab)^-1 (Atil S + Aak V)  with  Atil_i = a_i exp(G_{i-1}), i.e. X = u + w S;
      * O = (q . exp(G)) S + Aqb X + Aqk V;
      * S <- Diag(exp(G_C)) S + (k . exp(G_C - G))^T V + (b . exp(G_C - G))^T X.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    T, H, dk = k.shape
    dv = v.shape[-1]
    o = np.zeros((T, H, dv))
    S_T = np.zeros((H, dk, dv))
    for h in range(H):
        S = np.zeros((dk, dv)) if S0 is None else np.array(S0[h], dtype=np.float64)
        for c0 in range(0, T, chunk):
            c1 = min(T, c0 + chunk)
            L = c1 - c0
            Q, K, V = q[c0:c1, h] * scale, k[c0:c1, h], v[c0:c1, h]
            A, B, gg = a[c0:c1, h], b[c0:c1, h], g[c0:c1, h]
            G = np.cumsum(gg, axis=0)
            Gm = G - gg                                            # G_{i-1}
            Dq = np.exp(np.clip(G[:, None, :] - G[None, :, :], None, 0.0))     # exp(G_i - G_j), j <= i
            Da = np.exp(np.clip(Gm[:, None, :] - G[None, :, :], None, 0.0))    # exp(G_{i-1} - G_j), j < i
            Aqk = np.tril(np.einsum("id,jd,ijd->ij", Q, K, Dq))
            Aqb = np.tril(np.einsum("id,jd,ijd->ij", Q, B, Dq))
            Aab = np.tril(np.einsum("id,jd,ijd->ij", A, B, Da), -1)
            Aak = np.tril(np.einsum("id,jd,ijd->ij", A, K, Da), -1)
            X = np.linalg.solve(np.eye(L) - Aab, (A * np.exp(Gm)) @ S + Aak @ V)
            o[c0:c1, h] = (Q * np.exp(G)) @ S + Aqb @ X + Aqk @ V
            dec = np.exp(G[-1][None, :] - G)
            S = np.exp(G[-1])[:, None] * S + (K * dec).T @ V + (B * dec).T @ X
        S_T[h] = S
    return o, S_T
