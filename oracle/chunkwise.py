"""Chunkwise (WY / UT-transform) restatement of the linear branch in fp64 numpy.

TEST INFRASTRUCTURE ONLY.  It exists to cross-check the token-by-token recurrence of
``natsl_oracle.c``: Section 3's chunkwise form (S[t+1] = S[t] + g1(K,V,S),
O[t] = Q S[t]^T + (Q K^T . M_C) g2(K,V)) specialised to the Gated DeltaNet update of
Section 4.3 with the per-token route folded in as beta~ = (1 - route) * beta.

Per chunk, with G_i the inclusive cumulative log-decay inside the chunk,
gamma_i = exp(G_i) and Gamma_ij = exp(G_i - G_j) for i >= j:

    A_ij = beta~_i Gamma_ij (k_i . k_j)          (j <  i)
    T    = (I + A)^-1
    U    = T diag(beta~) V ,  W = T diag(beta~ gamma) K
    P_ij = scale (q_i . k_j) Gamma_ij            (j <= i)
    U~   = U - W S
    O    = scale diag(gamma) Q S + P U~
    S   <- gamma_C S + (diag(gamma_C / gamma) K)^T U~
"""
from __future__ import annotations

import numpy as np


def gdn_chunkwise(q, k, v, g, beta, route, C, scale, state_in=None):
    """q,k,v [L,d]; g,beta,route [L] for ONE (batch, head).  Returns (o_la [L,d], S [d,d])."""
    q, k, v, g, beta = (np.asarray(a, np.float64) for a in (q, k, v, g, beta))
    L, d = q.shape
    assert L % C == 0
    bt = beta * (1.0 - np.asarray(route, np.float64))
    S = np.zeros((d, d)) if state_in is None else np.array(state_in, np.float64)
    o = np.zeros((L, d))
    for c in range(L // C):
        sl = slice(c * C, (c + 1) * C)
        Q, K, V, b = q[sl], k[sl], v[sl], bt[sl]
        G = np.cumsum(g[sl])
        gam = np.exp(G)
        Gam = np.exp(np.minimum(G[:, None] - G[None, :], 0.0))  # only i >= j is used
        KK = K @ K.T
        A = np.tril(b[:, None] * Gam * KK, -1)
        T = np.linalg.solve(np.eye(C) + A, np.eye(C))
        U = T @ (b[:, None] * V)
        W = T @ ((b * gam)[:, None] * K)
        P = np.tril(scale * (Q @ K.T) * Gam, 0)
        Ut = U - W @ S
        o[sl] = scale * gam[:, None] * (Q @ S) + P @ Ut
        Kt = (np.exp(G[-1] - G))[:, None] * K
        S = gam[-1] * S + Kt.T @ Ut
    return o, S
