"""Brute-force forms for tiny sequences (L <= 16 or so), fp64 numpy.

TEST INFRASTRUCTURE ONLY.  The column masks of Section 4.1 are materialised as L x L
matrices and the Gated DeltaNet state is written as the explicit sum of matrix products
obtained by unrolling the recurrence of Section 4.3; nothing here is recurrent.
"""
from __future__ import annotations

import numpy as np


def masks(route):
    """M^nla_ij = 1 iff token j is a softmax token and i >= j; M^la likewise for linear tokens.

    (The second case line of the paper's mask equations is read as "0 otherwise".)
    """
    r = np.asarray(route).astype(bool)
    L = r.shape[0]
    causal = np.tril(np.ones((L, L), bool))
    return causal & r[None, :], causal & ~r[None, :]


def softmax_branch(q, k, v, route, scale):
    """O_nla = (exp(A) . M^nla / rowsum) V  for ONE (batch, head); empty rows give 0."""
    q, k, v = (np.asarray(a, np.float64) for a in (q, k, v))
    m_nla, _ = masks(route)
    A = scale * (q @ k.T)
    E = np.where(m_nla, np.exp(A - A.max()), 0.0)
    Z = E.sum(1, keepdims=True)
    Pm = np.divide(E, Z, out=np.zeros_like(E), where=Z > 0)
    return Pm @ v


def linear_branch(q, k, v, g, beta, route, scale, state_in=None):
    """o_la via the unrolled product form of the gated delta rule, ONE (batch, head).

    With M_m = alpha_m (I - beta~_m k_m^T k_m)  (dk x dk) and beta~ = beta where the token is
    linear (column of M^la) and 0 where it is a softmax token:
        S_i = (M_i ... M_0) S_in + sum_{j<=i} (M_i M_{i-1} ... M_{j+1}) beta~_j k_j^T v_j
    """
    q, k, v, g, beta = (np.asarray(a, np.float64) for a in (q, k, v, g, beta))
    L, d = q.shape
    bt = np.where(np.asarray(route).astype(bool), 0.0, beta)
    M = [np.exp(g[m]) * (np.eye(d) - bt[m] * np.outer(k[m], k[m])) for m in range(L)]
    o = np.zeros((L, d))
    S_last = None
    for i in range(L):
        S = np.zeros((d, d))
        for j in range(i + 1):
            prod = np.eye(d)
            for m in range(i, j, -1):       # M_i M_{i-1} ... M_{j+1}
                prod = prod @ M[m]
            S += prod @ (bt[j] * np.outer(k[j], v[j]))
        if state_in is not None:
            prod = np.eye(d)
            for m in range(i, -1, -1):
                prod = prod @ M[m]
            S += prod @ np.asarray(state_in, np.float64)
        o[i] = scale * (q[i] @ S)
        S_last = S
    return o, S_last


def combine(o_nla, o_la, w, eps):
    """out = w_nla Norm(o_nla) + w_la Norm(o_la), Norm = RMS normalisation over d."""
    def norm(x):
        return x / np.sqrt((x * x).mean(-1, keepdims=True) + eps)
    return w[..., 0:1] * norm(o_nla) + w[..., 1:2] * norm(o_la)
