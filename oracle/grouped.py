"""fp64 CPU oracle of the layer with grouped softmax heads and per-branch q/k normalisation --
TEST INFRASTRUCTURE ONLY (see the package docstring for who may import it).

Section 4.3: several softmax heads are grouped under one linear-attention head and share its
operation mask; q and k are L2-normalised for the linear operation and RMS-normalised for the
softmax operation; both operations share the same q, k, v.  Appendix (model hyper-parameters):
two or three softmax heads per linear head.

The paper does not say how one q, k, v splits into heads of two different counts.  The reading taken
here: the G softmax heads of a group are the G equal column slices of their linear head, i.e. for
q, k, v [B,L,H,d] the linear operation of head h uses all d columns and softmax head (h, s) uses the
columns [s d/G, (s+1) d/G); all of them use route[:, :, h].  The output of softmax head (h, s) fills
the same columns of o_nla[:, :, h]; the Norm of the output equation is taken per head of the operation
that produced it (each softmax head's slice on its own, the linear head's row as a whole), and the two
weights stay per linear head.

Everything is written as plain torch fp64 operations in the order of the definitions (token-by-token
delta rule, Section 4.3 GDN equation with decay on every token; masked softmax, Section 4.1 O_nla
equation; Norm equation), and the gradients come from reverse-mode differentiation of exactly these
statements.  With G = 1 and no normalisation this is the layer of `natsl_oracle.c`, against which
the tests pin it.
"""
from __future__ import annotations

import numpy as np
import torch


def l2_normalise(x, norm_eps):
    """x / sqrt(sum_d x^2 + norm_eps) over the last axis (linear operation, Section 4.3)."""
    return x / torch.sqrt((x * x).sum(-1, keepdim=True) + norm_eps)


def rms_normalise(x, norm_eps):
    """x / sqrt(mean_d x^2 + norm_eps) over the last axis, no gain (softmax operation, Section 4.3)."""
    return x / torch.sqrt((x * x).mean(-1, keepdim=True) + norm_eps)


def _forward(q, k, v, g, beta, route, w, G, qk_norm, scale_la, scale_sm, eps, norm_eps, state_in, block=None,
             masks=None):
    # masks (block mode only): [B, L/block, H, 2] of ones = (linear, softmax) operation masks of the blocks,
    # present so that their gradients can be taken (Section 4.2): the linear one multiplies the update a
    # linear block commits to the state, the softmax one multiplies the unnormalised probabilities of a
    # softmax block's keys.
    B, L, H, d = q.shape
    ds = d // G
    lin = (route == 0).to(q.dtype)                       # [B,L,H]: 1 for linear tokens
    # ---- linear operation: gated delta rule over all d columns of the head ----
    q_la = l2_normalise(q, norm_eps) if qk_norm else q
    k_la = l2_normalise(k, norm_eps) if qk_norm else k
    S = state_in if state_in is not None else q.new_zeros((B, H, d, d))
    o_la = []
    for i in range(L):
        if block and i % block == 0:
            S_start, decay = S, torch.ones_like(g[:, i])  # state and decay since the block began
        S = torch.exp(g[:, i])[:, :, None, None] * S     # decay on every token
        ki, vi = k_la[:, i], v[:, i]
        err = vi - torch.einsum("bha,bhac->bhc", ki, S)
        if block:
            # block-level routing (Section 4.1): the decision is known only at the block's end, so
            # every token of the block runs the delta rule ...
            bt = beta[:, i][:, :, None, None]
            decay = decay * torch.exp(g[:, i])
        else:
            bt = (beta[:, i] * lin[:, i])[:, :, None, None]  # softmax tokens do not write the state
        S = S + bt * ki[:, :, :, None] * err[:, :, None, :]
        o_la.append(scale_la * torch.einsum("bha,bhac->bhc", q_la[:, i], S))
        if block and i % block == block - 1:
            # ... and a softmax block's update is rolled back: only the decay remains
            keep = lin[:, i][:, :, None, None]
            rolled = decay[:, :, None, None] * S_start
            if masks is not None:        # S_next = decay S_start + m_la U, U = the block's update
                S = rolled + keep * masks[:, i // block, :, 0][:, :, None, None] * (S - rolled)
            else:
                S = keep * S + (1 - keep) * rolled
    o_la = torch.stack(o_la, 1)                          # [B,L,H,d]
    # ---- softmax operation: G heads per linear head, keys = retained tokens j <= i ----
    qs, ks, vs = (x.reshape(B, L, H, G, ds) for x in (q, k, v))
    if qk_norm:
        qs, ks = rms_normalise(qs, norm_eps), rms_normalise(ks, norm_eps)
    logits = scale_sm * torch.einsum("blhsa,bmhsa->bhslm", qs, ks)          # [B,H,G,L(query),L(key)]
    causal = torch.tril(torch.ones((L, L), dtype=torch.bool))
    vis = causal[None, None] & (route != 0).permute(0, 2, 1)[:, :, None, :]  # [B,H,L,L]
    if block:         # both operations read the query's own block
        blk = torch.arange(L) // block
        vis = vis | (causal & (blk[:, None] == blk[None, :]))[None, None]
    vis = vis[:, :, None]                                                    # same for every head of the group
    neg = torch.full_like(logits, -np.inf)
    masked = torch.where(vis, logits, neg)
    m = masked.max(-1, keepdim=True).values
    m_safe = torch.where(torch.isfinite(m), m, torch.zeros_like(m))
    p = torch.exp(masked - m_safe)                       # exp(-inf) = 0 at the keys a query does not see
    if masks is not None:
        # the softmax mask of key j's block, for every query that sees the key (what it does to the keys of a
        # linear block, seen inside their own block only, is discarded: that block did not choose softmax)
        blk = torch.arange(L) // block
        mk = masks[:, :, :, 1].permute(0, 2, 1)[:, :, blk]                    # [B,H,L(key)]
        p = p * mk[:, :, None, None, :]
    z = p.sum(-1, keepdim=True)
    any_key = z > 0
    p = p / torch.where(any_key, z, torch.ones_like(z))
    o_nla = torch.einsum("bhslm,bmhsc->blhsc", p, vs)                        # [B,L,H,G,ds]
    lse = torch.where(any_key, m_safe + torch.log(torch.where(any_key, z, torch.ones_like(z))),
                      torch.full_like(z, -np.inf))[..., 0]                   # [B,H,G,L]
    # ---- output: Norm per head of the producing operation, weights per linear head ----
    y_nla = o_nla * torch.rsqrt((o_nla * o_nla).mean(-1, keepdim=True) + eps)
    y_la = o_la * torch.rsqrt((o_la * o_la).mean(-1, keepdim=True) + eps)
    w_nla = w[..., 0:1] if w is not None else 0.5
    w_la = w[..., 1:2] if w is not None else 0.5
    out = w_nla * y_nla.reshape(B, L, H, d) + w_la * y_la
    return dict(out=out, o_la=o_la, o_nla=o_nla.reshape(B, L, H, d), lse=lse, state_out=S)


def _t(a, grad=False):
    if a is None:
        return None
    x = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64)).clone()
    return x.requires_grad_(grad)


def _check(q, route, G, block=None):
    B, L, H, d = q.shape
    if G < 1 or d % G:
        raise ValueError("G must divide the head dimension")
    if route.shape != (B, L, H):
        raise ValueError("route must be [B,L,H]")
    if block:
        r = np.asarray(route).reshape(B, L // block, block, H) if L % block == 0 else None
        if r is None or (r != r[:, :, :1]).any():
            raise ValueError("block mode: route must be constant within each block")


def hybrid_fwd(q, k, v, g, beta, route, w=None, *, G=1, qk_norm=False, scale_la, scale_sm, eps=1e-5,
               norm_eps=1e-6, state_in=None, block=None):
    """q,k,v [B,L,H,d]; g,beta,route [B,L,H]; w [B,L,H,2] or None; G softmax heads per linear head.
    block=R: block-level routing (route constant per block of R tokens, Section 4.1).
    Returns dict(out, o_la, o_nla [B,L,H,d]; lse [B,H,G,L]; state_out [B,H,d,d]) as numpy float64."""
    _check(np.asarray(q), np.asarray(route), G, block)
    with torch.no_grad():
        res = _forward(_t(q), _t(k), _t(v), _t(g), _t(beta), torch.from_numpy(np.asarray(route).astype(np.int64)),
                       _t(w), G, qk_norm, scale_la, scale_sm, eps, norm_eps, _t(state_in), block)
    return {n: x.numpy() for n, x in res.items()}


def hybrid_bwd(q, k, v, g, beta, route, w, dout, *, G=1, qk_norm=False, scale_la, scale_sm, eps=1e-5,
               norm_eps=1e-6, state_in=None, dstate_out=None, block=None, want_dscore=False):
    """Gradients of <out, dout> (+ <state_out, dstate_out>) with respect to q, k, v, g, beta, w and
    state_in.  Returns dict(dq, dk, dv, dg, dbeta, dw, dstate_in)."""
    _check(np.asarray(q), np.asarray(route), G, block)
    B, L, H, d = np.asarray(q).shape
    if w is None:
        w = np.full((B, L, H, 2), 0.5)
    if state_in is None:
        state_in = np.zeros((B, H, d, d))
    leaves = [_t(x, True) for x in (q, k, v, g, beta, w, state_in)]
    tq, tk, tv, tg, tb, tw, ts = leaves
    masks = None
    if want_dscore:
        if not block:
            raise ValueError("score gradients: one decision per block")
        masks = torch.ones((B, L // block, H, 2), dtype=torch.float64, requires_grad=True)
        leaves = leaves + [masks]
    res = _forward(tq, tk, tv, tg, tb, torch.from_numpy(np.asarray(route).astype(np.int64)), tw, G, qk_norm,
                   scale_la, scale_sm, eps, norm_eps, ts, block, masks)
    loss = (res["out"] * _t(dout)).sum()
    if dstate_out is not None:
        loss = loss + (res["state_out"] * _t(dstate_out)).sum()
    grads = torch.autograd.grad(loss, leaves, allow_unused=True)
    names = ("dq", "dk", "dv", "dg", "dbeta", "dw", "dstate_in", "dscore")
    out = {n: (np.zeros(tuple(x.shape)) if gr is None else gr.numpy()) for n, gr, x in zip(names, grads, leaves)}
    if want_dscore:      # only the operation a block chose has a mask gradient ("d score = 0 if the mask is 0")
        blocks = np.asarray(route)[:, ::block]                                # [B, L/block, H]
        out["dscore"][..., 0][blocks != 0] = 0.0
        out["dscore"][..., 1][blocks == 0] = 0.0
    return out
