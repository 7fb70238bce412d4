"""Pins of the fp64 oracle against things other than itself: closed forms, special cases that
reduce to a library routine (torch scaled_dot_product_attention, torch autograd), brute force on
tiny inputs, finite differences, and the mask structure of the paper's Fig. 1(c)."""
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import bruteforce, chunkwise

RNG = np.random.default_rng(1234)
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_inputs(B, L, H, d, p=0.3, seed=0, unit=True):
    r = np.random.default_rng(seed)
    q = r.standard_normal((B, L, H, d))
    k = r.standard_normal((B, L, H, d))
    if unit:
        q /= np.linalg.norm(q, axis=-1, keepdims=True)
        k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = r.standard_normal((B, L, H, d))
    g = -np.log1p(np.exp(r.standard_normal((B, L, H))))
    beta = 1 / (1 + np.exp(-r.standard_normal((B, L, H))))
    route = (r.random((B, L, H)) < p).astype(np.uint8)
    wz = np.exp(r.standard_normal((B, L, H, 2)))
    w = wz / wz.sum(-1, keepdims=True)
    return dict(q=q, k=k, v=v, g=g, beta=beta, route=route, w=w)


def fwd(x, scale_la=0.5, scale_sm=1.5, eps=1e-5, **kw):
    return oracle.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x.get("w"),
                             scale_la=scale_la, scale_sm=scale_sm, eps=eps, **kw)


# ------------------------------------------------------------------ compaction
def test_compaction_against_nonzero():
    for (B, L, H, C, p) in [(2, 256, 3, 64, 0.25), (1, 128, 2, 64, 0.0), (1, 128, 2, 64, 1.0),
                            (1, 24, 1, 4, 0.5)]:
        route = (RNG.random((B, L, H)) < p).astype(np.uint8)
        res = oracle.route_compact(route, C)
        NC = L // C
        for b in range(B):
            for h in range(H):
                col = route[b, :, h]
                pos = np.nonzero(col)[0]
                n_sm = len(pos)
                assert res["sm_chunk_prefix"][b, h, NC] == n_sm
                assert np.array_equal(res["sm_idx"][b, h, :n_sm], pos)
                assert n_sm + res["n_lin"][b, h].sum() == L
                cnt = col.reshape(NC, C).sum(1)
                assert np.array_equal(np.diff(res["sm_chunk_prefix"][b, h]), cnt)
                for c in range(NC):
                    lin = np.nonzero(col[c * C:(c + 1) * C] == 0)[0]
                    assert res["n_lin"][b, h, c] == len(lin)
                    assert np.array_equal(res["lin_idx"][b, h, c, :len(lin)], lin)
                    assert np.all(res["lin_idx"][b, h, c, len(lin):] == C)


def test_compaction_single_bit_and_reject():
    route = np.zeros((1, 128, 1), np.uint8)
    route[0, 77, 0] = 1
    res = oracle.route_compact(route, 64)
    assert res["sm_idx"][0, 0, 0] == 77 and list(res["sm_chunk_prefix"][0, 0]) == [0, 0, 1]
    assert list(res["n_lin"][0, 0]) == [64, 63]
    with pytest.raises(ValueError):
        oracle.route_compact(np.zeros((1, 100, 1), np.uint8), 64)


# ------------------------------------------------------------------ linear branch
def test_recurrent_equals_chunkwise():
    x = rand_inputs(2, 192, 2, 16, p=0.3, seed=1)
    S0 = RNG.standard_normal((2, 2, 16, 16))
    r = fwd(x, state_in=S0)
    for b in range(2):
        for h in range(2):
            o, S = chunkwise.gdn_chunkwise(x["q"][b, :, h], x["k"][b, :, h], x["v"][b, :, h],
                                           x["g"][b, :, h], x["beta"][b, :, h], x["route"][b, :, h],
                                           64, 0.5, state_in=S0[b, h])
            np.testing.assert_allclose(o, r["o_la"][b, :, h], rtol=1e-10, atol=1e-12)
            np.testing.assert_allclose(S, r["state_out"][b, h], rtol=1e-10, atol=1e-12)


def test_bruteforce_tiny():
    x = rand_inputs(1, 12, 2, 5, p=0.35, seed=2)
    S0 = RNG.standard_normal((1, 2, 5, 5))
    r = fwd(x, state_in=S0)
    for h in range(2):
        o_la, S = bruteforce.linear_branch(x["q"][0, :, h], x["k"][0, :, h], x["v"][0, :, h],
                                           x["g"][0, :, h], x["beta"][0, :, h], x["route"][0, :, h],
                                           0.5, state_in=S0[0, h])
        o_nla = bruteforce.softmax_branch(x["q"][0, :, h], x["k"][0, :, h], x["v"][0, :, h],
                                          x["route"][0, :, h], 1.5)
        np.testing.assert_allclose(o_la, r["o_la"][0, :, h], rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(S, r["state_out"][0, h], rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(o_nla, r["o_nla"][0, :, h], rtol=1e-10, atol=1e-13)
        out = bruteforce.combine(o_nla, o_la, x["w"][0, :, h], 1e-5)
        np.testing.assert_allclose(out, r["out"][0, :, h], rtol=1e-10, atol=1e-13)


def test_hybrid_equals_pure_gdn_with_masked_beta():
    x = rand_inputs(1, 96, 2, 8, p=0.4, seed=3)
    r = fwd(x)
    y = dict(x)
    y["beta"] = x["beta"] * (1 - x["route"])
    y["route"] = np.zeros_like(x["route"])
    r2 = fwd(y)
    np.testing.assert_allclose(r["o_la"], r2["o_la"], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(r["state_out"], r2["state_out"], rtol=1e-12, atol=1e-15)
    assert np.all(r2["o_nla"] == 0) and np.all(np.isneginf(r2["lse"]))


def test_alpha_one_reduces_to_deltanet_paper_orientation():
    """g = 0, all-linear: the DeltaNet equation of Section 4.3 in the paper's own orientation,
    S in R^{dv x dk}, S_t = S_{t-1}(I - beta k k^T) + beta v k^T, o = S q."""
    x = rand_inputs(1, 40, 1, 6, p=0.0, seed=4)
    x["g"] = np.zeros_like(x["g"])
    r = fwd(x, scale_la=1.0)
    d = 6
    S = np.zeros((d, d))
    for t in range(40):
        k, v, b = x["k"][0, t, 0], x["v"][0, t, 0], x["beta"][0, t, 0]
        S = S @ (np.eye(d) - b * np.outer(k, k)) + b * np.outer(v, k)
        np.testing.assert_allclose(S @ x["q"][0, t, 0], r["o_la"][0, t, 0], rtol=1e-11, atol=1e-14)
    np.testing.assert_allclose(S.T, r["state_out"][0, 0], rtol=1e-11, atol=1e-14)


def test_gdn_paper_orientation_with_decay():
    """All-linear, g != 0: S_t = S_{t-1} alpha_t (I - beta_t k k^T) + beta_t v k^T (Section 4.3)."""
    x = rand_inputs(1, 30, 1, 5, p=0.0, seed=5)
    r = fwd(x, scale_la=1.0)
    S = np.zeros((5, 5))
    for t in range(30):
        k, v, b, a = x["k"][0, t, 0], x["v"][0, t, 0], x["beta"][0, t, 0], np.exp(x["g"][0, t, 0])
        S = S @ (a * (np.eye(5) - b * np.outer(k, k))) + b * np.outer(v, k)
        np.testing.assert_allclose(S @ x["q"][0, t, 0], r["o_la"][0, t, 0], rtol=1e-11, atol=1e-14)


def test_state_invariants_beta_zero():
    x = rand_inputs(1, 64, 1, 8, p=0.3, seed=6)
    S0 = RNG.standard_normal((1, 1, 8, 8))
    x["beta"] = np.zeros_like(x["beta"])
    r = fwd(x, state_in=S0)
    np.testing.assert_allclose(r["state_out"], np.exp(x["g"].sum()) * S0, rtol=1e-12)
    x["g"] = np.zeros_like(x["g"])
    r = fwd(x, state_in=S0)
    assert np.array_equal(r["state_out"], S0)          # bit for bit


def test_decay_always_on_softmax_tokens():
    """All tokens routed to softmax: the state is never written, only decayed, and a softmax
    token's linear read sees the state after its own decay."""
    x = rand_inputs(1, 20, 1, 4, p=1.1, seed=7)
    S0 = RNG.standard_normal((1, 1, 4, 4))
    r = fwd(x, state_in=S0, scale_la=0.7)
    G = np.cumsum(x["g"][0, :, 0])
    np.testing.assert_allclose(r["state_out"][0, 0], np.exp(G[-1]) * S0[0, 0], rtol=1e-12)
    for i in range(20):
        np.testing.assert_allclose(r["o_la"][0, i, 0], 0.7 * np.exp(G[i]) * x["q"][0, i, 0] @ S0[0, 0],
                                   rtol=1e-12)


def test_delta_rule_writes_value():
    """beta = 1 and |k| = 1: after the update, k_t S_t = v_t exactly (delta rule)."""
    x = rand_inputs(1, 10, 1, 6, p=0.0, seed=8)
    x["beta"] = np.ones_like(x["beta"])
    y = dict(x)
    y["q"] = x["k"]
    r = fwd(y, scale_la=1.0)
    np.testing.assert_allclose(r["o_la"], x["v"], rtol=1e-12, atol=1e-13)


def test_orthonormal_keys_plain_linear_attention():
    d = 8
    Q, _ = np.linalg.qr(RNG.standard_normal((d, d)))
    x = rand_inputs(1, d, 1, d, p=0.0, seed=9)
    x["k"] = Q[None, :, None, :].copy()
    x["beta"] = np.ones_like(x["beta"])
    x["g"] = np.zeros_like(x["g"])
    r = fwd(x)
    S = sum(np.outer(Q[j], x["v"][0, j, 0]) for j in range(d))
    np.testing.assert_allclose(r["state_out"][0, 0], S, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ softmax branch
def test_all_softmax_equals_library_causal_attention():
    x = rand_inputs(2, 50, 3, 16, p=1.1, seed=10, unit=False)
    r = fwd(x, scale_sm=0.3)
    tq, tk, tv = (torch.from_numpy(x[n]).permute(0, 2, 1, 3) for n in ("q", "k", "v"))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=0.3)
    np.testing.assert_allclose(r["o_nla"], ref.permute(0, 2, 1, 3).numpy(), rtol=1e-10, atol=1e-12)
    # independent double loop for the log-sum-exp
    for i in (0, 7, 49):
        s = 0.3 * x["k"][1, :i + 1, 2] @ x["q"][1, i, 2]
        assert abs(np.log(np.exp(s).sum()) - r["lse"][1, 2, i]) < 1e-10


def test_mixed_route_equals_library_masked_attention():
    x = rand_inputs(1, 70, 2, 8, p=0.3, seed=11, unit=False)
    x["route"][0, 0, :] = 1                               # no empty rows
    r = fwd(x, scale_sm=0.9)
    tq, tk, tv = (torch.from_numpy(x[n]).permute(0, 2, 1, 3) for n in ("q", "k", "v"))
    L = 70
    keep = torch.from_numpy(x["route"].astype(bool)).permute(0, 2, 1)[:, :, None, :]  # [B,H,1,L]
    mask = torch.tril(torch.ones(L, L, dtype=torch.bool))[None, None] & keep
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask, scale=0.9)
    np.testing.assert_allclose(r["o_nla"], ref.permute(0, 2, 1, 3).numpy(), rtol=1e-10, atol=1e-12)


def test_single_retained_token_and_empty_rows():
    x = rand_inputs(1, 16, 1, 4, p=0.0, seed=12)
    x["route"][0, 5, 0] = 1
    r = fwd(x)
    assert np.all(r["o_nla"][0, :5] == 0) and np.all(np.isneginf(r["lse"][0, 0, :5]))
    for i in range(5, 16):
        np.testing.assert_allclose(r["o_nla"][0, i, 0], x["v"][0, 5, 0], rtol=1e-13)


# ------------------------------------------------------------------ combination
def test_combination_properties():
    x = rand_inputs(1, 32, 2, 16, p=0.3, seed=13)
    x["route"][0, 0, :] = 1
    x["w"] = np.zeros_like(x["w"])
    x["w"][..., 0] = 1.0
    r = fwd(x, eps=1e-12)
    np.testing.assert_allclose(np.sqrt((r["out"] ** 2).mean(-1)), 1.0, rtol=1e-8)
    x["w"][..., 0], x["w"][..., 1] = 0.0, 1.0
    r = fwd(x, eps=1e-12)
    rms = np.sqrt((r["out"] ** 2).mean(-1))
    nz = np.abs(r["o_la"]).max(-1) > 0                    # empty state: Norm(0) = 0
    np.testing.assert_allclose(rms[nz], 1.0, rtol=1e-6)
    assert np.all(rms[~nz] == 0) and nz.sum() > 50
    # all-linear: out = w_la Norm(GDN), the softmax branch contributes Norm(0) = 0
    y = rand_inputs(1, 32, 1, 8, p=0.0, seed=14)
    r = fwd(y)
    o = r["o_la"]
    ref = y["w"][..., 1:2] * o / np.sqrt((o * o).mean(-1, keepdims=True) + 1e-5)
    np.testing.assert_allclose(r["out"], ref, rtol=1e-12, atol=1e-15)
    # w = None means (1/2, 1/2)
    y2 = dict(y)
    y2["w"] = None
    y3 = dict(y)
    y3["w"] = np.full_like(y["w"], 0.5)
    assert np.array_equal(fwd(y2)["out"], fwd(y3)["out"])


# ------------------------------------------------------------------ Fig. 1(c)
def _influence(x, field, i_out, scale=1e-3):
    """|d o[i_out] / d v_j| > 0 pattern by perturbing v_j, j = 0..L-1."""
    base = fwd(x)[field][0, :, 0]
    L = base.shape[0]
    vis = np.zeros((L, L), bool)
    for j in range(L):
        y = {n: a.copy() if isinstance(a, np.ndarray) else a for n, a in x.items()}
        y["v"][0, j, 0] += scale
        vis[:, j] = np.abs(fwd(y)[field][0, :, 0] - base).max(-1) > 0
    return vis


def test_fig1c_visibility_pattern():
    rows = [ln.strip() for ln in open(os.path.join(GOLDEN, "fig1c_visibility.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 12 and all(len(r) == 12 for r in rows)
    fig = np.array([list(r) for r in rows])
    C = 2
    route = np.zeros(12, np.uint8)
    route[[0, 1, 6, 7]] = 1                               # chunks 1 and 4 are softmax chunks
    x = rand_inputs(1, 12, 1, 4, seed=15)
    x["route"] = route[None, :, None].copy()
    x["beta"] = np.full_like(x["beta"], 0.7)
    sm = _influence(x, "o_nla", None)
    la = _influence(x, "o_la", None)
    chunk = np.arange(12) // C
    earlier = chunk[:, None] > chunk[None, :]             # key in an earlier chunk than the query
    # softmax branch: cross-chunk cells are exactly the figure's S cells
    assert np.array_equal(sm & earlier, fig == "S")
    # linear branch: the state a query reads from earlier chunks holds linear tokens up to the
    # column where the figure draws its G cell, and nothing when the row has no G
    for i in range(12):
        cols = np.nonzero(la[i] & earlier[i])[0]
        gcol = np.nonzero(fig[i] == "G")[0]
        if len(gcol) == 0:
            assert len(cols) == 0
        else:
            assert cols.max() == gcol[0]
            assert np.all(route[cols] == 0)
    # each token is visible in exactly one branch, causally
    assert np.array_equal(sm | la, np.tril(np.ones((12, 12), bool)))
    assert not np.any(sm & la)
    m_nla, m_la = bruteforce.masks(route)
    assert np.array_equal(sm, m_nla) and np.array_equal(la, m_la)


# ------------------------------------------------------------------ decode
def test_decode_from_empty_equals_forward_rows():
    x = rand_inputs(2, 24, 2, 8, p=0.3, seed=16)
    r = fwd(x)
    B, L, H, d = x["q"].shape
    state = np.zeros((B, H, d, d))
    kc, vc = np.zeros((B, H, L, d)), np.zeros((B, H, L, d))
    n = np.zeros((B, H), np.int32)
    for t in range(L):
        o = oracle.decode_step(x["q"][:, t], x["k"][:, t], x["v"][:, t], x["g"][:, t],
                               x["beta"][:, t], x["route"][:, t], x["w"][:, t], state, kc, vc, n,
                               scale_la=0.5, scale_sm=1.5)
        np.testing.assert_allclose(o["out"], r["out"][:, t], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(state, r["state_out"], rtol=1e-12, atol=1e-15)
    assert np.array_equal(n, x["route"].sum(1).astype(np.int32))


def test_prefill_handoff_then_one_step():
    x = rand_inputs(1, 33, 2, 8, p=0.3, seed=17)
    full = fwd(x)
    head = {n: (a[:, :32] if a is not None else None) for n, a in x.items()}
    r = fwd(head, want_cache=True)
    state = r["state_out"].copy()
    cap = 40
    kc, vc = np.zeros((1, 2, cap, 8)), np.zeros((1, 2, cap, 8))
    kc[:, :, :32], vc[:, :, :32] = r["k_sm"], r["v_sm"]
    n = r["n_sm"].copy()
    o = oracle.decode_step(x["q"][:, 32], x["k"][:, 32], x["v"][:, 32], x["g"][:, 32],
                           x["beta"][:, 32], x["route"][:, 32], x["w"][:, 32], state, kc, vc, n,
                           scale_la=0.5, scale_sm=1.5)
    np.testing.assert_allclose(o["out"], full["out"][:, 32], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(state, full["state_out"], rtol=1e-12, atol=1e-15)


def test_decode_cache_full():
    x = rand_inputs(1, 1, 1, 4, p=1.1, seed=18)
    state = np.zeros((1, 1, 4, 4))
    kc, vc = np.zeros((1, 1, 2, 4)), np.zeros((1, 1, 2, 4))
    n = np.full((1, 1), 2, np.int32)
    with pytest.raises(OverflowError):
        oracle.decode_step(x["q"][:, 0], x["k"][:, 0], x["v"][:, 0], x["g"][:, 0], x["beta"][:, 0],
                           x["route"][:, 0], None, state, kc, vc, n, scale_la=1.0, scale_sm=1.0)


# ------------------------------------------------------------------ backward
def _loss(x, dout, S0, dS):
    r = fwd(x, state_in=S0)
    return (r["out"] * dout).sum() + (r["state_out"] * dS).sum()


def test_backward_finite_differences():
    B, L, H, d = 1, 20, 2, 6
    x = rand_inputs(B, L, H, d, p=0.3, seed=19, unit=False)
    x["q"] *= 0.5
    x["k"] *= 0.4
    x["route"][0, 0, 0] = 1
    x["route"][0, :3, 1] = 0                               # head 1 starts with empty softmax rows
    dout = RNG.standard_normal((B, L, H, d))
    S0 = RNG.standard_normal((B, H, d, d)) * 0.3
    dS = RNG.standard_normal((B, H, d, d))
    gr = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], dout,
                           scale_la=0.5, scale_sm=1.5, state_in=S0, dstate_out=dS)
    h = 1e-6
    checks = [("q", "dq"), ("k", "dk"), ("v", "dv"), ("g", "dg"), ("beta", "dbeta"), ("w", "dw")]
    pick = np.random.default_rng(5)
    for name, gname in checks:
        flat = x[name].reshape(-1)
        for idx in pick.choice(flat.size, size=min(40, flat.size), replace=False):
            old = flat[idx]
            flat[idx] = old + h
            lp = _loss(x, dout, S0, dS)
            flat[idx] = old - h
            lm = _loss(x, dout, S0, dS)
            flat[idx] = old
            fd = (lp - lm) / (2 * h)
            an = gr[gname].reshape(-1)[idx]
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)) + 1e-7, (name, idx, fd, an)
    flat = S0.reshape(-1)
    for idx in pick.choice(flat.size, size=20, replace=False):
        old = flat[idx]
        flat[idx] = old + h
        lp = _loss(x, dout, S0, dS)
        flat[idx] = old - h
        lm = _loss(x, dout, S0, dS)
        flat[idx] = old
        assert abs((lp - lm) / (2 * h) - gr["dstate_in"].reshape(-1)[idx]) < 2e-6


def _torch_forward(q, k, v, g, beta, route, w, scale_la, scale_sm, eps):
    """Same layer written with torch ops (masked library attention + a python recurrence) so that
    torch autograd differentiates it; one (batch, head)."""
    L, d = q.shape
    S = torch.zeros(d, d, dtype=torch.float64)
    o_la = []
    for i in range(L):
        S = torch.exp(g[i]) * S
        if not route[i]:
            S = S + beta[i] * torch.outer(k[i], v[i] - k[i] @ S)
        o_la.append(scale_la * (q[i] @ S))
    o_la = torch.stack(o_la)
    keep = torch.tensor(route.astype(bool))
    mask = torch.tril(torch.ones(L, L, dtype=torch.bool)) & keep[None, :]
    o_nla = torch.nn.functional.scaled_dot_product_attention(q[None], k[None], v[None],
                                                             attn_mask=mask[None], scale=scale_sm)[0]
    rows = mask.any(1)
    o_nla = torch.where(rows[:, None], o_nla, torch.zeros_like(o_nla))

    def norm(x):
        return x * torch.rsqrt((x * x).mean(-1, keepdim=True) + eps)
    return w[:, 0:1] * norm(o_nla) + w[:, 1:2] * norm(o_la)


def test_backward_equals_autograd():
    B, L, H, d = 1, 48, 1, 8
    x = rand_inputs(B, L, H, d, p=0.3, seed=20)
    x["route"][0, 0, 0] = 1
    dout = RNG.standard_normal((B, L, H, d))
    gr = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], dout,
                           scale_la=0.35, scale_sm=2.8)
    t = {n: torch.tensor(x[n][0, :, 0], dtype=torch.float64, requires_grad=True)
         for n in ("q", "k", "v", "g", "beta", "w")}
    out = _torch_forward(t["q"], t["k"], t["v"], t["g"], t["beta"], x["route"][0, :, 0], t["w"],
                         0.35, 2.8, 1e-5)
    np.testing.assert_allclose(out.detach().numpy(), fwd(x, 0.35, 2.8)["out"][0, :, 0], rtol=1e-10,
                               atol=1e-12)
    (out * torch.from_numpy(dout[0, :, 0])).sum().backward()
    for n, gn in [("q", "dq"), ("k", "dk"), ("v", "dv"), ("g", "dg"), ("beta", "dbeta"), ("w", "dw")]:
        np.testing.assert_allclose(gr[gn][0, :, 0], t[n].grad.numpy(), rtol=1e-8, atol=1e-11,
                                   err_msg=n)


def test_inactive_branch_gradients_vanish():
    """k, v gradients of an operation vanish for tokens that are inactive for it (Section 4.2)."""
    x = rand_inputs(1, 40, 2, 8, p=0.3, seed=21)
    x["route"][0, 0, :] = 1
    dout = RNG.standard_normal(x["q"].shape)
    lin = x["route"] == 0
    only_sm = dict(x)
    only_sm["w"] = np.stack([np.ones_like(x["g"]), np.zeros_like(x["g"])], -1)
    gs = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], only_sm["w"], dout,
                           scale_la=0.5, scale_sm=1.5)
    assert np.all(gs["dk"][lin] == 0) and np.all(gs["dv"][lin] == 0)
    assert np.all(gs["dbeta"] == 0) and np.all(gs["dg"] == 0)
    only_la = np.stack([np.zeros_like(x["g"]), np.ones_like(x["g"])], -1)
    gl = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], only_la, dout,
                           scale_la=0.5, scale_sm=1.5)
    assert np.all(gl["dk"][~lin] == 0) and np.all(gl["dv"][~lin] == 0)
    assert np.all(gl["dbeta"][~lin] == 0)
    assert np.abs(gl["dk"][lin]).min() > 0


# ------------------------------------------------------------------ block mode (Section 4.1)
def _block_route(B, L, H, R, p, seed):
    r = np.random.default_rng(seed)
    return np.repeat((r.random((B, L // R, H)) < p).astype(np.uint8), R, axis=1)


def test_block_mode_fig1c_visibility_pattern():
    """Fig. 1(c) with its D cells: the query's own chunk is read by both operations, the cells
    of earlier chunks by exactly one."""
    rows = [ln.strip() for ln in open(os.path.join(GOLDEN, "fig1c_visibility.txt"))
            if ln.strip() and not ln.startswith("#")]
    fig = np.array([list(r) for r in rows])
    C = 2
    route = np.zeros(12, np.uint8)
    route[[0, 1, 6, 7]] = 1
    x = rand_inputs(1, 12, 1, 4, seed=15)
    x["route"] = route[None, :, None].copy()
    x["beta"] = np.full_like(x["beta"], 0.7)

    def influence(field):
        base = fwd(x, block=C)[field][0, :, 0]
        vis = np.zeros((12, 12), bool)
        for j in range(12):
            y = {n: a.copy() for n, a in x.items()}
            y["v"][0, j, 0] += 1e-3
            vis[:, j] = np.abs(fwd(y, block=C)[field][0, :, 0] - base).max(-1) > 0
        return vis

    sm, la = influence("o_nla"), influence("o_la")
    chunk = np.arange(12) // C
    earlier = chunk[:, None] > chunk[None, :]
    own = (chunk[:, None] == chunk[None, :]) & np.tril(np.ones((12, 12), bool))
    assert np.array_equal(own, fig == "D")
    assert np.array_equal(sm & ~earlier, own) and np.array_equal(la & ~earlier, own)
    assert np.array_equal(sm & earlier, fig == "S")
    for i in range(12):
        cols = np.nonzero(la[i] & earlier[i])[0]
        gcol = np.nonzero(fig[i] == "G")[0]
        if len(gcol) == 0:
            assert len(cols) == 0
        else:
            assert cols.max() == gcol[0] and np.all(route[cols] == 0)
    # earlier chunks: every token in exactly one branch
    assert np.array_equal((sm | la) & earlier, earlier) and not np.any(sm & la & earlier)


def test_block_mode_all_softmax_is_causal_attention_and_blockwise_gdn():
    B, L, H, d, R = 2, 48, 2, 8, 8
    x = rand_inputs(B, L, H, d, seed=31)
    x["route"] = np.ones((B, L, H), np.uint8)
    S0 = RNG.standard_normal((B, H, d, d))
    r = fwd(x, block=R, state_in=S0)
    # softmax branch: plain causal attention (library routine)
    tq, tk, tv = (torch.from_numpy(x[n]).permute(0, 2, 1, 3) for n in ("q", "k", "v"))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=1.5)
    np.testing.assert_allclose(r["o_nla"], ref.permute(0, 2, 1, 3).numpy(), rtol=1e-10, atol=1e-12)
    # the state only decays
    G = x["g"].sum(1)                                          # [B,H]
    np.testing.assert_allclose(r["state_out"], np.exp(G)[..., None, None] * S0, rtol=1e-12)
    # linear branch: every block is a pure GDN run over the block alone, entered with the
    # decayed initial state (the token-level oracle with route 0 on that block)
    for c in range(L // R):
        sl = slice(c * R, (c + 1) * R)
        S_c = np.exp(x["g"][:, :c * R].sum(1))[..., None, None] * S0
        y = {n: x[n][:, sl] for n in ("q", "k", "v", "g", "beta", "w")}
        y["route"] = np.zeros((B, R, H), np.uint8)
        blk = fwd(y, state_in=S_c)
        np.testing.assert_allclose(r["o_la"][:, sl], blk["o_la"], rtol=1e-10, atol=1e-13)


def test_block_mode_all_linear_is_gdn_and_block_local_attention():
    B, L, H, d, R = 1, 40, 2, 8, 8
    x = rand_inputs(B, L, H, d, seed=32)
    x["route"] = np.zeros((B, L, H), np.uint8)
    r = fwd(x, block=R)
    tok = fwd(x)                                               # token level, all linear: pure GDN
    np.testing.assert_allclose(r["o_la"], tok["o_la"], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(r["state_out"], tok["state_out"], rtol=1e-12, atol=1e-15)
    for c in range(L // R):
        sl = slice(c * R, (c + 1) * R)
        tq, tk, tv = (torch.from_numpy(x[n][:, sl]).permute(0, 2, 1, 3) for n in ("q", "k", "v"))
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=1.5)
        np.testing.assert_allclose(r["o_nla"][:, sl], ref.permute(0, 2, 1, 3).numpy(), rtol=1e-10,
                                   atol=1e-12)


def test_block_mode_brute_force_mixed_routes():
    """Mixed routes, tiny: the softmax branch from its dense mask (retained earlier blocks plus
    the causal part of the own block), the linear branch from the paper's matrix form of the GDN
    update restarted at each block from the committed state."""
    B, L, H, d, R = 1, 24, 1, 6, 4
    x = rand_inputs(B, L, H, d, seed=33)
    x["route"] = _block_route(B, L, H, R, 0.4, seed=5)
    assert 0 < x["route"].sum() < L
    S0 = RNG.standard_normal((B, H, d, d))
    r = fwd(x, block=R, state_in=S0, want_cache=True)
    q, k, v = (x[n][0, :, 0] for n in ("q", "k", "v"))
    g, beta, route = (x[n][0, :, 0] for n in ("g", "beta", "route"))
    blk = np.arange(L) // R
    i, j = np.meshgrid(np.arange(L), np.arange(L), indexing="ij")
    mask = (j <= i) & ((route[j] == 1) | (blk[j] == blk[i]))
    logits = np.where(mask, 1.5 * q @ k.T, -np.inf)
    p = np.exp(logits - logits.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    np.testing.assert_allclose(r["o_nla"][0, :, 0], p @ v, rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(r["lse"][0, 0], np.log(np.exp(logits).sum(1)), rtol=1e-10)
    # linear branch, in the paper's orientation (its state is the transpose of ours):
    # S_t = S_{t-1} alpha_t (I - beta_t k_t k_t^T) + beta_t v_t k_t^T,  o_t = S_t q_t
    Sp = S0[0, 0].T.copy()
    o_la = np.zeros((L, d))
    eye = np.eye(d)
    for c in range(L // R):
        S_run = Sp.copy()
        for t in range(c * R, (c + 1) * R):
            S_run = S_run @ (np.exp(g[t]) * (eye - beta[t] * np.outer(k[t], k[t]))) \
                + beta[t] * np.outer(v[t], k[t])
            o_la[t] = 0.5 * S_run @ q[t]
        Sp = S_run if route[c * R] == 0 else np.exp(g[c * R:(c + 1) * R].sum()) * Sp
    np.testing.assert_allclose(r["o_la"][0, :, 0], o_la, rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(r["state_out"][0, 0], Sp.T, rtol=1e-10, atol=1e-13)
    # the retained set after the last block: the tokens of the softmax blocks, in order
    keep = np.nonzero(route)[0]
    assert r["n_sm"][0, 0] == len(keep)
    assert np.array_equal(r["k_sm"][0, 0, :len(keep)], k[keep])
    # combination: same Norm equation as the token-level mode
    def norm(o):
        return o / np.sqrt((o * o).mean(-1, keepdims=True) + 1e-5)
    w = x["w"][0, :, 0]
    np.testing.assert_allclose(r["out"][0, :, 0], w[:, :1] * norm(p @ v) + w[:, 1:] * norm(o_la),
                               rtol=1e-10, atol=1e-13)


def test_block_mode_rejects_route_that_changes_inside_a_block():
    x = rand_inputs(1, 16, 1, 4, seed=34)
    x["route"] = np.zeros((1, 16, 1), np.uint8)
    x["route"][0, 5, 0] = 1
    with pytest.raises(ValueError):
        fwd(x, block=4)


def test_block_mode_generation_protocol_equals_the_forward():
    """Decoding token by token with the decision open (route 2) and rolling back at each block's
    end gives what the block-mode forward gives: outputs, final state, kept K/V."""
    B, L, H, d, R = 2, 20, 2, 6, 4
    x = rand_inputs(B, L, H, d, seed=35)
    x["route"] = _block_route(B, L, H, R, 0.5, seed=6)
    S0 = RNG.standard_normal((B, H, d, d))
    ref = fwd(x, block=R, state_in=S0, want_cache=True)
    state, start = S0.copy(), S0.copy()
    kc, vc = np.zeros((B, H, L, d)), np.zeros((B, H, L, d))
    n = np.zeros((B, H), np.int32)
    undecided = np.full((B, H), 2, np.uint8)
    for t in range(L):
        r = oracle.decode_step(x["q"][:, t], x["k"][:, t], x["v"][:, t], x["g"][:, t], x["beta"][:, t],
                               undecided, x["w"][:, t], state, kc, vc, n, scale_la=0.5, scale_sm=1.5)
        np.testing.assert_allclose(r["out"], ref["out"][:, t], rtol=1e-11, atol=1e-14)
        if (t + 1) % R == 0:
            blk = slice(t + 1 - R, t + 1)
            oracle.block_end(x["route"][:, t], x["g"][:, blk].sum(1), state, start, n, R)
            assert np.array_equal(state, start)
    np.testing.assert_allclose(state, ref["state_out"], rtol=1e-11, atol=1e-14)
    assert np.array_equal(n, ref["n_sm"])
    # a linear block leaves its entries behind the length; the next block overwrites them
    for b in range(B):
        for h in range(H):
            assert np.array_equal(kc[b, h, :n[b, h]], ref["k_sm"][b, h, :n[b, h]])
            assert np.array_equal(vc[b, h, :n[b, h]], ref["v_sm"][b, h, :n[b, h]])


# ------------------------------------------------------------------ score layer (Section 4.1)
def test_score_layer_closed_forms_and_brute_force():
    from oracle import router
    r = np.random.default_rng(41)
    B, L, Dm, H, C = 2, 24, 10, 3, 4
    x = r.standard_normal((B, L, Dm))
    w = r.standard_normal((H, 2, Dm))
    res = router.score_layer(x, w, C)
    # brute force, loop by loop
    for b in range(B):
        for c in range(L // C):
            for h in range(H):
                for o in range(2):
                    s = 0.0
                    for dd in range(Dm):
                        m = sum(x[b, c * C + i, dd] for i in range(C)) / C
                        s += w[h, o, dd] * m
                    assert abs(res["scores"][b, c, h, o] - s) < 1e-12
                sm = np.exp(res["scores"][b, c, h]) / np.exp(res["scores"][b, c, h]).sum()
                assert np.all(res["route"][b, c * C:(c + 1) * C, h] == np.argmax(sm))
    # a chunk of identical tokens: the mean is the token, the score is W x
    xc = np.repeat(r.standard_normal((1, 3, Dm)), C, axis=1)
    rc = router.score_layer(xc, w, C)
    np.testing.assert_allclose(rc["scores"][0], np.einsum("cd,hod->cho", xc[0, ::C], w), rtol=1e-12)
    # one-hot rows pick out the mean of one feature; equal rows tie, and the tie goes to linear
    w1 = np.zeros((1, 2, Dm))
    w1[0, :, 7] = 1.0
    r1 = router.score_layer(x, w1, C)
    np.testing.assert_allclose(r1["scores"][..., 0, 1], x[..., 7].reshape(B, L // C, C).mean(-1), rtol=1e-12)
    assert not r1["route"].any()
    # scaling the softmax row up flips every chunk whose pooled feature is positive
    w1[0, 1, 7] = 2.0
    r2 = router.score_layer(x, w1, C)
    assert np.array_equal(r2["route"][:, ::C, 0] == 1, x[..., 7].reshape(B, L // C, C).mean(-1) > 0)


def test_block_mode_backward_finite_differences():
    B, L, H, d, R = 1, 20, 2, 5, 4
    x = rand_inputs(B, L, H, d, seed=36, unit=False)
    x["q"] *= 0.5
    x["k"] *= 0.4
    x["route"] = _block_route(B, L, H, R, 0.5, seed=7)
    assert 0 < x["route"].sum() < x["route"].size
    dout = RNG.standard_normal((B, L, H, d))
    S0 = RNG.standard_normal((B, H, d, d)) * 0.3
    dS = RNG.standard_normal((B, H, d, d))

    def loss():
        r = fwd(x, state_in=S0, block=R)
        return (r["out"] * dout).sum() + (r["state_out"] * dS).sum()

    gr = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], dout,
                           scale_la=0.5, scale_sm=1.5, state_in=S0, dstate_out=dS, block=R)
    h = 1e-6
    pick = np.random.default_rng(9)
    arrays = [(x[n], gr[gn], n) for n, gn in [("q", "dq"), ("k", "dk"), ("v", "dv"), ("g", "dg"),
                                              ("beta", "dbeta"), ("w", "dw")]]
    arrays.append((S0, gr["dstate_in"], "state_in"))
    for arr, grad, name in arrays:
        flat = arr.reshape(-1)
        for idx in pick.choice(flat.size, size=min(40, flat.size), replace=False):
            old = flat[idx]
            flat[idx] = old + h
            lp = loss()
            flat[idx] = old - h
            lm = loss()
            flat[idx] = old
            fd, an = (lp - lm) / (2 * h), grad.reshape(-1)[idx]
            assert abs(fd - an) <= 2e-6 * max(1.0, abs(an)) + 1e-7, (name, idx, fd, an)


def test_block_mode_backward_special_cases():
    B, L, H, d, R = 1, 24, 2, 6, 8
    x = rand_inputs(B, L, H, d, seed=37)
    dout = RNG.standard_normal((B, L, H, d))
    kw = dict(scale_la=0.5, scale_sm=1.5)
    args = lambda y: (y["q"], y["k"], y["v"], y["g"], y["beta"], y["route"], y["w"], dout)
    # all blocks linear, only the linear branch weighted: the token-level backward of pure GDN
    x["route"] = np.zeros((B, L, H), np.uint8)
    x["w"] = np.stack([np.zeros_like(x["g"]), np.ones_like(x["g"])], -1)
    gb = oracle.hybrid_bwd(*args(x), block=R, **kw)
    gt = oracle.hybrid_bwd(*args(x), **kw)
    for n in ("dq", "dk", "dv", "dg", "dbeta"):
        np.testing.assert_allclose(gb[n], gt[n], rtol=1e-10, atol=1e-13, err_msg=n)
    # all blocks softmax, only the softmax branch weighted: the token-level backward of causal
    # attention (every token retained); nothing reaches g or beta
    x["route"] = np.ones((B, L, H), np.uint8)
    x["w"] = np.stack([np.ones_like(x["g"]), np.zeros_like(x["g"])], -1)
    gb = oracle.hybrid_bwd(*args(x), block=R, **kw)
    gt = oracle.hybrid_bwd(*args(x), **kw)
    for n in ("dq", "dk", "dv"):
        np.testing.assert_allclose(gb[n], gt[n], rtol=1e-10, atol=1e-13, err_msg=n)
    assert np.all(gb["dg"] == 0) and np.all(gb["dbeta"] == 0)


def test_block_mode_score_gradients_against_a_relaxed_mask_forward():
    """d score per block (Section 4.2): finite differences of a forward in which the masks are
    real numbers -- mu_t multiplies e^A of the keys of softmax block t for every query, m_t scales
    the update a linear block commits to the state."""
    B, L, H, d, R = 1, 16, 1, 4, 4
    x = rand_inputs(B, L, H, d, seed=38)
    x["route"] = np.repeat(np.array([1, 0, 1, 0], np.uint8), R)[None, :, None]
    dout = RNG.standard_normal((B, L, H, d))
    q, k, v = (x[n][0, :, 0] for n in ("q", "k", "v"))
    g, beta, route, w = (x[n][0, :, 0] for n in ("g", "beta", "route", "w"))
    blk = np.arange(L) // R
    NB = L // R

    def loss(mu, m):
        i, j = np.meshgrid(np.arange(L), np.arange(L), indexing="ij")
        vis = (j <= i) & ((route[j] == 1) | (blk[j] == blk[i]))
        weight = np.where(route[j] == 1, mu[blk[j]], 1.0)              # mask value of the key's block
        e = np.where(vis, weight * np.exp(1.5 * q @ k.T), 0.0)
        o_nla = (e / e.sum(1, keepdims=True)) @ v
        S = np.zeros((d, d))                                          # ours: o = q S
        o_la = np.zeros((L, d))
        for c in range(NB):
            run = S.copy()
            for t in range(c * R, (c + 1) * R):
                run = np.exp(g[t]) * run
                run = run + beta[t] * np.outer(k[t], v[t] - k[t] @ run)
                o_la[t] = 0.5 * q[t] @ run
            decayed = np.exp(g[c * R:(c + 1) * R].sum()) * S
            S = decayed + (m[c] if route[c * R] == 0 else 0.0) * (run - decayed)
        norm = lambda o: o / np.sqrt((o * o).mean(-1, keepdims=True) + 1e-5)
        out = w[:, :1] * norm(o_nla) + w[:, 1:] * norm(o_la)
        return (out * dout[0, :, 0]).sum()

    ones = np.ones(NB)
    np.testing.assert_allclose(loss(ones, ones), (fwd(x, block=R)["out"] * dout).sum(), rtol=1e-10)
    gr = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], dout,
                           scale_la=0.5, scale_sm=1.5, block=R)["dscore"][0, :, 0]
    h = 1e-6
    for c in range(NB):
        for op in (0, 1):
            e = np.zeros(NB)
            e[c] = h
            fd = ((loss(ones, ones + e) - loss(ones, ones - e)) if op == 0
                  else (loss(ones + e, ones) - loss(ones - e, ones))) / (2 * h)
            active = (route[c * R] == 1) == (op == 1)
            if active:
                assert abs(fd - gr[c, op]) <= 1e-6 * max(1.0, abs(fd)), (c, op, fd, gr[c, op])
                assert abs(fd) > 1e-6 or c == NB - 1       # (the last linear block feeds nothing)
            else:
                assert gr[c, op] == 0.0                    # not computed for the inactive operation
