"""Pins of the oracle with grouped softmax heads and per-branch q/k normalisation
(`oracle/grouped.py`; Section 4.3, the paragraphs on head grouping and on the L2 / RMS
normalisation of q and k).  CPU only.

What fixes it, other than itself:
* G = 1 without normalisation is the plain layer: forward and gradients equal the C oracle's
  (an independent token-by-token implementation with a hand-derived backward);
* the softmax heads of a group are ordinary attention heads over column slices: o_nla equals the C
  oracle run on the slices as separate heads with the route repeated, and the library's masked attention;
* RMS-norm(q) . RMS-norm(k) = d (q^ . k^) for L2-normalised q^, k^: with G = 1 and norm_eps = 0 the
  normalised layer equals the plain layer on pre-normalised inputs with scale_sm d;
* a normalised layer does not see the lengths of the q and k rows: rescaling them changes nothing,
  and the gradient of every row is orthogonal to the row (Euler's relation, degree 0);
* an explicit loop over heads, queries and keys on a tiny case; central finite differences.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import grouped
from test_oracle_pins import rand_inputs

KW = dict(scale_la=0.5, scale_sm=1.5, eps=1e-5)


def gf(x, **kw):
    a = dict(KW)
    a.update(kw)
    return grouped.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], **a)


def gb(x, dout, **kw):
    a = dict(KW)
    a.update(kw)
    return grouped.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], dout, **a)


def test_one_head_per_group_is_the_plain_layer():
    x = rand_inputs(2, 96, 3, 16, p=0.3, seed=21)
    r = np.random.default_rng(5)
    s0 = 0.1 * r.standard_normal((2, 3, 16, 16))
    a = gf(x, G=1, state_in=s0)
    b = oracle.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], state_in=s0, **KW)
    for n in ("out", "o_la", "o_nla", "state_out"):
        np.testing.assert_allclose(a[n], b[n], rtol=1e-9, atol=1e-11, err_msg=n)
    np.testing.assert_allclose(a["lse"][:, :, 0], b["lse"], rtol=1e-10, atol=1e-12)
    dout = r.standard_normal(x["q"].shape)
    ds = 0.05 * r.standard_normal(s0.shape)
    ga = gb(x, dout, G=1, state_in=s0, dstate_out=ds)
    gbb = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], dout,
                            state_in=s0, dstate_out=ds, **KW)
    for n in ("dq", "dk", "dv", "dg", "dbeta", "dw", "dstate_in"):
        np.testing.assert_allclose(ga[n], gbb[n], rtol=1e-8, atol=1e-10, err_msg=n)


@pytest.mark.parametrize("G", [2, 3, 4])
def test_group_heads_are_attention_heads_over_column_slices(G):
    B, L, H, d = 2, 80, 3, 24
    x = rand_inputs(B, L, H, d, p=0.3, seed=22, unit=False)
    x["route"][:, 0] = 1
    a = gf(x, G=G, scale_sm=0.4)
    # (1) the C oracle on the slices as H*G separate heads, route repeated: its o_nla and lse
    sl = {n: x[n].reshape(B, L, H * G, d // G) for n in ("q", "k", "v")}
    rep = {n: np.repeat(x[n], G, axis=2) for n in ("g", "beta", "route")}
    b = oracle.hybrid_fwd(sl["q"], sl["k"], sl["v"], rep["g"], rep["beta"], rep["route"], None,
                          scale_la=0.5, scale_sm=0.4)
    np.testing.assert_allclose(a["o_nla"], b["o_nla"].reshape(B, L, H, d), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(a["lse"].reshape(B, H * G, L), b["lse"], rtol=1e-10, atol=1e-12)
    # (2) the library's masked attention on the same slices
    tq, tk, tv = (torch.from_numpy(sl[n]).permute(0, 2, 1, 3) for n in ("q", "k", "v"))
    keep = torch.from_numpy(rep["route"].astype(bool)).permute(0, 2, 1)[:, :, None, :]
    mask = torch.tril(torch.ones(L, L, dtype=torch.bool))[None, None] & keep
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask, scale=0.4)
    np.testing.assert_allclose(a["o_nla"], ref.permute(0, 2, 1, 3).reshape(B, L, H, d).numpy(),
                               rtol=1e-10, atol=1e-12)
    # (3) the linear operation does not know about the groups
    c = gf(x, G=1, scale_sm=0.4)
    np.testing.assert_array_equal(a["o_la"], c["o_la"])
    np.testing.assert_array_equal(a["state_out"], c["state_out"])
    # (4) the output: each softmax head's slice normalised on its own, the linear row as a whole
    on = a["o_nla"].reshape(B, L, H, G, d // G)
    yn = (on / np.sqrt((on ** 2).mean(-1, keepdims=True) + 1e-5)).reshape(B, L, H, d)
    yl = a["o_la"] / np.sqrt((a["o_la"] ** 2).mean(-1, keepdims=True) + 1e-5)
    np.testing.assert_allclose(a["out"], x["w"][..., :1] * yn + x["w"][..., 1:] * yl, rtol=1e-10, atol=1e-12)


def test_explicit_loops_tiny():
    B, L, H, d, G = 1, 10, 2, 8, 2
    x = rand_inputs(B, L, H, d, p=0.4, seed=23, unit=False)
    ne = 1e-3
    a = gf(x, G=G, qk_norm=True, norm_eps=ne, scale_sm=0.7)
    ds = d // G
    for h in range(H):
        for s in range(G):
            cols = slice(s * ds, (s + 1) * ds)
            for i in range(L):
                qi = x["q"][0, i, h, cols]
                qi = qi / np.sqrt((qi ** 2).mean() + ne)
                num, den = np.zeros(ds), 0.0
                for j in range(i + 1):
                    if not x["route"][0, j, h]:
                        continue
                    kj = x["k"][0, j, h, cols]
                    kj = kj / np.sqrt((kj ** 2).mean() + ne)
                    e = np.exp(0.7 * float(qi @ kj))
                    num += e * x["v"][0, j, h, cols]
                    den += e
                want = num / den if den > 0 else np.zeros(ds)
                np.testing.assert_allclose(a["o_nla"][0, i, h, cols], want, rtol=1e-10, atol=1e-12)
        # linear operation on L2-normalised rows: the plain layer's o_la with the rows normalised outside
    qn = x["q"] / np.sqrt((x["q"] ** 2).sum(-1, keepdims=True) + ne)
    kn = x["k"] / np.sqrt((x["k"] ** 2).sum(-1, keepdims=True) + ne)
    b = oracle.hybrid_fwd(qn, kn, x["v"], x["g"], x["beta"], x["route"], x["w"], scale_la=0.5, scale_sm=0.7)
    np.testing.assert_allclose(a["o_la"], b["o_la"], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(a["state_out"], b["state_out"], rtol=1e-9, atol=1e-11)


def test_rms_times_rms_is_d_times_cosine():
    B, L, H, d = 1, 64, 2, 16
    x = rand_inputs(B, L, H, d, p=0.3, seed=24, unit=False)
    a = gf(x, G=1, qk_norm=True, norm_eps=0.0, scale_sm=0.11)
    qn = x["q"] / np.linalg.norm(x["q"], axis=-1, keepdims=True)
    kn = x["k"] / np.linalg.norm(x["k"], axis=-1, keepdims=True)
    b = oracle.hybrid_fwd(qn, kn, x["v"], x["g"], x["beta"], x["route"], x["w"], scale_la=0.5,
                          scale_sm=0.11 * d)
    for n in ("out", "o_la", "o_nla"):
        np.testing.assert_allclose(a[n], b[n], rtol=1e-9, atol=1e-11, err_msg=n)


def test_normalised_layer_ignores_row_lengths():
    B, L, H, d, G = 1, 48, 2, 16, 2
    x = rand_inputs(B, L, H, d, p=0.3, seed=25, unit=False)
    r = np.random.default_rng(7)
    a = gf(x, G=G, qk_norm=True, norm_eps=0.0)
    y = dict(x)
    y["q"] = x["q"] * np.exp(r.standard_normal((B, L, H, 1)))
    y["k"] = x["k"] * np.exp(r.standard_normal((B, L, H, 1)))
    b = gf(y, G=G, qk_norm=True, norm_eps=0.0)
    np.testing.assert_allclose(a["out"], b["out"], rtol=1e-9, atol=1e-11)
    dout = r.standard_normal(x["q"].shape)
    gr = gb(x, dout, G=G, qk_norm=True, norm_eps=0.0)
    for n in ("q", "k"):
        dot = (gr["d" + n] * x[n]).sum(-1)
        assert np.abs(dot).max() <= 1e-9 * np.abs(gr["d" + n]).max() * np.abs(x[n]).max() * d
    # without the normalisation the lengths do matter (the test would notice a flag that does nothing)
    c, e = gf(x, G=G), gf(y, G=G)
    assert np.abs(c["out"] - e["out"]).max() > 1e-3


def test_backward_finite_differences():
    B, L, H, d, G = 1, 12, 2, 8, 2
    x = rand_inputs(B, L, H, d, p=0.35, seed=26, unit=False)
    r = np.random.default_rng(9)
    dout = r.standard_normal(x["q"].shape)
    s0 = 0.1 * r.standard_normal((B, H, d, d))
    dso = 0.1 * r.standard_normal((B, H, d, d))
    kw = dict(G=G, qk_norm=True, norm_eps=1e-4, state_in=s0)
    gr = gb(x, dout, dstate_out=dso, **kw)

    def loss(z):
        o = gf(z, **kw)
        return float((o["out"] * dout).sum() + (o["state_out"] * dso).sum())

    h = 1e-6
    for n, gname in (("q", "dq"), ("k", "dk"), ("v", "dv"), ("g", "dg"), ("beta", "dbeta"), ("w", "dw")):
        for _ in range(6):
            idx = tuple(int(r.integers(0, m)) for m in x[n].shape)
            zp, zm = dict(x), dict(x)
            zp[n] = x[n].copy(); zp[n][idx] += h
            zm[n] = x[n].copy(); zm[n][idx] -= h
            fd = (loss(zp) - loss(zm)) / (2 * h)
            assert abs(fd - gr[gname][idx]) <= 1e-5 * max(1.0, abs(fd)), (n, idx, fd, gr[gname][idx])


def block_route(B, L, H, R, p, seed):
    r = np.random.default_rng(seed)
    return np.repeat((r.random((B, L // R, H)) < p).astype(np.uint8), R, axis=1)


def test_block_mode_with_one_head_per_group_is_the_c_oracles_block_mode():
    B, L, H, d, R = 2, 96, 2, 16, 16
    x = rand_inputs(B, L, H, d, seed=28)
    x["route"] = block_route(B, L, H, R, 0.4, 1)
    r = np.random.default_rng(3)
    s0 = 0.1 * r.standard_normal((B, H, d, d))
    a = gf(x, G=1, state_in=s0, block=R)
    b = oracle.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], state_in=s0, block=R, **KW)
    for n in ("out", "o_la", "o_nla", "state_out"):
        np.testing.assert_allclose(a[n], b[n], rtol=1e-9, atol=1e-11, err_msg=n)
    dout = r.standard_normal(x["q"].shape)
    ds = 0.05 * r.standard_normal(s0.shape)
    ga = gb(x, dout, G=1, state_in=s0, dstate_out=ds, block=R)
    gc = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], dout, state_in=s0,
                           dstate_out=ds, block=R, **KW)
    for n in ("dq", "dk", "dv", "dg", "dbeta", "dw", "dstate_in"):
        np.testing.assert_allclose(ga[n], gc[n], rtol=1e-8, atol=1e-10, err_msg=n)
    # and it is not the token-level layer
    assert np.abs(a["out"] - gf(x, G=1, state_in=s0)["out"]).max() > 1e-3


def test_block_mode_group_heads_are_block_mode_heads_over_column_slices():
    B, L, H, d, R, G = 1, 64, 2, 16, 16, 2
    x = rand_inputs(B, L, H, d, seed=29, unit=False)
    x["route"] = block_route(B, L, H, R, 0.5, 2)
    a = gf(x, G=G, scale_sm=0.4, block=R)
    sl = {n: x[n].reshape(B, L, H * G, d // G) for n in ("q", "k", "v")}
    rep = {n: np.repeat(x[n], G, axis=2) for n in ("g", "beta", "route")}
    b = oracle.hybrid_fwd(sl["q"], sl["k"], sl["v"], rep["g"], rep["beta"], rep["route"], None, scale_la=0.5,
                          scale_sm=0.4, block=R)
    np.testing.assert_allclose(a["o_nla"], b["o_nla"].reshape(B, L, H, d), rtol=1e-10, atol=1e-12)
    c = oracle.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], scale_la=0.5,
                          scale_sm=0.4, block=R)
    np.testing.assert_allclose(a["o_la"], c["o_la"], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(a["state_out"], c["state_out"], rtol=1e-9, atol=1e-11)
    with pytest.raises(ValueError):
        y = dict(x)
        y["route"] = x["route"].copy()
        y["route"][0, 3, 0] ^= 1
        gf(y, G=G, block=R)


def test_block_mode_score_gradients_equal_the_c_oracles_and_add_over_the_group():
    B, L, H, d, R = 1, 96, 2, 16, 16
    x = rand_inputs(B, L, H, d, seed=30)
    x["route"] = block_route(B, L, H, R, 0.5, 4)
    r = np.random.default_rng(5)
    dout = r.standard_normal(x["q"].shape)
    a = gb(x, dout, G=1, block=R, want_dscore=True)
    c = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], dout, block=R, **KW)
    np.testing.assert_allclose(a["dscore"], c["dscore"], rtol=1e-8, atol=1e-10)
    assert np.abs(c["dscore"][..., 0]).max() > 0 and np.abs(c["dscore"][..., 1]).max() > 0
    for n in ("dq", "dk", "dg"):                           # the masks leave the other gradients alone
        np.testing.assert_allclose(a[n], c[n], rtol=1e-8, atol=1e-10, err_msg=n)
    # grouped heads share their linear head's mask: its gradient is the sum over the group's heads, i.e. what
    # the C oracle gives for the column slices run as separate heads, added up (softmax operation; weights 1, 0
    # keep the linear operation out of it)
    G = 2
    w1 = np.zeros((B, L, H, 2)); w1[..., 0] = 1.0
    y = dict(x); y["w"] = w1
    ag = gb(y, dout, G=G, block=R, want_dscore=True, scale_sm=0.4)
    sl = {n: x[n].reshape(B, L, H * G, d // G) for n in ("q", "k", "v")}
    rep = {n: np.repeat(x[n], G, axis=2) for n in ("g", "beta", "route")}
    cg = oracle.hybrid_bwd(sl["q"], sl["k"], sl["v"], rep["g"], rep["beta"], rep["route"], np.repeat(w1, G, axis=2),
                           dout.reshape(B, L, H * G, d // G), block=R, scale_la=0.5, scale_sm=0.4)
    np.testing.assert_allclose(ag["dscore"][..., 1], cg["dscore"][..., 1].reshape(B, L // R, H, G).sum(-1),
                               rtol=1e-8, atol=1e-10)


def test_rejects_group_count_that_does_not_divide():
    x = rand_inputs(1, 8, 1, 8, seed=27)
    with pytest.raises(ValueError):
        gf(x, G=3)
