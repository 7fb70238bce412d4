"""GPU parity of the forward with grouped softmax heads and in-kernel q/k normalisation
(Section 4.3: several softmax heads under one linear head's mask; L2-normalised q, k for the linear
operation, RMS-normalised for the softmax operation) against `oracle/grouped.py`, element by element
on the same seeded inputs:

* fp32 storage (CUDA-core kernels): d = 64 and 128, G = 1, 2, 4, with and without normalisation;
* bf16 storage (tensor-core kernels): d = 128 with G = 2 -- six linear heads with twelve softmax heads,
  the appendix's smaller model -- and G = 1 with normalisation, on shapes that take the one-pass scan,
  and the segmented scan;
* the backward for fp32 storage and for bf16 storage at d = 128, including the Jacobians of the two
  normalisations;
* generation: natsl_decode_step (and the block end) with grouped heads and the normalisation;
* requests that are not built come back as NATSL_ERR_UNSUPPORTED, before any launch.
"""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import grouped
from paper_2602_03681_b200 import inputs
from test_gpu_parity import TOL, check_stored, dev, rel_err, tdtype

pytestmark = pytest.mark.gpu


def make_inputs(wl, B, H, L, unnormalised, block_p=None, spread=0.7):
    route = None if block_p is None else inputs.route_blocks(wl.seed, (B, L, H), block_p)
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L, route=route)
    if unnormalised:      # rows of very different lengths (log-normal, sigma = spread): the normalisation has something to do
        r = np.random.default_rng(wl.seed + 100)
        for n in ("q", "k"):
            x[n] = (x[n] * np.exp(spread * r.standard_normal((B, L, H, 1)))).astype(np.float32)
            if wl.dtype == "bf16":
                x[n] = inputs.round_bf16(x[n])
    return x


def run_both(wl, x, G, norm, scale_sm, norm_eps=1e-6, flags=0, block=False):
    from paper_2602_03681_b200 import binding
    dt = tdtype(wl)
    f = flags | (binding.QK_NORM if norm else 0) | (binding.BLOCK_ROUTING if block else 0)
    res = binding.hybrid_fwd(dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt), dev(x["g"]), dev(x["beta"]),
                             dev(x["route"]), dev(x["w"]), scale_la=wl.scale_la, scale_sm=scale_sm,
                             want=("o_la", "o_nla", "lse", "state_out"), flags=f, G=G, norm_eps=norm_eps)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(res["ws"]) == 0
    got = {n: t.float().cpu().numpy() for n, t in res.items() if n != "ws"}
    ref = grouped.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], G=max(G, 1),
                             qk_norm=norm, scale_la=wl.scale_la, scale_sm=scale_sm, norm_eps=norm_eps,
                             block=64 if block else None)
    return got, ref


def check(wl, got, ref, tol, G):
    B, L, H, d = ref["out"].shape
    lse_g = got["lse"].reshape(B, H, max(G, 1), L)
    fin = np.isfinite(ref["lse"])
    assert np.array_equal(np.isneginf(lse_g), ~fin)
    assert np.abs(lse_g[fin] - ref["lse"][fin]).max() <= max(tol, 1e-3) * 2
    for n in ("o_la", "o_nla", "state_out"):
        e = rel_err(got[n], ref[n])
        assert e <= tol, (n, e)
    # every softmax head on its own: a head that is off must not hide behind the others' RMS
    ds = d // max(G, 1)
    for s in range(max(G, 1)):
        cols = slice(s * ds, (s + 1) * ds)
        e = rel_err(got["o_nla"][..., cols], ref["o_nla"][..., cols])
        assert e <= tol, ("o_nla slice", s, e)
    check_stored(got["out"], ref["out"], tol, wl.dtype)


@pytest.mark.parametrize("d,G,norm,B,H,L", [
    (64, 2, True, 1, 3, 256),
    (64, 2, False, 2, 2, 192),
    (128, 4, True, 1, 2, 192),
    (128, 2, True, 1, 3, 256),
    (128, 2, False, 1, 2, 128),
    (64, 1, True, 1, 2, 256),
])
def test_fp32_storage(d, G, norm, B, H, L):
    wl = dataclasses.replace(inputs.WORKLOADS["cfg0_f32_tiny_fwd"], d=d, seed=31 + d + G)
    x = make_inputs(wl, B, H, L, norm)
    scale_sm = (d / G) ** -0.5 if norm else wl.scale_sm
    got, ref = run_both(wl, x, G, norm, scale_sm)
    check(wl, got, ref, TOL["f32"], G)


@pytest.mark.parametrize("G,norm,B,H,L,flags", [
    (2, True, 1, 6, 1024, 0),        # six linear heads x two softmax heads; segmented scan (few heads)
    (2, False, 1, 6, 512, 0),
    (2, True, 8, 6, 512, 0),         # 48 (batch, head) pairs: one-pass scan
    (2, True, 2, 3, 320, 16),        # stages in sequence on the caller's stream; ragged last query tile
    (1, True, 2, 4, 384, 0),         # normalisation alone
    (2, True, 1, 2, 192, 2),         # one-pass scan with few heads
])
def test_bf16_tensor_cores(G, norm, B, H, L, flags):
    wl = dataclasses.replace(inputs.WORKLOADS["cfg1_bf16_prefill"], seed=41 + G + B)
    x = make_inputs(wl, B, H, L, norm)
    scale_sm = (wl.d / G) ** -0.5 if norm else wl.scale_sm
    got, ref = run_both(wl, x, G, norm, scale_sm, flags=flags)
    check(wl, got, ref, TOL["bf16"], G)


@pytest.mark.parametrize("storage,d,G,norm,B,H,L,p", [
    ("f32", 64, 2, True, 1, 2, 256, 0.4),
    ("f32", 128, 2, False, 1, 2, 192, 0.5),
    ("bf16", 128, 2, True, 1, 6, 512, 0.3),      # the paper's mode: one decision per block, grouped heads, normalised q, k
    ("bf16", 128, 2, True, 2, 3, 320, 0.6),      # ragged last query tile
    ("bf16", 128, 2, False, 1, 3, 384, 0.4),
    ("bf16", 128, 1, True, 1, 2, 256, 0.0),      # all blocks linear: every tile is an own-block tile
    ("bf16", 64, 1, True, 2, 2, 256, 0.4),
])
def test_block_level_routing_with_grouped_heads(storage, d, G, norm, B, H, L, p):
    """Block-level routing (Section 4.1) together with grouped heads and the normalisation: the own-block
    tile of a linear block reads the layer's own keys, which the kernel normalises in shared memory."""
    base = "cfg0_f32_tiny_fwd" if storage == "f32" else ("cfg1_bf16_prefill" if d == 128 else "cfg4_bf16_train")
    wl = dataclasses.replace(inputs.WORKLOADS[base], d=d, seed=71 + d + G)
    x = make_inputs(wl, B, H, L, norm, block_p=p)
    if p == 0.0:
        x["route"][:] = 0
    scale_sm = (d / G) ** -0.5 if norm else wl.scale_sm
    got, ref = run_both(wl, x, G, norm, scale_sm, block=True)
    check(wl, got, ref, TOL[storage], G)


def test_bf16_paper_mode_at_length():
    """Six linear x twelve softmax heads, one decision per block, normalised q, k, L = 2048: 16 query tiles per
    head with up to ~10 retained tiles and two own-block tiles each, several waves of CTAs."""
    wl = dataclasses.replace(inputs.WORKLOADS["cfg1_bf16_prefill"], seed=77)
    x = make_inputs(wl, 1, 6, 2048, True, block_p=0.3)
    got, ref = run_both(wl, x, 2, True, 64 ** -0.5, block=True)
    check(wl, got, ref, TOL["bf16"], 2)


def test_paper_mode_forward_repeated_calls_complete_and_agree():
    """Many back-to-back calls on shapes whose second query tile has two own-block tiles in most heads (the
    case in which the MMA thread waits for two rounds of in-kernel key normalisation): every call ends
    without a device-side time-out and returns the same bits.  With a short bound on the waits, so that a
    missed hand-over shows as a status, not as a two-second stall."""
    from paper_2602_03681_b200 import binding
    wl = dataclasses.replace(inputs.WORKLOADS["cfg1_bf16_prefill"], seed=83)
    B, H, L, G = 8, 6, 512, 2
    x = make_inputs(wl, B, H, L, True, block_p=0.15)
    dt = tdtype(wl)
    args = [dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt), dev(x["g"]), dev(x["beta"]), dev(x["route"]), dev(x["w"])]
    f = binding.QK_NORM | binding.BLOCK_ROUTING
    binding.natsl_debug_set_wait_limit(100000)           # ~0.05 s
    try:
        first, ws = None, None
        for it in range(60):
            res = binding.hybrid_fwd(*args, scale_la=wl.scale_la, scale_sm=64 ** -0.5, flags=f, G=G, norm_eps=1e-6, ws=ws)
            ws = res["ws"]
            if it % 10 == 9 or it == 0:
                torch.cuda.synchronize()
                assert binding.natsl_device_status(ws) == 0, it
                out = res["out"].clone()
                if first is None:
                    first = out
                assert torch.equal(out, first), it
    finally:
        binding.natsl_debug_set_wait_limit(0)


def test_bf16_tensor_cores_d64_normalisation():
    """The normalisation alone at d = 64 (one softmax head per linear head, the 64-column kernels)."""
    wl = dataclasses.replace(inputs.WORKLOADS["cfg4_bf16_train"], seed=47)
    x = make_inputs(wl, 2, 3, 448, True)
    got, ref = run_both(wl, x, 1, True, wl.d ** -0.5)
    check(wl, got, ref, TOL["bf16"], 1)


@pytest.mark.parametrize("d,G,norm,B,H,L,states", [
    (64, 2, True, 1, 3, 256, False),
    (128, 4, True, 1, 2, 192, True),
    (128, 2, False, 2, 2, 128, False),
    (64, 1, True, 1, 2, 192, True),
    (128, 2, True, 1, 2, 256, False),
])
def test_fp32_storage_backward(d, G, norm, B, H, L, states):
    """Backward with grouped heads and the normalisation's Jacobians (fp32 storage) against the gradients
    of the oracle's definition, with and without a carried state and its gradient."""
    from paper_2602_03681_b200 import binding
    from test_gpu_parity import check_bwd
    wl = dataclasses.replace(inputs.WORKLOADS["cfg0_f32_tiny_fwd"], d=d, seed=51 + d + G)
    x = make_inputs(wl, B, H, L, norm)
    scale_sm = (d / G) ** -0.5 if norm else wl.scale_sm
    r = np.random.default_rng(6)
    s0 = (0.1 * r.standard_normal((B, H, d, d))).astype(np.float32) if states else None
    dso = (0.05 * r.standard_normal((B, H, d, d))).astype(np.float32) if states else None
    p = binding.make_params(B, H, L, d, binding.NATSL_F32, wl.scale_la, scale_sm, w=dev(x["w"]),
                            flags=binding.QK_NORM if norm else 0, G=G, norm_eps=1e-6)
    keep = [dev(a) for a in (s0, dso) if a is not None]
    dstate_in = torch.empty((B, H, d, d), device="cuda")
    if states:
        p.state_in, p.dstate_out, p.dstate_in = keep[0].data_ptr(), keep[1].data_ptr(), dstate_in.data_ptr()
    w_dev = dev(x["w"])
    p.w = w_dev.data_ptr()
    ws = binding.alloc_workspace(p, binding.OP_BWD)
    t = {n: dev(x[n]) for n in ("q", "k", "v", "g", "beta", "route", "dout")}
    outs = {n: torch.empty_like(t["q"]) for n in ("dq", "dk", "dv")}
    outs.update(dg=torch.empty_like(t["g"]), dbeta=torch.empty_like(t["g"]),
                dw=torch.empty((B, L, H, 2), device="cuda"))
    binding.natsl_hybrid_bwd(t["q"], t["k"], t["v"], t["g"], t["beta"], t["route"], t["dout"], outs["dq"], outs["dk"],
                             outs["dv"], outs["dg"], outs["dbeta"], outs["dw"], p, ws)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(ws) == 0
    got = {n: v.cpu().numpy() for n, v in outs.items()}
    ref = grouped.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"], G=G,
                             qk_norm=norm, scale_la=wl.scale_la, scale_sm=scale_sm, norm_eps=1e-6,
                             state_in=s0, dstate_out=dso)
    check_bwd(wl, got, ref, TOL["f32"])
    if states:
        assert rel_err(dstate_in.cpu().numpy(), ref["dstate_in"]) <= TOL["f32"]
    if norm:      # Euler: a normalised layer's gradient is orthogonal to every q and k row
        for n in ("q", "k"):
            dot = np.abs((got["d" + n].astype(np.float64) * x[n]).sum(-1))
            scale = np.sqrt((got["d" + n].astype(np.float64) ** 2).sum(-1) * (x[n].astype(np.float64) ** 2).sum(-1))
            assert (dot <= 1e-3 * scale + 1e-9).all()


@pytest.mark.parametrize("G,norm,B,H,L", [
    (2, True, 1, 6, 256),        # six linear heads x two softmax heads
    (2, False, 2, 2, 320),
    (1, True, 1, 3, 192),
    (2, True, 2, 3, 384),
])
def test_bf16_tensor_cores_backward(G, norm, B, H, L):
    """Backward at d = 128 on tensor cores (softmax branch's kernels on column slices, reverse scan on the
    L2-normalised copies, chunk-level products as tile GEMMs, Jacobians of the normalisations last)."""
    from test_gpu_parity import check_bwd
    from paper_2602_03681_b200 import binding
    wl = dataclasses.replace(inputs.WORKLOADS["cfg1_bf16_prefill"], seed=61 + G + B)
    x = make_inputs(wl, B, H, L, norm)
    scale_sm = (wl.d / G) ** -0.5 if norm else wl.scale_sm
    dt = torch.bfloat16
    p = binding.make_params(B, H, L, wl.d, binding.NATSL_BF16, wl.scale_la, scale_sm,
                            flags=binding.QK_NORM if norm else 0, G=G, norm_eps=1e-6)
    w_dev = dev(x["w"])
    p.w = w_dev.data_ptr()
    ws = binding.alloc_workspace(p, binding.OP_BWD)
    t = {n: dev(x[n], dt) for n in ("q", "k", "v", "dout")}
    t.update({n: dev(x[n]) for n in ("g", "beta", "route")})
    outs = {n: torch.empty_like(t["q"]) for n in ("dq", "dk", "dv")}
    outs.update(dg=torch.empty_like(t["g"]), dbeta=torch.empty_like(t["g"]),
                dw=torch.empty((B, L, H, 2), device="cuda"))
    binding.natsl_hybrid_bwd(t["q"], t["k"], t["v"], t["g"], t["beta"], t["route"], t["dout"], outs["dq"], outs["dk"],
                             outs["dv"], outs["dg"], outs["dbeta"], outs["dw"], p, ws)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(ws) == 0
    got = {n: v.float().cpu().numpy() for n, v in outs.items()}
    ref = grouped.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"], G=G,
                             qk_norm=norm, scale_la=wl.scale_la, scale_sm=scale_sm, norm_eps=1e-6)
    # (with the normalisation the q, k rows differ in length by up to 16 x, and so do their gradient rows)
    check_bwd(wl, got, ref, TOL["bf16"], large_only=not norm)


@pytest.mark.parametrize("storage,d,G,norm,B,H,L,p", [
    ("f32", 64, 2, True, 1, 2, 256, 0.4),
    ("f32", 128, 2, False, 1, 2, 192, 0.5),
    ("f32", 128, 4, True, 1, 1, 128, 0.0),
    ("bf16", 128, 2, True, 1, 6, 256, 0.3),      # the paper's mode, trainable: blocks, grouped heads, normalised q, k
    ("bf16", 128, 2, False, 2, 2, 320, 0.5),
    ("bf16", 128, 1, True, 1, 2, 256, 0.4),
])
def test_block_level_routing_backward_with_grouped_heads(storage, d, G, norm, B, H, L, p):
    """Backward under block-level routing with grouped heads and the normalisation (every token's k
    reaches both operations there, through two different normalisations)."""
    from test_gpu_parity import check_bwd
    from paper_2602_03681_b200 import binding
    base = "cfg0_f32_tiny_fwd" if storage == "f32" else "cfg1_bf16_prefill"
    wl = dataclasses.replace(inputs.WORKLOADS[base], d=d, seed=81 + d + G)
    x = make_inputs(wl, B, H, L, norm, block_p=p)
    if p == 0.0:
        x["route"][:] = 0
    scale_sm = (d / G) ** -0.5 if norm else wl.scale_sm
    dt = tdtype(wl)
    pr = binding.make_params(B, H, L, d, binding.NATSL_F32 if storage == "f32" else binding.NATSL_BF16,
                             wl.scale_la, scale_sm, G=G, norm_eps=1e-6,
                             flags=binding.BLOCK_ROUTING | (binding.QK_NORM if norm else 0))
    w_dev = dev(x["w"])
    pr.w = w_dev.data_ptr()
    dscore = torch.zeros((B, L // 64, H, 2), device="cuda")
    pr.dscore = dscore.data_ptr()
    ws = binding.alloc_workspace(pr, binding.OP_BWD)
    t = {n: dev(x[n], dt) for n in ("q", "k", "v", "dout")}
    t.update({n: dev(x[n]) for n in ("g", "beta", "route")})
    outs = {n: torch.empty_like(t["q"]) for n in ("dq", "dk", "dv")}
    outs.update(dg=torch.empty_like(t["g"]), dbeta=torch.empty_like(t["g"]),
                dw=torch.empty((B, L, H, 2), device="cuda"))
    binding.natsl_hybrid_bwd(t["q"], t["k"], t["v"], t["g"], t["beta"], t["route"], t["dout"], outs["dq"], outs["dk"],
                             outs["dv"], outs["dg"], outs["dbeta"], outs["dw"], pr, ws)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(ws) == 0
    got = {n: v.float().cpu().numpy() for n, v in outs.items()}
    ref = grouped.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"], G=G,
                             qk_norm=norm, scale_la=wl.scale_la, scale_sm=scale_sm, norm_eps=1e-6, block=64,
                             want_dscore=True)
    check_bwd(wl, got, ref, TOL[storage], large_only=not norm)
    # score gradients (Section 4.2): the group's softmax heads share the block's mask
    gd = dscore.cpu().numpy()
    blocks = x["route"][:, ::64]
    assert np.all(gd[..., 0][blocks == 1] == 0) and np.all(gd[..., 1][blocks == 0] == 0)
    for op in (0, 1):
        if np.abs(ref["dscore"][..., op]).max() > 0:
            assert rel_err(gd[..., op], ref["dscore"][..., op]) <= TOL[storage], (op, rel_err(gd[..., op], ref["dscore"][..., op]))


def test_paper_mode_backward_on_one_stream_gives_the_same_bits():
    """Grouped heads, normalised q and k, one decision per block: the backward with every kernel on the caller's
    stream (NATSL_SINGLE_STREAM) and the default one, whose linear branch runs on a second stream beside the
    softmax branch, agree bit for bit (they would not if the two branches shared a buffer)."""
    from paper_2602_03681_b200 import binding
    d, G, B, H, L = 128, 2, 2, 3, 512
    wl = dataclasses.replace(inputs.WORKLOADS["cfg1_bf16_prefill"], seed=97)
    x = make_inputs(wl, B, H, L, True, block_p=0.3)
    dt = tdtype(wl)
    t = {n: dev(x[n], dt) for n in ("q", "k", "v", "dout")}
    t.update({n: dev(x[n]) for n in ("g", "beta", "route")})
    w_dev = dev(x["w"])
    results = []
    for extra in (0, binding.SINGLE_STREAM):
        pr = binding.make_params(B, H, L, d, binding.NATSL_BF16, wl.scale_la, (d / G) ** -0.5, w=w_dev, G=G,
                                 norm_eps=1e-6, flags=binding.BLOCK_ROUTING | binding.QK_NORM | extra)
        dscore = torch.zeros((B, L // 64, H, 2), device="cuda")
        pr.dscore = dscore.data_ptr()
        ws = binding.alloc_workspace(pr, binding.OP_BWD)
        outs = {n: torch.empty_like(t["q"]) for n in ("dq", "dk", "dv")}
        outs.update(dg=torch.empty_like(t["g"]), dbeta=torch.empty_like(t["g"]),
                    dw=torch.empty((B, L, H, 2), device="cuda"), dscore=dscore)
        binding.natsl_hybrid_bwd(t["q"], t["k"], t["v"], t["g"], t["beta"], t["route"], t["dout"], outs["dq"],
                                 outs["dk"], outs["dv"], outs["dg"], outs["dbeta"], outs["dw"], pr, ws)
        torch.cuda.synchronize()
        assert binding.natsl_device_status(ws) == 0
        results.append(outs)
    for n in results[0]:
        assert torch.equal(results[0][n], results[1][n]), n


@pytest.mark.parametrize("storage,block", [("bf16", False), ("bf16", True), ("f32", False)])
def test_saved_forward_then_backward_with_grouped_heads(storage, block):
    """The training step as two calls (NATSL_SAVE_FOR_BWD, then NATSL_SAVED_FWD) with grouped heads and the
    normalisation: same `out` as the plain forward's oracle, same gradients as the oracle's."""
    from test_gpu_parity import check_bwd
    from paper_2602_03681_b200 import binding
    d, G, B, H, L = 128, 2, 1, 3, 256
    base = "cfg0_f32_tiny_fwd" if storage == "f32" else "cfg1_bf16_prefill"
    wl = dataclasses.replace(inputs.WORKLOADS[base], d=d, seed=91)
    x = make_inputs(wl, B, H, L, True, block_p=0.4 if block else None)
    scale_sm = (d / G) ** -0.5
    dt = tdtype(wl)
    flags = binding.QK_NORM | (binding.BLOCK_ROUTING if block else 0)
    code = binding.NATSL_F32 if storage == "f32" else binding.NATSL_BF16
    w_dev = dev(x["w"])
    pr = binding.make_params(B, H, L, d, code, wl.scale_la, scale_sm, w=w_dev, G=G, norm_eps=1e-6,
                             flags=flags | binding.SAVE_FOR_BWD)
    ws = binding.alloc_workspace(pr, binding.OP_BWD)
    t = {n: dev(x[n], dt) for n in ("q", "k", "v", "dout")}
    t.update({n: dev(x[n]) for n in ("g", "beta", "route")})
    out = torch.empty_like(t["q"])
    binding.natsl_hybrid_fwd(t["q"], t["k"], t["v"], t["g"], t["beta"], t["route"], out, pr, ws)
    pb = binding.make_params(B, H, L, d, code, wl.scale_la, scale_sm, w=w_dev, G=G, norm_eps=1e-6,
                             flags=flags | binding.SAVED_FWD)
    outs = {n: torch.empty_like(t["q"]) for n in ("dq", "dk", "dv")}
    outs.update(dg=torch.empty_like(t["g"]), dbeta=torch.empty_like(t["g"]),
                dw=torch.empty((B, L, H, 2), device="cuda"))
    binding.natsl_hybrid_bwd(t["q"], t["k"], t["v"], t["g"], t["beta"], t["route"], t["dout"], outs["dq"], outs["dk"],
                             outs["dv"], outs["dg"], outs["dbeta"], outs["dw"], pb, ws)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(ws) == 0
    kw = dict(G=G, qk_norm=True, scale_la=wl.scale_la, scale_sm=scale_sm, norm_eps=1e-6, block=64 if block else None)
    ref_f = grouped.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], **kw)
    check_stored(out.float().cpu().numpy(), ref_f["out"], TOL[storage], wl.dtype)
    ref_b = grouped.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"], **kw)
    check_bwd(wl, {n: v.float().cpu().numpy() for n, v in outs.items()}, ref_b, TOL[storage], large_only=False)


@pytest.mark.parametrize("storage,d,G,norm,block,B,H,L", [
    ("bf16", 128, 2, True, True, 2, 3, 192),       # the paper's mode in generation: decision open, roll-back per block
    ("bf16", 128, 2, True, False, 2, 2, 160),
    ("bf16", 128, 2, False, False, 1, 2, 96),
    ("bf16", 64, 1, True, False, 2, 2, 96),
    ("f32", 128, 4, True, True, 1, 2, 128),
    ("f32", 64, 2, True, False, 2, 1, 96),
])
def test_generation_with_grouped_heads(storage, d, G, norm, block, B, H, L):
    """natsl_decode_step with grouped heads and the normalisation, from an empty state and cache: step t
    equals row t of the forward over the whole sequence (oracle/grouped.py); the cache keeps the keys as given."""
    from paper_2602_03681_b200 import binding
    base = "cfg0_f32_tiny_fwd" if storage == "f32" else ("cfg1_bf16_prefill" if d == 128 else "cfg4_bf16_train")
    wl = dataclasses.replace(inputs.WORKLOADS[base], d=d, seed=101 + d + G)
    x = make_inputs(wl, B, H, L, norm, block_p=0.4 if block else None)
    scale_sm = (d / G) ** -0.5 if norm else wl.scale_sm
    ref = grouped.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], G=G, qk_norm=norm,
                             scale_la=wl.scale_la, scale_sm=scale_sm, norm_eps=1e-6, block=64 if block else None)
    dt = tdtype(wl)
    code = binding.NATSL_F32 if storage == "f32" else binding.NATSL_BF16
    p = binding.make_params(B, H, 0, d, code, wl.scale_la, scale_sm, flags=binding.QK_NORM if norm else 0, G=G,
                            norm_eps=1e-6)
    ws = binding.alloc_workspace(p, binding.OP_DECODE)
    state = torch.zeros((B, H, d, d), device="cuda")
    start = state.clone()
    kc = torch.zeros((B, H, L, d), dtype=dt, device="cuda")
    vc = torch.zeros_like(kc)
    n = torch.zeros((B, H), dtype=torch.int32, device="cuda")
    undecided = torch.full((B, H), 2, dtype=torch.uint8, device="cuda")
    for t in range(L):
        w = dev(x["w"][:, t])
        p.w = w.data_ptr()
        out = torch.empty((B, H, d), dtype=dt, device="cuda")
        binding.natsl_decode_step(dev(x["q"][:, t], dt), dev(x["k"][:, t], dt), dev(x["v"][:, t], dt),
                                  dev(x["g"][:, t]), dev(x["beta"][:, t]),
                                  undecided if block else dev(x["route"][:, t]), state, kc, vc, n, out, p, ws)
        check_stored(out.float().cpu().numpy(), ref["out"][:, t], TOL[storage], wl.dtype, f"step{t}")
        if block and (t + 1) % 64 == 0:
            g_block = x["g"][:, t - 63:t + 1].astype(np.float64).sum(1).astype(np.float32)
            binding.natsl_decode_block_end(dev(x["route"][:, t]), dev(g_block), state, start, n, 64, p, ws)
    assert binding.natsl_device_status(ws) == 0
    assert rel_err(state.cpu().numpy(), ref["state_out"]) <= max(TOL[storage], 1e-3) * (1 if storage == "f32" else 1)
    kept = x["route"].sum(1).T if not block else x["route"][:, ::64].sum(1).T * 64      # [H,B] -> compare as [B,H]
    assert np.array_equal(n.cpu().numpy(), kept.T.astype(np.int32))
    b0, h0 = 0, H - 1                       # the cache rows are the retained tokens' keys as given
    rows = np.nonzero(x["route"][b0, :, h0])[0]
    assert np.array_equal(kc[b0, h0, :len(rows)].float().cpu().numpy(), x["k"][b0, rows, h0])


@pytest.mark.parametrize("storage,d,G,block,B,H,L0,L", [
    ("bf16", 128, 2, True, 2, 3, 256, 384),
    ("bf16", 128, 2, False, 1, 2, 192, 256),
    ("f32", 64, 2, True, 1, 2, 128, 192),
])
def test_prefill_then_generation_with_grouped_heads(storage, d, G, block, B, H, L0, L):
    """Prefill L0 tokens with the normalisation on, hand state and cache to natsl_decode_step, generate up to
    L: every generated step equals its row of the forward over the whole sequence.  The cache the prefill
    returns holds the keys as given; the prefill's own softmax kernel read a normalised copy."""
    from paper_2602_03681_b200 import binding
    base = "cfg0_f32_tiny_fwd" if storage == "f32" else "cfg1_bf16_prefill"
    wl = dataclasses.replace(inputs.WORKLOADS[base], d=d, seed=111 + d + G)
    x = make_inputs(wl, B, H, L, True, block_p=0.4 if block else None)
    scale_sm = (d / G) ** -0.5
    ref = grouped.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], G=G, qk_norm=True,
                             scale_la=wl.scale_la, scale_sm=scale_sm, norm_eps=1e-6, block=64 if block else None)
    dt = tdtype(wl)
    flags = binding.QK_NORM | (binding.BLOCK_ROUTING if block else 0)
    pre = binding.hybrid_fwd(*(dev(x[n][:, :L0], dt) for n in ("q", "k", "v")), dev(x["g"][:, :L0]),
                             dev(x["beta"][:, :L0]), dev(x["route"][:, :L0]), dev(x["w"][:, :L0]),
                             scale_la=wl.scale_la, scale_sm=scale_sm, want=("state_out", "cache"), sm_cap=L,
                             flags=flags, G=G, norm_eps=1e-6)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(pre["ws"]) == 0
    check_stored(pre["out"].float().cpu().numpy(), ref["out"][:, :L0], TOL[storage], wl.dtype, "prefill")
    state, kc, vc, n = pre["state_out"], pre["k_sm"], pre["v_sm"], pre["sm_len"]
    rows = np.nonzero(x["route"][0, :L0, 0])[0]
    assert np.array_equal(kc[0, 0, :len(rows)].float().cpu().numpy(), x["k"][0, rows, 0])      # as given
    code = binding.NATSL_F32 if storage == "f32" else binding.NATSL_BF16
    p = binding.make_params(B, H, 0, d, code, wl.scale_la, scale_sm, flags=binding.QK_NORM, G=G, norm_eps=1e-6)
    ws = binding.alloc_workspace(p, binding.OP_DECODE)
    start = state.clone()
    undecided = torch.full((B, H), 2, dtype=torch.uint8, device="cuda")
    for t in range(L0, L):
        w = dev(x["w"][:, t])
        p.w = w.data_ptr()
        out = torch.empty((B, H, d), dtype=dt, device="cuda")
        binding.natsl_decode_step(dev(x["q"][:, t], dt), dev(x["k"][:, t], dt), dev(x["v"][:, t], dt),
                                  dev(x["g"][:, t]), dev(x["beta"][:, t]),
                                  undecided if block else dev(x["route"][:, t]), state, kc, vc, n, out, p, ws)
        check_stored(out.float().cpu().numpy(), ref["out"][:, t], TOL[storage], wl.dtype, f"step{t}")
        if block and (t + 1) % 64 == 0:
            g_block = x["g"][:, t - 63:t + 1].astype(np.float64).sum(1).astype(np.float32)
            binding.natsl_decode_block_end(dev(x["route"][:, t]), dev(g_block), state, start, n, 64, p, ws)
    assert binding.natsl_device_status(ws) == 0
    assert rel_err(state.cpu().numpy(), ref["state_out"]) <= max(TOL[storage], 1e-3)


@pytest.mark.parametrize("G,norm,block,B,H,pieces", [
    (2, True, True, 1, 3, (256, 128, 320)),
    (2, True, False, 2, 2, (192, 320)),
    (2, False, False, 1, 2, (128, 256)),
    (1, True, False, 1, 2, (320, 192)),
])
def test_prefill_in_pieces_with_grouped_heads(G, norm, block, B, H, pieces):
    """NATSL_APPEND_CACHE with grouped heads and the normalisation: the pieces' outputs equal the forward over
    the whole sequence; the cache holds the keys as given, and a later piece reads normalised copies of the
    earlier pieces' keys made from it."""
    from paper_2602_03681_b200 import binding
    wl = dataclasses.replace(inputs.WORKLOADS["cfg1_bf16_prefill"], seed=121 + G)
    d, L = wl.d, sum(pieces)
    x = make_inputs(wl, B, H, L, norm, block_p=0.35 if block else None)
    scale_sm = (d / G) ** -0.5 if norm else wl.scale_sm
    ref = grouped.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], G=G, qk_norm=norm,
                             scale_la=wl.scale_la, scale_sm=scale_sm, norm_eps=1e-6, block=64 if block else None)
    dt = torch.bfloat16
    flags = binding.APPEND_CACHE | (binding.QK_NORM if norm else 0) | (binding.BLOCK_ROUTING if block else 0)
    k_sm = torch.zeros((B, H, L, d), dtype=dt, device="cuda")
    v_sm = torch.zeros_like(k_sm)
    sm_len = torch.zeros((B, H), dtype=torch.int32, device="cuda")
    state, outs, t0 = None, [], 0
    for n in pieces:
        sl = slice(t0, t0 + n)
        res = binding.hybrid_fwd(*(dev(x[m][:, sl], dt) for m in ("q", "k", "v")), dev(x["g"][:, sl]),
                                 dev(x["beta"][:, sl]), dev(x["route"][:, sl]), dev(x["w"][:, sl]),
                                 scale_la=wl.scale_la, scale_sm=scale_sm, state_in=state, want=("state_out",),
                                 cache=(k_sm, v_sm, sm_len), flags=flags, G=G, norm_eps=1e-6)
        torch.cuda.synchronize()
        assert binding.natsl_device_status(res["ws"]) == 0
        state = res["state_out"]
        outs.append(res["out"].float().cpu().numpy())
        t0 += n
    check_stored(np.concatenate(outs, 1), ref["out"], TOL["bf16"], "bf16")
    assert rel_err(state.cpu().numpy(), ref["state_out"]) <= TOL["bf16"]
    rows = np.nonzero(x["route"][0, :, 0])[0]
    assert sm_len[0, 0].item() == len(rows)
    assert np.array_equal(k_sm[0, 0, :len(rows)].float().cpu().numpy(), x["k"][0, rows, 0])


@pytest.mark.parametrize("block", [False, True])
def test_bf16_d64_normalised_backward(block):
    """bf16 storage at d = 64 with the normalisation: the backward takes the path with separate chunk-level
    products (the fused chunk kernel does not know the normalisation)."""
    from test_gpu_parity import check_bwd
    from paper_2602_03681_b200 import binding
    wl = dataclasses.replace(inputs.WORKLOADS["cfg4_bf16_train"], seed=131)
    B, H, L, d = 2, 2, 256, 64
    # (row lengths over a factor of ~5: a gradient row scales with 1 / its row's length, and the bound is
    # relative to the whole tensor's RMS; with sigma = 0.7 the shortest rows of this case sit 2 % above it)
    x = make_inputs(wl, B, H, L, True, block_p=0.4 if block else None, spread=0.4)
    scale_sm = d ** -0.5
    flags = binding.QK_NORM | (binding.BLOCK_ROUTING if block else 0)
    pr = binding.make_params(B, H, L, d, binding.NATSL_BF16, wl.scale_la, scale_sm, flags=flags, norm_eps=1e-6)
    w_dev = dev(x["w"])
    pr.w = w_dev.data_ptr()
    ws = binding.alloc_workspace(pr, binding.OP_BWD)
    t = {n: dev(x[n], torch.bfloat16) for n in ("q", "k", "v", "dout")}
    t.update({n: dev(x[n]) for n in ("g", "beta", "route")})
    outs = {n: torch.empty_like(t["q"]) for n in ("dq", "dk", "dv")}
    outs.update(dg=torch.empty_like(t["g"]), dbeta=torch.empty_like(t["g"]), dw=torch.empty((B, L, H, 2), device="cuda"))
    binding.natsl_hybrid_bwd(t["q"], t["k"], t["v"], t["g"], t["beta"], t["route"], t["dout"], outs["dq"], outs["dk"],
                             outs["dv"], outs["dg"], outs["dbeta"], outs["dw"], pr, ws)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(ws) == 0
    ref = grouped.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"], G=1,
                             qk_norm=True, scale_la=wl.scale_la, scale_sm=scale_sm, norm_eps=1e-6,
                             block=64 if block else None)
    check_bwd(wl, {n: v.float().cpu().numpy() for n, v in outs.items()}, ref, TOL["bf16"], large_only=False)


def test_normalisation_ignores_row_lengths_on_the_device():
    """Rescaling the q and k rows by powers of two changes no bf16 mantissa, so with norm_eps = 0 the
    normalised layer must return almost the same bits."""
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    x = make_inputs(wl, 1, 4, 256, False)
    r = np.random.default_rng(3)
    y = dict(x)
    y["q"] = x["q"] * 2.0 ** r.integers(-6, 7, size=(1, 256, 4, 1))
    y["k"] = x["k"] * 2.0 ** r.integers(-6, 7, size=(1, 256, 4, 1))
    outs = []
    for z in (x, y):
        res = binding.hybrid_fwd(*(dev(z[n], torch.bfloat16) for n in ("q", "k", "v")), dev(z["g"]), dev(z["beta"]),
                                 dev(z["route"]), dev(z["w"]), scale_la=wl.scale_la, scale_sm=0.125,
                                 flags=binding.QK_NORM, G=2, norm_eps=0.0)
        torch.cuda.synchronize()
        assert binding.natsl_device_status(res["ws"]) == 0
        outs.append(res["out"].float().cpu().numpy())
    assert np.abs(outs[0] - outs[1]).max() <= 2e-2 * np.sqrt((outs[0] ** 2).mean())
    assert np.abs(outs[0]).max() > 0.1


def test_requests_that_are_not_built_are_refused():
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    x = make_inputs(wl, 1, 2, 128, False)
    args = [dev(x[n], torch.bfloat16) for n in ("q", "k", "v")] + [dev(x["g"]), dev(x["beta"]), dev(x["route"]),
                                                                  dev(x["w"])]
    kw = dict(scale_la=wl.scale_la, scale_sm=wl.scale_sm)

    def refused(call):
        with pytest.raises(binding.NatslError) as e:
            call()
        return e.value.status == binding.ERR_UNSUPPORTED

    assert refused(lambda: binding.hybrid_fwd(*args, G=4, **kw))                                  # d/G = 32 on tensor cores
    assert refused(lambda: binding.hybrid_fwd(*args, G=2, flags=binding.FORCE_SIMT, **kw))        # bf16 on CUDA cores
    with pytest.raises(binding.NatslError):                                                       # G must divide d
        binding.hybrid_fwd(*args, G=3, **kw)
    # backward: two softmax heads of 32 columns (d = 64) are not built on tensor cores
    wl4 = inputs.WORKLOADS["cfg4_bf16_train"]
    x4 = make_inputs(wl4, 1, 2, 128, False)
    a4 = [dev(x4[n], torch.bfloat16) for n in ("q", "k", "v")] + [dev(x4["g"]), dev(x4["beta"]), dev(x4["route"])]
    p = binding.make_params(1, 2, 128, 64, binding.NATSL_BF16, wl4.scale_la, wl4.scale_sm, G=2)
    n = binding.natsl_workspace_size(p, binding.OP_BWD)
    ws = torch.zeros(n, dtype=torch.uint8, device="cuda")
    outs = [torch.empty_like(a4[0]) for _ in range(3)] + [torch.empty_like(a4[3]) for _ in range(2)]
    dw = torch.empty((1, 128, 2, 2), device="cuda")
    with pytest.raises(binding.NatslError) as e:
        binding.natsl_hybrid_bwd(*a4, a4[0], *outs, dw, p, ws)
    assert e.value.status == binding.ERR_UNSUPPORTED
