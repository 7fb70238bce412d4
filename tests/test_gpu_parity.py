"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle on the same seeded
inputs.  Indices bit-exact; floating outputs max|gpu - oracle| <= tol * RMS(oracle) with
tol = 1e-4 for fp32 storage and 2e-2 for bf16 storage."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_03681_b200 import inputs

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(dtype) if dtype is not None else t


def tdtype(wl):
    return torch.bfloat16 if wl.dtype == "bf16" else torch.float32


def rel_err(got, ref):
    ref = np.asarray(ref, np.float64)
    got = np.asarray(got, np.float64)
    rms = np.sqrt((ref ** 2).mean())
    return np.abs(got - ref).max() / max(rms, 1e-30)


def run_fwd(wl, x, want=("o_la", "o_nla", "lse", "state_out"), state_in=None, flags=0, w="given"):
    from paper_2602_03681_b200 import binding
    dt = tdtype(wl)
    res = binding.hybrid_fwd(dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt), dev(x["g"]),
                             dev(x["beta"]), dev(x["route"]),
                             dev(x["w"]) if w == "given" else None,
                             scale_la=wl.scale_la, scale_sm=wl.scale_sm,
                             state_in=None if state_in is None else dev(state_in), want=want,
                             flags=flags)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(res["ws"]) == 0
    return {n: t.float().cpu().numpy() for n, t in res.items() if n != "ws"}


def run_oracle(wl, x, state_in=None, w="given", **kw):
    return oracle.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"],
                             x["w"] if w == "given" else None, scale_la=wl.scale_la,
                             scale_sm=wl.scale_sm, state_in=state_in, **kw)


def half_ulp_bf16(x):
    """Exact half unit-in-the-last-place of bf16 (8 significant bits) at |x|."""
    x = np.abs(np.asarray(x, np.float64))
    e = np.floor(np.log2(np.maximum(x, 2.0 ** -126)))
    return 2.0 ** (e - 8)


def check_stored(got, ref, tol, storage, name="out", large_only=True):
    """A tensor stored in the workload's storage type: the computed value must be within
    tol * RMS of the oracle; storing it in bf16 adds at most half a bf16 ulp on top, which by
    itself already exceeds 2e-2 * RMS for the few elements with |x| >= 4.  Returns how many
    elements needed that allowance; each of them must be a large one, whose half ulp is at least
    half the plain bound (for the layer output, RMS about 0.77, that means |ref| >= 2).
    large_only=False drops that last requirement, for tensors whose rows differ in scale by an order of
    magnitude (gradients through a normalisation of rows of very different lengths), where "large" measured
    against the whole tensor's RMS says nothing about an element of a small row."""
    ref = np.asarray(ref, np.float64)
    err = np.abs(np.asarray(got, np.float64) - ref)
    plain = tol * np.sqrt((ref ** 2).mean())
    bound = plain + half_ulp_bf16(ref) if storage == "bf16" else plain
    worst = (err / bound).max()
    assert worst <= 1.0, (name, worst, rel_err(got, ref))
    needed = err > plain
    if storage == "bf16" and tol >= 1e-2 and large_only:     # (a caller with a tighter tolerance lives on the allowance)
        assert np.all(half_ulp_bf16(ref[needed]) >= 0.5 * plain), (name, "allowance used by a small element")
    return int(needed.sum())


def check_fwd(wl, got, ref, tol):
    lse_ok = np.isfinite(ref["lse"])
    assert np.array_equal(np.isneginf(got["lse"]), ~lse_ok)
    if lse_ok.any():
        assert np.abs(got["lse"][lse_ok] - ref["lse"][lse_ok]).max() <= max(tol, 1e-3) * 2
    for name in ("o_la", "o_nla", "state_out"):       # fp32 tensors: no storage rounding
        if name in got:
            e = rel_err(got[name], ref[name])
            assert e <= tol, (name, e)
    check_stored(got["out"], ref["out"], tol, wl.dtype)


# ------------------------------------------------------------------ compaction (bit-exact)
@pytest.mark.parametrize("B,L,H,p", [(1, 256, 2, 0.25), (2, 1024, 3, 0.1), (1, 64, 1, 0.0),
                                     (1, 128, 2, 1.0), (1, 4096 * 20, 1, 0.05)])
def test_route_compact_bit_exact(B, L, H, p):
    from paper_2602_03681_b200 import binding
    rng = np.random.default_rng(L + H)
    route = (rng.random((B, L, H)) < p).astype(np.uint8)
    if L == 128:
        route[0, 77, 0] = 0            # almost-all-softmax with one hole
    ref = oracle.route_compact(route, 64)
    NC = L // 64
    sm_idx = torch.full((B, H, L), -1, dtype=torch.int32, device="cuda")
    pre = torch.zeros((B, H, NC + 1), dtype=torch.int32, device="cuda")
    lin = torch.zeros((B, H, NC, 64), dtype=torch.int32, device="cuda")
    nl = torch.zeros((B, H, NC), dtype=torch.int32, device="cuda")
    prm = binding.make_params(B, H, L, 64, binding.NATSL_F32, 1.0, 1.0)
    binding.natsl_route_compact(dev(route), sm_idx, pre, lin, nl, prm)
    torch.cuda.synchronize()
    assert np.array_equal(sm_idx.cpu().numpy(), ref["sm_idx"])
    assert np.array_equal(pre.cpu().numpy(), ref["sm_chunk_prefix"])
    assert np.array_equal(lin.cpu().numpy(), ref["lin_idx"])
    assert np.array_equal(nl.cpu().numpy(), ref["n_lin"])


# ------------------------------------------------------------------ forward
def test_fwd_cfg0_fp32():
    wl = inputs.WORKLOADS["cfg0_f32_tiny_fwd"]
    x = inputs.make_layer_inputs(wl)
    check_fwd(wl, run_fwd(wl, x), run_oracle(wl, x), TOL["f32"])


@pytest.mark.parametrize("name,B,H,L", [("cfg0_f32_tiny_fwd", 2, 3, 192),
                                        ("cfg0_f32_tiny_fwd", 1, 1, 64),
                                        ("cfg1_bf16_prefill", 1, 2, 320),
                                        ("cfg4_bf16_train", 2, 2, 256),
                                        ("cfg2_bf16_long_prefill", 1, 2, 1024)])
def test_fwd_small_cases_simt(name, B, H, L):
    """The fp32 CUDA-core path on every storage type / head size, several chunks, state_in."""
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS[name]
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L)
    S0 = (0.1 * np.random.default_rng(3).standard_normal((B, H, wl.d, wl.d))).astype(np.float32)
    got = run_fwd(wl, x, state_in=S0, flags=binding.FORCE_SIMT)
    ref = run_oracle(wl, x, state_in=S0)
    # fp32 math throughout: only the bf16 rounding of `out` is left for bf16 storage
    check_fwd(wl, got, ref, 1e-4)


def test_fwd_degenerate_routes():
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg0_f32_tiny_fwd"]
    for fill in (0, 1):
        x = inputs.make_layer_inputs(wl, route=np.full((1, 256, 2), fill, np.uint8))
        got = run_fwd(wl, x, flags=binding.FORCE_SIMT, w=None)
        ref = run_oracle(wl, x, w=None)
        check_fwd(wl, got, ref, 1e-4)
        if fill == 0:
            assert np.all(got["o_nla"] == 0)


def test_fwd_rejects_bad_arguments():
    from paper_2602_03681_b200 import binding
    q = torch.zeros((1, 100, 1, 64), device="cuda")
    g = torch.zeros((1, 100, 1), device="cuda")
    r = torch.zeros((1, 100, 1), dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.NatslError) as e:
        binding.hybrid_fwd(q, q, q, g, g, r, scale_la=1.0, scale_sm=1.0)
    assert e.value.status == -2
    q = torch.zeros((1, 128, 1, 64), device="cuda")
    g = torch.zeros((1, 128, 1), device="cuda")
    r = torch.zeros((1, 128, 1), dtype=torch.uint8, device="cuda")
    p = binding.make_params(1, 1, 128, 64, 0, 1.0, 1.0)
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.NatslError) as e:
        binding.natsl_hybrid_fwd(q, q, q, g, g, r, torch.empty_like(q), p, small)
    assert e.value.status == -5


# ------------------------------------------------------------------ decode
def run_decode(wl, B, H, steps, n0, cap=None, route=None):
    from paper_2602_03681_b200 import binding
    x = inputs.make_decode_inputs(wl, B=B, H=H, steps=steps, ctx_retained=n0, cap=cap)
    if route is not None:
        x["route"] = np.ascontiguousarray(np.broadcast_to(route, x["route"].shape)).astype(np.uint8)
    dt = tdtype(wl)
    state = dev(x["state"])
    kc, vc = dev(x["k_cache"], dt), dev(x["v_cache"], dt)
    n = dev(x["cache_len"])
    p = binding.make_params(B, H, 0, wl.d, binding._dtype_code(kc), wl.scale_la, wl.scale_sm)
    ws = binding.alloc_workspace(p, binding.OP_DECODE)
    o_state = x["state"].astype(np.float64)
    o_kc, o_vc = x["k_cache"].astype(np.float64), x["v_cache"].astype(np.float64)
    o_n = x["cache_len"].copy()
    tol = TOL[wl.dtype]
    for t in range(steps):
        w = dev(x["w"][t])
        p.w = w.data_ptr()
        out = torch.empty((B, H, wl.d), dtype=dt, device="cuda")
        binding.natsl_decode_step(dev(x["q"][t], dt), dev(x["k"][t], dt), dev(x["v"][t], dt),
                                  dev(x["g"][t]), dev(x["beta"][t]), dev(x["route"][t]), state, kc,
                                  vc, n, out, p, ws)
        ref = oracle.decode_step(x["q"][t], x["k"][t], x["v"][t], x["g"][t], x["beta"][t],
                                 x["route"][t], x["w"][t], o_state, o_kc, o_vc, o_n,
                                 scale_la=wl.scale_la, scale_sm=wl.scale_sm)
        check_stored(out.float().cpu().numpy(), ref["out"], tol, wl.dtype, f"step{t}")
    assert binding.natsl_device_status(ws) == 0
    assert np.array_equal(n.cpu().numpy(), o_n)
    assert rel_err(state.cpu().numpy(), o_state) <= 1e-4
    for b in range(B):
        for h in range(H):
            m = o_n[b, h]
            assert np.array_equal(kc[b, h, :m].float().cpu().numpy(), o_kc[b, h, :m].astype(np.float32))
            assert np.array_equal(vc[b, h, :m].float().cpu().numpy(), o_vc[b, h, :m].astype(np.float32))


@pytest.mark.parametrize("name,B,H,steps,n0", [("cfg3_bf16_decode", 3, 4, 24, 333),
                                               ("cfg3_bf16_decode", 2, 2, 40, 0),
                                               ("cfg4_bf16_train", 2, 3, 16, 77),
                                               ("cfg0_f32_tiny_fwd", 2, 2, 20, 50)])
def test_decode_trajectory(name, B, H, steps, n0):
    run_decode(inputs.WORKLOADS[name], B, H, steps, n0)


@pytest.mark.parametrize("n0", [29, 125, 253])
def test_decode_growing_cache_crosses_tile_boundaries(n0):
    """Every token is appended (route 1) from three entries below a boundary of the kernel's
    32-key tiles: 32 (a second tile appears), 128 (the tiles per cache slice go from one to two)
    and 256; eight steps cross it, each step against the oracle."""
    run_decode(inputs.WORKLOADS["cfg3_bf16_decode"], 2, 2, 8, n0, route=1)


def test_decode_cache_full_is_reported_not_trapped():
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg3_bf16_decode"]
    x = inputs.make_decode_inputs(wl, B=1, H=2, steps=1, ctx_retained=4, cap=4)
    dt = torch.bfloat16
    state = dev(x["state"])
    kc, vc = dev(x["k_cache"], dt), dev(x["v_cache"], dt)
    n = dev(x["cache_len"])
    route = np.array([[1, 0]], np.uint8)
    p = binding.make_params(1, 2, 0, wl.d, binding.NATSL_BF16, wl.scale_la, wl.scale_sm)
    ws = binding.alloc_workspace(p, binding.OP_DECODE)
    out = torch.full((1, 2, wl.d), 7.0, dtype=dt, device="cuda")
    binding.natsl_decode_step(dev(x["q"][0], dt), dev(x["k"][0], dt), dev(x["v"][0], dt),
                              dev(x["g"][0]), dev(x["beta"][0]), dev(route), state, kc, vc, n, out,
                              p, ws)
    assert binding.natsl_device_status(ws) == binding.ERR_CACHE_FULL
    assert binding.natsl_device_status(ws) == 0           # cleared by the read
    assert np.array_equal(state[0, 0].cpu().numpy(), x["state"][0, 0])   # untouched
    assert torch.all(out[0, 0] == 0) and n[0, 0].item() == 4
    assert not np.array_equal(state[0, 1].cpu().numpy(), x["state"][0, 1])  # the other head ran


# ------------------------------------------------------------------ backward
def run_bwd(wl, x, w="given", flags=0):
    from paper_2602_03681_b200 import binding
    dt = tdtype(wl)
    res = binding.hybrid_bwd(dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt), dev(x["g"]),
                             dev(x["beta"]), dev(x["route"]), dev(x["w"]) if w == "given" else None,
                             dev(x["dout"], dt), scale_la=wl.scale_la, scale_sm=wl.scale_sm,
                             flags=flags)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(res["ws"]) == 0
    return {n: t.float().cpu().numpy() for n, t in res.items() if n != "ws"}


def check_bwd(wl, got, ref, tol, large_only=True):
    for name in ("dq", "dk", "dv"):
        check_stored(got[name], ref[name], tol, wl.dtype, name, large_only)
    for name in ("dg", "dbeta", "dw"):
        e = rel_err(got[name], ref[name])
        assert e <= tol, (name, e)


@pytest.mark.parametrize("name,B,H,L", [("cfg0_f32_tiny_fwd", 1, 2, 256),
                                        ("cfg0_f32_tiny_fwd", 2, 1, 64),
                                        ("cfg4_bf16_train", 2, 3, 320),
                                        ("cfg1_bf16_prefill", 1, 2, 192)])
def test_bwd_small_cases(name, B, H, L):
    """The fp32 CUDA-core backward (forced for bf16 storage, whose default runs the softmax branch
    on tensor cores)."""
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS[name]
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L)
    got = run_bwd(wl, x, flags=binding.FORCE_SIMT)
    ref = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"],
                            scale_la=wl.scale_la, scale_sm=wl.scale_sm)
    # fp32 arithmetic throughout; bf16 storage only rounds dq, dk, dv
    check_bwd(wl, got, ref, 1e-4 if wl.dtype == "f32" else 2e-4)
    lin = x["route"] == 0
    assert np.all(got["dbeta"][~lin] == 0)


def test_bwd_degenerate_routes():
    wl = inputs.WORKLOADS["cfg0_f32_tiny_fwd"]
    for fill in (0, 1):
        x = inputs.make_layer_inputs(wl, B=1, H=2, L=128, route=np.full((1, 128, 2), fill, np.uint8))
        got = run_bwd(wl, x, w=None)
        ref = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], None,
                                x["dout"], scale_la=wl.scale_la, scale_sm=wl.scale_sm)
        for name in ("dq", "dk", "dv", "dg", "dbeta"):
            ref_rms = np.sqrt((ref[name] ** 2).mean())
            if ref_rms == 0:
                assert np.all(got[name] == 0), name
            else:
                assert rel_err(got[name], ref[name]) <= 1e-4, name
