"""Parity of the block-routed forward (Section 4.1: one routing decision per block of 64 tokens,
both operations read the query's own block) with the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_03681_b200 import inputs
from test_gpu_parity import check_fwd, check_stored, dev, rel_err, run_fwd, tdtype

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2


def block_inputs(wl, B, H, L, p, seed=0):
    route = inputs.route_blocks(wl.seed + seed, (B, L, H), p)
    return inputs.make_layer_inputs(wl, B=B, H=H, L=L, route=route)


def oracle_block(wl, x, state_in=None, **kw):
    return oracle.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"],
                             scale_la=wl.scale_la, scale_sm=wl.scale_sm, state_in=state_in, block=64,
                             **kw)


@pytest.mark.parametrize("name,B,H,L,p,flags", [
    ("cfg4_bf16_train", 1, 2, 512, 0.3, 0),        # d = 64
    ("cfg1_bf16_prefill", 1, 2, 576, 0.3, 0),      # d = 128, ragged last query tile (9 blocks)
    ("cfg1_bf16_prefill", 2, 3, 1024, 0.15, 0),
    ("cfg1_bf16_prefill", 1, 1, 2048, 0.2, 0),     # few (batch, head) pairs: segmented scan
    ("cfg1_bf16_prefill", 1, 1, 2048, 0.2, 2),     # ... and the same in one pass
    ("cfg4_bf16_train", 1, 2, 64, 0.0, 0),         # a single block
])
def test_block_routed_forward_matches_oracle(name, B, H, L, p, flags):
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS[name]
    x = block_inputs(wl, B, H, L, p)
    rng = np.random.default_rng(7)
    S0 = (0.1 * rng.standard_normal((B, H, wl.d, wl.d))).astype(np.float32)
    ref = oracle_block(wl, x, state_in=S0.astype(np.float64))
    got = run_fwd(wl, x, state_in=S0, flags=binding.BLOCK_ROUTING | flags)
    check_fwd(wl, got, ref, TOL_BF16)
    # the mode is not the token-level one: with the same inputs the two differ visibly
    tok = run_fwd(wl, x, state_in=S0, flags=flags)
    assert rel_err(tok["out"], ref["out"]) > 10 * TOL_BF16 or x["route"].all()


@pytest.mark.parametrize("p", [0.0, 1.0])
def test_block_routing_all_linear_and_all_softmax(p):
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    x = block_inputs(wl, 1, 2, 384, 0.5)
    x["route"][:] = int(p)
    ref = oracle_block(wl, x)
    got = run_fwd(wl, x, flags=binding.BLOCK_ROUTING)
    check_fwd(wl, got, ref, TOL_BF16)


def test_block_routing_prefill_hands_over_the_kept_cache_and_state():
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    B, H, L = 1, 2, 512
    x = block_inputs(wl, B, H, L, 0.4)
    ref = oracle_block(wl, x, want_cache=True)
    dt = tdtype(wl)
    res = binding.hybrid_fwd(dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt), dev(x["g"]),
                             dev(x["beta"]), dev(x["route"]), dev(x["w"]), scale_la=wl.scale_la,
                             scale_sm=wl.scale_sm, want=("state_out", "cache"),
                             flags=binding.BLOCK_ROUTING)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(res["ws"]) == 0
    k_sm, v_sm, sm_len = res["k_sm"], res["v_sm"], res["sm_len"]
    n = sm_len.cpu().numpy()
    assert np.array_equal(n, ref["n_sm"])                  # integer work: exact
    for b in range(B):
        for h in range(H):
            assert np.array_equal(k_sm[b, h, :n[b, h]].float().cpu().numpy(), ref["k_sm"][b, h, :n[b, h]])
            assert np.array_equal(v_sm[b, h, :n[b, h]].float().cpu().numpy(), ref["v_sm"][b, h, :n[b, h]])
    assert rel_err(res["state_out"].cpu().numpy(), ref["state_out"]) <= TOL_BF16


def test_block_routing_reports_a_route_that_changes_inside_a_block():
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    x = block_inputs(wl, 1, 2, 256, 0.5)
    x["route"][0, 70, 1] ^= 1
    dt = tdtype(wl)
    res = binding.hybrid_fwd(dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt), dev(x["g"]),
                             dev(x["beta"]), dev(x["route"]), dev(x["w"]), scale_la=wl.scale_la,
                             scale_sm=wl.scale_sm, flags=binding.BLOCK_ROUTING)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(res["ws"]) == binding.ERR_ROUTE


@pytest.mark.parametrize("name,B,H,L,p,flags,tol", [
    ("cfg0_f32_tiny_fwd", 1, 2, 256, 0.3, 0, 1e-4),       # fp32 storage: CUDA-core path, fp32 bar
    ("cfg0_f32_tiny_fwd", 2, 1, 448, 0.5, 0, 1e-4),
    ("cfg1_bf16_prefill", 1, 2, 320, 0.3, 1, 2e-2),       # bf16 storage forced onto the CUDA-core path
])
def test_block_routed_forward_on_the_cuda_core_path(name, B, H, L, p, flags, tol):
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS[name]
    x = block_inputs(wl, B, H, L, p)
    rng = np.random.default_rng(8)
    S0 = (0.1 * rng.standard_normal((B, H, wl.d, wl.d))).astype(np.float32)
    ref = oracle_block(wl, x, state_in=S0.astype(np.float64))
    got = run_fwd(wl, x, state_in=S0, flags=binding.BLOCK_ROUTING | flags)
    check_fwd(wl, got, ref, tol)


# ------------------------------------------------------------------ generation
def decode_blocks(wl, x, t0, t1, state, kc, vc, n, ref, tol):
    """Decode tokens t0..t1 of x with the block decision open, rolling back at each block's end;
    every step's output is checked against row t of the block-mode forward `ref`."""
    from paper_2602_03681_b200 import binding
    dt = tdtype(wl)
    B, _, H, d = x["q"].shape
    p = binding.make_params(B, H, 0, d, binding._dtype_code(kc), wl.scale_la, wl.scale_sm)
    ws = binding.alloc_workspace(p, binding.OP_DECODE)
    start = state.clone()
    undecided = torch.full((B, H), 2, dtype=torch.uint8, device="cuda")
    for t in range(t0, t1):
        w = dev(x["w"][:, t])
        p.w = w.data_ptr()
        out = torch.empty((B, H, d), dtype=dt, device="cuda")
        binding.natsl_decode_step(dev(x["q"][:, t], dt), dev(x["k"][:, t], dt), dev(x["v"][:, t], dt),
                                  dev(x["g"][:, t]), dev(x["beta"][:, t]), undecided, state, kc, vc, n,
                                  out, p, ws)
        check_stored(out.float().cpu().numpy(), ref["out"][:, t], tol, wl.dtype, f"step{t}")
        if (t + 1) % 64 == 0:
            g_block = x["g"][:, t - 63:t + 1].astype(np.float64).sum(1).astype(np.float32)
            binding.natsl_decode_block_end(dev(x["route"][:, t]), dev(g_block), state, start, n, 64, p, ws)
            assert torch.equal(state, start)
    assert binding.natsl_device_status(ws) == 0


@pytest.mark.parametrize("name,B,H,L0,L", [("cfg3_bf16_decode", 2, 2, 256, 448),
                                           ("cfg4_bf16_train", 1, 3, 128, 256)])
def test_block_routed_prefill_then_generation(name, B, H, L0, L):
    """Prefill L0 tokens, then generate up to L with route 2 and block ends: every step equals the
    block-mode forward over the whole sequence; so do the final state and the kept K/V."""
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS[name]
    x = block_inputs(wl, B, H, L, 0.4)
    ref = oracle_block(wl, x, want_cache=True)
    dt = tdtype(wl)
    pre = binding.hybrid_fwd(*(dev(x[n][:, :L0], dt) for n in ("q", "k", "v")), dev(x["g"][:, :L0]),
                             dev(x["beta"][:, :L0]), dev(x["route"][:, :L0]), dev(x["w"][:, :L0]),
                             scale_la=wl.scale_la, scale_sm=wl.scale_sm, want=("state_out", "cache"),
                             sm_cap=L, flags=binding.BLOCK_ROUTING)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(pre["ws"]) == 0
    state, kc, vc, n = pre["state_out"], pre["k_sm"], pre["v_sm"], pre["sm_len"]
    decode_blocks(wl, x, L0, L, state, kc, vc, n, ref, TOL_BF16)
    assert np.array_equal(n.cpu().numpy(), ref["n_sm"])
    assert rel_err(state.cpu().numpy(), ref["state_out"]) <= TOL_BF16
    for b in range(B):
        for h in range(H):
            m = ref["n_sm"][b, h]
            assert np.array_equal(kc[b, h, :m].float().cpu().numpy(), ref["k_sm"][b, h, :m])
            assert np.array_equal(vc[b, h, :m].float().cpu().numpy(), ref["v_sm"][b, h, :m])


def test_block_routed_generation_from_scratch_fp32():
    """fp32 storage, no prefill: two blocks generated from an empty state and cache, 1e-4."""
    wl = inputs.WORKLOADS["cfg0_f32_tiny_fwd"]
    B, H, L = 2, 2, 128
    x = block_inputs(wl, B, H, L, 0.5)
    x["route"][:, :64] = 0                 # a linear block first: its entries are dropped again
    x["route"][:, 64:] = 1
    ref = oracle_block(wl, x, want_cache=True)
    state = torch.zeros((B, H, wl.d, wl.d), device="cuda")
    kc = torch.zeros((B, H, L, wl.d), device="cuda")
    vc = torch.zeros_like(kc)
    n = torch.zeros((B, H), dtype=torch.int32, device="cuda")
    decode_blocks(wl, x, 0, L, state, kc, vc, n, ref, 1e-4)
    assert np.array_equal(n.cpu().numpy(), ref["n_sm"]) and np.all(ref["n_sm"] == 64)
    assert rel_err(state.cpu().numpy(), ref["state_out"]) <= 1e-4
    assert np.array_equal(kc[:, :, :64].cpu().numpy(), ref["k_sm"][:, :, :64].astype(np.float32))


def test_block_end_without_the_blocks_entries_is_reported():
    from paper_2602_03681_b200 import binding
    p = binding.make_params(1, 1, 0, 64, binding.NATSL_F32, 1.0, 1.0)
    ws = binding.alloc_workspace(p, binding.OP_DECODE)
    state = torch.zeros((1, 1, 64, 64), device="cuda")
    n = torch.full((1, 1), 10, dtype=torch.int32, device="cuda")
    binding.natsl_decode_block_end(torch.zeros((1, 1), dtype=torch.uint8, device="cuda"),
                                   torch.zeros((1, 1), device="cuda"), state, state.clone(), n, 64, p, ws)
    assert binding.natsl_device_status(ws) == binding.ERR_ROUTE
    assert n.item() == 10


# ------------------------------------------------------------------ backward
BWD_PATHS = {     # workload, flags, tolerance
    "fused_d64": ("cfg4_bf16_train", 0, TOL_BF16),          # tensor cores, one fused kernel per chunk
    "tc_d128": ("cfg1_bf16_prefill", 0, TOL_BF16),          # tensor cores, chunk-level products as tile GEMMs
    "f32_d64": ("cfg0_f32_tiny_fwd", 0, 1e-4),              # fp32 storage, CUDA cores
    "bf16_simt": ("cfg4_bf16_train", 1, 2e-4),              # fp32 arithmetic on bf16 storage (FORCE_SIMT)
}


@pytest.mark.parametrize("path,B,H,L,p", [
    ("fused_d64", 1, 2, 256, 0.4), ("fused_d64", 2, 3, 512, 0.25), ("fused_d64", 1, 1, 64, 0.0),
    ("fused_d64", 1, 2, 192, 1.0),
    ("tc_d128", 1, 2, 256, 0.4), ("tc_d128", 2, 2, 320, 0.25), ("tc_d128", 1, 1, 128, 0.0), ("tc_d128", 1, 1, 128, 1.0),
    ("f32_d64", 1, 2, 256, 0.4), ("f32_d64", 2, 1, 192, 0.6), ("f32_d64", 1, 1, 128, 0.0), ("f32_d64", 1, 1, 128, 1.0),
    ("bf16_simt", 1, 2, 192, 0.4),
])
def test_block_routed_backward_matches_oracle(path, B, H, L, p):
    """Backward under block-level routing against the oracle's block-mode backward, on every path."""
    from paper_2602_03681_b200 import binding
    from test_gpu_parity import check_bwd, run_bwd
    name, flags, tol = BWD_PATHS[path]
    wl = inputs.WORKLOADS[name]
    x = block_inputs(wl, B, H, L, p)
    if p in (0.0, 1.0):
        x["route"][:] = int(p)
    ref = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"],
                            scale_la=wl.scale_la, scale_sm=wl.scale_sm, block=64)
    got = run_bwd(wl, x, flags=binding.BLOCK_ROUTING | flags)
    check_bwd(wl, got, ref, tol)
    tok = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"],
                            scale_la=wl.scale_la, scale_sm=wl.scale_sm)
    if 0 < p < 1:       # the mode differs visibly from token-level routing on the same inputs
        assert rel_err(tok["dk"], ref["dk"]) > 10 * TOL_BF16


def test_block_routed_backward_fp32_d128_with_states():
    """fp32 storage at d = 128, with an initial state, a gradient at the final state and the gradient of
    the initial state."""
    import dataclasses
    from paper_2602_03681_b200 import binding
    from test_gpu_parity import check_bwd
    wl = dataclasses.replace(inputs.WORKLOADS["cfg0_f32_tiny_fwd"], d=128, seed=17)
    B, H, L = 1, 2, 192
    x = block_inputs(wl, B, H, L, 0.4)
    r = np.random.default_rng(4)
    s0 = (0.1 * r.standard_normal((B, H, 128, 128))).astype(np.float32)
    ds = (0.05 * r.standard_normal((B, H, 128, 128))).astype(np.float32)
    ref = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"],
                            scale_la=wl.scale_la, scale_sm=wl.scale_sm, block=64, state_in=s0, dstate_out=ds)
    res = binding.hybrid_bwd(*(dev(x[m]) for m in ("q", "k", "v")), dev(x["g"]), dev(x["beta"]),
                             dev(x["route"]), dev(x["w"]), dev(x["dout"]), scale_la=wl.scale_la,
                             scale_sm=wl.scale_sm, flags=binding.BLOCK_ROUTING, state_in=dev(s0),
                             dstate_out=dev(ds), want_dstate_in=True)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(res["ws"]) == 0
    got = {n: t.float().cpu().numpy() for n, t in res.items() if n != "ws"}
    check_bwd(wl, got, ref, 1e-4)
    assert rel_err(got["dstate_in"], ref["dstate_in"]) <= 1e-4


@pytest.mark.parametrize("path,B,H,L,p", [("fused_d64", 1, 2, 256, 0.4), ("fused_d64", 2, 3, 512, 0.25),
                                          ("tc_d128", 1, 2, 320, 0.4), ("f32_d64", 2, 2, 256, 0.4),
                                          ("bf16_simt", 1, 2, 192, 0.4)])
def test_block_routed_backward_score_gradients(path, B, H, L, p):
    """d score per block and head (Section 4.2) against the oracle: nonzero only for the operation
    the block chose."""
    from paper_2602_03681_b200 import binding
    name, flags, tol = BWD_PATHS[path]
    wl = inputs.WORKLOADS[name]
    x = block_inputs(wl, B, H, L, p)
    ref = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"],
                            scale_la=wl.scale_la, scale_sm=wl.scale_sm, block=64)["dscore"]
    dt = tdtype(wl)
    res = binding.hybrid_bwd(*(dev(x[m], dt) for m in ("q", "k", "v")), dev(x["g"]), dev(x["beta"]),
                             dev(x["route"]), dev(x["w"]), dev(x["dout"], dt), scale_la=wl.scale_la,
                             scale_sm=wl.scale_sm, flags=binding.BLOCK_ROUTING | flags, want_dscore=True)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(res["ws"]) == 0
    got = res["dscore"].cpu().numpy()
    blocks = x["route"][:, ::64]                                   # [B, L/64, H]
    assert np.all(got[..., 0][blocks == 1] == 0) and np.all(got[..., 1][blocks == 0] == 0)
    for op in (0, 1):
        assert rel_err(got[..., op], ref[..., op]) <= tol, (op, rel_err(got[..., op], ref[..., op]))
    assert np.abs(ref[..., 1]).max() > 0 and np.abs(ref[..., 0]).max() > 0


def test_score_gradients_need_block_routing():
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg4_bf16_train"]
    x = inputs.make_layer_inputs(wl, B=1, H=1, L=128)
    dt = tdtype(wl)
    with pytest.raises(binding.NatslError) as e:
        binding.hybrid_bwd(*(dev(x[m], dt) for m in ("q", "k", "v")), dev(x["g"]), dev(x["beta"]),
                           dev(x["route"]), dev(x["w"]), dev(x["dout"], dt), scale_la=wl.scale_la,
                           scale_sm=wl.scale_sm, want_dscore=True)
    assert e.value.status == binding.ERR_UNSUPPORTED
