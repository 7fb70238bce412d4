"""GPU parity of the tensor-core (tcgen05) forward, the default path for bf16 storage, against the
fp64 oracle: small and ragged shapes (one chunk, odd chunk counts, half-filled last query tile),
both head sizes, degenerate routings, initial state, prefill -> decode cache hand-off, extreme
decays, and agreement with the library's fp32 CUDA-core path."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_03681_b200 import inputs
from test_gpu_parity import (TOL, check_bwd, check_fwd, check_stored, dev, rel_err, run_bwd, run_fwd,
                             run_oracle)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,B,H,L", [("cfg1_bf16_prefill", 1, 1, 64),      # a single chunk
                                        ("cfg1_bf16_prefill", 2, 3, 192),     # odd number of chunks
                                        ("cfg1_bf16_prefill", 1, 2, 1088),    # several K/V tiles + tail
                                        ("cfg4_bf16_train", 1, 1, 64),
                                        ("cfg4_bf16_train", 2, 2, 448),
                                        ("cfg2_bf16_long_prefill", 1, 3, 1536)])
def test_fwd_tensor_core_small_cases(name, B, H, L):
    wl = inputs.WORKLOADS[name]
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L)
    check_fwd(wl, run_fwd(wl, x), run_oracle(wl, x), TOL["bf16"])


@pytest.mark.parametrize("name", ["cfg1_bf16_prefill", "cfg4_bf16_train"])
def test_fwd_tensor_core_initial_state_and_default_weights(name):
    wl = inputs.WORKLOADS[name]
    B, H, L = 2, 2, 320
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L)
    S0 = (0.1 * np.random.default_rng(5).standard_normal((B, H, wl.d, wl.d))).astype(np.float32)
    check_fwd(wl, run_fwd(wl, x, state_in=S0, w=None), run_oracle(wl, x, state_in=S0, w=None),
              TOL["bf16"])


@pytest.mark.parametrize("name", ["cfg1_bf16_prefill", "cfg4_bf16_train"])
def test_fwd_tensor_core_degenerate_routes(name):
    wl = inputs.WORKLOADS[name]
    B, H, L = 1, 2, 256
    for fill in (0, 1):
        x = inputs.make_layer_inputs(wl, B=B, H=H, L=L, route=np.full((B, L, H), fill, np.uint8))
        got, ref = run_fwd(wl, x), run_oracle(wl, x)
        check_fwd(wl, got, ref, TOL["bf16"])
        if fill == 0:                      # nothing retained: the softmax branch is exactly empty
            assert np.all(got["o_nla"] == 0) and np.all(np.isneginf(got["lse"]))
        else:                              # nothing folded: the state only decays from zero
            assert np.all(got["o_la"] == 0) and np.all(got["state_out"] == 0)


def test_fwd_tensor_core_single_retained_token_and_late_first_token():
    """Queries before the first retained token see an empty set; after it, exactly v of that token."""
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    B, H, L = 1, 2, 256
    route = np.zeros((B, L, H), np.uint8)
    route[0, 70, 0] = 1
    route[0, 200, 1] = 1
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L, route=route)
    got, ref = run_fwd(wl, x), run_oracle(wl, x)
    check_fwd(wl, got, ref, TOL["bf16"])
    for h, first in ((0, 70), (1, 200)):
        assert np.all(got["o_nla"][0, :first, h] == 0)
        assert np.allclose(got["o_nla"][0, first:, h], x["v"][0, first, h], rtol=2e-3, atol=1e-6)


def test_fwd_tensor_core_cache_handoff_matches_oracle():
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    B, H, L = 2, 3, 512
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L)
    dt = torch.bfloat16
    cap = 160
    res = binding.hybrid_fwd(dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt), dev(x["g"]),
                             dev(x["beta"]), dev(x["route"]), dev(x["w"]), scale_la=wl.scale_la,
                             scale_sm=wl.scale_sm, want=("cache", "o_nla", "lse"), sm_cap=cap)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(res["ws"]) == 0
    ref = run_oracle(wl, x, want_cache=True)
    n = res["sm_len"].cpu().numpy()
    assert np.array_equal(n, ref["n_sm"]) and n.max() <= cap
    for b in range(B):
        for h in range(H):
            m = n[b, h]
            assert np.array_equal(res["k_sm"][b, h, :m].float().cpu().numpy(),
                                  ref["k_sm"][b, h, :m].astype(np.float32))
            assert np.array_equal(res["v_sm"][b, h, :m].float().cpu().numpy(),
                                  ref["v_sm"][b, h, :m].astype(np.float32))
    assert rel_err(res["o_nla"].cpu().numpy(), ref["o_nla"]) <= TOL["bf16"]
    check_stored(res["out"].float().cpu().numpy(), ref["out"], TOL["bf16"], "bf16")


def test_fwd_tensor_core_cache_too_small_is_reported():
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    x = inputs.make_layer_inputs(wl, B=1, H=1, L=256, route=np.ones((1, 256, 1), np.uint8))
    dt = torch.bfloat16
    res = binding.hybrid_fwd(dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt), dev(x["g"]),
                             dev(x["beta"]), dev(x["route"]), dev(x["w"]), scale_la=wl.scale_la,
                             scale_sm=wl.scale_sm, want=("cache",), sm_cap=64)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(res["ws"]) == binding.ERR_CACHE_FULL
    assert torch.isfinite(res["out"].float()).all()
    assert int(res["sm_len"].max()) <= 64         # the stored length never exceeds the cache's rows


def test_decode_after_an_overflowed_prefill_stays_inside_the_cache():
    """A prefill whose cache was too small reports it and leaves sm_len = sm_cap; a decode step that
    follows (queued before the host could look at the status) reads only the cache's own rows, and
    a stored length beyond the capacity is clamped and reported, not followed."""
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    B, H, L, cap = 1, 2, 256, 64
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L, route=np.ones((B, L, H), np.uint8))
    dt = torch.bfloat16
    res = binding.hybrid_fwd(dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt), dev(x["g"]),
                             dev(x["beta"]), dev(x["route"]), dev(x["w"]), scale_la=wl.scale_la,
                             scale_sm=wl.scale_sm, want=("cache", "state_out"), sm_cap=cap)
    p = binding.make_params(B, H, 0, wl.d, binding.NATSL_BF16, wl.scale_la, wl.scale_sm)
    dws = binding.alloc_workspace(p, binding.OP_DECODE)
    tok = inputs.make_layer_inputs(wl, B=B, H=H, L=64)
    q1, k1, v1 = (dev(tok[m][:, 0], dt) for m in ("q", "k", "v"))
    g1, b1 = dev(tok["g"][:, 0]), dev(tok["beta"][:, 0])
    r0 = torch.zeros((B, H), dtype=torch.uint8, device="cuda")          # linear token: no append
    out = torch.empty((B, H, wl.d), dtype=dt, device="cuda")
    state = res["state_out"].clone()
    binding.natsl_decode_step(q1, k1, v1, g1, b1, r0, state, res["k_sm"], res["v_sm"], res["sm_len"],
                              out, p, dws)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(res["ws"]) == binding.ERR_CACHE_FULL   # the prefill's report
    assert binding.natsl_device_status(dws) == 0                              # the step itself is clean
    assert res["sm_len"].cpu().tolist() == [[cap, cap]]
    assert torch.isfinite(out.float()).all()
    # the same step checked against the oracle's decode on the cache the prefill left
    import oracle
    ref = oracle.decode_step(tok["q"][:, 0], tok["k"][:, 0], tok["v"][:, 0], tok["g"][:, 0],
                             tok["beta"][:, 0], np.zeros((B, H), np.uint8), None,
                             res["state_out"].cpu().numpy().astype(np.float64),
                             res["k_sm"].float().cpu().numpy().astype(np.float64),
                             res["v_sm"].float().cpu().numpy().astype(np.float64),
                             np.full((B, H), cap, np.int32), scale_la=wl.scale_la, scale_sm=wl.scale_sm)
    check_stored(out.float().cpu().numpy(), ref["out"], TOL["bf16"], "bf16")
    # a length the caller corrupted: clamped to the capacity and reported
    bad = torch.full((B, H), cap + 1000, dtype=torch.int32, device="cuda")
    binding.natsl_decode_step(q1, k1, v1, g1, b1, r0, state, res["k_sm"], res["v_sm"], bad, out, p, dws)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(dws) == binding.ERR_CACHE_FULL
    assert torch.isfinite(out.float()).all()


@pytest.mark.parametrize("g_value", [0.0, -3.0])
def test_fwd_tensor_core_decay_extremes(g_value):
    """No decay at all, and a decay strong enough that in-chunk factors underflow to zero."""
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    B, H, L = 1, 2, 256
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L)
    x["g"] = np.full((B, L, H), g_value, np.float32)
    got, ref = run_fwd(wl, x), run_oracle(wl, x)
    assert np.isfinite(got["out"]).all() and np.isfinite(got["o_la"]).all()
    check_fwd(wl, got, ref, TOL["bf16"])


def test_fwd_tensor_core_agrees_with_cuda_core_path():
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    x = inputs.make_layer_inputs(wl, B=1, H=4, L=768)
    a = run_fwd(wl, x)
    b = run_fwd(wl, x, flags=binding.FORCE_SIMT)
    for name in ("o_la", "o_nla", "state_out"):
        assert rel_err(a[name], b[name]) <= TOL["bf16"], name
    assert np.array_equal(np.isneginf(a["lse"]), np.isneginf(b["lse"]))


def test_fwd_tensor_core_is_deterministic():
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    x = inputs.make_layer_inputs(wl, B=1, H=2, L=512)
    a, b = run_fwd(wl, x), run_fwd(wl, x)
    for name in ("out", "o_la", "o_nla", "lse", "state_out"):
        assert np.array_equal(a[name], b[name]), name


# ------------------------------------------------------------------ backward (softmax branch on tcgen05)
@pytest.mark.parametrize("name,B,H,L,route", [("cfg4_bf16_train", 2, 3, 320, None),
                                              ("cfg4_bf16_train", 1, 2, 64, None),
                                              ("cfg1_bf16_prefill", 1, 2, 448, None),
                                              # d = 128 (separate chunk-level kernels, two streams): one chunk;
                                              # odd batch and head counts; all tokens retained
                                              ("cfg1_bf16_prefill", 3, 1, 64, None),
                                              ("cfg1_bf16_prefill", 3, 5, 128, None),
                                              ("cfg1_bf16_prefill", 1, 3, 192, "all_softmax"),
                                              ("cfg4_bf16_train", 1, 2, 384, "all_softmax"),
                                              ("cfg1_bf16_prefill", 1, 2, 256, "all_linear"),
                                              ("cfg4_bf16_train", 1, 1, 256, "late")])
def test_bwd_tensor_core_softmax_branch(name, B, H, L, route):
    wl = inputs.WORKLOADS[name]
    r = None
    if route == "all_softmax":
        r = np.ones((B, L, H), np.uint8)
    elif route == "all_linear":
        r = np.zeros((B, L, H), np.uint8)
    elif route == "late":                         # queries before token 100 see nothing
        r = np.zeros((B, L, H), np.uint8)
        r[:, 100, :] = 1
        r[:, 101:, :] = (np.random.default_rng(1).random((B, L - 101, H)) < 0.3)
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L, route=r)
    got = run_bwd(wl, x)
    ref = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"],
                            scale_la=wl.scale_la, scale_sm=wl.scale_sm)
    for name_ in ("dq", "dk", "dv", "dg", "dbeta", "dw"):
        assert np.isfinite(got[name_]).all(), name_
    check_bwd(wl, got, ref, TOL["bf16"])
    lin = x["route"] == 0
    assert np.all(got["dbeta"][~lin] == 0)


@pytest.mark.parametrize("scale", [2.0 ** -20, 2.0 ** -6, 2.0 ** 6, 2.0 ** 20])
@pytest.mark.parametrize("name,block", [("cfg4_bf16_train", False), ("cfg4_bf16_train", True),
                                        ("cfg1_bf16_prefill", False)])
def test_bwd_tensor_core_is_linear_in_the_incoming_gradient(scale, name, block):
    """Every gradient is linear in dout.  A loss-scaled or a tiny dout must not leave the range of
    the fp16 operands: the read-out gradients are scaled by a power of two taken from max |dout|
    (reverse scan, softmax backward), the chunk kernel rescales its gradient tiles per chunk, and
    neither may show in the result."""
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS[name]
    B, H, L = 1, 2, 256
    route = inputs.route_blocks(wl.seed, (B, L, H), wl.p_softmax) if block else None
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L, route=route)
    x["dout"] = (x["dout"] * scale).astype(np.float32)      # power of two: still exact in bf16
    got = run_bwd(wl, x, flags=binding.BLOCK_ROUTING if block else 0)
    ref = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"],
                            scale_la=wl.scale_la, scale_sm=wl.scale_sm, block=64 if block else None)
    check_bwd(wl, got, ref, TOL["bf16"])


@pytest.mark.parametrize("name", ["cfg4_bf16_train", "cfg1_bf16_prefill"])
@pytest.mark.parametrize("block", [False, True])
def test_bwd_on_one_stream_gives_the_same_bits(name, block):
    """NATSL_SINGLE_STREAM puts every kernel of the backward on the caller's stream; by default independent
    stages run on a second stream beside it (d = 64: reverse scan and key-side softmax kernel beside the
    query-side and chunk kernels; d = 128: the whole linear branch beside the softmax branch).  Same kernels,
    same inputs: the gradients must agree bit for bit, or two stages share a buffer they should not."""
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS[name]
    B, H, L = 2, 3, 512
    route = inputs.route_blocks(wl.seed, (B, L, H), wl.p_softmax) if block else None
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L, route=route)
    f = binding.BLOCK_ROUTING if block else 0
    a = run_bwd(wl, x, flags=f)
    b = run_bwd(wl, x, flags=f | binding.SINGLE_STREAM)
    for n in ("dq", "dk", "dv", "dg", "dbeta", "dw"):
        assert np.array_equal(a[n], b[n]), n


@pytest.mark.parametrize("name", ["cfg4_bf16_train", "cfg1_bf16_prefill"])
def test_bwd_tensor_core_many_chunks(name):
    wl = inputs.WORKLOADS[name]
    x = inputs.make_layer_inputs(wl, B=1, H=2, L=1024)
    got = run_bwd(wl, x)
    ref = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"],
                            scale_la=wl.scale_la, scale_sm=wl.scale_sm)
    check_bwd(wl, got, ref, TOL["bf16"])


@pytest.mark.parametrize("name,L", [("cfg1_bf16_prefill", 704), ("cfg4_bf16_train", 448)])
def test_fwd_tensor_core_out_only(name, L):
    """The call as the bench makes it: no optional output requested (the raw branch outputs stay in
    the workspace), last query tile half filled."""
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS[name]
    x = inputs.make_layer_inputs(wl, B=2, H=2, L=L)
    dt = torch.bfloat16
    res = binding.hybrid_fwd(dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt), dev(x["g"]),
                             dev(x["beta"]), dev(x["route"]), dev(x["w"]), scale_la=wl.scale_la,
                             scale_sm=wl.scale_sm)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(res["ws"]) == 0
    ref = run_oracle(wl, x)
    check_stored(res["out"].float().cpu().numpy(), ref["out"], TOL["bf16"], "bf16")


@pytest.mark.parametrize("name,H,L", [("cfg1_bf16_prefill", 2, 2048), ("cfg4_bf16_train", 3, 1024)])
def test_fwd_tensor_core_segmented_scan_with_weak_decay(name, H, L):
    """With few (batch, head) pairs the scan runs as parallel segments chained by their state
    transitions.  With almost no decay a segment's entry state still matters at its end, so the
    transition matrices carry real weight here (with the workloads' decay they are ~0)."""
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS[name]
    x = inputs.make_layer_inputs(wl, B=1, H=H, L=L)
    x["g"] = np.full((1, L, H), -1e-3, np.float32)
    S0 = (0.2 * np.random.default_rng(11).standard_normal((1, H, wl.d, wl.d))).astype(np.float32)
    seg = run_fwd(wl, x, state_in=S0)
    one = run_fwd(wl, x, state_in=S0, flags=binding.SINGLE_PASS_SCAN)
    ref = run_oracle(wl, x, state_in=S0)
    check_fwd(wl, seg, ref, TOL["bf16"])
    check_fwd(wl, one, ref, TOL["bf16"])
    for n in ("o_la", "state_out"):
        assert rel_err(seg[n], one[n]) <= TOL["bf16"], n
    assert not np.array_equal(seg["state_out"], one["state_out"])   # the two paths really differ
