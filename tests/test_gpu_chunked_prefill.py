"""Prefill in pieces (state_in / state_out chained, retained K/V appended to one cache) against
the oracle's forward over the whole sequence, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_03681_b200 import inputs
from test_gpu_parity import check_stored, dev, rel_err, tdtype

pytestmark = pytest.mark.gpu

TOL = 2e-2


def prefill_in_pieces(wl, x, pieces, cap, flags):
    from paper_2602_03681_b200 import binding
    dt = tdtype(wl)
    B, L, H, d = x["q"].shape
    k_sm = torch.zeros((B, H, cap, d), dtype=dt, device="cuda")
    v_sm = torch.zeros_like(k_sm)
    sm_len = torch.zeros((B, H), dtype=torch.int32, device="cuda")
    state = None
    outs, lses = [], []
    t0 = 0
    for n in pieces:
        sl = slice(t0, t0 + n)
        res = binding.hybrid_fwd(*(dev(x[m][:, sl], dt) for m in ("q", "k", "v")), dev(x["g"][:, sl]),
                                 dev(x["beta"][:, sl]), dev(x["route"][:, sl]), dev(x["w"][:, sl]),
                                 scale_la=wl.scale_la, scale_sm=wl.scale_sm, state_in=state,
                                 want=("state_out", "lse"), cache=(k_sm, v_sm, sm_len),
                                 flags=flags | binding.APPEND_CACHE)
        torch.cuda.synchronize()
        assert binding.natsl_device_status(res["ws"]) == 0
        state = res["state_out"]
        outs.append(res["out"].float().cpu().numpy())
        lses.append(res["lse"].cpu().numpy())
        t0 += n
    assert t0 == L
    return dict(out=np.concatenate(outs, 1), lse=np.concatenate(lses, 2), state=state.cpu().numpy(),
                k_sm=k_sm, v_sm=v_sm, sm_len=sm_len.cpu().numpy())


@pytest.mark.parametrize("name,B,H,pieces,block", [
    ("cfg1_bf16_prefill", 1, 2, (256, 256, 256), False),
    ("cfg1_bf16_prefill", 2, 2, (128, 448, 64, 320), False),    # uneven pieces, odd tile counts
    ("cfg4_bf16_train", 1, 3, (192, 320), False),               # d = 64
    ("cfg1_bf16_prefill", 1, 2, (256, 128, 384), True),         # with block-level routing
    ("cfg1_bf16_prefill", 1, 1, (1024, 1024), False),           # segmented scan inside a piece
])
def test_prefill_in_pieces_equals_the_whole(name, B, H, pieces, block):
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS[name]
    L = sum(pieces)
    route = inputs.route_blocks(wl.seed, (B, L, H), 0.3) if block else None
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L, route=route)
    ref = oracle.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"],
                            scale_la=wl.scale_la, scale_sm=wl.scale_sm, want_cache=True,
                            block=64 if block else None)
    got = prefill_in_pieces(wl, x, pieces, cap=L, flags=binding.BLOCK_ROUTING if block else 0)
    check_stored(got["out"], ref["out"], TOL, wl.dtype)
    ok = np.isfinite(ref["lse"])
    assert np.array_equal(np.isfinite(got["lse"]), ok)
    assert np.abs(got["lse"][ok] - ref["lse"][ok]).max() <= 2 * TOL
    assert rel_err(got["state"], ref["state_out"]) <= TOL
    assert np.array_equal(got["sm_len"], ref["n_sm"])               # integer work: exact
    for b in range(B):
        for h in range(H):
            m = ref["n_sm"][b, h]
            assert np.array_equal(got["k_sm"][b, h, :m].float().cpu().numpy(), ref["k_sm"][b, h, :m])
            assert np.array_equal(got["v_sm"][b, h, :m].float().cpu().numpy(), ref["v_sm"][b, h, :m])


def test_appending_beyond_the_cache_capacity_is_reported():
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    x = inputs.make_layer_inputs(wl, B=1, H=1, L=256)
    x["route"][:] = 1
    dt = tdtype(wl)
    cache = (torch.zeros((1, 1, 384, wl.d), dtype=dt, device="cuda"),
             torch.zeros((1, 1, 384, wl.d), dtype=dt, device="cuda"),
             torch.zeros((1, 1), dtype=torch.int32, device="cuda"))
    args = [dev(x[m], dt) for m in ("q", "k", "v")] + [dev(x["g"]), dev(x["beta"]), dev(x["route"]), dev(x["w"])]
    r1 = binding.hybrid_fwd(*args, scale_la=wl.scale_la, scale_sm=wl.scale_sm, cache=cache,
                            flags=binding.APPEND_CACHE)
    assert binding.natsl_device_status(r1["ws"]) == 0 and cache[2].item() == 256
    r2 = binding.hybrid_fwd(*args, scale_la=wl.scale_la, scale_sm=wl.scale_sm, cache=cache,
                            flags=binding.APPEND_CACHE)
    assert binding.natsl_device_status(r2["ws"]) == binding.ERR_CACHE_FULL


def test_append_needs_a_cache_and_the_tensor_core_path():
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    x = inputs.make_layer_inputs(wl, B=1, H=1, L=128)
    dt = tdtype(wl)
    args = [dev(x[m], dt) for m in ("q", "k", "v")] + [dev(x["g"]), dev(x["beta"]), dev(x["route"]), dev(x["w"])]
    with pytest.raises(binding.NatslError) as e:
        binding.hybrid_fwd(*args, scale_la=1.0, scale_sm=1.0, flags=binding.APPEND_CACHE)
    assert e.value.status == -1
    with pytest.raises(binding.NatslError) as e:
        binding.hybrid_fwd(*args, scale_la=1.0, scale_sm=1.0, want=("cache",),
                           flags=binding.APPEND_CACHE | binding.FORCE_SIMT)
    assert e.value.status == binding.ERR_UNSUPPORTED
