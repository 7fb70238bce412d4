"""The decode step replayed from a CUDA graph: one step is captured once (static input buffers,
state and cache updated in place) and replayed for every token, as a serving loop would do."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_03681_b200 import inputs
from test_gpu_parity import TOL, check_stored, dev, rel_err

pytestmark = pytest.mark.gpu


def test_decode_steps_replayed_from_a_cuda_graph():
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg3_bf16_decode"]
    B, H, steps = 2, 4, 12
    x = inputs.make_decode_inputs(wl, B=B, H=H, steps=steps, ctx_retained=150)
    dt = torch.bfloat16
    state, n = dev(x["state"]), dev(x["cache_len"])
    kc, vc = dev(x["k_cache"], dt), dev(x["v_cache"], dt)
    o_state = x["state"].astype(np.float64)
    o_kc, o_vc, o_n = x["k_cache"].astype(np.float64), x["v_cache"].astype(np.float64), x["cache_len"].copy()
    # static buffers the captured step reads
    sq, sk, sv = (torch.zeros((B, H, wl.d), dtype=dt, device="cuda") for _ in range(3))
    sg, sb = torch.zeros((B, H), device="cuda"), torch.zeros((B, H), device="cuda")
    sr = torch.zeros((B, H), dtype=torch.uint8, device="cuda")
    sw = torch.zeros((B, H, 2), device="cuda")
    out = torch.zeros((B, H, wl.d), dtype=dt, device="cuda")
    p = binding.make_params(B, H, 0, wl.d, binding.NATSL_BF16, wl.scale_la, wl.scale_sm, w=sw)
    ws = binding.alloc_workspace(p, binding.OP_DECODE)

    def load(t):
        sq.copy_(dev(x["q"][t], dt)); sk.copy_(dev(x["k"][t], dt)); sv.copy_(dev(x["v"][t], dt))
        sg.copy_(dev(x["g"][t])); sb.copy_(dev(x["beta"][t])); sr.copy_(dev(x["route"][t]))
        sw.copy_(dev(x["w"][t]))

    def check(t):
        ref = oracle.decode_step(x["q"][t], x["k"][t], x["v"][t], x["g"][t], x["beta"][t], x["route"][t],
                                 x["w"][t], o_state, o_kc, o_vc, o_n, scale_la=wl.scale_la,
                                 scale_sm=wl.scale_sm)
        check_stored(out.float().cpu().numpy(), ref["out"], TOL[wl.dtype], wl.dtype, f"step{t}")

    # step 0 runs eagerly (first use of the kernel), step 1 is captured, the rest are replays
    load(0)
    binding.natsl_decode_step(sq, sk, sv, sg, sb, sr, state, kc, vc, n, out, p, ws)
    check(0)
    load(1)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.natsl_decode_step(sq, sk, sv, sg, sb, sr, state, kc, vc, n, out, p, ws)
    # capturing does not execute: state and cache are still those after step 0
    for t in range(1, steps):
        load(t)
        graph.replay()
        torch.cuda.synchronize()
        check(t)
    assert binding.natsl_device_status(ws) == 0
    assert np.array_equal(n.cpu().numpy(), o_n)
    assert rel_err(state.cpu().numpy(), o_state) <= 1e-4
