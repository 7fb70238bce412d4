"""GPU parity of two backward features against the fp64 oracle:

* the state carried across calls (Section 3, chunkwise recurrence): a backward that starts from a
  non-zero initial state, receives a gradient at its final state and returns the gradient of the
  initial state -- on the fused tensor-core path (d = 64), the tensor-core path with tile GEMMs
  (d = 128) and the fp32 CUDA-core path;
* the forward run with NATSL_SAVE_FOR_BWD in the backward's workspace, after which the backward
  (NATSL_SAVED_FWD) starts at the gradients: same `out` as the plain forward, same gradients as
  the self-contained backward, both within the oracle's tolerance.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_03681_b200 import inputs
from test_gpu_parity import TOL, check_bwd, check_stored, dev, rel_err, tdtype

pytestmark = pytest.mark.gpu


def _states(wl, B, H, seed):
    rng = np.random.default_rng(seed)
    s0 = (0.1 * rng.standard_normal((B, H, wl.d, wl.d))).astype(np.float32)
    ds = (0.05 * rng.standard_normal((B, H, wl.d, wl.d))).astype(np.float32)
    return s0, ds


@pytest.mark.parametrize("name,B,H,L,flags,tol", [
    ("cfg4_bf16_train", 2, 2, 320, 0, 2e-2),          # fused chunk kernel (d = 64)
    ("cfg1_bf16_prefill", 1, 2, 256, 0, 2e-2),        # tensor cores, d = 128
    ("cfg0_f32_tiny_fwd", 1, 2, 192, 0, 1e-4),        # fp32 CUDA cores
    ("cfg4_bf16_train", 1, 2, 128, 1, 2e-4),          # fp32 arithmetic on bf16 storage (FORCE_SIMT)
])
def test_bwd_through_initial_and_final_state(name, B, H, L, flags, tol):
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS[name]
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L)
    s0, ds = _states(wl, B, H, 11)
    dt = tdtype(wl)
    res = binding.hybrid_bwd(dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt), dev(x["g"]),
                             dev(x["beta"]), dev(x["route"]), dev(x["w"]), dev(x["dout"], dt),
                             scale_la=wl.scale_la, scale_sm=wl.scale_sm, flags=flags,
                             state_in=dev(s0), dstate_out=dev(ds), want_dstate_in=True)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(res["ws"]) == 0
    got = {n: t.float().cpu().numpy() for n, t in res.items() if n != "ws"}
    ref = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"],
                            scale_la=wl.scale_la, scale_sm=wl.scale_sm, state_in=s0, dstate_out=ds)
    check_bwd(wl, got, ref, tol)
    assert rel_err(got["dstate_in"], ref["dstate_in"]) <= tol
    # the state gradient really took part: without it dk of the last chunk differs
    ref0 = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"],
                             scale_la=wl.scale_la, scale_sm=wl.scale_sm, state_in=s0)
    assert rel_err(ref0["dk"], ref["dk"]) > 2 * tol


@pytest.mark.parametrize("name,B,H,L,block", [("cfg4_bf16_train", 2, 3, 448, False),
                                              ("cfg4_bf16_train", 1, 2, 256, True),
                                              ("cfg1_bf16_prefill", 1, 2, 256, True),
                                              ("cfg0_f32_tiny_fwd", 1, 2, 192, True),
                                              ("cfg1_bf16_prefill", 1, 2, 256, False),
                                              ("cfg0_f32_tiny_fwd", 1, 2, 128, False)])
def test_saved_forward_then_backward(name, B, H, L, block):
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS[name]
    route = inputs.route_blocks(wl.seed, (B, L, H), wl.p_softmax) if block else None
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L, route=route)
    dt = tdtype(wl)
    kind = wl.dtype
    base = binding.BLOCK_ROUTING if block else 0
    q, k, v = dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt)
    g, beta, r, w, dout = dev(x["g"]), dev(x["beta"]), dev(x["route"]), dev(x["w"]), dev(x["dout"], dt)
    kw = dict(scale_la=wl.scale_la, scale_sm=wl.scale_sm)
    plain = binding.hybrid_fwd(q, k, v, g, beta, r, w, flags=base, want=("state_out",), **kw)
    alone = binding.hybrid_bwd(q, k, v, g, beta, r, w, dout, flags=base, **kw)
    # forward in the backward's workspace, then the backward from what it left there
    p = binding.make_params(B, H, L, wl.d, binding._dtype_code(q), wl.scale_la, wl.scale_sm, w=w,
                            flags=base | binding.SAVE_FOR_BWD)
    state_out = torch.empty((B, H, wl.d, wl.d), dtype=torch.float32, device="cuda")
    p.state_out = state_out.data_ptr()
    ws = binding.alloc_workspace(p, binding.OP_BWD)
    out = torch.empty_like(q)
    binding.natsl_hybrid_fwd(q, k, v, g, beta, r, out, p, ws)
    saved = binding.hybrid_bwd(q, k, v, g, beta, r, w, dout, flags=base | binding.SAVED_FWD, ws=ws, **kw)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(ws) == 0
    ref_f = oracle.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"],
                              block=64 if block else None, **kw)
    check_stored(out.float().cpu().numpy(), ref_f["out"], TOL[kind], kind)
    assert rel_err(state_out.cpu().numpy(), ref_f["state_out"]) <= TOL[kind]
    assert rel_err(out.float().cpu().numpy(), plain["out"].float().cpu().numpy()) <= TOL[kind]
    ref_b = oracle.hybrid_bwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], x["dout"],
                              block=64 if block else None, **kw)
    got = {n: t.float().cpu().numpy() for n, t in saved.items() if n != "ws"}
    check_bwd(wl, got, ref_b, TOL[kind])
    for n in ("dq", "dk", "dv", "dg", "dbeta", "dw"):      # same kernels on the same inputs
        a = alone[n].float().cpu().numpy()
        assert np.abs(got[n] - a).max() <= 1e-3 * TOL[kind] * max(np.sqrt((a ** 2).mean()), 1e-30) + \
            (np.abs(a).max() * 2.0 ** -8 if kind == "bf16" and n in ("dq", "dk", "dv") else 0.0), n
