"""The allocation-free forward (natsl_hybrid_fwd_static) against the ordinary entry point.

Some hosts of the library cannot allocate device memory (a plug-in inside a server that owns the
pool; a loop that must avoid cudaMalloc's device-wide synchronisation), so this entry point takes
its scratch from a fixed array inside the library.  It must give what natsl_hybrid_fwd gives, also
on a second call that finds the previous call's leftovers in the shared array."""
import numpy as np
import pytest
import torch

from paper_2602_03681_b200 import inputs

pytestmark = pytest.mark.gpu


def _dev(a, dt=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t if dt is None else t.to(dt)


def _both(binding, wl, x, dt):
    q, k, v = _dev(x["q"], dt), _dev(x["k"], dt), _dev(x["v"], dt)
    g, beta, route, w = _dev(x["g"]), _dev(x["beta"]), _dev(x["route"]), _dev(x["w"])
    B, L, H, d = q.shape
    outs = []
    for static in (False, True):
        out = torch.zeros_like(q)
        o_la = torch.zeros((B, L, H, d), dtype=torch.float32, device="cuda")
        lse = torch.zeros((B, H, L), dtype=torch.float32, device="cuda")
        p = binding.make_params(B, H, L, d, binding._dtype_code(q), wl.scale_la, wl.scale_sm, w=w,
                                o_la=o_la, lse=lse)
        if static:
            binding.natsl_hybrid_fwd_static(q, k, v, g, beta, route, out, p)
        else:
            ws = binding.alloc_workspace(p, binding.OP_FWD)
            binding.natsl_hybrid_fwd(q, k, v, g, beta, route, out, p, ws)
        torch.cuda.synchronize()
        outs.append((out.float().cpu().numpy(), o_la.cpu().numpy(), lse.cpu().numpy()))
    return outs


def test_static_forward_matches_workspace_forward_twice():
    from paper_2602_03681_b200 import binding
    from test_gpu_parity import TOL, check_stored, rel_err, run_oracle
    # two different problems back to back: the second call sees the first one's scratch contents
    cases = [("cfg1_bf16_prefill", torch.bfloat16, dict(B=1, H=2, L=1024)),
             ("cfg0_f32_tiny_fwd", torch.float32, dict(B=1, H=2, L=256))]
    for name, dt, size in cases:
        wl = inputs.WORKLOADS[name]
        x = inputs.make_layer_inputs(wl, **size)
        (out_a, ola_a, lse_a), (out_b, ola_b, lse_b) = _both(binding, wl, x, dt)
        # the same kernels on the same stream, and the forward is deterministic: identical bits
        assert np.array_equal(out_a, out_b)
        assert np.array_equal(ola_a, ola_b)
        assert np.array_equal(lse_a, lse_b)
        # ... and the right ones: the static entry point against the oracle
        kind = "bf16" if dt == torch.bfloat16 else "f32"
        ref = run_oracle(wl, x)
        check_stored(out_b, ref["out"], TOL[kind], kind)
        assert rel_err(ola_b, ref["o_la"]) <= TOL[kind]
    assert binding.natsl_static_status() == 0


def test_static_forward_allocates_nothing_and_reports_device_side_errors():
    """After the first call on the device, a static call leaves the free device memory where it
    was although it launches kernels; and what only the device can detect (here: block-level
    routing with a route that changes inside a block) is read back through natsl_static_status."""
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    x = inputs.make_layer_inputs(wl, B=1, H=2, L=512)
    dt = torch.bfloat16
    q, k, v = _dev(x["q"], dt), _dev(x["k"], dt), _dev(x["v"], dt)
    g, beta, route, w = _dev(x["g"]), _dev(x["beta"]), _dev(x["route"]), _dev(x["w"])
    out = torch.zeros_like(q)
    B, L, H, d = q.shape
    p = binding.make_params(B, H, L, d, binding.NATSL_BF16, wl.scale_la, wl.scale_sm, w=w)
    binding.natsl_hybrid_fwd_static(q, k, v, g, beta, route, out, p)       # set-up call
    torch.cuda.synchronize()
    assert binding.natsl_static_status() == 0
    free0, _ = torch.cuda.mem_get_info()
    launches0 = binding.natsl_launch_count()
    for _ in range(3):
        binding.natsl_hybrid_fwd_static(q, k, v, g, beta, route, out, p)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert binding.natsl_launch_count() > launches0
    # token-level route handed to block-level routing: the route changes inside blocks
    pb = binding.make_params(B, H, L, d, binding.NATSL_BF16, wl.scale_la, wl.scale_sm, w=w,
                             flags=binding.BLOCK_ROUTING)
    binding.natsl_hybrid_fwd_static(q, k, v, g, beta, route, out, pb)
    assert binding.natsl_static_status() == binding.ERR_ROUTE
    assert binding.natsl_static_status() == 0                               # reading clears it


def test_static_forward_rejects_problems_beyond_its_scratch():
    from paper_2602_03681_b200 import binding
    B, H, L, d = 2, 8, 4096, 128
    q = torch.zeros((B, L, H, d), dtype=torch.bfloat16, device="cuda")
    g = torch.zeros((B, L, H), device="cuda")
    r = torch.zeros((B, L, H), dtype=torch.uint8, device="cuda")
    p = binding.make_params(B, H, L, d, binding.NATSL_BF16, 1.0, 1.0)
    assert binding.natsl_workspace_size(p, binding.OP_FWD) > binding.STATIC_WS_BYTES
    with pytest.raises(binding.NatslError) as e:
        binding.natsl_hybrid_fwd_static(q, q, q, g, g, r, torch.empty_like(q), p)
    assert e.value.status == binding.ERR_TOO_LARGE
    assert "scratch" in str(e.value)
