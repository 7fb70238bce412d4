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
    # two different problems back to back: the second call sees the first one's scratch contents
    cases = [("cfg1_bf16_prefill", torch.bfloat16, dict(B=1, H=2, L=1024)),
             ("cfg0_f32_tiny_fwd", torch.float32, dict(B=1, H=2, L=256))]
    for name, dt, size in cases:
        wl = inputs.WORKLOADS[name]
        x = inputs.make_layer_inputs(wl, **size)
        (out_a, ola_a, lse_a), (out_b, ola_b, lse_b) = _both(binding, wl, x, dt)
        tol = 2e-2 if dt == torch.bfloat16 else 1e-4
        rms = np.sqrt((out_a.astype(np.float64) ** 2).mean())
        assert np.abs(out_a - out_b).max() <= tol * rms
        assert np.abs(ola_a - ola_b).max() <= tol * np.sqrt((ola_a.astype(np.float64) ** 2).mean())
        fin = np.isfinite(lse_a)
        assert np.array_equal(fin, np.isfinite(lse_b))
        assert np.abs(lse_a[fin] - lse_b[fin]).max() <= 1e-3


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
