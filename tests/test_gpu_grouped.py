"""GPU parity of the forward with grouped softmax heads and in-kernel q/k normalisation
(Section 4.3: several softmax heads under one linear head's mask; L2-normalised q, k for the linear
operation, RMS-normalised for the softmax operation) against `oracle/grouped.py`, element by element
on the same seeded inputs:

* fp32 storage (CUDA-core kernels): d = 64 and 128, G = 1, 2, 4, with and without normalisation;
* bf16 storage (tensor-core kernels): d = 128 with G = 2 -- six linear heads with twelve softmax heads,
  the appendix's smaller model -- and G = 1 with normalisation, on shapes that take the one-pass scan,
  and the segmented scan;
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


def make_inputs(wl, B, H, L, unnormalised):
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L)
    if unnormalised:      # rows of very different lengths: the normalisation has something to do
        r = np.random.default_rng(wl.seed + 100)
        for n in ("q", "k"):
            x[n] = (x[n] * np.exp(0.7 * r.standard_normal((B, L, H, 1)))).astype(np.float32)
            if wl.dtype == "bf16":
                x[n] = inputs.round_bf16(x[n])
    return x


def run_both(wl, x, G, norm, scale_sm, norm_eps=1e-6, flags=0):
    from paper_2602_03681_b200 import binding
    dt = tdtype(wl)
    f = flags | (binding.QK_NORM if norm else 0)
    res = binding.hybrid_fwd(dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt), dev(x["g"]), dev(x["beta"]),
                             dev(x["route"]), dev(x["w"]), scale_la=wl.scale_la, scale_sm=scale_sm,
                             want=("o_la", "o_nla", "lse", "state_out"), flags=f, G=G, norm_eps=norm_eps)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(res["ws"]) == 0
    got = {n: t.float().cpu().numpy() for n, t in res.items() if n != "ws"}
    ref = grouped.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"], G=max(G, 1),
                             qk_norm=norm, scale_la=wl.scale_la, scale_sm=scale_sm, norm_eps=norm_eps)
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
    assert refused(lambda: binding.hybrid_fwd(*args, G=2, flags=binding.BLOCK_ROUTING, **kw))
    assert refused(lambda: binding.hybrid_fwd(*args, G=2, flags=binding.FORCE_SIMT, **kw))        # bf16 on CUDA cores
    assert refused(lambda: binding.hybrid_fwd(*args, flags=binding.QK_NORM, want=("cache",), **kw))
    with pytest.raises(binding.NatslError):                                                       # G must divide d
        binding.hybrid_fwd(*args, G=3, **kw)
    p = binding.make_params(1, 2, 128, 128, binding.NATSL_BF16, wl.scale_la, wl.scale_sm, G=2)
    n = binding.natsl_workspace_size(p, binding.OP_BWD)
    ws = torch.zeros(n, dtype=torch.uint8, device="cuda")
    outs = [torch.empty_like(args[0]) for _ in range(3)] + [torch.empty_like(args[3]) for _ in range(2)]
    dw = torch.empty((1, 128, 2, 2), device="cuda")
    with pytest.raises(binding.NatslError) as e:
        binding.natsl_hybrid_bwd(*args[:6], args[0], *outs, dw, p, ws)
    assert e.value.status == binding.ERR_UNSUPPORTED
