"""The time-out path of the tensor-core kernels, exercised without a fault and without a hang.

Every device-side wait of those kernels is bounded.  The test hook natsl_debug_set_wait_limit
shortens the bound to a few milliseconds and makes the scan withhold the per-chunk counters that
the softmax kernel's epilogue waits for: that one wait (a counter nothing raises) then runs out in
every CTA of the softmax kernel, the kernel records NATSL_ERR_TIMEOUT, lets its copies land,
frees its tensor memory and returns.  The next call on the same workspace, with the hook off, must
be correct."""
import numpy as np
import pytest
import torch

from paper_2602_03681_b200 import inputs
from test_gpu_parity import TOL, check_fwd, dev, run_fwd, run_oracle

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_workspace_stays_usable():
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    B, H, L = 1, 2, 128                       # one query tile per (batch, head): two CTAs wait
    x = inputs.make_layer_inputs(wl, B=B, H=H, L=L)
    dt = torch.bfloat16
    args = [dev(x["q"], dt), dev(x["k"], dt), dev(x["v"], dt), dev(x["g"]), dev(x["beta"]),
            dev(x["route"]), dev(x["w"])]
    first = binding.hybrid_fwd(*args, scale_la=wl.scale_la, scale_sm=wl.scale_sm)
    torch.cuda.synchronize()
    ws = first["ws"]
    assert binding.natsl_device_status(ws) == 0
    try:
        binding.natsl_debug_set_wait_limit(8192, withhold_scan_flags=True)    # 8 M cycles, ~4 ms
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        binding.hybrid_fwd(*args, scale_la=wl.scale_la, scale_sm=wl.scale_sm, ws=ws)
        t1.record()
        torch.cuda.synchronize()
        assert binding.natsl_device_status(ws) == binding.ERR_TIMEOUT
        assert t0.elapsed_time(t1) < 1000.0        # the bound, not the default two seconds
    finally:
        binding.natsl_debug_set_wait_limit(0, withhold_scan_flags=False)
    again = binding.hybrid_fwd(*args, scale_la=wl.scale_la, scale_sm=wl.scale_sm, ws=ws)
    torch.cuda.synchronize()
    assert binding.natsl_device_status(ws) == 0
    assert torch.equal(again["out"], first["out"])
    check_fwd(wl, run_fwd(wl, x), run_oracle(wl, x), TOL["bf16"])
