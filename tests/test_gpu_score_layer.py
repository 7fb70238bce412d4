"""Parity of the attention score layer (Section 4.1: mean pooling, linear map, arg max per chunk
and head) with the fp64 oracle, through the C ABI, and its use as the route of a block-routed
forward."""
import numpy as np
import pytest
import torch

import oracle
from oracle import router
from paper_2602_03681_b200 import inputs
from test_gpu_parity import check_fwd, dev, rel_err, run_fwd

pytestmark = pytest.mark.gpu


def features(seed, B, L, Dm, H, bf16):
    r = np.random.default_rng(seed)
    x = r.standard_normal((B, L, Dm)).astype(np.float32)
    if bf16:
        x = inputs.round_bf16(x)
    w = (r.standard_normal((H, 2, Dm)) / np.sqrt(Dm)).astype(np.float32)
    return x, w


def run_score_layer(x, w, H, bf16, want_scores=True):
    from paper_2602_03681_b200 import binding
    B, L, Dm = x.shape
    p = binding.make_params(B, H, L, 64, binding.NATSL_BF16 if bf16 else binding.NATSL_F32, 1.0, 1.0)
    scores = torch.zeros((B, L // 64, H, 2), device="cuda") if want_scores else None
    route = torch.full((B, L, H), 9, dtype=torch.uint8, device="cuda")
    binding.natsl_score_layer(dev(x, torch.bfloat16 if bf16 else None), dev(w), scores, route, p)
    torch.cuda.synchronize()
    return (scores.cpu().numpy() if want_scores else None), route.cpu().numpy()


@pytest.mark.parametrize("B,L,Dm,H,bf16", [(2, 256, 512, 4, True), (1, 64, 8, 1, True),
                                           (3, 640, 2048, 16, True), (2, 192, 1032, 3, True),
                                           (2, 128, 260, 5, False), (1, 4096, 1024, 12, False),
                                           # several column pieces per thread, the last one ragged; rows too
                                           # wide for the deep ring of staged rows, and for any ring
                                           (1, 192, 1544, 3, False), (1, 128, 4616, 2, True),
                                           (1, 192, 16896, 2, True)])
def test_score_layer_matches_oracle(B, L, Dm, H, bf16):
    x, w = features(B * L + Dm, B, L, Dm, H, bf16)
    ref = router.score_layer(x, w, 64)
    scores, route = run_score_layer(x, w, H, bf16)
    rms = np.sqrt((ref["scores"] ** 2).mean())
    assert np.abs(scores - ref["scores"]).max() <= 1e-4 * rms          # fp32 arithmetic
    # the decision is taken on the kernel's own fp32 scores: first maximum, linear on a tie
    assert np.array_equal(route[:, ::64], np.argmax(scores, -1).astype(np.uint8))
    assert np.array_equal(route, np.repeat(route[:, ::64], 64, axis=1))  # constant per chunk
    # and it is the oracle's wherever the oracle's margin exceeds the tolerance
    clear = np.abs(ref["scores"][..., 1] - ref["scores"][..., 0]) > 2e-4 * rms
    assert clear.mean() > 0.9
    assert np.array_equal(route[:, ::64][clear], ref["route"][:, ::64][clear])


def test_score_layer_tie_goes_to_linear_and_scores_are_optional():
    x, w = features(3, 1, 128, 64, 2, True)
    w[:, 1] = w[:, 0]                                       # identical rows: exact ties
    scores, route = run_score_layer(x, w, 2, True)
    assert np.array_equal(scores[..., 0], scores[..., 1]) and not route.any()
    w[:, 1] = w[:, 0] + 1.0
    x[:] = 0.25                                             # pooled = 0.25: softmax row wins by 16
    _, route = run_score_layer(x, w, 2, True, want_scores=False)
    assert route.all()


def test_score_layer_rejects_bad_shapes():
    from paper_2602_03681_b200 import binding
    p = binding.make_params(1, 2, 128, 64, binding.NATSL_BF16, 1.0, 1.0)
    x = torch.zeros((1, 128, 12), dtype=torch.bfloat16, device="cuda")    # 12 % 8 != 0
    w = torch.zeros((2, 2, 12), device="cuda")
    route = torch.zeros((1, 128, 2), dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.NatslError) as e:
        binding.natsl_score_layer(x, w, None, route, p)
    assert e.value.status == -2


def test_score_layer_feeds_the_block_routed_forward():
    """Scores -> route on the device, then the block-routed forward with that route; the oracle
    takes the same route (the arg max itself is checked above)."""
    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    B, H, L = 1, 4, 512
    x, w = features(11, B, L, H * wl.d, H, True)
    _, route = run_score_layer(x, w, H, True)
    assert 0 < route.mean() < 1
    y = inputs.make_layer_inputs(wl, B=B, H=H, L=L, route=route)
    got = run_fwd(wl, y, flags=binding.BLOCK_ROUTING)
    ref = oracle.hybrid_fwd(y["q"], y["k"], y["v"], y["g"], y["beta"], y["route"], y["w"],
                            scale_la=wl.scale_la, scale_sm=wl.scale_sm, block=64)
    check_fwd(wl, got, ref, 2e-2)
