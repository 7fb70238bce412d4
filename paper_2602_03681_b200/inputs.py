"""Seeded synthetic inputs for the hybrid layer -- shared by the tests, the oracle legs and
the benchmark.  This module holds NONE of the method's arithmetic: it only draws tensors
with the shapes, value distributions and routing structure of the five benchmark
workloads, from numpy's counter-based Philox generator (one sub-stream per tensor, so a
tensor's bits do not depend on which other tensors were drawn).

All floating tensors are returned as float32 numpy arrays.  For the bf16 workloads q, k, v
(and dout, cache K/V) are rounded to bf16 (round-to-nearest-even) and widened back, so the
CPU oracle and the GPU library consume exactly the same values.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

_STREAMS = dict(q=1, k=2, v=3, g=4, beta=5, route=6, w=7, dout=8, state=9, kc=10, vc=11, steps=12)


@dataclass(frozen=True)
class Workload:
    name: str
    call: str                  # "fwd" | "decode" | "fwd_bwd"
    B: int
    H: int
    L: int                     # sequence length (decode: number of steps)
    d: int
    C: int = 64
    dtype: str = "bf16"        # storage type of q,k,v,out: "f32" | "bf16"
    p_softmax: float = 0.1
    routing: str = "bernoulli"  # "bernoulli" | "runs"
    g_shift: float = 0.0       # g = -softplus(N(g_shift, 1))
    seed: int = 0
    ctx_retained: int = 0      # decode: retained tokens already in the cache
    extra: dict = field(default_factory=dict)

    @property
    def scale_la(self) -> float:
        return float(self.d) ** -0.5

    @property
    def scale_sm(self) -> float:
        # unit-norm q,k: sqrt(d) * (q.k) equals (1/sqrt(d)) * RMSnorm(q).RMSnorm(k)
        return float(self.d) ** 0.5


WORKLOADS = {
    "cfg0_f32_tiny_fwd": Workload("cfg0_f32_tiny_fwd", "fwd", 1, 2, 256, 64, dtype="f32",
                                  p_softmax=0.25, seed=0),
    "cfg1_bf16_prefill": Workload("cfg1_bf16_prefill", "fwd", 4, 16, 4096, 128, p_softmax=0.10,
                                  seed=1),
    "cfg2_bf16_long_prefill": Workload("cfg2_bf16_long_prefill", "fwd", 1, 16, 32768, 128,
                                       p_softmax=0.05, routing="runs", g_shift=-2.0, seed=2),
    "cfg3_bf16_decode": Workload("cfg3_bf16_decode", "decode", 64, 16, 256, 128, p_softmax=0.10,
                                 seed=3, ctx_retained=1638),
    "cfg4_bf16_train": Workload("cfg4_bf16_train", "fwd_bwd", 8, 12, 2048, 64, p_softmax=0.20,
                                seed=4),
}


def _rng(seed: int, stream: str) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, _STREAMS[stream]]))


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bf16 (ties to even) and return it widened to float32."""
    x = np.ascontiguousarray(x, np.float32)
    u = x.view(np.uint32)                       # finite inputs: the add below cannot wrap
    r = (u >> np.uint32(16)) & np.uint32(1)
    r += np.uint32(0x7FFF)
    r += u
    r &= np.uint32(0xFFFF0000)
    return r.view(np.float32).reshape(x.shape)


def _normal(seed, stream, shape):
    return _rng(seed, stream).standard_normal(shape, dtype=np.float32)


def _unit_rows(x):
    n = np.sqrt((x.astype(np.float64) ** 2).sum(-1, keepdims=True))
    return (x / n).astype(np.float32)


def _softplus(x):
    x = x.astype(np.float64)
    return np.where(x > 30, x, np.log1p(np.exp(np.minimum(x, 30))))


def route_bernoulli(seed, shape, p, force_first=True):
    """Independent Bernoulli(p) per (token, head); 1 = softmax.  shape = (B, L, H)."""
    r = (_rng(seed, "route").random(shape) < p).astype(np.uint8)
    if force_first and shape[1] > 0:
        r[:, 0, :] = 1
    return r


def route_runs(seed, shape, p, mean_run=8.0):
    """Clustered softmax tokens: alternating runs of 1s (geometric, mean `mean_run`) and gaps of
    0s (geometric, mean chosen so the long-run fraction of 1s is p), starting with a run at token
    0, drawn independently per (batch, head)."""
    B, L, H = shape
    rng = _rng(seed, "route")
    mean_gap = mean_run * (1.0 - p) / p
    r = np.zeros(shape, np.uint8)
    for b in range(B):
        for h in range(H):
            pos = 0
            while pos < L:
                run = int(rng.geometric(1.0 / mean_run))
                r[b, pos:pos + run, h] = 1
                pos += run
                pos += int(rng.geometric(1.0 / mean_gap))
    return r


def route_blocks(seed, shape, p, R=64, force_first=True):
    """One Bernoulli(p) decision per block of R tokens and head (block-level routing: the paper's
    chunk size equals the GDN chunk size), repeated over the block's tokens.  shape = (B, L, H)."""
    B, L, H = shape
    assert L % R == 0
    r = (_rng(seed, "route").random((B, L // R, H)) < p).astype(np.uint8)
    if force_first and L > 0:
        r[:, 0, :] = 1
    return np.repeat(r, R, axis=1)


def make_layer_inputs(wl: Workload, *, B=None, H=None, L=None, route=None):
    """Inputs of one forward (and backward) call.  B/H/L override the workload's sizes to get
    smaller cases with the same distributions.  Returns a dict of numpy arrays:
    q,k,v [B,L,H,d] f32 (bf16-representable for bf16 workloads); g,beta [B,L,H] f32;
    route [B,L,H] u8; w [B,L,H,2] f32; dout [B,L,H,d] f32."""
    B = wl.B if B is None else B
    H = wl.H if H is None else H
    L = wl.L if L is None else L
    d, s = wl.d, wl.seed
    q = _unit_rows(_normal(s, "q", (B, L, H, d)))
    k = _unit_rows(_normal(s, "k", (B, L, H, d)))
    v = _normal(s, "v", (B, L, H, d))
    g = (-_softplus(_normal(s, "g", (B, L, H)) + wl.g_shift)).astype(np.float32)
    beta = (1.0 / (1.0 + np.exp(-_normal(s, "beta", (B, L, H)).astype(np.float64)))).astype(
        np.float32)
    wz = _normal(s, "w", (B, L, H, 2)).astype(np.float64)
    wz = np.exp(wz - wz.max(-1, keepdims=True))
    w = (wz / wz.sum(-1, keepdims=True)).astype(np.float32)
    dout = _normal(s, "dout", (B, L, H, d))
    if route is None:
        if wl.routing == "runs":
            route = route_runs(s, (B, L, H), wl.p_softmax)
        else:
            route = route_bernoulli(s, (B, L, H), wl.p_softmax)
    if wl.dtype == "bf16":
        q, k, v, dout = (round_bf16(a) for a in (q, k, v, dout))
    return dict(q=q, k=k, v=v, g=g, beta=beta, route=np.ascontiguousarray(route, np.uint8), w=w,
                dout=dout)


def make_decode_inputs(wl: Workload, *, B=None, H=None, steps=None, ctx_retained=None, cap=None):
    """Initial decode state and the per-step token stream.
    state [B,H,d,d] f32 ~ N(0, 0.02^2); k_cache,v_cache [B,H,cap,d] ~ N(0,1) for the first
    `ctx_retained` rows (zeros after); cache_len [B,H] i32; per step: q,k,v [T,B,H,d];
    g,beta [T,B,H]; route [T,B,H] u8 ~ Bernoulli(p); w [T,B,H,2]."""
    B = wl.B if B is None else B
    H = wl.H if H is None else H
    T = wl.L if steps is None else steps
    n0 = wl.ctx_retained if ctx_retained is None else ctx_retained
    cap = (n0 + T) if cap is None else cap
    d, s = wl.d, wl.seed
    state = (0.02 * _normal(s, "state", (B, H, d, d))).astype(np.float32)
    kc = np.zeros((B, H, cap, d), np.float32)
    vc = np.zeros((B, H, cap, d), np.float32)
    kc[:, :, :n0] = _normal(s, "kc", (B, H, n0, d))
    vc[:, :, :n0] = _normal(s, "vc", (B, H, n0, d))
    cache_len = np.full((B, H), n0, np.int32)
    q = _unit_rows(_normal(s, "q", (T, B, H, d)))
    k = _unit_rows(_normal(s, "k", (T, B, H, d)))
    v = _normal(s, "v", (T, B, H, d))
    g = (-_softplus(_normal(s, "g", (T, B, H)) + wl.g_shift)).astype(np.float32)
    beta = (1.0 / (1.0 + np.exp(-_normal(s, "beta", (T, B, H)).astype(np.float64)))).astype(
        np.float32)
    wz = _normal(s, "w", (T, B, H, 2)).astype(np.float64)
    wz = np.exp(wz - wz.max(-1, keepdims=True))
    w = (wz / wz.sum(-1, keepdims=True)).astype(np.float32)
    route = (_rng(s, "steps").random((T, B, H)) < wl.p_softmax).astype(np.uint8)
    if wl.dtype == "bf16":
        q, k, v, kc, vc = (round_bf16(a) for a in (q, k, v, kc, vc))
    return dict(state=state, k_cache=kc, v_cache=vc, cache_len=cache_len, q=q, k=k, v=v, g=g,
                beta=beta, route=route, w=w)
