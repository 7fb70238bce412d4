"""Run one operation of the library a few times on a chosen (possibly reduced) workload.

Meant to be the command a profiler wraps: it draws the seeded synthetic inputs, runs `--iters`
calls of `--op` on the current device and exits.  Nothing is timed or checked here.

    python -m paper_2602_03681_b200.profile_case --op fwd --workload cfg1_bf16_prefill --B 1
    python -m paper_2602_03681_b200.profile_case --op decode --workload cfg3_bf16_decode --B 8 --iters 4
    python -m paper_2602_03681_b200.profile_case --op bwd --workload cfg4_bf16_train --B 1
    python -m paper_2602_03681_b200.profile_case --op fwd --flags 4        (block-level routing)
    python -m paper_2602_03681_b200.profile_case --op score --iters 6      (attention score layer)
    python -m paper_2602_03681_b200.profile_case --op train --workload cfg1_bf16_prefill --B 10 --H 6 --G 2 \
        --qk-norm --flags 4        (six linear x twelve softmax heads, normalised q, k, one route per block)
"""
from __future__ import annotations

import argparse

import torch

from . import binding, inputs


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", choices=["fwd", "bwd", "train", "decode", "score"], default="fwd",
                    help="train: forward with NATSL_SAVE_FOR_BWD, then the backward from what it saved")
    ap.add_argument("--workload", default=None, choices=sorted(inputs.WORKLOADS),
                    help="default: the workload that belongs to --op")
    ap.add_argument("--B", type=int, default=None, help="batch override (smaller case)")
    ap.add_argument("--L", type=int, default=None, help="sequence length override")
    ap.add_argument("--H", type=int, default=None, help="(linear) head count override")
    ap.add_argument("--G", type=int, default=0, help="softmax heads per linear head (fwd, bwd, train)")
    ap.add_argument("--qk-norm", action="store_true", help="NATSL_QK_NORM with norm_eps 1e-6; scale_sm = (d/G)^-1/2")
    ap.add_argument("--iters", type=int, default=2)
    ap.add_argument("--flags", type=int, default=0)
    ap.add_argument("--report", action="store_true", help="print CUDA-event time of each call")
    ap.add_argument("--stream", action="store_true", help="run on a stream of its own, not the default stream")
    args = ap.parse_args()
    if args.workload is None:
        args.workload = {"fwd": "cfg1_bf16_prefill", "bwd": "cfg4_bf16_train", "train": "cfg4_bf16_train",
                         "decode": "cfg3_bf16_decode", "score": "cfg1_bf16_prefill"}[args.op]
    if (inputs.WORKLOADS[args.workload].call == "decode") != (args.op == "decode"):
        ap.error(f"workload {args.workload} does not belong to --op {args.op}")

    wl = inputs.WORKLOADS[args.workload]
    dt = torch.float32 if wl.dtype == "f32" else torch.bfloat16
    code = binding.NATSL_F32 if wl.dtype == "f32" else binding.NATSL_BF16
    torch.cuda.set_device(0)
    binding.lib()
    if args.stream:
        torch.cuda.set_stream(torch.cuda.Stream())

    def dev(a, t=None):
        x = torch.from_numpy(a).cuda()
        return x if t is None else x.to(t)

    events = []

    def timed(call):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        call()
        e1.record()
        events.append((e0, e1))

    def finish(note=""):
        torch.cuda.synchronize()
        if args.report:
            print(f"{args.op} {args.workload}: ms per call",
                  [round(a.elapsed_time(b), 4) for a, b in events], note)

    if args.op == "score":      # the attention score layer on the workload's shapes, d_model = H d
        B, L, Dm = args.B or wl.B, args.L or wl.L, wl.H * wl.d
        gen = torch.Generator(device="cuda").manual_seed(wl.seed)
        xs = [torch.randn((B, L, Dm), device="cuda", generator=gen).to(dt) for _ in range(3)]
        w = torch.randn((wl.H, 2, Dm), device="cuda", generator=gen) / Dm ** 0.5
        route = torch.empty((B, L, wl.H), dtype=torch.uint8, device="cuda")
        p = binding.make_params(B, wl.H, L, wl.d, code, 1.0, 1.0)
        for i in range(args.iters):
            timed(lambda: binding.natsl_score_layer(xs[i % 3], w, None, route, p))
        finish()
        return

    if args.op == "decode":
        B = args.B or wl.B
        x = inputs.make_decode_inputs(wl, B=B, steps=args.iters)
        state, n = dev(x["state"]), dev(x["cache_len"])
        kc, vc = dev(x["k_cache"], dt), dev(x["v_cache"], dt)
        p = binding.make_params(B, wl.H, 0, wl.d, code, wl.scale_la,
                                float(wl.d // max(args.G, 1)) ** -0.5 if args.qk_norm else wl.scale_sm,
                                flags=args.flags | (binding.QK_NORM if args.qk_norm else 0), G=args.G,
                                norm_eps=1e-6 if args.qk_norm else 0.0)
        ws = binding.alloc_workspace(p, binding.OP_DECODE)
        out = torch.empty((B, wl.H, wl.d), dtype=dt, device="cuda")
        tok = {m: dev(x[m], dt if m in ("q", "k", "v") else None)
               for m in ("q", "k", "v", "g", "beta", "route", "w")}
        for t in range(args.iters):
            p.w = tok["w"][t].data_ptr()
            timed(lambda: binding.natsl_decode_step(
                tok["q"][t], tok["k"][t], tok["v"][t], tok["g"][t], tok["beta"][t],
                tok["route"][t], state, kc, vc, n, out, p, ws))
        finish(f"cache_len {int(n.min())}..{int(n.max())}")
        return

    kw = {}
    if args.B:
        kw["B"] = args.B
    if args.L:
        kw["L"] = args.L
    if args.H:
        kw["H"] = args.H
    gflags = args.flags | (binding.QK_NORM if args.qk_norm else 0)
    gkw = dict(G=args.G, norm_eps=1e-6 if args.qk_norm else 0.0)
    scale_sm = float(wl.d // max(args.G, 1)) ** -0.5 if args.qk_norm else wl.scale_sm
    if args.op in ("fwd", "bwd", "train") and args.flags & binding.BLOCK_ROUTING:   # one route per block of 64 tokens
        kw["route"] = inputs.route_blocks(wl.seed, (kw.get("B", wl.B), kw.get("L", wl.L), kw.get("H", wl.H)),
                                          wl.p_softmax)
    x = inputs.make_layer_inputs(wl, **kw)
    q, k, v = (dev(x[m], dt) for m in ("q", "k", "v"))
    g, beta, route, w = (dev(x[m]) for m in ("g", "beta", "route", "w"))
    if args.op == "fwd":
        ws = None
        for _ in range(args.iters):
            def call():
                nonlocal ws
                ws = binding.hybrid_fwd(q, k, v, g, beta, route, w, scale_la=wl.scale_la,
                                        scale_sm=scale_sm, flags=gflags, ws=ws, **gkw)["ws"]
            timed(call)
    elif args.op == "train":
        dout = dev(x["dout"], dt)
        B, L, H, d = q.shape
        p = binding.make_params(B, H, L, d, code, wl.scale_la, scale_sm, w=w,
                                flags=gflags | binding.SAVE_FOR_BWD, **gkw)
        pb = binding.make_params(B, H, L, d, code, wl.scale_la, scale_sm, w=w,
                                 flags=gflags | binding.SAVED_FWD, **gkw)
        ws = binding.alloc_workspace(p, binding.OP_BWD)
        out = torch.empty_like(q)
        grads = [torch.empty_like(q) for _ in range(3)] + [torch.empty_like(g) for _ in range(2)] + \
            [torch.empty((B, L, H, 2), dtype=torch.float32, device="cuda")]
        for _ in range(args.iters):
            def call():
                binding.natsl_hybrid_fwd(q, k, v, g, beta, route, out, p, ws)
                binding.natsl_hybrid_bwd(q, k, v, g, beta, route, dout, *grads, pb, ws)
            timed(call)
    else:
        dout = dev(x["dout"], dt)
        ws = None
        for _ in range(args.iters):
            def call():
                nonlocal ws
                ws = binding.hybrid_bwd(q, k, v, g, beta, route, w, dout, scale_la=wl.scale_la,
                                        scale_sm=wl.scale_sm, flags=args.flags, ws=ws)["ws"]
            timed(call)
    finish()


if __name__ == "__main__":
    main()
