#!/usr/bin/env python
"""Benchmark of the NAtS-L hybrid attention layer on B200.

`python bench.py --gpus N --steps K --warmup W` times K forward passes of the whole hot path
(route compaction -> chunkwise Gated DeltaNet -> sparse softmax -> combination) on the bf16
prefill workload (B=4, H=16, L=4096, d=128, C=64, 10 % softmax tokens) per GPU and prints ONE
JSON line.  With N > 1 (launched by torch.distributed.run) every rank runs its own batch
(independent (batch, head) problems, no collective on the data path): weak scaling.

`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2602_03681_b200 import inputs  # noqa: E402

METRIC = "hybrid_layer_fwd_tokens_per_s"
UNIT = "tokens/s"
WORKLOAD = "cfg1_bf16_prefill"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# ------------------------------------------------------------------------------------------
# algorithmic work (counted from the realised routing masks)
# ------------------------------------------------------------------------------------------
def useful_flops(route: np.ndarray, d: int, C: int = 64):
    """Useful FLOPs of one forward, per stage, from the compacted algorithm (1 FMA = 2 FLOPs).
    GDN per chunk with n linear tokens:
      prepare: 6 n^2 d [K K^T, T(beta V), T(beta gamma K)] + 2 C n d [Q K_lin^T]
      scan   : 2 d^2 (2 n + C) [W S, K~^T U~, Q S] + 2 C n d [P U~]
    softmax per (batch, head): 4 d sum_i |{j <= i : route_j = 1}|."""
    B, L, H = route.shape
    r = route.astype(np.int64)
    n = (C - r.reshape(B, L // C, C, H).sum(2)).astype(np.float64)       # linear tokens per chunk
    prepare = float((6 * n * n * d + 2 * C * n * d).sum())
    scan = float((2 * d * d * (2 * n + C) + 2 * C * n * d).sum())
    nvis = np.cumsum(r, axis=1)
    softmax = float(4 * d * nvis.sum())
    return {"gdn_prepare": prepare, "gdn_scan": scan, "softmax_combine": softmax}


BWD_FORMULA = ("per chunk with n linear tokens, C = 64: gradient products 8 C n d [P^T dO, dO U~^T, dP K, dP^T Q] "
               "+ 8 n d^2 [K~ dS, W^T dU~, U~ dS^T, dU~ S0^T] + 4 C d^2 [(s gamma Q)^T dO, dO S0^T] "
               "+ 12 n^2 d [T^T dU, T^T dW, dU (beta V)^T, dW (beta gamma K)^T, dA K, dA^T K] + 4 n^3 [T^T dT T^T]; "
               "plus the chunkwise quantities the backward needs again: 6 n^2 d + 2 C n d [K K^T, T beta V, "
               "T beta gamma K, Q K^T] + 2 n d^2 [W S0]  (all linear: 28 C^2 d + 14 C d^2 + 4 C^3); "
               "softmax branch: 2.5 x its forward = 10 d sum_i |{j <= i : route_j = 1}| [S, dP, dV, dQ, dK]")


def useful_flops_bwd(route: np.ndarray, d: int, C: int = 64):
    """Useful FLOPs of one backward from the realised routing mask (BWD_FORMULA)."""
    B, L, H = route.shape
    r = route.astype(np.int64)
    n = (C - r.reshape(B, L // C, C, H).sum(2)).astype(np.float64)
    grad = 8 * C * n * d + 8 * n * d * d + 4 * C * d * d + 12 * n * n * d + 4 * n ** 3
    again = 6 * n * n * d + 2 * C * n * d + 2 * n * d * d
    nvis = np.cumsum(r, axis=1)
    return {"gdn_bwd": float((grad + again).sum()), "softmax_bwd": float(10 * d * nvis.sum())}


def tensor_roofline(flops, ms, peaks, peak_kind, traffic=None):
    tf = flops / (ms * 1e-3) / 1e12
    return {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
            "frac": tf / peaks["bf16_tflops"], "frac_of_nominal_2250": tf / 2250.0,
            "peak_source": peak_kind, "traffic": traffic, "useful_gflop": flops / 1e9, "ms": ms}


def useful_flops_block(route: np.ndarray, d: int, C: int = 64):
    """The same count under block-level routing: every block runs the delta rule with all C of its
    tokens, and a query in a linear block also reads the causal part of its own block."""
    B, L, H = route.shape
    r = route.astype(np.int64)
    nblk = B * (L // C) * H
    prepare = float(nblk * (6 * C * C * d + 2 * C * C * d))
    scan = float(nblk * (2 * d * d * 3 * C + 2 * C * C * d))
    own = (np.arange(L) % C + 1)[None, :, None] * (1 - r)
    softmax = float(4 * d * (np.cumsum(r, axis=1) + own).sum())
    return {"gdn_prepare": prepare, "gdn_scan": scan, "softmax_combine": softmax}


def min_hbm_bytes_fwd(wl, B):
    """q, k, v read once + out written once + the small per-token tensors."""
    e = 2 if wl.dtype == "bf16" else 4
    tok = B * wl.L * wl.H
    return tok * wl.d * e * 4 + tok * (4 + 4 + 1 + 8)


def decode_bytes_per_step(B, H, d, cache_len_mean, e=2):
    """state read + written (fp32), retained K and V read once, per (sequence, head)."""
    return B * H * (2 * d * d * 4 + 2 * cache_len_mean * d * e)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def load_traffic():
    """DRAM bytes per launch from the committed profiler summaries (profiles/traffic.txt)."""
    path = os.path.join(ROOT, "profiles", "traffic.txt")
    out = {}
    if os.path.exists(path):
        with open(path) as f:
            for line in f:
                parts = line.split("#")[0].split()
                if len(parts) >= 2 and parts[1].isdigit():
                    out[parts[0]] = int(parts[1])
    return out


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 7:
                    continue
                try:
                    sm.append(float(f[0]))
                    mx.append(float(f[1]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), f[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ------------------------------------------------------------------------------------------
# reference arm: the fp64 CPU oracle on a bounded sample
# ------------------------------------------------------------------------------------------
def oracle_sample_inputs(wl, sample_B):
    x = inputs.make_layer_inputs(wl, B=sample_B)
    return x


def time_oracle(wl, x, repeats):
    import oracle
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        oracle.hybrid_fwd(x["q"], x["k"], x["v"], x["g"], x["beta"], x["route"], x["w"],
                          scale_la=wl.scale_la, scale_sm=wl.scale_sm)
        times.append(time.perf_counter() - t0)
    return times, oracle.num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = inputs.WORKLOADS[WORKLOAD]
    sample_B = 1
    x = oracle_sample_inputs(wl, sample_B)
    time_oracle(wl, x, 1)      # page in, spin up OpenMP
    times, cores = time_oracle(wl, x, args.steps)
    total = sum(times)
    value = sample_B * wl.L * args.steps / total
    sample = f"{sample_B} of {wl.B} sequences of the workload per step (all {wl.H} heads, L={wl.L})"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "B": sample_B, "H": wl.H, "L": wl.L, "d": wl.d, "C": wl.C,
                   "p_softmax": wl.p_softmax, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2602_03681_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    binding.lib()   # fail loudly here if the CUDA library is missing

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        if world == 1:
            return x
        t = torch.tensor([x], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    wl = inputs.WORKLOADS[WORKLOAD]
    wl_rank = inputs.Workload(**{**wl.__dict__, "seed": wl.seed + 1000 * rank})
    x = inputs.make_layer_inputs(wl_rank)
    dt = torch.bfloat16
    B, L, H, d = wl.B, wl.L, wl.H, wl.d

    host = {n: torch.from_numpy(x[n]) for n in ("q", "k", "v", "g", "beta", "route", "w")}
    for n in ("q", "k", "v"):
        host[n] = host[n].to(dt)
    host = {n: t.contiguous().pin_memory() for n, t in host.items()}
    devt = {n: t.cuda() for n, t in host.items()}
    out = torch.empty((B, L, H, d), dtype=dt, device="cuda")
    out_host = torch.empty((B, L, H, d), dtype=dt).pin_memory()

    p = binding.make_params(B, H, L, d, binding.NATSL_BF16, wl.scale_la, wl.scale_sm, w=devt["w"])
    ws = binding.alloc_workspace(p, binding.OP_FWD)

    def step():
        binding.natsl_hybrid_fwd(devt["q"], devt["k"], devt["v"], devt["g"], devt["beta"],
                                 devt["route"], out, p, ws)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert binding.natsl_device_status(ws) == 0

    # ---- timed region: K steps, inputs resident in HBM ----
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = binding.natsl_launch_count()
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    launches = binding.natsl_launch_count() - launches0
    ms = max_over_ranks(e0.elapsed_time(e1))
    clocks = sampler.stop() if rank == 0 else None
    if rank == 0 and clocks["samples"] < 3:
        # The timed region is shorter than nvidia-smi's sampling period: sample the clocks over an
        # identical back-to-back run of the same step instead (untimed), and say so.
        sampler = ClockSampler(local_rank)
        sampler.start()
        t_end, extra = time.perf_counter() + 1.0, 0
        while time.perf_counter() < t_end:
            for _ in range(50):
                step()
            torch.cuda.synchronize()
            extra += 50
        clocks = sampler.stop()
        clocks["note"] = (f"timed region ({ms:.1f} ms) shorter than the sampling period; sampled "
                          f"over {extra} further identical steps run right after it")
    ms_per_step = ms / args.steps
    value = world * B * L / (ms_per_step * 1e-3)

    # ---- per-stage device times (events recorded by the library between its kernels) ----
    names = binding.stage_names(binding.OP_FWD)
    n_ev = len(names) + 1
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(n_ev)] for _ in range(args.steps)]
    for row in evs:
        for e in row:
            e.record()
    torch.cuda.synchronize()
    for row in evs:
        keep = binding.attach_stage_events(p, row)
        step()
        del keep
    p.stage_events, p.n_stage_events = None, 0
    torch.cuda.synchronize()
    stage_ms = {nm: float(np.mean([row[i].elapsed_time(row[i + 1]) for row in evs]))
                for i, nm in enumerate(names)}

    # ---- end to end: pinned host buffers -> device -> layer -> host, every step ----
    # Two steps are in flight, each on its own stream with its own device buffers and workspace, so
    # that one step's host-to-device copies overlap the other's compute and device-to-host copy (the
    # link is full duplex); every step still copies all of its inputs in and its result out.
    class Lane:
        pass

    lanes = []
    for _ in range(2):
        ln = Lane()
        ln.stream = torch.cuda.Stream()
        ln.dev = {n: torch.empty_like(t, device="cuda") for n, t in host.items()}
        ln.out = torch.empty_like(out)
        ln.out_host = torch.empty((B, L, H, d), dtype=dt).pin_memory()
        ln.p = binding.make_params(B, H, L, d, binding.NATSL_BF16, wl.scale_la, wl.scale_sm, w=ln.dev["w"])
        ln.ws = binding.alloc_workspace(ln.p, binding.OP_FWD)
        lanes.append(ln)

    def e2e_step(i):
        ln = lanes[i % 2]
        with torch.cuda.stream(ln.stream):
            for n in ln.dev:
                ln.dev[n].copy_(host[n], non_blocking=True)
            binding.natsl_hybrid_fwd(ln.dev["q"], ln.dev["k"], ln.dev["v"], ln.dev["g"], ln.dev["beta"],
                                     ln.dev["route"], ln.out, ln.p, ln.ws)
            ln.out_host.copy_(ln.out, non_blocking=True)

    def join_lanes():
        for ln in lanes:
            torch.cuda.current_stream().wait_stream(ln.stream)

    for i in range(4):
        e2e_step(i)
    join_lanes()
    barrier()
    for ln in lanes:
        assert binding.natsl_device_status(ln.ws) == 0
        assert torch.equal(ln.out_host, out.cpu())       # same inputs, same result as the resident run
        ln.stream.wait_stream(torch.cuda.current_stream())
    e0.record()
    for ln in lanes:
        ln.stream.wait_event(e0)
    for i in range(args.steps):
        e2e_step(i)
    join_lanes()
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1)) / args.steps
    h2d = sum(host[n].numel() * host[n].element_size() for n in devt)
    d2h = lanes[0].out_host.numel() * lanes[0].out_host.element_size()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel ----
    peaks, peak_kind = load_peaks()
    traffic = load_traffic()
    flops = useful_flops(x["route"], d, wl.C)
    dom = max((n for n in names if n in flops), key=lambda n: stage_ms[n])
    tf = flops[dom] / (stage_ms[dom] * 1e-3) / 1e12
    peak_tf = peaks["bf16_tflops_sustained"] if ms > 2000 else peaks["bf16_tflops"]
    roofline = {"kernel": dom, "bound": "tensor", "achieved": tf, "peak": peak_tf, "unit": "TFLOP/s",
                "frac": tf / peak_tf, "peak_source": peak_kind,
                "traffic": traffic.get(f"{dom}:{WORKLOAD}"),
                "useful_flops_per_launch": flops[dom], "ms_per_launch": stage_ms[dom]}
    total_flops = sum(flops.values())
    step_tf = total_flops / (ms_per_step * 1e-3) / 1e12

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "B_per_gpu": B, "H": H, "L": L, "d": d, "C": wl.C,
                   "p_softmax": wl.p_softmax, "sharding": "independent (batch, head) per GPU",
                   "l2": "working set (q,k,v,out + workspace) > 126 MB L2; no flush between steps"},
        "e2e": {"value": world * B * L / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "pipelining": "two steps in flight on two streams"},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": roofline,
        "stages_ms": stage_ms,
        "stages_note": ("stage times are taken in a separate pass with the library's per-stage events, "
                        "which makes it run the stages in sequence; in the timed steps the compaction "
                        "and the gather run on a side stream beside the prepare kernel, so a step is "
                        "shorter than the sum of the stages"),
        "step": {"useful_tflops": step_tf, "frac_of_bf16_peak": step_tf / peak_tf,
                 "useful_gflop": total_flops / 1e9, "min_hbm_bytes": min_hbm_bytes_fwd(wl, B),
                 "hbm_floor_ms": min_hbm_bytes_fwd(wl, B) / (peaks["hbm_gbs"] * 1e9) * 1e3},
    }

    if world == 1 and not args.no_extras:
        line["decode"] = bench_decode(args, peaks, peak_kind, traffic)
        line["other_workloads"] = bench_other_workloads(peaks, peak_kind, traffic)
    if world == 1 and not args.no_cpu:
        xs = x if args.cpu_sample_B >= B else inputs.make_layer_inputs(wl_rank, B=args.cpu_sample_B)
        sb = min(args.cpu_sample_B, B)
        times, cores = time_oracle(wl, xs, 2)
        line["cpu_baseline"] = {"value": sb * L / min(times), "unit": UNIT, "cores": cores,
                                "kind": "oracle",
                                "sample": f"{sb} of {B} sequences (all {H} heads, L={L}), best of 2"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def bench_other_workloads(peaks, peak_kind="measured", traffic=None):
    """Forward of the long-context workload and forward + backward of the training workload
    (device-resident inputs, CUDA events, best of 3 after a warm-up), with useful FLOPs."""
    import torch

    from paper_2602_03681_b200 import binding
    res = {}
    dt = torch.bfloat16
    for name, ops in (("cfg2_bf16_long_prefill", ("fwd",)), ("cfg4_bf16_train", ("fwd", "bwd")),
                      ("cfg1_bf16_prefill/block_routing", ("fwd",)),
                      ("cfg4_bf16_train/block_routing", ("fwd", "bwd"))):
        block = name.endswith("/block_routing")          # the same shapes, one route per 64 tokens
        wl = inputs.WORKLOADS[name.split("/")[0]]
        x = inputs.make_layer_inputs(
            wl, route=inputs.route_blocks(wl.seed, (wl.B, wl.L, wl.H), wl.p_softmax) if block else None)
        d = {m: torch.from_numpy(x[m]).cuda() for m in ("g", "beta", "route", "w")}
        for m in ("q", "k", "v", "dout"):
            d[m] = torch.from_numpy(x[m]).cuda().to(dt)
        ws = {"fwd": None, "bwd": None}

        def call(op):
            if op == "fwd":
                ws["fwd"] = binding.hybrid_fwd(d["q"], d["k"], d["v"], d["g"], d["beta"], d["route"],
                                               d["w"], scale_la=wl.scale_la, scale_sm=wl.scale_sm,
                                               flags=binding.BLOCK_ROUTING if block else 0,
                                               ws=ws["fwd"])["ws"]
            else:
                ws["bwd"] = binding.hybrid_bwd(d["q"], d["k"], d["v"], d["g"], d["beta"], d["route"],
                                               d["w"], d["dout"], scale_la=wl.scale_la,
                                               scale_sm=wl.scale_sm,
                                               flags=binding.BLOCK_ROUTING if block else 0,
                                               ws=ws["bwd"])["ws"]

        ms = {}
        for op in ops:
            call(op)
            torch.cuda.synchronize()
            best = float("inf")
            for _ in range(3):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                call(op)
                e1.record()
                torch.cuda.synchronize()
                best = min(best, e0.elapsed_time(e1))
            ms[op] = best
        fl = sum((useful_flops_block if block else useful_flops)(x["route"], wl.d, wl.C).values())
        total_ms = sum(ms.values())
        traffic = traffic or {}
        base = name.split("/")[0]
        entry = {"ms": ms, "tokens_per_s": wl.B * wl.L / (total_ms * 1e-3),
                 "useful_fwd_gflop": fl / 1e9,
                 "fwd_useful_tflops": fl / (ms["fwd"] * 1e-3) / 1e12,
                 "fwd_frac_of_bf16_peak": fl / (ms["fwd"] * 1e-3) / 1e12 / peaks["bf16_tflops"],
                 "roofline": {"fwd": tensor_roofline(fl, ms["fwd"], peaks, peak_kind,
                                                     None if block else traffic.get(f"fwd:{base}"))}}
        if "bwd" in ops:
            # the training step as a user runs it: forward in the backward's workspace
            # (NATSL_SAVE_FOR_BWD), then the backward from what the forward left there
            bflags = binding.BLOCK_ROUTING if block else 0
            pt = binding.make_params(wl.B, wl.H, wl.L, wl.d, binding.NATSL_BF16, wl.scale_la, wl.scale_sm,
                                     w=d["w"], flags=bflags | binding.SAVE_FOR_BWD)
            wst = binding.alloc_workspace(pt, binding.OP_BWD)
            outt = torch.empty_like(d["q"])

            def train_step():
                binding.natsl_hybrid_fwd(d["q"], d["k"], d["v"], d["g"], d["beta"], d["route"], outt, pt, wst)
                binding.hybrid_bwd(d["q"], d["k"], d["v"], d["g"], d["beta"], d["route"], d["w"], d["dout"],
                                   scale_la=wl.scale_la, scale_sm=wl.scale_sm,
                                   flags=bflags | binding.SAVED_FWD, ws=wst)

            train_step()
            torch.cuda.synchronize()
            best = float("inf")
            for _ in range(3):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                train_step()
                e1.record()
                torch.cuda.synchronize()
                best = min(best, e0.elapsed_time(e1))
            assert binding.natsl_device_status(wst) == 0
            entry["ms"]["fwd_saved+bwd"] = best
            entry["train_tokens_per_s"] = wl.B * wl.L / (best * 1e-3)
            entry["bwd_workspace_bytes"] = int(wst.numel())
            del wst, outt
        if "bwd" in ops and not block:
            fb = sum(useful_flops_bwd(x["route"], wl.d, wl.C).values())
            entry["useful_bwd_gflop"] = fb / 1e9
            entry["bwd_flop_formula"] = BWD_FORMULA
            entry["roofline"]["bwd"] = tensor_roofline(fb, ms["bwd"], peaks, peak_kind, traffic.get(f"bwd:{base}"))
            entry["roofline"]["fwd+bwd"] = tensor_roofline(fl + fb, total_ms, peaks, peak_kind)
            entry["roofline"]["fwd_saved+bwd"] = tensor_roofline(fl + fb, entry["ms"]["fwd_saved+bwd"], peaks, peak_kind)
        res[name] = entry
        del d, ws
        torch.cuda.empty_cache()
    res["grouped_heads_6x2_qk_norm"] = bench_grouped_heads(peaks, peak_kind)
    res["score_layer"] = bench_score_layer(peaks)
    res["cfg2_bf16_long_prefill/in_4_pieces"] = bench_prefill_in_pieces()
    res["serving_131072_tokens"] = bench_long_context_serving()
    return res


def bench_grouped_heads(peaks, peak_kind, B=10, H=6, G=2):
    """Forward with grouped softmax heads and in-kernel q/k normalisation (Section 4.3) on the
    smaller model's head counts (appendix: six linear heads, twelve softmax heads) at the prefill
    workload's length and head size: H = 6 linear heads of d = 128, G = 2 softmax heads of 64 each,
    L = 4096, B = 10 (60 (batch, head) pairs, close to the prefill workload's 64).  The useful FLOPs
    are those of the ungrouped layer: G heads of d / G columns do the same logit and value products."""
    import dataclasses

    import torch

    from paper_2602_03681_b200 import binding
    wl = dataclasses.replace(inputs.WORKLOADS["cfg1_bf16_prefill"], B=B, H=H, seed=5)
    x = inputs.make_layer_inputs(wl)
    d = {m: torch.from_numpy(x[m]).cuda() for m in ("g", "beta", "route", "w")}
    for m in ("q", "k", "v"):
        d[m] = torch.from_numpy(x[m]).cuda().to(torch.bfloat16)
    ms = {}
    for label, kw in (("grouped_qk_norm", dict(G=G, flags=binding.QK_NORM, norm_eps=1e-6,
                                               scale_sm=float(wl.d // G) ** -0.5)),
                      ("plain_same_shapes", dict(scale_sm=wl.scale_sm))):
        ws = None
        best = float("inf")
        for it in range(5):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ws = binding.hybrid_fwd(d["q"], d["k"], d["v"], d["g"], d["beta"], d["route"], d["w"],
                                    scale_la=wl.scale_la, ws=ws, **kw)["ws"]
            e1.record()
            torch.cuda.synchronize()
            if it >= 2:
                best = min(best, e0.elapsed_time(e1))
        assert binding.natsl_device_status(ws) == 0
        ms[label] = best
    fl = sum(useful_flops(x["route"], wl.d, wl.C).values())
    res = {"B": B, "H_linear": H, "G": G, "L": wl.L, "d": wl.d, "ms": ms,
           "tokens_per_s": B * wl.L / (ms["grouped_qk_norm"] * 1e-3), "useful_fwd_gflop": fl / 1e9,
           "roofline": {"fwd": tensor_roofline(fl, ms["grouped_qk_norm"], peaks, peak_kind)}}
    # The mode the paper's models run in -- one routing decision per block, grouped heads, normalised q, k --
    # forward and training step (forward saved in the backward's workspace, then the backward; at d = 128
    # the backward's chunk-level products are CUDA-core tile GEMMs).
    xb = inputs.make_layer_inputs(wl, route=inputs.route_blocks(wl.seed, (B, wl.L, H), wl.p_softmax))
    rb = torch.from_numpy(xb["route"]).cuda()
    dout = torch.from_numpy(xb["dout"]).cuda().to(torch.bfloat16)
    flags = binding.QK_NORM | binding.BLOCK_ROUTING
    kw = dict(G=G, norm_eps=1e-6)
    scale_sm = float(wl.d // G) ** -0.5
    pf = binding.make_params(B, H, wl.L, wl.d, binding.NATSL_BF16, wl.scale_la, scale_sm, w=d["w"],
                             flags=flags | binding.SAVE_FOR_BWD, **kw)
    pb = binding.make_params(B, H, wl.L, wl.d, binding.NATSL_BF16, wl.scale_la, scale_sm, w=d["w"],
                             flags=flags | binding.SAVED_FWD, **kw)
    wsb = binding.alloc_workspace(pf, binding.OP_BWD)
    out = torch.empty_like(d["q"])
    grads = [torch.empty_like(d["q"]) for _ in range(3)] + [torch.empty_like(d["g"]) for _ in range(2)] + \
        [torch.empty((B, wl.L, H, 2), device="cuda")]
    wsf = None

    def fwd_block():
        nonlocal wsf
        wsf = binding.hybrid_fwd(d["q"], d["k"], d["v"], d["g"], d["beta"], rb, d["w"], scale_la=wl.scale_la,
                                 scale_sm=scale_sm, flags=flags, ws=wsf, **kw)["ws"]

    def train_step():
        binding.natsl_hybrid_fwd(d["q"], d["k"], d["v"], d["g"], d["beta"], rb, out, pf, wsb)
        binding.natsl_hybrid_bwd(d["q"], d["k"], d["v"], d["g"], d["beta"], rb, dout, *grads, pb, wsb)

    for label, call in (("block_routed_fwd", fwd_block), ("block_routed_fwd_saved+bwd", train_step)):
        best = float("inf")
        for it in range(4):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            call()
            e1.record()
            torch.cuda.synchronize()
            if it >= 1:
                best = min(best, e0.elapsed_time(e1))
        ms[label] = best
    assert binding.natsl_device_status(wsb) == 0 and binding.natsl_device_status(wsf) == 0
    res["bwd_workspace_bytes"] = int(wsb.numel())
    res["train_tokens_per_s"] = B * wl.L / (ms["block_routed_fwd_saved+bwd"] * 1e-3)
    del wsb, wsf, out, grads
    torch.cuda.empty_cache()
    return res


def bench_long_context_serving(L=131072, piece=16384, decode_steps=64):
    """A long-context serving loop on the long-context workload's head shapes (B=1, H=16, d=128,
    5 % clustered softmax tokens): the prompt is prefilled in pieces (state chained, retained K/V
    appended to one cache), then tokens are generated with one decode step captured in a CUDA graph
    and replayed.  Inputs are drawn on the device (seeded); the code path is the one the parity
    tests cover at 32768 tokens."""
    import torch

    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg2_bf16_long_prefill"]
    B, H, d, dt = 1, wl.H, wl.d, torch.bfloat16
    gen = torch.Generator(device="cuda").manual_seed(wl.seed)
    route_all = inputs.route_runs(wl.seed, (B, L + decode_steps, H), wl.p_softmax)
    cap = int(route_all.sum(1).max()) + 128

    def draw(n):
        q = torch.nn.functional.normalize(torch.randn((B, n, H, d), device="cuda", generator=gen), dim=-1)
        k = torch.nn.functional.normalize(torch.randn((B, n, H, d), device="cuda", generator=gen), dim=-1)
        v = torch.randn((B, n, H, d), device="cuda", generator=gen)
        g = -torch.nn.functional.softplus(torch.randn((B, n, H), device="cuda", generator=gen) + wl.g_shift)
        beta = torch.sigmoid(torch.randn((B, n, H), device="cuda", generator=gen))
        w = torch.softmax(torch.randn((B, n, H, 2), device="cuda", generator=gen), dim=-1)
        return [q.to(dt), k.to(dt), v.to(dt), g, beta, w]

    pieces = []
    for i in range(L // piece):
        q, k, v, g, beta, w = draw(piece)
        r = torch.from_numpy(np.ascontiguousarray(route_all[:, i * piece:(i + 1) * piece])).cuda()
        pieces.append([q, k, v, g, beta, r, w])
    cache = (torch.zeros((B, H, cap, d), dtype=dt, device="cuda"),
             torch.zeros((B, H, cap, d), dtype=dt, device="cuda"),
             torch.zeros((B, H), dtype=torch.int32, device="cuda"))
    ws = [None]
    state = [None]

    def prefill():
        cache[2].zero_()
        st = None
        for a in pieces:
            r = binding.hybrid_fwd(*a, scale_la=wl.scale_la, scale_sm=wl.scale_sm, state_in=st,
                                   want=("state_out",), cache=cache, flags=binding.APPEND_CACHE, ws=ws[0])
            st, ws[0] = r["state_out"], r["ws"]
        state[0] = st

    prefill()
    torch.cuda.synchronize()
    best = float("inf")
    for _ in range(2):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        prefill()
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    assert binding.natsl_device_status(ws[0]) == 0
    # generation: one captured step, replayed; per-step inputs are copied into its static buffers
    tq, tk, tv, tg, tb, tw = draw(decode_steps)
    troute = torch.from_numpy(np.ascontiguousarray(route_all[:, L:])).cuda()
    sq, sk, sv = (torch.zeros((B, H, d), dtype=dt, device="cuda") for _ in range(3))
    sg, sb = torch.zeros((B, H), device="cuda"), torch.zeros((B, H), device="cuda")
    sr = torch.zeros((B, H), dtype=torch.uint8, device="cuda")
    sw = torch.zeros((B, H, 2), device="cuda")
    out = torch.zeros((B, H, d), dtype=dt, device="cuda")
    p = binding.make_params(B, H, 0, d, binding.NATSL_BF16, wl.scale_la, wl.scale_sm, w=sw)
    dws = binding.alloc_workspace(p, binding.OP_DECODE)
    st, n = state[0], cache[2]

    def load(t):
        sq.copy_(tq[:, t]); sk.copy_(tk[:, t]); sv.copy_(tv[:, t])
        sg.copy_(tg[:, t]); sb.copy_(tb[:, t]); sr.copy_(troute[:, t]); sw.copy_(tw[:, t])

    load(0)
    binding.natsl_decode_step(sq, sk, sv, sg, sb, sr, st, cache[0], cache[1], n, out, p, dws)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.natsl_decode_step(sq, sk, sv, sg, sb, sr, st, cache[0], cache[1], n, out, p, dws)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(1, decode_steps):
        load(t)
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    assert binding.natsl_device_status(dws) == 0
    return {"prompt_tokens": L, "pieces": L // piece, "prefill_ms": best,
            "prefill_tokens_per_s": L / (best * 1e-3), "retained_per_head_max": cap - 128,
            "decode_ms_per_token": e0.elapsed_time(e1) / (decode_steps - 1),
            "decode": "one step captured in a CUDA graph, replayed; includes the copies of the step's inputs"}


def bench_prefill_in_pieces(n_pieces=4):
    """The long-context workload prefilled piece by piece: state chained through state_in /
    state_out, retained K/V appended to one cache (device-resident inputs, best of 3)."""
    import torch

    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg2_bf16_long_prefill"]
    x = inputs.make_layer_inputs(wl)
    n = wl.L // n_pieces
    dt = torch.bfloat16
    pieces = []
    for i in range(n_pieces):
        sl = slice(i * n, (i + 1) * n)
        pieces.append([torch.from_numpy(np.ascontiguousarray(x[m][:, sl])).cuda().to(dt) for m in ("q", "k", "v")] +
                      [torch.from_numpy(np.ascontiguousarray(x[m][:, sl])).cuda() for m in ("g", "beta", "route", "w")])
    cap = int(x["route"].sum(1).max()) + 128
    cache = (torch.zeros((wl.B, wl.H, cap, wl.d), dtype=dt, device="cuda"),
             torch.zeros((wl.B, wl.H, cap, wl.d), dtype=dt, device="cuda"),
             torch.zeros((wl.B, wl.H), dtype=torch.int32, device="cuda"))
    ws = [None]

    def run():
        cache[2].zero_()
        state = None
        for a in pieces:
            r = binding.hybrid_fwd(*a, scale_la=wl.scale_la, scale_sm=wl.scale_sm, state_in=state,
                                   want=("state_out",), cache=cache, flags=binding.APPEND_CACHE, ws=ws[0])
            state, ws[0] = r["state_out"], r["ws"]

    run()
    torch.cuda.synchronize()
    best = float("inf")
    for _ in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        run()
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    assert binding.natsl_device_status(ws[0]) == 0
    return {"ms": best, "pieces": n_pieces, "tokens_per_s": wl.B * wl.L / (best * 1e-3), "cache_rows": cap}


def bench_score_layer(peaks):
    """The attention score layer on the prefill shapes (d_model = H d): HBM-bound, X is read once."""
    import torch

    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg1_bf16_prefill"]
    Dm = wl.H * wl.d
    gen = torch.Generator(device="cuda").manual_seed(wl.seed)
    reps = 6                               # distinct inputs in turn: 6 x 67 MB > L2
    xs = [torch.randn((wl.B, wl.L, Dm), device="cuda", generator=gen).to(torch.bfloat16) for _ in range(reps)]
    w = torch.randn((wl.H, 2, Dm), device="cuda", generator=gen) / Dm ** 0.5
    route = torch.empty((wl.B, wl.L, wl.H), dtype=torch.uint8, device="cuda")
    p = binding.make_params(wl.B, wl.H, wl.L, wl.d, binding.NATSL_BF16, 1.0, 1.0)
    for x in xs[:3]:
        binding.natsl_score_layer(x, w, None, route, p)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n = 4 * reps
    e0.record()
    for i in range(n):
        binding.natsl_score_layer(xs[i % reps], w, None, route, p)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / n
    nbytes = wl.B * wl.L * Dm * 2 + wl.B * wl.L * wl.H
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"ms": ms, "d_model": Dm, "algorithmic_bytes": nbytes, "achieved_gbs": gbs,
            "frac_of_hbm_peak": gbs / peaks["hbm_gbs"]}


def bench_decode(args, peaks, peak_kind, traffic):
    """Decode workload: batch 64, H=16, d=128, 256 steps, 1638 retained tokens per cache."""
    import torch

    from paper_2602_03681_b200 import binding
    wl = inputs.WORKLOADS["cfg3_bf16_decode"]
    B, H, d, T = wl.B, wl.H, wl.d, wl.L
    x = inputs.make_decode_inputs(wl)
    dt = torch.bfloat16
    state0 = torch.from_numpy(x["state"]).cuda()
    state = state0.clone()
    kc = torch.from_numpy(x["k_cache"]).to(dt).cuda()
    vc = torch.from_numpy(x["v_cache"]).to(dt).cuda()
    n0 = torch.from_numpy(x["cache_len"]).cuda()
    n = n0.clone()
    tok = {m: torch.from_numpy(x[m]).cuda() for m in ("g", "beta", "route", "w")}
    for m in ("q", "k", "v"):
        tok[m] = torch.from_numpy(x[m]).to(dt).cuda()
    out = torch.empty((T, B, H, d), dtype=dt, device="cuda")
    p = binding.make_params(B, H, 0, d, binding.NATSL_BF16, wl.scale_la, wl.scale_sm)
    ws = binding.alloc_workspace(p, binding.OP_DECODE)

    def trajectory():
        for t in range(T):
            p.w = tok["w"][t].data_ptr()
            binding.natsl_decode_step(tok["q"][t], tok["k"][t], tok["v"][t], tok["g"][t],
                                      tok["beta"][t], tok["route"][t], state, kc, vc, n, out[t], p, ws)

    times = []
    for rep in range(3):
        state.copy_(state0)
        n.copy_(n0)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        trajectory()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    assert binding.natsl_device_status(ws) == 0
    ms = min(times[1:])
    mean_len = float(x["cache_len"].mean()) + 0.5 * float(x["route"].mean()) * T
    bytes_step = decode_bytes_per_step(B, H, d, mean_len)
    gbs = bytes_step / (ms / T * 1e-3) / 1e9
    # the same trajectory with two softmax heads per linear head and q, k normalised inside the kernel
    # (Section 4.3): same bytes, more arithmetic per cached key
    p = binding.make_params(B, H, 0, d, binding.NATSL_BF16, wl.scale_la, float(d // 2) ** -0.5,
                            flags=binding.QK_NORM, G=2, norm_eps=1e-6)
    ms_grouped = float("inf")
    for rep in range(2):          # (the first repetition loads the kernel)
        state.copy_(state0)
        n.copy_(n0)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        trajectory()
        e1.record()
        torch.cuda.synchronize()
        if rep:
            ms_grouped = e0.elapsed_time(e1)
    assert binding.natsl_device_status(ws) == 0
    return {"workload": wl.name, "value": B * T / (ms * 1e-3), "unit": "tokens/s",
            "ms_per_step": ms / T, "steps": T,
            "grouped_heads_G2_qk_norm": {"ms_per_step": ms_grouped / T,
                                         "frac_of_hbm_peak": bytes_step / (ms_grouped / T * 1e-3) / 1e9 / peaks["hbm_gbs"]},
            "roofline": {"kernel": "decode_step", "bound": "hbm", "achieved": gbs,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                         "peak_source": peak_kind, "algorithmic_bytes_per_launch": bytes_step,
                         "traffic": traffic.get(f"decode_step:{wl.name}")}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the decode workload")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--cpu-sample-B", type=int, default=4)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
