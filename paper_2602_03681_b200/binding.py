"""Thin ctypes binding of ``libnatsl.so`` -- same names as the C ABI (``include/natsl.h``).

Argument marshalling only: torch supplies device memory and streams, every step of the path
runs in the library's CUDA kernels.  There is no fallback of any kind: if the library is not
built, importing the entry points raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnatsl.so")

NATSL_F32, NATSL_BF16 = 0, 1
OP_FWD, OP_BWD, OP_DECODE, OP_COMPACT = 0, 1, 2, 3
FORCE_SIMT = 1
SINGLE_PASS_SCAN = 2
BLOCK_ROUTING = 4
APPEND_CACHE = 8
SINGLE_STREAM = 16
SAVE_FOR_BWD = 32
SAVED_FWD = 64
QK_NORM = 128
ERR_CACHE_FULL = -7
ERR_UNSUPPORTED = -8
ERR_ROUTE = -11

EXPORTS = ["natsl_workspace_size", "natsl_route_compact", "natsl_hybrid_fwd", "natsl_hybrid_bwd",
           "natsl_decode_step", "natsl_decode_block_end", "natsl_device_status", "natsl_hybrid_fwd_static",
           "natsl_score_layer", "natsl_static_status", "natsl_debug_set_wait_limit",
           "natsl_stage_name", "natsl_launch_count", "natsl_strerror"]
ERR_TIMEOUT = -10
ERR_TOO_LARGE = -9
STATIC_WS_BYTES = 32 << 20


class NatslError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"natsl status {status}: {msg}")
        self.status = status


class natsl_params(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("L", ctypes.c_int32),
                ("d", ctypes.c_int32), ("C", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("scale_la", ctypes.c_float), ("scale_sm", ctypes.c_float),
                ("eps", ctypes.c_float), ("flags", ctypes.c_uint32),
                ("w", ctypes.c_void_p), ("state_in", ctypes.c_void_p),
                ("state_out", ctypes.c_void_p), ("o_la", ctypes.c_void_p),
                ("o_nla", ctypes.c_void_p), ("lse", ctypes.c_void_p), ("k_sm", ctypes.c_void_p),
                ("v_sm", ctypes.c_void_p), ("sm_len", ctypes.c_void_p),
                ("sm_cap", ctypes.c_int32), ("stage_events", ctypes.c_void_p),
                ("n_stage_events", ctypes.c_int32), ("dstate_out", ctypes.c_void_p),
                ("dstate_in", ctypes.c_void_p), ("dscore", ctypes.c_void_p),
                ("G", ctypes.c_int32), ("norm_eps", ctypes.c_float)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library; raise loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2602_03681_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        _lib = ctypes.CDLL(LIB_PATH)
        _lib.natsl_strerror.restype = ctypes.c_char_p
        _lib.natsl_strerror.argtypes = [ctypes.c_int]
        _lib.natsl_stage_name.restype = ctypes.c_char_p
        _lib.natsl_stage_name.argtypes = [ctypes.c_int, ctypes.c_int]
        _lib.natsl_launch_count.restype = ctypes.c_uint64
        for name in EXPORTS[:7] + ["natsl_score_layer", "natsl_static_status"]:
            getattr(_lib, name).restype = ctypes.c_int
        _lib.natsl_debug_set_wait_limit.restype = None
        _lib.natsl_debug_set_wait_limit.argtypes = [ctypes.c_uint32, ctypes.c_int]
    return _lib


def natsl_strerror(status: int) -> str:
    return lib().natsl_strerror(int(status)).decode()


def natsl_stage_name(op: int, i: int):
    s = lib().natsl_stage_name(op, i)
    return None if s is None else s.decode()


def natsl_launch_count() -> int:
    return int(lib().natsl_launch_count())


def stage_names(op: int):
    names, i = [], 0
    while natsl_stage_name(op, i) is not None:
        names.append(natsl_stage_name(op, i))
        i += 1
    return names


def attach_stage_events(p, events):
    """Point p.stage_events at a list of recorded-once torch.cuda.Event(enable_timing=True).
    Returns the ctypes array, which the caller must keep alive while `p` is used."""
    arr = (ctypes.c_void_p * len(events))(*[ctypes.c_void_p(e.cuda_event) for e in events])
    p.stage_events = ctypes.cast(arr, ctypes.c_void_p).value
    p.n_stage_events = len(events)
    return arr


def _check(rc: int):
    if rc != 0:
        raise NatslError(rc, natsl_strerror(rc))


def _ptr(t):
    if t is None:
        return ctypes.c_void_p(0)
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensors only"
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype_code(t) -> int:
    if t.dtype == torch.float32:
        return NATSL_F32
    if t.dtype == torch.bfloat16:
        return NATSL_BF16
    raise NatslError(-3, "dtype must be float32 or bfloat16")


def make_params(B, H, L, d, dtype_code, scale_la, scale_sm, eps=1e-5, C=64, flags=0, w=None,
                state_in=None, state_out=None, o_la=None, o_nla=None, lse=None, k_sm=None,
                v_sm=None, sm_len=None, sm_cap=0, G=0, norm_eps=0.0) -> natsl_params:
    p = natsl_params()
    p.G, p.norm_eps = G, norm_eps
    p.B, p.H, p.L, p.d, p.C, p.dtype = B, H, L, d, C, dtype_code
    p.scale_la, p.scale_sm, p.eps, p.flags = scale_la, scale_sm, eps, flags
    for name, t in dict(w=w, state_in=state_in, state_out=state_out, o_la=o_la, o_nla=o_nla,
                        lse=lse, k_sm=k_sm, v_sm=v_sm, sm_len=sm_len).items():
        setattr(p, name, _ptr(t).value)
    p.sm_cap = sm_cap
    return p


def natsl_workspace_size(p: natsl_params, op: int) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().natsl_workspace_size(ctypes.byref(p), op, ctypes.byref(n)))
    return int(n.value)


def alloc_workspace(p: natsl_params, op: int, device="cuda") -> torch.Tensor:
    """Zero-filled byte tensor of the size the library asks for (at least 256 bytes)."""
    return torch.zeros(max(natsl_workspace_size(p, op), 256), dtype=torch.uint8, device=device)


def natsl_route_compact(route, sm_idx, sm_chunk_prefix, lin_idx, n_lin, p: natsl_params):
    _check(lib().natsl_route_compact(_ptr(route), _ptr(sm_idx), _ptr(sm_chunk_prefix),
                                     _ptr(lin_idx), _ptr(n_lin), ctypes.byref(p),
                                     ctypes.c_void_p(0), ctypes.c_size_t(0), _stream()))


def natsl_hybrid_fwd(q, k, v, g, beta, route, out, p: natsl_params, ws):
    _check(lib().natsl_hybrid_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(route),
                                  _ptr(out), ctypes.byref(p), _ptr(ws),
                                  ctypes.c_size_t(ws.numel()), _stream()))


def natsl_hybrid_fwd_static(q, k, v, g, beta, route, out, p: natsl_params):
    """natsl_hybrid_fwd without a caller workspace: the scratch is a fixed array inside the
    library, for hosts that cannot allocate device memory.  Raises NatslError(-9) when the
    problem needs more than STATIC_WS_BYTES of scratch."""
    _check(lib().natsl_hybrid_fwd_static(_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta),
                                         _ptr(route), _ptr(out), ctypes.byref(p), _stream()))


def natsl_hybrid_bwd(q, k, v, g, beta, route, dout, dq, dk, dv, dg, dbeta, dw, p: natsl_params, ws):
    _check(lib().natsl_hybrid_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(route),
                                  _ptr(dout), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dg), _ptr(dbeta),
                                  _ptr(dw), ctypes.byref(p), _ptr(ws),
                                  ctypes.c_size_t(ws.numel()), _stream()))


def natsl_decode_step(q, k, v, g, beta, route, state, k_cache, v_cache, cache_len, out,
                      p: natsl_params, ws):
    cap = k_cache.shape[2]
    _check(lib().natsl_decode_step(_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(route),
                                   _ptr(state), _ptr(k_cache), _ptr(v_cache), _ptr(cache_len),
                                   ctypes.c_int32(cap), _ptr(out), ctypes.byref(p), _ptr(ws),
                                   ctypes.c_size_t(ws.numel()), _stream()))


def natsl_decode_block_end(route_block, g_block, state, state_start, cache_len, block_len,
                           p: natsl_params, ws):
    _check(lib().natsl_decode_block_end(_ptr(route_block), _ptr(g_block), _ptr(state),
                                        _ptr(state_start), _ptr(cache_len), ctypes.c_int32(block_len),
                                        ctypes.byref(p), _ptr(ws), ctypes.c_size_t(ws.numel()),
                                        _stream()))


def natsl_score_layer(x, w_score, scores, route, p: natsl_params):
    _check(lib().natsl_score_layer(_ptr(x), _ptr(w_score), _ptr(scores), _ptr(route),
                                   ctypes.c_int32(x.shape[-1]), ctypes.byref(p), _stream()))


def natsl_device_status(ws) -> int:
    return int(lib().natsl_device_status(_ptr(ws), _stream()))


def natsl_static_status() -> int:
    """Status word of the library's built-in scratch on the current device (synchronises)."""
    return int(lib().natsl_static_status(_stream()))


def natsl_debug_set_wait_limit(kcycles: int, withhold_scan_flags: bool = False):
    """Test hook: bound of the device-side waits in units of 1024 cycles (0 = default) and whether
    the scan withholds the per-chunk flags the softmax kernel waits for."""
    lib().natsl_debug_set_wait_limit(int(kcycles), 1 if withhold_scan_flags else 0)


# ---------------------------------------------------------------------------------------------
# Convenience wrappers (allocation + marshalling; no arithmetic).
# ---------------------------------------------------------------------------------------------
def hybrid_fwd(q, k, v, g, beta, route, w=None, *, scale_la, scale_sm, eps=1e-5, state_in=None,
               want=(), flags=0, sm_cap=0, ws=None, cache=None, G=0, norm_eps=0.0):
    """Allocate outputs and run natsl_hybrid_fwd.  `want` may name optional outputs:
    "o_la", "o_nla", "lse", "state_out", "cache" (compacted K/V with capacity sm_cap or L).
    cache=(k_sm, v_sm, sm_len): use these existing cache tensors (with APPEND_CACHE: in and out).
    G: softmax heads per linear head (lse is then [B,H,G,L]); norm_eps goes with the QK_NORM flag."""
    B, L, H, d = q.shape
    dev = q.device
    out = torch.empty_like(q)
    opt = {}
    if "o_la" in want:
        opt["o_la"] = torch.empty((B, L, H, d), dtype=torch.float32, device=dev)
    if "o_nla" in want:
        opt["o_nla"] = torch.empty((B, L, H, d), dtype=torch.float32, device=dev)
    if "lse" in want:
        opt["lse"] = torch.empty((B, H, G, L) if G > 1 else (B, H, L), dtype=torch.float32, device=dev)
    if "state_out" in want:
        opt["state_out"] = torch.empty((B, H, d, d), dtype=torch.float32, device=dev)
    cap = 0
    if cache is not None:
        opt["k_sm"], opt["v_sm"], opt["sm_len"] = cache
        cap = cache[0].shape[2]
    elif "cache" in want:
        cap = sm_cap or L
        opt["k_sm"] = torch.zeros((B, H, cap, d), dtype=q.dtype, device=dev)
        opt["v_sm"] = torch.zeros((B, H, cap, d), dtype=q.dtype, device=dev)
        opt["sm_len"] = torch.zeros((B, H), dtype=torch.int32, device=dev)
    p = make_params(B, H, L, d, _dtype_code(q), scale_la, scale_sm, eps, flags=flags, w=w,
                    state_in=state_in, sm_cap=cap, G=G, norm_eps=norm_eps, **opt)
    if ws is None:
        ws = alloc_workspace(p, OP_FWD, dev)
    natsl_hybrid_fwd(q, k, v, g, beta, route, out, p, ws)
    res = dict(out=out, ws=ws, **opt)
    return res


def hybrid_bwd(q, k, v, g, beta, route, w, dout, *, scale_la, scale_sm, eps=1e-5, ws=None, flags=0,
               want_dscore=False, state_in=None, dstate_out=None, want_dstate_in=False):
    """Allocate gradients and run natsl_hybrid_bwd.  Returns dict(dq, dk, dv, dg, dbeta, dw, ws)
    (+ dscore, dstate_in when asked for)."""
    B, L, H, d = q.shape
    dev = q.device
    dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    dg = torch.empty((B, L, H), dtype=torch.float32, device=dev)
    dbeta = torch.empty((B, L, H), dtype=torch.float32, device=dev)
    dw = torch.empty((B, L, H, 2), dtype=torch.float32, device=dev)
    p = make_params(B, H, L, d, _dtype_code(q), scale_la, scale_sm, eps, w=w, flags=flags,
                    state_in=state_in)
    dstate_in = None
    if dstate_out is not None:
        p.dstate_out = dstate_out.data_ptr()
    if want_dstate_in:
        dstate_in = torch.empty((B, H, d, d), dtype=torch.float32, device=dev)
        p.dstate_in = dstate_in.data_ptr()
    dscore = None
    if want_dscore:
        dscore = torch.empty((B, L // 64, H, 2), dtype=torch.float32, device=dev)
        p.dscore = dscore.data_ptr()
    if ws is None:
        ws = alloc_workspace(p, OP_BWD, dev)
    natsl_hybrid_bwd(q, k, v, g, beta, route, dout, dq, dk, dv, dg, dbeta, dw, p, ws)
    res = dict(dq=dq, dk=dk, dv=dv, dg=dg, dbeta=dbeta, dw=dw, ws=ws)
    if dscore is not None:
        res["dscore"] = dscore
    if dstate_in is not None:
        res["dstate_in"] = dstate_in
    return res
