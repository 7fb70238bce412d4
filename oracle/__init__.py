"""fp64 CPU oracle of the NAtS-L hybrid attention layer -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  The CUDA library and its Python binding never do, and this package imports
nothing from them.

``natsl_oracle.c`` holds the token-by-token definition (forward, analytic backward,
decode step, route compaction); this module marshals numpy arrays into it.
``chunkwise.py`` restates the linear branch in the chunkwise (WY / UT-transform) form
and ``bruteforce.py`` materialises the column masks for tiny sequences; both exist
only to cross-check the recurrent definition.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "natsl_oracle.c")
_LIB_PATH = os.path.join(_HERE, "libnatsl_oracle.so")
_lib = None

_f64p = ctypes.POINTER(ctypes.c_double)
_u8p = ctypes.POINTER(ctypes.c_uint8)
_i32p = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over batch x head)."""
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC)):
        return _LIB_PATH
    tmp = _LIB_PATH + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB_PATH)
        _lib.natsl_oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().natsl_oracle_num_threads())


def _d(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def _p(a, ty=_f64p):
    return None if a is None else a.ctypes.data_as(ty)


def route_compact(route: np.ndarray, C: int):
    """Index lists of the softmax and linear tokens (Section 4.1, masks M^nla / M^la).

    route [B,L,H] uint8.  Returns dict(sm_idx [B,H,L] (first n_sm valid, rest -1),
    sm_chunk_prefix [B,H,L/C+1], lin_idx [B,H,L/C,C] padded with C, n_lin [B,H,L/C]).
    """
    route = np.ascontiguousarray(route, dtype=np.uint8)
    B, L, H = route.shape
    NC = L // C
    sm_idx = np.full((B, H, L), -1, np.int32)
    pre = np.zeros((B, H, NC + 1), np.int32)
    lin_idx = np.zeros((B, H, NC, C), np.int32)
    n_lin = np.zeros((B, H, NC), np.int32)
    rc = _load().natsl_oracle_route_compact(_p(route, _u8p), B, L, H, C, _p(sm_idx, _i32p),
                                            _p(pre, _i32p), _p(lin_idx, _i32p), _p(n_lin, _i32p))
    if rc != 0:
        raise ValueError(f"natsl_oracle_route_compact failed ({rc}): L % C must be 0")
    return dict(sm_idx=sm_idx, sm_chunk_prefix=pre, lin_idx=lin_idx, n_lin=n_lin)


def hybrid_fwd(q, k, v, g, beta, route, w=None, *, scale_la, scale_sm, eps=1e-5, state_in=None,
               want_cache=False, block=None):
    """Token-by-token forward (Section 4.1 masks, Section 4.3 GDN + decay-always + Norm).

    q,k,v [B,L,H,d]; g,beta [B,L,H]; route [B,L,H]; w [B,L,H,2] or None.
    block=R: one routing decision per block of R tokens; both operations see the query's own
    block and the one not chosen is rolled back at the block's end (Section 4.1, the paragraphs
    on intra-chunk correlations and per-token generation).  route must be constant per block.
    Returns dict(out, o_la, o_nla [B,L,H,d]; lse [B,H,L]; state_out [B,H,d,d];
    and with want_cache: k_sm, v_sm [B,H,L,d], n_sm [B,H]).
    """
    q, k, v, g, beta, w, state_in = map(_d, (q, k, v, g, beta, w, state_in))
    route = np.ascontiguousarray(route, dtype=np.uint8)
    B, L, H, d = q.shape
    out, o_la, o_nla = (np.zeros((B, L, H, d)) for _ in range(3))
    lse = np.zeros((B, H, L))
    state_out = np.zeros((B, H, d, d))
    kc = np.zeros((B, H, L, d)) if want_cache else None
    vc = np.zeros((B, H, L, d)) if want_cache else None
    n_sm = np.zeros((B, H), np.int32) if want_cache else None
    tail = (ctypes.c_double(scale_la), ctypes.c_double(scale_sm), ctypes.c_double(eps),
            _p(state_in), _p(out), _p(o_la), _p(o_nla), _p(lse), _p(state_out), _p(kc), _p(vc),
            _p(n_sm, _i32p))
    head = (_p(q), _p(k), _p(v), _p(g), _p(beta), _p(route, _u8p), _p(w), B, L, H, d)
    if block is None:
        rc = _load().natsl_oracle_hybrid_fwd(*head, *tail)
    else:
        rc = _load().natsl_oracle_hybrid_fwd_block(*head, int(block), *tail)
    if rc == -4:
        raise ValueError("block mode: route must be constant within each block")
    if rc != 0:
        raise RuntimeError(f"natsl_oracle_hybrid_fwd failed ({rc})")
    res = dict(out=out, o_la=o_la, o_nla=o_nla, lse=lse, state_out=state_out)
    if want_cache:
        res.update(k_sm=kc, v_sm=vc, n_sm=n_sm)
    return res


def hybrid_bwd(q, k, v, g, beta, route, w, dout, *, scale_la, scale_sm, eps=1e-5, state_in=None,
               dstate_out=None, block=None):
    """Analytic reverse-mode gradients of hybrid_fwd's `out` (and state_out) contraction.
    block=R: of the block-mode forward (hybrid_fwd with the same `block`).

    Returns dict(dq, dk, dv [B,L,H,d]; dg, dbeta [B,L,H]; dw [B,L,H,2]; dstate_in [B,H,d,d]).
    """
    q, k, v, g, beta, w, dout, state_in, dstate_out = map(
        _d, (q, k, v, g, beta, w, dout, state_in, dstate_out))
    route = np.ascontiguousarray(route, dtype=np.uint8)
    B, L, H, d = q.shape
    dq, dk, dv = (np.zeros((B, L, H, d)) for _ in range(3))
    dg, dbeta = np.zeros((B, L, H)), np.zeros((B, L, H))
    dw = np.zeros((B, L, H, 2))
    dstate_in = np.zeros((B, H, d, d))
    head = (_p(q), _p(k), _p(v), _p(g), _p(beta), _p(route, _u8p), _p(w), _p(dout), B, L, H, d)
    tail = (ctypes.c_double(scale_la), ctypes.c_double(scale_sm), ctypes.c_double(eps),
            _p(state_in), _p(dstate_out), _p(dq), _p(dk), _p(dv), _p(dg), _p(dbeta), _p(dw),
            _p(dstate_in))
    dscore = None
    if block is None:
        rc = _load().natsl_oracle_hybrid_bwd(*head, *tail)
    else:
        dscore = np.zeros((B, L // int(block), H, 2))
        rc = _load().natsl_oracle_hybrid_bwd_block(*head, int(block), *tail, _p(dscore))
    if rc == -4:
        raise ValueError("block mode: route must be constant within each block")
    if rc != 0:
        raise RuntimeError(f"natsl_oracle_hybrid_bwd failed ({rc})")
    res = dict(dq=dq, dk=dk, dv=dv, dg=dg, dbeta=dbeta, dw=dw, dstate_in=dstate_in)
    if dscore is not None:
        res["dscore"] = dscore      # [B, L/R, H, 2]: (linear, softmax) mask gradients per block
    return res


def decode_step(q, k, v, g, beta, route, w, state, k_cache, v_cache, cache_len, *, scale_la,
                scale_sm, eps=1e-5):
    """One generation step; `state`, `k_cache`, `v_cache`, `cache_len` are updated IN PLACE.
    route 0 / 1: linear / softmax token; 2: token of a block whose decision is still open (folded
    into the state and appended to the cache; see block_end).

    q,k,v [B,H,d]; g,beta,route [B,H]; w [B,H,2] or None; state [B,H,d,d] float64;
    k_cache,v_cache [B,H,cap,d] float64; cache_len [B,H] int32.
    Returns dict(out, o_la, o_nla [B,H,d]).
    """
    for a in (state, k_cache, v_cache):
        assert a.dtype == np.float64 and a.flags.c_contiguous
    assert cache_len.dtype == np.int32 and cache_len.flags.c_contiguous
    q, k, v, g, beta, w = map(_d, (q, k, v, g, beta, w))
    route = np.ascontiguousarray(route, dtype=np.uint8)
    B, H, d = q.shape
    cap = k_cache.shape[2]
    out, o_la, o_nla = (np.zeros((B, H, d)) for _ in range(3))
    rc = _load().natsl_oracle_decode_step(
        _p(q), _p(k), _p(v), _p(g), _p(beta), _p(route, _u8p), _p(w), B, H, d,
        ctypes.c_double(scale_la), ctypes.c_double(scale_sm), ctypes.c_double(eps),
        _p(state), _p(k_cache), _p(v_cache), _p(cache_len, _i32p), cap, _p(out), _p(o_la),
        _p(o_nla))
    if rc == -3:
        raise OverflowError("retained-KV cache full")
    if rc != 0:
        raise RuntimeError(f"natsl_oracle_decode_step failed ({rc})")
    return dict(out=out, o_la=o_la, o_nla=o_nla)


def block_end(route_block, g_block, state, state_start, cache_len, R):
    """End of a block of R tokens decoded with route 2 (Section 4.1, roll-back of the operation
    that was not chosen).  `state`, `state_start`, `cache_len` are updated IN PLACE."""
    for a in (state, state_start):
        assert a.dtype == np.float64 and a.flags.c_contiguous
    assert cache_len.dtype == np.int32 and cache_len.flags.c_contiguous
    route_block = np.ascontiguousarray(route_block, dtype=np.uint8)
    g_block = _d(g_block)
    B, H, d, _ = state.shape
    rc = _load().natsl_oracle_block_end(_p(route_block, _u8p), _p(g_block), B, H, d, int(R),
                                        _p(state), _p(state_start), _p(cache_len, _i32p))
    if rc != 0:
        raise RuntimeError(f"natsl_oracle_block_end failed ({rc})")
