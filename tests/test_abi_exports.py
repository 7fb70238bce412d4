"""The C-ABI library builds for sm_100a without a GPU, loads, and exports every entry point that
include/natsl.h declares.  No compute call is made here."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "natsl.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(natsl_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_header_symbols():
    from paper_2602_03681_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert "natsl_hybrid_fwd" in names and "natsl_decode_step" in names
    for name in names:
        assert hasattr(lib, name), name


def test_binding_lists_the_same_names():
    from paper_2602_03681_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    for name in binding.EXPORTS:
        assert hasattr(binding, name)


def test_host_side_validation_needs_no_gpu():
    """Shape / NULL / dtype errors are returned before anything is launched."""
    from paper_2602_03681_b200 import binding, build
    build.build()
    lib = binding.lib()
    p = binding.natsl_params()
    p.B, p.H, p.L, p.d, p.C, p.dtype, p.eps = 1, 1, 100, 64, 64, 0, 1e-5
    n = ctypes.c_size_t(0)
    assert lib.natsl_workspace_size(ctypes.byref(p), binding.OP_FWD, ctypes.byref(n)) == -2
    p.L = 128
    assert lib.natsl_workspace_size(ctypes.byref(p), binding.OP_FWD, ctypes.byref(n)) == 0
    assert n.value > 0
    p.d = 96
    assert lib.natsl_workspace_size(ctypes.byref(p), binding.OP_FWD, ctypes.byref(n)) == -2
    p.d, p.dtype = 64, 7
    assert lib.natsl_workspace_size(ctypes.byref(p), binding.OP_FWD, ctypes.byref(n)) == -3
    p.dtype = 1
    null = ctypes.c_void_p(0)
    rc = lib.natsl_hybrid_fwd(null, null, null, null, null, null, null, ctypes.byref(p), null,
                              ctypes.c_size_t(0), null)
    assert rc == -1
    assert b"NULL" in lib.natsl_strerror(-1)
