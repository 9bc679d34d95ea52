"""Host-side checks that need no GPU: the library builds, loads, exports every symbol the
header declares, and rejects bad arguments before any launch."""
import ctypes
import os
import re

import pytest

import paper_2605_11196_b200 as vla
from paper_2605_11196_b200 import build as vbuild
from paper_2605_11196_b200.binding import EXPORTS, VlaOpts

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "vla.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vla_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = vbuild.build()
    lib = ctypes.CDLL(path)
    names = declared_functions()
    assert set(names) == set(EXPORTS), (names, EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def test_version_and_support_query():
    assert vla.vla_version() >= 100
    for d in (16, 32, 64, 128):
        for dt in (vla.VLA_F32, vla.VLA_BF16):
            assert vla.vla_query_support(d, d, dt, 0) == vla.VLA_OK
            assert vla.vla_query_support(d, d, dt, vla.VLA_FLAG_IDENTITY_MAP) == vla.VLA_OK
    assert vla.vla_query_support(48, 48) == vla.VLA_ERR_UNSUPPORTED
    assert vla.vla_query_support(64, 32) == vla.VLA_ERR_UNSUPPORTED
    assert vla.vla_query_support(64, 64, 7) == vla.VLA_ERR_UNSUPPORTED
    assert vla.status_string(0) == "ok"
    assert "unknown" in vla.status_string(-99)


def _call(q=0x1000, k=0x2000, v=0x3000, lam=1.0, B=1, H=1, T=4, dk=32, dv=32, S0=None, A0=None,
          out=0x4000, opts=None):
    lib = vla.load_library()
    vp = ctypes.c_void_p
    return lib.vla_forward(vp(q), vp(k), vp(v), lam, B, H, T, dk, dv, vp(S0), vp(A0), vp(out),
                           None, None, opts, None)


def test_host_side_validation_returns_codes_before_any_launch():
    # none of these reaches a CUDA call: the fake pointers are never dereferenced
    assert _call(B=-1) == vla.VLA_ERR_INVALID_ARG
    assert _call(T=-5) == vla.VLA_ERR_INVALID_ARG
    assert _call(dk=48, dv=48) == vla.VLA_ERR_UNSUPPORTED
    assert _call(dk=64, dv=32) == vla.VLA_ERR_UNSUPPORTED
    assert _call(lam=0.0) == vla.VLA_ERR_INVALID_ARG
    assert _call(lam=-1.0) == vla.VLA_ERR_INVALID_ARG
    assert _call(q=None) == vla.VLA_ERR_INVALID_ARG
    assert _call(out=None) == vla.VLA_ERR_INVALID_ARG
    assert _call(q=0x1004) == vla.VLA_ERR_ALIGNMENT
    assert _call(S0=0x5008) == vla.VLA_ERR_ALIGNMENT
    o = VlaOpts(); o.struct_size = 4
    assert _call(opts=ctypes.byref(o)) == vla.VLA_ERR_INVALID_ARG
    o = VlaOpts(); o.struct_size = ctypes.sizeof(VlaOpts); o.qkv_dtype = 9
    assert _call(opts=ctypes.byref(o)) == vla.VLA_ERR_INVALID_ARG
    o = VlaOpts(); o.struct_size = ctypes.sizeof(VlaOpts); o.flags = 1 << 9
    assert _call(opts=ctypes.byref(o)) == vla.VLA_ERR_INVALID_ARG
    assert _call(B=0) == vla.VLA_OK          # no units: nothing to do
    assert vla.vla_host_workspace_bytes(-1, 1, 1, 32, 32) == 0
    assert vla.vla_host_workspace_bytes(2, 2, 8, 32, 32) >= 3 * 2 * 2 * 8 * 32 * 4


def test_missing_library_raises(monkeypatch):
    from paper_2605_11196_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding._build, "LIB", "/nonexistent/libvla.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.load_library()


def test_newer_entry_points_validate_on_the_host():
    """vla_make_u, vla_backward and vla_forward_seqpar refuse bad or unsupported arguments before
    any CUDA call (the fake pointers are never dereferenced)."""
    lib = vla.load_library()
    vp = ctypes.c_void_p
    f = ctypes.c_float
    mk = lambda **kw: lib.vla_make_u(vp(kw.get("k", 0x1000)), vp(kw.get("W", 0x2000)), kw.get("B", 1), kw.get("H", 1),
                                     kw.get("T", 4), kw.get("d", 32), kw.get("kd", 0), kw.get("ud", 0), f(1.0), f(1e-4),
                                     vp(kw.get("u", 0x3000)), None)
    assert mk(d=48) == vla.VLA_ERR_UNSUPPORTED
    assert mk(B=-1) == vla.VLA_ERR_INVALID_ARG
    assert mk(kd=7) == vla.VLA_ERR_INVALID_ARG
    assert mk(k=None) == vla.VLA_ERR_INVALID_ARG
    assert mk(u=0x3004) == vla.VLA_ERR_ALIGNMENT
    assert mk(T=0) == vla.VLA_OK and mk(B=0) == vla.VLA_OK

    def bwd(opts=None, d=32, dq=0x6000):
        return lib.vla_backward(vp(0x1000), vp(0x2000), vp(0x3000), 1.0, 1, 1, 4, d, d, None, None, vp(0x4000),
                                None, None, None, vp(dq), vp(0x7000), vp(0x8000), None, None, None, opts,
                                vp(0x10000), 1 << 30, None)
    o = VlaOpts(); o.struct_size = ctypes.sizeof(VlaOpts); o.flags = vla.VLA_FLAG_TOKEN_MAJOR
    assert bwd(ctypes.byref(o), d=16) == vla.VLA_ERR_UNSUPPORTED    # token-major tensors: d >= 32
    o = VlaOpts(); o.struct_size = ctypes.sizeof(VlaOpts); o.u = 0x9000
    assert bwd(ctypes.byref(o)) == vla.VLA_ERR_INVALID_ARG          # explicit u needs opts->du
    o.du = 0xa000
    assert bwd(ctypes.byref(o), d=16) == vla.VLA_ERR_UNSUPPORTED    # explicit u: d >= 32
    o = VlaOpts(); o.struct_size = ctypes.sizeof(VlaOpts); o.refresh_period = 4; o.refresh_eta = 1e-3
    assert bwd(ctypes.byref(o), d=16) == vla.VLA_ERR_UNSUPPORTED    # refresh: d >= 32
    assert bwd(dq=None) == vla.VLA_ERR_INVALID_ARG
    assert bwd(dq=0x6004) == vla.VLA_ERR_ALIGNMENT
    small = lib.vla_backward(vp(0x1000), vp(0x2000), vp(0x3000), 1.0, 1, 1, 4, 32, 32, None, None, vp(0x4000),
                             None, None, None, vp(0x6000), vp(0x7000), vp(0x8000), None, None, None, None,
                             vp(0x10000), 16, None)
    assert small == vla.VLA_ERR_INVALID_ARG                          # workspace too small
    # the workspace grows with every dimension and covers the per-token vectors
    w1 = vla.backward_workspace_bytes(2, 3, 64, 32)
    assert w1 >= 6 * 2 * 3 * 64 * 32 * 4
    assert vla.backward_workspace_bytes(2, 3, 128, 32) > w1 and vla.backward_workspace_bytes(2, 3, 64, 64) > w1
    assert vla.backward_workspace_bytes(-1, 3, 64, 32) == 0
    assert vla.vla_query_support(64, 64, vla.VLA_BF16, vla.VLA_FLAG_TOKEN_MAJOR) == vla.VLA_OK
