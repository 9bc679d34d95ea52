"""ctypes binding of the fp64 CPU oracle (``vla_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the CPU-baseline leg
of the benchmark load this; the CUDA package never does.  The binding only
marshals numpy arrays; all arithmetic is in the C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vla_oracle.c")
_HDR = os.path.join(_HERE, "vla_oracle.h")
_LIB = os.path.join(_HERE, "libvla_oracle.so")
_SRC_BWD = os.path.join(_HERE, "vla_oracle_bwd.c")
_HDR_BWD = os.path.join(_HERE, "vla_oracle_bwd.h")
_LIB_BWD = os.path.join(_HERE, "libvla_oracle_bwd.so")

F32, BF16, F64 = 0, 1, 2
IDENTITY_MAP = 1
LINEAR_ATTENTION = 2

_lock = threading.Lock()
_default = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no vector intrinsics) if it is stale."""
    newest_src = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest_src:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-std=c99", "-O2", "-fPIC", "-shared", "-Wall", "-Wextra",
             "-o", tmp, _SRC, "-lm", "-lpthread"])
        os.replace(tmp, _LIB)
    return _LIB


def build_bwd(force: bool = False, src: Optional[str] = None, out: Optional[str] = None) -> str:
    """Compile the backward oracle (a separate shared object; ``src``/``out`` let the mutation
    tests build a broken copy)."""
    src = src or _SRC_BWD
    out = out or _LIB_BWD
    newest = max(os.path.getmtime(src), os.path.getmtime(_HDR_BWD), os.path.getmtime(_HDR))
    if force or not os.path.exists(out) or os.path.getmtime(out) < newest:
        tmp = out + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-std=c99", "-O2", "-fPIC", "-shared", "-Wall", "-Wextra", "-I", _HERE,
             "-o", tmp, src, "-lm", "-lpthread"])
        os.replace(tmp, out)
    return out


class _Trace(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("A", "S", "khat", "u", "alpha", "e", "delta", "den")]


class _Refresh(ctypes.Structure):
    _fields_ = [("period", ctypes.c_int), ("eta", ctypes.c_double), ("step_offset", ctypes.c_long)]


def _refresh_arg(refresh):
    """refresh = None or (period, eta, step_offset)."""
    if refresh is None:
        return None
    period, eta, off = refresh
    return ctypes.byref(_Refresh(int(period), float(eta), int(off)))


def _bind(path):
    lib = ctypes.CDLL(path)
    vp, i, d, u = ctypes.c_void_p, ctypes.c_int, ctypes.c_double, ctypes.c_uint
    lib.vla_oracle_forward.restype = i
    lib.vla_oracle_forward.argtypes = [vp, vp, vp, vp, i, d, i, i, i, i, i,
                                       vp, vp, vp, u, d, vp, vp, vp, vp, i, vp]
    lib.vla_oracle_forward_trace.restype = i
    lib.vla_oracle_forward_trace.argtypes = [vp, vp, vp, vp, i, d, i, i, i,
                                             vp, vp, vp, u, d, vp, vp, vp, vp,
                                             ctypes.POINTER(_Trace), vp]
    return lib


def _np_dtype(in_dtype: int):
    return {F32: np.float32, BF16: np.uint16, F64: np.float64}[in_dtype]


def _in(a, in_dtype, shape):
    a = np.ascontiguousarray(a, dtype=_np_dtype(in_dtype))
    assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _opt64(a, shape):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=np.float64)
    assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


@dataclass
class OracleResult:
    out: np.ndarray   # [B,H,T,d_v] fp64
    S_T: np.ndarray   # [B,H,d_v,d_k]
    A_T: np.ndarray   # [B,H,d_k,d_k]
    z_T: np.ndarray   # [B,H,d_k]
    trace: Optional[dict] = None


class OracleLib:
    """One loaded build of the oracle.  ``load()`` gives the committed source's build;
    the mutation tests wrap deliberately broken builds of a copy of the C file."""

    def __init__(self, path: str):
        self.path = path
        self._lib = _bind(path)

    def forward(self, q, k, v, lam, *, u=None, in_dtype=F32, S0=None, A0=None, z0=None,
                flags=0, eps=1e-4, n_threads=1, refresh=None) -> OracleResult:
        """All units of ``q,k[,u]: [B,H,T,d_k]``, ``v: [B,H,T,d_v]``.

        bf16 inputs are passed as uint16 bit patterns (``in_dtype=BF16``).
        """
        lib = self._lib
        B, H, T, dk = np.shape(q)
        dv = np.shape(v)[-1]
        q = _in(q, in_dtype, (B, H, T, dk))
        k = _in(k, in_dtype, (B, H, T, dk))
        v = _in(v, in_dtype, (B, H, T, dv))
        u = None if u is None else _in(u, in_dtype, (B, H, T, dk))
        S0 = _opt64(S0, (B, H, dv, dk))
        A0 = _opt64(A0, (B, H, dk, dk))
        z0 = _opt64(z0, (B, H, dk))
        out = np.empty((B, H, T, dv), np.float64)
        S_T = np.empty((B, H, dv, dk), np.float64)
        A_T = np.empty((B, H, dk, dk), np.float64)
        z_T = np.empty((B, H, dk), np.float64)
        rc = lib.vla_oracle_forward(_ptr(q), _ptr(k), _ptr(v), _ptr(u), in_dtype, float(lam),
                                    B, H, T, dk, dv, _ptr(S0), _ptr(A0), _ptr(z0),
                                    flags, float(eps), _ptr(out), _ptr(S_T), _ptr(A_T),
                                    _ptr(z_T), int(n_threads), _refresh_arg(refresh))
        if rc != 0:
            raise ValueError("vla_oracle_forward: invalid argument")
        return OracleResult(out, S_T, A_T, z_T)


    def forward_trace(self, q, k, v, lam, *, u=None, in_dtype=F64, S0=None, A0=None, z0=None,
                      flags=0, eps=1e-4, refresh=None) -> OracleResult:
        """One unit (``q,k[,u]: [T,d_k]``, ``v: [T,d_v]``) with every per-step quantity dumped."""
        lib = self._lib
        T, dk = np.shape(q)
        dv = np.shape(v)[-1]
        q = _in(q, in_dtype, (T, dk))
        k = _in(k, in_dtype, (T, dk))
        v = _in(v, in_dtype, (T, dv))
        u = None if u is None else _in(u, in_dtype, (T, dk))
        S0 = _opt64(S0, (dv, dk))
        A0 = _opt64(A0, (dk, dk))
        z0 = _opt64(z0, (dk,))
        out = np.empty((T, dv), np.float64)
        S_T = np.empty((dv, dk), np.float64)
        A_T = np.empty((dk, dk), np.float64)
        z_T = np.empty((dk,), np.float64)
        tr = dict(A=np.empty((T, dk, dk)), S=np.empty((T, dv, dk)), khat=np.empty((T, dk)),
                  u=np.empty((T, dk)), alpha=np.empty((T, dk)), e=np.empty((T, dv)),
                  delta=np.empty((T,)), den=np.empty((T,)))
        ctr = _Trace(**{n: a.ctypes.data for n, a in tr.items()})
        rc = lib.vla_oracle_forward_trace(_ptr(q), _ptr(k), _ptr(v), _ptr(u), in_dtype,
                                          float(lam), T, dk, dv, _ptr(S0), _ptr(A0), _ptr(z0),
                                          flags, float(eps), _ptr(out), _ptr(S_T), _ptr(A_T),
                                          _ptr(z_T), ctypes.byref(ctr), _refresh_arg(refresh))
        if rc != 0:
            raise ValueError("vla_oracle_forward_trace: invalid argument")
        return OracleResult(out, S_T, A_T, z_T, tr)


def load() -> OracleLib:
    global _default
    with _lock:
        if _default is None:
            _default = OracleLib(build())
    return _default


def forward(*args, **kw) -> OracleResult:
    return load().forward(*args, **kw)


def forward_trace(*args, **kw) -> OracleResult:
    return load().forward_trace(*args, **kw)


def state_norms(q, k, v, lam, **kw):
    """Per-step Frobenius norms (||S_t||_F, ||A_t||_F) of one unit, the quantities of the
    paper's stability experiment (Section 6.2), from the traced oracle.  A diagnostic: the
    paper's printed trajectory does not reproduce under any stated u (only ||A_0||_F does)."""
    r = load().forward_trace(q, k, v, lam, **kw)
    T = r.trace["S"].shape[0]
    return (np.linalg.norm(r.trace["S"].reshape(T, -1), axis=1),
            np.linalg.norm(r.trace["A"].reshape(T, -1), axis=1))


@dataclass
class OracleGrads:
    dq: np.ndarray
    dk: np.ndarray
    dv: np.ndarray
    du: Optional[np.ndarray]
    dS0: np.ndarray
    dA0: np.ndarray
    dz0: np.ndarray


class OracleBwdLib:
    """One loaded build of the backward oracle (``vla_oracle_bwd.c``)."""

    def __init__(self, path: Optional[str] = None):
        self.path = path or build_bwd()
        lib = ctypes.CDLL(self.path)
        vp, i, d, u = ctypes.c_void_p, ctypes.c_int, ctypes.c_double, ctypes.c_uint
        lib.vla_oracle_backward.restype = i
        lib.vla_oracle_backward.argtypes = [vp, vp, vp, vp, i, d, i, i, i, i, i, vp, vp, vp, u, d,
                                            vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i, vp]
        self._lib = lib

    def backward(self, q, k, v, lam, d_out, *, u=None, in_dtype=F64, S0=None, A0=None, z0=None,
                 dS_T=None, dA_T=None, dz_T=None, flags=0, eps=1e-4, n_threads=1,
                 refresh=None) -> OracleGrads:
        """Gradients for ``q,k[,u]: [B,H,T,d_k]``, ``v, d_out: [B,H,T,d_v]``."""
        B, H, T, dk = np.shape(q)
        dv = np.shape(v)[-1]
        q = _in(q, in_dtype, (B, H, T, dk))
        k = _in(k, in_dtype, (B, H, T, dk))
        v = _in(v, in_dtype, (B, H, T, dv))
        u = None if u is None else _in(u, in_dtype, (B, H, T, dk))
        S0 = _opt64(S0, (B, H, dv, dk)); A0 = _opt64(A0, (B, H, dk, dk)); z0 = _opt64(z0, (B, H, dk))
        d_out = _opt64(d_out, (B, H, T, dv))
        dS_T = _opt64(dS_T, (B, H, dv, dk)); dA_T = _opt64(dA_T, (B, H, dk, dk))
        dz_T = _opt64(dz_T, (B, H, dk))
        dq = np.zeros((B, H, T, dk)); dkk = np.zeros((B, H, T, dk)); dvv = np.zeros((B, H, T, dv))
        du = None if u is None else np.zeros((B, H, T, dk))
        dS0 = np.zeros((B, H, dv, dk)); dA0 = np.zeros((B, H, dk, dk)); dz0 = np.zeros((B, H, dk))
        rc = self._lib.vla_oracle_backward(
            _ptr(q), _ptr(k), _ptr(v), _ptr(u), in_dtype, float(lam), B, H, T, dk, dv,
            _ptr(S0), _ptr(A0), _ptr(z0), flags, float(eps), _ptr(d_out), _ptr(dS_T), _ptr(dA_T),
            _ptr(dz_T), _ptr(dq), _ptr(dkk), _ptr(dvv), _ptr(du), _ptr(dS0), _ptr(dA0), _ptr(dz0),
            int(n_threads), _refresh_arg(refresh))
        if rc != 0:
            raise ValueError("vla_oracle_backward: invalid argument")
        return OracleGrads(dq, dkk, dvv, du, dS0, dA0, dz0)


_default_bwd = None


def load_bwd() -> OracleBwdLib:
    global _default_bwd
    with _lock:
        if _default_bwd is None:
            _default_bwd = OracleBwdLib()
        return _default_bwd


def backward(*args, **kwargs) -> OracleGrads:
    return load_bwd().backward(*args, **kwargs)
