"""Thin Python binding of the C ABI in ``include/vla.h``: argument marshalling only.

Every step of the scan runs in the CUDA kernels behind ``libvla.so``.  There is no
fallback: if the library is missing or a shape has no kernel, the call raises.
PyTorch is used for device memory and streams only.
"""
from __future__ import annotations

import ctypes
import os
import threading
from dataclasses import dataclass
from typing import NamedTuple, Optional

import torch

from . import build as _build

VLA_OK = 0
VLA_ERR_INVALID_ARG, VLA_ERR_UNSUPPORTED, VLA_ERR_ALIGNMENT = -1, -2, -3
VLA_ERR_CUDA, VLA_ERR_DEVICE_TIMEOUT, VLA_ERR_NONFINITE, VLA_ERR_TOO_LARGE = -4, -5, -6, -7
VLA_STATIC_SCRATCH_BYTES = 32 << 20
VLA_F32, VLA_BF16 = 0, 1
VLA_FLAG_IDENTITY_MAP, VLA_FLAG_CHECK_FINITE, VLA_FLAG_TOKEN_MAJOR, VLA_FLAG_LINEAR_ATTENTION = 1, 2, 4, 8
VLA_KERNEL_AUTO, VLA_KERNEL_TOKEN, VLA_KERNEL_CHUNK, VLA_KERNEL_DECODE, VLA_KERNEL_CHUNK_TC = 0, 1, 2, 3, 4

EXPORTS = ("vla_forward", "vla_forward_host", "vla_forward_host_static", "vla_host_workspace_bytes",
           "vla_forward_seqpar", "vla_seqpar_segments", "vla_seqpar_workspace_bytes",
           "vla_probe_fp32_fma", "vla_backward", "vla_backward_workspace_bytes", "vla_make_u",
           "vla_query_support", "vla_status_string", "vla_version", "vla_selftest_wait_timeout",
           "vla_last_launch")


class VlaOpts(ctypes.Structure):
    """Mirror of ``vla_opts_t``."""
    _fields_ = [("struct_size", ctypes.c_uint32), ("qkv_dtype", ctypes.c_int32),
                ("u", ctypes.c_void_p), ("flags", ctypes.c_uint32), ("eps", ctypes.c_float),
                ("z0", ctypes.c_void_p), ("zT", ctypes.c_void_p), ("status", ctypes.c_void_p),
                ("kernel", ctypes.c_int32), ("refresh_period", ctypes.c_int32),
                ("refresh_eta", ctypes.c_float), ("step_offset", ctypes.c_int64), ("du", ctypes.c_void_p),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
                ("wait_probe_limit", ctypes.c_uint32)]


class VlaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s: %s (%d)" % (where, status_string(code), code))


_lock = threading.Lock()
_lib = None


def library_path() -> str:
    return _build.LIB


def load_library():
    """dlopen ``libvla.so`` (built in-tree by ``build.build()``).  Raises if it is absent."""
    global _lib
    with _lock:
        if _lib is None:
            path = library_path()
            if not os.path.exists(path):
                raise RuntimeError(
                    "CUDA library %s is missing: run paper_2605_11196_b200.build.build() "
                    "(there is no fallback path)" % path)
            lib = ctypes.CDLL(path)
            vp, i, f = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
            lib.vla_forward.restype = i
            lib.vla_forward.argtypes = [vp, vp, vp, f, i, i, i, i, i, vp, vp, vp, vp, vp,
                                        ctypes.POINTER(VlaOpts), vp]
            lib.vla_forward_host.restype = i
            lib.vla_forward_host.argtypes = [vp, vp, vp, f, i, i, i, i, i, vp, vp, vp, vp, vp,
                                             ctypes.POINTER(VlaOpts), vp, ctypes.c_size_t, vp]
            lib.vla_forward_host_static.restype = i
            lib.vla_forward_host_static.argtypes = [vp, vp, vp, f, i, i, i, i, i, vp, vp, vp, vp, vp,
                                                    ctypes.POINTER(VlaOpts), vp]
            lib.vla_forward_seqpar.restype = i
            lib.vla_forward_seqpar.argtypes = [vp, vp, vp, f, i, i, i, i, i, vp, vp, vp, vp, vp, vp, i,
                                               vp, ctypes.c_size_t, vp]
            lib.vla_seqpar_segments.restype = i
            lib.vla_seqpar_segments.argtypes = [i, i, i, i, i]
            lib.vla_seqpar_workspace_bytes.restype = ctypes.c_size_t
            lib.vla_seqpar_workspace_bytes.argtypes = [i, i, i, i, i]
            lib.vla_backward.restype = i
            lib.vla_backward.argtypes = [vp, vp, vp, f, i, i, i, i, i] + [vp] * 13 + [vp, ctypes.c_size_t, vp]
            lib.vla_backward_workspace_bytes.restype = ctypes.c_size_t
            lib.vla_backward_workspace_bytes.argtypes = [i, i, i, i]
            lib.vla_make_u.restype = i
            lib.vla_make_u.argtypes = [vp, vp, i, i, i, i, i, i, ctypes.c_float, ctypes.c_float, vp, vp]
            lib.vla_probe_fp32_fma.restype = i
            lib.vla_probe_fp32_fma.argtypes = [i, vp, ctypes.POINTER(ctypes.c_double), vp]
            lib.vla_host_workspace_bytes.restype = ctypes.c_size_t
            lib.vla_host_workspace_bytes.argtypes = [i, i, i, i, i, i, i]
            lib.vla_query_support.restype = i
            lib.vla_query_support.argtypes = [i, i, i, ctypes.c_uint32]
            lib.vla_status_string.restype = ctypes.c_char_p
            lib.vla_status_string.argtypes = [i]
            lib.vla_version.restype = i
            lib.vla_version.argtypes = []
            lib.vla_selftest_wait_timeout.restype = i
            lib.vla_selftest_wait_timeout.argtypes = [ctypes.c_uint32, vp, vp]
            lib.vla_last_launch.restype = i
            lib.vla_last_launch.argtypes = [ctypes.c_char_p, ctypes.c_size_t]
            _lib = lib
    return _lib


def last_launch() -> str:
    """Name, instantiation and grid of the kernel this thread's last library call launched last."""
    buf = ctypes.create_string_buffer(160)
    rc = load_library().vla_last_launch(buf, len(buf))
    if rc != VLA_OK:
        raise VlaError(rc, "vla_last_launch")
    return buf.value.decode()


def selftest_wait_timeout(probe_limit: int, status: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Enqueue the library's bounded-wait test kernel (``vla_selftest_wait_timeout``): ``status``
    (device int32, zero on entry) reads ``VLA_ERR_DEVICE_TIMEOUT`` once the stream has run it."""
    st = stream if stream is not None else torch.cuda.current_stream(status.device)
    with torch.cuda.device(status.device):
        rc = load_library().vla_selftest_wait_timeout(int(probe_limit), _ptr(status), ctypes.c_void_p(st.cuda_stream))
    if rc != VLA_OK:
        raise VlaError(rc, "vla_selftest_wait_timeout")


def status_string(code: int) -> str:
    return load_library().vla_status_string(int(code)).decode()


def vla_version() -> int:
    return load_library().vla_version()


def vla_query_support(d_k: int, d_v: int, qkv_dtype: int = VLA_F32, flags: int = 0) -> int:
    return load_library().vla_query_support(d_k, d_v, qkv_dtype, flags)


def vla_make_u(k, W_u, *, scale: Optional[float] = None, eps: float = 1e-4, out=None, out_dtype=None,
               stream: Optional[torch.cuda.Stream] = None):
    """``u = scale * L2norm(W_u[h] k)`` for CUDA tensors ``k: [B,H,T,d]``, ``W_u: [H,d,d]`` fp32.
    ``scale`` defaults to Algorithm 1's ``1/sqrt(d)``; the result has ``out_dtype`` (default: k's)."""
    lib = load_library()
    B, H, T, d = k.shape
    if out_dtype is None:
        out_dtype = k.dtype if out is None else out.dtype
    _chk(k, (B, H, T, d), k.dtype, "k"); _chk(W_u, (H, d, d), torch.float32, "W_u")
    if out is None:
        out = torch.empty((B, H, T, d), dtype=out_dtype, device=k.device)
    _chk(out, (B, H, T, d), out_dtype, "out")
    if scale is None:
        scale = float(d) ** -0.5
    st = stream if stream is not None else torch.cuda.current_stream(k.device)
    with torch.cuda.device(k.device):
        rc = lib.vla_make_u(_ptr(k), _ptr(W_u), B, H, T, d, _dtype_code(k), _dtype_code(out),
                            float(scale), float(eps), _ptr(out), ctypes.c_void_p(st.cuda_stream))
    if rc != VLA_OK:
        raise VlaError(rc, "vla_make_u")
    return out


def vla_host_workspace_bytes(B, H, T, d_k, d_v, qkv_dtype=VLA_F32, has_u=False) -> int:
    return load_library().vla_host_workspace_bytes(B, H, T, d_k, d_v, qkv_dtype, int(has_u))


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return VLA_F32
    if t.dtype == torch.bfloat16:
        return VLA_BF16
    raise TypeError("q, k, v must be float32 or bfloat16, got %s" % t.dtype)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _chk(t, shape, dtype, name, cuda=True):
    if t is None:
        return
    if tuple(t.shape) != tuple(shape):
        raise ValueError("%s: shape %s, expected %s" % (name, tuple(t.shape), tuple(shape)))
    if t.dtype != dtype:
        raise TypeError("%s: dtype %s, expected %s" % (name, t.dtype, dtype))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    if cuda != t.is_cuda:
        raise ValueError("%s must be a %s tensor" % (name, "CUDA" if cuda else "CPU"))


@dataclass
class VlaResult:
    out: torch.Tensor              # [B,H,T,d_v] fp32
    S_T: torch.Tensor              # [B,H,d_v,d_k] fp32
    A_T: torch.Tensor              # [B,H,d_k,d_k] fp32
    z_T: torch.Tensor              # [B,H,d_k] fp32
    status: Optional[torch.Tensor]  # device int32 scalar; read after synchronising


def _make_opts(dt, u, flags, eps, z0, zT, status, kernel, refresh=None, wait_probe_limit=0):
    o = VlaOpts()
    o.struct_size = ctypes.sizeof(VlaOpts)
    o.qkv_dtype = dt
    o.u = None if u is None else u.data_ptr()
    o.flags = flags
    o.eps = eps
    o.z0 = None if z0 is None else z0.data_ptr()
    o.zT = None if zT is None else zT.data_ptr()
    o.status = None if status is None else status.data_ptr()
    o.kernel = kernel
    o.wait_probe_limit = int(wait_probe_limit)
    if refresh is not None:     # (period, eta, step_offset): Algorithm 1's periodic A += eta I
        o.refresh_period, o.refresh_eta, o.step_offset = int(refresh[0]), float(refresh[1]), int(refresh[2])
    return o


def vla_forward(q, k, v, lam: float, *, u=None, S0=None, A0=None, z0=None, flags: int = 0,
                eps: float = 1e-4, out=None, S_T=None, A_T=None, z_T=None, status=None,
                kernel: int = VLA_KERNEL_AUTO, stream: Optional[torch.cuda.Stream] = None,
                want_status: bool = True, refresh=None, workspace=None, wait_probe_limit: int = 0) -> VlaResult:
    """Enqueue the scan for CUDA tensors ``q,k[,u]: [B,H,T,d_k]``, ``v: [B,H,T,d_v]``
    (``[B,T,H,d]`` for all of them and ``out`` with ``VLA_FLAG_TOKEN_MAJOR``).

    Output tensors are allocated with torch unless passed in.  Nothing is synchronised.
    ``workspace``: device scratch the library may use to cut the sequences of a problem with few
    units into concurrently scanned segments (``opts->workspace``); ``True`` allocates what the
    library asks for with torch, ``None`` / ``False`` passes none.
    """
    lib = load_library()
    if q.dim() != 4:
        raise ValueError("q must be [B,H,T,d_k]")
    if flags & VLA_FLAG_TOKEN_MAJOR:
        B, T, H, dk = q.shape
        tok = lambda d_: (B, T, H, d_)
    else:
        B, H, T, dk = q.shape
        tok = lambda d_: (B, H, T, d_)
    dv = v.shape[-1]
    dt = _dtype_code(q)
    dev = q.device
    _chk(q, tok(dk), q.dtype, "q"); _chk(k, tok(dk), q.dtype, "k")
    _chk(v, tok(dv), q.dtype, "v"); _chk(u, tok(dk), q.dtype, "u")
    f32 = torch.float32
    _chk(S0, (B, H, dv, dk), f32, "S0"); _chk(A0, (B, H, dk, dk), f32, "A0")
    _chk(z0, (B, H, dk), f32, "z0")
    if out is None:
        out = torch.empty(tok(dv), dtype=f32, device=dev)
    if S_T is None:
        S_T = torch.empty((B, H, dv, dk), dtype=f32, device=dev)
    if A_T is None:
        A_T = torch.empty((B, H, dk, dk), dtype=f32, device=dev)
    if z_T is None:
        z_T = torch.empty((B, H, dk), dtype=f32, device=dev)
    _chk(out, tok(dv), f32, "out"); _chk(S_T, (B, H, dv, dk), f32, "S_T")
    _chk(A_T, (B, H, dk, dk), f32, "A_T"); _chk(z_T, (B, H, dk), f32, "z_T")
    if status is None and want_status:
        status = torch.zeros((), dtype=torch.int32, device=dev)
    st = stream if stream is not None else torch.cuda.current_stream(dev)
    opts = _make_opts(dt, u, flags, eps, z0, z_T, status, kernel, refresh, wait_probe_limit)
    if workspace is True:
        P = int(lib.vla_seqpar_segments(B, H, T, dk, dt)) if kernel == VLA_KERNEL_AUTO else 1
        workspace = None if P <= 1 else torch.empty((int(lib.vla_seqpar_workspace_bytes(B, H, T, dk, P)),),
                                                    dtype=torch.uint8, device=dev)
    if workspace is not None and workspace is not False:
        opts.workspace, opts.workspace_bytes = workspace.data_ptr(), workspace.numel()
    with torch.cuda.device(dev):
        rc = lib.vla_forward(_ptr(q), _ptr(k), _ptr(v), float(lam), B, H, T, dk, dv,
                             _ptr(S0), _ptr(A0), _ptr(out), _ptr(S_T), _ptr(A_T),
                             ctypes.byref(opts), ctypes.c_void_p(st.cuda_stream))
    if rc != VLA_OK:
        raise VlaError(rc, "vla_forward")
    return VlaResult(out, S_T, A_T, z_T, status)


def backward_workspace_bytes(B: int, H: int, T: int, d_k: int) -> int:
    return int(load_library().vla_backward_workspace_bytes(B, H, T, d_k))


class VlaGrads(NamedTuple):
    dq: torch.Tensor
    dk: torch.Tensor
    dv: torch.Tensor
    dS0: torch.Tensor
    dA0: torch.Tensor
    dz0: torch.Tensor
    status: Optional[torch.Tensor]
    du: Optional[torch.Tensor] = None


def vla_backward(q, k, v, lam: float, d_out, *, u=None, S0=None, A0=None, z0=None, dS_T=None, dA_T=None,
                 dz_T=None, flags: int = 0, eps: float = 1e-4, workspace=None, status=None,
                 stream: Optional[torch.cuda.Stream] = None, want_status: bool = True,
                 refresh=None) -> VlaGrads:
    """Gradients of the forward scan for CUDA tensors (u = k_hat: d in {16, 32, 64, 128}; explicit
    ``u`` (its gradient is returned as ``du``) and / or the periodic ``refresh`` = (period, eta,
    step_offset): d in {32, 64, 128}); the forward is recomputed inside.  ``d_out`` is dL/d(out); ``dS_T, dA_T, dz_T`` default to zero."""
    lib = load_library()
    if flags & VLA_FLAG_TOKEN_MAJOR:      # sequence tensors and their gradients as [B, T, H, d]
        B, T, H, dk = q.shape
        tok = lambda d_: (B, T, H, d_)
    else:
        B, H, T, dk = q.shape
        tok = lambda d_: (B, H, T, d_)
    dv_ = v.shape[-1]
    dt = _dtype_code(q)
    dev = q.device
    f32 = torch.float32
    _chk(q, tok(dk), q.dtype, "q"); _chk(k, tok(dk), q.dtype, "k")
    _chk(v, tok(dv_), q.dtype, "v"); _chk(d_out, tok(dv_), f32, "d_out")
    _chk(u, tok(dk), q.dtype, "u")
    _chk(S0, (B, H, dv_, dk), f32, "S0"); _chk(A0, (B, H, dk, dk), f32, "A0"); _chk(z0, (B, H, dk), f32, "z0")
    _chk(dS_T, (B, H, dv_, dk), f32, "dS_T"); _chk(dA_T, (B, H, dk, dk), f32, "dA_T")
    _chk(dz_T, (B, H, dk), f32, "dz_T")
    dq = torch.empty(tok(dk), dtype=f32, device=dev)
    dkk = torch.empty(tok(dk), dtype=f32, device=dev)
    dvv = torch.empty(tok(dv_), dtype=f32, device=dev)
    dS0 = torch.empty((B, H, dv_, dk), dtype=f32, device=dev)
    dA0 = torch.empty((B, H, dk, dk), dtype=f32, device=dev)
    dz0 = torch.empty((B, H, dk), dtype=f32, device=dev)
    if status is None and want_status:
        status = torch.zeros((), dtype=torch.int32, device=dev)
    st = stream if stream is not None else torch.cuda.current_stream(dev)
    need = int(lib.vla_backward_workspace_bytes(B, H, T, dk))
    if workspace is None:
        workspace = torch.empty((need,), dtype=torch.uint8, device=dev)
    du = None if u is None else torch.empty(tok(dk), dtype=f32, device=dev)
    opts = _make_opts(dt, u, flags, eps, z0, None, status, VLA_KERNEL_AUTO, refresh)
    opts.du = None if du is None else du.data_ptr()
    with torch.cuda.device(dev):
        rc = lib.vla_backward(_ptr(q), _ptr(k), _ptr(v), float(lam), B, H, T, dk, dv_, _ptr(S0), _ptr(A0),
                              _ptr(d_out), _ptr(dS_T), _ptr(dA_T), _ptr(dz_T), _ptr(dq), _ptr(dkk),
                              _ptr(dvv), _ptr(dS0), _ptr(dA0), _ptr(dz0), ctypes.byref(opts),
                              _ptr(workspace), workspace.numel(), ctypes.c_void_p(st.cuda_stream))
    if rc != VLA_OK:
        raise VlaError(rc, "vla_backward")
    return VlaGrads(dq, dkk, dvv, dS0, dA0, dz0, status, du)


def measure_fp32_fma_tflops(device=None, iters: int = 4096, reps: int = 5) -> float:
    """fp32 FMA rate of the device at its current clocks (register-only loop, best of ``reps``)."""
    lib = load_library()
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    sink = torch.zeros((4,), dtype=torch.float32, device=dev)
    flops = ctypes.c_double(0.0)
    best = 0.0
    with torch.cuda.device(dev):
        st = torch.cuda.current_stream(dev)
        for r in range(reps + 1):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(st)
            rc = lib.vla_probe_fp32_fma(int(iters), _ptr(sink), ctypes.byref(flops),
                                        ctypes.c_void_p(st.cuda_stream))
            b.record(st)
            if rc != VLA_OK:
                raise VlaError(rc, "vla_probe_fp32_fma")
            b.synchronize()
            if r > 0:
                best = max(best, flops.value / (a.elapsed_time(b) * 1e-3) / 1e12)
    return best


def seqpar_segments(B: int, H: int, T: int, d_k: int, dtype: torch.dtype) -> int:
    """Segments per unit that ``vla_forward_seqpar`` would choose on the current device."""
    code = VLA_BF16 if dtype == torch.bfloat16 else VLA_F32
    return int(load_library().vla_seqpar_segments(B, H, T, d_k, code))


def seqpar_workspace_bytes(B: int, H: int, T: int, d_k: int, segments: int) -> int:
    return int(load_library().vla_seqpar_workspace_bytes(B, H, T, d_k, segments))


def vla_forward_seqpar(q, k, v, lam: float, *, segments: int = 0, workspace=None, u=None, S0=None,
                       A0=None, z0=None, flags: int = 0, eps: float = 1e-4, out=None, S_T=None, A_T=None,
                       z_T=None, status=None, stream: Optional[torch.cuda.Stream] = None,
                       want_status: bool = True) -> VlaResult:
    """Sequence-parallel scan of CUDA tensors: each unit's sequence is cut into ``segments``
    pieces that are scanned concurrently (0 = let the library choose).  ``workspace`` is a CUDA
    uint8 tensor of at least ``seqpar_workspace_bytes`` bytes (allocated with torch if absent)."""
    lib = load_library()
    if q.dim() != 4:
        raise ValueError("q must be [B,H,T,d_k]")
    B, H, T, dk = q.shape
    dv = v.shape[-1]
    dt = _dtype_code(q)
    dev = q.device
    _chk(q, (B, H, T, dk), q.dtype, "q"); _chk(k, (B, H, T, dk), q.dtype, "k")
    _chk(v, (B, H, T, dv), q.dtype, "v"); _chk(u, (B, H, T, dk), q.dtype, "u")
    f32 = torch.float32
    _chk(S0, (B, H, dv, dk), f32, "S0"); _chk(z0, (B, H, dk), f32, "z0")
    _chk(A0, (B, H, dk, dk), f32, "A0")
    if out is None:
        out = torch.empty((B, H, T, dv), dtype=f32, device=dev)
    if S_T is None:
        S_T = torch.empty((B, H, dv, dk), dtype=f32, device=dev)
    if A_T is None:
        A_T = torch.empty((B, H, dk, dk), dtype=f32, device=dev)
    if z_T is None:
        z_T = torch.empty((B, H, dk), dtype=f32, device=dev)
    _chk(out, (B, H, T, dv), f32, "out"); _chk(S_T, (B, H, dv, dk), f32, "S_T")
    _chk(A_T, (B, H, dk, dk), f32, "A_T"); _chk(z_T, (B, H, dk), f32, "z_T")
    if status is None and want_status:
        status = torch.zeros((), dtype=torch.int32, device=dev)
    st = stream if stream is not None else torch.cuda.current_stream(dev)
    with torch.cuda.device(dev):
        P = segments if segments > 0 else int(lib.vla_seqpar_segments(B, H, T, dk, dt))
        need = int(lib.vla_seqpar_workspace_bytes(B, H, T, dk, max(P, 1)))
        if workspace is None:
            workspace = torch.empty((need,), dtype=torch.uint8, device=dev)
        if workspace.device != dev or workspace.dtype != torch.uint8 or not workspace.is_contiguous():
            raise ValueError("workspace must be a contiguous CUDA uint8 tensor on the inputs' device")
        opts = _make_opts(dt, u, flags, eps, z0, z_T, status, VLA_KERNEL_AUTO, None)
        rc = lib.vla_forward_seqpar(_ptr(q), _ptr(k), _ptr(v), float(lam), B, H, T, dk, dv,
                                    _ptr(S0), _ptr(A0), _ptr(out), _ptr(S_T), _ptr(A_T), ctypes.byref(opts),
                                    int(segments), _ptr(workspace), workspace.numel(),
                                    ctypes.c_void_p(st.cuda_stream))
    if rc != VLA_OK:
        raise VlaError(rc, "vla_forward_seqpar")
    return VlaResult(out, S_T, A_T, z_T, status)


def vla_forward_host(q, k, v, lam: float, workspace: torch.Tensor, *, u=None, S0=None, A0=None,
                     z0=None, flags: int = 0, eps: float = 1e-4, out=None, S_T=None, A_T=None,
                     z_T=None, status=None, kernel: int = VLA_KERNEL_AUTO,
                     stream: Optional[torch.cuda.Stream] = None) -> VlaResult:
    """The same for HOST tensors (pinned for asynchronous copies); ``workspace`` is a CUDA
    uint8 tensor of at least ``vla_host_workspace_bytes(...)`` bytes.  Copies in, the scan
    and copies out are enqueued on the stream; synchronise it before reading the results."""
    lib = load_library()
    if flags & VLA_FLAG_TOKEN_MAJOR:          # q, k, v, u, out are [B,T,H,d]
        B, T, H, dk = q.shape
        tok = lambda d_: (B, T, H, d_)
    else:
        B, H, T, dk = q.shape
        tok = lambda d_: (B, H, T, d_)
    dv = v.shape[-1]
    dt = _dtype_code(q)
    f32 = torch.float32
    _chk(q, tok(dk), q.dtype, "q", cuda=False); _chk(k, tok(dk), q.dtype, "k", cuda=False)
    _chk(v, tok(dv), q.dtype, "v", cuda=False); _chk(u, tok(dk), q.dtype, "u", cuda=False)
    _chk(S0, (B, H, dv, dk), f32, "S0", cuda=False); _chk(A0, (B, H, dk, dk), f32, "A0", cuda=False)
    _chk(z0, (B, H, dk), f32, "z0", cuda=False)
    pin = torch.cuda.is_available()
    mk = lambda shape: torch.empty(shape, dtype=f32, pin_memory=pin)
    out = mk(tok(dv)) if out is None else out
    S_T = mk((B, H, dv, dk)) if S_T is None else S_T
    A_T = mk((B, H, dk, dk)) if A_T is None else A_T
    z_T = mk((B, H, dk)) if z_T is None else z_T
    _chk(out, tok(dv), f32, "out", cuda=False); _chk(S_T, (B, H, dv, dk), f32, "S_T", cuda=False)
    _chk(A_T, (B, H, dk, dk), f32, "A_T", cuda=False); _chk(z_T, (B, H, dk), f32, "z_T", cuda=False)
    if not workspace.is_cuda or workspace.dtype != torch.uint8 or not workspace.is_contiguous():
        raise ValueError("workspace must be a contiguous CUDA uint8 tensor")
    dev = workspace.device
    st = stream if stream is not None else torch.cuda.current_stream(dev)
    opts = _make_opts(dt, u, flags, eps, z0, z_T, status, kernel)
    with torch.cuda.device(dev):
        rc = lib.vla_forward_host(_ptr(q), _ptr(k), _ptr(v), float(lam), B, H, T, dk, dv,
                                  _ptr(S0), _ptr(A0), _ptr(out), _ptr(S_T), _ptr(A_T),
                                  ctypes.byref(opts), _ptr(workspace), workspace.numel(),
                                  ctypes.c_void_p(st.cuda_stream))
    if rc != VLA_OK:
        raise VlaError(rc, "vla_forward_host")
    return VlaResult(out, S_T, A_T, z_T, status)


def vla_forward_host_static(q, k, v, lam: float, *, u=None, S0=None, A0=None, z0=None,
                            flags: int = 0, eps: float = 1e-4, out=None, S_T=None, A_T=None,
                            z_T=None, status=None, kernel: int = VLA_KERNEL_AUTO,
                            device=None, stream: Optional[torch.cuda.Stream] = None) -> VlaResult:
    """``vla_forward_host`` without a workspace argument: the staging memory is the library's
    built-in device array (``VLA_STATIC_SCRATCH_BYTES``), so the call allocates nothing on the
    device.  For callers that hold host tensors and a stream but cannot get device memory
    where they stand (no allocator handle, a committed memory cap, a loop that must not
    allocate).  Problems whose staging need exceeds the array raise ``VLA_ERR_TOO_LARGE``.
    Calls on one device share the array: do not let two of them overlap on the GPU."""
    lib = load_library()
    if flags & VLA_FLAG_TOKEN_MAJOR:          # q, k, v, u, out are [B,T,H,d]
        B, T, H, dk = q.shape
        tok = lambda d_: (B, T, H, d_)
    else:
        B, H, T, dk = q.shape
        tok = lambda d_: (B, H, T, d_)
    dv = v.shape[-1]
    dt = _dtype_code(q)
    f32 = torch.float32
    _chk(q, tok(dk), q.dtype, "q", cuda=False); _chk(k, tok(dk), q.dtype, "k", cuda=False)
    _chk(v, tok(dv), q.dtype, "v", cuda=False); _chk(u, tok(dk), q.dtype, "u", cuda=False)
    _chk(S0, (B, H, dv, dk), f32, "S0", cuda=False); _chk(A0, (B, H, dk, dk), f32, "A0", cuda=False)
    _chk(z0, (B, H, dk), f32, "z0", cuda=False)
    pin = torch.cuda.is_available()
    mk = lambda shape: torch.empty(shape, dtype=f32, pin_memory=pin)
    out = mk(tok(dv)) if out is None else out
    S_T = mk((B, H, dv, dk)) if S_T is None else S_T
    A_T = mk((B, H, dk, dk)) if A_T is None else A_T
    z_T = mk((B, H, dk)) if z_T is None else z_T
    _chk(out, tok(dv), f32, "out", cuda=False); _chk(S_T, (B, H, dv, dk), f32, "S_T", cuda=False)
    _chk(A_T, (B, H, dk, dk), f32, "A_T", cuda=False); _chk(z_T, (B, H, dk), f32, "z_T", cuda=False)
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    st = stream if stream is not None else torch.cuda.current_stream(dev)
    opts = _make_opts(dt, u, flags, eps, z0, z_T, status, kernel)
    with torch.cuda.device(dev):
        rc = lib.vla_forward_host_static(_ptr(q), _ptr(k), _ptr(v), float(lam), B, H, T, dk, dv,
                                         _ptr(S0), _ptr(A0), _ptr(out), _ptr(S_T), _ptr(A_T),
                                         ctypes.byref(opts), ctypes.c_void_p(st.cuda_stream))
    if rc != VLA_OK:
        raise VlaError(rc, "vla_forward_host_static")
    return VlaResult(out, S_T, A_T, z_T, status)
