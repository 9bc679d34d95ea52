"""``torch.autograd`` face of the scan: ``vla_scan`` runs ``vla_forward`` and, under autograd,
``vla_backward``.  Marshalling only; every step of both passes runs in the CUDA library.

Differentiable inputs: ``q, k, v``, explicit penalty directions ``u`` (so a learned
``u = L2norm(W_u k) / sqrt(d)`` built with torch ops, or with ``vla_make_u`` outside autograd,
trains through it), and the carried states ``S0, A0, z0``.  Outputs ``(out, S_T, A_T, z_T)``;
gradients may flow into any of them.  Head-major ``[B,H,T,d]`` or, with
``VLA_FLAG_TOKEN_MAJOR``, ``[B,T,H,d]`` tensors; ``d >= 32`` for explicit ``u``, the refresh and
token-major tensors (the limits of ``vla_backward``).
"""
from typing import Optional

import torch

from . import binding as _b

# One device-side status word per device, shared by every forward and backward call made through
# vla_scan: the kernels record a device-side problem in it (a bounded wait that ran out, a
# non-finite value with VLA_FLAG_CHECK_FINITE); nothing here reads it back, so no call
# synchronises.  check_status() reads and clears it.
_status = {}


def _status_word(device: torch.device) -> torch.Tensor:
    key = (device.type, device.index if device.index is not None else torch.cuda.current_device())
    if key not in _status:
        _status[key] = torch.zeros((), dtype=torch.int32, device=device)
    return _status[key]


def check_status(device=None) -> None:
    """Synchronise `device` and raise ``VlaError`` if any ``vla_scan`` forward or backward pass on it
    has reported a device-side problem since the last check (the word is cleared)."""
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    word = _status_word(device)
    code = int(word.item())
    if code != 0:
        word.zero_()
        raise _b.VlaError(code, "vla_scan (device-side status)")


class _VlaScan(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, u, S0, A0, z0, lam, flags, eps, refresh):
        r = _b.vla_forward(q, k, v, lam, u=u, S0=S0, A0=A0, z0=z0, flags=flags, eps=eps, refresh=refresh,
                           status=_status_word(q.device))
        ctx.save_for_backward(q, k, v, u, S0, A0, z0)
        ctx.args = (lam, flags, eps, refresh)
        return r.out, r.S_T, r.A_T, r.z_T

    @staticmethod
    def backward(ctx, d_out, dS_T, dA_T, dz_T):
        q, k, v, u, S0, A0, z0 = ctx.saved_tensors
        lam, flags, eps, refresh = ctx.args
        f32c = lambda x: None if x is None else x.to(torch.float32).contiguous()
        if d_out is None:
            d_out = torch.zeros(v.shape, dtype=torch.float32, device=v.device)
        g = _b.vla_backward(q, k, v, lam, f32c(d_out), u=u, S0=S0, A0=A0, z0=z0, dS_T=f32c(dS_T),
                            dA_T=f32c(dA_T), dz_T=f32c(dz_T), flags=flags, eps=eps, refresh=refresh,
                            status=_status_word(q.device))
        need = ctx.needs_input_grad
        pick = lambda i, x, like: x.to(like.dtype) if (need[i] and x is not None and like is not None) else None
        return (pick(0, g.dq, q), pick(1, g.dk, k), pick(2, g.dv, v), pick(3, g.du, u), pick(4, g.dS0, S0),
                pick(5, g.dA0, A0), pick(6, g.dz0, z0), None, None, None, None)


def vla_scan(q, k, v, lam: float, *, u: Optional[torch.Tensor] = None, S0=None, A0=None, z0=None,
             flags: int = 0, eps: float = 1e-4, refresh=None):
    """``(out, S_T, A_T, z_T)`` of the VLA forward scan for CUDA tensors, differentiable with
    respect to ``q, k, v, u, S0, A0, z0``.  Device-side problems of either pass land in a status
    word that ``check_status()`` reads (the calls themselves never synchronise)."""
    return _VlaScan.apply(q, k, v, u, S0, A0, z0, float(lam), int(flags), float(eps), refresh)
