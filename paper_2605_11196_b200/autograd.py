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


class _VlaScan(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, u, S0, A0, z0, lam, flags, eps, refresh):
        r = _b.vla_forward(q, k, v, lam, u=u, S0=S0, A0=A0, z0=z0, flags=flags, eps=eps, refresh=refresh,
                           want_status=False)
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
                            want_status=False)
        need = ctx.needs_input_grad
        pick = lambda i, x, like: x.to(like.dtype) if (need[i] and x is not None and like is not None) else None
        return (pick(0, g.dq, q), pick(1, g.dk, k), pick(2, g.dv, v), pick(3, g.du, u), pick(4, g.dS0, S0),
                pick(5, g.dA0, A0), pick(6, g.dz0, z0), None, None, None, None)


def vla_scan(q, k, v, lam: float, *, u: Optional[torch.Tensor] = None, S0=None, A0=None, z0=None,
             flags: int = 0, eps: float = 1e-4, refresh=None):
    """``(out, S_T, A_T, z_T)`` of the VLA forward scan for CUDA tensors, differentiable with
    respect to ``q, k, v, u, S0, A0, z0``."""
    return _VlaScan.apply(q, k, v, u, S0, A0, z0, float(lam), int(flags), float(eps), refresh)
