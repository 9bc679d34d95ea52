"""Shared helpers of the GPU parity tests: run the CUDA path and the CPU oracle on the
same seeded inputs and compare element by element."""
import os

import numpy as np
import torch

import oracle
import paper_2605_11196_b200 as vla
from paper_2605_11196_b200 import workloads as W

NTHREADS = max(1, len(os.sched_getaffinity(0)))


def to_oracle_array(t: torch.Tensor):
    """Storage-exact view for the oracle: fp32 as is, bf16 as uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16), oracle.BF16
    return t.numpy(), oracle.F32


def run_oracle(q, k, v, lam, u=None, S0=None, A0=None, z0=None, flags=0, eps=1e-4, refresh=None):
    qa, dt = to_oracle_array(q)
    ka, _ = to_oracle_array(k)
    va, _ = to_oracle_array(v)
    ua = None if u is None else to_oracle_array(u)[0]
    f64 = lambda x: None if x is None else x.detach().cpu().double().numpy()
    # the library's flag bits -> the oracle's (it knows the two that change the arithmetic)
    flags = (oracle.IDENTITY_MAP if flags & vla.VLA_FLAG_IDENTITY_MAP else 0) | \
            (oracle.LINEAR_ATTENTION if flags & vla.VLA_FLAG_LINEAR_ATTENTION else 0)
    return oracle.forward(qa, ka, va, lam, u=ua, in_dtype=dt, S0=f64(S0), A0=f64(A0), z0=f64(z0),
                          flags=flags, eps=eps, n_threads=NTHREADS, refresh=refresh)


def rel_err(x_gpu: torch.Tensor, x_ref: np.ndarray) -> float:
    """max|x_gpu - x_ref| / max|x_ref| over the whole tensor."""
    x = x_gpu.detach().cpu().double().numpy()
    assert x.shape == x_ref.shape, (x.shape, x_ref.shape)
    if x_ref.size == 0:
        return 0.0
    assert np.all(np.isfinite(x)), "non-finite value from the CUDA path"
    den = np.abs(x_ref).max()
    return float(np.abs(x - x_ref).max() / (den if den > 0 else 1.0))


def run_gpu(q, k, v, lam, u=None, S0=None, A0=None, z0=None, flags=0, eps=1e-4, kernel=0, refresh=None):
    dev = torch.device("cuda:0")
    mv = lambda x: None if x is None else x.to(dev).contiguous()
    r = vla.vla_forward(mv(q), mv(k), mv(v), lam, u=mv(u), S0=mv(S0), A0=mv(A0), z0=mv(z0),
                        flags=flags, eps=eps, kernel=kernel, refresh=refresh)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0, vla.status_string(int(r.status.item()))
    return r


def check_parity(q, k, v, lam, tol, *, u=None, S0=None, A0=None, z0=None, flags=0, eps=1e-4,
                 kernel=0, label="", refresh=None):
    ref = run_oracle(q, k, v, lam, u, S0, A0, z0, flags, eps, refresh)
    got = run_gpu(q, k, v, lam, u, S0, A0, z0, flags, eps, kernel, refresh)
    errs = {"o": rel_err(got.out, ref.out), "S_T": rel_err(got.S_T, ref.S_T),
            "A_T": rel_err(got.A_T, ref.A_T), "z_T": rel_err(got.z_T, ref.z_T)}
    for name, e in errs.items():
        assert e <= tol, "%s %s: rel err %.3e > %.1e (%s)" % (label, name, e, tol, errs)
    return errs, got, ref
