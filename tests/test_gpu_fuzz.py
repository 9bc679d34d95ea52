"""Seeded random walks over the call surface: shapes, layouts, options and kernels drawn at
random, every call compared with the fp64 oracles.  The cases are fixed by their seeds."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_11196_b200 as vla
from paper_2605_11196_b200 import workloads as W
from parity_util import NTHREADS, rel_err, run_oracle, to_oracle_array

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _seeds(default):
    """Seeds per test; VLA_FUZZ_SEEDS=N runs N of each (a longer hunt, by hand)."""
    import os
    return int(os.environ.get("VLA_FUZZ_SEEDS", default))


def _draw(rng):
    d = int(rng.choice([16, 32, 64, 128]))
    B, H = int(rng.integers(1, 4)), int(rng.integers(1, 6))
    if rng.random() < 0.25:     # more units than one wave of CTAs: schedules that cut units, late A sides
        B, H = 1, int(rng.choice([37, 151, 307]))
    T = int(rng.choice([1, 3, 15, 16, 17, 31, 33, 48, 70, 129, 200]))
    dtype = str(rng.choice(["f32", "bf16"]))
    flags = int(rng.choice([0, vla.VLA_FLAG_IDENTITY_MAP]))
    lam = float(rng.choice([0.1, 0.5, 1.0, 3.0]))
    return d, B, H, T, dtype, flags, lam


def _states(rng, B, H, d, seed):
    g = torch.Generator().manual_seed(seed)
    S0 = torch.randn((B, H, d, d), generator=g) * 0.1 if rng.random() < 0.5 else None
    z0 = torch.rand((B, H, d), generator=g) + 0.05 if rng.random() < 0.5 else None
    A0 = None
    if rng.random() < 0.4:
        h = torch.randn((B, H, d, d), generator=g) * 0.1
        A0 = h @ h.transpose(-1, -2) + 0.4 * torch.eye(d)
    return S0, A0, z0


@pytest.mark.parametrize("seed", range(_seeds(40)))
def test_forward_random_calls(seed):
    rng = np.random.default_rng(1000 + seed)
    d, B, H, T, dtype, flags, lam = _draw(rng)
    w = W.Workload("f", B, H, d, T, dtype, 5000 + seed)
    q, k, v = W.make_inputs(w)
    u = W.make_u(w, float(rng.choice([1.0, d ** -0.5]))) if rng.random() < 0.4 else None
    refresh = (int(rng.integers(1, 25)), float(rng.choice([1e-3, 1e-2])), int(rng.integers(0, 30))) \
        if rng.random() < 0.3 else None
    S0, A0, z0 = _states(rng, B, H, d, seed)
    kernel = int(rng.choice([vla.VLA_KERNEL_AUTO, vla.VLA_KERNEL_TOKEN, vla.VLA_KERNEL_CHUNK]))
    if d == 16 and kernel == vla.VLA_KERNEL_CHUNK:
        kernel = vla.VLA_KERNEL_AUTO
    tmaj = rng.random() < 0.4
    ref = run_oracle(q, k, v, lam, u=u, S0=S0, A0=A0, z0=z0, flags=flags, refresh=refresh)
    mv = lambda x: None if x is None else x.to(DEV)
    tm = (lambda x: None if x is None else x.permute(0, 2, 1, 3).contiguous().to(DEV)) if tmaj else mv
    r = vla.vla_forward(tm(q), tm(k), tm(v), lam, u=tm(u), S0=mv(S0), A0=mv(A0), z0=mv(z0), kernel=kernel,
                        flags=flags | (vla.VLA_FLAG_TOKEN_MAJOR if tmaj else 0), refresh=refresh)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    out = r.out.permute(0, 2, 1, 3) if tmaj else r.out
    label = "seed %d: d=%d B=%d H=%d T=%d %s flags=%d u=%s refresh=%s kernel=%d tm=%s" % (
        seed, d, B, H, T, dtype, flags, u is not None, refresh, kernel, tmaj)
    for name, got, want in (("o", out, ref.out), ("S_T", r.S_T, ref.S_T), ("A_T", r.A_T, ref.A_T),
                            ("z_T", r.z_T, ref.z_T)):
        e = rel_err(got, want)
        assert e <= 1e-4, "%s %s rel err %.3e" % (label, name, e)


@pytest.mark.parametrize("seed", range(_seeds(24)))
def test_tc_random_calls(seed):
    """The tensor-core kernel, forced: unit counts on both schedules, ragged lengths, both input
    types and readings, carried states, either layout."""
    rng = np.random.default_rng(3000 + seed)
    B, H = (int(rng.integers(1, 4)), int(rng.integers(1, 6))) if rng.random() < 0.6 else (1, int(rng.choice([149, 163, 301])))
    T = int(rng.choice([1, 5, 16, 17, 47, 64, 130, 257, 600]))
    if B * H > 100:
        T = min(T, 130)
    dtype = str(rng.choice(["f32", "bf16"]))
    flags = int(rng.choice([0, vla.VLA_FLAG_IDENTITY_MAP]))
    lam = float(rng.choice([0.1, 0.5, 1.0, 3.0]))
    w = W.Workload("f", B, H, 128, T, dtype, 7000 + seed)
    q, k, v = W.make_inputs(w)
    S0, A0, z0 = _states(rng, B, H, 128, seed)
    tmaj = rng.random() < 0.4
    sel = list(range(H)) if B * H <= 100 else sorted(set(int(x) for x in rng.integers(0, H, 6)) | {0, H - 1})
    pick = lambda x: None if x is None else x[:, sel].contiguous()
    ref = run_oracle(pick(q), pick(k), pick(v), lam, S0=pick(S0), A0=pick(A0), z0=pick(z0), flags=flags)
    mv = lambda x: None if x is None else x.to(DEV)
    tm = (lambda x: None if x is None else x.permute(0, 2, 1, 3).contiguous().to(DEV)) if tmaj else mv
    r = vla.vla_forward(tm(q), tm(k), tm(v), lam, S0=mv(S0), A0=mv(A0), z0=mv(z0), kernel=vla.VLA_KERNEL_CHUNK_TC,
                        flags=flags | (vla.VLA_FLAG_TOKEN_MAJOR if tmaj else 0))
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    out = r.out.permute(0, 2, 1, 3) if tmaj else r.out
    label = "seed %d: B=%d H=%d T=%d %s flags=%d lam=%g tm=%s %s" % (seed, B, H, T, dtype, flags, lam, tmaj, vla.last_launch())
    for name, got, want in (("o", out[:, sel], ref.out), ("S_T", r.S_T[:, sel], ref.S_T), ("A_T", r.A_T[:, sel], ref.A_T),
                            ("z_T", r.z_T[:, sel], ref.z_T)):
        e = rel_err(got, want)
        assert e <= 1e-4, "%s %s rel err %.3e" % (label, name, e)


@pytest.mark.parametrize("seed", range(_seeds(30)))
def test_backward_random_calls(seed):
    rng = np.random.default_rng(2000 + seed)
    d, B, H, T, dtype, flags, lam = _draw(rng)
    w = W.Workload("f", B, H, d, T, dtype, 6000 + seed)
    q, k, v = W.make_inputs(w)
    general_ok = d >= 32
    u = W.make_u(w, float(rng.choice([1.0, d ** -0.5]))) if general_ok and rng.random() < 0.4 else None
    refresh = (int(rng.integers(1, 25)), float(rng.choice([1e-3, 1e-2])), int(rng.integers(0, 30))) \
        if general_ok and rng.random() < 0.3 else None
    tmaj = general_ok and rng.random() < 0.4
    S0, A0, z0 = _states(rng, B, H, d, seed)
    g = torch.Generator().manual_seed(seed)
    d_out = torch.randn((B, H, T, d), generator=g)
    dS_T = torch.randn((B, H, d, d), generator=g) if rng.random() < 0.5 else None
    dA_T = torch.randn((B, H, d, d), generator=g) if rng.random() < 0.5 else None
    dz_T = torch.randn((B, H, d), generator=g) if rng.random() < 0.5 else None
    f64 = lambda x: None if x is None else x.detach().cpu().double().numpy()
    qa, dt = to_oracle_array(q)
    ref = oracle.backward(qa, to_oracle_array(k)[0], to_oracle_array(v)[0], lam, f64(d_out),
                          u=None if u is None else to_oracle_array(u)[0], in_dtype=dt, S0=f64(S0), A0=f64(A0),
                          z0=f64(z0), dS_T=f64(dS_T), dA_T=f64(dA_T), dz_T=f64(dz_T), flags=flags,
                          n_threads=NTHREADS, refresh=refresh)
    mv = lambda x: None if x is None else x.to(DEV)
    tm = (lambda x: None if x is None else x.permute(0, 2, 1, 3).contiguous().to(DEV)) if tmaj else mv
    r = vla.vla_backward(tm(q), tm(k), tm(v), lam, tm(d_out), u=tm(u), S0=mv(S0), A0=mv(A0), z0=mv(z0),
                         dS_T=mv(dS_T), dA_T=mv(dA_T), dz_T=mv(dz_T), refresh=refresh,
                         flags=flags | (vla.VLA_FLAG_TOKEN_MAJOR if tmaj else 0))
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    back = (lambda x: x.permute(0, 2, 1, 3)) if tmaj else (lambda x: x)
    label = "seed %d: d=%d B=%d H=%d T=%d %s flags=%d u=%s refresh=%s tm=%s" % (
        seed, d, B, H, T, dtype, flags, u is not None, refresh, tmaj)
    pairs = [("dq", back(r.dq), ref.dq), ("dk", back(r.dk), ref.dk), ("dv", back(r.dv), ref.dv),
             ("dS0", r.dS0, ref.dS0), ("dA0", r.dA0, ref.dA0), ("dz0", r.dz0, ref.dz0)]
    if u is not None:
        pairs.append(("du", back(r.du), ref.du))
    for name, got, want in pairs:
        x = got.detach().cpu().double().numpy()
        assert np.all(np.isfinite(x))
        e = float(np.abs(x - want).max() / max(np.abs(want).max(), 1e-3))
        assert e <= 3e-4, "%s %s rel err %.3e" % (label, name, e)


@pytest.mark.parametrize("seed", range(_seeds(20)))
def test_seqpar_random_calls(seed):
    rng = np.random.default_rng(3000 + seed)
    d = int(rng.choice([32, 64, 128]))
    B, H = int(rng.integers(1, 3)), int(rng.integers(1, 5))
    P = int(rng.choice([2, 3, 4, 8]))
    T = 16 * P * int(rng.integers(1, 5))
    dtype = str(rng.choice(["f32", "bf16"]))
    flags = int(rng.choice([0, vla.VLA_FLAG_IDENTITY_MAP]))
    lam = float(rng.choice([0.1, 1.0, 3.0]))
    w = W.Workload("f", B, H, d, T, dtype, 7000 + seed)
    q, k, v = W.make_inputs(w)
    u = W.make_u(w, float(rng.choice([1.0, d ** -0.5]))) if rng.random() < 0.4 else None
    S0, A0, z0 = _states(rng, B, H, d, seed)
    ref = run_oracle(q, k, v, lam, u=u, S0=S0, A0=A0, z0=z0, flags=flags)
    mv = lambda x: None if x is None else x.to(DEV)
    r = vla.vla_forward_seqpar(mv(q), mv(k), mv(v), lam, segments=P, u=mv(u), S0=mv(S0), A0=mv(A0), z0=mv(z0),
                               flags=flags)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    label = "seed %d: d=%d B=%d H=%d T=%d P=%d %s flags=%d u=%s" % (seed, d, B, H, T, P, dtype, flags, u is not None)
    for name, got, want in (("o", r.out, ref.out), ("S_T", r.S_T, ref.S_T), ("A_T", r.A_T, ref.A_T),
                            ("z_T", r.z_T, ref.z_T)):
        e = rel_err(got, want)
        assert e <= 1e-4, "%s %s rel err %.3e" % (label, name, e)
