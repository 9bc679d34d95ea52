"""Backward kernel (vla_backward) against the fp64 backward oracle, which is itself pinned by
finite differences of the forward oracle (tests/test_oracle_bwd_pins.py)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_11196_b200 as vla
from paper_2605_11196_b200 import workloads as W
from parity_util import NTHREADS, rel_err, to_oracle_array

pytestmark = pytest.mark.gpu
IDENT = vla.VLA_FLAG_IDENTITY_MAP


def _small(d, T, dtype, units=(1, 2), seed=1):
    return W.Workload("t", units[0], units[1], d, T, dtype, seed)


def _run_both(q, k, v, lam, d_out, flags=0, S0=None, A0=None, z0=None, dS_T=None, dA_T=None, dz_T=None, u=None,
              refresh=None):
    dev = torch.device("cuda:0")
    mv = lambda x: None if x is None else x.to(dev).contiguous()
    g = vla.vla_backward(mv(q), mv(k), mv(v), lam, mv(d_out), u=mv(u), S0=mv(S0), A0=mv(A0), z0=mv(z0),
                         dS_T=mv(dS_T), dA_T=mv(dA_T), dz_T=mv(dz_T), flags=flags, refresh=refresh)
    torch.cuda.synchronize()
    assert int(g.status.item()) == 0
    qa, dt = to_oracle_array(q)
    ka, _ = to_oracle_array(k)
    va, _ = to_oracle_array(v)
    f64 = lambda x: None if x is None else x.detach().cpu().double().numpy()
    ua = None if u is None else to_oracle_array(u)[0]
    ref = oracle.backward(qa, ka, va, lam, f64(d_out), u=ua, in_dtype=dt, S0=f64(S0), A0=f64(A0), z0=f64(z0),
                          dS_T=f64(dS_T), dA_T=f64(dA_T), dz_T=f64(dz_T), flags=flags, n_threads=NTHREADS,
                          refresh=refresh)
    return g, ref


def _err(x_gpu, x_ref):
    """max|x - ref| / max|ref|, with a floor on the denominator: a gradient that is exactly
    zero in exact arithmetic (dq of a single token written into an empty memory) comes out as
    rounding noise on both sides."""
    x = x_gpu.detach().cpu().double().numpy()
    assert x.shape == x_ref.shape and np.all(np.isfinite(x))
    return float(np.abs(x - x_ref).max() / max(np.abs(x_ref).max(), 1e-3)) if x_ref.size else 0.0


def _check(g, ref, tol, label):
    errs = {"dq": _err(g.dq, ref.dq), "dk": _err(g.dk, ref.dk), "dv": _err(g.dv, ref.dv),
            "dS0": _err(g.dS0, ref.dS0), "dA0": _err(g.dA0, ref.dA0), "dz0": _err(g.dz0, ref.dz0)}
    if ref.du is not None:
        errs["du"] = _err(g.du, ref.du)
    for name, e in errs.items():
        assert e <= tol, "%s %s: rel err %.3e > %.1e (%s)" % (label, name, e, tol, errs)
    return errs


@pytest.mark.parametrize("d", [16, 32, 64, 128])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [0, IDENT])
@pytest.mark.parametrize("T", [1, 7, 64, 200])
def test_gradients_agree_with_the_backward_oracle(d, dtype, flags, T):
    w = _small(d, T, dtype, units=(2, 3), seed=3000 + d + T)
    q, k, v = W.make_inputs(w)
    g = torch.Generator().manual_seed(d * 7 + T)
    d_out = torch.randn((2, 3, T, d), generator=g)
    for lam in (1.0, 0.1):
        got, ref = _run_both(q, k, v, lam, d_out, flags=flags)
        _check(got, ref, 2e-4, "backward d=%d T=%d lam=%g" % (d, T, lam))


@pytest.mark.parametrize("d", [16, 32, 64, 128])
@pytest.mark.parametrize("flags", [0, IDENT])
def test_carried_states_and_incoming_state_gradients(d, flags):
    w = _small(d, 96, "f32", units=(1, 4), seed=3100 + d)
    q, k, v = W.make_inputs(w)
    g = torch.Generator().manual_seed(d)
    shape = (1, 4)
    S0 = torch.randn(shape + (d, d), generator=g) * 0.2
    h = torch.randn(shape + (d, d), generator=g) * 0.1
    A0 = h @ h.transpose(-1, -2) + 0.5 * torch.eye(d)
    z0 = torch.rand(shape + (d,), generator=g) + 0.1
    d_out = torch.randn(shape + (96, d), generator=g)
    dS_T = torch.randn(shape + (d, d), generator=g)
    dA_T = torch.randn(shape + (d, d), generator=g)
    dz_T = torch.randn(shape + (d,), generator=g)
    got, ref = _run_both(q, k, v, 0.5, d_out, flags=flags, S0=S0, A0=A0, z0=z0, dS_T=dS_T, dA_T=dA_T, dz_T=dz_T)
    _check(got, ref, 2e-4, "backward carried d=%d" % d)


def test_mid_workload_gradients_and_what_is_not_covered():
    """The `mid` workload (32 units, d = 64, T = 4096) whole, and a shape without kernels."""
    w = W.WORKLOADS["mid"]
    q, k, v = W.make_inputs(w)
    g = torch.Generator().manual_seed(11)
    d_out = torch.randn((w.B, w.H, w.T, w.d), generator=g)
    got, ref = _run_both(q, k, v, w.lam, d_out)
    print("mid backward", _check(got, ref, 1e-3, "backward mid"))
    dev = torch.device("cuda:0")
    w48 = _small(48, 16, "f32")
    q, k, v = [x.to(dev) for x in W.make_inputs(w48)]
    with pytest.raises(vla.VlaError) as ei:
        vla.vla_backward(q, k, v, 1.0, torch.zeros((1, 2, 16, 48), device=dev))
    assert ei.value.code == vla.VLA_ERR_UNSUPPORTED


@pytest.mark.parametrize("flags", [0, IDENT])
def test_throughput_shape_sampled_units(flags):
    """Units of the headline shape (d = 128, T = 8192, bf16), whole sequences: the longest walk
    back through undone updates the workloads ask for.  Three units (the oracle's fp64 reverse
    pass takes seconds per unit); the kernels are launched one CTA per unit as at full size."""
    w = W.Workload("t", 1, 3, 128, 8192, "bf16", 4)
    q, k, v = W.make_inputs(w)
    d_out = torch.randn((1, 3, 8192, 128), generator=torch.Generator().manual_seed(5))
    got, ref = _run_both(q, k, v, w.lam, d_out, flags=flags)
    errs = _check(got, ref, 1e-3, "backward throughput-shaped")
    print(flags, errs)


@pytest.mark.parametrize("d,T", [(16, 4096), (32, 4099)])
def test_long_walk_back_keeps_the_early_tokens(d, T):
    """Paper mode over thousands of tokens: the readout denominators of the early tokens are
    small against the final key sum, so they must come from the forward's checkpoints, not
    from subtracting every key from the final sum."""
    w = W.Workload("t", 1, 2, d, T, "f32", 9)
    q, k, v = W.make_inputs(w)
    d_out = torch.randn((1, 2, T, d), generator=torch.Generator().manual_seed(6))
    got, ref = _run_both(q, k, v, w.lam, d_out)
    _check(got, ref, 1e-3, "backward long d=%d" % d)
    early = slice(0, 64)
    e = np.abs(got.dq.cpu().double().numpy()[:, :, early] - ref.dq[:, :, early]).max() / np.abs(ref.dq[:, :, early]).max()
    assert e <= 1e-3, e


# ---- explicit penalty directions (the paper's learned-u setting): gradients of q, k, v and u
@pytest.mark.parametrize("d", [32, 64, 128])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [0, IDENT])
@pytest.mark.parametrize("T", [1, 7, 64, 200])
def test_gradients_with_explicit_u(d, dtype, flags, T):
    w = _small(d, T, dtype, units=(2, 3), seed=3300 + d + T)
    q, k, v = W.make_inputs(w)
    d_out = torch.randn((2, 3, T, d), generator=torch.Generator().manual_seed(d * 5 + T))
    for scale, lam in ((d ** -0.5, 0.1), (1.0, 1.0)):
        u = W.make_u(w, scale)
        got, ref = _run_both(q, k, v, lam, d_out, flags=flags, u=u)
        _check(got, ref, 2e-4, "backward explicit u d=%d T=%d" % (d, T))


@pytest.mark.parametrize("d", [32, 128])
def test_explicit_u_with_carried_states_and_state_gradients(d):
    w = _small(d, 96, "f32", units=(1, 4), seed=3400 + d)
    q, k, v = W.make_inputs(w)
    u = W.make_u(w, d ** -0.5)
    g = torch.Generator().manual_seed(d)
    shape = (1, 4)
    S0 = torch.randn(shape + (d, d), generator=g) * 0.2
    h = torch.randn(shape + (d, d), generator=g) * 0.1
    A0 = h @ h.transpose(-1, -2) + 0.5 * torch.eye(d)
    z0 = torch.rand(shape + (d,), generator=g) + 0.1
    d_out = torch.randn(shape + (96, d), generator=g)
    dS_T = torch.randn(shape + (d, d), generator=g)
    dA_T = torch.randn(shape + (d, d), generator=g)
    dz_T = torch.randn(shape + (d,), generator=g)
    got, ref = _run_both(q, k, v, 0.5, d_out, S0=S0, A0=A0, z0=z0, dS_T=dS_T, dA_T=dA_T, dz_T=dz_T, u=u)
    _check(got, ref, 2e-4, "backward explicit u carried d=%d" % d)


def test_explicit_u_equal_to_k_hat_splits_the_key_gradient():
    """u given as the normalised keys themselves: q, v gradients as in the u = k_hat call."""
    w = _small(64, 50, "f32", units=(1, 2), seed=3500)
    q, k, v = W.make_inputs(w)
    u = k / k.norm(dim=-1, keepdim=True)
    d_out = torch.randn((1, 2, 50, 64), generator=torch.Generator().manual_seed(1))
    dev = torch.device("cuda:0")
    a = vla.vla_backward(q.to(dev), k.to(dev), v.to(dev), 1.0, d_out.to(dev), flags=IDENT)
    b = vla.vla_backward(q.to(dev), k.to(dev), v.to(dev), 1.0, d_out.to(dev), flags=IDENT, u=u.to(dev))
    torch.cuda.synchronize()
    assert torch.allclose(a.dq, b.dq, rtol=1e-3, atol=1e-5) and torch.allclose(a.dv, b.dv, rtol=1e-3, atol=1e-5)
    assert b.du is not None and torch.isfinite(b.du).all()
    w16 = _small(16, 8, "f32")
    q, k, v = [x.to(dev) for x in W.make_inputs(w16)]
    with pytest.raises(vla.VlaError) as ei:
        vla.vla_backward(q, k, v, 1.0, torch.zeros((1, 2, 8, 16), device=dev), u=k)
    assert ei.value.code == vla.VLA_ERR_UNSUPPORTED


@pytest.mark.parametrize("umode", ["khat", "unit_over_sqrt_d"])
def test_long_walk_back_with_a_weak_prior(umode):
    """lambda = 0.1 (the paper's value): A starts at 10 I and shrinks by two orders of magnitude
    over the sequence; the reverse sweep rebuilds it by adding the downdates back."""
    d, T = 64, 4096
    w = W.Workload("t", 1, 2, d, T, "f32", 12)
    q, k, v = W.make_inputs(w)
    u = None if umode == "khat" else W.make_u(w, d ** -0.5)
    d_out = torch.randn((1, 2, T, d), generator=torch.Generator().manual_seed(8))
    for flags in (0, IDENT):
        got, ref = _run_both(q, k, v, 0.1, d_out, flags=flags, u=u)
        errs = _check(got, ref, 1e-3, "backward lambda=0.1 %s" % umode)
        print(umode, flags, errs)


# ---- Algorithm 1's periodic refresh A += eta I in the backward pass
@pytest.mark.parametrize("d", [32, 64, 128])
@pytest.mark.parametrize("umode", ["khat", "unit_over_sqrt_d"])
@pytest.mark.parametrize("flags", [0, IDENT])
@pytest.mark.parametrize("refresh", [(20, 1e-3, 0), (3, 5e-2, 2), (1, 1e-2, 0), (16, 1e-2, 7)])
def test_gradients_with_the_periodic_refresh(d, umode, flags, refresh):
    T = 75
    w = _small(d, T, "f32", units=(1, 3), seed=3600 + d)
    q, k, v = W.make_inputs(w)
    u = None if umode == "khat" else W.make_u(w, d ** -0.5)
    g = torch.Generator().manual_seed(d + refresh[0])
    d_out = torch.randn((1, 3, T, d), generator=g)
    dA_T = torch.randn((1, 3, d, d), generator=g)
    got, ref = _run_both(q, k, v, 0.1, d_out, flags=flags, u=u, refresh=refresh, dA_T=dA_T)
    _check(got, ref, 2e-4, "backward refresh %s d=%d %s" % (refresh, d, umode))


def test_refresh_is_refused_where_there_is_no_general_path():
    dev = torch.device("cuda:0")
    w16 = _small(16, 8, "f32")
    q, k, v = [x.to(dev) for x in W.make_inputs(w16)]
    with pytest.raises(vla.VlaError) as ei:
        vla.vla_backward(q, k, v, 1.0, torch.zeros((1, 2, 8, 16), device=dev), refresh=(4, 1e-3, 0))
    assert ei.value.code == vla.VLA_ERR_UNSUPPORTED


# ---- token-major tensors ([B, T, H, d]) in the backward pass
@pytest.mark.parametrize("d", [32, 64, 128])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("option", ["plain", "explicit_u", "refresh"])
def test_token_major_gradients(d, dtype, option):
    """The same backward call with the sequence tensors and their gradients transposed to
    [B, T, H, d]: bit-identical to the head-major call, and within tolerance of the oracle."""
    T = 83
    w = _small(d, T, dtype, units=(2, 3), seed=3700 + d)
    q, k, v = W.make_inputs(w)
    u = W.make_u(w, d ** -0.5) if option == "explicit_u" else None
    refresh = (20, 1e-3, 3) if option == "refresh" else None
    g = torch.Generator().manual_seed(d)
    d_out = torch.randn((2, 3, T, d), generator=g)
    dS_T = torch.randn((2, 3, d, d), generator=g)
    got, ref = _run_both(q, k, v, 0.5, d_out, u=u, refresh=refresh, dS_T=dS_T)
    _check(got, ref, 2e-4, "backward head-major")
    dev = torch.device("cuda:0")
    tm = lambda x: None if x is None else x.permute(0, 2, 1, 3).contiguous().to(dev)
    r = vla.vla_backward(tm(q), tm(k), tm(v), 0.5, tm(d_out), u=tm(u), dS_T=dS_T.to(dev), refresh=refresh,
                         flags=vla.VLA_FLAG_TOKEN_MAJOR)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    back = lambda x: x.permute(0, 2, 1, 3)
    assert torch.equal(back(r.dq), got.dq) and torch.equal(back(r.dk), got.dk) and torch.equal(back(r.dv), got.dv)
    assert torch.equal(r.dS0, got.dS0) and torch.equal(r.dA0, got.dA0) and torch.equal(r.dz0, got.dz0)
    if u is not None:
        assert torch.equal(back(r.du), got.du)


def test_token_major_is_refused_without_the_reverse_scans():
    dev = torch.device("cuda:0")
    x = torch.zeros((1, 8, 2, 16), device=dev)
    with pytest.raises(vla.VlaError) as ei:
        vla.vla_backward(x, x, x, 1.0, x, flags=vla.VLA_FLAG_TOKEN_MAJOR)
    assert ei.value.code == vla.VLA_ERR_UNSUPPORTED


@pytest.mark.parametrize("umode", ["khat", "unit_over_sqrt_d"])
def test_more_units_than_resident_ctas(umode):
    """More units than the SMs hold at once, not a multiple of them: the forward that leaves the
    stash runs on the schedule that cuts units at chunk boundaries, and the reverse scans' second
    halves (the A sides) start as CTAs of the first wave retire."""
    d, T = 128, 80
    w = W.Workload("t", 1, 151, d, T, "bf16", 21)
    q, k, v = W.make_inputs(w)
    u = None if umode == "khat" else W.make_u(w, d ** -0.5)
    d_out = torch.randn((1, 151, T, d), generator=torch.Generator().manual_seed(3))
    got, ref = _run_both(q, k, v, w.lam, d_out, u=u)
    _check(got, ref, 2e-4, "backward 151 units")


def test_backward_replays_from_a_cuda_graph():
    """Captured once, replayed on new inputs: the launch that runs both reverse scans zeroes its
    progress words and ticket counter with a memset node of the same graph."""
    dev = torch.device("cuda:0")
    w = W.Workload("t", 1, 151, 64, 48, "f32", 41)
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    d_out = torch.randn((1, 151, 48, 64), generator=torch.Generator().manual_seed(1)).to(dev)
    ws = torch.empty((vla.backward_workspace_bytes(1, 151, 48, 64),), dtype=torch.uint8, device=dev)
    status = torch.zeros((), dtype=torch.int32, device=dev)
    call = lambda: vla.vla_backward(q, k, v, w.lam, d_out, workspace=ws, status=status)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        call()
    torch.cuda.current_stream().wait_stream(s)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        g = call()
    for seed in (42, 43):
        q2, k2, v2 = W.make_inputs(W.Workload("t", 1, 151, 64, 48, "f32", seed))
        q.copy_(q2); k.copy_(k2); v.copy_(v2)
        graph.replay()
        torch.cuda.synchronize()
        got = [x.clone() for x in (g.dq, g.dk, g.dv, g.dA0)]
        fresh = vla.vla_backward(q, k, v, w.lam, d_out)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for a, b in zip(got, (fresh.dq, fresh.dk, fresh.dv, fresh.dA0)):
            assert torch.equal(a, b)


@pytest.mark.parametrize("flags", [0, IDENT])
def test_long_shape_one_unit(flags):
    """One unit of the `long` shape (d = 64, T = 65536, bf16): 65536 undone updates in a row and
    an adjoint of A that sums 65536 fp32 updates.  With the normalised keys of Section 3.1 that
    adjoint grows to ~1e4 while the early tokens' z are O(1); the A side sums it in two levels
    (folded every 256 tokens) so that its rounding stays below 1e-3 of max|dk| (a single
    accumulator: 1.4e-3)."""
    w = W.Workload("t", 1, 1, 64, 65536, "bf16", 3)
    q, k, v = W.make_inputs(w)
    d_out = torch.randn((1, 1, 65536, 64), generator=torch.Generator().manual_seed(9))
    got, ref = _run_both(q, k, v, w.lam, d_out, flags=flags)
    errs = {"dq": _err(got.dq, ref.dq), "dk": _err(got.dk, ref.dk), "dv": _err(got.dv, ref.dv),
            "dS0": _err(got.dS0, ref.dS0), "dA0": _err(got.dA0, ref.dA0), "dz0": _err(got.dz0, ref.dz0)}
    print(flags, errs)
    for name, e in errs.items():
        assert e <= 1e-3, (name, e, errs)


def test_throughput_workload_full_launch_sampled_units():
    """The backward pass of the whole headline workload (512 units, the launch the benchmark
    times: 1024 CTAs drawing tickets, A sides following S sides, the forward on the balanced
    schedule); the oracle recomputes a sample of whole units."""
    w = W.WORKLOADS["throughput"]
    dev = torch.device("cuda:0")
    q, k, v = W.make_inputs(w)
    d_out = torch.randn((w.B, w.H, w.T, w.d), generator=torch.Generator().manual_seed(17))
    g = vla.vla_backward(q.to(dev), k.to(dev), v.to(dev), w.lam, d_out.to(dev))
    torch.cuda.synchronize()
    assert int(g.status.item()) == 0
    units = [(0, 0), (31, 15), (13, 7), (20, 3)]
    pick = lambda x: torch.stack([x[b, h] for (b, h) in units]).unsqueeze(0).contiguous()
    f64 = lambda x: x.detach().cpu().double().numpy()
    ref = oracle.backward(to_oracle_array(pick(q))[0], to_oracle_array(pick(k))[0], to_oracle_array(pick(v))[0],
                          w.lam, f64(pick(d_out)), in_dtype=oracle.BF16, n_threads=NTHREADS)
    for name, got, want in (("dq", g.dq, ref.dq), ("dk", g.dk, ref.dk), ("dv", g.dv, ref.dv),
                            ("dA0", g.dA0, ref.dA0), ("dS0", g.dS0, ref.dS0)):
        for n, (b, h) in enumerate(units):
            e = _err(got[b, h], want[0, n])
            assert e <= 1e-3, "unit (%d,%d) %s rel err %.3e" % (b, h, name, e)
