"""Tensor-core form of the chunk kernel (VLA_KERNEL_CHUNK_TC, d = 128) vs the fp64 CPU oracle,
element by element, through the C ABI (-m gpu).

The kernel is opt-in: the library's own kernel choice never takes it.  It computes the same
chunk algebra as the FMA kernel with the d x d products on the tensor cores (TF32 operands in
hi/lo pairs, fp32 accumulation).  The tensor core truncates when it aligns and accumulates
its addends, so sums of many like-signed products come out slightly low; with Section 3.1's
normalised keys (mixed signs) it holds the bounds of the specification at every length, with
Algorithm 1's feature map (all-positive keys, which share a dominant direction) the final S
drifts beyond 1e-4 of its maximum on long sequences.  The tests assert the specification's
bounds wherever the kernel meets them and pin the measured drift where it does not.
"""
import numpy as np
import pytest
import torch

import paper_2605_11196_b200 as vla
from paper_2605_11196_b200 import workloads as W
from parity_util import check_parity, rel_err, run_gpu, run_oracle

pytestmark = pytest.mark.gpu

IDENT = vla.VLA_FLAG_IDENTITY_MAP
TC = vla.VLA_KERNEL_CHUNK_TC


def _carried(w, seed):
    """Carried-in states: random S0, a symmetric positive definite A0, a positive key sum."""
    g = torch.Generator().manual_seed(seed)
    B, H, d = w.B, w.H, w.d
    S0 = torch.randn((B, H, d, d), generator=g) * 0.3
    M = torch.randn((B, H, d, d), generator=g) * 0.05
    A0 = torch.eye(d) * 0.5 + M @ M.transpose(-1, -2)
    z0 = torch.rand((B, H, d), generator=g) * 3.0
    return S0, A0, z0


@pytest.mark.parametrize("T", [1, 2, 15, 16, 17, 31, 32, 33, 83, 256])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [0, IDENT])
def test_tc_small_and_ragged(T, dtype, flags):
    """One chunk, several chunks, ragged tails: the specification's 1e-4 on o, S_T, A_T, z_T."""
    w = W.Workload("tc", 2, 3, 128, T, dtype, 900 + T)
    q, k, v = W.make_inputs(w)
    for lam in (1.0, 0.1):
        check_parity(q, k, v, lam, 1e-4, flags=flags, kernel=TC, label="tc T=%d lam=%g" % (T, lam))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [0, IDENT])
def test_tc_carried_states_and_split_invariance(dtype, flags):
    """States carried in (S0, A0, z0) and out; a sequence run in two calls equals one call."""
    w = W.Workload("tc", 2, 2, 128, 200, dtype, 31)
    q, k, v = W.make_inputs(w)
    S0, A0, z0 = _carried(w, 77)
    errs, got, ref = check_parity(q, k, v, 1.0, 1e-4, S0=S0, A0=A0, z0=z0, flags=flags, kernel=TC, label="tc carried")
    T1 = 112   # a multiple of the chunk: the second call starts on the same chunk boundaries
    a = run_gpu(q[:, :, :T1], k[:, :, :T1], v[:, :, :T1], 1.0, S0=S0, A0=A0, z0=z0, flags=flags, kernel=TC)
    b = run_gpu(q[:, :, T1:], k[:, :, T1:], v[:, :, T1:], 1.0, S0=a.S_T, A0=a.A_T, z0=a.z_T, flags=flags, kernel=TC)
    assert torch.equal(torch.cat([a.out, b.out], dim=2), got.out)
    assert torch.equal(b.S_T, got.S_T) and torch.equal(b.A_T, got.A_T) and torch.equal(b.z_T, got.z_T)


def test_tc_is_deterministic_and_leaves_canaries_alone():
    """Two runs are bit-identical; nothing is written outside out / S_T / A_T / z_T."""
    dev = torch.device("cuda:0")
    w = W.Workload("tc", 1, 5, 128, 70, "bf16", 5)
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    pad = 64
    def run():
        out = torch.full((w.B * w.H * w.T * 128 + 2 * pad,), 7.25, device=dev)
        view = out[pad:-pad].view(w.B, w.H, w.T, 128)
        r = vla.vla_forward(q, k, v, 1.0, kernel=TC, out=view)
        torch.cuda.synchronize()
        assert int(r.status.item()) == 0
        assert torch.all(out[:pad] == 7.25) and torch.all(out[-pad:] == 7.25)
        return r
    a, b = run(), run()
    for x, y in ((a.out, b.out), (a.S_T, b.S_T), (a.A_T, b.A_T), (a.z_T, b.z_T)):
        assert torch.equal(x, y)


def test_tc_rejects_what_it_does_not_cover():
    dev = torch.device("cuda:0")
    def call(d, **kw):
        w = W.Workload("tc", 1, 2, d, 32, "f32", 3)
        q, k, v = [x.to(dev) for x in W.make_inputs(w)]
        u = W.make_u(w, 1.0).to(dev) if kw.pop("with_u", False) else None
        return vla.vla_forward(q, k, v, 1.0, kernel=TC, u=u, **kw)
    for bad in (dict(d=64), dict(d=128, with_u=True), dict(d=128, refresh=(20, 1e-3, 0))):
        with pytest.raises(vla.VlaError) as ei:
            call(**bad)
        assert ei.value.code == vla.VLA_ERR_UNSUPPORTED


def test_tc_many_units_more_than_one_wave():
    """More units than SMs (CTAs queue for the SM's tensor memory): every unit against the oracle."""
    w = W.Workload("tc", 20, 16, 128, 48, "bf16", 12)
    q, k, v = W.make_inputs(w)
    check_parity(q, k, v, 1.0, 1e-4, kernel=TC, label="tc 320 units")


@pytest.mark.parametrize("dtype,T,tol", [("f32", 4096, 1e-4), ("bf16", 8192, 1e-3)])
def test_tc_long_sequences_normalised_keys(dtype, T, tol):
    """Section 3.1's keys: the specification's bounds hold at full length."""
    w = W.Workload("tc", 1, 2, 128, T, dtype, 44)
    q, k, v = W.make_inputs(w)
    errs, _, _ = check_parity(q, k, v, 1.0, tol, flags=IDENT, kernel=TC, label="tc long, normalised keys")
    assert max(errs.values()) <= 2e-5, errs     # measured <= 6e-6


def test_tc_long_sequence_feature_map_drift_is_as_measured():
    """Algorithm 1's feature map at T = 4096: the readout, A_T and z_T hold 1e-4; the final S does
    not (measured 2.5e-4 of its maximum, against 3e-6 on the FMA kernel), which is why the
    library never chooses this kernel by itself.  The bound asserted for S_T is the measured
    drift with margin, not the specification's."""
    w = W.Workload("tc", 1, 1, 128, 4096, "bf16", 5)
    q, k, v = W.make_inputs(w)
    ref = run_oracle(q, k, v, 1.0)
    got = run_gpu(q, k, v, 1.0, kernel=TC)
    assert rel_err(got.out, ref.out) <= 1e-4
    assert rel_err(got.A_T, ref.A_T) <= 1e-4
    assert rel_err(got.z_T, ref.z_T) <= 1e-4
    assert rel_err(got.S_T, ref.S_T) <= 1e-3
    fma = run_gpu(q, k, v, 1.0, kernel=vla.VLA_KERNEL_CHUNK)
    assert rel_err(fma.S_T, ref.S_T) <= 1e-4      # the default kernel holds the bound on the same input


def test_auto_never_picks_the_tc_kernel():
    """The library's own choice at d = 128 is bit-identical to the FMA chunk kernel."""
    dev = torch.device("cuda:0")
    w = W.Workload("tc", 1, 3, 128, 96, "bf16", 8)
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    a = vla.vla_forward(q, k, v, 1.0)
    b = vla.vla_forward(q, k, v, 1.0, kernel=vla.VLA_KERNEL_CHUNK)
    torch.cuda.synchronize()
    assert torch.equal(a.out, b.out) and torch.equal(a.S_T, b.S_T) and torch.equal(a.A_T, b.A_T)
