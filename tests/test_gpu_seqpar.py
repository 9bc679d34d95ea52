"""Sequence-parallel forward (vla_forward_seqpar) against the fp64 oracle: the segments of a
unit are scanned concurrently and stitched with the composition of Section 3.4 written for a
map that acts on the right (S_end = S_start P + G); A at the segment starts comes from the
prefix sums of u u^T."""
import numpy as np
import pytest
import torch

import paper_2605_11196_b200 as vla
from paper_2605_11196_b200 import workloads as W
from parity_util import rel_err, run_gpu, run_oracle

pytestmark = pytest.mark.gpu
IDENT = vla.VLA_FLAG_IDENTITY_MAP


def _small(d, T, dtype, units=(1, 2), seed=1):
    return W.Workload("t", units[0], units[1], d, T, dtype, seed)


def _run_seqpar(q, k, v, lam, segments, u=None, S0=None, A0=None, z0=None, flags=0):
    dev = torch.device("cuda:0")
    mv = lambda x: None if x is None else x.to(dev).contiguous()
    r = vla.vla_forward_seqpar(mv(q), mv(k), mv(v), lam, segments=segments, u=mv(u), S0=mv(S0), A0=mv(A0), z0=mv(z0),
                               flags=flags)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0, vla.status_string(int(r.status.item()))
    return r


def _check(r, ref, tol, label):
    errs = {"o": rel_err(r.out, ref.out), "S_T": rel_err(r.S_T, ref.S_T), "A_T": rel_err(r.A_T, ref.A_T),
            "z_T": rel_err(r.z_T, ref.z_T)}
    for name, e in errs.items():
        assert e <= tol, "%s %s: rel err %.3e > %.1e (%s)" % (label, name, e, tol, errs)
    return errs


@pytest.mark.parametrize("d", [32, 64, 128])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [0, IDENT])
@pytest.mark.parametrize("segments", [2, 4, 8])
def test_segments_agree_with_the_oracle(d, dtype, flags, segments):
    w = _small(d, 256, dtype, units=(2, 3), seed=40 + d + segments)
    q, k, v = W.make_inputs(w)
    for lam in (1.0, 0.1):
        ref = run_oracle(q, k, v, lam, flags=flags)
        r = _run_seqpar(q, k, v, lam, segments, flags=flags)
        _check(r, ref, 1e-4, "seqpar d=%d P=%d lam=%g" % (d, segments, lam))


@pytest.mark.parametrize("d", [32, 128])
@pytest.mark.parametrize("flags", [0, IDENT])
def test_carried_state_and_explicit_u(d, flags):
    """S0, z0 and a symmetric positive definite A0 carried in, explicit penalty directions, many
    short segments (one chunk each)."""
    w = _small(d, 192, "f32", units=(1, 3), seed=70 + d)
    q, k, v = W.make_inputs(w)
    g = torch.Generator().manual_seed(d)
    S0 = torch.randn((1, 3, d, d), generator=g) * 0.1
    z0 = torch.rand((1, 3, d), generator=g)
    h = torch.randn((1, 3, d, d), generator=g) * 0.1
    A0s = h @ h.transpose(-1, -2) + 0.3 * torch.eye(d)
    for u in (None, W.make_u(w, d ** -0.5)):
        for A0 in (None, A0s):
            ref = run_oracle(q, k, v, 0.5, u=u, S0=S0, A0=A0, z0=z0, flags=flags)
            for segments in (3, 12):
                r = _run_seqpar(q, k, v, 0.5, segments, u=u, S0=S0, A0=A0, z0=z0, flags=flags)
                _check(r, ref, 1e-4, "seqpar carried d=%d P=%d" % (d, segments))


def test_one_segment_is_the_plain_scan_and_bad_arguments_are_refused():
    dev = torch.device("cuda:0")
    w = _small(64, 96, "f32", seed=5)
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    a = vla.vla_forward_seqpar(q, k, v, 1.0, segments=1)
    b = vla.vla_forward(q, k, v, 1.0)
    torch.cuda.synchronize()
    assert torch.equal(a.out, b.out) and torch.equal(a.S_T, b.S_T) and torch.equal(a.A_T, b.A_T)
    with pytest.raises(vla.VlaError) as ei:            # 6 chunks do not split in 4
        vla.vla_forward_seqpar(q, k, v, 1.0, segments=4)
    assert ei.value.code == vla.VLA_ERR_INVALID_ARG
    with pytest.raises(vla.VlaError) as ei:            # workspace too small
        vla.vla_forward_seqpar(q, k, v, 1.0, segments=2,
                               workspace=torch.empty((1024,), dtype=torch.uint8, device=dev))
    assert ei.value.code == vla.VLA_ERR_INVALID_ARG
    w16 = _small(16, 64, "f32")
    q, k, v = [x.to(dev) for x in W.make_inputs(w16)]
    with pytest.raises(vla.VlaError) as ei:            # d = 16 has no chunk kernel
        vla.vla_forward_seqpar(q, k, v, 1.0, segments=2)
    assert ei.value.code == vla.VLA_ERR_UNSUPPORTED
    assert vla.seqpar_workspace_bytes(1, 2, 96, 64, 2) > 0


def test_library_picks_segments_for_few_long_units():
    B, H, T, d = 1, 16, 65536, 64
    P = vla.seqpar_segments(B, H, T, d, torch.bfloat16)
    assert P >= 2 and (T // 16) % P == 0 and T // P >= 256
    assert vla.seqpar_segments(32, 16, 8192, 128, torch.bfloat16) == 1   # the GPU is full already
    assert vla.seqpar_segments(1, 1, 100, 64, torch.float32) == 1        # T not a multiple of 16


@pytest.mark.parametrize("name", ["mid", "long"])
@pytest.mark.parametrize("flags", [0, IDENT])
def test_few_unit_workloads_full_size(name, flags):
    """The two workloads with fewer units than SMs, whole, with the library's own choice of
    segments, against the oracle and against the plain scan."""
    w = W.WORKLOADS[name]
    q, k, v = W.make_inputs(w)
    ref = run_oracle(q, k, v, w.lam, flags=flags)
    r = _run_seqpar(q, k, v, w.lam, 0, flags=flags)
    errs = _check(r, ref, w.tol, "seqpar " + name)
    plain = run_gpu(q, k, v, w.lam, flags=flags)
    print(name, flags, errs, "plain o err", rel_err(plain.out, ref.out))
    assert np.isfinite(r.out.cpu().numpy()).all()


def test_vla_forward_takes_the_segmented_route_when_given_scratch():
    """kernel AUTO + opts->workspace: a problem with few long units runs as vla_forward_seqpar
    (the scratch is used, the result is that call's up to the order of its atomic sums), one
    that fills the device, or too little scratch, leaves it to the plain scan."""
    dev = torch.device("cuda:0")
    w = W.Workload("t", 1, 6, 64, 2048, "bf16", 91)
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    P = vla.seqpar_segments(1, 6, 2048, 64, torch.bfloat16)
    assert P > 1
    ws = torch.full((vla.seqpar_workspace_bytes(1, 6, 2048, 64, P),), 0x5A, dtype=torch.uint8, device=dev)
    a = vla.vla_forward(q, k, v, w.lam, workspace=ws)
    b = vla.vla_forward_seqpar(q, k, v, w.lam, segments=P)
    c = vla.vla_forward(q, k, v, w.lam)
    a2 = vla.vla_forward(q, k, v, w.lam, workspace=True)        # scratch allocated by the binding
    torch.cuda.synchronize()
    assert bool((ws != 0x5A).any())                              # the segmented route ran
    f64 = lambda x: x.cpu().double().numpy()
    assert rel_err(a.out, f64(b.out)) <= 1e-6 and rel_err(a.S_T, f64(b.S_T)) <= 1e-6
    assert rel_err(a2.out, f64(b.out)) <= 1e-6
    assert rel_err(a.out, f64(c.out)) <= 1e-4                    # the same scan in another order
    small = torch.full((1024,), 0x5A, dtype=torch.uint8, device=dev)   # too little scratch: the plain scan
    d2 = vla.vla_forward(q, k, v, w.lam, workspace=small)
    torch.cuda.synchronize()
    assert torch.equal(d2.out, c.out) and bool((small == 0x5A).all())
    wf = W.Workload("t", 4, 80, 32, 64, "f32", 92)               # the device is full: nothing to cut
    q, k, v = [x.to(dev) for x in W.make_inputs(wf)]
    big = torch.full((1 << 20,), 0x5A, dtype=torch.uint8, device=dev)
    e = vla.vla_forward(q, k, v, wf.lam, workspace=big)
    f = vla.vla_forward(q, k, v, wf.lam)
    torch.cuda.synchronize()
    assert torch.equal(e.out, f.out) and bool((big == 0x5A).all())
