"""CUDA path vs the fp64 CPU oracle, element by element, through the C ABI (-m gpu)."""
import numpy as np
import pytest
import torch

import paper_2605_11196_b200 as vla
from paper_2605_11196_b200 import workloads as W
from parity_util import check_parity, rel_err, run_gpu, run_oracle

pytestmark = pytest.mark.gpu

IDENT = vla.VLA_FLAG_IDENTITY_MAP


def _small(d, T, dtype, units=(2, 3), seed=100, kind="normal"):
    return W.Workload("small", units[0], units[1], d, T, dtype, seed, kind=kind)


KERNELS = {"token": vla.VLA_KERNEL_TOKEN, "chunk": vla.VLA_KERNEL_CHUNK}


def _chunk_covers(d, umode="khat"):
    return d >= 32


@pytest.mark.parametrize("kernel", ["token", "chunk"])
@pytest.mark.parametrize("d", [16, 32, 64, 128])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [0, IDENT])
@pytest.mark.parametrize("umode", ["khat", "unit", "unit_over_sqrt_d"])
def test_small_shapes(kernel, d, dtype, flags, umode):
    """Several chunks plus a ragged tail (T = 83 = 5*16 + 3), 6 units, both kernels."""
    if kernel == "chunk" and not _chunk_covers(d, umode):
        pytest.skip("the chunk kernel covers d >= 32")
    w = _small(d, 83, dtype, seed=7 * d + len(umode))
    q, k, v = W.make_inputs(w)
    u = None
    if umode != "khat":
        u = W.make_u(w, 1.0 if umode == "unit" else d ** -0.5)
    for lam in (1.0, 0.1):
        check_parity(q, k, v, lam, 1e-4, u=u, flags=flags, kernel=KERNELS[kernel],
                     label="%s %s d=%d lam=%g" % (kernel, umode, d, lam))


def test_forced_chunk_kernel_rejects_what_it_does_not_cover():
    dev = torch.device("cuda:0")
    w = _small(16, 8, "f32")
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    with pytest.raises(vla.VlaError) as ei:
        vla.vla_forward(q, k, v, 1.0, kernel=vla.VLA_KERNEL_CHUNK)
    assert ei.value.code == vla.VLA_ERR_UNSUPPORTED
    with pytest.raises(vla.VlaError):          # with the periodic refresh as well
        vla.vla_forward(q, k, v, 1.0, refresh=(20, 1e-3, 0), kernel=vla.VLA_KERNEL_CHUNK)


@pytest.mark.parametrize("T", [0, 1, 2, 15, 16, 17, 31, 32, 33, 48, 49, 63, 64, 65, 97])
@pytest.mark.parametrize("d", [16, 32, 64, 128])
def test_ragged_and_degenerate_lengths(T, d):
    w = _small(d, T, "f32", units=(1, 5), seed=T + d)
    q, k, v = W.make_inputs(w)
    g = torch.Generator().manual_seed(5)
    S0 = torch.randn((1, 5, d, d), generator=g) * 0.1
    z0 = torch.rand((1, 5, d), generator=g)
    for flags in (0, IDENT):
        for kern in (vla.VLA_KERNEL_TOKEN, vla.VLA_KERNEL_CHUNK):
            if kern == vla.VLA_KERNEL_CHUNK and not _chunk_covers(d):
                continue
            check_parity(q, k, v, 0.5, 1e-4, S0=S0, z0=z0, flags=flags, kernel=kern, label="T=%d" % T)


def test_zero_units_and_status_strings():
    dev = torch.device("cuda:0")
    z = torch.zeros((0, 4, 8, 32), device=dev)
    r = vla.vla_forward(z, z, z, 1.0)
    assert r.out.shape == (0, 4, 8, 32)
    assert "unsupported" in vla.status_string(vla.VLA_ERR_UNSUPPORTED)


def test_state_carry_split_invariance():
    """forward(T) == forward(T1) then forward(T - T1) with (S, A, zkey) carried (paper mode
    carries the key sum as well)."""
    w = _small(32, 100, "f32", seed=11)
    q, k, v = W.make_inputs(w)
    u = W.make_u(w)
    for flags in (0, IDENT):
        for uu in (None, u):
            # one kernel for all three calls (AUTO would pick by length), so that a
            # chunk-aligned split can be compared bit for bit
            kern = vla.VLA_KERNEL_CHUNK
            full = run_gpu(q, k, v, 0.1, u=uu, flags=flags, kernel=kern)
            ref = run_oracle(q, k, v, 0.1, u=uu, flags=flags)
            for T1 in (16, 37, 64):
                sl = lambda x, a, b: None if x is None else x[:, :, a:b].contiguous()
                a = run_gpu(sl(q, 0, T1), sl(k, 0, T1), sl(v, 0, T1), 0.1, u=sl(uu, 0, T1), flags=flags,
                            kernel=kern)
                b = run_gpu(sl(q, T1, 100), sl(k, T1, 100), sl(v, T1, 100), 0.1, u=sl(uu, T1, 100),
                            S0=a.S_T, A0=a.A_T, z0=a.z_T, flags=flags, kernel=kern)
                cat = torch.cat([a.out, b.out], dim=2)
                assert rel_err(cat, ref.out) <= 1e-4
                assert rel_err(b.S_T, ref.S_T) <= 1e-4 and rel_err(b.A_T, ref.A_T) <= 1e-4
                assert rel_err(b.z_T, ref.z_T) <= 1e-4
                if T1 % 16 == 0:   # chunk-aligned split: the same instruction stream
                    assert torch.equal(cat, full.out) and torch.equal(b.A_T, full.A_T)


@pytest.mark.parametrize("d,units", [(128, (7, 43)), (64, (1, 601)), (32, (3, 401))])
@pytest.mark.parametrize("flags", [0, IDENT])
def test_more_units_than_resident_ctas(d, units, flags):
    """More units than the GPU can hold at once, not a multiple of it: the chunk kernel then
    runs a persistent grid that cuts units at chunk boundaries and hands their state from one
    CTA to the next.  Every unit is checked, with carried-in state, T not a multiple of 16."""
    w = _small(d, 90, "bf16", units=units, seed=1000 + d)
    q, k, v = W.make_inputs(w)
    B, H = units
    g = torch.Generator().manual_seed(d)
    S0 = torch.randn((B, H, d, d), generator=g) * 0.05
    z0 = torch.rand((B, H, d), generator=g)
    errs, got, ref = check_parity(q, k, v, 1.0, 1e-4, S0=S0, z0=z0, flags=flags,
                                  kernel=vla.VLA_KERNEL_CHUNK, label="balanced d=%d" % d)
    if flags == 0:   # and with an explicit penalty direction (the paper's u / sqrt(d_h))
        check_parity(q, k, v, 0.1, 1e-4, u=W.make_u(w, d ** -0.5), S0=S0, z0=z0, flags=flags,
                     kernel=vla.VLA_KERNEL_CHUNK, label="balanced explicit-u d=%d" % d)
    # the same launch twice is bitwise reproducible (the cut points are fixed by the shape)
    again = run_gpu(q, k, v, 1.0, S0=S0, z0=z0, flags=flags, kernel=vla.VLA_KERNEL_CHUNK)
    assert torch.equal(got.out, again.out) and torch.equal(got.S_T, again.S_T)
    # and it agrees with the token kernel (one CTA per unit, no hand-off)
    tok = run_gpu(q, k, v, 1.0, S0=S0, z0=z0, flags=flags, kernel=vla.VLA_KERNEL_TOKEN)
    assert rel_err(tok.out, ref.out) <= 1e-4


@pytest.mark.parametrize("d", [16, 32, 128])
@pytest.mark.parametrize("flags", [0, IDENT])
@pytest.mark.parametrize("umode", ["khat", "unit_over_sqrt_d"])
@pytest.mark.parametrize("kernel", ["token", "chunk"])
def test_periodic_refresh_as_in_algorithm_1(d, flags, umode, kernel):
    """Algorithm 1 to the letter: lambda_0 = 0.1, A += 1e-3 I every 20 steps, with and without an
    explicit u, in one call and split in two with the step offset carried, on both kernels."""
    if kernel == "chunk" and d < 32:
        pytest.skip("the chunk kernel starts at d = 32")
    kern = KERNELS[kernel]
    w = _small(d, 130, "f32", units=(1, 3), seed=500 + d)
    q, k, v = W.make_inputs(w)
    u = None if umode == "khat" else W.make_u(w, d ** -0.5)
    rf = (20, 1e-3, 0)
    errs, got, ref = check_parity(q, k, v, 0.1, 1e-4, u=u, flags=flags, refresh=rf, kernel=kern,
                                  label="refresh %s d=%d" % (kernel, d))
    plain = run_oracle(q, k, v, 0.1, u=u, flags=flags)
    assert np.abs(plain.A_T - ref.A_T).max() > 1e-4           # the refresh is visible in A_T
    T1 = 53
    sl = lambda x, a, b: None if x is None else x[:, :, a:b].contiguous()
    a = run_gpu(sl(q, 0, T1), sl(k, 0, T1), sl(v, 0, T1), 0.1, u=sl(u, 0, T1), flags=flags, refresh=rf,
                kernel=kern)
    b = run_gpu(sl(q, T1, 130), sl(k, T1, 130), sl(v, T1, 130), 0.1, u=sl(u, T1, 130), flags=flags,
                S0=a.S_T, A0=a.A_T, z0=a.z_T, refresh=(20, 1e-3, T1), kernel=kern)
    assert rel_err(torch.cat([a.out, b.out], dim=2), ref.out) <= 1e-4
    assert rel_err(b.A_T, ref.A_T) <= 1e-4 and rel_err(b.S_T, ref.S_T) <= 1e-4


@pytest.mark.parametrize("period,eta,offset", [(1, 1e-3, 0), (3, 5e-3, 2), (16, 1e-2, 0), (17, 1e-2, 16),
                                               (20, 1e-3, 19), (37, 0.05, 1000003), (500, 0.1, 0)])
@pytest.mark.parametrize("d,dtype", [(32, "f32"), (64, "bf16"), (128, "bf16")])
def test_refresh_periods_and_offsets_on_the_chunk_kernel(period, eta, offset, d, dtype):
    """Several refreshes inside one 16-token chunk, none at all, refreshes that fall on chunk
    boundaries and on the ragged last chunk, and a large carried step offset."""
    w = _small(d, 83, dtype, units=(1, 2), seed=900 + d + period)
    q, k, v = W.make_inputs(w)
    rf = (period, eta, offset)
    for u in (None, W.make_u(w, d ** -0.5)):
        check_parity(q, k, v, 0.1, 1e-4, u=u, refresh=rf, kernel=vla.VLA_KERNEL_CHUNK,
                     label="chunk refresh P=%d d=%d" % (period, d))


def test_refresh_on_the_balanced_schedule():
    """More units than resident CTAs with the refresh: cut units carry the refresh phase."""
    w = _small(64, 200, "bf16", units=(5, 61), seed=77)
    q, k, v = W.make_inputs(w)
    check_parity(q, k, v, 0.1, 1e-4, refresh=(20, 1e-3, 7), kernel=vla.VLA_KERNEL_CHUNK,
                 label="balanced refresh")


def test_in_place_state_and_canaries():
    """S_T/A_T may alias S0/A0; nothing is written outside the output tensors."""
    dev = torch.device("cuda:0")
    w = _small(64, 40, "bf16", seed=13)
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    B, H, T, d = q.shape
    g = torch.Generator().manual_seed(3)
    S = (torch.randn((B, H, d, d), generator=g) * 0.1).to(dev)
    Ah = torch.randn((B, H, d, d), generator=g) * 0.05
    A = (Ah @ Ah.transpose(-1, -2) + torch.eye(d)).to(dev)
    ref = run_oracle(q, k, v, 1.0, S0=S, A0=A)
    pad = 1024
    buf = torch.full((B * H * T * d + 2 * pad,), 12345.0, device=dev)
    out = buf[pad:pad + B * H * T * d].view(B, H, T, d)
    r = vla.vla_forward(q, k, v, 1.0, S0=S, A0=A, S_T=S, A_T=A, out=out)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    assert torch.all(buf[:pad] == 12345.0) and torch.all(buf[-pad:] == 12345.0)
    assert rel_err(out, ref.out) <= 1e-4 and rel_err(S, ref.S_T) <= 1e-4 and rel_err(A, ref.A_T) <= 1e-4


def test_bitwise_determinism():
    w = _small(128, 200, "bf16", units=(3, 3), seed=17)
    q, k, v = W.make_inputs(w)
    a = run_gpu(q, k, v, 1.0)
    b = run_gpu(q, k, v, 1.0)
    assert torch.equal(a.out, b.out) and torch.equal(a.S_T, b.S_T) and torch.equal(a.A_T, b.A_T)


def test_zero_key_is_a_no_op():
    """A zero key (identity map) gives k_hat = 0, alpha = 0: no update, finite outputs."""
    w = _small(32, 20, "f32", units=(1, 2), seed=19)
    q, k, v = W.make_inputs(w)
    k[:, :, 7] = 0
    for kern in KERNELS.values():
        check_parity(q, k, v, 1.0, 1e-4, flags=IDENT, kernel=kern)


def test_nonfinite_inputs_are_reported():
    dev = torch.device("cuda:0")
    w = _small(32, 20, "f32", units=(1, 2), seed=23)
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    k[0, 1, 5, 3] = float("nan")
    for kern in KERNELS.values():
        r = vla.vla_forward(q, k, v, 1.0, flags=vla.VLA_FLAG_CHECK_FINITE, kernel=kern)
        torch.cuda.synchronize()
        assert int(r.status.item()) == vla.VLA_ERR_NONFINITE
        assert torch.isfinite(r.out[0, 0]).all()        # the other unit is untouched by it


def test_host_entry_point_matches_device_entry_point():
    dev = torch.device("cuda:0")
    w = _small(64, 70, "bf16", seed=29)
    q, k, v = W.make_inputs(w)
    u = W.make_u(w)
    B, H, T, d = q.shape
    g = torch.Generator().manual_seed(31)
    S0 = torch.randn((B, H, d, d), generator=g) * 0.1
    z0 = torch.rand((B, H, d), generator=g)
    nbytes = vla.vla_host_workspace_bytes(B, H, T, d, d, vla.VLA_BF16, True)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    pin = lambda x: x.pin_memory()
    rh = vla.vla_forward_host(pin(q), pin(k), pin(v), 1.0, ws, u=pin(u), S0=pin(S0), z0=pin(z0))
    torch.cuda.synchronize()
    rd = run_gpu(q, k, v, 1.0, u=u, S0=S0, z0=z0)
    assert torch.equal(rh.out, rd.out.cpu()) and torch.equal(rh.S_T, rd.S_T.cpu())
    assert torch.equal(rh.A_T, rd.A_T.cpu()) and torch.equal(rh.z_T, rd.z_T.cpu())


def test_host_entry_point_pipelines_large_batches_in_slices():
    """Above 64 MB and one unit per SM the host entry point cuts the batch into slices of
    whole units on three internal streams; results must equal the device entry point's."""
    dev = torch.device("cuda:0")
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    w = _small(64, 512, "bf16", units=(1, 2 * sms + 5), seed=37)
    q, k, v = W.make_inputs(w)
    B, H, T, d = q.shape
    g = torch.Generator().manual_seed(41)
    S0 = torch.randn((B, H, d, d), generator=g) * 0.1
    nbytes = vla.vla_host_workspace_bytes(B, H, T, d, d, vla.VLA_BF16, False)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    pin = lambda x: x.pin_memory()
    rh = vla.vla_forward_host(pin(q), pin(k), pin(v), 1.0, ws, S0=pin(S0))
    torch.cuda.synchronize()
    rd = run_gpu(q, k, v, 1.0, S0=S0)
    # each slice runs with its own grid, so the cut points of the balanced schedule differ
    # from the single launch: equal within rounding, not bitwise
    assert rel_err(rh.out, rd.out.cpu().double().numpy()) <= 1e-5
    assert rel_err(rh.S_T, rd.S_T.cpu().double().numpy()) <= 1e-5
    assert rel_err(rh.A_T, rd.A_T.cpu().double().numpy()) <= 1e-5
    assert rel_err(rh.z_T, rd.z_T.cpu().double().numpy()) <= 1e-5
    # and against the oracle on a few units of the first and of the last slice
    for h in (0, 3, H - 1):
        sl = lambda x: x[:, h:h + 1].contiguous()
        ref = run_oracle(sl(q), sl(k), sl(v), 1.0, S0=sl(S0))
        assert rel_err(rh.out[:, h:h + 1], ref.out) <= 1e-4


# ---------------------------------------------------------------- the five workloads
@pytest.mark.parametrize("name", ["tiny", "mid", "recall", "long"])
@pytest.mark.parametrize("flags", [0, IDENT])
def test_workload_full(name, flags):
    """Whole workload, every unit, both readings of the feature map."""
    w = W.WORKLOADS[name]
    q, k, v = W.make_inputs(w)
    errs, _, _ = check_parity(q, k, v, w.lam, w.tol, flags=flags, label=name)
    print(name, flags, errs)


@pytest.mark.parametrize("flags", [0, IDENT])
def test_workload_throughput_sampled_units(flags):
    """The full-size launch the benchmark times (512 units); the oracle recomputes a sample
    of whole units (units are independent), compared element by element."""
    w = W.WORKLOADS["throughput"]
    dev = torch.device("cuda:0")
    q, k, v = W.make_inputs(w)
    r = vla.vla_forward(q.to(dev), k.to(dev), v.to(dev), w.lam, flags=flags)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    assert torch.isfinite(r.out).all()
    # 24 whole units spread over the batch, recomputed by the oracle in one threaded call
    units = [(b, (5 * b + 3) % w.H) for b in range(0, w.B, 2)] + [(31, 15), (0, 0), (17, 8), (8, 1),
                                                                  (30, 2), (1, 14), (15, 15), (22, 7)]
    pick = lambda x: torch.stack([x[b, h] for (b, h) in units]).unsqueeze(0).contiguous()
    ref = run_oracle(pick(q), pick(k), pick(v), w.lam, flags=flags)
    for name, got, want in (("o", r.out, ref.out), ("S_T", r.S_T, ref.S_T), ("A_T", r.A_T, ref.A_T)):
        for n, (b, h) in enumerate(units):
            e = rel_err(got[b, h], want[0, n])
            assert e <= w.tol, "unit (%d,%d) %s rel err %.3e" % (b, h, name, e)


# ---------------------------------------------------------------- single-step kernel
def _spd(shape, g, d):
    h = torch.randn(shape + (d, d), generator=g) * 0.05
    return h @ h.transpose(-1, -2) + 0.5 * torch.eye(d)


@pytest.mark.parametrize("d,units", [(32, (3, 5)), (64, (2, 331)), (128, (7, 29)), (128, (1, 1))])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [0, IDENT])
def test_single_step_kernel(d, units, dtype, flags):
    """T = 1 with carried states: the kernel that streams S and A through shared memory, with
    fewer and more units than persistent CTAs, against the oracle and the token kernel."""
    w = _small(d, 1, dtype, units=units, seed=2000 + d)
    q, k, v = W.make_inputs(w)
    B, H = units
    g = torch.Generator().manual_seed(d + B)
    S0 = torch.randn((B, H, d, d), generator=g) * 0.3
    A0 = _spd((B, H), g, d)
    z0 = torch.rand((B, H, d), generator=g) * 3.0
    errs, got, ref = check_parity(q, k, v, 1.0, 1e-5, S0=S0, A0=A0, z0=z0, flags=flags,
                                  kernel=vla.VLA_KERNEL_DECODE, label="decode d=%d" % d)
    tok = run_gpu(q, k, v, 1.0, S0=S0, A0=A0, z0=z0, flags=flags, kernel=vla.VLA_KERNEL_TOKEN)
    assert rel_err(tok.out, ref.out) <= 1e-5
    auto = run_gpu(q, k, v, 1.0, S0=S0, A0=A0, z0=z0, flags=flags)     # AUTO takes the same kernel
    assert torch.equal(auto.out, got.out) and torch.equal(auto.S_T, got.S_T) and torch.equal(auto.A_T, got.A_T)


def test_single_step_kernel_in_a_decode_loop_and_its_limits():
    """Five steps, one call each, states updated in place; then the shapes it does not take."""
    dev = torch.device("cuda:0")
    d, T = 128, 5
    w = _small(d, T, "bf16", units=(2, 100), seed=77)
    q, k, v = W.make_inputs(w)
    g = torch.Generator().manual_seed(1)
    S0 = torch.randn((2, 100, d, d), generator=g) * 0.1
    A0 = _spd((2, 100), g, d)
    z0 = torch.rand((2, 100, d), generator=g)
    ref = run_oracle(q, k, v, 1.0, S0=S0, A0=A0, z0=z0)
    S, A, z = S0.to(dev), A0.to(dev), z0.to(dev)
    outs = []
    for t in range(T):
        sl = lambda x: x[:, :, t:t + 1].contiguous().to(dev)
        r = vla.vla_forward(sl(q), sl(k), sl(v), 1.0, S0=S, A0=A, z0=z, S_T=S, A_T=A, z_T=z,
                            kernel=vla.VLA_KERNEL_DECODE)
        outs.append(r.out)
    torch.cuda.synchronize()
    assert rel_err(torch.cat(outs, dim=2), ref.out) <= 1e-5
    assert rel_err(S, ref.S_T) <= 1e-5 and rel_err(A, ref.A_T) <= 1e-5 and rel_err(z, ref.z_T) <= 1e-5
    sl = lambda x: x[:, :, :1].contiguous().to(dev)
    with pytest.raises(vla.VlaError) as ei:      # no carried state: nothing to stream
        vla.vla_forward(sl(q), sl(k), sl(v), 1.0, kernel=vla.VLA_KERNEL_DECODE)
    assert ei.value.code == vla.VLA_ERR_UNSUPPORTED
    with pytest.raises(vla.VlaError):            # more than one step
        vla.vla_forward(q.to(dev), k.to(dev), v.to(dev), 1.0, S0=S, A0=A, kernel=vla.VLA_KERNEL_DECODE)


# ---- token-major tensors: q, k, v, u, out as [B, T, H, d] (the layout a projection writes)
TOKEN_MAJOR = vla.VLA_FLAG_TOKEN_MAJOR


@pytest.mark.parametrize("kernel", ["token", "chunk"])
@pytest.mark.parametrize("d", [16, 32, 64, 128])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [0, IDENT])
@pytest.mark.parametrize("umode", ["khat", "unit_over_sqrt_d"])
def test_token_major_layout(kernel, d, dtype, flags, umode):
    """The same scan with the sequence tensors transposed to [B, T, H, d]: bit-identical to the
    head-major call (the layout changes addresses, not arithmetic) and within tolerance of the
    oracle, which is given the head-major arrays."""
    if kernel == "chunk" and not _chunk_covers(d, umode):
        pytest.skip("no chunk kernel for this shape")
    kcode = vla.VLA_KERNEL_TOKEN if kernel == "token" else vla.VLA_KERNEL_CHUNK
    w = _small(d, 83, dtype, units=(2, 3), seed=300 + d)
    q, k, v = W.make_inputs(w)
    u = None if umode == "khat" else W.make_u(w, d ** -0.5)
    dev = torch.device("cuda:0")
    tm = lambda x: None if x is None else x.permute(0, 2, 1, 3).contiguous().to(dev)
    g = torch.Generator().manual_seed(d)
    S0 = torch.randn((2, 3, d, d), generator=g) * 0.1
    z0 = torch.rand((2, 3, d), generator=g)
    plain = run_gpu(q, k, v, w.lam, u=u, S0=S0, z0=z0, flags=flags, kernel=kcode)
    r = vla.vla_forward(tm(q), tm(k), tm(v), w.lam, u=tm(u), S0=S0.to(dev), z0=z0.to(dev),
                        flags=flags | TOKEN_MAJOR, kernel=kcode)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    assert r.out.shape == (2, 83, 3, d)
    assert torch.equal(r.out.permute(0, 2, 1, 3), plain.out)
    assert torch.equal(r.S_T, plain.S_T) and torch.equal(r.A_T, plain.A_T) and torch.equal(r.z_T, plain.z_T)
    ref = run_oracle(q, k, v, w.lam, u=u, S0=S0, z0=z0, flags=flags)
    assert rel_err(r.out.permute(0, 2, 1, 3), ref.out) <= 1e-4
    assert rel_err(r.S_T, ref.S_T) <= 1e-4 and rel_err(r.A_T, ref.A_T) <= 1e-4


def test_token_major_long_units_and_where_it_is_refused():
    """Long units with a ragged tail in [B, T, H, d], on the plain grid and on the schedule that
    cuts units into pieces; the calls that do not take the layout say so."""
    dev = torch.device("cuda:0")
    w = W.Workload("t", 1, 5, 64, 4096 + 37, "bf16", 77)
    q, k, v = W.make_inputs(w)
    tm = lambda x: x.permute(0, 2, 1, 3).contiguous().to(dev)
    plain = run_gpu(q, k, v, w.lam)
    r = vla.vla_forward(tm(q), tm(k), tm(v), w.lam, flags=TOKEN_MAJOR)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    assert torch.equal(r.out.permute(0, 2, 1, 3), plain.out) and torch.equal(r.S_T, plain.S_T)
    ref = run_oracle(q, k, v, w.lam)
    assert rel_err(r.out.permute(0, 2, 1, 3), ref.out) <= 1e-4
    wb = W.Workload("t", 1, 151, 128, 256 + 5, "bf16", 79)      # more units than resident CTAs
    q, k, v = W.make_inputs(wb)
    for kern in (vla.VLA_KERNEL_CHUNK, vla.VLA_KERNEL_AUTO):        # the FMA form, and the library's choice
        plain = run_gpu(q, k, v, wb.lam, kernel=kern)               # the same kernel, head-major
        r = vla.vla_forward(tm(q), tm(k), tm(v), wb.lam, flags=TOKEN_MAJOR, kernel=kern)
        torch.cuda.synchronize()
        assert int(r.status.item()) == 0
        assert torch.equal(r.out.permute(0, 2, 1, 3), plain.out) and torch.equal(r.A_T, plain.A_T)
    assert vla.vla_query_support(64, 64, vla.VLA_BF16, TOKEN_MAJOR) == vla.VLA_OK
    w2 = W.Workload("t", 1, 2, 64, 64, "f32", 78)
    q, k, v = [x.to(dev) for x in W.make_inputs(w2)]
    with pytest.raises(vla.VlaError) as ei:
        vla.vla_forward_seqpar(q, k, v, 1.0, segments=2, flags=TOKEN_MAJOR)
    assert ei.value.code == vla.VLA_ERR_UNSUPPORTED


@pytest.mark.parametrize("option", ["explicit_u", "refresh", "explicit_u_refresh"])
@pytest.mark.parametrize("flags", [0, IDENT])
def test_throughput_shape_with_algorithm_1_options(option, flags):
    """Whole sequences of the headline shape (d = 128, T = 8192, bf16) on the general path of
    the chunk kernel: explicit u = unit / sqrt(d), the periodic refresh every 20 steps, both."""
    w = W.Workload("t", 1, 4, 128, 8192, "bf16", 4)
    q, k, v = W.make_inputs(w)
    u = W.make_u(w, 128 ** -0.5) if "explicit_u" in option else None
    refresh = (20, 1e-3, 0) if "refresh" in option else None
    errs, _, _ = check_parity(q, k, v, w.lam, 1e-3, u=u, flags=flags, refresh=refresh,
                              kernel=vla.VLA_KERNEL_CHUNK, label=option)
    print(option, flags, errs)


def test_forward_and_backward_replay_from_a_cuda_graph():
    """The calls allocate nothing and never synchronise, so they can be captured; a replayed
    graph must give what a fresh call gives on the buffers' current contents (more units than
    resident CTAs: the shape on which a plain call would cut units across CTAs)."""
    dev = torch.device("cuda:0")
    w = W.Workload("t", 1, 151, 128, 64, "bf16", 31)
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    out = torch.empty((1, 151, 64, 128), device=dev)
    S_T = torch.empty((1, 151, 128, 128), device=dev)
    A_T = torch.empty_like(S_T)
    z_T = torch.empty((1, 151, 128), device=dev)
    status = torch.zeros((), dtype=torch.int32, device=dev)
    call = lambda: vla.vla_forward(q, k, v, w.lam, out=out, S_T=S_T, A_T=A_T, z_T=z_T, status=status)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        call()                                  # warm-up outside the capture
    torch.cuda.current_stream().wait_stream(s)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call()
    for seed in (32, 33, 34):
        q2, k2, v2 = W.make_inputs(W.Workload("t", 1, 151, 128, 64, "bf16", seed))
        q.copy_(q2); k.copy_(k2); v.copy_(v2)
        graph.replay()
        torch.cuda.synchronize()
        got = (out.clone(), S_T.clone(), A_T.clone())
        fresh = vla.vla_forward(q, k, v, w.lam)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        # the captured launch runs one CTA per unit, the fresh one cuts units across CTAs; at
        # d = 128 (tensor-core kernel) a cut re-forms (state . 1) from the handed-over state, so
        # the two agree to rounding there, and bit for bit on the FMA kernel
        f64 = lambda x: x.cpu().double().numpy()
        for a, b in zip(got, (fresh.out, fresh.S_T, fresh.A_T)):
            assert rel_err(a, f64(b)) <= 1e-5
        fma = vla.vla_forward(q, k, v, w.lam, kernel=vla.VLA_KERNEL_CHUNK)
        torch.cuda.synchronize()
        assert rel_err(fma.out, f64(fresh.out)) <= 1e-4


# ---------------------------------------------------------------- reduction modes (Section 4.4)
@pytest.mark.parametrize("kernel", ["token", "chunk"])
@pytest.mark.parametrize("d,dtype", [(32, "f32"), (64, "bf16"), (128, "f32")])
@pytest.mark.parametrize("flags", [0, IDENT])
def test_zero_penalty_directions_give_the_normalised_delta_rule(kernel, d, dtype, flags):
    """u = 0 passed explicitly (Section 4.4's remark; Eq. "deltanet" without the gate): the
    penalty never grows, A stays A_0 = I/lambda exactly, the write direction is k_hat and
    S_t = S_{t-1} + (v_t - S_{t-1} k_hat_t) k_hat_t^T.  Checked against the oracle and against
    that recurrence written out here in fp64."""
    w = _small(d, 70, dtype, units=(1, 3), seed=300 + d)
    q, k, v = W.make_inputs(w)
    u0 = torch.zeros_like(k)
    lam = 0.5
    errs, got, ref = check_parity(q, k, v, lam, 1e-4, u=u0, flags=flags, kernel=KERNELS[kernel],
                                  label="u=0 %s d=%d" % (kernel, d))
    A_T = got.A_T.cpu()
    assert torch.equal(A_T, (torch.eye(d) / lam).expand_as(A_T)), "A must not move when u = 0"
    kk, vv = k.double().numpy(), v.double().numpy()
    for h in range(w.H):
        S = np.zeros((d, d))
        for t in range(w.T):
            kf = kk[0, h, t] if flags & IDENT else np.where(kk[0, h, t] > 0, kk[0, h, t] + 1.0, np.exp(kk[0, h, t]))
            kh = kf / np.linalg.norm(kf)
            S += np.outer(vv[0, h, t] - S @ kh, kh)
        assert np.abs(got.S_T[0, h].cpu().double().numpy() - S).max() <= 1e-4 * np.abs(S).max()


LINATT = vla.VLA_FLAG_LINEAR_ATTENTION


@pytest.mark.parametrize("d", [16, 32, 64, 128])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [LINATT, LINATT | IDENT])
def test_linear_attention_mode(d, dtype, flags):
    """Section 2, Eq. "linear-attn" as a mode of the same scan: additive write S += v phi(k)^T, the
    readout of Eq. "output"; A passes through.  Against the oracle (whose additive mode is pinned
    by direct double sums) with carried S0, z0, and the layouts."""
    w = _small(d, 83, dtype, units=(2, 3), seed=500 + d)
    q, k, v = W.make_inputs(w)
    g = torch.Generator().manual_seed(d)
    S0 = torch.randn((2, 3, d, d), generator=g) * 0.1
    z0 = torch.rand((2, 3, d), generator=g)
    A0 = _spd((2, 3), g, d)
    errs, got, ref = check_parity(q, k, v, 1.0, 1e-4, S0=S0, A0=A0, z0=z0, flags=flags, label="linear attention d=%d" % d)
    assert torch.equal(got.A_T.cpu(), A0)                       # no penalty matrix in this mode
    assert vla.last_launch().startswith("vla_scan_token_kernel")
    dev = torch.device("cuda:0")
    tm = lambda x: x.permute(0, 2, 1, 3).contiguous().to(dev)
    r = vla.vla_forward(tm(q), tm(k), tm(v), 1.0, S0=S0.to(dev), A0=A0.to(dev), z0=z0.to(dev),
                        flags=flags | TOKEN_MAJOR)
    torch.cuda.synchronize()
    assert torch.equal(r.out.permute(0, 2, 1, 3), got.out) and torch.equal(r.S_T, got.S_T)


def test_linear_attention_mode_is_refused_where_it_has_no_meaning():
    dev = torch.device("cuda:0")
    w = _small(64, 32, "f32")
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    for kw in (dict(u=W.make_u(w).to(dev)), dict(refresh=(20, 1e-3, 0)), dict(kernel=vla.VLA_KERNEL_CHUNK)):
        with pytest.raises(vla.VlaError) as ei:
            vla.vla_forward(q, k, v, 1.0, flags=LINATT, **kw)
        assert ei.value.code == vla.VLA_ERR_UNSUPPORTED
    with pytest.raises(vla.VlaError):
        vla.vla_backward(q, k, v, 1.0, torch.zeros_like(q), flags=LINATT)
