"""vla_scan under torch.autograd: the gradients that loss.backward() leaves on the inputs are
those of the fp64 backward oracle, also through penalty directions built with torch ops from a
weight (the learned-u setting)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_11196_b200 as vla
from oracle import make_u as OU
from paper_2605_11196_b200 import workloads as W
from parity_util import NTHREADS

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _rel(x, ref):
    x = x.detach().cpu().double().numpy()
    return float(np.abs(x - ref).max() / max(np.abs(ref).max(), 1e-3))


@pytest.mark.parametrize("d,flags", [(16, 0), (64, 0), (64, vla.VLA_FLAG_IDENTITY_MAP), (128, 0)])
def test_backward_through_the_function(d, flags):
    T = 60
    w = W.Workload("t", 2, 2, d, T, "f32", 900 + d)
    q, k, v = [x.to(DEV).requires_grad_(True) for x in W.make_inputs(w)]
    g = torch.Generator().manual_seed(d)
    S0 = (torch.randn((2, 2, d, d), generator=g) * 0.1).to(DEV).requires_grad_(True)
    c_out = torch.randn((2, 2, T, d), generator=g)
    c_S = torch.randn((2, 2, d, d), generator=g)
    out, S_T, A_T, z_T = vla.vla_scan(q, k, v, 0.5, S0=S0, flags=flags)
    loss = (out * c_out.to(DEV)).sum() + (S_T * c_S.to(DEV)).sum()
    loss.backward()
    f64 = lambda x: x.detach().cpu().double().numpy()
    ref = oracle.backward(f64(q).astype(np.float32), f64(k).astype(np.float32), f64(v).astype(np.float32), 0.5,
                          f64(c_out), in_dtype=oracle.F32, S0=f64(S0), dS_T=f64(c_S), flags=flags,
                          n_threads=NTHREADS)
    assert _rel(q.grad, ref.dq) <= 2e-4 and _rel(k.grad, ref.dk) <= 2e-4 and _rel(v.grad, ref.dv) <= 2e-4
    assert _rel(S0.grad, ref.dS0) <= 2e-4


def test_learned_penalty_directions_train_through_it():
    """u = L2norm(W_u k) / sqrt(d) built with torch ops: the weight's gradient is the oracle's du
    pulled back through the fp64 make_u step (finite differences of its oracle)."""
    d, T = 32, 40
    w = W.Workload("t", 1, 2, d, T, "f32", 950)
    q, k, v = [x.to(DEV) for x in W.make_inputs(w)]
    Wu = (torch.randn((2, d, d), generator=torch.Generator().manual_seed(1)) / d ** 0.5).to(DEV).requires_grad_(True)
    y = torch.einsum("hcj,bhtj->bhtc", Wu, k)
    u = y / y.norm(dim=-1, keepdim=True) * d ** -0.5
    c_out = torch.randn((1, 2, T, d), generator=torch.Generator().manual_seed(2))
    out, _, _, _ = vla.vla_scan(q, k, v, 0.1, u=u)
    (out * c_out.to(DEV)).sum().backward()
    f64 = lambda x: x.detach().cpu().double().numpy()
    u_ref = OU.make_u(f64(k).astype(np.float32), f64(Wu), d ** -0.5, 1e-4).astype(np.float32)
    ref = oracle.backward(f64(q).astype(np.float32), f64(k).astype(np.float32), f64(v).astype(np.float32), 0.1,
                          f64(c_out), u=u_ref, in_dtype=oracle.F32, n_threads=NTHREADS)
    # directional derivative of sum(du . make_u(W)) along a few weight perturbations
    W0 = f64(Wu)
    rng = np.random.default_rng(0)
    for _ in range(3):
        dW = rng.standard_normal(W0.shape)
        h = 1e-6
        fd = (OU.make_u(f64(k).astype(np.float32), W0 + h * dW, d ** -0.5, 1e-4) -
              OU.make_u(f64(k).astype(np.float32), W0 - h * dW, d ** -0.5, 1e-4)) / (2 * h)
        want = float((ref.du * fd).sum())
        got = float((f64(Wu.grad) * dW).sum())
        assert abs(got - want) <= 2e-3 * max(abs(want), 1e-3), (got, want)


def test_device_side_problems_of_vla_scan_are_reported_by_check_status():
    """vla_scan never synchronises; what a kernel reports on the device (here: a non-finite value
    under VLA_FLAG_CHECK_FINITE) is read back by check_status(), which clears it."""
    dev = torch.device("cuda:0")
    vla.check_status(dev)                               # clean to begin with
    w = W.Workload("ag", 1, 2, 64, 40, "f32", 9)
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    vla.vla_scan(q, k, v, 1.0, flags=vla.VLA_FLAG_CHECK_FINITE)
    vla.check_status(dev)                               # a finite run leaves the word at 0
    k_bad = k.clone()
    k_bad[0, 1, 7, 3] = float("nan")
    vla.vla_scan(q, k_bad, v, 1.0, flags=vla.VLA_FLAG_CHECK_FINITE)
    with pytest.raises(vla.VlaError) as ei:
        vla.check_status(dev)
    assert ei.value.code == vla.VLA_ERR_NONFINITE
    vla.check_status(dev)                               # cleared
