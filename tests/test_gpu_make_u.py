"""vla_make_u (u = scale * L2norm(W_u k), Algorithm 1) against the fp64 oracle, and the scan
driven by those directions end to end."""
import numpy as np
import pytest
import torch

import paper_2605_11196_b200 as vla
from oracle import make_u as OU
from paper_2605_11196_b200 import workloads as W
from parity_util import rel_err, run_oracle, to_oracle_array

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _weights(H, d, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn((H, d, d), generator=g) / d ** 0.5


@pytest.mark.parametrize("d", [16, 32, 64, 128])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("T", [1, 63, 64, 65, 1100])
def test_make_u_matches_the_oracle(d, dtype, T):
    w = W.Workload("t", 2, 3, d, T, dtype, 500 + d)
    _, k, _ = W.make_inputs(w)
    Wu = _weights(3, d, d)
    ka, dt = to_oracle_array(k)
    for scale in (d ** -0.5, 1.0):
        ref = OU.make_u(ka, Wu.double().numpy(), scale, 1e-4, in_dtype=dt)
        # fp32 result
        u32 = vla.vla_make_u(k.to(DEV), Wu.to(DEV), scale=scale, out_dtype=torch.float32)
        torch.cuda.synchronize()
        assert np.abs(u32.cpu().double().numpy() - ref).max() <= 2e-6 * scale
        # stored in the keys' own type: bf16 results are within one rounding of the exact value
        u = vla.vla_make_u(k.to(DEV), Wu.to(DEV), scale=scale)
        torch.cuda.synchronize()
        assert u.dtype == k.dtype and u.shape == k.shape
        err = np.abs(u.cpu().double().numpy() - ref)
        bound = 2e-6 * scale if dtype == "f32" else 2.0 ** -8 * np.abs(ref) + 1e-6 * scale
        assert np.all(err <= bound)


@pytest.mark.parametrize("d", [16, 64, 128])
@pytest.mark.parametrize("flags", [0, vla.VLA_FLAG_IDENTITY_MAP])
def test_scan_with_projected_directions(d, flags):
    """Algorithm 1 with its learned penalty direction: u from W_u on the device, then the scan;
    the oracle forms u in fp64 and stores it as fp32 like the device buffer."""
    w = W.Workload("t", 2, 2, d, 150, "f32", 600 + d)
    q, k, v = W.make_inputs(w)
    Wu = _weights(2, d, 7 * d)
    u_ref = OU.make_u(k.numpy(), Wu.double().numpy(), d ** -0.5, 1e-4)
    ref = run_oracle(q, k, v, 0.1, u=torch.from_numpy(u_ref.astype(np.float32)), flags=flags)
    u = vla.vla_make_u(k.to(DEV), Wu.to(DEV))
    r = vla.vla_forward(q.to(DEV), k.to(DEV), v.to(DEV), 0.1, u=u, flags=flags)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    for got, want in ((r.out, ref.out), (r.S_T, ref.S_T), (r.A_T, ref.A_T)):
        assert rel_err(got, want) <= 1e-4


def test_make_u_arguments():
    k = torch.zeros((1, 2, 4, 48), device=DEV)
    with pytest.raises(vla.VlaError) as ei:
        vla.vla_make_u(k, torch.zeros((2, 48, 48), device=DEV))
    assert ei.value.code == vla.VLA_ERR_UNSUPPORTED
    k = torch.zeros((1, 2, 4, 32), device=DEV)
    u = vla.vla_make_u(k, torch.ones((2, 32, 32), device=DEV))    # zero keys: u = 0, no NaN
    torch.cuda.synchronize()
    assert torch.all(u == 0)
    e = vla.vla_make_u(torch.zeros((0, 2, 4, 32), device=DEV), torch.ones((2, 32, 32), device=DEV))
    assert e.numel() == 0
