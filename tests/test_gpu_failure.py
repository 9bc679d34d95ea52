"""Failure detection on the device (-m gpu): a bounded wait that is made to run out.

Nothing here faults, traps or hangs the GPU: the wait gives up by itself after its probe limit,
the kernel writes a status code and returns, and the context stays usable."""
import pytest
import torch

import paper_2605_11196_b200 as vla
from paper_2605_11196_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _scan(dev, kernel=vla.VLA_KERNEL_AUTO, **kw):
    w = W.Workload("f", 2, 3, 64, 100, "f32", 21)
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    r = vla.vla_forward(q, k, v, 1.0, kernel=kernel, **kw)
    torch.cuda.synchronize()
    return r


def test_bounded_wait_runs_out_and_the_device_stays_usable():
    """The library's own bounded wait (the function every scan kernel waits with) on a barrier
    that can never complete: after `probe_limit` probes the kernel reports
    VLA_ERR_DEVICE_TIMEOUT through the status word and ends normally.  A scan before and a scan
    after it on the same device give bit-identical results."""
    dev = torch.device("cuda:0")
    before = _scan(dev)
    for limit in (1, 1000):
        status = torch.zeros((), dtype=torch.int32, device=dev)
        vla.selftest_wait_timeout(limit, status)
        torch.cuda.synchronize()                       # returns: the wait gave up by itself
        assert int(status.item()) == vla.VLA_ERR_DEVICE_TIMEOUT
        assert "wait" in vla.status_string(int(status.item()))
    after = _scan(dev)
    assert int(after.status.item()) == 0
    for a, b in ((before.out, after.out), (before.S_T, after.S_T), (before.A_T, after.A_T), (before.z_T, after.z_T)):
        assert torch.equal(a, b)


def test_a_status_word_already_set_is_not_overwritten():
    """First error wins: the kernels set the status with compare-and-swap against 0."""
    dev = torch.device("cuda:0")
    status = torch.full((), vla.VLA_ERR_NONFINITE, dtype=torch.int32, device=dev)
    vla.selftest_wait_timeout(10, status)
    torch.cuda.synchronize()
    assert int(status.item()) == vla.VLA_ERR_NONFINITE


@pytest.mark.parametrize("kernel", [vla.VLA_KERNEL_CHUNK, vla.VLA_KERNEL_CHUNK_TC])
def test_probe_limit_is_a_launch_parameter(kernel):
    """opts->wait_probe_limit reaches the kernels: a generous explicit limit changes nothing (the
    waits complete long before it), results are bit-identical to the default."""
    dev = torch.device("cuda:0")
    d = 128 if kernel == vla.VLA_KERNEL_CHUNK_TC else 64
    w = W.Workload("f", 1, 4, d, 90, "bf16", 22)
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    a = vla.vla_forward(q, k, v, 1.0, kernel=kernel)
    b = vla.vla_forward(q, k, v, 1.0, kernel=kernel, wait_probe_limit=1 << 20)
    torch.cuda.synchronize()
    assert int(a.status.item()) == 0 and int(b.status.item()) == 0
    assert torch.equal(a.out, b.out) and torch.equal(a.S_T, b.S_T) and torch.equal(a.A_T, b.A_T)


def test_selftest_rejects_bad_arguments():
    dev = torch.device("cuda:0")
    status = torch.zeros((), dtype=torch.int32, device=dev)
    with pytest.raises(vla.VlaError) as ei:
        vla.selftest_wait_timeout(0, status)
    assert ei.value.code == vla.VLA_ERR_INVALID_ARG


def test_last_launch_names_the_kernel_that_ran():
    dev = torch.device("cuda:0")
    _scan(dev, kernel=vla.VLA_KERNEL_CHUNK)
    assert vla.last_launch().startswith("vla_scan_chunk_kernel<64,f32>")
    _scan(dev, kernel=vla.VLA_KERNEL_TOKEN)
    assert vla.last_launch().startswith("vla_scan_token_kernel<64,f32>")
    w = W.Workload("f", 1, 2, 128, 40, "bf16", 23)
    q, k, v = [x.to(dev) for x in W.make_inputs(w)]
    vla.vla_forward(q, k, v, 1.0, kernel=vla.VLA_KERNEL_CHUNK_TC)
    assert vla.last_launch().startswith("vla_scan_tc_kernel<128,bf16>")
    torch.cuda.synchronize()
