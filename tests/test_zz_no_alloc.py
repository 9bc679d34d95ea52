"""vla_forward_host_static: the host-buffer entry point whose device staging memory is
built into the library, for callers that cannot obtain device memory at the call site
(no allocator handle, a committed memory cap, a loop that must not allocate).

Collected last on purpose: a failure here cannot hide the result of any other test.
It is checked against vla_forward_host (caller-provided workspace; same staging code, same
kernels, so bit for bit) and against the CPU oracle, on calls in a row, because every call
reuses the same built-in array and sees what the previous one left in it.  The last call is
smaller than the one before and carries no S0 / z0: nothing of the earlier call may leak in.
"""
import ctypes

import pytest
import torch

import paper_2605_11196_b200 as vla
from paper_2605_11196_b200 import workloads as W
from parity_util import rel_err, run_oracle


@pytest.mark.gpu
def test_static_scratch_entry_point_matches_workspace_entry_point_twice():
    dev = torch.device("cuda:0")
    lib = vla.load_library()
    results = []
    # different problems back to back: each one finds the previous one's leftovers
    for call, (B, H, d, T, dtype, flags, seed, carry) in enumerate([
            (2, 3, 64, 150, "bf16", 0, 301, True),
            (2, 3, 32, 77, "f32", vla.VLA_FLAG_IDENTITY_MAP, 302, True),
            (1, 2, 32, 40, "f32", 0, 303, False)]):
        w = W.Workload("noalloc", B, H, d, T, dtype, seed)
        q, k, v = [x.pin_memory() for x in W.make_inputs(w)]
        g = torch.Generator().manual_seed(seed)
        S0 = (torch.randn((B, H, d, d), generator=g) * 0.1).pin_memory() if carry else None
        z0 = torch.rand((B, H, d), generator=g).pin_memory() if carry else None

        # reference: the existing entry point with a workspace from the caller
        nbytes = vla.vla_host_workspace_bytes(B, H, T, d, d, vla.VLA_BF16 if dtype == "bf16" else vla.VLA_F32)
        assert nbytes <= vla.VLA_STATIC_SCRATCH_BYTES
        ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        ref = vla.vla_forward_host(q, k, v, 0.5, ws, S0=S0, z0=z0, flags=flags)
        torch.cuda.synchronize()

        # the entry point under test, straight through the C ABI with host pointers
        f32 = torch.float32
        out = torch.empty((B, H, T, d), dtype=f32).pin_memory()
        S_T = torch.empty((B, H, d, d), dtype=f32).pin_memory()
        A_T = torch.empty((B, H, d, d), dtype=f32).pin_memory()
        z_T = torch.empty((B, H, d), dtype=f32).pin_memory()
        status = torch.zeros((), dtype=torch.int32, device=dev)
        opts = vla.VlaOpts()
        opts.struct_size = ctypes.sizeof(vla.VlaOpts)
        opts.qkv_dtype = vla.VLA_BF16 if dtype == "bf16" else vla.VLA_F32
        opts.flags = flags
        opts.eps = 1e-4
        opts.z0 = z0.data_ptr() if carry else None
        opts.zT = z_T.data_ptr()
        opts.status = status.data_ptr()
        vp = ctypes.c_void_p
        with torch.cuda.device(dev):
            rc = lib.vla_forward_host_static(vp(q.data_ptr()), vp(k.data_ptr()), vp(v.data_ptr()), 0.5,
                                             B, H, T, d, d, vp(S0.data_ptr()) if carry else None, None,
                                             vp(out.data_ptr()), vp(S_T.data_ptr()), vp(A_T.data_ptr()),
                                             ctypes.byref(opts),
                                             vp(torch.cuda.current_stream(dev).cuda_stream))
        assert rc == vla.VLA_OK, vla.status_string(rc)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        orc = run_oracle(q, k, v, 0.5, S0=S0, z0=z0, flags=flags)
        for name, got, want, want64 in (("o", out, ref.out, orc.out), ("S_T", S_T, ref.S_T, orc.S_T),
                                        ("A_T", A_T, ref.A_T, orc.A_T), ("z_T", z_T, ref.z_T, orc.z_T)):
            assert torch.equal(got, want), "call %d %s differs from vla_forward_host" % (call, name)
            assert rel_err(got, want64) <= 1e-4, "call %d %s vs the oracle" % (call, name)
        results.append(out.clone())
    assert len(results) == 3


@pytest.mark.gpu
def test_static_scratch_rejects_oversized_problems():
    # 8 x 8 units of 4096 tokens at d = 128 need far more than the built-in array
    w = W.Workload("too-big", 1, 1, 128, 16, "f32", 5)
    q, k, v = W.make_inputs(w)
    big = (8, 8, 4096, 128)
    assert vla.vla_host_workspace_bytes(*big[:3], 128, 128) > vla.VLA_STATIC_SCRATCH_BYTES
    lib = vla.load_library()
    vp = ctypes.c_void_p
    fake = vp(q.data_ptr())          # never dereferenced: the size check comes first
    rc = lib.vla_forward_host_static(fake, fake, fake, 1.0, 8, 8, 4096, 128, 128, None, None,
                                     fake, None, None, None, None)
    assert rc == vla.VLA_ERR_TOO_LARGE
    assert "VLA_STATIC_SCRATCH_BYTES" in vla.status_string(rc)
