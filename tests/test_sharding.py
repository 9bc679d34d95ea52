"""The multi-GPU path shards (batch, head) units over ranks with no collective on the data
path.  This checks the host-side logic with two gloo ranks on CPU: each rank draws its own
batch (rank-offset seed), the per-rank results concatenate to what one process computes for
both batches, and the max-over-ranks timing reduction works."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import numpy as np, torch, torch.distributed as dist
    import oracle
    from paper_2605_11196_b200 import workloads as W
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    w = W.Workload("shard", 2, 2, 16, 40, "f32", 77)
    q, k, v = W.make_inputs(w, rank=rank)              # weak scaling: one batch per rank
    r = oracle.forward(q.numpy(), k.numpy(), v.numpy(), w.lam)   # stands in for the GPU call
    mine = torch.from_numpy(r.out)
    gathered = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine)                    # a caller-side gather, not part of the path
    t = torch.tensor([1.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        for rr in range(world):
            q2, k2, v2 = W.make_inputs(w, rank=rr)
            ref = oracle.forward(q2.numpy(), k2.numpy(), v2.numpy(), w.lam).out
            assert np.array_equal(gathered[rr].numpy(), ref), rr
        assert not np.array_equal(gathered[0].numpy(), gathered[1].numpy())   # different batches
        assert float(t) == float(world)
        print("SHARD_OK tokens", world * w.tokens)
    dist.barrier()
    dist.destroy_process_group()
""") % ROOT


STRONG_WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import numpy as np, torch, torch.distributed as dist
    import oracle
    from paper_2605_11196_b200 import workloads as W, sharding as SH
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    # ONE problem, the same on every rank (same seed), split contiguously by batch index
    w = W.Workload("strong", 5, 2, 16, 33, "f32", 78)
    q, k, v = W.make_inputs(w)
    g = torch.Generator().manual_seed(5)
    S0 = torch.randn((w.B, w.H, w.d, w.d), generator=g, dtype=torch.float64) * 0.1
    b0, b1 = SH.batch_bounds(w.B, world, rank)
    assert (b0, b1) == ((0, 2), (2, 5))[rank]
    qs, ks, vs, S0s = SH.shard_batch([q, k, v, S0], world, rank)
    assert qs.is_contiguous() and S0s.is_contiguous()          # contiguous blocks of the caller's tensors
    r = oracle.forward(qs.numpy(), ks.numpy(), vs.numpy(), w.lam, S0=S0s.numpy())   # stands in for the GPU call
    parts = {}
    for name, mine in (("out", r.out), ("S_T", r.S_T), ("A_T", r.A_T)):
        sizes = [SH.batch_bounds(w.B, world, rr) for rr in range(world)]
        bufs = [torch.empty((e - b,) + mine.shape[1:], dtype=torch.float64) for (b, e) in sizes]
        bufs[rank] = torch.from_numpy(mine).clone()
        for rr in range(world):                                # unequal shards: one broadcast per rank
            dist.broadcast(bufs[rr], src=rr)                   # (a caller-side gather, not part of the path)
        parts[name] = SH.assemble_batch(bufs, w.B)
    if rank == 0:
        ref = oracle.forward(q.numpy(), k.numpy(), v.numpy(), w.lam, S0=S0.numpy())
        for name in ("out", "S_T", "A_T"):
            assert np.array_equal(parts[name].numpy(), getattr(ref, name)), name   # bit for bit
        print("STRONG_OK", tuple(parts["out"].shape))
    dist.barrier()
    dist.destroy_process_group()
""") % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_ranks_shard_units_without_a_collective(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=300)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert "SHARD_OK tokens 320" in outs[0]


def test_one_problem_split_by_batch_index_reassembles_bit_exactly(tmp_path):
    """Strong scaling's partition: one [B,H,T,d] problem cut contiguously by b over two ranks
    (unequal shards: 2 and 3 batches), each shard scanned on its own, the pieces put back in
    rank order: identical to the unsplit result, with no exchange during the scan."""
    script = tmp_path / "strong_worker.py"
    script.write_text(STRONG_WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=300)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert "STRONG_OK (5, 2, 33, 16)" in outs[0]


def test_batch_bounds_cover_the_batch_once():
    from paper_2605_11196_b200 import sharding as SH
    for B in (0, 1, 5, 8, 64):
        for world in (1, 2, 3, 8):
            spans = [SH.batch_bounds(B, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1


def test_reference_arm_prints_one_json_line_and_other_ranks_stay_silent():
    import json
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
           "--steps", "2", "--warmup", "1"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300,
                         env=dict(os.environ, RANK="0", WORLD_SIZE="2"))
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
    out1 = subprocess.run(cmd, capture_output=True, text=True, timeout=300,
                          env=dict(os.environ, RANK="1", WORLD_SIZE="2"))
    assert out1.returncode == 0 and out1.stdout.strip() == ""
