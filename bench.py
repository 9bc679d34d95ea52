#!/usr/bin/env python
"""Benchmark of the VLA forward scan on B200.

A "step" is one pass of the whole hot path (stream in, prep, per-token Sherman-Morrison /
residual update / readout, stream out, final states) over one batch of synthetic input.
Default workload: "throughput" (B=32, H=16, d=128, T=8192, bf16 in, fp32 state) -- the
largest of the five workloads, and the one that fills the GPU.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--scaling weak|strong]
                  [--no-per-workload]
  python bench.py --impl reference ...     # the fp64 CPU oracle, as it stands, on host cores

For N > 1 launch with torch.distributed.run; by default every rank scans its own batch (weak
scaling), with --scaling strong the ranks split ONE batch contiguously by batch index; no
data-path collective either way.  Rank 0 prints ONE JSON line.  At N = 1 the line also carries
`per_workload`: kernel timings of the other four workloads and of the other entry points
(segmented forward, single-step decode, backward, projection of u, the opt-in tensor-core
kernel), each with the kernel name the library reports for what it launched.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

METRIC = "vla_forward_tokens_per_s"
UNIT = "tokens/s"

# FP32 FMA peak: SMs x 128 lanes x 2 flop x clock.  Nominal at the maximum SM clock; the
# achieved fraction is also reported at the clock sampled during the timed region.
FP32_LANES_PER_SM = 128


def alg_flops_per_token(d: int, has_u: bool = False) -> float:
    """Algorithmic fp32 work per token (u = k_hat): A u (d^2 FMA), the symmetric rank-1
    downdate (d(d+1)/2), S k_hat, S q_f and the S update (3 d^2); 2 flop per FMA."""
    fma = d * d + d * (d + 1) / 2 + 3 * d * d + (d * d if has_u else 0)
    return 2.0 * fma


def alg_bytes_per_token(d: int, in_bytes: int, has_u: bool = False) -> float:
    """q, k, v (and u) read once in their storage type, o written once in fp32."""
    return (3 + (1 if has_u else 0)) * d * in_bytes + 4 * d


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            pk = json.load(f)
        return float(pk["hbm_gbs"]), float(pk.get("sm_max_mhz", 1965.0)), "measured", float(pk.get("bf16_tflops", 1590.0))
    return 6650.0, 1965.0, "fallback", 1590.0


def ncu_traffic_per_token(kernel_key: str):
    """DRAM bytes per token of one ncu capture (profiles/ncu_traffic.txt: key, bytes, tokens, source)."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.txt")
    try:
        with open(path) as f:
            for ln in f:
                ln = ln.split("#")[0].split()
                if len(ln) >= 3 and ln[0] == kernel_key:
                    return float(ln[1]) / float(ln[2])
    except OSError:
        pass
    return None


def timed_ms(call, stream, dev, warm, reps, flush=None):
    """Median CUDA-event time of `call` on `stream` after `warm` untimed calls; `flush` (a buffer
    larger than L2) is rewritten before every timed call."""
    evs = []
    with torch.cuda.stream(stream):
        for _ in range(warm):
            call()
        for _ in range(reps):
            if flush is not None:
                flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); call(); b.record(stream)
            evs.append((a, b))
    torch.cuda.synchronize(dev)
    return float(np.median([a.elapsed_time(b) for a, b in evs]))


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.idx = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [r for (ts, r) in self.rows if t0 <= ts <= t1 + 0.2] or [r for (_, r) in self.rows]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except Exception:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_arrays(q, k, v):
    import oracle
    if q.dtype == torch.bfloat16:
        f = lambda x: x.contiguous().view(torch.int16).numpy().view(np.uint16)
        return f(q), f(k), f(v), oracle.BF16
    return q.contiguous().numpy(), k.contiguous().numpy(), v.contiguous().numpy(), oracle.F32


def time_oracle(w, q, k, v, budget_units=None):
    """The oracle as it stands on this machine's host cores, on a bounded sample of whole units
    of the same workload (units are independent; tokens/s scales with units)."""
    import oracle
    cores = max(1, len(os.sched_getaffinity(0)))
    # about 15 s of wall time: ~ 1 ns per fp64 multiply-add per core, 5 d^2 of them per token
    per_unit_s = w.T * 5 * w.d * w.d * 1.0e-9
    n_units = budget_units or int(max(1, min(w.units, round(15.0 * cores / max(per_unit_s, 1e-9)))))
    n_units = max(min(n_units, w.units), min(cores, w.units))
    qs = q.reshape(w.units, 1, w.T, w.d)[:n_units]
    ks = k.reshape(w.units, 1, w.T, w.d)[:n_units]
    vs = v.reshape(w.units, 1, w.T, w.d)[:n_units]
    qa, ka, va, dt = oracle_arrays(qs, ks, vs)
    threads = min(cores, n_units)
    t0 = time.perf_counter()
    oracle.forward(qa, ka, va, w.lam, in_dtype=dt, n_threads=threads)
    dt_s = time.perf_counter() - t0
    return {"value": n_units * w.T / dt_s, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "%d of %d units x T=%d tokens (whole units, first in batch order), fp64, %.1f s"
                      % (n_units, w.units, w.T, dt_s)}, dt_s, n_units


def run_reference(args):
    """--impl reference: the CPU oracle timed on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2605_11196_b200 import workloads as W
    w = W.WORKLOADS[args.workload]
    cores = max(1, len(os.sched_getaffinity(0)))
    # a step = a bounded sample of whole units, sized for ~3 s of wall time per step
    per_unit_s = w.T * 5 * w.d * w.d * 1.0e-9
    n_units = int(max(1, min(w.units, round(3.0 * cores / per_unit_s))))
    n_units = max(min(n_units, w.units), min(cores, w.units))
    ws = W.scaled(w, B=1, H=n_units)
    q, k, v = W.make_inputs(ws)
    times = []
    for it in range(args.warmup + args.steps):
        _, dt_s, _ = time_oracle(ws, q, k, v, budget_units=n_units)
        if it >= args.warmup:
            times.append(dt_s)
    total = sum(times)
    val = args.steps * n_units * w.T / total
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic (seeded N(0,1), the workload's recipe)",
            "config": {"workload": w.name, "B": w.B, "H": w.H, "d_k": w.d, "d_v": w.d, "T": w.T,
                       "in_dtype": w.dtype, "lambda": w.lam,
                       "sample": "%d of %d units per step" % (n_units, w.units)},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": min(cores, n_units), "kind": "oracle",
                             "sample": "%d of %d whole units x T=%d per step" % (n_units, w.units, w.T)},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def bench_one(vla, w, dev, q, k, v, steps, warmup, stream, kernel="auto"):
    """Device-resident timing of `steps` launches; returns (seconds for all steps, per-launch ms list)."""
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    out = torch.empty((w.B, w.H, w.T, w.d), dtype=torch.float32, device=dev)
    S_T = torch.empty((w.B, w.H, w.d, w.d), dtype=torch.float32, device=dev)
    A_T = torch.empty_like(S_T)
    z_T = torch.empty((w.B, w.H, w.d), dtype=torch.float32, device=dev)
    status = torch.zeros((), dtype=torch.int32, device=dev)
    kern = {"auto": vla.VLA_KERNEL_AUTO, "token": vla.VLA_KERNEL_TOKEN, "chunk": vla.VLA_KERNEL_CHUNK,
            "chunk_tc": vla.VLA_KERNEL_CHUNK_TC}[kernel]
    call = lambda: vla.vla_forward(qd, kd, vd, w.lam, out=out, S_T=S_T, A_T=A_T, z_T=z_T,
                                   status=status, stream=stream, kernel=kern)
    return (qd, kd, vd, out, S_T, A_T, z_T, status), call


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="throughput")
    ap.add_argument("--all-workloads", action="store_true", help="(default at N = 1; kept for old command lines)")
    ap.add_argument("--no-per-workload", action="store_true",
                    help="skip 'per_workload' (the other four workloads and entry points, kernel only)")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="N > 1: every rank its own batch (weak) or one batch split by batch index (strong)")
    ap.add_argument("--B", type=int, default=None, help="override the workload's batch (profiling cases)")
    ap.add_argument("--H", type=int, default=None, help="override the workload's heads")
    ap.add_argument("--T", type=int, default=None, help="override the workload's sequence length")
    ap.add_argument("--kernel", default="auto", choices=["auto", "token", "chunk", "chunk_tc"],
                    help="force a kernel for the headline call (profiling; the default is the library's own choice)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()

    if args.impl == "reference":
        run_reference(args)
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)

    import paper_2605_11196_b200 as vla
    from paper_2605_11196_b200 import workloads as W
    vla.load_library()                        # raises if the CUDA library is missing
    w = W.WORKLOADS[args.workload]
    over = {n: getattr(args, n) for n in ("B", "H", "T") if getattr(args, n) is not None}
    if over:
        w = W.scaled(w, name=w.name + "-resized", **over)
    hbm_peak, sm_max_mhz, peak_src, bf16_peak = measured_peaks()
    n_sm = torch.cuda.get_device_properties(dev).multi_processor_count

    strong = args.scaling == "strong" and world > 1
    if strong:
        # ONE batch (the same seed on every rank), split contiguously by batch index
        from paper_2605_11196_b200 import sharding as SH
        w_full = w
        q, k, v = [x.contiguous() for x in SH.shard_batch(W.make_inputs(w), world, rank)]
        b0, b1 = SH.batch_bounds(w.B, world, rank)
        if b1 == b0:
            raise SystemExit("--scaling strong: rank %d of %d has no batch of B = %d (replicas only)" % (rank, world, w.B))
        w = W.scaled(w, B=b1 - b0)
    else:
        w_full = w
        q, k, v = W.make_inputs(w, rank=rank)
    stream = torch.cuda.Stream(dev)
    bufs, call = bench_one(vla, w, dev, q, k, v, args.steps, args.warmup, stream, args.kernel)
    qd, kd, vd, out, S_T, A_T, z_T, status = bufs
    in_bytes = 2 if w.dtype == "bf16" else 4
    working_set = 3 * w.tokens * w.d * in_bytes + w.tokens * w.d * 4
    l2_bytes = 126 * 2 ** 20
    flush = None
    if working_set <= 2 * l2_bytes:           # small workloads: flush L2 between timed steps
        flush = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device=dev)

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 0)):
            call()
    barrier()

    # ---- kernel-only timed region: K steps, events on the launching stream
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
          for _ in range(args.steps)]
    barrier()
    t_wall0 = time.time()
    with torch.cuda.stream(stream):
        for (e0, e1) in ev:
            if flush is not None:
                flush.fill_(1)
            e0.record(stream)
            call()
            e1.record(stream)
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    per_launch_ms = [e0.elapsed_time(e1) for (e0, e1) in ev]
    total_s = sum(per_launch_ms) / 1e3
    assert int(status.item()) == 0, vla.status_string(int(status.item()))
    tt = torch.tensor([total_s], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    total_s_max = float(tt.item())
    job_tokens = w_full.tokens if strong else world * w.tokens
    value = args.steps * job_tokens / total_s_max
    launched = vla.last_launch()              # what the library launched for the timed call

    # ---- end to end: pinned host buffers in, host buffers out, through vla_forward_host
    e2e = None
    if not args.no_e2e:
        ws_bytes = vla.vla_host_workspace_bytes(w.B, w.H, w.T, w.d, w.d,
                                                vla.VLA_BF16 if w.dtype == "bf16" else vla.VLA_F32)
        wsbuf = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        qp, kp, vp = q.pin_memory(), k.pin_memory(), v.pin_memory()
        outp = torch.empty((w.B, w.H, w.T, w.d), dtype=torch.float32).pin_memory()
        STp = torch.empty((w.B, w.H, w.d, w.d), dtype=torch.float32).pin_memory()
        ATp = torch.empty_like(STp).pin_memory()
        zTp = torch.empty((w.B, w.H, w.d), dtype=torch.float32).pin_memory()
        e2e_steps = max(1, min(args.steps, 3))
        hcall = lambda: vla.vla_forward_host(qp, kp, vp, w.lam, wsbuf, out=outp, S_T=STp, A_T=ATp,
                                             z_T=zTp, status=status, stream=stream)
        with torch.cuda.stream(stream):
            hcall()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _ in range(e2e_steps):
                hcall()
            e1.record(stream)
        barrier()
        t = torch.tensor([e0.elapsed_time(e1) / 1e3], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        h2d = 3 * w.tokens * w.d * in_bytes
        d2h = w.tokens * w.d * 4 + w.units * (2 * w.d * w.d + w.d) * 4
        e2e = {"value": e2e_steps * job_tokens / float(t.item()), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "api": "vla_forward_host (pinned host q,k,v in; out, S_T, A_T, z_T to pinned host)"}
        # the copy ceiling of this machine: the same byte counts, one pinned copy per direction, alone
        if rank == 0:
            stage = wsbuf[:max(h2d, w.tokens * w.d * 4)]
            src = torch.empty(h2d, dtype=torch.uint8).pin_memory()
            dst = outp.view(torch.uint8).view(-1)
            def copy_ms(fn):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                with torch.cuda.stream(stream):
                    fn(); a.record(stream); fn(); b.record(stream)
                torch.cuda.synchronize(dev)
                return a.elapsed_time(b)
            t_h2d = copy_ms(lambda: stage[:h2d].copy_(src, non_blocking=True))
            t_d2h = copy_ms(lambda: dst.copy_(stage[:dst.numel()], non_blocking=True))
            e2e["pcie_h2d_gbs"] = h2d / (t_h2d * 1e-3) / 1e9
            e2e["pcie_d2h_gbs"] = dst.numel() / (t_d2h * 1e-3) / 1e9
            # both directions at once (what a fully overlapped pipeline sees): the same two copies
            # on two streams, timed together
            s2 = torch.cuda.Stream(dev)
            stage2 = torch.empty(dst.numel(), dtype=torch.uint8, device=dev)
            def both():
                s2.wait_stream(stream)
                with torch.cuda.stream(s2):
                    dst.copy_(stage2, non_blocking=True)
                stage[:h2d].copy_(src, non_blocking=True)
                stream.wait_stream(s2)
            t_both = copy_ms(both)
            e2e["pcie_both_directions_ms"] = t_both
            e2e["frac_of_concurrent_copy_time"] = (t_both * 1e-3) / (job_tokens / e2e["value"])   # copies alone / a whole step
            del stage2
            floor_s = max(h2d / (e2e["pcie_h2d_gbs"] * 1e9), d2h / (e2e["pcie_d2h_gbs"] * 1e9))
            e2e["copy_bound_tokens_per_s"] = w.tokens / floor_s       # both directions fully overlapped
            e2e["frac_of_copy_bound"] = (e2e["value"] * w.tokens / job_tokens) / e2e["copy_bound_tokens_per_s"]
            del src
        del wsbuf

    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    # ---- roofline of the (single) scan kernel, from the live event timings
    launch_ms = float(np.mean(per_launch_ms))
    flops = alg_flops_per_token(w.d) * w.tokens
    byts = alg_bytes_per_token(w.d, in_bytes) * w.tokens + w.units * (2 * w.d * w.d) * 4
    fp32_peak_nominal = n_sm * FP32_LANES_PER_SM * 2 * sm_max_mhz * 1e6 / 1e12       # TFLOP/s
    t_alu = flops / (fp32_peak_nominal * 1e12)
    t_hbm = byts / (hbm_peak * 1e9)
    bound = "alu" if t_alu >= t_hbm else "hbm"
    achieved_tflops = flops / (launch_ms * 1e-3) / 1e12
    achieved_gbs = byts / (launch_ms * 1e-3) / 1e9
    traffic_pt = ncu_traffic_per_token("%s<%d,%s>" % (launched.split("<")[0], w.d, w.dtype))
    fp32_src = "fp32 FMA: %d SMs x 128 lanes x 2 x %.0f MHz (derived, nominal max clock)" % (n_sm, sm_max_mhz)
    on_tensor_cores = launched.startswith("vla_scan_tc_kernel")
    if on_tensor_cores and bound == "alu":
        # The d x d products of the chunk algebra run as tcgen05.mma kind::tf32, each as three TF32
        # products (hi*hi, hi*lo, lo*hi) for fp32 accuracy: the peak for the algorithmic flops is
        # the dense TF32 rate / 3.  TF32 rate = the measured bf16 GEMM rate x the nominal
        # TF32 : bf16 ratio (1.1 : 2.25 PFLOP/s).
        tf32_peak = bf16_peak * (1.1 / 2.25)
        roof = {"bound": "tensor", "kernel": launched, "achieved": achieved_tflops, "peak": tf32_peak / 3.0,
                "unit": "TFLOP/s", "frac": achieved_tflops / (tf32_peak / 3.0),
                "peak_source": ("dense TF32 / 3 passes (hi/lo operand pairs): bf16_tflops of %s (%.0f) x 1.1/2.25 / 3"
                                % (peak_src, bf16_peak)),
                "fp32_alu_peak": fp32_peak_nominal, "fp32_alu_frac": achieved_tflops / fp32_peak_nominal,
                "fp32_alu_peak_source": fp32_src}
    else:
        roof = {"bound": bound, "kernel": launched,
                "achieved": achieved_tflops if bound == "alu" else achieved_gbs,
                "peak": fp32_peak_nominal if bound == "alu" else hbm_peak,
                "unit": "TFLOP/s" if bound == "alu" else "GB/s",
                "frac": (achieved_tflops / fp32_peak_nominal) if bound == "alu" else achieved_gbs / hbm_peak,
                "peak_source": fp32_src if bound == "alu" else "hbm_gbs of %s" % peak_src}
    roof.update({
            # dram__bytes_read + write of one ncu capture of this kernel, scaled by tokens
            # (profiles/ncu_traffic.txt names the capture)
            "traffic": traffic_pt * w.tokens if traffic_pt else None,
            "alg_flops_per_token": alg_flops_per_token(w.d),
            "alg_bytes_per_token": alg_bytes_per_token(w.d, in_bytes),
            "hbm_achieved_gbs": achieved_gbs, "hbm_peak_gbs": hbm_peak, "hbm_peak_source": peak_src,
            "hbm_frac": achieved_gbs / hbm_peak,
            "launch_ms": launch_ms,
            "unit_limited_frac_bound": min(w.units, n_sm) / n_sm})
    if clocks and clocks.get("sm_mhz"):
        roof["frac_at_sampled_clock"] = achieved_tflops / (fp32_peak_nominal * clocks["sm_mhz"] / sm_max_mhz)
    # the fp32 FMA rate this device sustains right now (register-only loop in the library),
    # measured after the timed region so that it cannot disturb it
    try:
        measured = vla.measure_fp32_fma_tflops(dev)
        roof["fp32_peak_measured_tflops"] = measured
        roof["frac_of_measured_fp32"] = achieved_tflops / measured
    except Exception as exc:   # the roofline above stands on the derived peak
        roof["fp32_peak_measured_tflops"] = None
        roof["fp32_peak_measured_error"] = str(exc)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * total_s_max / args.steps,
            "higher_is_better": True, "scaling": "strong" if strong else "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic (seeded N(0,1) q,k,v rounded to %s; %s)"
                    % (w.dtype, "one batch split by batch index over the ranks" if strong else "each rank its own batch"),
            "config": {"workload": w_full.name, "B": w_full.B, "H": w_full.H, "d_k": w.d, "d_v": w.d, "T": w.T,
                       "in_dtype": w.dtype, "state_dtype": "f32", "lambda": w.lam, "u": "k_hat",
                       "mode": "Algorithm 1 (phi = ELU+1, normalised readout)",
                       "parallelism": "dp%d over (batch, head) units, no collective%s"
                                      % (world, ", B split %s per rank" % (w.B,) if strong else ""),
                       "l2": ("inputs+outputs %.0f MB > L2" % (working_set / 1e6)) if flush is None
                             else "L2 flushed between timed steps (256 MB write)",
                       **({"kernel_forced": args.kernel} if args.kernel != "auto" else {})},
            "ns_per_scan_step": 1e6 * launch_ms / w.T,
            "roofline": roof, "e2e": e2e, "gpu_launches": args.steps, "clocks": clocks}

    if world == 1 and not args.no_per_workload:
        per = {}
        fl = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device=dev)     # L2 flush between timed calls
        frac = lambda ww, ms, has_u=False: alg_flops_per_token(ww.d, has_u) * ww.tokens / (ms * 1e-3) / 1e12 / fp32_peak_nominal

        def entry(ww, ms, **kw):
            e = {"ms": ms, "tokens_per_s": ww.tokens / (ms * 1e-3), "ns_per_scan_step": 1e6 * ms / ww.T,
                 "units": ww.units, "kernel": vla.last_launch()}
            e.update(kw)
            return e

        # ---- the other four workloads: plain call, the library's choice of kernel
        for name in W.ORDER:
            if name == w.name:
                continue
            ww = W.WORKLOADS[name]
            q2, k2, v2 = W.make_inputs(ww)
            _, call2 = bench_one(vla, ww, dev, q2, k2, v2, 0, 0, stream)
            ms = timed_ms(call2, stream, dev, 3, 10, fl)
            ib = 2 if ww.dtype == "bf16" else 4
            per[name] = entry(ww, ms, fp32_frac_nominal=frac(ww, ms),
                              hbm_frac=alg_bytes_per_token(ww.d, ib) * ww.tokens / (ms * 1e-3) / 1e9 / hbm_peak,
                              unit_limited_frac_bound=min(ww.units, n_sm) / n_sm)
            qd2, kd2, vd2 = q2.to(dev), k2.to(dev), v2.to(dev)
            # backward pass: forward recomputed inside (chunk kernel leaving the per-token stash),
            # both reverse scans as one launch, the dA0 kernel
            if name in ("mid", "recall"):
                go3 = torch.randn((ww.B, ww.H, ww.T, ww.d), device=dev)
                ms = timed_ms(lambda: vla.vla_backward(qd2, kd2, vd2, ww.lam, go3, stream=stream), stream, dev, 1, 3, fl)
                per[name + "_backward"] = entry(ww, ms, gpu_launches_per_step=3,
                                                forward_ms=per[name]["ms"], ratio_to_forward=ms / per[name]["ms"])
                del go3
            # fewer units than SMs: with scratch memory the plain call cuts each sequence into
            # segments that are scanned concurrently (twice the arithmetic, P times the CTAs)
            P = vla.seqpar_segments(ww.B, ww.H, ww.T, ww.d, q2.dtype)
            if P > 1:
                ws = torch.empty((vla.seqpar_workspace_bytes(ww.B, ww.H, ww.T, ww.d, P),), dtype=torch.uint8, device=dev)
                o2 = torch.empty((ww.B, ww.H, ww.T, ww.d), dtype=torch.float32, device=dev)
                S2 = torch.empty((ww.B, ww.H, ww.d, ww.d), dtype=torch.float32, device=dev)
                A2 = torch.empty_like(S2)
                z2 = torch.empty((ww.B, ww.H, ww.d), dtype=torch.float32, device=dev)
                st2 = torch.zeros((), dtype=torch.int32, device=dev)
                call3 = lambda: vla.vla_forward(qd2, kd2, vd2, ww.lam, workspace=ws, out=o2, S_T=S2, A_T=A2,
                                                z_T=z2, status=st2, stream=stream)
                ms = timed_ms(call3, stream, dev, 3, 10, fl)
                per[name + "_auto_with_workspace"] = entry(
                    ww, ms, segments=P, fp32_frac_nominal=frac(ww, ms), status=int(st2.item()),
                    api="vla_forward, kernel AUTO, opts->workspace given (runs as vla_forward_seqpar)",
                    gpu_launches_per_step=5, unit_limited_frac_bound=min(ww.units * P, n_sm) / n_sm)
                del ws, o2, S2, A2, z2
            del qd2, kd2, vd2

        # ---- the headline workload through the other entry points and options
        go_h = torch.randn((w.B, w.H, w.T, w.d), device=dev)
        wsb = torch.empty((vla.backward_workspace_bytes(w.B, w.H, w.T, w.d),), dtype=torch.uint8, device=dev)
        ms = timed_ms(lambda: vla.vla_backward(qd, kd, vd, w.lam, go_h, workspace=wsb, stream=stream), stream, dev, 1, 2)
        per[w.name + "_backward"] = entry(w, ms, gpu_launches_per_step=3, forward_ms=launch_ms,
                                          ratio_to_forward=ms / launch_ms)
        uu = W.make_u(w, w.d ** -0.5).to(dev)      # explicit penalty directions u = unit / sqrt(d_h)
        ms = timed_ms(lambda: vla.vla_backward(qd, kd, vd, w.lam, go_h, u=uu, workspace=wsb, stream=stream), stream, dev, 1, 2)
        per[w.name + "_backward_explicit_u"] = entry(w, ms, gpu_launches_per_step=3)
        del go_h, wsb
        fwd = dict(out=out, S_T=S_T, A_T=A_T, z_T=z_T, status=status, stream=stream)
        ms = timed_ms(lambda: vla.vla_forward(qd, kd, vd, w.lam, u=uu, **fwd), stream, dev, 2, 3)
        per[w.name + "_explicit_u"] = entry(w, ms, fp32_frac_nominal=frac(w, ms, True))
        # u formed on the device from a projection (Algorithm 1: u = L2norm(W_u k) / sqrt(d_h))
        Wu = (torch.randn((w.H, w.d, w.d), generator=torch.Generator().manual_seed(11)) / w.d ** 0.5).to(dev)
        ms_mk = timed_ms(lambda: vla.vla_make_u(kd, Wu, out=uu, stream=stream), stream, dev, 1, 3)
        in_b = 2 if w.dtype == "bf16" else 4
        per[w.name + "_make_u"] = {"ms": ms_mk, "tokens_per_s": w.tokens / (ms_mk * 1e-3),
                                   "kernel": "vla_make_u_tc_kernel (tcgen05, TF32 hi/lo)" if w.d == 128 else "vla_make_u_kernel",
                                   "tflops": 2.0 * w.d * w.d * w.tokens / (ms_mk * 1e-3) / 1e12,
                                   "hbm_frac": 2.0 * w.tokens * w.d * in_b / (ms_mk * 1e-3) / 1e9 / hbm_peak}
        def wcall():
            vla.vla_make_u(kd, Wu, out=uu, stream=stream)
            vla.vla_forward(qd, kd, vd, w.lam, u=uu, **fwd)
        ms = timed_ms(wcall, stream, dev, 1, 3)
        per[w.name + "_projected_u"] = entry(w, ms, gpu_launches_per_step=2)
        del uu, Wu
        # Algorithm 1's periodic refresh (every 20 tokens, + 1e-3 I)
        ms = timed_ms(lambda: vla.vla_forward(qd, kd, vd, w.lam, refresh=(20, 1e-3, 0), **fwd), stream, dev, 2, 3)
        per[w.name + "_refresh_20"] = entry(w, ms, fp32_frac_nominal=frac(w, ms))
        # q, k, v, out as [B, T, H, d]
        qt, kt, vt = [x.view(w.B, w.H, w.T, w.d).permute(0, 2, 1, 3).contiguous() for x in (qd, kd, vd)]
        out_t = torch.empty((w.B, w.T, w.H, w.d), dtype=torch.float32, device=dev)
        ms = timed_ms(lambda: vla.vla_forward(qt, kt, vt, w.lam, out=out_t, S_T=S_T, A_T=A_T, z_T=z_T, status=status,
                                              stream=stream, flags=vla.VLA_FLAG_TOKEN_MAJOR), stream, dev, 1, 3)
        per[w.name + "_token_major"] = entry(w, ms, fp32_frac_nominal=frac(w, ms))
        del qt, kt, vt, out_t
        # the fp32-FMA form of the chunk kernel on the same workload (the library's choice at
        # d = 128 is the tensor-core form)
        if w.d == 128:
            ms = timed_ms(lambda: vla.vla_forward(qd, kd, vd, w.lam, kernel=vla.VLA_KERNEL_CHUNK, **fwd), stream, dev, 2, 3)
            per[w.name + "_chunk_fma"] = entry(w, ms, fp32_frac_nominal=frac(w, ms))
            ms = timed_ms(lambda: vla.vla_forward(qd, kd, vd, w.lam, flags=vla.VLA_FLAG_IDENTITY_MAP, **fwd), stream, dev, 2, 3)
            per[w.name + "_identity_map"] = entry(w, ms, fp32_frac_nominal=frac(w, ms))
        # single-step decode (T = 1, carried states): bound by moving S and A through HBM once
        wd = W.EXTRA["decode"]
        q2, k2, v2 = [x.to(dev) for x in W.make_inputs(wd)]
        S0 = torch.zeros((wd.B, wd.H, wd.d, wd.d), device=dev)
        A0 = torch.eye(wd.d, device=dev).expand(wd.B, wd.H, wd.d, wd.d).contiguous()
        bufs = dict(out=torch.empty((wd.B, wd.H, 1, wd.d), device=dev), S_T=torch.empty_like(S0),
                    A_T=torch.empty_like(A0), z_T=torch.empty((wd.B, wd.H, wd.d), device=dev), status=status)
        state_bytes = wd.units * (4 * wd.d * wd.d * 4 + 2 * wd.d * 4)       # S, A read and written; z
        io_bytes = wd.units * (3 * wd.d * 2 + wd.d * 4)
        for key, kern in (("decode", vla.VLA_KERNEL_AUTO), ("decode_token_kernel", vla.VLA_KERNEL_TOKEN)):
            dcall = lambda: vla.vla_forward(q2, k2, v2, wd.lam, S0=S0, A0=A0, stream=stream, kernel=kern, **bufs)
            ms = timed_ms(dcall, stream, dev, 3, 10, fl)
            per[key] = {"ms": ms, "units": wd.units, "steps_per_s": wd.units / (ms * 1e-3),
                        "kernel": vla.last_launch(), "bound": "hbm",
                        "hbm_gbs": (state_bytes + io_bytes) / (ms * 1e-3) / 1e9,
                        "hbm_frac": (state_bytes + io_bytes) / (ms * 1e-3) / 1e9 / hbm_peak,
                        "hbm_peak_source": peak_src}
        assert int(status.item()) == 0, vla.status_string(int(status.item()))
        line["per_workload"] = per

    if not args.no_cpu_baseline:
        cb, _, _ = time_oracle(w, q, k, v)
        line["cpu_baseline"] = cb

    print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
