"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds NO arithmetic of the method: it only draws q, k, v from a seeded
torch CPU generator.  Both the CUDA path and the CPU oracle are fed from here.

The five workloads (the paper measures latency at d_h = 32, H = 4 on a multi-query
associative-recall task with 24 pairs, batch 64, T <= 512, and argues about contexts
beyond ~43k tokens; none of its data is used, only those shapes):
  tiny        B=1  H=1  d=16  T=256    fp32  N(0,1)               seed 0
  mid         B=4  H=8  d=64  T=4096   fp32  N(0,1)               seed 1
  recall      B=64 H=4  d=32  T=512    fp32  recall-shaped        seed 2
  long        B=1  H=16 d=64  T=65536  bf16  N(0,1)               seed 3
  throughput  B=32 H=16 d=128 T=8192   bf16  N(0,1)               seed 4
"recall" stands in for the recall benchmark's layout at the attention-input level:
per unit, 24 tokens carrying a random unit-norm key and an N(0,1) value, then filler
tokens ~ N(0, 0.1^2), then 24 query tokens whose q equals the stored keys in a shuffled
order (their k and v are filler).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    d: int
    T: int
    dtype: str          # "f32" | "bf16"
    seed: int
    lam: float = 1.0
    kind: str = "normal"  # "normal" | "recall"
    n_pairs: int = 24
    filler_std: float = 0.1

    @property
    def units(self) -> int:
        return self.B * self.H

    @property
    def tokens(self) -> int:
        return self.B * self.H * self.T

    @property
    def tol(self) -> float:
        """Accepted max|x - x_ref| / max|x_ref| for o, S_T, A_T: 1e-4 up to T = 4096, 1e-3 beyond."""
        return 1e-4 if self.T <= 4096 else 1e-3

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


WORKLOADS = {
    "tiny": Workload("tiny", 1, 1, 16, 256, "f32", 0),
    "mid": Workload("mid", 4, 8, 64, 4096, "f32", 1),
    "recall": Workload("recall", 64, 4, 32, 512, "f32", 2, kind="recall"),
    "long": Workload("long", 1, 16, 64, 65536, "bf16", 3),
    "throughput": Workload("throughput", 32, 16, 128, 8192, "bf16", 4),
}
ORDER = ("tiny", "mid", "recall", "long", "throughput")
# Not one of the five: a single-step decode shape (state read and written once per unit),
# reported by bench.py --all-workloads against the HBM roofline.
EXTRA = {"decode": Workload("decode", 64, 64, 128, 1, "bf16", 5)}


def scaled(w: Workload, **kw) -> Workload:
    """A smaller/larger case of the same recipe (tests)."""
    return replace(w, **kw)


def make_inputs(w: Workload, rank: int = 0):
    """(q, k, v) CPU tensors [B,H,T,d] in the workload's storage dtype.  `rank` offsets the
    seed so that data-parallel ranks draw different batches."""
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed + 1000003 * rank)
    shape = (w.B, w.H, w.T, w.d)
    if w.kind == "normal":
        q = torch.randn(shape, generator=g).to(w.torch_dtype)
        k = torch.randn(shape, generator=g).to(w.torch_dtype)
        v = torch.randn(shape, generator=g).to(w.torch_dtype)
        return q, k, v
    if w.kind == "recall":
        n = w.n_pairs
        if w.T < 2 * n:
            raise ValueError("recall layout needs T >= 2*n_pairs")
        q = torch.randn(shape, generator=g) * w.filler_std
        k = torch.randn(shape, generator=g) * w.filler_std
        v = torch.randn(shape, generator=g) * w.filler_std
        keys = torch.randn((w.B, w.H, n, w.d), generator=g)
        keys = keys / keys.norm(dim=-1, keepdim=True)
        vals = torch.randn((w.B, w.H, n, w.d), generator=g)
        k[:, :, :n] = keys
        v[:, :, :n] = vals
        # per-unit shuffled order of the queries
        perm = torch.stack([torch.randperm(n, generator=g) for _ in range(w.units)])
        perm = perm.view(w.B, w.H, n, 1).expand(-1, -1, -1, w.d)
        q[:, :, w.T - n:] = torch.gather(keys, 2, perm)
        return q.to(w.torch_dtype), k.to(w.torch_dtype), v.to(w.torch_dtype)
    raise ValueError(w.kind)


def make_u(w: Workload, scale: float = 1.0, rank: int = 0):
    """Random unit-norm penalty directions times `scale` (explicit-u tests)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed + 7919 + 1000003 * rank)
    u = torch.randn((w.B, w.H, w.T, w.d), generator=g)
    u = u / u.norm(dim=-1, keepdim=True) * scale
    return u.to(w.torch_dtype)
