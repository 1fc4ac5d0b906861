"""Seeded synthetic inputs with the shapes and norm structure of the five workloads.

This module holds no arithmetic of the method: it only draws tensors.  Both the
CUDA tests / benchmark and the CPU oracle tests take their inputs from here, so
that both sides see the same values (already rounded to the workload's dtype).

Recipe (per workload, seed = 20260218 + workload number):
  c1  fp32, B1 H4 Hkv4 d64 N512 C64 k16   Q,K,V iid N(0,1)
  c2  bf16, B4 H32 Hkv8 d64 N4096 C64 k64 Q,K,V iid N(0,1), then one scalar
      U(0.5,2) per (tensor, head) multiplies that head
  c3  bf16, B2 H32 Hkv8 d128 N32768 C64 k64  iid N(0,1); a Bernoulli(0.01) mask
      per (batch, position), shared by the KV heads, multiplies those K rows by 5
  c4  bf16, B1 H32 Hkv8 d128 N131072 C128 k128  K rows scaled by |t|, t ~
      Student-t(3) per row; Q,V iid N(0,1)
  c5  bf16, B64 H32 Hkv8 d128, prefix 32768, 256 decode steps, C64 k64, iid N(0,1)
NP-Map weights are N(0, 0.02^2), no bias; no gate; sm_scale = d^-1/2; eps = 1e-6.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    Hkv: int
    d: int
    N: int
    C: int
    k: int
    dtype: str  # "fp32" | "bf16"
    recipe: str  # "iid" | "head_scale" | "outlier_keys" | "student_t_keys"
    seed: int
    steps: int = 0  # decode steps (c5)

    @property
    def d_f(self) -> int:
        return self.d

    @property
    def sm_scale(self) -> float:
        return float(self.d) ** -0.5

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


_SEED0 = 20260218

WORKLOADS = {
    "c1": Workload("c1", 1, 4, 4, 64, 512, 64, 16, "fp32", "iid", _SEED0 + 1),
    "c2": Workload("c2", 4, 32, 8, 64, 4096, 64, 64, "bf16", "head_scale", _SEED0 + 2),
    "c3": Workload("c3", 2, 32, 8, 128, 32768, 64, 64, "bf16", "outlier_keys", _SEED0 + 3),
    "c4": Workload("c4", 1, 32, 8, 128, 131072, 128, 128, "bf16", "student_t_keys", _SEED0 + 4),
    "c5": Workload("c5", 64, 32, 8, 128, 32768, 64, 64, "bf16", "iid", _SEED0 + 5, steps=256),
}


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def make_qkv(w: Workload, device="cpu"):
    """Q [B,H,N,d], K,V [B,Hkv,N,d] drawn in fp32 and rounded once to the workload dtype."""
    g = _gen(device, w.seed)
    kw = dict(generator=g, device=device, dtype=torch.float32)
    Q = torch.randn(w.B, w.H, w.N, w.d, **kw)
    K = torch.randn(w.B, w.Hkv, w.N, w.d, **kw)
    V = torch.randn(w.B, w.Hkv, w.N, w.d, **kw)
    if w.recipe == "head_scale":
        Q *= torch.rand(1, w.H, 1, 1, **kw) * 1.5 + 0.5
        K *= torch.rand(1, w.Hkv, 1, 1, **kw) * 1.5 + 0.5
        V *= torch.rand(1, w.Hkv, 1, 1, **kw) * 1.5 + 0.5
    elif w.recipe == "outlier_keys":
        m = torch.rand(w.B, 1, w.N, 1, **kw) < 0.01
        K = torch.where(m, K * 5.0, K)
    elif w.recipe == "student_t_keys":
        z = torch.randn(w.B, w.Hkv, w.N, 1, **kw)
        c = torch.randn(w.B, w.Hkv, w.N, 3, **kw).square().sum(-1, keepdim=True) / 3.0
        K *= (z / c.sqrt()).abs()
    dt = w.torch_dtype
    return Q.to(dt), K.to(dt), V.to(dt)


def make_npmap_weights(w: Workload, device="cpu"):
    """Wq [H,d,d_f], Wk [Hkv,d,d_f] ~ N(0, 0.02^2), rounded to the workload dtype."""
    g = _gen(device, w.seed + 1000)
    kw = dict(generator=g, device=device, dtype=torch.float32)
    Wq = torch.randn(w.H, w.d, w.d_f, **kw) * 0.02
    Wk = torch.randn(w.Hkv, w.d, w.d_f, **kw) * 0.02
    return Wq.to(w.torch_dtype), Wk.to(w.torch_dtype)


def make_gate(w: Workload, device="cpu"):
    """Gate values in (0,1), [B,H,N,d] (used by the tests that exercise the gate)."""
    g = _gen(device, w.seed + 2000)
    return torch.rand(w.B, w.H, w.N, w.d, generator=g, device=device, dtype=torch.float32).to(w.torch_dtype)


def make_decode_inputs(w: Workload, step: int, device="cpu"):
    """One decode step's q [B,H,d], k,v [B,Hkv,d] ~ N(0,1)."""
    g = _gen(device, w.seed + 5000 + step)
    kw = dict(generator=g, device=device, dtype=torch.float32)
    q = torch.randn(w.B, w.H, w.d, **kw)
    k = torch.randn(w.B, w.Hkv, w.d, **kw)
    v = torch.randn(w.B, w.Hkv, w.d, **kw)
    dt = w.torch_dtype
    return q.to(dt), k.to(dt), v.to(dt)
