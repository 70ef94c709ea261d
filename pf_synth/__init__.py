"""Seeded synthetic inputs for the delta-rule forward pass.

This module holds NO arithmetic of the method: it only draws random tensors with the shapes and
value distributions of the benchmark workloads, so that the fp64 oracle and the CUDA path can be
fed bit-identical inputs.  Recipe (drawn on the host in fp32 from one ``torch.Generator`` seeded
with ``seed``, in the fixed order q, k, v, beta, S0):

    q, v  ~ N(0, 1/d)            (variance 1/d, i.e. std d**-0.5, d = d_k for q and d_v for v)
    k     ~ N(0, 1), then every key vector k[b,h,t,j,:] divided by its L2 norm (fp32)
    beta  = beta_scale * sigmoid(N(0, 1))        (beta_scale 1 -> (0,1); 2 -> (0,2))
    S0    = None, or N(0, s0_std**2) with shape [B,H,d_k,d_v]   (always kept fp32)

For the bf16 workloads q, k, v and beta are then rounded once to bf16 (round-to-nearest-even);
those rounded values are what both sides consume.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    L: int
    d_k: int
    d_v: int
    r: int
    chunk: int
    dtype: str = "bf16"          # "bf16" or "f32": dtype of q, k, v, beta as handed to the kernels
    beta_scale: float = 1.0
    s0_std: float = 0.0          # 0 -> S0 is None
    seed: int = 0

    @property
    def token_heads(self) -> int:
        return self.B * self.H * self.L

    @property
    def tokens(self) -> int:
        return self.B * self.L

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five benchmark configurations (index = seed).
CONFIGS = {
    "c0": Workload("c0", B=1, H=1, L=256, d_k=64, d_v=64, r=1, chunk=64, dtype="f32", seed=0),
    "c1": Workload("c1", B=4, H=8, L=2048, d_k=128, d_v=128, r=1, chunk=64, s0_std=0.1, seed=1),
    "c2": Workload("c2", B=2, H=16, L=8192, d_k=128, d_v=128, r=2, chunk=64, seed=2),
    "c3": Workload("c3", B=8, H=16, L=4096, d_k=64, d_v=64, r=4, chunk=64, beta_scale=2.0, seed=3),
    "c3_chunk32": Workload("c3_chunk32", B=8, H=16, L=4096, d_k=64, d_v=64, r=4, chunk=32,
                           beta_scale=2.0, seed=3),
    "c4": Workload("c4", B=1, H=32, L=65536, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=4),
}


@dataclass
class Inputs:
    q: torch.Tensor       # [B,H,L,d_k]
    k: torch.Tensor       # [B,H,L,r,d_k]
    v: torch.Tensor       # [B,H,L,r,d_v]
    beta: torch.Tensor    # [B,H,L,r]
    S0: Optional[torch.Tensor]   # [B,H,d_k,d_v] fp32 or None

    def to(self, device, non_blocking: bool = False) -> "Inputs":
        mv = lambda t: None if t is None else t.to(device, non_blocking=non_blocking)
        return Inputs(mv(self.q), mv(self.k), mv(self.v), mv(self.beta), mv(self.S0))

    def pin(self) -> "Inputs":
        pm = lambda t: None if t is None else t.pin_memory()
        return Inputs(pm(self.q), pm(self.k), pm(self.v), pm(self.beta), pm(self.S0))

    def nbytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in (self.q, self.k, self.v, self.beta, self.S0)
                   if t is not None)


def make_inputs(w: Workload, seed: Optional[int] = None) -> Inputs:
    """Host tensors for workload ``w`` (see the module docstring for the recipe)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed if seed is None else seed)
    B, H, L, r = w.B, w.H, w.L, w.r
    q = torch.randn(B, H, L, w.d_k, generator=g, dtype=torch.float32) * (w.d_k ** -0.5)
    k = torch.randn(B, H, L, r, w.d_k, generator=g, dtype=torch.float32)
    k = k / k.norm(dim=-1, keepdim=True)
    v = torch.randn(B, H, L, r, w.d_v, generator=g, dtype=torch.float32) * (w.d_v ** -0.5)
    beta = torch.sigmoid(torch.randn(B, H, L, r, generator=g, dtype=torch.float32)) * w.beta_scale
    S0 = None
    if w.s0_std > 0:
        S0 = torch.randn(B, H, w.d_k, w.d_v, generator=g, dtype=torch.float32) * w.s0_std
    if w.dtype == "bf16":
        q, k, v, beta = (t.to(torch.bfloat16) for t in (q, k, v, beta))
    elif w.dtype != "f32":
        raise ValueError(f"unknown dtype {w.dtype!r}")
    return Inputs(q.contiguous(), k.contiguous(), v.contiguous(), beta.contiguous(), S0)
