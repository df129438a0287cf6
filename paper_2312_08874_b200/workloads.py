"""Workload shapes and seeded synthetic inputs for the Agent Attention forward pass.

This module holds shapes and random draws only: it contains none of the method's
arithmetic, so both the CUDA path's tests and the CPU oracle's tests can take their
inputs from it without sharing any computation.

Shapes follow the paper's architecture tables (App. G: the DeiT-T block with a 14x14
window, 3 heads and 49 agents; the PVT stage-1 geometry with a 56x56 grid and a
64-channel single head), the Stable Diffusion 512^2 setting of App. C.2 (64x64 latent
grid) and the high-resolution argument of Sec. 5.5.  The tensors themselves are i.i.d.
normal draws standing in for activations of trained networks.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    """One problem size.  N = grid_h * grid_w tokens, n = pool * pool agents."""

    name: str
    batch: int
    heads: int
    grid_h: int
    grid_w: int
    head_dim: int
    pool: int                 # agents form a pool x pool grid
    dtype: str                # "f32" | "bf16" | "f16"
    bias: bool                # dense agent biases B1, B2 present
    dwc: bool                 # 3x3 depthwise-conv term present
    qkv_scale: float = 1.0    # multiplier applied to the N(0,1) draws of Q, K, V
    seed: int = 0

    @property
    def tokens(self) -> int:
        return self.grid_h * self.grid_w

    @property
    def agents(self) -> int:
        return self.pool * self.pool

    @property
    def slabs(self) -> int:
        return self.batch * self.heads

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def algorithmic_bytes(self) -> int:
        """Q, K, V read once, O written once, each bias and the filter once per head."""
        s = self.elem_bytes
        b = 4 * self.slabs * self.tokens * self.head_dim * s
        if self.bias:
            b += 2 * self.heads * self.agents * self.tokens * s
        if self.dwc:
            b += 9 * self.heads * self.head_dim * s
        return b

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


WORKLOADS: Dict[str, Workload] = {
    w.name: w
    for w in [
        Workload("cfg1_deit_f32", 1, 3, 14, 14, 64, 7, "f32", False, True, 1.0, 0),
        Workload("cfg2_deit_bf16", 128, 3, 14, 14, 64, 7, "bf16", True, True, 1.0, 1),
        Workload("cfg3_pvt_bf16", 64, 1, 56, 56, 64, 7, "bf16", True, True, 1.0, 2),
        Workload("cfg4_sd_f16", 2, 8, 64, 64, 40, 16, "f16", False, False,
                 1.0 / math.sqrt(40.0), 3),
        Workload("cfg5a_hires_bf16", 2, 8, 128, 128, 64, 16, "bf16", True, True, 1.0, 4),
        Workload("cfg5b_hires_bf16", 2, 8, 256, 256, 64, 16, "bf16", True, True, 1.0, 5),
    ]
}

TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}


def make_inputs(w: Workload, seed: Optional[int] = None,
                bias_std: float = 0.02, dwc_std: float = 0.02) -> Dict[str, Optional[torch.Tensor]]:
    """Draw one input set on the CPU, already rounded to the storage dtype.

    Draw order is fixed: Q, K, V, B1, B2, Wd, each as fp32 standard normals from one
    `torch.Generator`, then scaled, then cast.  Layouts (all dense, last index fastest):
    Q, K, V [B, heads, N, d]; B1 [heads, n, N]; B2 [heads, N, n]; Wd [heads, d, 3, 3].
    Entries that the workload does not use are None.
    """
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed if seed is None else seed)
    dt = TORCH_DTYPE[w.dtype]
    B, h, N, d, n = w.batch, w.heads, w.tokens, w.head_dim, w.agents

    def draw(shape, mult):
        t = torch.randn(shape, generator=g, dtype=torch.float32)
        if mult != 1.0:
            t.mul_(mult)
        return t.to(dt).contiguous()

    out: Dict[str, Optional[torch.Tensor]] = {}
    out["q"] = draw((B, h, N, d), w.qkv_scale)
    out["k"] = draw((B, h, N, d), w.qkv_scale)
    out["v"] = draw((B, h, N, d), w.qkv_scale)
    out["b1"] = draw((h, n, N), bias_std) if w.bias else None
    out["b2"] = draw((h, N, n), bias_std) if w.bias else None
    out["dwc"] = draw((h, d, 3, 3), dwc_std) if w.dwc else None
    return out


def make_upstream_grad(w: Workload, seed: Optional[int] = None) -> torch.Tensor:
    """Upstream gradient dL/dO [B, heads, N, d] for the backward pass: fp32 standard normals from a
    generator of its own (seed + 1000003), cast to the storage dtype."""
    g = torch.Generator(device="cpu")
    g.manual_seed((w.seed if seed is None else seed) + 1000003)
    t = torch.randn((w.batch, w.heads, w.tokens, w.head_dim), generator=g, dtype=torch.float32)
    return t.to(TORCH_DTYPE[w.dtype]).contiguous()


def shard_slabs(total_batch: int, world_size: int, rank: int) -> range:
    """Batch entries owned by `rank` when a batch is split over `world_size` processes.

    Slabs (batch x head pairs) are independent, so a multi-GPU job only partitions the
    batch; earlier ranks take the remainder.  No data crosses ranks.
    """
    base, rem = divmod(total_batch, world_size)
    start = rank * base + min(rank, rem)
    return range(start, start + base + (1 if rank < rem else 0))
