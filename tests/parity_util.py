"""Helpers shared by the GPU parity tests: run one workload through the C ABI (via the binding)
and through the fp64 oracle on the same seeded inputs, and measure the difference."""
from __future__ import annotations

import math
from typing import Dict, Optional

import numpy as np
import torch

from oracle import agent_attention_oracle as orc
from paper_2312_08874_b200 import AA_PATH_AUTO, AgentAttention, Workload, make_inputs

# Acceptance thresholds: fp32 path max-abs 1e-4; 16-bit paths max-abs 2e-2 and relative L2 5e-3,
# relative L2 = ||O_gpu - O_ref||_2 / ||O_ref||_2 over the compared tensor.
TOL = {"f32": dict(max_abs=1e-4, rel_l2=1e-5), "bf16": dict(max_abs=2e-2, rel_l2=5e-3),
       "f16": dict(max_abs=2e-2, rel_l2=5e-3)}


def errors(got: torch.Tensor, ref: np.ndarray) -> Dict[str, float]:
    g = got.detach().double().cpu().numpy()
    assert g.shape == ref.shape, (g.shape, ref.shape)
    assert np.all(np.isfinite(g)), "non-finite values in the GPU result"
    diff = g - ref
    den = float(np.linalg.norm(ref.ravel()))
    return {"max_abs": float(np.abs(diff).max()),
            "rel_l2": float(np.linalg.norm(diff.ravel()) / den) if den > 0 else float(np.abs(diff).max())}


def assert_close(got: torch.Tensor, ref: np.ndarray, dtype: str, what: str = "", scale: float = 1.0):
    e = errors(got, ref)
    tol = TOL[dtype]
    assert e["max_abs"] <= tol["max_abs"] * scale and e["rel_l2"] <= tol["rel_l2"] * scale, \
        f"{what}: {e} exceeds {tol} (x{scale})"
    return e


def to_np(t: Optional[torch.Tensor]) -> Optional[np.ndarray]:
    return None if t is None else t.double().numpy()


def to_dev(t: Optional[torch.Tensor]) -> Optional[torch.Tensor]:
    return None if t is None else t.cuda()


def make_module(w: Workload, path: int = AA_PATH_AUTO, scale1: float = 0.0, scale2: float = 0.0,
                max_agents: Optional[int] = None) -> AgentAttention:
    from paper_2312_08874_b200.workloads import TORCH_DTYPE
    return AgentAttention(w.batch, w.heads, w.head_dim, w.tokens, max_agents or w.agents,
                          TORCH_DTYPE[w.dtype], scale1=scale1, scale2=scale2, device=0, path=path)


def oracle_forward(w: Workload, inp, threads: int = 0, slabs=None, **kw):
    """Oracle on the storage-rounded inputs.  `slabs` = list of (b, head) to evaluate, else all."""
    threads = threads or orc.max_threads()
    if slabs is None:
        return orc.forward(to_np(inp["q"]), to_np(inp["k"]), to_np(inp["v"]), w.grid_h, w.grid_w,
                           pool_hw=(w.pool, w.pool), b1=to_np(inp["b1"]), b2=to_np(inp["b2"]),
                           dwc_weight=to_np(inp["dwc"]), threads=threads, **kw)
    outs = []
    for (b, h) in slabs:
        sl = lambda t: None if t is None else to_np(t[b:b + 1, h:h + 1])
        hd = lambda t: None if t is None else to_np(t[h:h + 1])
        outs.append(orc.forward(sl(inp["q"]), sl(inp["k"]), sl(inp["v"]), w.grid_h, w.grid_w,
                                pool_hw=(w.pool, w.pool), b1=hd(inp["b1"]), b2=hd(inp["b2"]),
                                dwc_weight=hd(inp["dwc"]), threads=1, **kw))
    return outs


def gpu_forward(mod: AgentAttention, w: Workload, inp, agents=None, return_workspace: bool = False):
    """One forward call through the C ABI on poisoned buffers: `out` starts as NaN and the workspace as 0xFF bytes
    (NaN in every element type), so an element the kernels do not write, or read before writing, shows."""
    dev = {k: to_dev(v) for k, v in inp.items()}
    out = torch.full_like(dev["q"], float("nan"))
    ws = torch.full((mod.workspace_bytes(w.grid_h, w.grid_w, w.agents),), 0xFF, dtype=torch.uint8, device="cuda")
    mod.forward(dev["q"], dev["k"], dev["v"], w.grid_h, w.grid_w, w.agents, agents=agents,
                b1=dev["b1"], b2=dev["b2"], dwc_weight=dev["dwc"], out=out, workspace=ws)
    torch.cuda.synchronize()
    assert mod.query_status() == 0, "a device-side bounded wait expired"
    return (out, ws) if return_workspace else out
