"""The allocation-free aggregation entry point (collected last on purpose).

`agent_attn_aggregate_static` serves callers that cannot call cudaMalloc where they need the
aggregation (a plugin inside an application that owns the device memory pool, a loop with a
fixed memory budget, a caller holding only its inputs and outputs): its split partials live in
a fixed array inside the library instead of a caller-provided workspace.  It must return what
`agent_attn_aggregate` returns, on consecutive calls that reuse the array, and must refuse
shapes that do not fit the array.
"""
import numpy as np
import pytest
import torch

from paper_2312_08874_b200 import WORKLOADS, AgentAttnError, make_inputs
from oracle import agent_attention_oracle as orc
from tests.parity_util import TOL, assert_close, make_module, to_dev, to_np

pytestmark = pytest.mark.gpu


def _close(a: torch.Tensor, b: torch.Tensor, dtype: str):
    diff = (a.double() - b.double())
    max_abs = float(diff.abs().max())
    rel = float(diff.norm() / b.double().norm())
    assert max_abs <= TOL[dtype]["max_abs"] and rel <= TOL[dtype]["rel_l2"], (max_abs, rel)


def test_static_scratch_aggregation_matches_workspace_aggregation_twice_in_a_row():
    w = WORKLOADS["cfg3_pvt_bf16"].scaled(batch=8)
    mod = make_module(w)
    for call, seed in enumerate((31, 32)):               # two different inputs, back to back
        inp = make_inputs(w, seed=seed)
        q, k, v, b1 = (to_dev(inp[x]) for x in ("q", "k", "v", "b1"))
        agents = mod.pool(q, w.grid_h, w.grid_w, w.pool, w.pool)
        expect = mod.aggregate(agents, k, v, b1=b1)
        out = torch.full_like(agents, float("nan"))      # stale or unwritten elements would show
        got = mod.aggregate_static(agents, k, v, b1=b1, out=out)
        torch.cuda.synchronize()
        assert torch.isfinite(got.float()).all(), f"call {call}"
        _close(got, expect, w.dtype)
        # and against the oracle's aggregation (Eq. 3 with the bias of Eq. 5) on the same agents
        a_np, k_np, v_np, b_np = to_np(agents.cpu()), to_np(inp["k"]), to_np(inp["v"]), to_np(inp["b1"])
        ref = np.stack([np.stack([orc.softmax_attention(a_np[b, h], k_np[b, h], v_np[b, h], bias=b_np[h],
                                                        scale=w.head_dim ** -0.5)
                                  for h in range(w.heads)]) for b in range(w.batch)])
        assert_close(got, ref, w.dtype, f"static-scratch aggregation, call {call}")
    # same inputs again: the array keeps the previous call's contents and that must not matter
    again = mod.aggregate_static(agents, k, v, b1=b1)
    torch.cuda.synchronize()
    assert torch.equal(again, got)


def test_static_scratch_rejects_shapes_beyond_its_size():
    lib_bytes = int(make_module(WORKLOADS["cfg1_deit_f32"]).lib.agent_attn_static_scratch_bytes())
    assert lib_bytes == 32 * 1024 * 1024
    w = WORKLOADS["cfg2_deit_bf16"].scaled(batch=2048)   # partial states far beyond 32 MiB
    mod = make_module(w)
    agents = torch.zeros((w.batch, w.heads, w.agents, w.head_dim), dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros((w.batch, w.heads, w.tokens, w.head_dim), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(AgentAttnError) as e:
        mod.aggregate_static(agents, kv, kv)
    assert e.value.status == 3 and "built-in scratch" in str(e.value)
