"""Backward pass through the C ABI against the fp64 oracle's chain rule, element by element."""
import numpy as np
import pytest
import torch

from oracle import agent_attention_oracle as orc
from paper_2312_08874_b200 import (AA_PATH_AUTO, AA_PATH_SIMT, WORKLOADS, AgentAttnError, Workload, make_inputs,
                                   make_upstream_grad)
from tests.parity_util import make_module, to_dev, to_np

pytestmark = pytest.mark.gpu

# The kernels compute in fp32 from the same storage-rounded inputs the oracle reads, for every element
# type: relative L2 error 5e-5 and max-abs error 1e-4 of the largest reference magnitude (sums of up to
# N = 65536 fp32 terms in an order that is not fixed, exponentials of fp32 logits).
REL_L2 = 5e-5
MAX_REL = 1e-4
# Handles created with AA_PATH_AUTO run the two gradient stages on the tensor cores for 16-bit inputs with
# n <= 64 and d = 64: A, V_A, dV_A, P and dS are then rounded to the storage type (2^-9 relative for bf16)
# before they enter a product, as in the forward pass, whose tolerance (relative L2 5e-3 per rounding stage)
# is doubled here for the two chained stages; max-abs 5e-2 of the largest reference magnitude.
TC_REL_L2 = 1e-2
TC_MAX_REL = 5e-2


def tensor_core_path(w: Workload, path: int) -> bool:
    return path == AA_PATH_AUTO and w.dtype in ("bf16", "f16") and w.agents <= 64 and w.head_dim == 64


def check(got: dict, ref: dict, what: str, tc: bool = False):
    rel_tol, max_tol = (TC_REL_L2, TC_MAX_REL) if tc else (REL_L2, MAX_REL)
    assert set(got) == set(ref), (sorted(got), sorted(ref))
    for key in sorted(ref):
        g = got[key].double().cpu().numpy()
        r = ref[key]
        assert g.shape == r.shape, (key, g.shape, r.shape)
        assert np.all(np.isfinite(g)), f"{what} {key}: non-finite"
        diff = g - r
        den = float(np.linalg.norm(r.ravel()))
        rel = float(np.linalg.norm(diff.ravel())) / den if den > 0 else float(np.abs(diff).max())
        mx = float(np.abs(diff).max()) / max(float(np.abs(r).max()), 1e-30)
        print(f"{what} {key}: rel_l2={rel:.3e} max_rel={mx:.3e}")
        assert rel <= rel_tol and mx <= max_tol, f"{what} {key}: rel_l2={rel:.3e} max_rel={mx:.3e}"


def run_both(w: Workload, inp, scale1=0.0, scale2=0.0, path=AA_PATH_AUTO):
    go = make_upstream_grad(w)
    mod = make_module(w, scale1=scale1, scale2=scale2, path=path)
    got = mod.backward(to_dev(inp["q"]), to_dev(inp["k"]), to_dev(inp["v"]), to_dev(go), w.grid_h, w.grid_w,
                       w.agents, b1=to_dev(inp["b1"]), b2=to_dev(inp["b2"]), dwc_weight=to_dev(inp["dwc"]))
    torch.cuda.synchronize()
    assert mod.query_status() == 0
    ref = orc.backward(to_np(inp["q"]), to_np(inp["k"]), to_np(inp["v"]), to_np(go), w.grid_h, w.grid_w,
                       (w.pool, w.pool), b1=to_np(inp["b1"]), b2=to_np(inp["b2"]), dwc_weight=to_np(inp["dwc"]),
                       scale1=scale1 or None, scale2=scale2 or None)
    return mod, got, ref


CASES = [
    # batch heads H  W   d   pool dtype  bias  dwc
    (2, 2, 7, 9, 8, 2, "f32", True, True),          # pooling windows overlap (7 and 9 rows / columns over 2 cells)
    (1, 3, 10, 10, 40, 4, "f32", True, True),
    (2, 1, 5, 5, 128, 5, "f32", False, True),       # every token its own agent, d = 128
    (3, 2, 14, 14, 64, 7, "bf16", True, True),
    (2, 2, 9, 11, 40, 3, "f16", True, True),
    (2, 1, 31, 29, 64, 6, "bf16", True, True),      # ragged last tile, odd N
    (1, 2, 36, 36, 64, 12, "bf16", True, True),     # n = 144: five agents per lane, the last lanes idle
    (1, 1, 32, 32, 64, 16, "f16", True, True),      # n = 256, d = 64: the largest n * d
    (2, 1, 3, 3, 16, 1, "bf16", True, True),        # one agent: P2 = 1, dS2 = 0
    (1, 1, 1, 1, 64, 1, "bf16", True, True),        # a single token
    (2, 2, 20, 20, 32, 5, "bf16", False, False),    # no bias, no depthwise term
    (6, 1, 56, 56, 64, 7, "bf16", True, True),      # the headline grid, several blocks per slab
    (2, 2, 16, 12, 64, 8, "f16", True, True),       # n = 64: every agent column of the tensor-core tiles in use
    (2, 1, 20, 20, 64, 5, "bf16", False, False),    # tensor-core kernels without bias and depthwise term
]


@pytest.mark.parametrize("path", [AA_PATH_AUTO, AA_PATH_SIMT], ids=["auto", "simt"])
@pytest.mark.parametrize("case", CASES, ids=[f"B{c[0]}h{c[1]}_{c[2]}x{c[3]}_d{c[4]}_p{c[5]}_{c[6]}" for c in CASES])
def test_backward_matches_oracle(case, path):
    B, heads, H, W, d, pool, dtype, bias, dwc = case
    w = Workload("bwd", B, heads, H, W, d, pool, dtype, bias, dwc, 1.0, seed=300 + H * W + d)
    if path == AA_PATH_SIMT and not tensor_core_path(w, AA_PATH_AUTO):
        pytest.skip("this shape runs the fp32 kernels on either path")
    inp = make_inputs(w, bias_std=0.5, dwc_std=0.2)
    _, got, ref = run_both(w, inp, path=path)
    check(got, ref, str(case), tc=tensor_core_path(w, path))


def test_backward_with_distinct_scales_and_optional_outputs():
    w = Workload("bwd", 2, 2, 12, 10, 32, 3, "bf16", True, True, 1.0, seed=11)
    inp = make_inputs(w, bias_std=0.5, dwc_std=0.2)
    mod, got, ref = run_both(w, inp, scale1=0.7, scale2=0.4)
    check(got, ref, "distinct scales")
    go = to_dev(make_upstream_grad(w))
    part = mod.backward(to_dev(inp["q"]), to_dev(inp["k"]), to_dev(inp["v"]), go, w.grid_h, w.grid_w, w.agents,
                        b1=to_dev(inp["b1"]), b2=to_dev(inp["b2"]), dwc_weight=to_dev(inp["dwc"]),
                        need_bias_grads=False, need_filter_grad=False)
    torch.cuda.synchronize()
    assert set(part) == {"dq", "dk", "dv"}
    check(part, {k: ref[k] for k in part}, "without optional gradients")


def test_backward_headline_configuration_full_size():
    w = WORKLOADS["cfg3_pvt_bf16"]
    inp = make_inputs(w)
    go = make_upstream_grad(w)
    ref = orc.backward(to_np(inp["q"]), to_np(inp["k"]), to_np(inp["v"]), to_np(go), w.grid_h, w.grid_w,
                       (w.pool, w.pool), b1=to_np(inp["b1"]), b2=to_np(inp["b2"]), dwc_weight=to_np(inp["dwc"]))
    for path in (AA_PATH_AUTO, AA_PATH_SIMT):
        mod = make_module(w, path=path)
        got = mod.backward(to_dev(inp["q"]), to_dev(inp["k"]), to_dev(inp["v"]), to_dev(go), w.grid_h, w.grid_w,
                           w.agents, b1=to_dev(inp["b1"]), b2=to_dev(inp["b2"]), dwc_weight=to_dev(inp["dwc"]))
        torch.cuda.synchronize()
        check(got, ref, f"cfg3 path {path}", tc=tensor_core_path(w, path))


def test_backward_large_grid_sampled_batch_entry():
    w = WORKLOADS["cfg5a_hires_bf16"].scaled(batch=1, heads=1)
    inp = make_inputs(w)
    _, got, ref = run_both(w, inp)
    check(got, ref, "cfg5a, one slab")


def test_backward_rejects_what_it_cannot_do():
    w = Workload("bwd", 1, 1, 32, 32, 128, 16, "bf16", False, True, 1.0, seed=5)     # n * d = 32768
    mod = make_module(w)
    assert mod.lib.agent_attn_backward_workspace_bytes(mod._h, 32, 32, 256) == 0
    inp = make_inputs(w)
    go = to_dev(make_upstream_grad(w))
    with pytest.raises(AgentAttnError) as e:
        mod.backward(to_dev(inp["q"]), to_dev(inp["k"]), to_dev(inp["v"]), go, 32, 32, 256,
                     dwc_weight=to_dev(inp["dwc"]), workspace=torch.empty(1 << 20, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 2
    w2 = Workload("bwd", 1, 1, 8, 8, 64, 2, "bf16", False, False, 1.0, seed=5)
    mod2 = make_module(w2, max_agents=8)
    inp2 = make_inputs(w2)
    go2 = to_dev(make_upstream_grad(w2))
    with pytest.raises(AgentAttnError) as e:          # 5 agents cannot come from pooling
        mod2.backward(to_dev(inp2["q"]), to_dev(inp2["k"]), to_dev(inp2["v"]), go2, 8, 8, 5,
                      workspace=torch.empty(1 << 20, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 1
