"""GPU-vs-oracle parity through the C ABI, element by element on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import agent_attention_oracle as orc
from paper_2312_08874_b200 import AA_PATH_AUTO, AA_PATH_SIMT, AA_PATH_UNFUSED, WORKLOADS, AgentAttention, Workload, make_inputs
from tests.parity_util import (assert_close, errors, gpu_forward, make_module, oracle_forward, to_dev, to_np)

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------ the five configurations
@pytest.mark.parametrize("path", [AA_PATH_AUTO, AA_PATH_UNFUSED], ids=["auto", "unfused"])
@pytest.mark.parametrize("name", ["cfg1_deit_f32", "cfg2_deit_bf16", "cfg3_pvt_bf16", "cfg4_sd_f16",
                                  "cfg5a_hires_bf16"])
def test_full_size_configs_match_oracle(name, path):
    w = WORKLOADS[name]
    if path == AA_PATH_UNFUSED and name not in ("cfg2_deit_bf16", "cfg3_pvt_bf16"):
        pytest.skip("only the small-agent-count configurations have two launch plans")
    inp = make_inputs(w)
    mod = make_module(w, path=path)
    out = gpu_forward(mod, w, inp)
    ref, a_ref, va_ref = oracle_forward(w, inp, return_intermediates=True)
    assert_close(out, ref, w.dtype, name)
    # intermediates through the step entry points
    a = mod.pool(to_dev(inp["q"]), w.grid_h, w.grid_w, w.pool, w.pool)
    assert_close(a, a_ref, w.dtype, name + " agents")
    va = mod.aggregate(a, to_dev(inp["k"]), to_dev(inp["v"]), b1=to_dev(inp["b1"]))
    torch.cuda.synchronize()
    assert_close(va, va_ref, w.dtype, name + " agent features")


def test_largest_config_matches_oracle_on_sampled_slabs():
    w = WORKLOADS["cfg5b_hires_bf16"]
    inp = make_inputs(w)
    mod = make_module(w)
    out = gpu_forward(mod, w, inp)
    assert torch.isfinite(out.float()).all()
    slabs = [(0, 0), (1, 5)]
    for (b, h), ref in zip(slabs, oracle_forward(w, inp, slabs=slabs)):
        assert_close(out[b:b + 1, h:h + 1], ref, w.dtype, f"cfg5b slab {(b, h)}")


def test_more_slabs_than_the_queue_lag_interleaves_task_kinds():
    """With more slabs than the queue's lag (the L2 budget: 83 slabs of this shape) aggregation and broadcast tasks
    alternate in the queue, so blocks take tickets of one kind while finishing a task of the other and broadcast
    tasks may find their slab's flag not yet set: sampled slabs against the oracle, repeatable bit for bit, and no
    bounded wait expired."""
    w = WORKLOADS["cfg3_pvt_bf16"].scaled(batch=160, seed=77)
    inp = make_inputs(w)
    mod = make_module(w)
    out = gpu_forward(mod, w, inp).clone()
    again = gpu_forward(mod, w, inp)
    assert torch.equal(out, again)
    assert torch.isfinite(out.float()).all()
    slabs = [(0, 0), (82, 0), (83, 0), (121, 0), (159, 0)]
    for (b, h), ref in zip(slabs, oracle_forward(w, inp, slabs=slabs)):
        assert_close(out[b:b + 1, h:h + 1], ref, w.dtype, f"slab {(b, h)} of 160")


# ------------------------------------------------------- attention term must not hide under DWC
@pytest.mark.parametrize("name", ["cfg3_pvt_bf16", "cfg5a_hires_bf16"])
@pytest.mark.parametrize("variant", ["no_dwc", "shifted_v"])
def test_attention_term_alone_and_with_nonzero_mean_values(name, variant):
    w = WORKLOADS[name].scaled(batch=2)
    inp = make_inputs(w)
    if variant == "no_dwc":
        inp["dwc"] = None
    else:
        inp["v"] = (inp["v"].float() + 1.0).to(inp["v"].dtype)
    mod = make_module(w)
    out = gpu_forward(mod, w, inp)
    assert_close(out, oracle_forward(w, inp), w.dtype, f"{name} {variant}")


# ------------------------------------------------------------------------------ shape sweep
SWEEP = [
    # batch heads H  W   d   pool dtype  bias  dwc
    (2, 2, 7, 9, 8, 2, "f32", True, True),
    (1, 3, 10, 10, 40, 4, "f32", True, True),
    (2, 1, 5, 5, 128, 5, "f32", False, True),
    (1, 2, 33, 17, 16, 3, "f32", True, False),
    (3, 2, 14, 14, 64, 7, "bf16", True, True),
    (2, 2, 9, 11, 40, 3, "f16", True, True),
    (1, 2, 20, 20, 32, 5, "bf16", True, True),
    (2, 1, 31, 29, 64, 6, "bf16", True, True),      # odd N: bias rows unaligned
    (1, 1, 40, 40, 128, 9, "f16", True, True),
    (1, 2, 36, 36, 96, 10, "bf16", False, True),
    (1, 2, 48, 48, 8, 12, "bf16", True, True),
    (1, 1, 64, 64, 24, 16, "f16", True, False),
    (5, 2, 28, 56, 64, 7, "bf16", True, True),      # fused path: H != W, ragged last 128-token tile
    (40, 2, 64, 64, 32, 8, "f16", True, True),      # fused path: widest grid, n = 64, more slabs than lag
    (3, 1, 56, 56, 64, 7, "bf16", False, False),    # fused path: no bias, no DWC
    (7, 3, 14, 14, 64, 7, "f16", True, True),       # fused path: one G task per slab, odd-head bias misaligned
    (2, 1, 3, 3, 16, 1, "bf16", True, True),        # one agent, nine tokens
    (1, 1, 1, 1, 64, 1, "bf16", True, True),        # a single token
    (2, 2, 36, 36, 64, 12, "bf16", True, True),     # tensor-memory kernels: n = 144 (two agent blocks, second ragged), ragged last tiles
    (1, 2, 48, 32, 40, 16, "f16", True, True),      # tensor-memory kernels: n = 256, d = 40 zero-filled to 64, bias and DWC
    (1, 3, 40, 40, 64, 10, "bf16", True, False),    # n = 100: one agent block on tcgen05 for the aggregation, n % 8 != 0 for the broadcast
    (2, 1, 27, 27, 64, 9, "bf16", True, True),      # n = 81 with odd N: stays on the mma.sync kernels
    (1, 1, 32, 32, 64, 16, "bf16", False, False),   # tensor-memory kernels without bias and DWC
]


@pytest.mark.parametrize("path", [AA_PATH_AUTO, AA_PATH_UNFUSED, AA_PATH_SIMT], ids=["auto", "unfused", "simt"])
@pytest.mark.parametrize("case", SWEEP, ids=[f"B{c[0]}h{c[1]}_{c[2]}x{c[3]}_d{c[4]}_p{c[5]}_{c[6]}" for c in SWEEP])
def test_shape_sweep(case, path):
    B, heads, H, W, d, pool, dtype, bias, dwc = case
    w = Workload("sweep", B, heads, H, W, d, pool, dtype, bias, dwc, 1.0, seed=100 + H * W + d)
    inp = make_inputs(w, bias_std=0.5, dwc_std=0.2)
    mod = make_module(w, path=path)
    out = gpu_forward(mod, w, inp)
    ref, a_ref, va_ref = oracle_forward(w, inp, return_intermediates=True)
    assert_close(out, ref, dtype, f"{case}")
    a = mod.pool(to_dev(inp["q"]), H, W, pool, pool)
    assert_close(a, a_ref, dtype, "agents")
    va = mod.aggregate(a, to_dev(inp["k"]), to_dev(inp["v"]), b1=to_dev(inp["b1"]))
    torch.cuda.synchronize()
    assert_close(va, va_ref, dtype, "agent features")


# ------------------------------------------------------------------- method-level properties
def test_user_supplied_agents_non_square_count():
    w = Workload("user_a", 2, 2, 12, 10, 64, 1, "bf16", True, True, 1.0, seed=7)
    n = 23
    inp = make_inputs(w)
    g = torch.Generator().manual_seed(8)
    agents = torch.randn((2, 2, n, 64), generator=g).to(torch.bfloat16)
    b1 = (torch.randn((2, n, w.tokens), generator=g) * 0.3).to(torch.bfloat16)
    b2 = (torch.randn((2, w.tokens, n), generator=g) * 0.3).to(torch.bfloat16)
    mod = make_module(w, max_agents=n)
    out = mod.forward(to_dev(inp["q"]), to_dev(inp["k"]), to_dev(inp["v"]), 12, 10, n, agents=agents.cuda(),
                      b1=b1.cuda(), b2=b2.cuda(), dwc_weight=to_dev(inp["dwc"]))
    torch.cuda.synchronize()
    ref = orc.forward(to_np(inp["q"]), to_np(inp["k"]), to_np(inp["v"]), 12, 10, agents=to_np(agents),
                      b1=to_np(b1), b2=to_np(b2), dwc_weight=to_np(inp["dwc"]), threads=4)
    assert_close(out, ref, "bf16", "user agents")


def test_separate_scales_follow_the_stable_diffusion_variant():
    # App. C.1: larger scale in the broadcast only, shortcut k*V = centre-tap filter.
    w = Workload("sd", 1, 2, 16, 16, 40, 4, "f16", False, True, 1.0, seed=9)
    inp = make_inputs(w)
    wd = torch.zeros((2, 40, 3, 3), dtype=torch.float16)
    wd[:, :, 1, 1] = 0.075
    inp["dwc"] = wd
    s2 = 40.0 ** -0.15
    mod = make_module(w, scale2=s2)
    out = gpu_forward(mod, w, inp)
    ref = oracle_forward(w, inp, scale2=s2)
    assert_close(out, ref, "f16", "sd variant")
    ref_default = oracle_forward(w, inp)
    assert errors(out, ref_default)["rel_l2"] > 2e-2      # the larger broadcast scale really is used


def test_constant_values_are_reproduced_and_single_agent_rows_are_identical():
    w = Workload("const_v", 1, 1, 16, 16, 64, 4, "bf16", True, False, 1.0, seed=10)
    inp = make_inputs(w)
    const = (torch.arange(64, dtype=torch.float32) / 16.0 - 2.0).to(torch.bfloat16)
    inp["v"] = const.expand(1, 1, 256, 64).contiguous()
    out = gpu_forward(make_module(w), w, inp)
    assert_close(out, to_np(inp["v"]), "bf16", "constant V", scale=0.5)
    w1 = Workload("one_agent", 1, 2, 8, 8, 32, 1, "f16", False, False, 1.0, seed=11)
    inp1 = make_inputs(w1)
    out1 = gpu_forward(make_module(w1), w1, inp1)
    assert torch.equal(out1, out1[:, :, :1].expand_as(out1))


def test_key_value_permutation_changes_split_boundaries_not_the_result():
    w = WORKLOADS["cfg3_pvt_bf16"].scaled(batch=1, bias=False, dwc=False)
    inp = make_inputs(w)
    mod = make_module(w)
    out1 = gpu_forward(mod, w, inp).float()
    perm = torch.randperm(w.tokens, generator=torch.Generator().manual_seed(3))
    inp2 = dict(inp, k=inp["k"][:, :, perm].contiguous(), v=inp["v"][:, :, perm].contiguous())
    out2 = gpu_forward(mod, w, inp2).float()
    ref = oracle_forward(w, inp)
    assert_close(out1, ref, "bf16", "original order")
    assert_close(out2, ref, "bf16", "permuted keys")


def test_zero_bias_tensors_equal_null_bias_and_runs_are_bitwise_repeatable():
    w = WORKLOADS["cfg2_deit_bf16"].scaled(batch=4, bias=False)
    inp = make_inputs(w)
    mod = make_module(w)
    out_null = gpu_forward(mod, w, inp).clone()
    again = gpu_forward(mod, w, inp).clone()
    assert torch.equal(out_null, again)
    inp0 = dict(inp, b1=torch.zeros((w.heads, w.agents, w.tokens), dtype=torch.bfloat16),
                b2=torch.zeros((w.heads, w.tokens, w.agents), dtype=torch.bfloat16))
    out_zero = gpu_forward(mod, w, inp0)
    assert torch.equal(out_null, out_zero)


def test_large_logits_stay_finite():
    w = Workload("hot", 1, 1, 16, 16, 64, 4, "bf16", False, False, 6.0, seed=12)
    inp = make_inputs(w)
    out = gpu_forward(make_module(w), w, inp)
    ref = oracle_forward(w, inp)
    assert torch.isfinite(out.float()).all()
    # peaked softmaxes amplify the rounding of A and V_A to bf16: only a loose bound is claimed
    assert errors(out, ref)["rel_l2"] < 5e-2


def test_forward_host_matches_forward():
    w = WORKLOADS["cfg2_deit_bf16"].scaled(batch=3)
    inp = make_inputs(w)
    mod = make_module(w)
    out_dev = gpu_forward(mod, w, inp).cpu()
    pin = {k: (None if v is None else v.pin_memory()) for k, v in inp.items()}
    out_host = mod.forward_host(pin["q"], pin["k"], pin["v"], w.grid_h, w.grid_w, w.agents, b1=pin["b1"],
                                b2=pin["b2"], dwc_weight=pin["dwc"])
    assert torch.equal(out_dev, out_host)
    assert mod.last_launch_count() == 1            # the fused persistent kernel
    assert mod.query_status() == 0


# ------------------------------------------------------------------ App. B: bias composition
@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("transpose", [False, True])
def test_bias_composition_matches_oracle(dtype, transpose):
    from paper_2312_08874_b200.workloads import TORCH_DTYPE
    heads, n, H, W, h0, w0 = 3, 49, 14, 20, 5, 7
    g = torch.Generator().manual_seed(40)
    dt = TORCH_DTYPE[dtype]
    col = torch.randn((heads, n, W), generator=g).to(dt)
    row = torch.randn((heads, n, H), generator=g).to(dt)
    blk = torch.randn((heads, n, h0, w0), generator=g).to(dt)
    mod = AgentAttention(1, heads, 64, H * W, n, dt)
    got = mod.compose_bias(col.cuda(), row.cuda(), blk.cuda(), H, W, n, transpose=transpose)
    torch.cuda.synchronize()
    ref = np.stack([orc.compose_bias(to_np(col[h]), to_np(row[h]), to_np(blk[h]), H, W, transpose=transpose)
                    for h in range(heads)])
    assert_close(got, ref, dtype, "composed bias", scale=1.0 if dtype != "f32" else 1.0)
    only_blk = mod.compose_bias(None, None, blk.cuda(), H, W, n, transpose=transpose)
    ref_blk = np.stack([orc.compose_bias(None, None, to_np(blk[h]), H, W, transpose=transpose) for h in range(heads)])
    assert_close(only_blk, ref_blk, dtype, "block bias alone")


# --------------------------------------------------------------------------------- error paths
def test_invalid_arguments_are_rejected_without_launching():
    from paper_2312_08874_b200 import AgentAttnError
    w = WORKLOADS["cfg1_deit_f32"]
    inp = make_inputs(w)
    mod = make_module(w)
    q, k, v = to_dev(inp["q"]), to_dev(inp["k"]), to_dev(inp["v"])
    big = torch.empty(1 << 22, dtype=torch.uint8, device="cuda")
    with pytest.raises(AgentAttnError) as e:                # n not a square when pooling
        mod.forward(q, k, v, 14, 14, 48, workspace=big)
    assert e.value.status == 1
    with pytest.raises(AgentAttnError) as e:                # more agents than the handle allows
        mod.forward(q, k, v, 14, 14, 64, workspace=big)
    assert e.value.status == 2
    with pytest.raises(AgentAttnError) as e:                # workspace too small
        mod.forward(q, k, v, 14, 14, 49, workspace=torch.empty(64, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 3
    with pytest.raises(AgentAttnError) as e:                # out aliases an input
        mod.forward(q, k, v, 14, 14, 49, out=q)
    assert e.value.status == 1
    with pytest.raises(AgentAttnError):                     # unsupported head dim
        AgentAttention(1, 1, 136, 64, 16, torch.bfloat16)
    with pytest.raises(AgentAttnError):
        AgentAttention(1, 1, 64, 64, 257, torch.bfloat16)
    torch.cuda.synchronize()


# ------------------------------------------------------------- token-major layouts with strides
STRIDED = [
    # batch heads H  W   d   pool dtype   bias  dwc     kernel that takes it
    (2, 3, 28, 28, 64, 7, "bf16", True, True),       # fused persistent kernel
    (3, 2, 14, 14, 64, 7, "f16", True, True),        # fused, one G task per slab, unaligned bias rows
    (2, 2, 32, 32, 64, 16, "bf16", True, True),      # tensor-memory kernels, n = 256
    (1, 4, 36, 36, 40, 12, "f16", True, True),       # tensor-memory kernels, n = 144, d = 40
    (2, 1, 24, 24, 64, 12, "bf16", False, False),    # one head, no bias, no DWC
    (1, 2, 56, 56, 64, 7, "bf16", True, True),       # fused, the 56x56 shape-specialised instantiation for strides
]


@pytest.mark.parametrize("packed", [False, True], ids=["bnhd", "qkv_interleaved"])
@pytest.mark.parametrize("case", STRIDED, ids=[f"B{c[0]}h{c[1]}_{c[2]}x{c[3]}_d{c[4]}_p{c[5]}_{c[6]}" for c in STRIDED])
def test_strided_token_major_layouts(case, packed):
    """Q, K, V read in place from [B, N, heads, d] (or interleaved [B, N, 3, heads, d]) and O written as
    [B, N, heads, d]: same result as the dense call on transposed copies, and within tolerance of the oracle."""
    B, heads, H, W, d, pool, dtype, bias, dwc = case
    w = Workload("strided", B, heads, H, W, d, pool, dtype, bias, dwc, 1.0, seed=300 + H * W + d)
    inp = make_inputs(w, bias_std=0.5, dwc_std=0.2)
    mod = make_module(w)
    dense = gpu_forward(mod, w, inp)
    q, k, v = (to_dev(inp[x]) for x in ("q", "k", "v"))                 # [B, heads, N, d]
    if packed:
        qkv = torch.stack([t.permute(0, 2, 1, 3) for t in (q, k, v)], dim=2).contiguous()    # [B, N, 3, heads, d]
        views = [qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3)]
    else:
        views = [t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) for t in (q, k, v)]  # [B, N, heads, d] storage
    assert not views[0].is_contiguous() or heads == 1
    out = mod.forward_strided(views[0], views[1], views[2], H, W, w.agents, b1=to_dev(inp["b1"]), b2=to_dev(inp["b2"]),
                              dwc_weight=to_dev(inp["dwc"]))
    torch.cuda.synchronize()
    assert mod.query_status() == 0
    assert out.permute(0, 2, 1, 3).is_contiguous()                       # stored as [B, N, heads, d]
    assert torch.equal(out, dense), "the strided call must match the dense call bit for bit"
    assert_close(out.contiguous(), oracle_forward(w, inp), dtype, f"strided {case}")


def test_strided_call_with_dense_strides_is_the_dense_call_and_fp32_is_refused():
    w = WORKLOADS["cfg3_pvt_bf16"].scaled(batch=2)
    inp = make_inputs(w)
    mod = make_module(w)
    dense = gpu_forward(mod, w, inp)
    out = torch.empty_like(dense)
    mod.forward_strided(to_dev(inp["q"]), to_dev(inp["k"]), to_dev(inp["v"]), w.grid_h, w.grid_w, w.agents,
                        b1=to_dev(inp["b1"]), b2=to_dev(inp["b2"]), dwc_weight=to_dev(inp["dwc"]), out=out)
    torch.cuda.synchronize()
    assert torch.equal(out, dense)
    w32 = Workload("strided32", 1, 2, 8, 8, 32, 2, "f32", False, False, 1.0, seed=9)
    i32 = make_inputs(w32)
    m32 = make_module(w32)
    qv = to_dev(i32["q"]).permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    with pytest.raises(RuntimeError, match="AA_ERR_UNSUPPORTED"):
        m32.forward_strided(qv, qv, qv, 8, 8, 4)
