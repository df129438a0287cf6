"""GPU-vs-oracle parity through the C ABI, element by element on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import agent_attention_oracle as orc
from paper_2312_08874_b200 import (AA_PATH_AUTO, AA_PATH_QUEUE, AA_PATH_SIMT, AA_PATH_UNFUSED, WORKLOADS, AgentAttention, Workload,
                                   make_inputs)
from tests.parity_util import (assert_close, errors, gpu_forward, make_module, oracle_forward, to_dev, to_np)

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------ the five configurations
@pytest.mark.parametrize("path", [AA_PATH_AUTO, AA_PATH_QUEUE, AA_PATH_UNFUSED], ids=["auto", "queue", "unfused"])
@pytest.mark.parametrize("name", ["cfg1_deit_f32", "cfg2_deit_bf16", "cfg3_pvt_bf16", "cfg4_sd_f16",
                                  "cfg5a_hires_bf16"])
def test_full_size_configs_match_oracle(name, path):
    w = WORKLOADS[name]
    if path == AA_PATH_UNFUSED and name not in ("cfg2_deit_bf16", "cfg3_pvt_bf16"):
        pytest.skip("only the small-agent-count configurations have two launch plans")
    if path == AA_PATH_QUEUE and name != "cfg3_pvt_bf16":
        pytest.skip("the task-queue kernel differs from the automatic choice only on long grids with few agents")
    inp = make_inputs(w)
    mod = make_module(w, path=path)
    out, ws = gpu_forward(mod, w, inp, return_workspace=True)
    ref, a_ref, va_ref = oracle_forward(w, inp, return_intermediates=True)
    assert_close(out, ref, w.dtype, name)
    # the agents and agent features that this very call left in its workspace (whichever kernels ran)
    a_ws, va_ws = mod.intermediates(ws, w.agents)
    assert_close(a_ws, a_ref, w.dtype, name + " agents in the workspace")
    assert_close(va_ws, va_ref, w.dtype, name + " agent features in the workspace")
    # intermediates through the step entry points
    a = mod.pool(to_dev(inp["q"]), w.grid_h, w.grid_w, w.pool, w.pool)
    assert_close(a, a_ref, w.dtype, name + " agents")
    va = mod.aggregate(a, to_dev(inp["k"]), to_dev(inp["v"]), b1=to_dev(inp["b1"]))
    torch.cuda.synchronize()
    assert_close(va, va_ref, w.dtype, name + " agent features")


def test_largest_config_matches_oracle_on_every_slab():
    w = WORKLOADS["cfg5b_hires_bf16"]
    inp = make_inputs(w)
    mod = make_module(w)
    out = gpu_forward(mod, w, inp)
    assert torch.isfinite(out.float()).all()
    ref = oracle_forward(w, inp)                       # all 16 slabs (about 70 G fp64 multiply-adds over the host threads)
    assert_close(out, ref, w.dtype, "cfg5b")
    for b in range(w.batch):
        for h in range(w.heads):
            assert_close(out[b:b + 1, h:h + 1], ref[b:b + 1, h:h + 1], w.dtype, f"cfg5b slab {(b, h)}")


@pytest.mark.parametrize("path", [AA_PATH_QUEUE, AA_PATH_AUTO], ids=["queue", "auto"])
def test_more_slabs_than_the_queue_lag_interleaves_task_kinds(path):
    """With more slabs than the queue's lag (the L2 budget: 83 slabs of this shape) aggregation and broadcast tasks
    alternate in the queue, so blocks take tickets of one kind while finishing a task of the other and broadcast
    tasks may find their slab's flag not yet set: sampled slabs against the oracle, repeatable bit for bit, and no
    bounded wait expired."""
    w = WORKLOADS["cfg3_pvt_bf16"].scaled(batch=160, seed=77)      # (streaming kernels: one aggregation block per slab)
    inp = make_inputs(w)
    mod = make_module(w, path=path)
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
    mod = make_module(w)
    out, ws = gpu_forward(mod, w, inp, return_workspace=True)
    ref = oracle_forward(w, inp)
    assert torch.isfinite(out.float()).all()
    # peaked softmaxes amplify the rounding of the agents to bf16 (a logit of 40 carries an error of 0.1): only a
    # loose bound against the exact oracle ...
    assert errors(out, ref)["rel_l2"] < 5e-2
    # ... and the usual one against the oracle run on the very agents the GPU used (its rounded A), which leaves
    # the kernels' own arithmetic: probabilities and V_A in 16 bits, fp32 accumulation
    a_ws, _ = mod.intermediates(ws, w.agents)
    ref_a = orc.forward(to_np(inp["q"]), to_np(inp["k"]), to_np(inp["v"]), w.grid_h, w.grid_w, agents=to_np(a_ws.cpu()),
                        threads=2)
    e = errors(out, ref_a)
    assert e["rel_l2"] <= 5e-3 and e["max_abs"] <= 3e-2 * float(np.abs(ref_a).max()), e


def test_forward_host_matches_forward():
    w = WORKLOADS["cfg2_deit_bf16"].scaled(batch=3)
    inp = make_inputs(w)
    mod = make_module(w)
    out_dev = gpu_forward(mod, w, inp).cpu()
    pin = {k: (None if v is None else v.pin_memory()) for k, v in inp.items()}
    out_host = mod.forward_host(pin["q"], pin["k"], pin["v"], w.grid_h, w.grid_w, w.agents, b1=pin["b1"],
                                b2=pin["b2"], dwc_weight=pin["dwc"])
    assert torch.equal(out_dev, out_host)
    assert mod.last_launch_count() == 1            # the persistent task-queue kernel (short grids)
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
    # strided tensors are read in place by the task-queue and tensor-memory kernels: the dense reference call is
    # pinned to the same kernels (AA_PATH_AUTO would take long grids with few agents to the streaming kernels)
    mod = make_module(w, path=AA_PATH_QUEUE)
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
    out = torch.full_like(dense, float("nan"))
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


# ------------------------------------------------ streaming kernels (long grids, few agents: n <= 64, d = 64)
STREAM = [
    # batch heads H   W   pool dtype  bias  dwc
    (2, 2, 32, 32, 4, "f16", True, True),        # four grid rows per tile
    (1, 3, 66, 24, 6, "bf16", True, True),       # ragged last tile of every slab (66 rows, 4 per tile), three heads
    (2, 1, 40, 40, 5, "bf16", False, False),     # no bias, no depthwise term
    (5, 2, 28, 56, 7, "bf16", True, True),       # H != W
    (2, 2, 64, 64, 8, "f16", True, True),        # widest grid, 64 agents, one grid row per tile
    (1, 2, 128, 8, 1, "bf16", True, True),       # narrowest grid, a single agent, twelve rows per tile
    (3, 1, 48, 48, 6, "bf16", True, False),      # bias without the depthwise term
    (1, 2, 36, 60, 6, "f16", False, True),       # depthwise term without bias
    (1, 1, 64, 64, 7, "bf16", True, True),       # one slab: a cluster of eight aggregation blocks; 64 % 7 != 0: see below
    (200, 1, 32, 32, 4, "bf16", True, True),     # more slabs than SMs: two aggregation waves, blocks that cross slabs
]


@pytest.mark.parametrize("case", STREAM, ids=[f"B{c[0]}h{c[1]}_{c[2]}x{c[3]}_p{c[4]}_{c[5]}" for c in STREAM])
def test_streaming_kernels_match_oracle(case):
    B, heads, H, W, pool, dtype, bias, dwc = case
    if H % pool or W % pool:
        pool = 8                                          # block pooling needs windows that tile the grid
    w = Workload("stream", B, heads, H, W, 64, pool, dtype, bias, dwc, 1.0, seed=500 + H * W + pool)
    inp = make_inputs(w, bias_std=0.5, dwc_std=0.2)
    mod = make_module(w)
    out, ws = gpu_forward(mod, w, inp, return_workspace=True)
    assert mod.last_launch_count() == 3, "expected the three streaming kernels"
    sample = None if B <= 8 else [(0, 0), (B // 2, 0), (B - 1, heads - 1)]
    if sample is None:
        ref, a_ref, va_ref = oracle_forward(w, inp, return_intermediates=True)
        assert_close(out, ref, dtype, f"{case}")
        a_ws, va_ws = mod.intermediates(ws, w.agents)
        assert_close(a_ws, a_ref, dtype, "agents in the workspace")
        assert_close(va_ws, va_ref, dtype, "agent features in the workspace")
    else:
        for (b, h), ref in zip(sample, oracle_forward(w, inp, slabs=sample)):
            assert_close(out[b:b + 1, h:h + 1], ref, dtype, f"slab {(b, h)}")
        assert torch.isfinite(out.float()).all()
    again = gpu_forward(mod, w, inp)
    assert torch.equal(out, again), "the streaming kernels must be bit-reproducible"


def test_streaming_kernels_with_caller_supplied_agents_and_separate_scales():
    w = Workload("stream_user_a", 2, 2, 40, 32, 64, 1, "bf16", True, True, 1.0, seed=21)
    n = 23                                                # not a square: no pooling grid exists for it
    inp = make_inputs(w)
    g = torch.Generator().manual_seed(22)
    agents = torch.randn((2, 2, n, 64), generator=g).to(torch.bfloat16)
    inp["b1"] = (torch.randn((2, n, w.tokens), generator=g) * 0.3).to(torch.bfloat16)
    inp["b2"] = (torch.randn((2, w.tokens, n), generator=g) * 0.3).to(torch.bfloat16)
    s1, s2 = 0.1, 64.0 ** -0.15
    w = Workload("stream_user_a", 2, 2, 40, 32, 64, 1, "bf16", True, True, 1.0, seed=21)
    mod = AgentAttention(2, 2, 64, w.tokens, n, torch.bfloat16, scale1=s1, scale2=s2)
    dev = {k: to_dev(v) for k, v in inp.items()}
    out = torch.full_like(dev["q"], float("nan"))
    mod.forward(dev["q"], dev["k"], dev["v"], 40, 32, n, agents=agents.cuda(), b1=dev["b1"], b2=dev["b2"],
                dwc_weight=dev["dwc"], out=out)
    torch.cuda.synchronize()
    assert mod.query_status() == 0 and mod.last_launch_count() == 3
    ref = orc.forward(to_np(inp["q"]), to_np(inp["k"]), to_np(inp["v"]), 40, 32, agents=to_np(agents), b1=to_np(inp["b1"]),
                      b2=to_np(inp["b2"]), dwc_weight=to_np(inp["dwc"]), scale1=s1, scale2=s2, threads=4)
    assert_close(out, ref, "bf16", "user agents, separate scales")
    ref_default = orc.forward(to_np(inp["q"]), to_np(inp["k"]), to_np(inp["v"]), 40, 32, agents=to_np(agents),
                              b1=to_np(inp["b1"]), b2=to_np(inp["b2"]), dwc_weight=to_np(inp["dwc"]), threads=4)
    assert errors(out, ref_default)["rel_l2"] > 1e-2      # the scales really are used


def test_streaming_aggregation_moves_its_reference_when_logits_grow():
    """Logits with a standard deviation of several units: rows outgrow the reference taken on their first tile, so
    the rescaling path of the aggregation runs (and the broadcast softmax is peaked)."""
    w = Workload("stream_hot", 2, 1, 48, 48, 64, 6, "bf16", True, False, 3.0, seed=23)
    inp = make_inputs(w, bias_std=2.0)
    mod = make_module(w)
    out, ws = gpu_forward(mod, w, inp, return_workspace=True)
    assert mod.last_launch_count() == 3
    ref, a_ref, va_ref = oracle_forward(w, inp, return_intermediates=True)
    assert torch.isfinite(out.float()).all()
    _, va_ws = mod.intermediates(ws, w.agents)
    # peaked softmaxes amplify the 16-bit rounding of A (a logit of 30 carries an error of 0.1): loose bounds
    assert errors(va_ws, va_ref)["rel_l2"] < 5e-2
    assert errors(out, ref)["rel_l2"] < 5e-2


def test_masked_keys_and_agents_through_infinite_bias_entries():
    """An infinite negative bias entry removes a key (or an agent) from a softmax.  The streaming kernels add the
    bias inside a tensor-core product, so they clamp it to a large finite value first: same result."""
    w = Workload("stream_mask", 1, 2, 32, 32, 64, 4, "bf16", True, True, 1.0, seed=24)
    inp = make_inputs(w, bias_std=0.5)
    b1, b2 = inp["b1"].clone(), inp["b2"].clone()
    b1[:, :, 100:400] = float("-inf")                     # every agent ignores these keys
    b1[0, 3, :1000] = float("-inf")                       # one agent sees only the last 24 keys
    b2[:, :, 5] = float("-inf")                           # no query listens to agent 5
    b2[1, 17, :15] = float("-inf")
    inp["b1"], inp["b2"] = b1, b2
    mod = make_module(w)
    out = gpu_forward(mod, w, inp)
    assert mod.last_launch_count() == 3
    assert_close(out, oracle_forward(w, inp), "bf16", "infinite bias entries")


@pytest.mark.parametrize("path,case", [(AA_PATH_AUTO, (3, 1, 32, 32, 4)), (AA_PATH_QUEUE, (3, 1, 14, 14, 7)),
                                       (AA_PATH_QUEUE, (3, 1, 32, 32, 4))], ids=["stream", "queue_ragged_tile", "queue"])
def test_non_finite_values_in_one_slab_do_not_leak_into_another(path, case):
    """Tiles are cut from a flat token axis, so the last tile of a slab may run into the next slab's rows; their
    weights are zero, and 0 * NaN must not reach the slab's result."""
    B, heads, H, W, pool = case
    w = Workload("leak", B, heads, H, W, 64, pool, "bf16", True, True, 1.0, seed=25)
    inp = make_inputs(w)
    clean = gpu_forward(make_module(w, path=path), w, inp).clone()
    bad = {k: (v.clone() if v is not None else None) for k, v in inp.items()}
    for name in ("q", "k", "v"):
        bad[name][1] = float("nan")                       # the middle slab is poison
    out = gpu_forward(make_module(w, path=path), w, bad)
    assert torch.equal(out[0], clean[0]) and torch.equal(out[2], clean[2])
    assert torch.isnan(out[1].float()).all()


def test_an_expired_flag_wait_is_reported_and_the_next_call_is_clean():
    """Failure detection without a fault: with the poll limit of the task-queue kernel set to 0 the first poll of a
    counter that the slab's other blocks have not reached yet gives up; the call returns, the status query reports
    AA_ERR_TIMEOUT once, and a normal call afterwards matches the oracle."""
    w = WORKLOADS["cfg3_pvt_bf16"].scaled(batch=2)        # seven aggregation tasks per slab wait for one another
    inp = make_inputs(w)
    mod = make_module(w, path=AA_PATH_QUEUE)
    dev = {k: to_dev(v) for k, v in inp.items()}
    mod.set_poll_limit(0)
    ws = torch.zeros((mod.workspace_bytes(w.grid_h, w.grid_w, w.agents),), dtype=torch.uint8, device="cuda")
    mod.forward(dev["q"], dev["k"], dev["v"], w.grid_h, w.grid_w, w.agents, b1=dev["b1"], b2=dev["b2"],
                dwc_weight=dev["dwc"], workspace=ws)
    torch.cuda.synchronize()
    assert mod.query_status() == 5, "AA_ERR_TIMEOUT expected"
    assert mod.query_status() == 0, "the status word is cleared by the query"
    mod.set_poll_limit(0xffffffff)
    out = gpu_forward(mod, w, inp)
    assert_close(out, oracle_forward(w, inp), w.dtype, "after the expired wait")
