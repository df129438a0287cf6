"""Host-side checks that need no GPU: the library builds, loads and exports the declared ABI;
construction fails loudly without a GPU; workload bookkeeping; rank sharding over gloo."""
import ctypes
import os
import re
import socket
import subprocess
import sys

import pytest
import torch

import paper_2312_08874_b200 as pkg
from paper_2312_08874_b200 import WORKLOADS, make_inputs, shard_slabs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "agent_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(agent_attn_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = pkg.load_library()
    names = declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/agent_attn.h but not exported"
    assert sorted(pkg.EXPORTS) == names


def test_config_struct_matches_header_field_order():
    text = open(os.path.join(ROOT, "include", "agent_attn.h")).read()
    body = re.search(r"typedef struct \{(.*?)\} agent_attn_config;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = re.findall(r"(?:int|float)\s+(\w+)\s*;", body)
    from paper_2312_08874_b200.binding import AgentAttnConfig
    assert fields == [f[0] for f in AgentAttnConfig._fields_]


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_create_fails_loudly_without_a_gpu():
    with pytest.raises(pkg.AgentAttnError) as e:
        pkg.AgentAttention(1, 3, 64, 196, 49, torch.float32)
    assert e.value.status == 4


def test_null_and_bad_arguments_at_the_abi():
    lib = pkg.load_library()
    assert lib.agent_attn_create(None, None) == 1
    assert lib.agent_attn_destroy(None) == 0
    assert lib.agent_attn_workspace_bytes(None, 14, 14, 49) == 0
    assert lib.agent_attn_last_error(None) == b"agent_attn: null handle"
    from paper_2312_08874_b200.binding import AgentAttnConfig
    h = ctypes.c_void_p()
    bad = AgentAttnConfig(1, 1, 136, 64, 16, 1, 0.0, 0.0, 0, 0)        # head_dim > 128
    assert lib.agent_attn_create(ctypes.byref(h), ctypes.byref(bad)) == 2
    bad = AgentAttnConfig(1, 1, 64, 64, 300, 1, 0.0, 0.0, 0, 0)        # too many agents
    assert lib.agent_attn_create(ctypes.byref(h), ctypes.byref(bad)) == 2
    bad = AgentAttnConfig(0, 1, 64, 64, 16, 1, 0.0, 0.0, 0, 0)         # empty batch
    assert lib.agent_attn_create(ctypes.byref(h), ctypes.byref(bad)) == 1
    bad = AgentAttnConfig(1, 1, 60, 64, 16, 1, 0.0, 0.0, 0, 0)         # rows not 16-byte multiples
    assert lib.agent_attn_create(ctypes.byref(h), ctypes.byref(bad)) == 2


def test_workload_bytes_match_the_roofline_table():
    # Q, K, V, O once each, both biases and the filter once per head.
    assert WORKLOADS["cfg1_deit_f32"].algorithmic_bytes() == 602112 + 9 * 3 * 64 * 4
    assert WORKLOADS["cfg3_pvt_bf16"].algorithmic_bytes() == 102760448 + 614656 + 9 * 64 * 2
    assert WORKLOADS["cfg4_sd_f16"].algorithmic_bytes() == 20971520
    assert WORKLOADS["cfg5a_hires_bf16"].algorithmic_bytes() == 2 * 134217728 + 9 * 8 * 64 * 2


def test_inputs_are_seeded_and_shaped():
    w = WORKLOADS["cfg2_deit_bf16"].scaled(batch=2)
    a, b = make_inputs(w), make_inputs(w)
    for k in a:
        assert torch.equal(a[k], b[k])
    assert a["q"].shape == (2, 3, 196, 64) and a["q"].dtype == torch.bfloat16
    assert a["b1"].shape == (3, 49, 196) and a["b2"].shape == (3, 196, 49) and a["dwc"].shape == (3, 64, 3, 3)
    assert abs(float(a["b1"].float().std()) - 0.02) < 2e-3
    c = make_inputs(w, seed=99)
    assert not torch.equal(a["q"], c["q"])
    w4 = WORKLOADS["cfg4_sd_f16"].scaled(batch=1)
    i4 = make_inputs(w4)
    assert i4["b1"] is None and i4["dwc"] is None
    assert abs(float(i4["q"].float().std()) - 40 ** -0.5) < 5e-3


def test_shard_slabs_partitions_the_batch():
    for total, world in [(64, 1), (64, 8), (10, 4), (3, 8)]:
        seen = []
        for r in range(world):
            seen += list(shard_slabs(total, world, r))
        assert seen == list(range(total))


_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
from paper_2312_08874_b200 import dist as d, shard_slabs
rank, local, world = d.init("gloo")
d.barrier()
mine = list(shard_slabs(10, world, rank))
t = d.max_over_ranks(1.0 + rank)          # the slowest rank defines the job's time
n = d.sum_over_ranks(len(mine))
d.barrier()
print(f"rank={{rank}} world={{world}} max={{t}} total={{n}} mine={{mine}}")
d.shutdown()
"""


def test_two_rank_gloo_timing_reduction_and_sharding(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER.format(root=ROOT))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert "rank=0 world=2 max=2.0 total=10.0 mine=[0, 1, 2, 3, 4]" in outs[0]
    assert "rank=1 world=2 max=2.0 total=10.0 mine=[5, 6, 7, 8, 9]" in outs[1]
