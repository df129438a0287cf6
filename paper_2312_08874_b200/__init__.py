"""Agent Attention forward pass for NVIDIA B200: CUDA kernels behind a C ABI, plus this binding."""
from .binding import (AA_PATH_AUTO, AA_PATH_QUEUE, AA_PATH_SIMT, AA_PATH_UNFUSED, AgentAttention, AgentAttnError, EXPORTS,
                      load_library)
from .workloads import WORKLOADS, Workload, make_inputs, make_upstream_grad, shard_slabs

__all__ = ["AA_PATH_AUTO", "AA_PATH_QUEUE", "AA_PATH_SIMT", "AA_PATH_UNFUSED", "AgentAttention", "AgentAttnError", "EXPORTS", "load_library",
           "WORKLOADS", "Workload", "make_inputs", "make_upstream_grad", "shard_slabs"]
