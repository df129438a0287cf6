"""Thin ctypes binding of `libagent_attn.so` (declared in `include/agent_attn.h`).

Argument marshalling only: every step of the forward pass runs in the library's CUDA kernels.
torch is used for device memory (`data_ptr()`), streams and dtype bookkeeping.  There is no
fallback: if the library is missing or no sm_100 GPU is present, construction raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from .build import LIB_PATH, build_library

AA_F32, AA_BF16, AA_F16 = 0, 1, 2
AA_PATH_AUTO, AA_PATH_SIMT, AA_PATH_UNFUSED, AA_PATH_QUEUE = 0, 1, 2, 3
STATUS_NAMES = {0: "AA_OK", 1: "AA_ERR_INVALID_ARG", 2: "AA_ERR_UNSUPPORTED", 3: "AA_ERR_WORKSPACE",
                4: "AA_ERR_CUDA", 5: "AA_ERR_TIMEOUT"}
_DTYPES = {torch.float32: AA_F32, torch.bfloat16: AA_BF16, torch.float16: AA_F16}

EXPORTS = [
    "agent_attn_create", "agent_attn_destroy", "agent_attn_last_error", "agent_attn_workspace_bytes",
    "agent_attn_forward", "agent_attn_pool", "agent_attn_aggregate", "agent_attn_broadcast",
    "agent_attn_staging_bytes", "agent_attn_forward_host", "agent_attn_query_status",
    "agent_attn_last_launch_count", "agent_attn_aggregate_static", "agent_attn_static_scratch_bytes",
    "agent_attn_compose_bias", "agent_attn_forward_strided",
    "agent_attn_backward_workspace_bytes", "agent_attn_backward", "agent_attn_test_set_poll_limit",
    "agent_attn_test_set_stage_mask",
]


class AgentAttnConfig(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int), ("heads", ctypes.c_int), ("head_dim", ctypes.c_int),
                ("max_tokens", ctypes.c_int), ("max_agents", ctypes.c_int), ("dtype", ctypes.c_int),
                ("scale1", ctypes.c_float), ("scale2", ctypes.c_float), ("device", ctypes.c_int),
                ("path", ctypes.c_int)]


class AgentAttnBias(ctypes.Structure):
    _fields_ = [("b1", ctypes.c_void_p), ("b2", ctypes.c_void_p)]


class AgentAttnGrads(ctypes.Structure):
    _fields_ = [("dq", ctypes.c_void_p), ("dk", ctypes.c_void_p), ("dv", ctypes.c_void_p),
                ("db1", ctypes.c_void_p), ("db2", ctypes.c_void_p), ("dwd", ctypes.c_void_p)]


class AgentAttnError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


_lib: Optional[ctypes.CDLL] = None


def load_library(build_if_missing: bool = True) -> ctypes.CDLL:
    """dlopen the in-tree library (building it first if its sources are newer)."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing:
        try:
            build_library()
        except Exception:
            if not os.path.exists(LIB_PATH):
                raise
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} is missing: run `python -m paper_2312_08874_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.agent_attn_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(AgentAttnConfig)]
    lib.agent_attn_create.restype = ci
    lib.agent_attn_destroy.argtypes = [vp]
    lib.agent_attn_destroy.restype = ci
    lib.agent_attn_last_error.argtypes = [vp]
    lib.agent_attn_last_error.restype = ctypes.c_char_p
    lib.agent_attn_workspace_bytes.argtypes = [vp, ci, ci, ci]
    lib.agent_attn_workspace_bytes.restype = sz
    lib.agent_attn_forward.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ctypes.POINTER(AgentAttnBias), vp,
                                       vp, vp, sz, vp]
    lib.agent_attn_forward.restype = ci
    ll3 = ctypes.POINTER(ctypes.c_longlong)
    lib.agent_attn_forward_strided.argtypes = [vp, vp, vp, vp, vp, ll3, ci, ci, ci, ctypes.POINTER(AgentAttnBias), vp,
                                               vp, ll3, vp, ctypes.c_size_t, vp]
    lib.agent_attn_forward_strided.restype = ci
    lib.agent_attn_pool.argtypes = [vp, vp, ci, ci, ci, ci, vp, vp]
    lib.agent_attn_pool.restype = ci
    lib.agent_attn_aggregate.argtypes = [vp, vp, vp, vp, vp, ci, ci, vp, vp, sz, vp]
    lib.agent_attn_aggregate.restype = ci
    lib.agent_attn_broadcast.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, vp, vp]
    lib.agent_attn_broadcast.restype = ci
    lib.agent_attn_staging_bytes.argtypes = [vp, ci, ci, ci]
    lib.agent_attn_staging_bytes.restype = sz
    lib.agent_attn_forward_host.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ctypes.POINTER(AgentAttnBias), vp,
                                            vp, vp, sz, vp]
    lib.agent_attn_forward_host.restype = ci
    lib.agent_attn_query_status.argtypes = [vp, vp]
    lib.agent_attn_query_status.restype = ci
    lib.agent_attn_last_launch_count.argtypes = [vp]
    lib.agent_attn_last_launch_count.restype = ci
    lib.agent_attn_aggregate_static.argtypes = [vp, vp, vp, vp, vp, ci, ci, vp, vp]
    lib.agent_attn_aggregate_static.restype = ci
    lib.agent_attn_compose_bias.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, vp]
    lib.agent_attn_compose_bias.restype = ci
    lib.agent_attn_backward_workspace_bytes.argtypes = [vp, ci, ci, ci]
    lib.agent_attn_backward_workspace_bytes.restype = sz
    lib.agent_attn_backward.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ctypes.POINTER(AgentAttnBias), vp,
                                        ctypes.POINTER(AgentAttnGrads), vp, sz, vp]
    lib.agent_attn_backward.restype = ci
    lib.agent_attn_test_set_stage_mask.argtypes = [vp, ctypes.c_uint]
    lib.agent_attn_test_set_stage_mask.restype = ci
    lib.agent_attn_test_set_poll_limit.argtypes = [vp, ctypes.c_uint]
    lib.agent_attn_test_set_poll_limit.restype = ci
    lib.agent_attn_static_scratch_bytes.argtypes = []
    lib.agent_attn_static_scratch_bytes.restype = sz
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream: Optional[torch.cuda.Stream]):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


class AgentAttention:
    """One `agent_attn_handle`.  Methods mirror the C entry points of the same names."""

    def __init__(self, batch: int, heads: int, head_dim: int, max_tokens: int, max_agents: int,
                 dtype: torch.dtype, scale1: float = 0.0, scale2: float = 0.0,
                 device: int = 0, path: int = AA_PATH_AUTO):
        self.lib = load_library()
        self.cfg = AgentAttnConfig(batch, heads, head_dim, max_tokens, max_agents, _DTYPES[dtype],
                                   scale1, scale2, device, path)
        self.dtype = dtype
        self.device = torch.device("cuda", device)
        self.batch, self.heads, self.head_dim = batch, heads, head_dim
        self._h = ctypes.c_void_p()
        rc = self.lib.agent_attn_create(ctypes.byref(self._h), ctypes.byref(self.cfg))
        if rc != 0:
            self._h = ctypes.c_void_p()
            raise AgentAttnError(rc, "agent_attn_create failed (is an sm_100 GPU present?)")
        self._ws: Optional[torch.Tensor] = None
        self._staging: Optional[torch.Tensor] = None

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self.lib.agent_attn_destroy(self._h)
            self._h = ctypes.c_void_p()

    __del__ = close

    # ------------------------------------------------------------------ helpers
    def _check(self, rc: int):
        if rc != 0:
            raise AgentAttnError(rc, self.lib.agent_attn_last_error(self._h).decode())

    def _chk_tensor(self, t: Optional[torch.Tensor], shape, name: str, cuda: bool = True):
        if t is None:
            return
        if tuple(t.shape) != tuple(shape) or t.dtype != self.dtype or not t.is_contiguous() or t.is_cuda != cuda:
            raise ValueError(f"{name}: expected contiguous {'cuda' if cuda else 'cpu'} {self.dtype} tensor of "
                             f"shape {tuple(shape)}, got {tuple(t.shape)} {t.dtype} on {t.device}")

    def workspace_bytes(self, grid_h: int, grid_w: int, n_agents: int) -> int:
        return int(self.lib.agent_attn_workspace_bytes(self._h, grid_h, grid_w, n_agents))

    def staging_bytes(self, grid_h: int, grid_w: int, n_agents: int) -> int:
        return int(self.lib.agent_attn_staging_bytes(self._h, grid_h, grid_w, n_agents))

    def workspace(self, grid_h: int, grid_w: int, n_agents: int) -> torch.Tensor:
        need = self.workspace_bytes(grid_h, grid_w, n_agents)
        if need == 0:
            raise ValueError("shape not supported by this handle")
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        return self._ws

    def intermediates(self, workspace: torch.Tensor, n_agents: int):
        """Views of the agents A and the agent features V_A ([B, heads, n, d] each) that `forward` left in its
        workspace: A occupies the first B*heads*n*d elements, V_A starts at the next multiple of 256 bytes."""
        count = self.batch * self.heads * n_agents * self.head_dim
        nbytes = count * workspace.new_empty(0, dtype=self.dtype).element_size()
        va_off = (nbytes + 255) // 256 * 256
        shape = (self.batch, self.heads, n_agents, self.head_dim)
        return (workspace[:nbytes].view(self.dtype).view(shape), workspace[va_off:va_off + nbytes].view(self.dtype).view(shape))

    def set_stage_mask(self, mask: int):
        """Measurement hook: which of the three streaming kernels `forward` launches (1 prep | 2 aggregation | 4 broadcast)."""
        self._check(self.lib.agent_attn_test_set_stage_mask(self._h, mask))

    def set_poll_limit(self, polls: int):
        """Test hook: polls of another block's counter before a wait of the task-queue kernel gives up."""
        self._check(self.lib.agent_attn_test_set_poll_limit(self._h, polls & 0xffffffff))

    def last_launch_count(self) -> int:
        return int(self.lib.agent_attn_last_launch_count(self._h))

    def query_status(self, stream=None) -> int:
        return int(self.lib.agent_attn_query_status(self._h, _stream_ptr(stream)))

    # ------------------------------------------------------------------ entry points
    def forward(self, q, k, v, grid_h: int, grid_w: int, n_agents: int, agents=None, b1=None, b2=None,
                dwc_weight=None, out=None, workspace=None, stream=None) -> torch.Tensor:
        B, h, d, N = self.batch, self.heads, self.head_dim, grid_h * grid_w
        for t, nm in ((q, "q"), (k, "k"), (v, "v")):
            self._chk_tensor(t, (B, h, N, d), nm)
        self._chk_tensor(agents, (B, h, n_agents, d), "agents")
        self._chk_tensor(b1, (h, n_agents, N), "b1")
        self._chk_tensor(b2, (h, N, n_agents), "b2")
        self._chk_tensor(dwc_weight, (h, d, 3, 3), "dwc_weight")
        if out is None:
            out = torch.empty_like(q)
        self._chk_tensor(out, (B, h, N, d), "out")
        ws = self.workspace(grid_h, grid_w, n_agents) if workspace is None else workspace
        bias = AgentAttnBias(_ptr(b1), _ptr(b2)) if (b1 is not None or b2 is not None) else None
        self._check(self.lib.agent_attn_forward(
            self._h, _ptr(q), _ptr(k), _ptr(v), _ptr(agents), grid_h, grid_w, n_agents,
            ctypes.byref(bias) if bias is not None else None, _ptr(dwc_weight), _ptr(out), _ptr(ws),
            ws.numel(), _stream_ptr(stream)))
        return out

    def forward_strided(self, q, k, v, grid_h: int, grid_w: int, n_agents: int, agents=None, b1=None, b2=None,
                        dwc_weight=None, out=None, workspace=None, stream=None) -> torch.Tensor:
        """Eq. 6 on VIEWS of shape [B, heads, N, d] with any batch / head / token strides (last dim contiguous).

        Typical use: `qkv` of shape [B, N, 3, heads, d] straight from a projection, passed as
        `qkv[:, :, i].permute(0, 2, 1, 3)`; `out` may be such a view of a [B, N, heads, d] tensor (that is
        what is allocated when `out` is None).  Q, K and V must share their strides.
        """
        B, h, d, N = self.batch, self.heads, self.head_dim, grid_h * grid_w
        for t, nm in ((q, "q"), (k, "k"), (v, "v"), (out, "out")):
            if t is None:
                continue
            if tuple(t.shape) != (B, h, N, d) or t.dtype != self.dtype or not t.is_cuda or t.stride(3) != 1:
                raise ValueError(f"{nm}: expected a cuda {self.dtype} view of shape {(B, h, N, d)} with contiguous channels")
        if q.stride() != k.stride() or q.stride() != v.stride():
            raise ValueError("q, k and v must have the same strides")
        self._chk_tensor(agents, (B, h, n_agents, d), "agents")
        self._chk_tensor(b1, (h, n_agents, N), "b1")
        self._chk_tensor(b2, (h, N, n_agents), "b2")
        self._chk_tensor(dwc_weight, (h, d, 3, 3), "dwc_weight")
        if out is None:
            out = torch.empty((B, N, h, d), dtype=self.dtype, device=self.device).permute(0, 2, 1, 3)
        ws = self.workspace(grid_h, grid_w, n_agents) if workspace is None else workspace
        bias = AgentAttnBias(_ptr(b1), _ptr(b2)) if (b1 is not None or b2 is not None) else None
        sin = (ctypes.c_longlong * 3)(q.stride(0), q.stride(1), q.stride(2))
        sout = (ctypes.c_longlong * 3)(out.stride(0), out.stride(1), out.stride(2))
        self._check(self.lib.agent_attn_forward_strided(
            self._h, _ptr(q), _ptr(k), _ptr(v), _ptr(agents), sin, grid_h, grid_w, n_agents,
            ctypes.byref(bias) if bias is not None else None, _ptr(dwc_weight), _ptr(out), sout, _ptr(ws),
            ws.numel(), _stream_ptr(stream)))
        return out

    def backward_workspace(self, grid_h: int, grid_w: int, n_agents: int) -> torch.Tensor:
        nbytes = self.lib.agent_attn_backward_workspace_bytes(self._h, grid_h, grid_w, n_agents)
        if nbytes == 0:
            raise AgentAttnError(2, f"backward does not support grid {grid_h}x{grid_w} with {n_agents} agents")
        return torch.empty(nbytes, dtype=torch.uint8, device=self.device)

    def backward(self, q, k, v, d_out, grid_h: int, grid_w: int, n_agents: int, b1=None, b2=None,
                 dwc_weight=None, need_bias_grads: bool = True, need_filter_grad: bool = True,
                 workspace=None, stream=None) -> dict:
        """`agent_attn_backward`: fp32 gradients of Eq. 6 (pooled agents) for the upstream gradient `d_out`.

        Returns a dict with `dq`, `dk`, `dv` ([B, heads, N, d]) and, for the inputs that were given and asked
        for, `db1` ([heads, n, N]), `db2` ([heads, N, n]) and `dwd` ([heads, d, 3, 3]).
        """
        B, h, d, N = self.batch, self.heads, self.head_dim, grid_h * grid_w
        for t, nm in ((q, "q"), (k, "k"), (v, "v"), (d_out, "d_out")):
            if t is None:
                raise ValueError(f"{nm} is required")
            self._chk_tensor(t, (B, h, N, d), nm)
        self._chk_tensor(b1, (h, n_agents, N), "b1")
        self._chk_tensor(b2, (h, N, n_agents), "b2")
        self._chk_tensor(dwc_weight, (h, d, 3, 3), "dwc_weight")
        f32 = dict(dtype=torch.float32, device=self.device)
        g = {"dq": torch.empty((B, h, N, d), **f32), "dk": torch.empty((B, h, N, d), **f32),
             "dv": torch.empty((B, h, N, d), **f32)}
        if b1 is not None and need_bias_grads:
            g["db1"] = torch.empty((h, n_agents, N), **f32)
        if b2 is not None and need_bias_grads:
            g["db2"] = torch.empty((h, N, n_agents), **f32)
        if dwc_weight is not None and need_filter_grad:
            g["dwd"] = torch.empty((h, d, 3, 3), **f32)
        ws = self.backward_workspace(grid_h, grid_w, n_agents) if workspace is None else workspace
        bias = AgentAttnBias(_ptr(b1), _ptr(b2)) if (b1 is not None or b2 is not None) else None
        grads = AgentAttnGrads(_ptr(g["dq"]), _ptr(g["dk"]), _ptr(g["dv"]), _ptr(g.get("db1")), _ptr(g.get("db2")),
                               _ptr(g.get("dwd")))
        self._check(self.lib.agent_attn_backward(
            self._h, _ptr(q), _ptr(k), _ptr(v), _ptr(d_out), grid_h, grid_w, n_agents,
            ctypes.byref(bias) if bias is not None else None, _ptr(dwc_weight), ctypes.byref(grads), _ptr(ws),
            ws.numel(), _stream_ptr(stream)))
        return g

    def pool(self, q, grid_h: int, grid_w: int, pool_h: int, pool_w: int, out=None, stream=None):
        B, h, d = self.batch, self.heads, self.head_dim
        self._chk_tensor(q, (B, h, grid_h * grid_w, d), "q")
        if out is None:
            out = torch.empty((B, h, pool_h * pool_w, d), dtype=self.dtype, device=self.device)
        self._chk_tensor(out, (B, h, pool_h * pool_w, d), "out")
        self._check(self.lib.agent_attn_pool(self._h, _ptr(q), grid_h, grid_w, pool_h, pool_w, _ptr(out),
                                             _stream_ptr(stream)))
        return out

    def aggregate(self, agents, k, v, b1=None, out=None, workspace=None, stream=None):
        B, h, d = self.batch, self.heads, self.head_dim
        n, N = agents.shape[2], k.shape[2]
        self._chk_tensor(agents, (B, h, n, d), "agents")
        self._chk_tensor(k, (B, h, N, d), "k")
        self._chk_tensor(v, (B, h, N, d), "v")
        self._chk_tensor(b1, (h, n, N), "b1")
        if out is None:
            out = torch.empty_like(agents)
        ws = self.workspace(1, N, n) if workspace is None else workspace
        self._check(self.lib.agent_attn_aggregate(self._h, _ptr(agents), _ptr(k), _ptr(v), _ptr(b1), N, n,
                                                  _ptr(out), _ptr(ws), ws.numel(), _stream_ptr(stream)))
        return out

    def aggregate_static(self, agents, k, v, b1=None, out=None, stream=None):
        """`agent_attn_aggregate_static`: the aggregation for callers that cannot allocate.

        Same result as `aggregate`, but the split partials live in the library's fixed 32 MiB
        array instead of a workspace, so this call allocates nothing when `out` is given.
        Calls that overlap on the GPU share that array and must be serialised.
        """
        B, h, d = self.batch, self.heads, self.head_dim
        n, N = agents.shape[2], k.shape[2]
        self._chk_tensor(agents, (B, h, n, d), "agents")
        self._chk_tensor(k, (B, h, N, d), "k")
        self._chk_tensor(v, (B, h, N, d), "v")
        self._chk_tensor(b1, (h, n, N), "b1")
        if out is None:
            out = torch.empty_like(agents)
        self._check(self.lib.agent_attn_aggregate_static(self._h, _ptr(agents), _ptr(k), _ptr(v), _ptr(b1),
                                                         N, n, _ptr(out), _stream_ptr(stream)))
        return out

    def broadcast(self, q, agents, va, v, grid_h: int, grid_w: int, b2=None, dwc_weight=None, out=None,
                  stream=None):
        B, h, d, N = self.batch, self.heads, self.head_dim, grid_h * grid_w
        n = agents.shape[2]
        self._chk_tensor(q, (B, h, N, d), "q")
        self._chk_tensor(agents, (B, h, n, d), "agents")
        self._chk_tensor(va, (B, h, n, d), "va")
        self._chk_tensor(v, (B, h, N, d), "v")
        self._chk_tensor(b2, (h, N, n), "b2")
        self._chk_tensor(dwc_weight, (h, d, 3, 3), "dwc_weight")
        if out is None:
            out = torch.empty_like(q)
        self._check(self.lib.agent_attn_broadcast(self._h, _ptr(q), _ptr(agents), _ptr(va), _ptr(v), _ptr(b2),
                                                  _ptr(dwc_weight), grid_h, grid_w, n, _ptr(out),
                                                  _stream_ptr(stream)))
        return out

    def compose_bias(self, col, row, blk, grid_h: int, grid_w: int, n_agents: int, transpose: bool = False,
                     out=None, stream=None):
        """`agent_attn_compose_bias`: dense B1 ([heads, n, N]) or B2 ([heads, N, n], transpose=True)
        from column [heads, n, w], row [heads, n, h] and block [heads, n, h0, w0] components (App. B)."""
        h, N = self.heads, grid_h * grid_w
        self._chk_tensor(col, (h, n_agents, grid_w), "col")
        self._chk_tensor(row, (h, n_agents, grid_h), "row")
        h0, w0 = (blk.shape[2], blk.shape[3]) if blk is not None else (1, 1)
        self._chk_tensor(blk, (h, n_agents, h0, w0), "blk")
        shape = (h, N, n_agents) if transpose else (h, n_agents, N)
        if out is None:
            out = torch.empty(shape, dtype=self.dtype, device=self.device)
        self._chk_tensor(out, shape, "out")
        self._check(self.lib.agent_attn_compose_bias(self._h, _ptr(col), _ptr(row), _ptr(blk), h0, w0, grid_h, grid_w,
                                                     n_agents, int(transpose), _ptr(out), _stream_ptr(stream)))
        return out

    def forward_host(self, q, k, v, grid_h: int, grid_w: int, n_agents: int, agents=None, b1=None, b2=None,
                     dwc_weight=None, out=None, stream=None, synchronize: bool = True, staging=None) -> torch.Tensor:
        """Eq. 6 on host (ideally pinned) tensors: copies in, runs, copies the result back.

        Everything is queued on `stream`.  `staging` is the device scratch of the call (uint8, at least
        `staging_bytes(...)`); calls that are in flight at the same time on different streams (to overlap one
        step's copies with the next) need a staging buffer each.  By default the module keeps one of its own.
        """
        B, h, d, N = self.batch, self.heads, self.head_dim, grid_h * grid_w
        for t, nm in ((q, "q"), (k, "k"), (v, "v")):
            self._chk_tensor(t, (B, h, N, d), nm, cuda=False)
        self._chk_tensor(agents, (B, h, n_agents, d), "agents", cuda=False)
        self._chk_tensor(b1, (h, n_agents, N), "b1", cuda=False)
        self._chk_tensor(b2, (h, N, n_agents), "b2", cuda=False)
        self._chk_tensor(dwc_weight, (h, d, 3, 3), "dwc_weight", cuda=False)
        if out is None:
            out = torch.empty((B, h, N, d), dtype=self.dtype).pin_memory()
        self._chk_tensor(out, (B, h, N, d), "out", cuda=False)
        need = self.staging_bytes(grid_h, grid_w, n_agents)
        if need == 0:
            raise ValueError("shape not supported by this handle")
        if staging is not None:
            if staging.dtype != torch.uint8 or not staging.is_cuda or staging.numel() < need:
                raise ValueError(f"staging must be a CUDA uint8 tensor of at least {need} bytes")
        else:
            if self._staging is None or self._staging.numel() < need:
                self._staging = torch.empty(need, dtype=torch.uint8, device=self.device)
            staging = self._staging
        bias = AgentAttnBias(_ptr(b1), _ptr(b2)) if (b1 is not None or b2 is not None) else None
        s = torch.cuda.current_stream() if stream is None else stream
        self._check(self.lib.agent_attn_forward_host(
            self._h, _ptr(q), _ptr(k), _ptr(v), _ptr(agents), grid_h, grid_w, n_agents,
            ctypes.byref(bias) if bias is not None else None, _ptr(dwc_weight), _ptr(out),
            _ptr(staging), staging.numel(), ctypes.c_void_p(s.cuda_stream)))
        if synchronize:
            s.synchronize()
        return out
