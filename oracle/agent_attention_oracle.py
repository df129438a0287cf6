"""ctypes front end of the fp64 CPU oracle (`agent_attention_oracle.c`).

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke check and by the benchmark's
CPU-baseline leg; never by the CUDA package.  Arguments and results are numpy float64
arrays; every function here only marshals them to the C routine of the same name.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "agent_attention_oracle.c")
_LIB = os.path.join(_HERE, "libagent_attention_oracle.so")
_lib: Optional[ctypes.CDLL] = None

_DP = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP for the loop over slabs)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        # The mutation test points this at deliberately broken builds of the C file to
        # show that the pins notice; nothing else sets it.
        lib = ctypes.CDLL(os.environ.get("AGENT_ATTENTION_ORACLE_LIB") or build())
        lib.aa_oracle_pool.argtypes = [_DP] + [ctypes.c_int] * 5 + [_DP]
        lib.aa_oracle_pool.restype = None
        lib.aa_oracle_softmax_attention.argtypes = (
            [_DP] * 4 + [ctypes.c_int] * 4 + [ctypes.c_double, _DP, _DP])
        lib.aa_oracle_softmax_attention.restype = None
        lib.aa_oracle_dwc_add.argtypes = [_DP, _DP] + [ctypes.c_int] * 3 + [_DP]
        lib.aa_oracle_dwc_add.restype = None
        lib.aa_oracle_forward.argtypes = (
            [_DP] * 4 + [ctypes.c_int] * 8 + [_DP] * 3 + [ctypes.c_double] * 2
            + [_DP] * 3 + [ctypes.c_int])
        lib.aa_oracle_forward.restype = ctypes.c_int
        lib.aa_oracle_explicit.argtypes = (
            [_DP] * 6 + [ctypes.c_int] * 3 + [ctypes.c_double] * 2 + [_DP] * 2)
        lib.aa_oracle_explicit.restype = None
        lib.aa_oracle_macs.argtypes = [ctypes.c_longlong] * 4 + [ctypes.POINTER(ctypes.c_longlong)]
        lib.aa_oracle_macs.restype = ctypes.c_longlong
        lib.aa_oracle_compose_bias.argtypes = [_DP] * 3 + [ctypes.c_int] * 6 + [_DP]
        lib.aa_oracle_compose_bias.restype = None
        lib.aa_oracle_backward.argtypes = ([_DP] * 4 + [ctypes.c_int] * 8 + [_DP] * 3 + [ctypes.c_double] * 2 + [_DP] * 6)
        lib.aa_oracle_backward.restype = ctypes.c_int
        lib.aa_oracle_max_threads.argtypes = []
        lib.aa_oracle_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _c(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_DP)


def max_threads() -> int:
    return int(_load().aa_oracle_max_threads())


def pool(q: np.ndarray, grid_h: int, grid_w: int, ph: int, pw: int) -> np.ndarray:
    """A = Pooling(Q) for one slab.  q [N, d] -> [ph*pw, d]."""
    q = _c(q)
    d = q.shape[-1]
    assert q.shape == (grid_h * grid_w, d)
    a = np.empty((ph * pw, d), dtype=np.float64)
    _load().aa_oracle_pool(_p(q), grid_h, grid_w, d, ph, pw, _p(a))
    return a


def softmax_attention(qm, km, vm, bias=None, scale: float = 1.0,
                      return_probs: bool = False):
    """One Softmax attention (Eq. 1 / Eq. 3) with an additive bias (Eq. 5), one slab."""
    qm, km, vm = _c(qm), _c(km), _c(vm)
    rows, d = qm.shape
    cols, dv = vm.shape
    assert km.shape == (cols, d)
    b = None if bias is None else _c(bias)
    assert b is None or b.shape == (rows, cols)
    out = np.empty((rows, dv), dtype=np.float64)
    probs = np.empty((rows, cols), dtype=np.float64) if return_probs else None
    _load().aa_oracle_softmax_attention(_p(qm), _p(km), _p(vm), _p(b), rows, cols, d, dv,
                                        float(scale), _p(out), _p(probs))
    return (out, probs) if return_probs else out


def dwc(v: np.ndarray, wd: np.ndarray, grid_h: int, grid_w: int) -> np.ndarray:
    """DWC(V) of Eq. 6 for one slab.  v [N, d], wd [d, 3, 3] -> [N, d]."""
    v, wd = _c(v), _c(wd)
    d = v.shape[-1]
    assert v.shape == (grid_h * grid_w, d) and wd.shape == (d, 3, 3)
    out = np.zeros_like(v)
    _load().aa_oracle_dwc_add(_p(v), _p(wd), grid_h, grid_w, d, _p(out))
    return out


def forward(q, k, v, grid_h: int, grid_w: int, *, pool_hw: Optional[Tuple[int, int]] = None,
            agents=None, b1=None, b2=None, dwc_weight=None,
            scale1: Optional[float] = None, scale2: Optional[float] = None,
            threads: int = 1, return_intermediates: bool = False):
    """Eq. 6 over a batch.  q, k, v [B, heads, N, d]; returns O [B, heads, N, d] (fp64).

    Exactly one of `pool_hw` (agents pooled from Q on a ph x pw grid) and `agents`
    ([B, heads, n, d]) is given.  scale1/scale2 default to 1/sqrt(d) (Sec. 3.2).
    """
    q, k, v = _c(q), _c(k), _c(v)
    B, heads, N, d = q.shape
    assert N == grid_h * grid_w and k.shape == q.shape and v.shape == q.shape
    assert (pool_hw is None) != (agents is None)
    if agents is not None:
        agents = _c(agents)
        n = agents.shape[2]
        assert agents.shape == (B, heads, n, d)
        ph = pw = 0
    else:
        ph, pw = pool_hw
        n = ph * pw
    b1 = None if b1 is None else _c(b1)
    b2 = None if b2 is None else _c(b2)
    wd = None if dwc_weight is None else _c(dwc_weight)
    assert b1 is None or b1.shape == (heads, n, N)
    assert b2 is None or b2.shape == (heads, N, n)
    assert wd is None or wd.shape == (heads, d, 3, 3)
    s1 = d ** -0.5 if scale1 is None else float(scale1)
    s2 = d ** -0.5 if scale2 is None else float(scale2)
    o = np.empty_like(q)
    a_out = np.empty((B, heads, n, d), dtype=np.float64)
    va_out = np.empty((B, heads, n, d), dtype=np.float64)
    used = _load().aa_oracle_forward(_p(q), _p(k), _p(v), _p(agents), B, heads, grid_h, grid_w,
                                     d, n, ph, pw, _p(b1), _p(b2), _p(wd), s1, s2,
                                     _p(o), _p(a_out), _p(va_out), int(threads))
    if used < 0:
        raise ValueError("aa_oracle_forward rejected its arguments")
    forward.last_threads = used
    if return_intermediates:
        return o, a_out, va_out
    return o


forward.last_threads = 1


def backward(q, k, v, d_out, grid_h: int, grid_w: int, pool_hw: Tuple[int, int], b1=None, b2=None,
             dwc_weight=None, scale1: Optional[float] = None, scale2: Optional[float] = None):
    """Gradients of Eq. 6 with pooled agents for an upstream gradient d_out [B, heads, N, d].

    Returns a dict with dq, dk, dv [B, heads, N, d] and, for the inputs that were given, db1 [heads, n, N],
    db2 [heads, N, n], dwd [heads, d, 3, 3] (fp64).
    """
    q, k, v, g = _c(q), _c(k), _c(v), _c(d_out)
    B, heads, N, d = q.shape
    assert N == grid_h * grid_w and k.shape == q.shape and v.shape == q.shape and g.shape == q.shape
    ph, pw = pool_hw
    n = ph * pw
    b1 = None if b1 is None else _c(b1)
    b2 = None if b2 is None else _c(b2)
    wd = None if dwc_weight is None else _c(dwc_weight)
    assert b1 is None or b1.shape == (heads, n, N)
    assert b2 is None or b2.shape == (heads, N, n)
    assert wd is None or wd.shape == (heads, d, 3, 3)
    s1 = d ** -0.5 if scale1 is None else float(scale1)
    s2 = d ** -0.5 if scale2 is None else float(scale2)
    out = {"dq": np.empty_like(q), "dk": np.empty_like(q), "dv": np.empty_like(q)}
    if b1 is not None: out["db1"] = np.empty((heads, n, N), dtype=np.float64)
    if b2 is not None: out["db2"] = np.empty((heads, N, n), dtype=np.float64)
    if wd is not None: out["dwd"] = np.empty((heads, d, 3, 3), dtype=np.float64)
    rc = _load().aa_oracle_backward(_p(q), _p(k), _p(v), _p(g), B, heads, grid_h, grid_w, d, n, ph, pw,
                                    _p(b1), _p(b2), _p(wd), s1, s2, _p(out["dq"]), _p(out["dk"]), _p(out["dv"]),
                                    _p(out.get("db1")), _p(out.get("db2")), _p(out.get("dwd")))
    if rc != 0:
        raise ValueError("aa_oracle_backward rejected its arguments")
    return out


def explicit(q, a, k, v, b1=None, b2=None, scale1: Optional[float] = None,
             scale2: Optional[float] = None):
    """Eq. 4 for one tiny slab: returns (M [N, N], O [N, d]) with M = s(QA^T+B2) s(AK^T+B1)."""
    q, a, k, v = _c(q), _c(a), _c(k), _c(v)
    N, d = q.shape
    n = a.shape[0]
    b1 = None if b1 is None else _c(b1)
    b2 = None if b2 is None else _c(b2)
    s1 = d ** -0.5 if scale1 is None else float(scale1)
    s2 = d ** -0.5 if scale2 is None else float(scale2)
    m = np.empty((N, N), dtype=np.float64)
    o = np.empty((N, d), dtype=np.float64)
    _load().aa_oracle_explicit(_p(q), _p(a), _p(k), _p(v), _p(b1), _p(b2), N, n, d, s1, s2,
                               _p(m), _p(o))
    return m, o


def macs(N: int, C: int, n: int, k: int = 3):
    """Eq. 7 in multiply-accumulates: (total, [proj, agents, aggregation, broadcast, dwc])."""
    parts = (ctypes.c_longlong * 5)()
    total = _load().aa_oracle_macs(N, C, n, k, parts)
    return int(total), [int(x) for x in parts]


def compose_bias(col, row, blk, grid_h: int, grid_w: int, transpose: bool = False):
    """App. B for one head: col [n, w], row [n, h], blk [n, h0, w0] (any may be None) -> [n, N] or [N, n]."""
    parts = [x for x in (col, row, blk) if x is not None]
    assert parts, "at least one component is needed"
    n = parts[0].shape[0]
    col = None if col is None else _c(col)
    row = None if row is None else _c(row)
    blk = None if blk is None else _c(blk)
    assert col is None or col.shape == (n, grid_w)
    assert row is None or row.shape == (n, grid_h)
    h0, w0 = (blk.shape[1], blk.shape[2]) if blk is not None else (1, 1)
    N = grid_h * grid_w
    out = np.empty((N, n) if transpose else (n, N), dtype=np.float64)
    _load().aa_oracle_compose_bias(_p(col), _p(row), _p(blk), n, grid_h, grid_w, h0, w0, int(bool(transpose)), _p(out))
    return out
