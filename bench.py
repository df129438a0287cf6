#!/usr/bin/env python
"""Benchmark of the Agent Attention forward pass (one JSON line on stdout, printed by rank 0).

A step is one forward pass of the whole module (pool -> aggregation -> broadcast + DWC) over one
batch of synthetic input of the headline shape (N = 3136 tokens on a 56x56 grid, n = 49 agents,
d = 64, bf16, batch 64).  Inputs are resident in HBM before the timed region; the buffer sets
rotate so that no step finds its inputs in L2.  `--impl reference` times the fp64 CPU oracle on
the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2312_08874_b200 import WORKLOADS, make_inputs  # noqa: E402
from paper_2312_08874_b200 import dist as pdist  # noqa: E402
from paper_2312_08874_b200.workloads import TORCH_DTYPE  # noqa: E402

METRIC = "agent-attention fwd tokens/s and % of HBM roofline at N=3136,n=49,d=64"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "cfg3_pvt_bf16"
# dram__bytes_read.sum + dram__bytes_write.sum per forward pass of the streaming path (three launches), from the ncu
# capture summarised under profiles/, with the digest of the kernel sources it was taken from: the figure is
# reported only while those sources are unchanged
NCU_TRAFFIC = {"cfg3_pvt_bf16": {"bytes": 117.3e6, "sources_sha256": "59cc6ac0f570fe83"}}
TRAFFIC_SOURCES = ("stream_prep.cu", "stream_aggregate.cu", "stream_broadcast.cu", "stream_common.cuh")


def kernel_sources_digest() -> str:
    import hashlib
    h = hashlib.sha256()
    for f in TRAFFIC_SOURCES:
        with open(os.path.join(ROOT, "paper_2312_08874_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def traffic_of(name: str):
    t = NCU_TRAFFIC.get(name)
    if not t or t["bytes"] is None or t["sources_sha256"] != kernel_sources_digest():
        return None
    return t["bytes"]


def measured_peaks():
    """(HBM GB/s, sustained bf16 TFLOP/s, source) from the generated peaks file, else the machine's fallback figures."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            j = json.load(f)
        return float(j["hbm_gbs"]), float(j.get("bf16_tflops_sustained", 1400.0)), "measured"
    except Exception:
        return 6650.0, 1400.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while a region runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    bits = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    bits = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, nm in names.items():
                    if bits & bit:
                        self.reasons.add(nm)
            except Exception:
                pass
            time.sleep(0.002)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2.0)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def flops_of(w) -> int:
    """2 x the multiply-accumulates of Eq. 7 without the projections, per forward pass."""
    per_slab = 8 * w.tokens * w.agents * w.head_dim + w.tokens * w.head_dim
    if w.dwc:
        per_slab += 18 * w.tokens * w.head_dim
    return w.slabs * per_slab


def oracle_sample_run(w, inp_np, threads):
    from oracle import agent_attention_oracle as orc
    t0 = time.perf_counter()
    orc.forward(inp_np["q"], inp_np["k"], inp_np["v"], w.grid_h, w.grid_w, pool_hw=(w.pool, w.pool),
                b1=inp_np["b1"], b2=inp_np["b2"], dwc_weight=inp_np["dwc"], threads=threads)
    return time.perf_counter() - t0, orc.forward.last_threads


def oracle_inputs(w):
    inp = make_inputs(w)
    return {k: (None if v is None else v.double().numpy()) for k, v in inp.items()}


def oracle_baseline(w, passes: int, warmup: int):
    """The oracle as it stands on the host cores, the same way for the GPU arm's `cpu_baseline` and for
    `--impl reference`: one pass = the forward pass over a bounded sample of the workload (as many whole batch
    entries as there are host threads, one slab per thread); the value is sample tokens / mean pass time."""
    from oracle import agent_attention_oracle as orc
    threads = orc.max_threads()
    sample_batch = max(1, min(w.batch, threads // max(1, w.heads)))
    ws = w.scaled(batch=sample_batch)
    inp = oracle_inputs(ws)
    for _ in range(warmup):
        oracle_sample_run(ws, inp, threads)
    t0 = time.perf_counter()
    used = 1
    for _ in range(passes):
        _, used = oracle_sample_run(ws, inp, threads)
    total = time.perf_counter() - t0
    sample = f"{ws.batch} of {w.batch} batch entries ({ws.slabs} slabs) of {w.name} per pass, mean of {passes} passes"
    return {"value": passes * ws.batch * ws.tokens / total, "unit": UNIT, "cores": used, "kind": "oracle",
            "sample": sample, "ms_per_pass": 1e3 * total / passes}


def run_reference(args, w):
    """The oracle as it stands on the host cores; each step is one pass over a bounded sample."""
    rank, _, world = pdist.env_rank()
    if rank != 0:
        return
    base = oracle_baseline(w, passes=args.steps, warmup=min(args.warmup, 3))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": base["ms_per_pass"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "sample": base["sample"]},
        "cpu_baseline": {k: base[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def backward_flops(w) -> int:
    """Algorithmic flops of the backward pass: eleven n x N x d products per slab (S1, V_A, S2 recomputed;
    dV_A, dP2, dQ, dA (two terms), dP1, dK, dV), two flops per multiply-add, plus the two depthwise terms."""
    mm = 11 * 2 * w.slabs * w.agents * w.tokens * w.head_dim
    dw = 2 * 2 * 9 * w.slabs * w.tokens * w.head_dim if w.dwc else 0
    return mm + dw


def run_backward(args, w, mod, sets, rank, local_rank, world):
    """Times agent_attn_backward on device-resident inputs (two rotating sets, each larger than the L2)."""
    from paper_2312_08874_b200 import make_upstream_grad
    dev = torch.device("cuda", local_rank)
    go = make_upstream_grad(w, seed=w.seed + 1000 * rank).to(dev)
    ws = mod.backward_workspace(w.grid_h, w.grid_w, w.agents)
    stream = torch.cuda.current_stream()
    steps = min(args.steps, 200)

    def step(i):
        d = sets[i % len(sets)]
        return mod.backward(d["q"], d["k"], d["v"], go, w.grid_h, w.grid_w, w.agents, b1=d["b1"], b2=d["b2"],
                            dwc_weight=d["dwc"], workspace=ws, stream=stream)

    t_w = time.perf_counter()
    i = 0
    while i < args.warmup or time.perf_counter() - t_w < args.min_warmup_seconds:
        g = step(i)
        i += 1
        if i % 16 == 0:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    launches = mod.last_launch_count()
    sampler = ClockSampler(local_rank)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    pdist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    e0.record(stream)
    for i in range(steps):
        g = step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    pdist.barrier()
    clocks = sampler.stop()
    ms_step = pdist.max_over_ranks(e0.elapsed_time(e1)) / steps
    tokens_per_step = world * w.batch * w.tokens
    # fp32 multiply-add peak of the CUDA cores: SMs x 128 lanes x 2 flops x the SM clock seen under load
    props = torch.cuda.get_device_properties(dev)
    mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965
    peak = props.multi_processor_count * 128 * 2 * mhz * 1e6 / 1e12
    tfl = backward_flops(w) / (ms_step * 1e-3) / 1e12
    set_bytes = sum(t.numel() * t.element_size() for t in list(sets[0].values()) + list(g.values()) + [go]
                    if t is not None) - sets[0]["out"].numel() * sets[0]["out"].element_size()
    hbm_peak, _, peak_src = measured_peaks()
    gbs = set_bytes / (ms_step * 1e-3) / 1e9
    tensor_path = w.dtype in ("bf16", "f16") and w.agents <= 64 and w.head_dim == 64
    if tensor_path:
        # tensor-core kernels: 14 GFLOP per step is microseconds of tensor time, the bytes touched bound the pass
        roofline = {"bound": "hbm", "kernel": "backward_path", "achieved": gbs, "peak": hbm_peak, "unit": "GB/s",
                    "frac": gbs / hbm_peak, "traffic": None, "peak_source": peak_src,
                    "algorithmic_bytes": set_bytes, "algorithmic_flops": backward_flops(w), "tflops": tfl}
    else:
        roofline = {"bound": "alu", "kernel": "backward_path", "achieved": tfl, "peak": peak, "unit": "TFLOP/s",
                    "frac": tfl / peak, "traffic": None,
                    "peak_source": "SMs x 128 fp32 lanes x 2 x sampled SM clock",
                    "algorithmic_flops": backward_flops(w), "algorithmic_bytes": set_bytes,
                    "hbm_frac_if_bandwidth_bound": gbs / hbm_peak}
    if rank == 0:
        print(json.dumps({
            "pass": "backward", "metric": "backward tokens/s", "value": tokens_per_step / (ms_step * 1e-3),
            "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": args.warmup, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": w.dtype if tensor_path else "f32", "data": "synthetic",
            "config": {"workload": w.name, "batch_per_gpu": w.batch, "heads": w.heads, "tokens": w.tokens,
                       "head_dim": w.head_dim, "agents": w.agents, "bias": w.bias, "dwc": w.dwc,
                       "gradients": sorted(g), "l2": f"2 rotating input sets, {set_bytes / 1e6:.1f} MB touched per step"},
            "clocks": clocks, "gpu_launches": launches * steps,
            "roofline": roofline,
        }))


def make_sets(w, dev, n_sets, rank, layout="dense"):
    """`n_sets` device-resident buffer sets of the workload (distinct contents, same distribution)."""
    dt = TORCH_DTYPE[w.dtype]
    host = make_inputs(w, seed=w.seed + 1000 * rank)
    sets = []
    for s in range(n_sets):
        g = torch.Generator(device="cpu").manual_seed(17 + s)
        roll = int(torch.randint(1, w.tokens, (1,), generator=g))
        d = {k: (None if v is None else v.to(dev)) for k, v in host.items()}
        if s:  # a roll along the token axis
            for k in ("q", "k", "v"):
                d[k] = torch.roll(d[k], roll, dims=2).contiguous()
        d["out"] = torch.empty_like(d["q"])
        if layout != "dense":      # the same values behind token-major storage; views keep the [B,h,N,d] shape
            if layout == "qkv":
                packed = torch.stack([d[k].permute(0, 2, 1, 3) for k in ("q", "k", "v")], dim=2).contiguous()
                for j, k in enumerate(("q", "k", "v")):
                    d[k] = packed[:, :, j].permute(0, 2, 1, 3)
            else:
                for k in ("q", "k", "v"):
                    d[k] = d[k].permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
            d["out"] = torch.empty((w.batch, w.tokens, w.heads, w.head_dim), dtype=dt, device=dev).permute(0, 2, 1, 3)
        sets.append(d)
    return host, sets


def n_sets_for(w, l2_bytes):
    """Rotating buffer sets: together more than 4x the L2, so no step re-reads a resident set."""
    return max(2, -(-4 * l2_bytes // w.algorithmic_bytes()))


def time_forward(mod, w, sets, ws, stream, steps, repeats, layout="dense", min_seconds=0.0, max_repeats=400):
    """`repeats` timed regions of exactly `steps` forward calls each, between CUDA events on the launching stream
    (more repeats until `min_seconds` of device time are covered).  Returns the per-step times in ms, one per repeat."""
    fwd = mod.forward if layout == "dense" else mod.forward_strided

    def step(i):
        d = sets[i % len(sets)]
        fwd(d["q"], d["k"], d["v"], w.grid_h, w.grid_w, w.agents, b1=d["b1"], b2=d["b2"],
            dwc_weight=d["dwc"], out=d["out"], workspace=ws, stream=stream)

    times, i, spent = [], 0, 0.0
    while len(times) < repeats or (spent < min_seconds and len(times) < max_repeats):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            step(i)
            i += 1
        e1.record(stream)
        e1.synchronize()
        ms = e0.elapsed_time(e1)
        times.append(ms / steps)
        spent += ms * 1e-3
    return times


def bound_of(w, ms_step, hbm_peak, tensor_peak):
    """Slower of (algorithmic bytes at the HBM peak) and (algorithmic flops at the sustained bf16 tensor peak)."""
    t_hbm = w.algorithmic_bytes() / (hbm_peak * 1e9)
    t_tensor = flops_of(w) / (tensor_peak * 1e12)
    t_bound = max(t_hbm, t_tensor)
    return {"bound": "hbm" if t_hbm >= t_tensor else "tensor", "t_hbm_us": 1e6 * t_hbm, "t_tensor_us": 1e6 * t_tensor,
            "frac": t_bound / (ms_step * 1e-3)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--repeats", type=int, default=5, help="timed regions of --steps forwards each (median reported)")
    ap.add_argument("--min-seconds", type=float, default=0.5, help="keep repeating until this much device time is covered")
    ap.add_argument("--layout", choices=["dense", "bnhd", "qkv"], default="dense",
                    help="storage of Q, K, V and out: dense [B,h,N,d]; bnhd = [B,N,h,d] (forward_strided); "
                         "qkv = Q, K, V interleaved as [B,N,3,h,d], out [B,N,h,d] (forward_strided)")
    ap.add_argument("--direction", choices=["forward", "backward"], default="forward",
                    help="backward: time agent_attn_backward (fp32 gradients of Q, K, V, both biases and the filter) "
                         "instead of the forward pass; prints a line with \"pass\": \"backward\"")
    ap.add_argument("--path", choices=["auto", "queue", "unfused", "simt"], default="auto",
                    help="kernel family: auto (the library's choice), queue (the persistent task-queue kernel wherever it "
                         "applies), unfused (one kernel per step), simt (fp32 FMA kernels)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--no-kernel-split", action="store_true",
                    help="skip the per-kernel timing of the streaming path (for short runs under a profiler)")
    ap.add_argument("--min-warmup-seconds", type=float, default=0.2)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    w = WORKLOADS[args.workload]

    if args.impl == "reference":
        run_reference(args, w)
        return

    from paper_2312_08874_b200 import AgentAttention
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the forward pass has no CPU path")
    rank, local_rank, world = pdist.init()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dt = TORCH_DTYPE[w.dtype]
    l2_bytes = int(torch.cuda.get_device_properties(dev).L2_cache_size)     # cudaDevAttrL2CacheSize

    set_bytes = w.algorithmic_bytes()
    n_sets = n_sets_for(w, l2_bytes)
    host, sets = make_sets(w, dev, n_sets, rank, args.layout)
    path = {"auto": 0, "simt": 1, "unfused": 2, "queue": 3}[args.path]
    mod = AgentAttention(w.batch, w.heads, w.head_dim, w.tokens, w.agents, dt, device=local_rank, path=path)
    ws = mod.workspace(w.grid_h, w.grid_w, w.agents)
    stream = torch.cuda.current_stream()
    if args.direction == "backward":
        if args.layout != "dense":
            raise SystemExit("the backward pass takes dense tensors")
        run_backward(args, w, mod, sets[:2], rank, local_rank, world)
        pdist.shutdown()
        return

    # warm-up: W steps, and at least 0.2 s so that clocks have ramped
    t_w = time.perf_counter()
    done = 0
    while done < args.warmup or time.perf_counter() - t_w < args.min_warmup_seconds:
        time_forward(mod, w, sets, ws, stream, 16, 1, args.layout)
        done += 16
    torch.cuda.synchronize()
    launches_per_step = mod.last_launch_count()

    # the timed region: `repeats` x exactly `steps` forward calls, device time by CUDA events, max over ranks
    sampler = ClockSampler(local_rank)
    pdist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    times = time_forward(mod, w, sets, ws, stream, args.steps, args.repeats, args.layout, args.min_seconds)
    torch.cuda.synchronize()
    pdist.barrier()
    clocks = sampler.stop()
    if mod.query_status() != 0:
        raise SystemExit("a device-side bounded wait expired during the timed region: the timing is void")
    ms_step = pdist.max_over_ranks(statistics.median(times))
    ms_min = pdist.max_over_ranks(min(times))
    tokens_per_step = world * w.batch * w.tokens
    value = tokens_per_step / (ms_step * 1e-3)

    s = w.elem_bytes
    unit = w.slabs * w.tokens * w.head_dim * s                       # one [B,h,N,d] tensor
    bias_b = w.heads * w.agents * w.tokens * s if w.bias else 0
    wd_b = 9 * w.heads * w.head_dim * s if w.dwc else 0
    peak, tensor_peak, peak_src = measured_peaks()
    kb_steps = min(args.steps, 200)
    kern_note = None
    if launches_per_step == 3 and args.layout == "dense" and not args.no_kernel_split:
        # three streaming kernels per forward call: each timed by itself between events through the stage mask
        # (a later stage alone reads what the last full call left in the workspace)
        names = ("prep", "aggregate", "broadcast_dwc")
        kern_ms = {}
        for bit, nm in enumerate(names):
            mod.set_stage_mask(1 << bit)
            time_forward(mod, w, sets, ws, stream, 8, 1)
            kern_ms[nm] = statistics.median(time_forward(mod, w, sets, ws, stream, kb_steps, 3))
        mod.set_stage_mask(7)
        # what each kernel itself has to touch (the second reads of Q and V are meant to come from L2)
        kern_bytes = {"prep": unit + 2 * bias_b + wd_b, "aggregate": 2 * unit + bias_b,
                      "broadcast_dwc": 3 * unit + bias_b + wd_b}
        kern_note = ("kernel_ms: each kernel launched alone, back to back with itself (so without the overlap that "
                     "programmatic dependent launch gives the path); kernel_algorithmic_bytes counts what a kernel "
                     "touches, second reads of Q and V included, so it sums to more than the path's bytes")
        dominant = "forward_path"
    elif launches_per_step in (1, 3) or args.layout != "dense":
        dominant = "fused_kernel" if launches_per_step == 1 else "forward_path"
        kern_ms = {dominant: ms_step}
        kern_bytes = {dominant: set_bytes}
    else:
        # one kernel per step of the path: time each between events on the launching stream, through the
        # step-level entry points
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(kb_steps)]
        a_buf = torch.empty((w.batch, w.heads, w.agents, w.head_dim), dtype=dt, device=dev)
        va_buf = torch.empty_like(a_buf)
        torch.cuda.synchronize()
        for i in range(kb_steps):
            d = sets[i % n_sets]
            evs[i][0].record(stream)
            mod.pool(d["q"], w.grid_h, w.grid_w, w.pool, w.pool, out=a_buf, stream=stream)
            evs[i][1].record(stream)
            mod.aggregate(a_buf, d["k"], d["v"], b1=d["b1"], out=va_buf, workspace=ws, stream=stream)
            evs[i][2].record(stream)
            mod.broadcast(d["q"], a_buf, va_buf, d["v"], w.grid_h, w.grid_w, b2=d["b2"], dwc_weight=d["dwc"],
                          out=d["out"], stream=stream)
            evs[i][3].record(stream)
        torch.cuda.synchronize()
        kern_ms = {nm: statistics.mean(evs[i][j].elapsed_time(evs[i][j + 1]) for i in range(kb_steps))
                   for j, nm in enumerate(("pool", "aggregate", "broadcast_dwc"))}
        kern_bytes = {"pool": unit, "aggregate": 2 * unit + bias_b, "broadcast_dwc": unit + bias_b + wd_b}
        dominant = max(kern_ms, key=kern_ms.get)
    path_gbs = set_bytes / (ms_step * 1e-3) / 1e9
    if dominant == "forward_path":
        dom_gbs, dom_ms, dom_bytes = path_gbs, ms_step, set_bytes
    else:
        dom_ms, dom_bytes = kern_ms[dominant], kern_bytes[dominant]
        dom_gbs = dom_bytes / (dom_ms * 1e-3) / 1e9
    roofline = {
        "bound": "hbm", "kernel": dominant, "achieved": dom_gbs, "peak": peak, "unit": "GB/s",
        "frac": dom_gbs / peak, "traffic": traffic_of(w.name) if launches_per_step == 3 else None, "peak_source": peak_src,
        "launches_per_step": launches_per_step,
        "kernel_ms": kern_ms, "kernel_algorithmic_bytes": kern_bytes,
        "kernel_frac": {k: kern_bytes[k] / (kern_ms[k] * 1e-3) / 1e9 / peak for k in kern_ms},
        "path_achieved": path_gbs, "path_frac": path_gbs / peak, "path_frac_nominal_8TBs": path_gbs / 8000.0,
        "path_algorithmic_bytes": set_bytes, "path_tflops": flops_of(w) / (ms_step * 1e-3) / 1e12,
    }
    if kern_note:
        roofline["note"] = kern_note

    # the other configurations, briefly (same protocol, fewer repeats): tokens/s against N for the high-resolution pair
    configs = None
    if not args.no_configs and world == 1 and args.layout == "dense":
        configs = [{"workload": w.name, "tokens": w.tokens, "agents": w.agents, "dtype": w.dtype, "ms_per_step": ms_step,
                    "tokens_per_s": value, "algorithmic_bytes": set_bytes, **bound_of(w, ms_step, peak, tensor_peak)}]
        del sets
        torch.cuda.empty_cache()
        for name in ("cfg2_deit_bf16", "cfg4_sd_f16", "cfg5a_hires_bf16", "cfg5b_hires_bf16"):
            if name == w.name:
                continue
            wc = WORKLOADS[name]
            _, sc = make_sets(wc, dev, n_sets_for(wc, l2_bytes), rank)
            mc = AgentAttention(wc.batch, wc.heads, wc.head_dim, wc.tokens, wc.agents, TORCH_DTYPE[wc.dtype], device=local_rank)
            wsc = mc.workspace(wc.grid_h, wc.grid_w, wc.agents)
            time_forward(mc, wc, sc, wsc, stream, 20, 1)
            est = statistics.median(time_forward(mc, wc, sc, wsc, stream, 10, 2))
            k = max(10, min(200, int(0.05 / (est * 1e-3))))
            tc = time_forward(mc, wc, sc, wsc, stream, k, 3)
            if mc.query_status() != 0:
                raise SystemExit(f"a device-side bounded wait expired on {name}")
            msc = statistics.median(tc)
            configs.append({"workload": name, "tokens": wc.tokens, "agents": wc.agents, "dtype": wc.dtype, "ms_per_step": msc,
                            "ms_per_step_min": min(tc), "steps": k, "repeats": 3, "launches_per_step": mc.last_launch_count(),
                            "tokens_per_s": wc.batch * wc.tokens / (msc * 1e-3), "algorithmic_bytes": wc.algorithmic_bytes(),
                            **bound_of(wc, msc, peak, tensor_peak)})
            del sc, mc, wsc
            torch.cuda.empty_cache()
        _, sets = make_sets(w, dev, 2, rank)          # (the end-to-end leg below needs no device sets)

    # end to end through the host-buffer entry point: pinned inputs in, result out, every step
    e2e = None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.e2e_steps > 0:
        pin = {k: (None if v is None else v.pin_memory()) for k, v in host.items()}
        out_h = torch.empty_like(pin["q"]).pin_memory()
        for _ in range(2):
            mod.forward_host(pin["q"], pin["k"], pin["v"], w.grid_h, w.grid_w, w.agents, b1=pin["b1"],
                             b2=pin["b2"], dwc_weight=pin["dwc"], out=out_h, stream=stream)
        # two calls in flight on two streams, each with its own staging and result buffer: the copy back of one
        # step overlaps the copy in of the next (the copies of a step itself stay in order on its stream)
        need = mod.staging_bytes(w.grid_h, w.grid_w, w.agents)
        lanes = [(torch.cuda.Stream(device=dev), torch.empty(need, dtype=torch.uint8, device=dev),
                  torch.empty_like(pin["q"]).pin_memory()) for _ in range(2)]
        pdist.barrier()
        torch.cuda.synchronize()
        e0.record(stream)
        for st, _, _ in lanes:
            st.wait_stream(stream)
        for i in range(args.e2e_steps):
            st, stg, oh = lanes[i & 1]
            mod.forward_host(pin["q"], pin["k"], pin["v"], w.grid_h, w.grid_w, w.agents, b1=pin["b1"],
                             b2=pin["b2"], dwc_weight=pin["dwc"], out=oh, stream=st, synchronize=False, staging=stg)
        for st, _, _ in lanes:
            stream.wait_stream(st)
        e1.record(stream)
        torch.cuda.synchronize()
        if mod.query_status() != 0:
            raise SystemExit("a device-side bounded wait expired during the end-to-end region")
        ms_e2e = pdist.max_over_ranks(e0.elapsed_time(e1)) / args.e2e_steps
        h2d = sum(v.numel() * v.element_size() for v in pin.values() if v is not None)
        e2e = {"value": tokens_per_step / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": out_h.numel() * out_h.element_size(), "ms_per_step": ms_e2e,
               "steps": args.e2e_steps, "streams": 2}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        base = oracle_baseline(w, passes=3, warmup=1)
        cpu_baseline = {k: base[k] for k in ("value", "unit", "cores", "kind", "sample")}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "ms_per_step_min": ms_min, "repeats": len(times),
            "timed_steps_total": len(times) * args.steps,
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": w.name, "batch_per_gpu": w.batch, "heads": w.heads, "tokens": w.tokens,
                       "grid": [w.grid_h, w.grid_w], "head_dim": w.head_dim, "agents": w.agents,
                       "bias": w.bias, "dwc": w.dwc, "layout": args.layout, "path": args.path,
                       "l2": f"{n_sets} rotating buffer sets of {set_bytes / 1e6:.1f} MB (> 4x the {l2_bytes / 2**20:.0f} MiB L2)",
                       "timing": f"median of {len(times)} regions of {args.steps} forward calls each, CUDA events",
                       "parallelism": f"batch-sharded x{world}, no collective"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * len(times) * args.steps,
            "roofline": roofline, "configs": configs, "cpu_baseline": cpu_baseline,
        }))
    pdist.shutdown()


if __name__ == "__main__":
    main()
