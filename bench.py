#!/usr/bin/env python
"""Benchmark of the 3D-DSA library: forward + backward Mtokens/s on synthetic latent video.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one forward plus one backward over one video of the workload (default: the
1080p x 256-frame bf16 configuration).  With N > 1 (launched by torch.distributed.run,
one rank per GPU) every rank processes its own video of a batch of N: videos are
independent, there is no collective on the data path, and the result is weak scaling.

The printed JSON line carries: `value` (Mtokens/s with the inputs resident in HBM, CUDA
events on the launching stream, max over ranks), `e2e` (the same through dsa3d_step_host
with pinned HOST buffers, copies inside the timed region), `roofline` (algorithmic bytes
of the dominant kernel / its event-timed duration, against the measured HBM copy rate),
`cpu_baseline` (the CPU oracle timed on a bounded sample, rank 0, N = 1 only), `clocks`
(nvidia-smi samples taken during the timed region) and `gpu_launches`.

`--impl reference` times the CPU oracle alone on the host cores on bounded samples of the
same workload and prints the same kind of line with "impl": "reference".
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2607_22696_b200 import inputs

METRIC = "3D-DSA fwd+bwd Mtokens/s at 1080p\u00d7256f (bf16); achieved HBM GB/s vs peak"
UNIT = "Mtokens/s"
FALLBACK_HBM_GBS = 6650.0

# Counters of one ncu capture per kernel on the small profiling workload (profile_small_bf16: a
# 3 GB cut of the default workload, d = 128, window 3x3x3), per (token, head) item:
#   dram    dram__bytes_read.sum + dram__bytes_write.sum
#   l2_sm   l1tex__m_xbar2l1tex_read_bytes.sum (what the corner gathers pull through the L2-to-SM
#           port after L1 hits; the algorithmic figure P*8*2*d*elt is computed live below)
#   inst    smsp__inst_executed.sum (warp instructions)
# Each entry names the kernel's source files and their SHA-256 (first 12 hex digits of the
# digest over the files in that order) at the time of the capture; when the sources on disk
# differ, every figure derived from the entry is printed with "stale": true.  A launch on another
# workload with the same d and window is reported as items x these figures, which understates the
# DRAM traffic of grids whose K/V and accumulators no longer fit the 126 MB L2 (a one-off capture
# at 1080p gave 1.7x / 1.6x / 1.8x the small case's bytes per item for the three kernels).
NCU_PER_ITEM = {
    "forward_kernel": {"dram": 1525.0, "l2_sm": 83815.0, "inst": 5509.0,
                       "sources": ["dsa3d_forward.cu", "dsa3d_common.cuh"], "sha": "a335f85dc533"},
    "backward_kernel": {"dram": 3003.0, "l2_sm": 92009.0, "inst": 5901.0,
                        "sources": ["dsa3d_backward.cu", "dsa3d_common.cuh"], "sha": "ac74993402dc"},
    "scatter_tile_kernel": {"dram": 13000.0, "inst": 5980.0,
                            "sources": ["dsa3d_backward.cu", "dsa3d_common.cuh"], "sha": "ac74993402dc"},
}


def source_sha(files) -> str:
    import hashlib
    h = hashlib.sha256()
    for name in files:
        with open(os.path.join(ROOT, "paper_2607_22696_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:12]


def ncu_figures(kernel: str):
    """The recorded per-item counters of `kernel` and whether its sources changed since."""
    rec = NCU_PER_ITEM[kernel]
    try:
        stale = source_sha(rec["sources"]) != rec["sha"]
    except OSError:
        stale = True
    return rec, stale


def launches_per_step(wl, fixed_window: bool, bounded: bool, tiled: bool) -> int:
    """Kernels of the library launched by one forward (+ backward) of the workload."""
    tensor_shape = wl.dtype == torch.bfloat16 and wl.d in (64, 128)
    if fixed_window:
        if not wl.backward:
            return 1
        # forward; then tables + per-query kernel + tile sums, or (shapes the table kernel does not cover)
        # per-query kernel + per-key kernel
        return 4 if tensor_shape and tuple(wl.window) in ((2, 2, 2), (3, 3, 3), (3, 5, 5), (3, 7, 7)) else 3
    if bounded and tensor_shape and tuple(wl.window) == (3, 3, 3):
        # forward: offsets check, tile kernel, general kernel (gated off); backward: offsets check, tables,
        # per-sample kernel, plane products, then gated off: accumulator clear, gather, tile scatter, two conversions
        return 3 + (9 if wl.backward else 0)
    if not wl.backward:
        return 1
    if wl.dtype == torch.bfloat16:
        return 5 if tiled else 4            # forward, gather, (tile scatter,) two conversions
    return 2


def tile_geometry(wl):
    """Tiles and key rows per tile of the dK/dV pre-reduction as the library lays them out
    (4 x 8 x 8 queries, halo 6, unless DSA3D_TILE overrides it)."""
    tt, ty, tx, halo = 4, 8, 8, 6
    env = os.environ.get("DSA3D_TILE", "")
    parts = env.split(",") if env else []
    if len(parts) == 4:
        try:
            tt, ty, tx, halo = (int(x) for x in parts)
        except ValueError:
            pass
    tiles = -(-wl.T // tt) * -(-wl.H // ty) * -(-wl.W // tx) * wl.heads
    rows = (tt + 2 * halo) * (ty + 2 * halo) * (tx + 2 * halo)
    return tiles, rows


def measure_ceilings(dev):
    """On-chip ceilings of this GPU, measured now with the library's probe kernels."""
    from paper_2607_22696_b200 import binding
    buf = torch.zeros(48 << 20, dtype=torch.uint8, device=dev)        # well inside the 126 MB L2
    out = {"l2_row_gather_gbs": binding.dsa3d_probe_gather(buf, buf.numel()),
           "l2_red_v4_f32_gbs": binding.dsa3d_probe_red(buf, buf.numel()),
           "fma_f32_tfma": binding.dsa3d_probe_fma(buf, 0),
           "fma_bf16_mixed_tfma": binding.dsa3d_probe_fma(buf, 1),
           "working_set_mb": 48}
    del buf
    return out


# ----------------------------------------------------------------------------- utilities

def metric_name(wl) -> str:
    """BASELINE's metric for its own workload; the same quantity named by workload otherwise."""
    if wl.name == "1080p_256f_bf16":
        return METRIC
    kind = "fwd+bwd" if wl.backward else "fwd"
    return f"3D-DSA {kind} Mtokens/s on {wl.name}; achieved HBM GB/s vs peak"


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json)"


class ClockSampler:
    """nvidia-smi samples every 200 ms while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200", "-i", str(gpu_index)], stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), power_w_max=max(power),
                       reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------- CPU oracle sampling

def oracle_sample(wl, rows: int, device_for_generation, frames: int = 1):
    """A bounded, exact sample of the workload for the CPU oracle: the first `rows` grid rows
    of `frames` consecutive frames from the middle one on as queries, evaluated on the crop of
    frames that their samples can reach (exact, because no sample leaves the crop: |offset_t|
    is bounded by the largest offset actually drawn for these queries).  Returns the cropped
    problem as CPU tensors."""
    tq = wl.T // 2
    rows = max(1, min(rows, wl.H))
    nf = max(1, min(frames, wl.T - tq))
    off_q = inputs.make_offsets(wl, device_for_generation, frames=(tq, tq + nf))[:, :rows].contiguous()
    finite = off_q[torch.isfinite(off_q)]
    reach = int(math.floor(2 + wl.window[0] // 2 + (float(finite.abs().max()) if finite.numel() else 0.0)))
    t0, t1 = max(0, tq - reach), min(wl.T, tq + nf - 1 + reach + 1)
    k = inputs.make_rows(wl, "k", device_for_generation, frames=(t0, t1)).cpu()
    v = inputs.make_rows(wl, "v", device_for_generation, frames=(t0, t1)).cpu()
    q = inputs.make_rows(wl, "q", device_for_generation, frames=(tq, tq + nf))[:, :rows].contiguous().cpu()
    dout = inputs.make_rows(wl, "dout", device_for_generation, frames=(tq, tq + nf))[:, :rows].contiguous().cpu()
    Tc = t1 - t0
    qtok = torch.cat([((tq + f - t0) * wl.H * wl.W + torch.arange(rows * wl.W)) for f in range(nf)]).to(torch.int64)
    return dict(q=q.view(-1, wl.heads, wl.d), k=k, v=v, offsets=off_q.cpu().view(-1, wl.heads, wl.P, 3),
                dout=dout.view(-1, wl.heads, wl.d), qtok=qtok, dims=(Tc, wl.H, wl.W, wl.heads, wl.d),
                tokens=nf * rows * wl.W,
                desc=f"{rows} grid rows of each of {nf} frame(s) from frame {tq} on ({nf * rows * wl.W} query tokens, "
                     f"all {wl.heads} heads), {'fwd+bwd incl. dK/dV' if wl.backward else 'forward only'}, on the exact "
                     f"{Tc}-frame crop their samples reach")


def time_oracle(sample, wl, backward=True):
    import oracle
    T, H, W, heads, d = sample["dims"]
    t0 = time.perf_counter()
    oracle.forward(sample["q"], sample["k"], sample["v"], sample["offsets"], T, H, W, heads, d, wl.window,
                   qtok=sample["qtok"])
    threads = oracle.last_threads()
    if backward:
        oracle.backward(sample["q"], sample["k"], sample["v"], sample["offsets"], sample["dout"], T, H, W,
                        heads, d, wl.window, qtok=sample["qtok"])
    return time.perf_counter() - t0, threads


def run_reference(args, wl):
    """The CPU oracle as it stands, on the host cores, on bounded samples of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
    probe = oracle_sample(wl, 1, gen_dev)
    dt, _ = time_oracle(probe, wl, wl.backward)                       # sizes the sample; not reported
    per_row = max(dt, 1e-3)
    target = min(4.0, 150.0 / max(1, args.steps + args.warmup))
    rows = max(1, min(wl.H, int(target / per_row)))
    sample = oracle_sample(wl, rows, gen_dev)
    for _ in range(args.warmup):
        time_oracle(sample, wl, wl.backward)
    times, threads = [], 1
    for _ in range(args.steps):
        dt, threads = time_oracle(sample, wl, wl.backward)
        times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = sample["tokens"] / (ms * 1e-3) / 1e6
    line = {
        "impl": "reference", "metric": metric_name(wl), "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "grid": [wl.T, wl.H, wl.W], "heads": wl.heads, "d": wl.d,
                   "window": list(wl.window), "storage": str(wl.dtype).replace("torch.", ""),
                   "offsets": f"{wl.offsets} sigma={wl.sigma}", "step": "one bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": sample["desc"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------- multi-rank plumbing

def rank_workload(wl, rank: int):
    """The video rank `rank` processes: the same shape for every rank (weak scaling), its own
    seed, so that no two ranks hold the same data.  Videos are independent, so there is no
    collective on the data path; ranks only meet in the timing barrier and the max below."""
    return wl if rank == 0 else inputs.dataclasses.replace(wl, seed=wl.seed + 1000 * rank)


def max_over_ranks(x: float, world: int, device=None) -> float:
    """Largest value of `x` over the ranks of the default process group (x itself when
    there is one rank)."""
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_mtokens_per_s(wl, world: int, step_ms: float) -> float:
    """Whole-job throughput: every rank processed one video of wl.N tokens in step_ms."""
    return wl.N * world / (step_ms * 1e-3) / 1e6


# ------------------------------------------------------------------------------ GPU arm

def measure_producer(wl, dev, reps: int = 5):
    """Times the layers around the operator (Eq. 1 first term and the offset predictor) on the
    workload's grid with hidden size heads*d: two 3x3x3 depthwise convolutions, the
    offset-producing linear layer on the tensor cores, and the forward with the convolution
    term added.  Buffers are freed before the main measurement allocates its own."""
    from paper_2607_22696_b200 import binding
    T, H, W, heads, d = wl.T, wl.H, wl.W, wl.heads, wl.d
    C, O, N = heads * d, heads * wl.P * 3, wl.N
    x = inputs.normal((T, H, W, C), wl.seed, 20, 1.0, wl.dtype, dev)
    wc = inputs.normal((27, C), wl.seed, 21, 0.2, torch.float32, dev)
    wlin = inputs.normal((O, C), wl.seed, 22, wl.sigma / math.sqrt(C), wl.dtype, dev)
    blin = inputs.normal((O,), wl.seed, 23, 0.1, torch.float32, dev)
    u = torch.empty_like(x)
    off = torch.empty((N, O), dtype=torch.float32, device=dev)

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) / reps

    conv_ms = timed(lambda: binding.dsa3d_dwconv3d_forward(x, wc, None, T, H, W, C, (3, 3, 3), u))
    gemm_ms = timed(lambda: binding.dsa3d_offsets_linear_forward(u, wlin, blin, N, C, O, off))
    # backward of both layers: dy of the convolution = the activations themselves (any tensor of
    # that shape and dtype does), doffsets of the linear layer = the offsets it just produced
    dxc = torch.empty_like(x)
    dwc = torch.empty((27, C), dtype=torch.float32, device=dev)
    dbc = torch.empty((C,), dtype=torch.float32, device=dev)
    wsc = torch.empty(binding.dsa3d_dwconv3d_backward_workspace_bytes(C, (3, 3, 3)), dtype=torch.uint8, device=dev)
    conv_dx_ms = timed(lambda: binding.dsa3d_dwconv3d_backward(None, wc, u, T, H, W, C, (3, 3, 3), dxc, None, None, wsc))
    conv_dw_ms = timed(lambda: binding.dsa3d_dwconv3d_backward(x, None, u, T, H, W, C, (3, 3, 3), None, dwc, dbc, None))
    del dxc, wsc
    du = torch.empty_like(u)
    dwl = torch.empty((O, C), dtype=torch.float32, device=dev)
    dbl = torch.empty((O,), dtype=torch.float32, device=dev)
    wsl = torch.empty(binding.dsa3d_offsets_linear_backward_workspace_bytes(N, C, O, wl.dtype), dtype=torch.uint8,
                      device=dev)
    lin_du_ms = timed(lambda: binding.dsa3d_offsets_linear_backward(None, wlin, off, N, C, O, du, None, None, wsl))
    lin_dw_ms = timed(lambda: binding.dsa3d_offsets_linear_backward(u, None, off, N, C, O, None, dwl, dbl, wsl))
    del du, dwl, dbl, wsl
    flag = binding.dsa3d_device_timeout_flag()
    elt = wl.elt
    peaks = {}
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            peaks = json.load(f)
    except (OSError, ValueError):
        pass
    tf_peak = float(peaks.get("bf16_tflops", 1590.0))
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    gemm_tf = 2.0 * N * C * O / (gemm_ms * 1e-3) / 1e12
    conv_gbs = 2.0 * N * C * elt / (conv_ms * 1e-3) / 1e9
    res = {"hidden": C, "offset_outputs": O, "timeout_flag": flag,
           "dwconv3d_3x3x3": {"ms": conv_ms, "bound": "hbm", "achieved": conv_gbs, "peak": hbm_peak, "unit": "GB/s",
                              "frac": conv_gbs / hbm_peak, "algorithmic_bytes": 2.0 * N * C * elt},
           "offsets_linear": {"ms": gemm_ms, "bound": "tensor", "achieved": gemm_tf, "peak": tf_peak,
                              "unit": "TFLOP/s", "frac": gemm_tf / tf_peak, "dtype": "bf16 x bf16 -> f32",
                              "peak_source": "measured burst (MEASURED_PEAKS.json bf16_tflops)" if peaks else "fallback"},
           "per_layer_ms": 2 * conv_ms + gemm_ms,
           "backward": {"dwconv3d_dx_ms": conv_dx_ms, "dwconv3d_dweight_dbias_ms": conv_dw_ms,
                        "offsets_linear_du_ms": lin_du_ms, "offsets_linear_dw_dbias_ms": lin_dw_ms,
                        "offsets_linear_tflops": {"du": 2.0 * N * C * O / (lin_du_ms * 1e-3) / 1e12,
                                                  "dw": 2.0 * N * C * O / (lin_dw_ms * 1e-3) / 1e12},
                        "note": "linear-layer times include the bf16 conversion and transposes of doffsets and u"}}
    del x, wc, wlin, blin, u, off
    torch.cuda.empty_cache()
    return res


def run_ours(args, wl):
    from paper_2607_22696_b200 import binding
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the operator has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()

    def max_ranks(x: float) -> float:
        return max_over_ranks(x, world, dev)

    binding.load()
    # --shard heads: ONE video over all ranks, rank r taking heads [r*h/G, (r+1)*h/G) of every
    # token (no exchange inside the operator: heads are independent) - strong scaling.  Default:
    # every rank its own video - weak scaling.
    sharded = args.shard == "heads" and world > 1
    if sharded:
        from paper_2607_22696_b200 import sharding
        lo, hi = sharding.head_range(wl.heads, world, rank)
        if hi == lo:
            raise RuntimeError("more ranks than heads")
        wl = inputs.dataclasses.replace(wl, heads=hi - lo)
    videos = 1 if sharded else world
    dims = (wl.T, wl.H, wl.W, wl.heads, wl.d)
    producer = None
    if args.producer and rank == 0 and wl.dtype == torch.bfloat16:
        producer = measure_producer(wl, dev)
    barrier()
    # every rank takes its own video of the batch: same shape, its own seed
    wl_rank = rank_workload(wl, rank)
    t = inputs.make_inputs(wl_rank, dev, with_dout=True)
    ws_bytes = binding.dsa3d_backward_workspace_bytes(*dims, wl.window, wl.dtype)
    if wl.offsets == "zero" and wl.backward:        # the fixed-window backward keeps its dot-product tables there
        ws_bytes = max(ws_bytes, binding.dsa3d_backward_fixed_window_workspace_bytes(*dims, wl.window, wl.dtype))
    if wl.offsets == "small" and wl.backward:       # tables and coefficient planes of the bounded-offsets backward
        ws_bytes = max(ws_bytes, binding.dsa3d_backward_bounded_offsets_workspace_bytes(*dims, wl.window, wl.dtype))
    b = {"out": torch.empty_like(t["q"]),
         "lse": torch.empty(wl.T, wl.H, wl.W, wl.heads, dtype=torch.float32, device=dev),
         "dq": torch.empty_like(t["q"]), "dk": torch.empty_like(t["q"]), "dv": torch.empty_like(t["q"]),
         "doff": torch.empty_like(t["offsets"]),
         "ws": torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=dev)}

    # A workload whose offsets are all zero IS the fixed-window variant: its forward goes through
    # the entry point that takes no offsets tensor (tensor-core tile kernel where the shape
    # allows); the backward is the general one on the zero offsets tensor.
    fixed_window = wl.offsets == "zero" and not args.no_fixed_window
    # offsets below 1 in size: the entry points that decide on the device between the tensor-core tile
    # kernels and the general kernels
    bounded = wl.offsets == "small" and not args.no_fixed_window

    def step():
        if fixed_window:
            binding.dsa3d_forward_fixed_window(t["q"], t["k"], t["v"], *dims, wl.window, b["out"], b["lse"])
        elif bounded:
            binding.dsa3d_forward_bounded_offsets(t["q"], t["k"], t["v"], t["offsets"], *dims, wl.window, b["out"], b["lse"])
        else:
            binding.dsa3d_forward(t["q"], t["k"], t["v"], t["offsets"], *dims, wl.window, b["out"], b["lse"])
        if wl.backward and fixed_window:
            binding.dsa3d_backward_fixed_window(t["q"], t["k"], t["v"], b["lse"], t["dout"], *dims, wl.window,
                                                b["dq"], b["dk"], b["dv"], b["doff"], b["ws"])
        elif wl.backward and bounded:
            binding.dsa3d_backward_bounded_offsets(t["q"], t["k"], t["v"], t["offsets"], b["lse"], t["dout"], *dims,
                                                   wl.window, b["dq"], b["dk"], b["dv"], b["doff"], b["ws"])
        elif wl.backward:
            binding.dsa3d_backward(t["q"], t["k"], t["v"], t["offsets"], b["lse"], t["dout"], *dims,
                                   wl.window, b["dq"], b["dk"], b["dv"], b["doff"], b["ws"])

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(8)] for _ in range(K)]
    for row in ev:                      # give every event a handle before the hook sees it
        for e in row:
            e.record()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    barrier()
    torch.cuda.synchronize()
    for i in range(K):
        binding.dsa3d_set_profile_events(*ev[i][2:8])
        ev[i][0].record()
        step()
        ev[i][1].record()
    torch.cuda.synchronize()
    barrier()
    binding.dsa3d_set_profile_events()
    clocks = sampler.stop() if sampler else None

    step_ms = ev[0][0].elapsed_time(ev[K - 1][1]) / K
    fwd_ms = sum(ev[i][2].elapsed_time(ev[i][3]) for i in range(K)) / K
    bwd_ms = sum(ev[i][4].elapsed_time(ev[i][5]) for i in range(K)) / K if wl.backward else 0.0
    tiled = (wl.backward and wl.dtype == torch.bfloat16 and os.environ.get("DSA3D_TILE", "") != "0"
             and not fixed_window and not bounded)
    sct_ms = sum(ev[i][6].elapsed_time(ev[i][7]) for i in range(K)) / K if tiled else 0.0
    step_ms = max_ranks(step_ms)
    fwd_ms, bwd_ms, sct_ms = max_ranks(fwd_ms), max_ranks(bwd_ms), max_ranks(sct_ms)
    value = aggregate_mtokens_per_s(wl, videos, step_ms)

    # ---------------------------------------------------------------- end to end (host)
    e2e = None
    b.clear()                           # the end-to-end leg brings its own device arena
    torch.cuda.empty_cache()
    if not args.no_e2e:
        e2e = run_e2e(args, wl, t, dims, dev, barrier, max_ranks, world, videos)
    # --------------------------------------------------------------------- CPU baseline
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        sample = oracle_sample(wl, args.cpu_rows, dev, args.cpu_frames)
        dt, threads = time_oracle(sample, wl, wl.backward)
        cpu = {"value": sample["tokens"] / dt / 1e6, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": sample["desc"], "seconds": dt}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak, peak_src = measured_hbm_peak()
    # the fixed-window forward reads no offsets tensor
    fwd_bytes = wl.fwd_bytes() - (wl.N * wl.heads * 12 * wl.P if fixed_window else 0)
    fwd_gbs = fwd_bytes / (fwd_ms * 1e-3) / 1e9
    # The backward's algorithmic bytes belong to its two kernels together (gather: dQ,
    # dOffsets; tile scatter: dK, dV), so they are set against the sum of the two durations.
    bwd_pair_ms = bwd_ms + sct_ms
    bwd_bytes = wl.bwd_bytes() - (wl.N * wl.heads * 12 * wl.P if fixed_window else 0)
    bwd_gbs = bwd_bytes / (bwd_pair_ms * 1e-3) / 1e9 if wl.backward else None
    dominant_bwd = wl.backward and bwd_pair_ms >= fwd_ms
    dom = {"kernel": ("backward_kernel + scatter_tile_kernel" if tiled else
                      "kernels of dsa3d_backward_fixed_window (tables, per-query arithmetic, tile sums)" if fixed_window else
                      "kernels of dsa3d_backward_bounded_offsets (tables, per-sample arithmetic, plane products)" if bounded
                      else "backward_kernel")
                     if dominant_bwd else ("kernel of dsa3d_forward_fixed_window" if fixed_window else
                                           "kernel of dsa3d_forward_bounded_offsets" if bounded else "forward_kernel"),
           "achieved": bwd_gbs if dominant_bwd else fwd_gbs,
           "ms": bwd_pair_ms if dominant_bwd else fwd_ms,
           "bytes": bwd_bytes if dominant_bwd else fwd_bytes}
    step_bytes = fwd_bytes + (bwd_bytes if wl.backward else 0)
    # Fractions of the ceilings that actually bind (the path is on-chip bound, not HBM bound).
    # Computed from the workload where the quantity follows from the method (rows gathered per
    # sample, rows reduced per tile, FMAs per corner); where only a counter can tell (bytes left
    # after L1 hits, warp instructions), from the recorded capture, marked stale when the kernel's
    # sources changed since.
    ceil = measure_ceilings(dev)
    items_all = wl.N * wl.heads
    general = not fixed_window and not bounded       # the on-chip ceilings below are those of the general kernels
    gather_bytes = items_all * wl.P * 8 * 2 * wl.d * wl.elt         # 8 corner rows of K and of V per sample
    fma_fwd = items_all * wl.P * 8 * 2 * wl.d
    fma_peak = ceil["fma_bf16_mixed_tfma"] if wl.dtype == torch.bfloat16 else ceil["fma_f32_tfma"]
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    mhz = (clocks or {}).get("sm_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0
    issue_peak = 4.0 * sms * mhz * 1e6                              # warp instructions per second
    captured = wl.dtype == torch.bfloat16 and wl.d == 128 and wl.P == 27 and general
    onchip = {"ceilings": ceil, "issue_rate_peak_ginst": issue_peak / 1e9}

    def kernel_fracs(name, ms, fma, gathers):
        out = {"fma_frac": fma / (ms * 1e-3) / 1e12 / fma_peak}
        if gathers and general:
            out["l2_gather_algorithmic_frac"] = gather_bytes / (ms * 1e-3) / 1e9 / ceil["l2_row_gather_gbs"]
        if captured:
            rec, stale = ncu_figures(name)
            out["issue_frac"] = items_all * rec["inst"] / (ms * 1e-3) / issue_peak
            if "l2_sm" in rec:
                out["l2_gather_gbs"] = items_all * rec["l2_sm"] / (ms * 1e-3) / 1e9
                out["l2_gather_frac"] = out["l2_gather_gbs"] / ceil["l2_row_gather_gbs"]
            out["counters_stale"] = stale
        return out

    if not general:
        onchip["note"] = ("the ceilings are those of the general gather kernels; this workload runs through the tile "
                          "kernels of the fixed-window / bounded-offsets entry points (counters under profiles/)")
    else:
        onchip["forward_kernel"] = kernel_fracs("forward_kernel", fwd_ms, fma_fwd, True)
    if wl.backward and general:
        onchip["backward_kernel"] = kernel_fracs("backward_kernel", bwd_ms, items_all * wl.P * 8 * 3 * wl.d, True)
        if tiled:
            onchip["scatter_tile_kernel"] = kernel_fracs("scatter_tile_kernel", sct_ms, fma_fwd, False)
            tiles, rows = tile_geometry(wl)
            red_gbs = tiles * rows * 2.0 * wl.d * 4 / (sct_ms * 1e-3) / 1e9     # every region row, dK and dV, fp32
            onchip["scatter_tile_kernel"].update(red_gbs_upper=red_gbs, red_frac_upper=red_gbs / ceil["l2_red_v4_f32_gbs"])
    # the ceiling that binds the dominant kernel: its largest on-chip fraction
    dom_names = ((["backward_kernel"] + (["scatter_tile_kernel"] if tiled else [])) if dominant_bwd else ["forward_kernel"])
    binding_name, binding_frac, binding_kernel = None, 0.0, None
    if general:
        for kname in dom_names:
            for key, label in (("l2_gather_frac", "l2_gather"), ("l2_gather_algorithmic_frac", "l2_gather"),
                               ("issue_frac", "issue"), ("red_frac_upper", "l2_red"), ("fma_frac", "fma")):
                if key == "l2_gather_algorithmic_frac" and "l2_gather_frac" in onchip[kname]:
                    continue                      # the counter-based figure (after L1 hits) is the tighter one
                val = onchip[kname].get(key)
                if val is not None and val > binding_frac:
                    binding_name, binding_frac, binding_kernel = label, val, kname
    traffic, traffic_source = None, None
    if captured:
        kernels = dom_names
        traffic = sum(items_all * ncu_figures(kn)[0]["dram"] for kn in kernels)
        stale = any(ncu_figures(kn)[1] for kn in kernels)
        traffic_source = ("dram__bytes_read.sum + dram__bytes_write.sum per item of an ncu capture on the 3 GB cut "
                          "profile_small_bf16 x items of this launch; understates grids whose K/V and accumulators "
                          "exceed the 126 MB L2 (about 1.6-1.8x more per item at 1080p)"
                          + ("; STALE: kernel sources changed since the capture" if stale else ""))
    line = {
        "metric": metric_name(wl), "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
        "ms_per_step": step_ms, "higher_is_better": True, "scaling": "strong" if sharded else "weak",
        "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "grid": [wl.T, wl.H, wl.W], "tokens": wl.N, "heads": wl.heads,
                   "d": wl.d, "window": list(wl.window), "storage": str(wl.dtype).replace("torch.", ""),
                   "offsets": f"{wl.offsets} sigma={wl.sigma}", "batch_per_gpu": 1,
                   "forward_entry": ("dsa3d_forward_fixed_window" if fixed_window else
                                     "dsa3d_forward_bounded_offsets" if bounded else "dsa3d_forward"),
                   "backward_entry": ("dsa3d_backward_fixed_window" if fixed_window else
                                      "dsa3d_backward_bounded_offsets" if bounded else "dsa3d_backward")
                                     if wl.backward else None,
                   "parallelism": (f"one video, heads sharded over {world} ranks (heads of rank 0: {wl.heads})"
                                   if sharded else f"independent videos x{world}"),
                   "l2": "inputs (tens of GB) exceed the 126 MB L2; no flush needed"},
        "roofline": {"bound": "hbm", "kernel": dom["kernel"], "achieved": dom["achieved"], "peak": peak,
                     "unit": "GB/s", "frac": dom["achieved"] / peak, "traffic": traffic,
                     "traffic_source": traffic_source,
                     "binding": ({"ceiling": binding_name, "kernel": binding_kernel, "frac": binding_frac}
                                 if binding_name else None),
                     "peak_source": peak_src, "algorithmic_bytes_per_launch": dom["bytes"],
                     "kernel_ms": dom["ms"],
                     "forward_kernel": {"ms": fwd_ms, "achieved": fwd_gbs, "frac": fwd_gbs / peak},
                     "backward_kernels": ({"gather_ms": bwd_ms, "tile_scatter_ms": sct_ms, "achieved": bwd_gbs,
                                          "frac": bwd_gbs / peak} if wl.backward else None),
                     "onchip": onchip,
                     "whole_step": {"bytes": step_bytes, "achieved": step_bytes / (step_ms * 1e-3) / 1e9,
                                    "frac": step_bytes / (step_ms * 1e-3) / 1e9 / peak}},
        "cpu_baseline": cpu, "e2e": e2e, "clocks": clocks, "producer": producer,
        "gpu_launches": K * launches_per_step(wl, fixed_window, bounded, tiled),
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def host_memory_available() -> int:
    """Bytes of host memory this process can still take: the smaller of what the kernel
    reports as available and what the container's memory cgroup leaves."""
    avail = None
    try:
        with open("/proc/meminfo") as f:
            for line in f:
                if line.startswith("MemAvailable:"):
                    avail = int(line.split()[1]) * 1024
    except OSError:
        pass
    try:
        limit = open("/sys/fs/cgroup/memory.max").read().strip()
        used = int(open("/sys/fs/cgroup/memory.current").read().strip())
        if limit != "max":
            room = int(limit) - used
            avail = room if avail is None else min(avail, room)
    except (OSError, ValueError):
        pass
    return avail if avail is not None else 0


def run_e2e(args, wl, t, dims, dev, barrier, max_ranks, world, videos=None):
    """Forward + backward through dsa3d_step_host: inputs start in pinned host memory and
    every output ends in pinned host memory, each step."""
    from paper_2607_22696_b200 import binding
    # a forward-only workload goes through the forward-only host entry point
    names_in = ["q", "k", "v", "offsets", "dout"] if wl.backward else ["q", "k", "v", "offsets"]
    # The step keeps every input and every output in page-locked host memory (about twice the
    # input bytes per rank).  Page-locking more than the host can spare takes the machine
    # down, so the leg is skipped, on all ranks together, unless every rank's share fits
    # with a third to spare.
    need = 2 * sum(t[n].numel() * t[n].element_size() for n in names_in)
    fits = 1.0 if host_memory_available() >= 1.5 * need * world else 0.0
    if -max_ranks(-fits) < 1.0:                           # min over ranks
        return {"value": None, "unit": UNIT, "skipped": f"needs {need * world / 1e9:.0f} GB of pinned host "
                "memory over all ranks; not available", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    host_in = {}
    for n in names_in:
        h = torch.empty(t[n].shape, dtype=t[n].dtype, pin_memory=True)
        h.copy_(t[n])
        host_in[n] = h
    shapes = {n: (t[n].shape, t[n].dtype) for n in names_in}
    for n in names_in:
        t[n] = None
    torch.cuda.synchronize()
    torch.cuda.empty_cache()
    row_shape, row_dtype = shapes["q"]
    out_names = ("out", "dq", "dk", "dv") if wl.backward else ("out",)
    host_out = {n: torch.empty(row_shape, dtype=row_dtype, pin_memory=True) for n in out_names}
    host_out["lse"] = torch.empty(dims[:4], dtype=torch.float32, pin_memory=True)
    if wl.backward:
        host_out["doffsets"] = torch.empty(shapes["offsets"][0], dtype=torch.float32, pin_memory=True)
    arena_bytes = (binding.dsa3d_step_host_arena_bytes if wl.backward else
                   binding.dsa3d_forward_host_arena_bytes)(*dims, wl.window, wl.dtype)
    arena = torch.empty(arena_bytes, dtype=torch.uint8, device=dev)

    def step():
        if not wl.backward:
            binding.dsa3d_forward_host(host_in["q"], host_in["k"], host_in["v"], host_in["offsets"], *dims, wl.window,
                                       host_out["out"], host_out["lse"], arena)
            return
        binding.dsa3d_step_host(host_in["q"], host_in["k"], host_in["v"], host_in["offsets"], host_in["dout"],
                                *dims, wl.window, host_out["out"], host_out["lse"], host_out["dq"],
                                host_out["dk"], host_out["dv"], host_out["doffsets"], arena)

    def step_pipelined():
        binding.dsa3d_step_host_pipelined(host_in["q"], host_in["k"], host_in["v"], host_in["offsets"], host_in["dout"],
                                          *dims, wl.window, host_out["out"], host_out["lse"], host_out["dq"],
                                          host_out["dk"], host_out["dv"], host_out["doffsets"], arena)

    steps = max(1, min(args.steps, args.e2e_steps))
    step()
    torch.cuda.synchronize()

    def timed(fn, finish=None):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        torch.cuda.synchronize()
        wall0 = time.perf_counter()
        e0.record()
        for _ in range(steps):
            fn()
        if finish is not None:
            finish()                                  # the stream waits for every queued transfer
        e1.record()
        torch.cuda.synchronize()
        wall = (time.perf_counter() - wall0) / steps
        barrier()
        return max_ranks(e0.elapsed_time(e1) / steps), wall

    # one call at a time (each complete before the next starts) ...
    single_ms, single_wall = timed(step)
    ms, wall = single_ms, single_wall
    # ... and, for a step with a backward, the same calls queued as a sequence: the next step's
    # uploads and the previous step's last downloads overlap the kernels.  The timed region still
    # holds every step's host-to-device and device-to-host copies, the first step's unhidden
    # upload and the last step's unhidden download included.
    if wl.backward:
        ms, wall = timed(step_pipelined, binding.dsa3d_step_host_flush)
    h2d = sum(h.numel() * h.element_size() for h in host_in.values())
    d2h = sum(h.numel() * h.element_size() for h in host_out.values())
    return {"value": aggregate_mtokens_per_s(wl, world if videos is None else videos, ms), "unit": UNIT,
            "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": ms, "wall_ms_per_step": wall * 1e3, "steps": steps,
            "entry_point": ("dsa3d_step_host_pipelined x steps + dsa3d_step_host_flush" if wl.backward
                            else "dsa3d_forward_host"),
            "one_call_at_a_time": {"value": aggregate_mtokens_per_s(wl, world if videos is None else videos, single_ms),
                                   "ms_per_step": single_ms, "entry_point": "dsa3d_step_host" if wl.backward
                                   else "dsa3d_forward_host"}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="1080p_256f_bf16", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--cpu-rows", type=int, default=68, help="grid rows per frame the CPU baseline processes")
    ap.add_argument("--cpu-frames", type=int, default=4, help="consecutive frames the CPU baseline takes its rows from")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--shard", default="videos", choices=["videos", "heads"],
                    help="N > 1: every rank its own video (weak scaling, default) or one video with its heads "
                         "split over the ranks (strong scaling)")
    ap.add_argument("--no-fixed-window", action="store_true",
                    help="zero-offset workloads: use dsa3d_forward on the zero tensor instead of dsa3d_forward_fixed_window")
    ap.add_argument("--producer", action="store_true",
                    help="also time the depthwise convolution and the offset-producing linear layer (bf16 workloads)")
    args = ap.parse_args()
    wl = inputs.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
