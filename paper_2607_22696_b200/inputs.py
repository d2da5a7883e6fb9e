"""Seeded synthetic inputs for 3D-DSA: the workload table and a counter-based generator.

This module holds none of the operator's arithmetic.  It serves both the CUDA library's
tests/benchmark and the CPU oracle's tests, and imports neither.

Every element is a pure function of (seed, tensor id, flat index): a splitmix64 hash of
the counter gives two 32-bit uniforms, Box-Muller turns them into a standard normal in
fp64, which is scaled and rounded once to the storage type.  Generation is chunked so a
45 GB workload never needs more than a few hundred MB of temporaries, and it runs on
whichever device the caller asks for.  CPU and GPU evaluations of log/cos may differ in
the last fp64 bit, so a test always generates a tensor ONCE and hands the same bytes to
both sides.

The shapes stand in for the paper's workloads: latent-video token grids of a diffusion
transformer (1080p, 256 frames, patch 16 gives about 2.07 M tokens; head dims 64 and 128)
with iid normal activations and iid normal learned offsets.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Tuple

import torch

TENSOR_IDS = {"q": 0, "k": 1, "v": 2, "offsets": 3, "dout": 4}

_MASK64 = (1 << 64) - 1


def _i64(x: int) -> int:
    """Reinterpret an unsigned 64-bit constant as the signed value torch.int64 stores."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _i64(0x9E3779B97F4A7C15)
_M1 = _i64(0xBF58476D1CE4E5B9)
_M2 = _i64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64 (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _splitmix64(ctr: torch.Tensor) -> torch.Tensor:
    z = ctr * _GOLDEN + _GOLDEN          # wraps modulo 2^64
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def _stream_base(seed: int, tensor_id: int) -> int:
    return _i64((seed * 0x632BE59BD9B4E019 + tensor_id * 0xD1342543DE82EF95 + 0x2545F4914F6CDD1D))


def _hash_chunk(seed: int, tensor_id: int, start: int, count: int, device) -> torch.Tensor:
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return _splitmix64(idx + _stream_base(seed, tensor_id))


def normal(shape, seed: int, tensor_id: int, sigma: float, dtype: torch.dtype, device="cpu",
           chunk: int = 1 << 24, first: int = 0) -> torch.Tensor:
    """iid N(0, sigma^2) tensor, rounded once (RNE) to ``dtype``.  ``first`` is the flat index
    of the tensor's first element inside a larger logical tensor, so a slice of a big
    workload can be produced without the rest."""
    n = math.prod(shape)
    out = torch.empty(n, dtype=dtype, device=device)
    for start in range(0, n, chunk):
        cnt = min(chunk, n - start)
        h = _hash_chunk(seed, tensor_id, first + start, cnt, device)
        u1 = (_lsr(h, 32).to(torch.float64) + 0.5) * (1.0 / 4294967296.0)
        u2 = ((h & 0xFFFFFFFF).to(torch.float64) + 0.5) * (1.0 / 4294967296.0)
        z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
        out[start:start + cnt] = (z * sigma).to(dtype)
    return out.view(*shape)


def uniform_int(shape, seed: int, tensor_id: int, lo: int, hi: int, dtype: torch.dtype,
                device="cpu", chunk: int = 1 << 24, first: int = 0) -> torch.Tensor:
    """iid integers uniform on {lo..hi}, stored as ``dtype``."""
    n = math.prod(shape)
    out = torch.empty(n, dtype=dtype, device=device)
    span = hi - lo + 1
    for start in range(0, n, chunk):
        cnt = min(chunk, n - start)
        h = _lsr(_hash_chunk(seed, tensor_id, first + start, cnt, device), 16)
        out[start:start + cnt] = (h % span + lo).to(dtype)
    return out.view(*shape)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One synthetic 3D-DSA problem.  ``offsets`` is 'normal', 'zero', 'int' (uniform
    integers in [-int_range, int_range]) or 'drift' (one velocity per (token, head) plus a
    small per-sample jitter)."""
    name: str
    T: int
    H: int
    W: int
    heads: int
    d: int
    window: Tuple[int, int, int]
    dtype: torch.dtype
    sigma: float
    seed: int
    backward: bool = True
    offsets: str = "normal"
    int_range: int = 2

    @property
    def N(self) -> int:
        return self.T * self.H * self.W

    @property
    def P(self) -> int:
        return self.window[0] * self.window[1] * self.window[2]

    @property
    def elt(self) -> int:
        return 2 if self.dtype == torch.bfloat16 else 4

    def fwd_bytes(self) -> int:
        """Algorithmic bytes of one forward: Q, K, V, offsets read once; out, lse written."""
        return self.N * self.heads * (4 * self.d * self.elt + 12 * self.P + 4)

    def bwd_bytes(self) -> int:
        """Algorithmic bytes of one backward: Q, K, V, dOut, offsets, lse read once; dQ, dK,
        dV, dOffsets written once."""
        return self.N * self.heads * (7 * self.d * self.elt + 24 * self.P + 4)


_BF16, _F32 = torch.bfloat16, torch.float32

WORKLOADS: Dict[str, Workload] = {w.name: w for w in [
    Workload("tiny_f32", 4, 8, 8, 2, 32, (3, 3, 3), _F32, 0.5, 0),
    Workload("480p_bf16_fwd", 16, 30, 52, 16, 64, (3, 3, 3), _BF16, 1.0, 1, backward=False),
    Workload("720p_bf16", 64, 45, 80, 24, 128, (3, 3, 3), _BF16, 1.5, 2),
    Workload("1080p_256f_bf16", 256, 68, 120, 16, 128, (3, 3, 3), _BF16, 2.0, 3),
    # a 3 GB cut of the 1080p workload (same heads' row size, window and offset spread, inputs
    # still several times the L2) for profiler captures that must stay small
    Workload("profile_small_bf16", 32, 45, 80, 8, 128, (3, 3, 3), _BF16, 2.0, 5),
    # the window the paper itself runs, (3,7,7) = 147 samples, on 64 frames of the 1080p grid
    # (at 256 frames the offsets alone would be 59 GB)
    Workload("1080p_64f_w377_bf16", 64, 68, 120, 16, 128, (3, 7, 7), _BF16, 2.0, 6),
    # not a BASELINE config: the head shape of the paper's 1B model (2048 hidden, 32 heads of 64
    # channels) on 128 frames of the 1080p grid, same bytes per token as 16 heads of 128
    Workload("1080p_128f_h32d64_bf16", 128, 68, 120, 32, 64, (3, 3, 3), _BF16, 2.0, 8),
    # not a BASELINE config: offsets with the coherence of a motion field (structured-motion
    # data of the paper's quality ablation), same grid and spread as the 1080p workload
    Workload("1080p_256f_drift_bf16", 256, 68, 120, 16, 128, (3, 3, 3), _BF16, 2.0, 7, offsets="drift"),
] + [
    Workload(f"sweep_w{kt}{kh}{kw}_{kind}", 64, 45, 80, 16, 128, (kt, kh, kw), _BF16,
             3.0 if kind == "normal" else 0.0, 4, offsets=kind)
    for (kt, kh, kw) in [(2, 2, 2), (3, 3, 3), (3, 5, 5)] for kind in ["zero", "int", "normal"]
] + [
    # not a BASELINE config: the fixed-window variant of the paper's ablation on the effect of offsets
    # (window (3,7,7), all offsets zero) on the grid of the sweep
    Workload("sweep_w377_zero", 64, 45, 80, 16, 128, (3, 7, 7), _BF16, 0.0, 4, offsets="zero"),
    # not a BASELINE config: offsets as small perturbations of the window (every component below 1 in
    # size), the regime in which the forward runs as tile attention on the tensor cores
    Workload("sweep_w333_small", 64, 45, 80, 16, 128, (3, 3, 3), _BF16, 0.4, 4, offsets="small"),
    # cuts of the fixed-window and small-offset cases for profiler captures (a few GB on the device)
    Workload("profile_small_w333_zero_bf16", 32, 45, 80, 8, 128, (3, 3, 3), _BF16, 0.0, 5, offsets="zero"),
    Workload("profile_small_w377_zero_bf16", 16, 45, 80, 8, 128, (3, 7, 7), _BF16, 0.0, 5, offsets="zero"),
    Workload("profile_small_w333_small_bf16", 32, 45, 80, 8, 128, (3, 3, 3), _BF16, 0.4, 5, offsets="small"),
]}


def make_offsets(wl: Workload, device="cpu", frames=None) -> torch.Tensor:
    """Offsets of the whole grid, or of frames [frames[0], frames[1]) only."""
    t0, t1 = (0, wl.T) if frames is None else frames
    shape = (t1 - t0, wl.H, wl.W, wl.heads, wl.P, 3)
    first = t0 * wl.H * wl.W * wl.heads * wl.P * 3
    if wl.offsets == "zero":
        return torch.zeros(shape, dtype=torch.float32, device=device)
    if wl.offsets == "int":
        return uniform_int(shape, wl.seed, TENSOR_IDS["offsets"], -wl.int_range, wl.int_range,
                           torch.float32, device, first=first)
    if wl.offsets == "drift":
        # every sample of a (token, head) shares one velocity ~N(0, sigma^2) per axis and adds
        # its own small jitter ~N(0, 0.3^2): what offsets that follow motion would look like
        vel = normal((t1 - t0, wl.H, wl.W, wl.heads, 1, 3), wl.seed, TENSOR_IDS["offsets"] + 16, wl.sigma,
                     torch.float32, device, first=t0 * wl.H * wl.W * wl.heads * 3)
        jit = normal(shape, wl.seed, TENSOR_IDS["offsets"], 0.3, torch.float32, device, first=first)
        return jit.add_(vel)
    if wl.offsets == "small":
        # learned offsets as small perturbations of the fixed window: N(0, sigma^2) cut off below 1 in size
        return normal(shape, wl.seed, TENSOR_IDS["offsets"], wl.sigma, torch.float32, device, first=first).clamp_(-0.999, 0.999)
    return normal(shape, wl.seed, TENSOR_IDS["offsets"], wl.sigma, torch.float32, device, first=first)


def make_rows(wl: Workload, name: str, device="cpu", frames=None) -> torch.Tensor:
    """Tensor ``name`` in (q, k, v, dout) for the whole grid or for frames [t0, t1) only; the
    slice equals the same frames of the full tensor generated on the same kind of device."""
    t0, t1 = (0, wl.T) if frames is None else frames
    shape = (t1 - t0, wl.H, wl.W, wl.heads, wl.d)
    first = t0 * wl.H * wl.W * wl.heads * wl.d
    return normal(shape, wl.seed, TENSOR_IDS[name], 1.0, wl.dtype, device, first=first)


def make_inputs(wl: Workload, device="cpu", with_dout: bool | None = None) -> Dict[str, torch.Tensor]:
    """q, k, v [T,H,W,heads,d] ~N(0,1) in the workload's dtype, offsets [T,H,W,heads,P,3]
    fp32, and dout ~N(0,1) when the workload has a backward pass."""
    shape = (wl.T, wl.H, wl.W, wl.heads, wl.d)
    t = {name: normal(shape, wl.seed, TENSOR_IDS[name], 1.0, wl.dtype, device) for name in "qkv"}
    t["offsets"] = make_offsets(wl, device)
    if wl.backward if with_dout is None else with_dout:
        t["dout"] = normal(shape, wl.seed, TENSOR_IDS["dout"], 1.0, wl.dtype, device)
    return t
