"""Helpers of the GPU parity tests: run the CUDA library through its binding, run the CPU
oracle on the same bytes, and compare with the tolerances the tests state.

Tolerances.  fp32 storage: max abs error 1e-5 for out and lse, 1e-4 for gradients.  bf16
storage (fp32 accumulation on the GPU, results rounded to bf16): every element must satisfy
|gpu - oracle| <= 2e-2 * max(|oracle|, rms(oracle tensor)); the rms floor keeps the bound
meaningful for elements near zero.  A tensor the oracle gives as exactly zero everywhere (dq
and dk of a one-cell window) has no relative bound at all - fp32 accumulation leaves rounding
noise of order 1e-7 there - and takes the fp32 bound above instead.  lse and doffsets are fp32
tensors of a bf16 problem and use the same rule.
"""
from __future__ import annotations

import math

import torch

import oracle
from paper_2607_22696_b200 import binding

F32_FWD_ATOL = 1e-5
F32_BWD_ATOL = 1e-4
BF16_REL = 2e-2


def gpu_forward(q, k, v, off, dims, window):
    T, H, W, heads, d = dims
    out = torch.empty_like(q)
    lse = torch.empty(T, H, W, heads, dtype=torch.float32, device=q.device)
    binding.dsa3d_forward(q, k, v, off, T, H, W, heads, d, window, out, lse)
    return out, lse


def gpu_backward(q, k, v, off, lse, dout, dims, window):
    T, H, W, heads, d = dims
    dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    doff = torch.empty_like(off)
    nbytes = binding.dsa3d_backward_workspace_bytes(T, H, W, heads, d, window, q.dtype)
    ws = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=q.device)
    # poison the outputs and the workspace: the library must overwrite everything
    for z in (dq, dk, dv, doff):
        z.fill_(float("nan"))
    ws.fill_(0xFF)
    binding.dsa3d_backward(q, k, v, off, lse, dout, T, H, W, heads, d, window, dq, dk, dv, doff, ws)
    torch.cuda.synchronize()
    del ws
    return dq, dk, dv, doff


def assert_close(name, got, ref, dtype, backward=False):
    """got: GPU result (any float dtype, any device); ref: fp64 oracle result."""
    got = got.detach().to("cpu", torch.float64).reshape(-1)
    ref = ref.detach().to(torch.float64).reshape(-1)
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    assert torch.isfinite(got).all(), f"{name}: non-finite values in the GPU result"
    err = (got - ref).abs()
    if dtype == torch.float32:
        atol = F32_BWD_ATOL if backward else F32_FWD_ATOL
        worst = float(err.max()) if err.numel() else 0.0
        assert worst <= atol, f"{name}: max abs error {worst:.3e} > {atol:.1e}"
    else:
        rms = float(ref.pow(2).mean().sqrt()) if ref.numel() else 0.0
        bound = BF16_REL * torch.clamp(ref.abs(), min=rms)
        if rms == 0.0:                     # an all-zero oracle tensor: only the absolute fp32 bound applies
            bound = bound + (F32_BWD_ATOL if backward else F32_FWD_ATOL)
        excess = err - bound
        if excess.numel() and float(excess.max()) > 0:
            i = int(excess.argmax())
            raise AssertionError(f"{name}: |gpu - oracle| = {float(err[i]):.4e} at {i} exceeds "
                                 f"the bound {float(bound[i]):.4e} "
                                 f"(oracle {float(ref[i]):.4e}, rms {rms:.4e})")


def full_parity(q, k, v, off, dout, window, check_backward=True):
    """Whole-tensor comparison on a problem small enough for the oracle."""
    T, H, W, heads, d = q.shape
    dims = (T, H, W, heads, d)
    dtype = q.dtype
    dev = [z.cuda() for z in (q, k, v, off)]
    out, lse = gpu_forward(*dev, dims, window)
    torch.cuda.synchronize()
    o_ref, l_ref = oracle.forward(q, k, v, off, T, H, W, heads, d, window)
    assert_close("out", out, o_ref, dtype)
    assert_close("lse", lse, l_ref, dtype)
    if not check_backward:
        return
    dq, dk, dv, doff = gpu_backward(*dev, lse, dout.cuda(), dims, window)
    r = oracle.backward(q, k, v, off, dout, T, H, W, heads, d, window)
    for name, got, ref in zip(("dq", "dk", "dv", "doffsets"), (dq, dk, dv, doff), r):
        assert_close(name, got, ref, dtype, backward=True)


def max_abs_offset(off: torch.Tensor) -> float:
    """Largest finite |offset| (a statistic of the input, used to bound which queries can
    reach a given key row)."""
    best = 0.0
    flat = off.reshape(-1)
    step = 1 << 28
    for s in range(0, flat.numel(), step):
        c = flat[s:s + step]
        c = c[torch.isfinite(c)]
        if c.numel():
            best = max(best, float(c.abs().max()))
    return best


def box_tokens(lo, hi, dims):
    T, H, W = dims[:3]
    t = torch.arange(max(lo[0], 0), min(hi[0], T))
    y = torch.arange(max(lo[1], 0), min(hi[1], H))
    x = torch.arange(max(lo[2], 0), min(hi[2], W))
    return ((t[:, None, None] * H + y[None, :, None]) * W + x[None, None, :]).reshape(-1)


def sampled_parity(tens, dims, window, lse, grads, heads_sel, n_random=1024, key_boxes=(), seed=0):
    """Parity on a workload too large for a full oracle run.

    Per-query results (out, lse, dq, doffsets) are compared on the first, middle and last
    few tokens plus `n_random` random tokens; dk / dv on the key rows of `key_boxes`
    ((lo, hi) index triples), for which the oracle processes every query that can reach
    them: a query at coordinate c touches key row j only if |c - j| < 1 + window radius +
    max |offset| on every axis.  Only the heads in `heads_sel` are checked; heads are
    independent, so slicing them out gives the oracle an exact smaller problem.
    """
    T, H, W, heads, d = dims
    N = T * H * W
    P = window[0] * window[1] * window[2]
    dtype = tens["q"].dtype
    hs = torch.tensor(heads_sel, device=tens["q"].device)
    nh = len(heads_sel)
    k_sub = tens["k"].view(N, heads, d)[:, hs].contiguous().cpu()
    v_sub = tens["v"].view(N, heads, d)[:, hs].contiguous().cpu()

    def rows(z, tail, tok):
        tok = tok.to(z.device)
        return z.view(N, heads, *tail)[tok][:, hs].contiguous().cpu()

    g = torch.Generator().manual_seed(seed)
    edge = min(N, 3 * W)
    qtok = torch.cat([torch.arange(0, edge), torch.arange(N // 2, min(N, N // 2 + edge)),
                      torch.arange(N - edge, N), torch.randint(0, N, (n_random,), generator=g)]).unique()
    q_r, off_r = rows(tens["q"], (d,), qtok), rows(tens["offsets"], (P, 3), qtok)
    o_ref, l_ref = oracle.forward(q_r, k_sub, v_sub, off_r, T, H, W, nh, d, window, qtok=qtok)
    assert_close("out[sampled]", rows(tens["out"], (d,), qtok), o_ref, dtype)
    assert_close("lse[sampled]", rows(lse, (), qtok), l_ref, dtype)
    if grads is None:
        return
    dq, dk, dv, doff = grads
    dout_r = rows(tens["dout"], (d,), qtok)
    dq_ref, _, _, doff_ref = oracle.backward(q_r, k_sub, v_sub, off_r, dout_r, T, H, W, nh, d, window,
                                             qtok=qtok, ktok=torch.zeros(0, dtype=torch.int64))
    assert_close("dq[sampled]", rows(dq, (d,), qtok), dq_ref, dtype, backward=True)
    assert_close("doffsets[sampled]", rows(doff, (P, 3), qtok), doff_ref, dtype, backward=True)

    reach = int(math.floor(1 + max(w // 2 for w in window) + max_abs_offset(tens["offsets"]))) + 1
    for lo, hi in key_boxes:
        ktok = box_tokens(lo, hi, dims)
        qbox = box_tokens([a - reach for a in lo], [b + reach for b in hi], dims)
        _, dk_ref, dv_ref, _ = oracle.backward(
            rows(tens["q"], (d,), qbox), k_sub, v_sub, rows(tens["offsets"], (P, 3), qbox),
            rows(tens["dout"], (d,), qbox), T, H, W, nh, d, window, qtok=qbox, ktok=ktok)
        assert float(dk_ref.abs().max()) > 0
        assert_close(f"dk[box {lo}]", rows(dk, (d,), ktok), dk_ref, dtype, backward=True)
        assert_close(f"dv[box {lo}]", rows(dv, (d,), ktok), dv_ref, dtype, backward=True)


def head_inner(a: torch.Tensor, b: torch.Tensor):
    """Per head, over tokens and channels: (sum of a*b, sqrt of the sum of (a*b)^2), fp64,
    chunked over the leading axis."""
    heads = a.shape[-2]
    tot = torch.zeros(heads, dtype=torch.float64, device=a.device)
    tot_sq = torch.zeros_like(tot)
    for t in range(a.shape[0]):
        prod = a[t].to(torch.float64) * b[t].to(torch.float64)
        tot += prod.sum(dim=(0, 1, 3))
        tot_sq += prod.pow(2).sum(dim=(0, 1, 3))
    return tot, tot_sq.sqrt()


def assert_bilinearity_invariants(tens, out, grads, ulp=2.0 ** -9):
    """sum <q,dQ> = sum <K,dK> and sum <V,dV> = sum <out,dO> per head: properties of the exact
    operator for any offsets, checked on the GPU result over every element.  The GPU tensors
    are rounded to their storage type, each element by at most `ulp` relative; independent
    roundings add in quadrature, so the two sides may differ by a few ulp * sqrt(sum of
    squared products)."""
    dq, dk, dv, _ = grads
    a, a_rss = head_inner(tens["q"], dq)
    b, b_rss = head_inner(tens["k"], dk)
    c, c_rss = head_inner(tens["v"], dv)
    e, e_rss = head_inner(out, tens["dout"])
    assert bool(((a - b).abs() <= 8 * ulp * (a_rss + b_rss)).all()), (a, b, a_rss, b_rss)
    assert bool(((c - e).abs() <= 8 * ulp * (c_rss + e_rss)).all()), (c, e, c_rss, e_rss)
