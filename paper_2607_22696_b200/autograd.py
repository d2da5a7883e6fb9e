"""torch.autograd wrappers around the C-ABI entry points (argument marshalling only: every
step of the operator runs in the library's kernels; there is no PyTorch fallback).

    out = dsa3d(q, k, v, offsets, window)                 # 3D deformable slide attention
    out = dsa3d(q, k, v, offsets, window, residual=r)     # with the first term of Eq. 1 added
    out = dsa3d_fixed_window(q, k, v, window)             # all offsets zero, no offsets tensor

q, k, v: CUDA tensors [T, H, W, heads, d] (bf16 or fp32, contiguous); offsets: fp32
[T, H, W, heads, P, 3].  Gradients flow to q, k, v, offsets (and to `residual`, whose gradient
is the incoming one).  The log-sum-exp saved by the forward is not differentiable.
"""
from __future__ import annotations

import torch

from . import binding


def _dims(q):
    if q.dim() != 5:
        raise ValueError("q, k, v must be [T, H, W, heads, d]")
    return tuple(int(s) for s in q.shape)


class _Dsa3d(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, offsets, residual, window):
        T, H, W, heads, d = _dims(q)
        q, k, v, offsets = q.contiguous(), k.contiguous(), v.contiguous(), offsets.contiguous()
        out = torch.empty_like(q)
        lse = torch.empty((T, H, W, heads), dtype=torch.float32, device=q.device)
        if residual is None:
            binding.dsa3d_forward(q, k, v, offsets, T, H, W, heads, d, window, out, lse)
        else:
            binding.dsa3d_forward_residual(q, k, v, offsets, residual.contiguous(), T, H, W, heads, d, window, out, lse)
        ctx.save_for_backward(q, k, v, offsets, lse)
        ctx.window = tuple(window)
        ctx.has_residual = residual is not None
        return out

    @staticmethod
    def backward(ctx, dout):
        q, k, v, offsets, lse = ctx.saved_tensors
        T, H, W, heads, d = _dims(q)
        dout = dout.contiguous()
        dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
        doff = torch.empty_like(offsets)
        nbytes = binding.dsa3d_backward_workspace_bytes(T, H, W, heads, d, ctx.window, q.dtype)
        ws = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=q.device)
        binding.dsa3d_backward(q, k, v, offsets, lse, dout, T, H, W, heads, d, ctx.window, dq, dk, dv, doff, ws)
        return dq, dk, dv, doff, (dout if ctx.has_residual else None), None


class _Dsa3dFixedWindow(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, window):
        T, H, W, heads, d = _dims(q)
        q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
        out = torch.empty_like(q)
        lse = torch.empty((T, H, W, heads), dtype=torch.float32, device=q.device)
        binding.dsa3d_forward_fixed_window(q, k, v, T, H, W, heads, d, window, out, lse)
        ctx.save_for_backward(q, k, v, lse)
        ctx.window = tuple(window)
        return out

    @staticmethod
    def backward(ctx, dout):
        q, k, v, lse = ctx.saved_tensors
        T, H, W, heads, d = _dims(q)
        dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
        nbytes = binding.dsa3d_backward_fixed_window_workspace_bytes(T, H, W, heads, d, ctx.window, q.dtype)
        ws = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=q.device)
        binding.dsa3d_backward_fixed_window(q, k, v, lse, dout.contiguous(), T, H, W, heads, d, ctx.window, dq, dk, dv,
                                            None, ws)
        return dq, dk, dv, None


def dsa3d(q, k, v, offsets, window, residual=None):
    """3D deformable slide attention (Eq. 1, second term; plus `residual` if given)."""
    return _Dsa3d.apply(q, k, v, offsets, residual, tuple(window))


def dsa3d_fixed_window(q, k, v, window):
    """The operator with all offsets zero (no offsets tensor, no offset gradient)."""
    return _Dsa3dFixedWindow.apply(q, k, v, tuple(window))
