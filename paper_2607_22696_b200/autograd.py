"""torch.autograd wrappers around the C-ABI entry points (argument marshalling only: every
step of the operator runs in the library's kernels; there is no PyTorch fallback).

    out = dsa3d(q, k, v, offsets, window)                 # 3D deformable slide attention
    out = dsa3d(q, k, v, offsets, window, residual=r)     # with the first term of Eq. 1 added
    out = dsa3d_fixed_window(q, k, v, window)             # all offsets zero, no offsets tensor
    y = dwconv3d(x, weight, bias, kernel)                 # depthwise 3-D convolution, channels-last
    offsets = offsets_linear(u, w, bias)                  # linear layer of the offset predictor

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


class _DwConv3d(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, weight, bias, kernel):
        if x.dim() != 4:
            raise ValueError("x must be [T, H, W, C] (channels-last)")
        T, H, W, C = (int(s) for s in x.shape)
        x, weight = x.contiguous(), weight.contiguous()
        y = torch.empty_like(x)
        binding.dsa3d_dwconv3d_forward(x, weight, None if bias is None else bias.contiguous(), T, H, W, C, kernel, y)
        ctx.save_for_backward(x, weight)
        ctx.kernel = tuple(kernel)
        ctx.has_bias = bias is not None
        return y

    @staticmethod
    def backward(ctx, dy):
        x, weight = ctx.saved_tensors
        T, H, W, C = (int(s) for s in x.shape)
        need_x, need_w, need_b = ctx.needs_input_grad[0], ctx.needs_input_grad[1], ctx.has_bias and ctx.needs_input_grad[2]
        dx = torch.empty_like(x) if need_x else None
        dw = torch.empty_like(weight) if (need_w or need_b) else None
        db = torch.empty((C,), dtype=torch.float32, device=x.device) if need_b else None
        nbytes = binding.dsa3d_dwconv3d_backward_workspace_bytes(C, ctx.kernel)
        ws = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=x.device) if need_x else None
        binding.dsa3d_dwconv3d_backward(x, weight, dy.contiguous(), T, H, W, C, ctx.kernel, dx, dw, db, ws)
        return dx, (dw if need_w else None), db, None


class _OffsetsLinear(torch.autograd.Function):
    @staticmethod
    def forward(ctx, u, w, bias):
        if u.dim() != 2 or w.dim() != 2 or u.shape[1] != w.shape[1]:
            raise ValueError("u must be [tokens, C] and w [O, C]")
        u, w, bias = u.contiguous(), w.contiguous(), bias.contiguous()
        tokens, C, O = int(u.shape[0]), int(u.shape[1]), int(w.shape[0])
        out = torch.empty((tokens, O), dtype=torch.float32, device=u.device)
        binding.dsa3d_offsets_linear_forward(u, w, bias, tokens, C, O, out)
        ctx.save_for_backward(u, w)
        return out

    @staticmethod
    def backward(ctx, doffsets):
        u, w = ctx.saved_tensors
        tokens, C, O = int(u.shape[0]), int(u.shape[1]), int(w.shape[0])
        need_u, need_w, need_b = ctx.needs_input_grad
        du = torch.empty_like(u) if need_u else None
        dw = torch.empty((O, C), dtype=torch.float32, device=u.device) if need_w else None
        db = torch.empty((O,), dtype=torch.float32, device=u.device) if need_b else None
        nbytes = binding.dsa3d_offsets_linear_backward_workspace_bytes(tokens, C, O, u.dtype)
        ws = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=u.device)
        binding.dsa3d_offsets_linear_backward(u, w, doffsets.contiguous(), tokens, C, O, du, dw, db, ws)
        return du, (None if dw is None else dw.to(w.dtype)), db


def dwconv3d(x, weight, bias, kernel):
    """Depthwise 3-D convolution of x [T, H, W, C] (first term of Eq. 1; first stage of the
    offset predictor); weight fp32 [kt*kh*kw, C], bias fp32 [C] or None."""
    return _DwConv3d.apply(x, weight, bias, tuple(kernel))


def offsets_linear(u, w, bias):
    """offsets [tokens, O] (fp32) = u [tokens, C] . w [O, C]^T + bias [O] (fp32); the gradient of
    w is accumulated in fp32 and rounded once to w's dtype."""
    return _OffsetsLinear.apply(u, w, bias)


def dsa3d(q, k, v, offsets, window, residual=None):
    """3D deformable slide attention (Eq. 1, second term; plus `residual` if given)."""
    return _Dsa3d.apply(q, k, v, offsets, residual, tuple(window))


def dsa3d_fixed_window(q, k, v, window):
    """The operator with all offsets zero (no offsets tensor, no offset gradient)."""
    return _Dsa3dFixedWindow.apply(q, k, v, tuple(window))
