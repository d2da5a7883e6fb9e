"""Eq. 1 as a torch.nn.Module: Attn(X) = DWConv3D(X) + 3D-DSA(Q, K, V; offsets) with
offsets = Linear(DWConv3D'(X)) (the offset predictor of the Formulation section).  Parameter
holding and argument marshalling only: every tensor operation runs in the library's kernels
through the autograd wrappers; there is no PyTorch fallback.

Q, K and V are inputs (their projections from X are dense layers outside this operator).  The
offset predictor's linear layer starts at zero, so a fresh module attends over the fixed
window (the zero-offset variant of the paper's ablation) and learns its deformation from there.
"""
from __future__ import annotations

import math

import torch

from . import autograd as ops


class DeformableSlideAttention3D(torch.nn.Module):
    def __init__(self, heads: int, d: int, window=(3, 3, 3), conv_kernel=(3, 3, 3), dtype=torch.bfloat16,
                 device="cuda", seed: int = 0):
        super().__init__()
        self.heads, self.d = int(heads), int(d)
        self.window = tuple(int(s) for s in window)
        self.conv_kernel = tuple(int(s) for s in conv_kernel)
        hidden = self.heads * self.d
        P = self.window[0] * self.window[1] * self.window[2]
        taps = self.conv_kernel[0] * self.conv_kernel[1] * self.conv_kernel[2]
        g = torch.Generator().manual_seed(seed)
        f32 = torch.float32

        def normal(shape, std):
            return (torch.randn(*shape, generator=g, dtype=f32) * std).to(device)

        # the two depthwise convolutions: fp32 parameters [taps, hidden] and [hidden]
        self.offset_conv_weight = torch.nn.Parameter(normal((taps, hidden), 1.0 / math.sqrt(taps)))
        self.offset_conv_bias = torch.nn.Parameter(torch.zeros(hidden, dtype=f32, device=device))
        self.term_conv_weight = torch.nn.Parameter(normal((taps, hidden), 1.0 / math.sqrt(taps)))
        self.term_conv_bias = torch.nn.Parameter(torch.zeros(hidden, dtype=f32, device=device))
        # the offset predictor's linear layer: weight in the storage type, bias fp32; zero at the start
        self.offset_weight = torch.nn.Parameter(torch.zeros(self.heads * P * 3, hidden, dtype=dtype, device=device))
        self.offset_bias = torch.nn.Parameter(torch.zeros(self.heads * P * 3, dtype=f32, device=device))

    def offsets(self, x: torch.Tensor) -> torch.Tensor:
        """Offsets [T, H, W, heads, P, 3] (fp32, grid units) predicted from x [T, H, W, heads*d]."""
        T, H, W, hidden = x.shape
        u = ops.dwconv3d(x, self.offset_conv_weight, self.offset_conv_bias, self.conv_kernel)
        off = ops.offsets_linear(u.view(T * H * W, hidden), self.offset_weight, self.offset_bias)
        return off.view(T, H, W, self.heads, -1, 3)

    def forward(self, x: torch.Tensor, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor) -> torch.Tensor:
        """x: [T, H, W, heads*d]; q, k, v: [T, H, W, heads, d]; returns [T, H, W, heads, d]."""
        T, H, W, hidden = x.shape
        if hidden != self.heads * self.d:
            raise ValueError("x must have heads*d channels")
        term = ops.dwconv3d(x, self.term_conv_weight, self.term_conv_bias, self.conv_kernel)
        return ops.dsa3d(q, k, v, self.offsets(x), self.window, residual=term.view(T, H, W, self.heads, self.d))
