"""CPU oracle for the two layers around the attention operator in Eq. 1: the depthwise 3-D
convolution (first term of Eq. 1, and the first stage of the offset predictor of the
Formulation section) and the linear layer that turns its output into offsets.

TEST INFRASTRUCTURE ONLY, like the rest of this package: plain fp64 PyTorch CPU ops written
from the definitions, no blocking or fusion; nothing here is imported by the CUDA path.

Conventions (the paper fixes none of them beyond "depthwise 3D convolution followed by a
linear layer"; the implementation section names nn.Conv3d with groups = hidden size):
  * activations are channels-last, x[t, y, x, c];
  * the convolution is a cross-correlation with zero padding and unit stride that keeps the
    grid size; tap (i, j, l) of a (kt, kh, kw) kernel reads the input at displacement
    (i - kt//2, j - kh//2, l - kw//2), the same centring as the attention window;
  * weight[tap, c] with tap = (i*kh + j)*kw + l, bias[c];
  * the linear layer is offsets[n, o] = bias[o] + sum_c u[n, c] * w[o, c].
"""
from __future__ import annotations

import torch


def dwconv3d(x: torch.Tensor, weight: torch.Tensor, bias, kernel) -> torch.Tensor:
    """Depthwise 3-D convolution of x [T, H, W, C]; returns fp64 [T, H, W, C]."""
    kt, kh, kw = (int(s) for s in kernel)
    T, H, W, C = x.shape
    if tuple(weight.shape) != (kt * kh * kw, C):
        raise ValueError("weight must be [kt*kh*kw, C]")
    xd = x.to(torch.float64)
    wd = weight.to(torch.float64)
    y = torch.zeros(T, H, W, C, dtype=torch.float64)
    if bias is not None:
        y += bias.to(torch.float64)
    for i in range(kt):
        for j in range(kh):
            for l in range(kw):
                dt, dy, dx = i - kt // 2, j - kh // 2, l - kw // 2
                # output positions whose displaced input position lies inside the grid
                t0, t1 = max(0, -dt), min(T, T - dt)
                y0, y1 = max(0, -dy), min(H, H - dy)
                x0, x1 = max(0, -dx), min(W, W - dx)
                if t0 >= t1 or y0 >= y1 or x0 >= x1:
                    continue
                tap = (i * kh + j) * kw + l
                y[t0:t1, y0:y1, x0:x1] += wd[tap] * xd[t0 + dt:t1 + dt, y0 + dy:y1 + dy, x0 + dx:x1 + dx]
    return y


def offsets_linear(u: torch.Tensor, w: torch.Tensor, bias) -> torch.Tensor:
    """offsets[n, o] = bias[o] + sum_c u[n, c] w[o, c] in fp64; u [N, C], w [O, C]."""
    out = u.to(torch.float64) @ w.to(torch.float64).t()
    if bias is not None:
        out = out + bias.to(torch.float64)
    return out


def dwconv3d_backward(x: torch.Tensor, weight: torch.Tensor, dy: torch.Tensor, kernel):
    """Gradients of L = sum(dy * dwconv3d(x, weight, bias)) with respect to x, weight and
    bias, written from the definition: tap (i, j, l) couples output position s with input
    position s + disp, so dx[s + disp] += w[tap] * dy[s], dw[tap] = sum_s x[s + disp] * dy[s]
    over the output positions whose displaced position lies inside the grid, and
    dbias[c] = sum_s dy[s, c].  Returns fp64 (dx [T, H, W, C], dw [taps, C], dbias [C])."""
    kt, kh, kw = (int(s) for s in kernel)
    T, H, W, C = x.shape
    xd = x.to(torch.float64)
    wd = weight.to(torch.float64)
    g = dy.to(torch.float64)
    dx = torch.zeros(T, H, W, C, dtype=torch.float64)
    dw = torch.zeros(kt * kh * kw, C, dtype=torch.float64)
    for i in range(kt):
        for j in range(kh):
            for l in range(kw):
                dt, dyy, dxx = i - kt // 2, j - kh // 2, l - kw // 2
                t0, t1 = max(0, -dt), min(T, T - dt)
                y0, y1 = max(0, -dyy), min(H, H - dyy)
                x0, x1 = max(0, -dxx), min(W, W - dxx)
                if t0 >= t1 or y0 >= y1 or x0 >= x1:
                    continue
                tap = (i * kh + j) * kw + l
                gs = g[t0:t1, y0:y1, x0:x1]
                dx[t0 + dt:t1 + dt, y0 + dyy:y1 + dyy, x0 + dxx:x1 + dxx] += wd[tap] * gs
                dw[tap] = (xd[t0 + dt:t1 + dt, y0 + dyy:y1 + dyy, x0 + dxx:x1 + dxx] * gs).sum(dim=(0, 1, 2))
    return dx, dw, g.sum(dim=(0, 1, 2))


def offsets_linear_backward(u: torch.Tensor, w: torch.Tensor, doffsets: torch.Tensor):
    """Gradients of L = sum(doffsets * offsets_linear(u, w, bias)): du[n, c] = sum_o
    doffsets[n, o] w[o, c]; dw[o, c] = sum_n doffsets[n, o] u[n, c]; dbias[o] = sum_n
    doffsets[n, o].  Returns fp64 (du [N, C], dw [O, C], dbias [O])."""
    g = doffsets.to(torch.float64)
    return g @ w.to(torch.float64), g.t() @ u.to(torch.float64), g.sum(dim=0)
