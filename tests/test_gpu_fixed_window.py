"""GPU parity of the fixed-window forward (all offsets zero, no offsets tensor): the
tensor-core tile kernels for bf16 with 64 or 128 channels (windows (3,3,3) and (2,2,2) in one
score tile; (3,5,5) and (3,7,7) plane by plane), the general kernel with a NULL offsets tensor
for everything else.  The oracle is run with an all-zero
offsets tensor."""
import os

import pytest
import torch

import oracle
from paper_2607_22696_b200 import binding, inputs

import parity_util as pu

pytestmark = pytest.mark.gpu

BF16, F32 = torch.bfloat16, torch.float32


def _case(shape, window, dtype, seed, sigma_q=1.0):
    T, H, W, heads, d = shape
    q, k, v = (inputs.normal(shape, seed, i, sigma_q if i == 0 else 1.0, dtype) for i in range(3))
    P = window[0] * window[1] * window[2]
    zeros = torch.zeros(T * H * W, heads, P, 3, dtype=F32)
    ref_out, ref_lse = oracle.forward(q.view(-1, heads, d), k, v, zeros, T, H, W, heads, d, window)
    out = torch.full(shape, float("nan"), dtype=dtype, device="cuda")
    lse = torch.full((T, H, W, heads), float("nan"), dtype=F32, device="cuda")
    guard = torch.full((64,), 5.0, dtype=F32, device="cuda")
    binding.dsa3d_forward_fixed_window(q.cuda(), k.cuda(), v.cuda(), T, H, W, heads, d, window, out, lse)
    torch.cuda.synchronize()
    assert binding.dsa3d_device_timeout_flag() == 0
    pu.assert_close("out", out, ref_out.view(shape), dtype)
    pu.assert_close("lse", lse, ref_lse.view(T, H, W, heads), dtype)
    assert torch.equal(guard.cpu(), torch.full((64,), 5.0))
    return q, k, v, out, lse


@pytest.mark.parametrize("shape", [(6, 9, 13, 2, 128), (4, 4, 8, 1, 128), (1, 1, 1, 1, 128), (9, 5, 17, 3, 128),
                                   (2, 13, 7, 2, 128), (6, 9, 13, 2, 64), (5, 4, 19, 3, 64), (1, 2, 3, 1, 64)])
@pytest.mark.parametrize("window", [(3, 3, 3), (2, 2, 2)])
def test_tensor_core_tile_kernel_matches_the_oracle(shape, window):
    """Grids that are not multiples of the 4 x 4 x 8 tile, a grid smaller than one tile, a
    single token (every window cell but the centre is a dead sample with logit 0)."""
    _case(shape, window, BF16, 140)


@pytest.mark.parametrize("shape", [(6, 9, 13, 2, 128), (4, 4, 8, 1, 128), (1, 1, 1, 1, 128), (9, 5, 17, 3, 128),
                                   (2, 13, 7, 2, 128), (8, 8, 16, 2, 64), (5, 4, 19, 3, 64), (1, 2, 3, 1, 64)])
@pytest.mark.parametrize("window", [(3, 5, 5), (3, 7, 7)])
def test_plane_by_plane_tensor_core_kernel_matches_the_oracle(shape, window):
    """Windows (3,5,5) and the paper's (3,7,7): scores and weighted sum both on the tensor cores,
    the halo region taken one plane at a time.  Grids that are not multiples of the tile, smaller
    than one tile, a single token (all but the centre cell dead), several tiles per CTA."""
    _case(shape, window, BF16, 144)


@pytest.mark.parametrize("window", [(3, 5, 5), (3, 7, 7)])
def test_plane_kernel_sharp_softmax_many_tiles_and_agreement_with_the_general_kernel(window):
    """One dominant key per query (weights close to 1 and close to 0 next to each other: the bf16
    head/remainder split of the weights must hold), on a grid of several hundred tiles so that
    every CTA walks through many of them; then the same problem through the general kernel."""
    shape = (12, 20, 40, 4, 128)
    T, H, W, heads, d = shape
    q, k, v, out_tc, lse_tc = _case(shape, window, BF16, 145, sigma_q=5.0)
    os.environ["DSA3D_NO_TENSOR_FIXED_WINDOW"] = "1"
    try:
        out_g, lse_g = torch.empty_like(out_tc), torch.empty_like(lse_tc)
        binding.dsa3d_forward_fixed_window(q.cuda(), k.cuda(), v.cuda(), T, H, W, heads, d, window, out_g, lse_g)
        torch.cuda.synchronize()
    finally:
        del os.environ["DSA3D_NO_TENSOR_FIXED_WINDOW"]
    assert float((lse_tc - lse_g).abs().max()) <= 1e-4
    ulp = (out_g.float().abs() * 2.0 ** -7).clamp_min(2e-3)
    assert bool(((out_tc.float() - out_g.float()).abs() <= ulp).all())      # within one bf16 step of each other


def test_sharp_softmax_and_border_samples():
    """Large logits (one key dominates) next to rows at the border whose dead samples hold
    logit 0 in the softmax."""
    _case((5, 6, 9, 2, 128), (3, 3, 3), BF16, 141, sigma_q=6.0)


@pytest.mark.parametrize("shape,window,dtype", [((4, 6, 7, 2, 32), (3, 3, 3), BF16), ((3, 5, 6, 2, 32), (3, 3, 3), F32),
                                                ((4, 6, 9, 2, 128), (5, 5, 5), BF16), ((4, 6, 9, 2, 128), (1, 3, 3), BF16),
                                                ((4, 6, 9, 2, 32), (3, 5, 5), BF16)])
def test_other_shapes_run_the_general_kernel_without_an_offsets_tensor(shape, window, dtype):
    _case(shape, window, dtype, 142)


def test_tile_kernel_agrees_with_the_general_kernel_on_zero_offsets():
    """Same problem through the tile kernel, through the general kernel forced by the
    environment switch, and through dsa3d_forward with a zero offsets tensor."""
    shape, window = (8, 10, 20, 3, 128), (3, 3, 3)
    T, H, W, heads, d = shape
    q, k, v, out_tc, lse_tc = _case(shape, window, BF16, 143)
    dq, dk, dv = q.cuda(), k.cuda(), v.cuda()
    os.environ["DSA3D_NO_TENSOR_FIXED_WINDOW"] = "1"
    try:
        out_g, lse_g = torch.empty_like(out_tc), torch.empty_like(lse_tc)
        binding.dsa3d_forward_fixed_window(dq, dk, dv, T, H, W, heads, d, window, out_g, lse_g)
    finally:
        del os.environ["DSA3D_NO_TENSOR_FIXED_WINDOW"]
    zeros = torch.zeros(T, H, W, heads, 27, 3, dtype=F32, device="cuda")
    out_z, lse_z = torch.empty_like(out_tc), torch.empty_like(lse_tc)
    binding.dsa3d_forward(dq, dk, dv, zeros, T, H, W, heads, d, window, out_z, lse_z)
    torch.cuda.synchronize()
    assert torch.equal(out_g, out_z) and torch.equal(lse_g, lse_z)          # same kernel, same arithmetic
    assert float((lse_tc - lse_z).abs().max()) <= 1e-4
    ulp = (out_z.float().abs() * 2.0 ** -7).clamp_min(1e-3)
    assert bool(((out_tc.float() - out_z.float()).abs() <= ulp).all())      # within one bf16 step of each other


# ------------------------------------------------------------------ fixed-window backward

def _backward_case(shape, window, dtype, seed, with_doffsets=True):
    T, H, W, heads, d = shape
    P = window[0] * window[1] * window[2]
    q, k, v = (inputs.normal(shape, seed, i, 1.0, dtype) for i in range(3))
    dout = inputs.normal(shape, seed, 4, 1.0, dtype)
    zeros = torch.zeros(T * H * W, heads, P, 3, dtype=F32)
    _, ref_lse = oracle.forward(q.view(-1, heads, d), k, v, zeros, T, H, W, heads, d, window)
    ref = oracle.backward(q.view(-1, heads, d), k, v, zeros, dout.view(-1, heads, d), T, H, W, heads, d, window)
    dq_, dk_, dv_, dout_ = (z.cuda() for z in (q, k, v, dout))
    out = torch.empty(shape, dtype=dtype, device="cuda")
    lse = torch.empty((T, H, W, heads), dtype=F32, device="cuda")
    binding.dsa3d_forward_fixed_window(dq_, dk_, dv_, T, H, W, heads, d, window, out, lse)
    g = [torch.full(shape, float("nan"), dtype=dtype, device="cuda") for _ in range(3)]
    doff = torch.full((T, H, W, heads, P, 3), float("nan"), dtype=F32, device="cuda") if with_doffsets else None
    ws = torch.full((binding.dsa3d_backward_fixed_window_workspace_bytes(T, H, W, heads, d, window, dtype),), 0xFF,
                    dtype=torch.uint8, device="cuda")
    guard = torch.full((64,), 9.0, dtype=F32, device="cuda")
    binding.dsa3d_backward_fixed_window(dq_, dk_, dv_, lse, dout_, T, H, W, heads, d, window, g[0], g[1], g[2], doff, ws)
    torch.cuda.synchronize()
    pu.assert_close("lse", lse, ref_lse.view(T, H, W, heads), dtype)
    for name, got, want in zip(("dq", "dk", "dv"), g, ref[:3]):
        pu.assert_close(name, got, want.view(shape), dtype, backward=True)
    if with_doffsets:
        pu.assert_close("doffsets", doff, ref[3].view(T, H, W, heads, P, 3), dtype, backward=True)
    assert torch.equal(guard.cpu(), torch.full((64,), 9.0))
    return (dq_, dk_, dv_, dout_, lse), g, doff


@pytest.mark.parametrize("shape,window,dtype", [
    ((6, 9, 13, 2, 128), (3, 3, 3), BF16), ((4, 5, 6, 2, 64), (3, 3, 3), BF16), ((3, 5, 6, 2, 32), (3, 3, 3), F32),
    ((5, 6, 7, 2, 128), (2, 2, 2), BF16), ((4, 6, 9, 1, 64), (3, 5, 5), BF16), ((1, 1, 1, 1, 32), (3, 3, 3), F32),
    ((9, 10, 19, 2, 128), (3, 5, 5), BF16), ((4, 4, 8, 1, 128), (3, 5, 5), BF16), ((6, 13, 9, 3, 64), (3, 5, 5), BF16),
    ((9, 10, 19, 2, 128), (3, 7, 7), BF16), ((4, 4, 8, 1, 128), (3, 7, 7), BF16), ((6, 13, 9, 3, 64), (3, 7, 7), BF16),
    ((1, 2, 3, 1, 64), (3, 7, 7), BF16),
    ((2, 3, 4, 2, 32), (1, 1, 1), BF16), ((3, 8, 9, 2, 64), (1, 7, 7), F32), ((4, 4, 5, 3, 128), (5, 3, 1), F32)])
def test_fixed_window_backward_matches_the_oracle(shape, window, dtype):
    """Against the oracle on an all-zero offsets tensor: odd and even windows, windows that reach
    two positions outside the grid (dead samples), a single token, every dtype and head size."""
    _backward_case(shape, window, dtype, 150)


@pytest.mark.parametrize("shape,window", [((13, 22, 37, 3, 64), (3, 7, 7)), ((16, 21, 40, 3, 128), (3, 5, 5))])
def test_plane_gradient_kernel_over_several_tiles_per_block(shape, window):
    """More (tile, head) items than the GPU has SMs: every persistent block of the plane-by-plane gradient
    kernel walks several tiles, so its stream of planes, the rotation of its coefficient buffers and the
    clearing of cells between sweeps carry over from tile to tile."""
    T, H, W, heads, _ = shape
    assert ((T + 3) // 4) * ((H + 3) // 4) * ((W + 7) // 8) * heads > 2 * 148
    _backward_case(shape, window, BF16, 152)


def test_fixed_window_backward_without_doffsets_and_determinism():
    """doffsets may be NULL (only the window's own positions are visited then); dk and dv are
    gathered, not accumulated with atomics, so two runs agree bit for bit."""
    shape, window = (5, 7, 9, 2, 128), (3, 3, 3)
    T, H, W, heads, d = shape
    (q, k, v, dout, lse), g1, doff = _backward_case(shape, window, BF16, 151)
    (_, _, _, _, _), g0, none = _backward_case(shape, window, BF16, 151, with_doffsets=False)
    assert none is None
    for a, b in zip(g0, g1):
        assert torch.equal(a, b)
    g2 = [torch.empty_like(z) for z in g1]
    ws = torch.empty((binding.dsa3d_backward_fixed_window_workspace_bytes(T, H, W, heads, d, window, BF16),),
                     dtype=torch.uint8, device="cuda")
    doff2 = torch.empty_like(doff)
    binding.dsa3d_backward_fixed_window(q, k, v, lse, dout, T, H, W, heads, d, window, g2[0], g2[1], g2[2], doff2, ws)
    torch.cuda.synchronize()
    for a, b in zip(g1, g2):
        assert torch.equal(a, b)
    assert torch.equal(doff, doff2)


def test_fixed_window_backward_agrees_with_the_general_backward_on_zero_offsets():
    shape, window = (6, 8, 12, 2, 128), (3, 3, 3)
    T, H, W, heads, d = shape
    (q, k, v, dout, lse), g, doff = _backward_case(shape, window, BF16, 152)
    zeros = torch.zeros(T, H, W, heads, 27, 3, dtype=F32, device="cuda")
    gg = pu.gpu_backward(q, k, v, zeros, lse, dout, shape, window)
    for name, a, b in zip(("dq", "dk", "dv"), g, gg[:3]):
        step = (b.float().abs() * 2.0 ** -7).clamp_min(2e-3)
        assert bool(((a.float() - b.float()).abs() <= step).all()), name
    assert float((doff - gg[3]).abs().max()) <= 1e-4 * max(1.0, float(gg[3].abs().max()))


def test_fixed_window_entry_points_agree_with_the_general_kernels_at_a_larger_size():
    """57,600 tokens x 4 heads (450 tiles per head, several per persistent CTA, ragged in y):
    forward and backward through the fixed-window entry points against the general kernels on
    a zero offsets tensor; every element within one bf16 step."""
    shape, window = (16, 45, 80, 4, 128), (3, 3, 3)
    T, H, W, heads, d = shape
    q, k, v = (inputs.normal(shape, 160, i, 1.0, BF16, device="cuda") for i in range(3))
    dout = inputs.normal(shape, 160, 4, 1.0, BF16, device="cuda")
    zeros = torch.zeros(T, H, W, heads, 27, 3, dtype=F32, device="cuda")
    out_g, lse_g = pu.gpu_forward(q, k, v, zeros, shape, window)
    g_g = pu.gpu_backward(q, k, v, zeros, lse_g, dout, shape, window)
    out_f, lse_f = torch.empty_like(out_g), torch.empty_like(lse_g)
    binding.dsa3d_forward_fixed_window(q, k, v, T, H, W, heads, d, window, out_f, lse_f)
    g_f = [torch.empty_like(q) for _ in range(3)]
    doff_f = torch.empty_like(zeros)
    ws = torch.empty((binding.dsa3d_backward_fixed_window_workspace_bytes(T, H, W, heads, d, window, BF16),),
                     dtype=torch.uint8, device="cuda")
    binding.dsa3d_backward_fixed_window(q, k, v, lse_f, dout, T, H, W, heads, d, window, g_f[0], g_f[1], g_f[2], doff_f, ws)
    torch.cuda.synchronize()
    assert binding.dsa3d_device_timeout_flag() == 0
    assert float((lse_f - lse_g).abs().max()) <= 1e-4
    for name, a, b in zip(("out", "dq", "dk", "dv"), [out_f] + g_f, [out_g] + list(g_g[:3])):
        step = (b.float().abs() * 2.0 ** -7).clamp_min(4e-3)
        assert bool(((a.float() - b.float()).abs() <= step).all()), name
    assert float((doff_f - g_g[3]).abs().max()) <= 2e-4 * max(1.0, float(g_g[3].abs().max()))
