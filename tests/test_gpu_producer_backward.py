"""GPU parity of the backward passes of the layers around the operator in Eq. 1: gradients of
the depthwise 3-D convolution (input, weights, bias) and of the offset-producing linear layer
(input, weights, bias; tensor-core contractions for bf16).  Every case has its own seeded
inputs; the expected values come from the fp64 oracle only."""
import pytest
import torch

from oracle import producer
from paper_2607_22696_b200 import binding, inputs

import parity_util as pu

pytestmark = pytest.mark.gpu

BF16, F32 = torch.bfloat16, torch.float32


def _normal(shape, seed, tid, sigma, dtype):
    return inputs.normal(shape, seed, tid, sigma, dtype)


def _sum_close(name, got, ref, rel):
    """fp32 sums of exact products: the error scales with the size of the sums."""
    got = got.detach().cpu().double()
    assert torch.isfinite(got).all(), name
    scale = max(float(ref.pow(2).mean().sqrt()), 1.0)
    worst = float((got - ref).abs().max())
    assert worst <= rel * scale, f"{name}: max abs error {worst:.3e} > {rel * scale:.3e}"


def _workspace(nbytes):
    return torch.empty(max(nbytes, 16), dtype=torch.uint8, device="cuda")


@pytest.mark.parametrize("dtype", [BF16, F32])
@pytest.mark.parametrize("shape,kernel", [((5, 7, 9, 16), (3, 3, 3)), ((3, 4, 13, 24), (1, 5, 3)),
                                          ((4, 5, 6, 8), (2, 2, 2)), ((3, 9, 10, 32), (3, 7, 7)),
                                          ((1, 1, 1, 8), (3, 3, 3)), ((2, 3, 2, 8), (5, 1, 7)),
                                          ((3, 4, 5, 72), (2, 4, 6)),
                                          ((6, 7, 19, 64), (3, 3, 3)), ((40, 6, 17, 64), (2, 4, 3)),
                                          ((5, 9, 33, 128), (3, 7, 7)), ((70, 3, 5, 64), (3, 3, 1)),
                                          ((48, 4, 16, 64), (3, 3, 3)), ((9, 10, 35, 128), (3, 3, 3)),
                                          ((1, 1, 1, 64), (3, 3, 3)), ((2, 5, 17, 192), (3, 3, 3))])
def test_dwconv3d_backward_matches_the_oracle(dtype, shape, kernel):
    """Odd, even and mixed kernel sizes (the flipped kernel's centre differs from the forward's
    for even sizes), widths with and without a compiled-in slide, channel counts that take the
    staged kernels (bf16, multiples of 64 channels; the 3 x 3 x 3 weight gradient has one of its
    own, here with grids that are not multiples of its 4 x 16 tile, a single frame, and enough
    frames that the march is cut into chunks) and ones that do not, more grid rows than one
    warp's chunk."""
    T, H, W, C = shape
    taps = kernel[0] * kernel[1] * kernel[2]
    x = _normal(shape, 300, 0, 1.0, dtype)
    w = _normal((taps, C), 300, 1, 0.3, F32)
    dy = _normal(shape, 300, 2, 1.0, dtype)
    ref_dx, ref_dw, ref_db = producer.dwconv3d_backward(x, w, dy, kernel)
    dx = torch.full(shape, float("nan"), dtype=dtype, device="cuda")
    dw = torch.full((taps, C), float("nan"), dtype=F32, device="cuda")
    db = torch.full((C,), float("nan"), dtype=F32, device="cuda")
    ws = _workspace(binding.dsa3d_dwconv3d_backward_workspace_bytes(C, kernel))
    xd, wd, dyd = x.cuda(), w.cuda(), dy.cuda()
    binding.dsa3d_dwconv3d_backward(xd, wd, dyd, T, H, W, C, kernel, dx, dw, db, ws)
    torch.cuda.synchronize()
    assert binding.dsa3d_device_timeout_flag() == 0
    pu.assert_close("dx", dx, ref_dx, dtype, backward=True)
    _sum_close("dweight", dw, ref_dw, 1e-4)
    _sum_close("dbias", db, ref_db, 1e-4)
    # inputs untouched; each output can be left out
    assert torch.equal(xd.cpu(), x) and torch.equal(dyd.cpu(), dy) and torch.equal(wd.cpu(), w)
    dw2 = torch.full((taps, C), float("nan"), dtype=F32, device="cuda")
    binding.dsa3d_dwconv3d_backward(xd, None, dyd, T, H, W, C, kernel, None, dw2, None, None)
    dx2 = torch.full(shape, float("nan"), dtype=dtype, device="cuda")
    binding.dsa3d_dwconv3d_backward(None, wd, dyd, T, H, W, C, kernel, dx2, None, None, ws)
    torch.cuda.synchronize()
    _sum_close("dweight alone", dw2, ref_dw, 1e-4)
    assert torch.equal(dx2, dx)


@pytest.fixture(params=["tma_stores", "plain_stores"])
def store_variant(request):
    """du leaves the contraction by TMA stores (default) or by plain stores (environment switch
    read at every call)."""
    import os
    if request.param == "plain_stores":
        os.environ["DSA3D_GEMM_PLAIN_STORES"] = "1"
    yield request.param
    os.environ.pop("DSA3D_GEMM_PLAIN_STORES", None)


@pytest.mark.parametrize("tokens,C,O", [(300, 192, 162), (128, 64, 32), (1000, 256, 1296), (77, 200, 40),
                                        (513, 128, 520), (1, 8, 1), (260, 2048, 81), (2500, 72, 300)])
def test_offsets_linear_backward_bf16_on_tensor_cores(tokens, C, O, store_variant):
    """Ragged sizes on every axis: output counts that are not a multiple of 8 (padded row
    pitch of the transposed copies), token counts that are not a multiple of the 64-token
    k-block, one and several column tiles, k-ranges split over several CTA pairs.  doffsets is
    rounded to bf16 once (2^-9 relative per element), hence the bf16 bound on du and dw; dbias
    is summed in fp32 from the unrounded values."""
    u = _normal((tokens, C), 310, 0, 1.0, BF16)
    w = _normal((O, C), 310, 1, 0.2, BF16)
    g = _normal((tokens, O), 310, 2, 0.5, F32)
    ref_du, ref_dw, ref_db = producer.offsets_linear_backward(u, w, g)
    du = torch.full((tokens, C), float("nan"), dtype=BF16, device="cuda")
    dw = torch.full((O, C), float("nan"), dtype=F32, device="cuda")
    db = torch.full((O,), float("nan"), dtype=F32, device="cuda")
    guard = torch.full((64,), 7.0, dtype=F32, device="cuda")
    ws = _workspace(binding.dsa3d_offsets_linear_backward_workspace_bytes(tokens, C, O, BF16))
    ud, wd, gd = u.cuda(), w.cuda(), g.cuda()
    binding.dsa3d_offsets_linear_backward(ud, wd, gd, tokens, C, O, du, dw, db, ws)
    torch.cuda.synchronize()
    assert binding.dsa3d_device_timeout_flag() == 0
    pu.assert_close("du", du, ref_du, BF16, backward=True)
    pu.assert_close("dw", dw, ref_dw, BF16, backward=True)
    _sum_close("dbias", db, ref_db, 1e-5)
    assert torch.equal(guard.cpu(), torch.full((64,), 7.0))
    assert torch.equal(ud.cpu(), u) and torch.equal(wd.cpu(), w) and torch.equal(gd.cpu(), g)
    # a second call gives the same du (deterministic) and dw within summation-order noise
    du2 = torch.empty_like(du)
    dw2 = torch.empty_like(dw)
    binding.dsa3d_offsets_linear_backward(ud, wd, gd, tokens, C, O, du2, dw2, None, ws)
    torch.cuda.synchronize()
    assert torch.equal(du2, du)
    _sum_close("dw again", dw2, dw.cpu().double(), 1e-5)


def test_offsets_linear_backward_over_several_token_slabs():
    """More tokens than one slab of the backward (262144): du is written slab by slab, dw and
    dbias accumulate over the slabs, and the last slab is short and ragged."""
    tokens, C, O = 262144 * 2 + 1000 + 3, 64, 40
    u = _normal((tokens, C), 311, 0, 1.0, BF16)
    w = _normal((O, C), 311, 1, 0.2, BF16)
    g = _normal((tokens, O), 311, 2, 0.5, F32)
    ref_du, ref_dw, ref_db = producer.offsets_linear_backward(u, w, g)
    du = torch.full((tokens, C), float("nan"), dtype=BF16, device="cuda")
    dw = torch.full((O, C), float("nan"), dtype=F32, device="cuda")
    db = torch.full((O,), float("nan"), dtype=F32, device="cuda")
    ws = _workspace(binding.dsa3d_offsets_linear_backward_workspace_bytes(tokens, C, O, BF16))
    binding.dsa3d_offsets_linear_backward(u.cuda(), w.cuda(), g.cuda(), tokens, C, O, du, dw, db, ws)
    torch.cuda.synchronize()
    assert binding.dsa3d_device_timeout_flag() == 0
    pu.assert_close("du", du, ref_du, BF16, backward=True)
    pu.assert_close("dw", dw, ref_dw, BF16, backward=True)
    _sum_close("dbias", db, ref_db, 1e-4)


def test_offsets_linear_backward_fp32():
    tokens, C, O = 37, 24, 54
    u = _normal((tokens, C), 312, 0, 1.0, F32)
    w = _normal((O, C), 312, 1, 0.2, F32)
    g = _normal((tokens, O), 312, 2, 0.5, F32)
    ref_du, ref_dw, ref_db = producer.offsets_linear_backward(u, w, g)
    du = torch.empty((tokens, C), dtype=F32, device="cuda")
    dw = torch.empty((O, C), dtype=F32, device="cuda")
    db = torch.empty((O,), dtype=F32, device="cuda")
    binding.dsa3d_offsets_linear_backward(u.cuda(), w.cuda(), g.cuda(), tokens, C, O, du, dw, db, None)
    torch.cuda.synchronize()
    pu.assert_close("du", du, ref_du, F32, backward=True)
    pu.assert_close("dw", dw, ref_dw, F32, backward=True)
    pu.assert_close("dbias", db, ref_db, F32, backward=True)


def test_producer_backward_rejects_bad_arguments():
    x = torch.zeros(2, 2, 2, 8, dtype=BF16, device="cuda")
    w = torch.zeros(27, 8, dtype=F32, device="cuda")
    dw = torch.zeros(27, 8, dtype=F32, device="cuda")
    db = torch.zeros(8, dtype=F32, device="cuda")
    small = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.Dsa3dError):          # dx without a workspace
        binding.dsa3d_dwconv3d_backward(x, w, x, 2, 2, 2, 8, (3, 3, 3), torch.empty_like(x), None, None, None)
    with pytest.raises(binding.Dsa3dError):          # workspace too small
        binding.dsa3d_dwconv3d_backward(x, w, x, 2, 2, 2, 8, (3, 3, 3), torch.empty_like(x), None, None, small)
    with pytest.raises(binding.Dsa3dError):          # dbias without dweight
        binding.dsa3d_dwconv3d_backward(x, w, x, 2, 2, 2, 8, (3, 3, 3), None, None, db, None)
    with pytest.raises(binding.Dsa3dError):          # kernel wider than supported
        binding.dsa3d_dwconv3d_backward(x, None, x, 2, 2, 2, 8, (3, 3, 9), None,
                                        torch.zeros(81, 8, dtype=F32, device="cuda"), None, None)
    u = torch.zeros(16, 8, dtype=BF16, device="cuda")
    wl = torch.zeros(4, 8, dtype=BF16, device="cuda")
    g = torch.zeros(16, 4, dtype=F32, device="cuda")
    with pytest.raises(binding.Dsa3dError):          # bf16 needs its workspace
        binding.dsa3d_offsets_linear_backward(u, wl, g, 16, 8, 4, torch.empty_like(u), None, None, small)
    torch.cuda.synchronize()
