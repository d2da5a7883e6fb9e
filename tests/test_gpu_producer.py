"""GPU parity of the layers around the operator in Eq. 1: the depthwise 3-D convolution, the
linear layer that produces the offsets (tensor-core kernel for bf16) and the forward with the
convolution term added.  Each stage is compared on its own seeded inputs, never on another
stage's GPU output."""
import pytest
import torch

import oracle
from oracle import producer
from paper_2607_22696_b200 import binding, inputs

import parity_util as pu

pytestmark = pytest.mark.gpu

BF16, F32 = torch.bfloat16, torch.float32


def _normal(shape, seed, tid, sigma, dtype):
    return inputs.normal(shape, seed, tid, sigma, dtype)


@pytest.mark.parametrize("dtype", [BF16, F32])
@pytest.mark.parametrize("shape,kernel", [((5, 7, 9, 16), (3, 3, 3)), ((3, 4, 13, 24), (1, 5, 3)),
                                          ((4, 5, 6, 8), (2, 2, 2)), ((3, 9, 10, 32), (3, 7, 7)),
                                          ((1, 1, 1, 8), (3, 3, 3)), ((2, 3, 2, 8), (5, 1, 7))])
def test_dwconv3d_matches_the_oracle(dtype, shape, kernel):
    T, H, W, C = shape
    taps = kernel[0] * kernel[1] * kernel[2]
    x = _normal(shape, 100, 0, 1.0, dtype)
    w = _normal((taps, C), 100, 1, 0.3, F32)
    bias = _normal((C,), 100, 2, 0.5, F32)
    for b in (bias, None):
        ref = producer.dwconv3d(x, w, b, kernel)
        y = torch.full(shape, float("nan"), dtype=dtype, device="cuda")
        binding.dsa3d_dwconv3d_forward(x.cuda(), w.cuda(), None if b is None else b.cuda(), T, H, W, C, kernel, y)
        torch.cuda.synchronize()
        pu.assert_close("dwconv3d", y, ref, dtype)


@pytest.fixture(params=["default", "general"])
def conv_variant(request):
    """3 x 3 x 3 kernels take a kernel of their own by default (weights in registers); the
    general staged kernel is forced by an environment switch read at every call."""
    import os
    if request.param == "general":
        os.environ["DSA3D_CONV_GENERAL"] = "1"
    yield request.param
    os.environ.pop("DSA3D_CONV_GENERAL", None)


@pytest.mark.parametrize("shape,kernel", [((6, 7, 19, 64), (3, 3, 3)), ((48, 4, 16, 64), (3, 3, 3)),
                                          ((1, 1, 1, 64), (3, 3, 3)), ((9, 10, 35, 128), (3, 3, 3)),
                                          ((5, 9, 33, 128), (3, 7, 7)), ((4, 5, 6, 64), (1, 1, 1)),
                                          ((9, 3, 40, 192), (5, 3, 5)), ((2, 1, 1, 64), (7, 5, 7)),
                                          ((40, 6, 17, 64), (2, 4, 3))])
def test_dwconv3d_staged_kernel_matches_the_oracle(shape, kernel, conv_variant):
    """bf16 with a multiple of 64 channels takes the kernel that stages planes in shared
    memory with TMA and marches along t: grids that are not multiples of the 4 x 16 tile,
    fewer frames than kernel taps, even kernel sizes, and grids small enough that the march
    is cut into several chunks of frames (whose first planes are real data, not padding)."""
    T, H, W, C = shape
    taps = kernel[0] * kernel[1] * kernel[2]
    x = _normal(shape, 101, 0, 1.0, BF16)
    w = _normal((taps, C), 101, 1, 0.3, F32)
    bias = _normal((C,), 101, 2, 0.5, F32)
    ref = producer.dwconv3d(x, w, bias, kernel)
    y = torch.full(shape, float("nan"), dtype=BF16, device="cuda")
    guard = torch.full((64,), 3.0, dtype=F32, device="cuda")
    xd, wd, bd = x.cuda(), w.cuda(), bias.cuda()
    for _ in range(2):
        binding.dsa3d_dwconv3d_forward(xd, wd, bd, T, H, W, C, kernel, y)
    torch.cuda.synchronize()
    assert binding.dsa3d_device_timeout_flag() == 0
    pu.assert_close("dwconv3d", y, ref, BF16)
    assert torch.equal(guard.cpu(), torch.full((64,), 3.0))


@pytest.fixture(params=["pair", "pair_plain_stores", "one_cta"])
def gemm_variant(request):
    """The tilings of the tensor-core linear layer: pairs of CTAs with the epilogue leaving by
    TMA stores (the default; output counts that are not a multiple of 4 take plain stores by
    themselves), the same with plain stores forced, and one CTA per tile (environment switches
    read at every call)."""
    import os
    switch = {"one_cta": "DSA3D_GEMM_ONE_CTA", "pair_plain_stores": "DSA3D_GEMM_PLAIN_STORES"}.get(request.param)
    if switch:
        os.environ[switch] = "1"
    yield request.param
    if switch:
        os.environ.pop(switch, None)


@pytest.mark.parametrize("tokens,C,O", [(300, 192, 162), (128, 64, 32), (1000, 256, 1296), (77, 200, 40),
                                        (513, 128, 520), (1, 8, 1), (260, 2048, 81)])
def test_offsets_linear_bf16_on_tensor_cores(tokens, C, O, gemm_variant):
    """Ragged token counts, channel counts that are not a multiple of the 64-channel stage
    (zero-filled by the tile loads), one to six column tiles of 32 to 256 columns.  The
    products are exact and the accumulation is fp32 in the tensor core's own order, so the
    bound is a small multiple of fp32 accumulation error over C terms, relative to the size
    of the result."""
    u = _normal((tokens, C), 110, 0, 1.0, BF16)
    w = _normal((O, C), 110, 1, 0.2, BF16)
    bias = _normal((O,), 110, 2, 1.0, F32)
    ref = producer.offsets_linear(u, w, bias)
    out = torch.full((tokens, O), float("nan"), dtype=F32, device="cuda")
    guard = torch.full((64,), 7.0, dtype=F32, device="cuda")       # allocated right after: must stay intact
    binding.dsa3d_offsets_linear_forward(u.cuda(), w.cuda(), bias.cuda(), tokens, C, O, out)
    torch.cuda.synchronize()
    assert binding.dsa3d_device_timeout_flag() == 0
    binding.dsa3d_check_device_timeout()                       # the same as a status: raises on a timeout
    got = out.cpu().double()
    assert torch.isfinite(got).all()
    scale = float(ref.pow(2).mean().sqrt())
    assert float((got - ref).abs().max()) <= 1e-3 * max(scale, 1.0)
    assert torch.equal(guard.cpu(), torch.full((64,), 7.0))


def test_offsets_linear_twice_in_a_row_and_large(gemm_variant):
    """Two launches back to back on one stream (barrier phases and TMEM are per launch), on a
    problem with more tiles than SMs so that every CTA loops over several tiles and both
    accumulator buffers."""
    tokens, C, O = 148 * 128 * 3 + 5, 128, 300
    u = _normal((tokens, C), 111, 0, 1.0, BF16).cuda()
    w = _normal((O, C), 111, 1, 0.2, BF16).cuda()
    bias = _normal((O,), 111, 2, 1.0, F32).cuda()
    out1 = torch.empty((tokens, O), dtype=F32, device="cuda")
    out2 = torch.empty((tokens, O), dtype=F32, device="cuda")
    binding.dsa3d_offsets_linear_forward(u, w, bias, tokens, C, O, out1)
    binding.dsa3d_offsets_linear_forward(u, w, bias, tokens, C, O, out2)
    torch.cuda.synchronize()
    assert binding.dsa3d_device_timeout_flag() == 0
    assert torch.equal(out1, out2)
    rows = torch.tensor([0, 1, 127, 128, 5000, tokens // 2, tokens - 6, tokens - 1])
    ref = producer.offsets_linear(u[rows.cuda()].cpu(), w.cpu(), bias.cpu())
    assert float((out1[rows.cuda()].cpu().double() - ref).abs().max()) <= 1e-3 * max(float(ref.pow(2).mean().sqrt()), 1.0)


def test_offsets_linear_fp32():
    tokens, C, O = 37, 24, 54
    u = _normal((tokens, C), 112, 0, 1.0, F32)
    w = _normal((O, C), 112, 1, 0.2, F32)
    bias = _normal((O,), 112, 2, 1.0, F32)
    out = torch.empty((tokens, O), dtype=F32, device="cuda")
    binding.dsa3d_offsets_linear_forward(u.cuda(), w.cuda(), bias.cuda(), tokens, C, O, out)
    torch.cuda.synchronize()
    pu.assert_close("offsets", out, producer.offsets_linear(u, w, bias), F32)


def test_producer_rejects_bad_arguments():
    x = torch.zeros(2, 2, 2, 8, dtype=BF16, device="cuda")
    w = torch.zeros(27, 8, dtype=F32, device="cuda")
    with pytest.raises(binding.Dsa3dError):       # channels not a multiple of 8
        binding.dsa3d_dwconv3d_forward(torch.zeros(2, 2, 2, 4, dtype=BF16, device="cuda"),
                                       torch.zeros(27, 4, dtype=F32, device="cuda"), None, 2, 2, 2, 4, (3, 3, 3),
                                       torch.zeros(2, 2, 2, 4, dtype=BF16, device="cuda"))
    with pytest.raises(binding.Dsa3dError):       # kernel wider than supported along x
        binding.dsa3d_dwconv3d_forward(x, torch.zeros(27, 8, dtype=F32, device="cuda"), None, 2, 2, 2, 8, (1, 3, 9),
                                       torch.zeros_like(x))
    with pytest.raises(binding.Dsa3dError):       # bias is required by the linear layer
        binding.dsa3d_offsets_linear_forward(torch.zeros(4, 8, dtype=BF16, device="cuda"),
                                             torch.zeros(3, 8, dtype=BF16, device="cuda"), None, 4, 8, 3,
                                             torch.zeros(4, 3, dtype=F32, device="cuda"))
    del w


@pytest.mark.parametrize("dtype,d", [(BF16, 128), (BF16, 64), (F32, 32)])
def test_forward_with_the_convolution_term(dtype, d):
    """Eq. 1 with its first term: out = residual + attention, added in fp32 before the one
    rounding; also with the residual living in the output buffer."""
    T, H, W, heads, window = 4, 6, 7, 2, (3, 3, 3)
    shape = (T, H, W, heads, d)
    q, k, v = (_normal(shape, 120, i, 1.0, dtype) for i in range(3))
    off = _normal((T, H, W, heads, 27, 3), 120, 3, 1.2, F32)
    res = _normal(shape, 120, 5, 2.0, dtype)
    ref_out, ref_lse = oracle.forward(q.view(-1, heads, d), k, v, off.view(-1, heads, 27, 3), T, H, W, heads, d, window)
    ref_out = ref_out.view(shape) + res.double()
    dq, dk, dv, doff, dres = (z.cuda() for z in (q, k, v, off, res))
    out = torch.full(shape, float("nan"), dtype=dtype, device="cuda")
    lse = torch.empty((T, H, W, heads), dtype=F32, device="cuda")
    binding.dsa3d_forward_residual(dq, dk, dv, doff, dres, T, H, W, heads, d, window, out, lse)
    torch.cuda.synchronize()
    pu.assert_close("out", out, ref_out, dtype)
    pu.assert_close("lse", lse, ref_lse.view(T, H, W, heads), dtype)
    inplace = dres.clone()
    binding.dsa3d_forward_residual(dq, dk, dv, doff, inplace, T, H, W, heads, d, window, inplace, lse)
    torch.cuda.synchronize()
    assert torch.equal(inplace, out)


def test_offset_predictor_then_attention_runs_end_to_end():
    """Layer input -> depthwise convolution -> linear layer -> offsets -> attention with the
    convolution term, all through the library on one stream: shapes and layouts chain
    without any reshaping, every output is finite and no bounded wait ran out."""
    T, H, W, heads, d, window = 4, 6, 8, 2, 64, (3, 3, 3)
    C, O = heads * d, heads * 27 * 3
    x = _normal((T, H, W, C), 130, 0, 1.0, BF16).cuda()
    q, k, v = (_normal((T, H, W, heads, d), 130, i + 1, 1.0, BF16).cuda() for i in range(3))
    w_off_conv = _normal((27, C), 130, 4, 0.2, F32).cuda()
    w_lin = _normal((O, C), 130, 5, 0.05, BF16).cuda()
    b_lin = _normal((O,), 130, 6, 0.3, F32).cuda()
    w_term = _normal((27, C), 130, 7, 0.2, F32).cuda()
    u = torch.empty_like(x)
    binding.dsa3d_dwconv3d_forward(x, w_off_conv, None, T, H, W, C, (3, 3, 3), u)
    off = torch.empty((T, H, W, heads, 27, 3), dtype=F32, device="cuda")
    binding.dsa3d_offsets_linear_forward(u, w_lin, b_lin, T * H * W, C, O, off)
    term = torch.empty_like(x)
    binding.dsa3d_dwconv3d_forward(x, w_term, None, T, H, W, C, (3, 3, 3), term)
    out = torch.empty_like(q)
    lse = torch.empty((T, H, W, heads), dtype=F32, device="cuda")
    binding.dsa3d_forward_residual(q, k, v, off, term, T, H, W, heads, d, window, out, lse)
    torch.cuda.synchronize()
    assert binding.dsa3d_device_timeout_flag() == 0
    assert torch.isfinite(off).all() and torch.isfinite(out.float()).all() and torch.isfinite(lse).all()
