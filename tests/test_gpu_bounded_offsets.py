"""dsa3d_forward_bounded_offsets: the forward for learned offsets that are small perturbations of the
fixed window.  When every offset component is finite and below 1 in size the operator runs as dense
tile attention on the tensor cores (logits = trilinear combinations of entries of the Q.K^T tile,
weighted sum as a second tcgen05 product); otherwise the general kernel runs.  Both roads are
compared with the CPU oracle on the same offsets, element by element."""
import os

import pytest
import torch

import oracle
import parity_util as pu
from paper_2607_22696_b200 import binding, inputs

pytestmark = pytest.mark.gpu
BF16, F32 = torch.bfloat16, torch.float32


def _bounded_offsets(shape, seed, kind):
    """Offsets with |component| < 1: uniform in (-1, 1), tiny, zero, or pushed against the bound."""
    n = 1
    for x in shape:
        n *= x
    g = torch.Generator().manual_seed(seed)
    if kind == "uniform":
        off = torch.rand(n, generator=g, dtype=torch.float64) * 2 - 1
        off = off.clamp(-0.999999, 0.999999).to(F32)
    elif kind == "tiny":
        off = ((torch.rand(n, generator=g, dtype=torch.float64) * 2 - 1) * 1e-3).to(F32)
    elif kind == "zero":
        off = torch.zeros(n, dtype=F32)
    elif kind == "edge":                      # values next to -1, 0 and +1, where the cell of a sample changes
        pick = torch.randint(0, 6, (n,), generator=g)
        table = torch.tensor([-0.99999994, -1e-7, 0.0, 1e-7, 0.99999994, 0.5], dtype=F32)
        off = table[pick]
    else:
        raise ValueError(kind)
    assert float(off.abs().max()) < 1.0
    return off.view(shape)


def _run(shape, window, dtype, seed, offsets, sigma_q=1.0):
    T, H, W, heads, d = shape
    q, k, v = (inputs.normal(shape, seed, i, sigma_q if i == 0 else 1.0, dtype) for i in range(3))
    out = torch.full(shape, float("nan"), dtype=dtype, device="cuda")
    lse = torch.full((T, H, W, heads), float("nan"), dtype=F32, device="cuda")
    binding.dsa3d_forward_bounded_offsets(q.cuda(), k.cuda(), v.cuda(), offsets.cuda(), T, H, W, heads, d, window, out, lse)
    torch.cuda.synchronize()
    assert binding.dsa3d_device_timeout_flag() == 0
    P = window[0] * window[1] * window[2]
    o_ref, l_ref = oracle.forward(q.view(-1, heads, d), k, v, offsets.view(-1, heads, P, 3), T, H, W, heads, d, window)
    pu.assert_close("out", out, o_ref.view(shape), dtype)
    pu.assert_close("lse", lse, l_ref.view(T, H, W, heads), dtype)
    return q, k, v, out, lse


@pytest.mark.parametrize("shape", [(6, 9, 13, 2, 128), (4, 4, 8, 1, 128), (1, 1, 1, 1, 128), (9, 5, 17, 3, 128),
                                   (2, 13, 7, 2, 128), (8, 8, 16, 2, 64), (5, 4, 19, 3, 64)])
@pytest.mark.parametrize("kind", ["uniform", "edge"])
def test_tile_kernel_for_offsets_below_one_matches_the_oracle(shape, kind):
    T, H, W, heads, d = shape
    off = _bounded_offsets((T, H, W, heads, 27, 3), 700 + T * W, kind)
    _run(shape, (3, 3, 3), BF16, 170, off)


@pytest.mark.parametrize("kind", ["tiny", "zero"])
def test_tile_kernel_many_tiles_sharp_softmax(kind):
    shape = (12, 20, 40, 4, 128)
    T, H, W, heads, d = shape
    off = _bounded_offsets((T, H, W, heads, 27, 3), 710, kind)
    _run(shape, (3, 3, 3), BF16, 171, off, sigma_q=5.0)


def test_the_two_roads_agree_and_one_large_offset_switches_to_the_general_kernel():
    """The same bounded problem through the tile kernel and through the general kernel (forced by the
    environment switch): within one bf16 step of each other.  Then a single offset of size 1.5, a NaN
    and an infinity: the device-side check must send the whole call to the general kernel, whose result
    is dsa3d_forward's bit for bit."""
    shape, window = (8, 10, 20, 3, 128), (3, 3, 3)
    T, H, W, heads, d = shape
    off = _bounded_offsets((T, H, W, heads, 27, 3), 720, "uniform")
    q, k, v, out_tc, lse_tc = _run(shape, window, BF16, 172, off)
    dq, dk, dv = q.cuda(), k.cuda(), v.cuda()
    os.environ["DSA3D_NO_TENSOR_FIXED_WINDOW"] = "1"
    try:
        out_g, lse_g = torch.empty_like(out_tc), torch.empty_like(lse_tc)
        binding.dsa3d_forward_bounded_offsets(dq, dk, dv, off.cuda(), T, H, W, heads, d, window, out_g, lse_g)
        torch.cuda.synchronize()
    finally:
        del os.environ["DSA3D_NO_TENSOR_FIXED_WINDOW"]
    assert float((lse_tc - lse_g).abs().max()) <= 1e-4
    ulp = (out_g.float().abs() * 2.0 ** -7).clamp_min(2e-3)
    assert bool(((out_tc.float() - out_g.float()).abs() <= ulp).all())
    for bad in (1.5, float("nan"), float("inf"), -1.0):
        off2 = off.clone()
        off2.view(-1)[off2.numel() // 2 + 1] = bad
        out_a, lse_a = torch.full_like(out_tc, float("nan")), torch.full_like(lse_tc, float("nan"))
        out_b, lse_b = torch.empty_like(out_tc), torch.empty_like(lse_tc)
        binding.dsa3d_forward_bounded_offsets(dq, dk, dv, off2.cuda(), T, H, W, heads, d, window, out_a, lse_a)
        binding.dsa3d_forward(dq, dk, dv, off2.cuda(), T, H, W, heads, d, window, out_b, lse_b)
        torch.cuda.synchronize()
        assert torch.equal(out_a, out_b) and torch.equal(lse_a, lse_b), bad


@pytest.mark.parametrize("shape,window,dtype", [((4, 6, 7, 2, 32), (3, 3, 3), BF16), ((3, 5, 6, 2, 32), (3, 3, 3), F32),
                                                ((4, 6, 9, 2, 128), (2, 2, 2), BF16), ((4, 6, 9, 2, 64), (3, 5, 5), BF16)])
def test_other_shapes_take_the_general_kernel(shape, window, dtype):
    T, H, W, heads, d = shape
    P = window[0] * window[1] * window[2]
    off = _bounded_offsets((T, H, W, heads, P, 3), 730, "uniform")
    _run(shape, window, dtype, 173, off)


# ------------------------------------------------------------------------------------------------
# dsa3d_backward_bounded_offsets: dot-product tables on the tensor cores, per-sample arithmetic from
# the tables, dq / dk / dv as the sums of a fixed 5 x 5 x 5 window on the tensor cores
# ------------------------------------------------------------------------------------------------
def _run_backward(shape, window, dtype, seed, offsets, sigma_q=1.0, entry=None):
    T, H, W, heads, d = shape
    P = window[0] * window[1] * window[2]
    q, k, v, dout = (inputs.normal(shape, seed, i, sigma_q if i == 0 else 1.0, dtype) for i in range(4))
    dev = [z.cuda() for z in (q, k, v, offsets, dout)]
    out, lse = pu.gpu_forward(*dev[:4], shape, window)
    grads = [torch.full(shape, float("nan"), dtype=dtype, device="cuda") for _ in range(3)]
    doff = torch.full((T, H, W, heads, P, 3), float("nan"), dtype=F32, device="cuda")
    nbytes = binding.dsa3d_backward_bounded_offsets_workspace_bytes(T, H, W, heads, d, window, dtype)
    ws = torch.full((nbytes + 64,), 0xA5, dtype=torch.uint8, device="cuda")       # poisoned, with a guard band behind it
    call = entry or binding.dsa3d_backward_bounded_offsets
    call(dev[0], dev[1], dev[2], dev[3], lse, dev[4], T, H, W, heads, d, window, grads[0], grads[1], grads[2], doff,
         ws[:nbytes] if nbytes else None, nbytes)
    torch.cuda.synchronize()
    assert binding.dsa3d_device_timeout_flag() == 0
    assert torch.equal(ws[nbytes:].cpu(), torch.full((64,), 0xA5, dtype=torch.uint8))
    refs = oracle.backward(q, k, v, offsets, dout, T, H, W, heads, d, window)
    for name, got, ref in zip(("dq", "dk", "dv", "doffsets"), (*grads, doff), refs):
        pu.assert_close(name, got, ref, dtype, backward=True)
    return dev, lse, grads, doff


@pytest.mark.parametrize("shape", [(6, 9, 13, 2, 128), (4, 4, 8, 1, 128), (1, 1, 1, 1, 128), (9, 5, 17, 3, 128),
                                   (2, 13, 7, 2, 128), (8, 8, 16, 2, 64), (5, 4, 19, 3, 64)])
@pytest.mark.parametrize("kind", ["uniform", "edge"])
def test_backward_tile_kernels_for_offsets_below_one_match_the_oracle(shape, kind):
    T, H, W, heads, d = shape
    off = _bounded_offsets((T, H, W, heads, 27, 3), 740 + T * W, kind)
    _run_backward(shape, (3, 3, 3), BF16, 174, off)


@pytest.mark.parametrize("kind", ["tiny", "zero", "uniform"])
def test_backward_tile_kernels_many_tiles_per_block(kind):
    """More (tile, head) items than SMs, a sharp softmax: the persistent blocks walk several tiles."""
    shape = (12, 20, 40, 4, 128)
    T, H, W, heads, d = shape
    off = _bounded_offsets((T, H, W, heads, 27, 3), 750, kind)
    _run_backward(shape, (3, 3, 3), BF16, 175, off, sigma_q=3.0)


def test_backward_roads_agree_and_one_large_offset_switches_to_the_general_kernels():
    """The bounded problem through the tile kernels and through dsa3d_backward: within a bf16 step of each
    other.  Then one offset of size 1.5, a NaN, an infinity, exactly -1: the device-side check must hand
    the whole call to the general kernels (which were queued behind the tile kernels), and dq and doffsets
    are dsa3d_backward's bit for bit, dk and dv up to the order of its atomic sums."""
    shape, window = (8, 10, 20, 3, 128), (3, 3, 3)
    T, H, W, heads, d = shape
    off = _bounded_offsets((T, H, W, heads, 27, 3), 760, "uniform")
    dev, lse, g_tc, doff_tc = _run_backward(shape, window, BF16, 176, off)
    g_gen = pu.gpu_backward(dev[0], dev[1], dev[2], dev[3], lse, dev[4], shape, window)
    for a, b in zip((*g_tc, doff_tc), g_gen):
        a, b = a.float(), b.float()
        step = (b.abs() * 2.0 ** -7).clamp_min(float(b.pow(2).mean().sqrt()) * 2.0 ** -7)
        assert bool(((a - b).abs() <= step).all())
    nbytes = binding.dsa3d_backward_bounded_offsets_workspace_bytes(T, H, W, heads, d, window, BF16)
    ws = torch.empty((nbytes,), dtype=torch.uint8, device="cuda")
    for bad in (1.5, float("nan"), float("inf"), -1.0):
        off2 = off.clone()
        off2.view(-1)[off2.numel() // 2 + 1] = bad
        o2 = off2.cuda()
        _, lse2 = pu.gpu_forward(dev[0], dev[1], dev[2], o2, shape, window)
        ga = [torch.full(shape, float("nan"), dtype=BF16, device="cuda") for _ in range(3)]
        da = torch.full((T, H, W, heads, 27, 3), float("nan"), dtype=F32, device="cuda")
        binding.dsa3d_backward_bounded_offsets(dev[0], dev[1], dev[2], o2, lse2, dev[4], T, H, W, heads, d, window,
                                               ga[0], ga[1], ga[2], da, ws, nbytes)
        gb = pu.gpu_backward(dev[0], dev[1], dev[2], o2, lse2, dev[4], shape, window)
        torch.cuda.synchronize()
        for a, b in ((ga[0], gb[0]), (da, gb[3])):          # per-query results: the same kernel, the same bits
            assert bool(((a == b) | (torch.isnan(a) & torch.isnan(b))).all()), bad
        for a, b in ((ga[1], gb[1]), (ga[2], gb[2])):
            fa, fb = a.float(), b.float()
            finite = torch.isfinite(fb)
            assert torch.equal(torch.isfinite(fa), finite)
            step = (fb[finite].abs() * 2.0 ** -7).clamp_min(2e-3)
            assert bool(((fa[finite] - fb[finite]).abs() <= step).all()), bad


@pytest.mark.parametrize("shape,window,dtype", [((4, 6, 7, 2, 32), (3, 3, 3), BF16), ((3, 5, 6, 2, 32), (3, 3, 3), F32),
                                                ((4, 6, 9, 2, 128), (2, 2, 2), BF16), ((4, 6, 9, 2, 64), (3, 5, 5), BF16)])
def test_backward_other_shapes_take_the_general_kernels(shape, window, dtype):
    T, H, W, heads, d = shape
    P = window[0] * window[1] * window[2]
    off = _bounded_offsets((T, H, W, heads, P, 3), 770, "uniform")
    _run_backward(shape, window, dtype, 177, off)


def test_two_calls_in_flight_on_two_streams_do_not_share_a_gate():
    """One call whose offsets pass the check and one whose offsets do not, queued on two streams before either
    has run: each takes its own gate word, so each must equal the same call made alone."""
    shape, window = (8, 12, 24, 2, 128), (3, 3, 3)
    T, H, W, heads, d = shape
    off_ok = _bounded_offsets((T, H, W, heads, 27, 3), 780, "uniform")
    off_big = off_ok.clone()
    off_big.view(-1)[7::101] = 2.5
    q, k, v, dout = (inputs.normal(shape, 178, i, 1.0, BF16).cuda() for i in range(4))
    nbytes = binding.dsa3d_backward_bounded_offsets_workspace_bytes(T, H, W, heads, d, window, BF16)

    def run(off, stream):
        out = torch.empty(shape, dtype=BF16, device="cuda")
        lse = torch.empty((T, H, W, heads), dtype=F32, device="cuda")
        g = [torch.empty(shape, dtype=BF16, device="cuda") for _ in range(3)]
        doff = torch.empty((T, H, W, heads, 27, 3), dtype=F32, device="cuda")
        ws = torch.empty((nbytes,), dtype=torch.uint8, device="cuda")
        with torch.cuda.stream(stream):
            binding.dsa3d_forward_bounded_offsets(q, k, v, off, T, H, W, heads, d, window, out, lse, stream=stream)
            binding.dsa3d_backward_bounded_offsets(q, k, v, off, lse, dout, T, H, W, heads, d, window, g[0], g[1], g[2], doff, ws,
                                                   stream=stream)
        return out, lse, g, doff, ws

    offs = [off_ok.cuda(), off_big.cuda()]
    torch.cuda.synchronize()
    alone = []
    for off in offs:
        alone.append(run(off, torch.cuda.current_stream()))
        torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    together = [run(offs[0], s1), run(offs[1], s2)]
    torch.cuda.synchronize()
    assert binding.dsa3d_device_timeout_flag() == 0
    for a, b in zip(alone, together):
        assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])               # out, lse
        assert torch.equal(a[2][0], b[2][0]) and torch.equal(a[3], b[3])         # dq, doffsets
    # the tile route writes dk and dv without atomics: bit for bit; the general route up to the order of its sums
    for i in (1, 2):
        assert torch.equal(alone[0][2][i], together[0][2][i])
        fa, fb = alone[1][2][i].float(), together[1][2][i].float()
        assert bool(((fa - fb).abs() <= (fb.abs() * 2.0 ** -7).clamp_min(2e-3)).all())
