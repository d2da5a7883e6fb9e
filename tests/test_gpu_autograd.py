"""The torch.autograd wrappers only marshal arguments: gradients obtained through
loss.backward() are the library's backward results, checked here against the oracle."""
import pytest
import torch

import oracle
from oracle import producer
from paper_2607_22696_b200 import autograd as ops, inputs

import parity_util as pu

pytestmark = pytest.mark.gpu

BF16, F32 = torch.bfloat16, torch.float32


@pytest.mark.parametrize("dtype,d", [(BF16, 128), (F32, 32)])
def test_autograd_wrapper_with_residual_matches_the_oracle(dtype, d):
    T, H, W, heads, window = 4, 5, 7, 2, (3, 3, 3)
    shape = (T, H, W, heads, d)
    q, k, v, dout, res = (inputs.normal(shape, 170, i, 1.0, dtype) for i in range(5))
    off = inputs.normal((T, H, W, heads, 27, 3), 170, 6, 1.1, F32)
    leaves = [z.cuda().requires_grad_(True) for z in (q, k, v, off, res)]
    out = ops.dsa3d(leaves[0], leaves[1], leaves[2], leaves[3], window, residual=leaves[4])
    out.backward(dout.cuda())
    torch.cuda.synchronize()
    o_ref, _ = oracle.forward(q.view(-1, heads, d), k, v, off.view(-1, heads, 27, 3), T, H, W, heads, d, window)
    refs = oracle.backward(q.view(-1, heads, d), k, v, off.view(-1, heads, 27, 3), dout.view(-1, heads, d),
                           T, H, W, heads, d, window)
    pu.assert_close("out", out, o_ref.view(shape) + res.double(), dtype)
    for name, leaf, ref in zip(("dq", "dk", "dv", "doffsets"), leaves[:4], refs):
        pu.assert_close(name, leaf.grad, ref.view(leaf.shape), dtype, backward=True)
    assert torch.equal(leaves[4].grad, dout.cuda())               # the convolution term passes the gradient through


def test_fixed_window_autograd_wrapper_matches_the_oracle():
    T, H, W, heads, d, window = 5, 6, 9, 2, 128, (3, 3, 3)
    shape = (T, H, W, heads, d)
    q, k, v, dout = (inputs.normal(shape, 171, i, 1.0, BF16) for i in range(4))
    zeros = torch.zeros(T * H * W, heads, 27, 3, dtype=F32)
    leaves = [z.cuda().requires_grad_(True) for z in (q, k, v)]
    out = ops.dsa3d_fixed_window(*leaves, window)
    out.backward(dout.cuda())
    torch.cuda.synchronize()
    o_ref, _ = oracle.forward(q.view(-1, heads, d), k, v, zeros, T, H, W, heads, d, window)
    refs = oracle.backward(q.view(-1, heads, d), k, v, zeros, dout.view(-1, heads, d), T, H, W, heads, d, window)
    pu.assert_close("out", out, o_ref.view(shape), BF16)
    for name, leaf, ref in zip(("dq", "dk", "dv"), leaves, refs):
        pu.assert_close(name, leaf.grad, ref.view(shape), BF16, backward=True)


@pytest.mark.parametrize("dtype", [BF16, F32])
def test_producer_autograd_wrappers_match_the_oracle(dtype):
    """Gradients of the convolution and of the linear layer through loss.backward()."""
    T, H, W, C, kernel = 4, 5, 18, 64, (3, 3, 3)
    x = inputs.normal((T, H, W, C), 172, 0, 1.0, dtype)
    wc = inputs.normal((27, C), 172, 1, 0.3, F32)
    bc = inputs.normal((C,), 172, 2, 0.5, F32)
    dy = inputs.normal((T, H, W, C), 172, 3, 1.0, dtype)
    leaves = [z.cuda().requires_grad_(True) for z in (x, wc, bc)]
    y = ops.dwconv3d(*leaves, kernel)
    y.backward(dy.cuda())
    torch.cuda.synchronize()
    pu.assert_close("y", y, producer.dwconv3d(x, wc, bc, kernel), dtype)
    dx, dw, db = producer.dwconv3d_backward(x, wc, dy, kernel)
    pu.assert_close("dx", leaves[0].grad, dx, dtype, backward=True)
    for name, got, ref in (("dweight", leaves[1].grad, dw), ("dbias", leaves[2].grad, db)):
        assert float((got.cpu().double() - ref).abs().max()) <= 1e-4 * max(float(ref.pow(2).mean().sqrt()), 1.0), name

    tokens, O = 300, 54
    u = inputs.normal((tokens, C), 173, 0, 1.0, dtype)
    wl = inputs.normal((O, C), 173, 1, 0.2, dtype)
    bl = inputs.normal((O,), 173, 2, 1.0, F32)
    g = inputs.normal((tokens, O), 173, 3, 0.5, F32)
    leaves = [z.cuda().requires_grad_(True) for z in (u, wl, bl)]
    off = ops.offsets_linear(*leaves)
    off.backward(g.cuda())
    torch.cuda.synchronize()
    ref = producer.offsets_linear(u, wl, bl)
    assert float((off.detach().cpu().double() - ref).abs().max()) <= 1e-3 * max(float(ref.pow(2).mean().sqrt()), 1.0)
    du, dwl, dbl = producer.offsets_linear_backward(u, wl, g)
    pu.assert_close("du", leaves[0].grad, du, dtype, backward=True)
    pu.assert_close("dw", leaves[1].grad, dwl, dtype, backward=True)
    assert leaves[1].grad.dtype == dtype
    assert float((leaves[2].grad.cpu().double() - dbl).abs().max()) <= 1e-4 * max(float(dbl.abs().max()), 1.0)


def test_layer_module_equals_its_parts_and_its_gradients_follow_the_loss():
    """The Eq. 1 module only chains the wrappers: its output equals the entry points called by
    hand on the same tensors (bitwise), every parameter and input receives a finite gradient,
    and output and gradients equal the same chain evaluated stage by stage in the fp64 oracle."""
    from paper_2607_22696_b200 import binding
    from paper_2607_22696_b200.layer import DeformableSlideAttention3D
    T, H, W, heads, d, window = 4, 5, 6, 2, 32, (3, 3, 3)
    hidden, N = heads * d, T * H * W
    layer = DeformableSlideAttention3D(heads, d, window, (3, 3, 3), dtype=F32, seed=5)
    with torch.no_grad():          # leave the zero start: offsets of a fraction of a cell, off the lattice
        layer.offset_weight.copy_(inputs.normal(tuple(layer.offset_weight.shape), 180, 0, 0.05, F32).cuda())
        layer.offset_bias.copy_(inputs.normal(tuple(layer.offset_bias.shape), 180, 1, 0.3, F32).cuda())
    x = inputs.normal((T, H, W, hidden), 181, 0, 1.0, F32).cuda().requires_grad_(True)
    q, k, v = (inputs.normal((T, H, W, heads, d), 181, i, 1.0, F32).cuda().requires_grad_(True) for i in (1, 2, 3))
    probe = inputs.normal((T, H, W, heads, d), 181, 4, 1.0, F32).cuda()

    out = layer(x, q, k, v)
    # by hand through the binding
    u = torch.empty_like(x)
    binding.dsa3d_dwconv3d_forward(x.detach(), layer.offset_conv_weight.detach(), layer.offset_conv_bias.detach(),
                                   T, H, W, hidden, (3, 3, 3), u)
    off = torch.empty((N, heads * 27 * 3), dtype=F32, device="cuda")
    binding.dsa3d_offsets_linear_forward(u, layer.offset_weight.detach(), layer.offset_bias.detach(), N, hidden,
                                         heads * 27 * 3, off)
    term = torch.empty_like(x)
    binding.dsa3d_dwconv3d_forward(x.detach(), layer.term_conv_weight.detach(), layer.term_conv_bias.detach(),
                                   T, H, W, hidden, (3, 3, 3), term)
    ref = torch.empty_like(out)
    lse = torch.empty((T, H, W, heads), dtype=F32, device="cuda")
    binding.dsa3d_forward_residual(q.detach(), k.detach(), v.detach(), off, term, T, H, W, heads, d, window, ref, lse)
    torch.cuda.synchronize()
    assert torch.equal(out.detach(), ref)

    (out * probe).sum().backward()
    torch.cuda.synchronize()
    leaves = dict(layer.named_parameters(), x=x, q=q, k=k, v=v)
    for name, leaf in leaves.items():
        assert leaf.grad is not None and torch.isfinite(leaf.grad).all(), name
        assert float(leaf.grad.abs().max()) > 0, name

    # the same chain in the fp64 oracle, stage by stage on its own intermediate results (fp32
    # storage keeps the GPU's offsets within 1e-6 of the oracle's, so no sample changes cell)
    par = {n: p.detach().cpu() for n, p in layer.named_parameters()}
    xc, qc, kc, vc, pc = (z.detach().cpu() for z in (x, q, k, v, probe))
    u_o = producer.dwconv3d(xc, par["offset_conv_weight"], par["offset_conv_bias"], (3, 3, 3))
    off_o = producer.offsets_linear(u_o.view(N, hidden), par["offset_weight"], par["offset_bias"])
    term_o = producer.dwconv3d(xc, par["term_conv_weight"], par["term_conv_bias"], (3, 3, 3))
    off4 = off_o.view(N, heads, 27, 3).float()            # the operator takes its offsets in fp32
    o_ref, _ = oracle.forward(qc.view(-1, heads, d), kc, vc, off4, T, H, W, heads, d, window)
    pu.assert_close("layer output", out, o_ref.view(T, H, W, heads, d) + term_o.view(T, H, W, heads, d), F32)
    dq_o, dk_o, dv_o, doff_o = oracle.backward(qc.view(-1, heads, d), kc, vc, off4, pc.view(-1, heads, d),
                                               T, H, W, heads, d, window)
    du_o, dwl_o, dbl_o = producer.offsets_linear_backward(u_o.view(N, hidden), par["offset_weight"], doff_o.view(N, -1))
    dx1, dwc1, dbc1 = producer.dwconv3d_backward(xc, par["offset_conv_weight"], du_o.view(T, H, W, hidden), (3, 3, 3))
    dx2, dwc2, dbc2 = producer.dwconv3d_backward(xc, par["term_conv_weight"], pc.view(T, H, W, hidden), (3, 3, 3))
    want = {"offset_conv_weight": dwc1, "offset_conv_bias": dbc1, "term_conv_weight": dwc2, "term_conv_bias": dbc2,
            "offset_weight": dwl_o, "offset_bias": dbl_o, "x": dx1 + dx2, "q": dq_o, "k": dk_o, "v": dv_o}
    for name, ref in want.items():
        got = leaves[name].grad.detach().cpu().double().reshape(-1)
        ref = ref.reshape(-1)
        bound = 1e-4 * max(float(ref.abs().max()), 1.0)
        assert float((got - ref).abs().max()) <= bound, (name, float((got - ref).abs().max()), bound)
