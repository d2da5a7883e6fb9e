"""The torch.autograd wrappers only marshal arguments: gradients obtained through
loss.backward() are the library's backward results, checked here against the oracle."""
import pytest
import torch

import oracle
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
