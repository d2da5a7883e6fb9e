"""Seeded random sweep over small problems: grid extents (including 1), head counts, head sizes,
storage types, windows and offset kinds are drawn at random and every entry point that applies
(general forward/backward; the fixed-window pair when the offsets are zero) is compared with the
oracle.  Catches indexing slips that hand-picked shapes miss; the draws are fixed by the seed."""
import random

import pytest
import torch

import oracle
from paper_2607_22696_b200 import binding, inputs

import parity_util as pu

pytestmark = pytest.mark.gpu

BF16, F32 = torch.bfloat16, torch.float32


def _draw(rng, it):
    T, H, W = rng.randint(1, 9), rng.randint(1, 11), rng.randint(1, 19)
    heads = rng.randint(1, 3)
    d = rng.choice([32, 64, 128])
    dtype = rng.choice([BF16, BF16, F32])
    window = (rng.randint(1, 3), rng.randint(1, 3), rng.randint(1, 3))
    if rng.random() < 0.15:
        window = rng.choice([(3, 5, 5), (1, 7, 7), (2, 2, 2), (4, 2, 3)])
    sigma = rng.choice([0.0, 0.3, 1.0, 2.5])
    kind = rng.choice(["normal", "int", "zero"]) if sigma > 0 else "zero"
    return (T, H, W, heads, d), dtype, window, sigma, kind, 1000 + it


@pytest.mark.parametrize("seed", [1, 2])
def test_random_small_problems_match_the_oracle(seed):
    rng = random.Random(seed)
    for it in range(40):
        shape, dtype, window, sigma, kind, s = _draw(rng, it)
        T, H, W, heads, d = shape
        P = window[0] * window[1] * window[2]
        q, k, v, dout = (inputs.normal(shape, s, i, 1.0, dtype) for i in range(4))
        if kind == "normal":
            off = inputs.normal((T, H, W, heads, P, 3), s, 5, sigma, F32)
        elif kind == "int":
            off = inputs.uniform_int((T, H, W, heads, P, 3), s, 5, -2, 2, F32)
        else:
            off = torch.zeros((T, H, W, heads, P, 3), dtype=F32)
        pu.full_parity(q, k, v, off, dout, window)
        if kind != "zero":
            continue
        o_ref, l_ref = oracle.forward(q.view(-1, heads, d), k, v, off.view(-1, heads, P, 3), T, H, W, heads, d, window)
        refs = oracle.backward(q.view(-1, heads, d), k, v, off.view(-1, heads, P, 3), dout.view(-1, heads, d),
                               T, H, W, heads, d, window)
        qd, kd, vd, dd = (z.cuda() for z in (q, k, v, dout))
        out = torch.empty(shape, dtype=dtype, device="cuda")
        lse = torch.empty((T, H, W, heads), dtype=F32, device="cuda")
        binding.dsa3d_forward_fixed_window(qd, kd, vd, T, H, W, heads, d, window, out, lse)
        g = [torch.empty(shape, dtype=dtype, device="cuda") for _ in range(3)]
        doff = torch.empty((T, H, W, heads, P, 3), dtype=F32, device="cuda")
        ws = torch.empty((binding.dsa3d_backward_fixed_window_workspace_bytes(T, H, W, heads, d, window, dtype),),
                         dtype=torch.uint8, device="cuda")
        binding.dsa3d_backward_fixed_window(qd, kd, vd, lse, dd, T, H, W, heads, d, window, g[0], g[1], g[2], doff, ws)
        torch.cuda.synchronize()
        assert binding.dsa3d_device_timeout_flag() == 0
        pu.assert_close("out", out, o_ref.view(shape), dtype)
        pu.assert_close("lse", lse, l_ref.view(T, H, W, heads), dtype)
        for name, got, want in zip(("dq", "dk", "dv"), g, refs[:3]):
            pu.assert_close(name, got, want.view(shape), dtype, backward=True)
        pu.assert_close("doffsets", doff, refs[3].view(T, H, W, heads, P, 3), dtype, backward=True)
