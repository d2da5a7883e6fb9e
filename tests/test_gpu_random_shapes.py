"""Seeded random sweep over small problems: grid extents (including 1), head counts, head sizes,
storage types, windows and offset kinds are drawn at random and every entry point that applies
(general forward/backward; the fixed-window pair when the offsets are zero; the bounded-offsets pair on
offsets below 1 in size) is compared with the
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


@pytest.mark.parametrize("seed", [3])
def test_random_small_offset_problems_match_the_oracle(seed):
    """The pair of entry points for learned offsets below 1 in size (window (3,3,3), bf16) on random small
    grids: offsets uniform in (-1, 1), or drawn from values next to -1, 0 and +1 where a sample changes cell."""
    rng = random.Random(seed)
    window, P = (3, 3, 3), 27
    edge = torch.tensor([-0.99999994, -1e-7, 0.0, 1e-7, 0.99999994, 0.5, -0.5], dtype=F32)
    for it in range(24):
        shape = (rng.randint(1, 9), rng.randint(1, 11), rng.randint(1, 19), rng.randint(1, 3), rng.choice([64, 128]))
        T, H, W, heads, d = shape
        s = 2000 + it
        q, k, v, dout = (inputs.normal(shape, s, i, rng.choice([1.0, 3.0]) if i == 0 else 1.0, BF16) for i in range(4))
        gen = torch.Generator().manual_seed(s)
        if rng.random() < 0.5:
            off = (torch.rand((T, H, W, heads, P, 3), generator=gen, dtype=torch.float64) * 2 - 1).clamp(-0.999999, 0.999999).to(F32)
        else:
            off = edge[torch.randint(0, edge.numel(), (T, H, W, heads, P, 3), generator=gen)]
        o_ref, l_ref = oracle.forward(q.view(-1, heads, d), k, v, off.view(-1, heads, P, 3), T, H, W, heads, d, window)
        refs = oracle.backward(q.view(-1, heads, d), k, v, off.view(-1, heads, P, 3), dout.view(-1, heads, d),
                               T, H, W, heads, d, window)
        qd, kd, vd, od, dd = (z.cuda() for z in (q, k, v, off, dout))
        out = torch.full(shape, float("nan"), dtype=BF16, device="cuda")
        lse = torch.full((T, H, W, heads), float("nan"), dtype=F32, device="cuda")
        binding.dsa3d_forward_bounded_offsets(qd, kd, vd, od, T, H, W, heads, d, window, out, lse)
        g = [torch.full(shape, float("nan"), dtype=BF16, device="cuda") for _ in range(3)]
        doff = torch.full((T, H, W, heads, P, 3), float("nan"), dtype=F32, device="cuda")
        ws = torch.empty((binding.dsa3d_backward_bounded_offsets_workspace_bytes(T, H, W, heads, d, window, BF16),),
                         dtype=torch.uint8, device="cuda")
        binding.dsa3d_backward_bounded_offsets(qd, kd, vd, od, lse, dd, T, H, W, heads, d, window, g[0], g[1], g[2], doff, ws)
        torch.cuda.synchronize()
        assert binding.dsa3d_device_timeout_flag() == 0
        pu.assert_close("out", out, o_ref.view(shape), BF16)
        pu.assert_close("lse", lse, l_ref.view(T, H, W, heads), BF16)
        for name, got, want in zip(("dq", "dk", "dv"), g, refs[:3]):
            pu.assert_close(name, got, want.view(shape), BF16, backward=True)
        pu.assert_close("doffsets", doff, refs[3].view(T, H, W, heads, P, 3), BF16, backward=True)


def _sum_close(name, got, ref, rel):
    got = got.detach().cpu().double()
    assert torch.isfinite(got).all(), name
    worst = float((got - ref).abs().max())
    bound = rel * max(float(ref.pow(2).mean().sqrt()), 1.0)
    assert worst <= bound, f"{name}: max abs error {worst:.3e} > {bound:.3e}"


@pytest.mark.parametrize("seed", [3, 4])
def test_random_layers_around_the_operator_match_the_oracle(seed):
    """The convolution and the linear layer, forward and backward, on random shapes: grids with
    extents of 1, channel counts that are and are not multiples of 64 (staged and plain kernels),
    kernel sizes with and without kernels of their own, token and output counts that are ragged
    against every tile size of the contractions."""
    from oracle import producer
    rng = random.Random(seed)
    for it in range(30):
        dtype = rng.choice([BF16, BF16, F32])
        T, H, W = rng.randint(1, 10), rng.randint(1, 9), rng.randint(1, 37)
        C = rng.choice([8, 16, 24, 64, 64, 128, 192])
        kernel = rng.choice([(3, 3, 3), (3, 3, 3), (1, 1, 1), (2, 2, 2), (3, 5, 5), (1, 3, 7), (5, 3, 1), (2, 3, 4)])
        taps = kernel[0] * kernel[1] * kernel[2]
        s = 2000 + 100 * seed + it
        x = inputs.normal((T, H, W, C), s, 0, 1.0, dtype)
        wc = inputs.normal((taps, C), s, 1, 0.3, F32)
        bc = inputs.normal((C,), s, 2, 0.5, F32) if rng.random() < 0.7 else None
        dy = inputs.normal((T, H, W, C), s, 3, 1.0, dtype)
        xd, wd, dyd = x.cuda(), wc.cuda(), dy.cuda()
        y = torch.full((T, H, W, C), float("nan"), dtype=dtype, device="cuda")
        binding.dsa3d_dwconv3d_forward(xd, wd, None if bc is None else bc.cuda(), T, H, W, C, kernel, y)
        dx = torch.full((T, H, W, C), float("nan"), dtype=dtype, device="cuda")
        dw = torch.full((taps, C), float("nan"), dtype=F32, device="cuda")
        db = torch.full((C,), float("nan"), dtype=F32, device="cuda")
        ws = torch.empty(max(binding.dsa3d_dwconv3d_backward_workspace_bytes(C, kernel), 16), dtype=torch.uint8, device="cuda")
        binding.dsa3d_dwconv3d_backward(xd, wd, dyd, T, H, W, C, kernel, dx, dw, db, ws)
        torch.cuda.synchronize()
        tag = f"case {it}: {dtype} grid {(T, H, W)} C {C} kernel {kernel}"
        pu.assert_close(tag + " y", y, producer.dwconv3d(x, wc, bc, kernel), dtype)
        r_dx, r_dw, r_db = producer.dwconv3d_backward(x, wc, dy, kernel)
        pu.assert_close(tag + " dx", dx, r_dx, dtype, backward=True)
        _sum_close(tag + " dweight", dw, r_dw, 1e-4)
        _sum_close(tag + " dbias", db, r_db, 1e-4)

        tokens, O = rng.randint(1, 700), rng.choice([1, 3, 27, 40, 81, 162, 300, 648])
        u = inputs.normal((tokens, C), s, 4, 1.0, dtype)
        wl = inputs.normal((O, C), s, 5, 0.2, dtype)
        bl = inputs.normal((O,), s, 6, 1.0, F32)
        g = inputs.normal((tokens, O), s, 7, 0.5, F32)
        ud, wld, gd = u.cuda(), wl.cuda(), g.cuda()
        off = torch.full((tokens, O), float("nan"), dtype=F32, device="cuda")
        binding.dsa3d_offsets_linear_forward(ud, wld, bl.cuda(), tokens, C, O, off)
        du = torch.full((tokens, C), float("nan"), dtype=dtype, device="cuda")
        dwl = torch.full((O, C), float("nan"), dtype=F32, device="cuda")
        dbl = torch.full((O,), float("nan"), dtype=F32, device="cuda")
        wsl = torch.empty(max(binding.dsa3d_offsets_linear_backward_workspace_bytes(tokens, C, O, dtype), 16),
                          dtype=torch.uint8, device="cuda")
        binding.dsa3d_offsets_linear_backward(ud, wld, gd, tokens, C, O, du, dwl, dbl, wsl)
        torch.cuda.synchronize()
        assert binding.dsa3d_device_timeout_flag() == 0
        tag = f"case {it}: {dtype} tokens {tokens} C {C} O {O}"
        _sum_close(tag + " offsets", off, producer.offsets_linear(u, wl, bl), 1e-3 if dtype == BF16 else 1e-5)
        r_du, r_dwl, r_dbl = producer.offsets_linear_backward(u, wl, g)
        pu.assert_close(tag + " du", du, r_du, dtype, backward=True)
        pu.assert_close(tag + " dw", dwl, r_dwl, dtype, backward=True)
        _sum_close(tag + " dbias", dbl, r_dbl, 1e-5)
