"""Pins for the oracle of the depthwise convolution and the offset-producing linear layer
(first term of Eq. 1; the offset predictor of the Formulation section): identities, closed
forms, a brute-force triple loop and the library routine the paper's implementation section
names, chosen so that a wrong centring, a flipped kernel, a transposed weight or a dropped
bias fails at least one."""
import itertools

import torch

from oracle import producer


def _rand(shape, seed, dtype=torch.float64):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(*shape, generator=g, dtype=dtype)


def test_centre_tap_is_the_identity():
    x = _rand((4, 5, 6, 3), 1)
    for kernel in [(3, 3, 3), (1, 5, 3), (2, 2, 2), (3, 7, 7)]:
        taps = kernel[0] * kernel[1] * kernel[2]
        w = torch.zeros(taps, 3, dtype=torch.float64)
        centre = ((kernel[0] // 2) * kernel[1] + kernel[1] // 2) * kernel[2] + kernel[2] // 2
        w[centre] = 1.0
        assert torch.equal(producer.dwconv3d(x, w, None, kernel), x)


def test_single_tap_shifts_with_zero_fill_and_correlation_sign():
    """Tap (i, j, l) reads the input at +(i - kt//2, ...): output[t] = x[t + dt] inside the
    grid, 0 where t + dt falls outside.  A convolution (flipped kernel) would shift the other
    way and fail here."""
    T, H, W, C = 5, 4, 6, 2
    x = _rand((T, H, W, C), 2)
    kernel = (3, 3, 3)
    for (i, j, l) in [(0, 1, 1), (2, 1, 1), (1, 0, 1), (1, 1, 2), (2, 0, 2)]:
        w = torch.zeros(27, C, dtype=torch.float64)
        w[(i * 3 + j) * 3 + l] = 1.0
        got = producer.dwconv3d(x, w, None, kernel)
        dt, dy, dx = i - 1, j - 1, l - 1
        for t, y, xx in itertools.product(range(T), range(H), range(W)):
            st, sy, sx = t + dt, y + dy, xx + dx
            inside = 0 <= st < T and 0 <= sy < H and 0 <= sx < W
            want = x[st, sy, sx] if inside else torch.zeros(C, dtype=torch.float64)
            assert torch.equal(got[t, y, xx], want), (i, j, l, t, y, xx)


def test_constant_input_counts_the_taps_inside_the_grid():
    """x = 1 and w = 1 give, at each position, the number of taps that stay inside the grid: a
    product of per-axis counts; the bias adds on top."""
    T, H, W, C = 4, 3, 5, 2
    kernel = (3, 2, 5)
    x = torch.ones(T, H, W, C, dtype=torch.float64)
    w = torch.ones(kernel[0] * kernel[1] * kernel[2], C, dtype=torch.float64)
    bias = torch.tensor([0.5, -2.0], dtype=torch.float64)
    got = producer.dwconv3d(x, w, bias, kernel)

    def count(pos, size, k):
        return sum(1 for i in range(k) if 0 <= pos + i - k // 2 < size)

    for t, y, xx in itertools.product(range(T), range(H), range(W)):
        n = count(t, T, kernel[0]) * count(y, H, kernel[1]) * count(xx, W, kernel[2])
        assert torch.equal(got[t, y, xx], n + bias)


def test_brute_force_loops_and_channel_independence():
    T, H, W, C = 3, 4, 3, 3
    kernel = (3, 3, 2)
    x = _rand((T, H, W, C), 3)
    w = _rand((18, C), 4)
    bias = _rand((C,), 5)
    got = producer.dwconv3d(x, w, bias, kernel)
    for t, y, xx, c in itertools.product(range(T), range(H), range(W), range(C)):
        acc = float(bias[c])
        for i, j, l in itertools.product(range(3), range(3), range(2)):
            st, sy, sx = t + i - 1, y + j - 1, xx + l - 1
            if 0 <= st < T and 0 <= sy < H and 0 <= sx < W:
                acc += float(w[(i * 3 + j) * 2 + l, c]) * float(x[st, sy, sx, c])
        assert abs(float(got[t, y, xx, c]) - acc) < 1e-12
    # depthwise: changing channel 1 of the input leaves channels 0 and 2 of the output alone
    x2 = x.clone()
    x2[..., 1] += 1.0
    got2 = producer.dwconv3d(x2, w, bias, kernel)
    assert torch.equal(got2[..., 0], got[..., 0]) and torch.equal(got2[..., 2], got[..., 2])
    assert not torch.equal(got2[..., 1], got[..., 1])


def test_matches_the_grouped_conv3d_of_the_implementation_section():
    """nn.Conv3d(groups = channels) with padding k//2 on odd kernels is the routine the paper
    builds on; the oracle never calls it."""
    T, H, W, C = 4, 5, 6, 4
    kernel = (3, 3, 3)
    x = _rand((T, H, W, C), 6)
    w = _rand((27, C), 7)
    bias = _rand((C,), 8)
    got = producer.dwconv3d(x, w, bias, kernel)
    xt = x.permute(3, 0, 1, 2).unsqueeze(0)                       # [1, C, T, H, W]
    wt = w.t().reshape(C, 1, 3, 3, 3)
    ref = torch.nn.functional.conv3d(xt, wt, bias, padding=1, groups=C)[0].permute(1, 2, 3, 0)
    assert torch.allclose(got, ref, rtol=0, atol=1e-12)


def test_linear_layer_against_loops_and_the_library_routine():
    u = _rand((7, 5), 9)
    w = _rand((4, 5), 10)
    bias = _rand((4,), 11)
    got = producer.offsets_linear(u, w, bias)
    for n, o in itertools.product(range(7), range(4)):
        acc = float(bias[o]) + sum(float(u[n, c]) * float(w[o, c]) for c in range(5))
        assert abs(float(got[n, o]) - acc) < 1e-12
    assert torch.allclose(got, torch.nn.functional.linear(u, w, bias), rtol=0, atol=1e-12)
    # identity weight returns the input plus the bias; a transposed weight would not fit here
    eye = torch.eye(5, dtype=torch.float64)
    assert torch.equal(producer.offsets_linear(u, eye, None), u)
    one_hot = torch.zeros(2, 5, dtype=torch.float64)
    one_hot[1, 3] = 2.0
    out = producer.offsets_linear(u, one_hot, None)
    assert torch.equal(out[:, 0], torch.zeros(7, dtype=torch.float64)) and torch.equal(out[:, 1], 2.0 * u[:, 3])


def test_inputs_in_storage_precision_are_read_exactly():
    """bf16 / fp32 inputs are widened, never re-rounded: the result equals the fp64 result on
    the widened values."""
    x = _rand((3, 3, 3, 2), 12).to(torch.bfloat16)
    w = _rand((27, 2), 13).to(torch.float32)
    got = producer.dwconv3d(x, w, None, (3, 3, 3))
    ref = producer.dwconv3d(x.to(torch.float64), w.to(torch.float64), None, (3, 3, 3))
    assert torch.equal(got, ref)


def test_convolution_gradients_against_autograd_of_the_library_routine():
    """The gradient formulas are checked against reverse-mode differentiation of the grouped
    Conv3d (odd kernels, where padding k//2 is the oracle's centring), which the oracle never
    calls."""
    T, H, W, C = 4, 5, 3, 3
    kernel = (3, 3, 3)
    x = _rand((T, H, W, C), 20).requires_grad_(True)
    w = _rand((27, C), 21).requires_grad_(True)
    bias = _rand((C,), 22).requires_grad_(True)
    dy = _rand((T, H, W, C), 23)
    xt = x.permute(3, 0, 1, 2).unsqueeze(0)
    wt = w.t().reshape(C, 1, 3, 3, 3)
    y = torch.nn.functional.conv3d(xt, wt, bias, padding=1, groups=C)[0].permute(1, 2, 3, 0)
    (y * dy).sum().backward()
    dx, dw, db = producer.dwconv3d_backward(x.detach(), w.detach(), dy, kernel)
    assert torch.allclose(dx, x.grad, rtol=0, atol=1e-12)
    assert torch.allclose(dw, w.grad, rtol=0, atol=1e-11)
    assert torch.allclose(db, bias.grad, rtol=0, atol=1e-12)


def test_convolution_gradients_by_the_adjoint_identity_and_single_entries():
    """Even and mixed kernel sizes (no library routine with this centring): the map x -> y is
    linear, so <dy, conv(x)> = <dx, x> for every x, and likewise in the weights; a single
    non-zero dy entry and a single tap give gradients that can be read off by hand."""
    T, H, W, C = 3, 4, 5, 2
    for kernel in [(2, 2, 2), (1, 4, 3), (3, 2, 5)]:
        taps = kernel[0] * kernel[1] * kernel[2]
        x, w, dy = _rand((T, H, W, C), 30), _rand((taps, C), 31), _rand((T, H, W, C), 32)
        dx, dw, db = producer.dwconv3d_backward(x, w, dy, kernel)
        x2, w2 = _rand((T, H, W, C), 33), _rand((taps, C), 34)
        zero = torch.zeros_like(x)
        assert abs(float((dy * producer.dwconv3d(x2, w, None, kernel)).sum() - (dx * x2).sum())) < 1e-10
        assert abs(float((dy * producer.dwconv3d(x, w2, None, kernel)).sum() - (dw * w2).sum())) < 1e-10
        assert torch.equal(producer.dwconv3d_backward(zero, w, dy, kernel)[1], torch.zeros_like(w))
        assert torch.allclose(db, dy.sum(dim=(0, 1, 2)), rtol=0, atol=1e-13)
    # one tap, one output entry: dx is w*dy at the displaced position, dw is x there times dy
    kernel = (2, 2, 2)                                   # displacements -1 and 0 on each axis
    w = torch.zeros(8, C, dtype=torch.float64)
    w[0] = torch.tensor([2.0, -3.0], dtype=torch.float64)   # tap (0,0,0): displacement (-1,-1,-1)
    x = _rand((T, H, W, C), 35)
    dy = torch.zeros(T, H, W, C, dtype=torch.float64)
    dy[2, 3, 4] = torch.tensor([1.0, 0.5], dtype=torch.float64)
    dx, dw, _ = producer.dwconv3d_backward(x, w, dy, kernel)
    want = torch.zeros_like(dx)
    want[1, 2, 3] = torch.tensor([2.0, -1.5], dtype=torch.float64)
    assert torch.equal(dx, want)
    for i, j, l in itertools.product(range(2), range(2), range(2)):     # dw does not depend on w
        assert torch.equal(dw[(i * 2 + j) * 2 + l], x[1 + i, 2 + j, 3 + l] * dy[2, 3, 4])
    # the same output entry at the corner of the grid has no displaced position: no gradient
    dy0 = torch.zeros_like(dy)
    dy0[0, 0, 0] = 1.0
    dx0, dw0, _ = producer.dwconv3d_backward(x, w, dy0, kernel)
    assert torch.equal(dx0, torch.zeros_like(dx0)) and torch.equal(dw0[0], torch.zeros(C, dtype=torch.float64))
    assert torch.equal(dw0[7], x[0, 0, 0] * dy0[0, 0, 0])           # tap (1,1,1) has displacement 0


def test_convolution_gradients_by_central_differences():
    T, H, W, C = 3, 3, 4, 2
    kernel = (3, 2, 3)
    x, w, dy = _rand((T, H, W, C), 40), _rand((18, C), 41), _rand((T, H, W, C), 42)
    dx, dw, _ = producer.dwconv3d_backward(x, w, dy, kernel)
    loss = lambda xx, ww: float((dy * producer.dwconv3d(xx, ww, None, kernel)).sum())
    eps = 1e-6
    for idx in [(0, 0, 0, 0), (1, 2, 3, 1), (2, 1, 0, 0)]:
        xp, xm = x.clone(), x.clone()
        xp[idx] += eps
        xm[idx] -= eps
        assert abs((loss(xp, w) - loss(xm, w)) / (2 * eps) - float(dx[idx])) < 1e-7
    for idx in [(0, 0), (7, 1), (17, 0)]:
        wp, wm = w.clone(), w.clone()
        wp[idx] += eps
        wm[idx] -= eps
        assert abs((loss(x, wp) - loss(x, wm)) / (2 * eps) - float(dw[idx])) < 1e-7


def test_linear_layer_gradients_against_loops_and_autograd():
    u, w, g = _rand((6, 5), 50), _rand((4, 5), 51), _rand((6, 4), 52)
    du, dw, db = producer.offsets_linear_backward(u, w, g)
    for n, c in itertools.product(range(6), range(5)):
        assert abs(float(du[n, c]) - sum(float(g[n, o]) * float(w[o, c]) for o in range(4))) < 1e-12
    for o, c in itertools.product(range(4), range(5)):
        assert abs(float(dw[o, c]) - sum(float(g[n, o]) * float(u[n, c]) for n in range(6))) < 1e-12
    for o in range(4):
        assert abs(float(db[o]) - sum(float(g[n, o]) for n in range(6))) < 1e-12
    ua, wa, ba = u.clone().requires_grad_(True), w.clone().requires_grad_(True), _rand((4,), 53).requires_grad_(True)
    (torch.nn.functional.linear(ua, wa, ba) * g).sum().backward()
    assert torch.allclose(du, ua.grad, rtol=0, atol=1e-12)
    assert torch.allclose(dw, wa.grad, rtol=0, atol=1e-12)
    assert torch.allclose(db, ba.grad, rtol=0, atol=1e-12)
