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
