"""Pins for the CPU oracle: each test checks it against something other than itself.

The paper prints no worked values for the operator, so the pins are: the zero-offset
reduction to fixed local attention (Ablations, "Effect of offsets"), brute-force masked
dense softmax attention, exact gathers for integer offsets, closed forms on affine fields,
the library routine the paper names for the sampling (grid_sample, Implementation
considerations) together with autograd through it, hand-computable padding cases, P = 1,
softmax invariances, central finite differences, bilinearity invariants and translation
equivariance.  All reference code in this file is written independently of oracle/.
"""
import itertools
import math

import pytest
import torch
import torch.nn.functional as F

import oracle

torch.manual_seed(1234)
F64 = torch.float64


def rand_problem(T, H, W, heads, d, window, sigma, dtype=F64, seed=0):
    g = torch.Generator().manual_seed(seed)
    P = window[0] * window[1] * window[2]
    q = torch.randn(T, H, W, heads, d, generator=g, dtype=F64).to(dtype)
    k = torch.randn(T, H, W, heads, d, generator=g, dtype=F64).to(dtype)
    v = torch.randn(T, H, W, heads, d, generator=g, dtype=F64).to(dtype)
    off_dtype = F64 if dtype == F64 else torch.float32
    off = (torch.randn(T, H, W, heads, P, 3, generator=g, dtype=F64) * sigma).to(off_dtype)
    dout = torch.randn(T, H, W, heads, d, generator=g, dtype=F64).to(dtype)
    return q, k, v, off, dout


def displacements(window):
    """Window displacement of each cell, cell index u-major and w-minor."""
    return [(u - window[0] // 2, vv - window[1] // 2, w - window[2] // 2)
            for u in range(window[0]) for vv in range(window[1]) for w in range(window[2])]


def tokens(T, H, W):
    return list(itertools.product(range(T), range(H), range(W)))


# ---------------------------------------------------------------- independent references

def slide_window_attention(q, k, v, window, int_off=None):
    """Fixed 3D sliding-window attention by integer gathers (zero rows outside the grid).
    int_off [T,H,W,heads,P,3] optional integer shifts of each cell."""
    T, H, W, heads, d = q.shape
    disp = displacements(window)
    P = len(disp)
    out = torch.zeros(T, H, W, heads, d, dtype=F64)
    lse = torch.zeros(T, H, W, heads, dtype=F64)
    for (t, y, x) in tokens(T, H, W):
        for m in range(heads):
            ks = torch.zeros(P, d, dtype=F64)
            vs = torch.zeros(P, d, dtype=F64)
            for p, (bt, by, bx) in enumerate(disp):
                tt, yy, xx = t + bt, y + by, x + bx
                if int_off is not None:
                    tt += int(int_off[t, y, x, m, p, 0])
                    yy += int(int_off[t, y, x, m, p, 1])
                    xx += int(int_off[t, y, x, m, p, 2])
                if 0 <= tt < T and 0 <= yy < H and 0 <= xx < W:
                    ks[p] = k[tt, yy, xx, m].to(F64)
                    vs[p] = v[tt, yy, xx, m].to(F64)
            s = ks @ q[t, y, x, m].to(F64) / math.sqrt(d)
            lse[t, y, x, m] = torch.logsumexp(s, 0)
            out[t, y, x, m] = torch.softmax(s, 0) @ vs
    return out, lse


def dense_masked_attention(q, k, v, window):
    """Brute force: softmax over ALL N keys with a window mask; a query whose window sticks
    out of the grid also sees one zero-logit, zero-value sink per outside cell."""
    T, H, W, heads, d = q.shape
    N = T * H * W
    toks = tokens(T, H, W)
    disp = set(displacements(window))
    out = torch.zeros(N, heads, d, dtype=F64)
    for m in range(heads):
        Q, K, V = (z[..., m, :].reshape(N, d).to(F64) for z in (q, k, v))
        S = Q @ K.T / math.sqrt(d)
        mask = torch.zeros(N, N, dtype=torch.bool)
        for i, (t, y, x) in enumerate(toks):
            for j, (t2, y2, x2) in enumerate(toks):
                mask[i, j] = (t2 - t, y2 - y, x2 - x) in disp
        n_sink = len(disp) - mask.sum(1)
        E = torch.where(mask, torch.exp(S), torch.zeros_like(S))
        denom = E.sum(1) + n_sink.to(F64)          # exp(0) = 1 per sink
        out[:, m] = (E @ V) / denom[:, None]
    return out.view(T, H, W, heads, d)


def torch_grid_sample_dsa(q, k, v, off, window):
    """The operator composed the way the paper's implementation does it: grid_sample
    ('bilinear' on 5-D input, zeros padding) for K and V, then softmax and weighted sum.
    Differentiable; index-space positions are mapped to normalised coordinates with
    align_corners=True."""
    T, H, W, heads, d = q.shape
    disp = torch.tensor(displacements(window), dtype=F64)            # [P,3] (t,y,x)
    P = disp.shape[0]
    coords = torch.tensor(tokens(T, H, W), dtype=F64)                # [N,3]
    N = coords.shape[0]
    pos = coords[:, None, None, :] + disp[None, None, :, :] + off.reshape(N, heads, P, 3)
    size = torch.tensor([T, H, W], dtype=F64)
    norm = 2.0 * pos / (size - 1.0) - 1.0                            # (t,y,x) normalised
    grid = norm.flip(-1)                                             # grid_sample wants (x,y,z)
    outs, lses = [], []
    for m in range(heads):
        vol_k = k[..., m, :].permute(3, 0, 1, 2)[None]               # [1,d,T,H,W]
        vol_v = v[..., m, :].permute(3, 0, 1, 2)[None]
        gm = grid[:, m][None, :, :, None, :]                         # [1,N,P,1,3]
        ks = F.grid_sample(vol_k, gm, mode="bilinear", padding_mode="zeros", align_corners=True)
        vs = F.grid_sample(vol_v, gm, mode="bilinear", padding_mode="zeros", align_corners=True)
        ks = ks[0, :, :, :, 0].permute(1, 2, 0)                      # [N,P,d]
        vs = vs[0, :, :, :, 0].permute(1, 2, 0)
        s = torch.einsum("nd,npd->np", q[..., m, :].reshape(N, d), ks) / math.sqrt(d)
        a = torch.softmax(s, -1)
        outs.append(torch.einsum("np,npd->nd", a, vs))
        lses.append(torch.logsumexp(s, -1))
    out = torch.stack(outs, 1).view(T, H, W, heads, d)
    lse = torch.stack(lses, 1).view(T, H, W, heads)
    return out, lse


def run_oracle(q, k, v, off, window, dout=None):
    T, H, W, heads, d = q.shape
    out, lse = oracle.forward(q, k, v, off, T, H, W, heads, d, window)
    res = [out.view(T, H, W, heads, d), lse.view(T, H, W, heads)]
    if dout is not None:
        dq, dk, dv, doff = oracle.backward(q, k, v, off, dout, T, H, W, heads, d, window)
        res += [dq.view_as(q), dk.view_as(k), dv.view_as(v), doff.view_as(off)]
    return res


# ------------------------------------------------------------------------------- the pins

@pytest.mark.parametrize("window", [(3, 3, 3), (2, 2, 2), (1, 3, 5), (3, 1, 1)])
def test_zero_offsets_equal_fixed_window_attention(window):
    q, k, v, off, _ = rand_problem(3, 4, 5, 2, 4, window, 0.0, seed=1)
    out, lse = run_oracle(q, k, v, torch.zeros_like(off), window)
    ref_out, ref_lse = slide_window_attention(q, k, v, window)
    assert torch.allclose(out, ref_out, rtol=0, atol=1e-14)
    assert torch.allclose(lse, ref_lse, rtol=0, atol=1e-14)


@pytest.mark.parametrize("window", [(3, 3, 3), (2, 2, 2)])
def test_zero_offsets_equal_masked_dense_attention(window):
    q, k, v, off, _ = rand_problem(3, 3, 4, 2, 3, window, 0.0, seed=2)
    out, _ = run_oracle(q, k, v, torch.zeros_like(off), window)
    ref = dense_masked_attention(q, k, v, window)
    assert torch.allclose(out, ref, rtol=0, atol=1e-14)


@pytest.mark.parametrize("dtype", [F64, torch.float32])
def test_integer_offsets_are_exact_gathers(dtype):
    window = (3, 3, 3)
    q, k, v, off, _ = rand_problem(4, 4, 5, 2, 4, window, 0.0, dtype=dtype, seed=3)
    g = torch.Generator().manual_seed(7)
    ioff = torch.randint(-3, 4, off.shape, generator=g)
    out, lse = run_oracle(q, k, v, ioff.to(off.dtype), window)
    ref_out, ref_lse = slide_window_attention(q, k, v, window, ioff)
    assert torch.allclose(out, ref_out, rtol=0, atol=1e-14)
    assert torch.allclose(lse, ref_lse, rtol=0, atol=1e-14)


def test_affine_fields_closed_form_value_and_gradients():
    """K[pos] = A pos + k0 and V[pos] = B pos + v0 are reproduced exactly by trilinear
    interpolation at interior positions, which gives every output in closed form."""
    T, H, W, heads, d, window = 7, 7, 7, 1, 3, (3, 3, 3)
    g = torch.Generator().manual_seed(4)
    A, B = torch.randn(d, 3, generator=g, dtype=F64), torch.randn(d, 3, generator=g, dtype=F64)
    k0, v0 = torch.randn(d, generator=g, dtype=F64), torch.randn(d, generator=g, dtype=F64)
    coords = torch.tensor(tokens(T, H, W), dtype=F64)
    k = (coords @ A.T + k0).view(T, H, W, heads, d)
    v = (coords @ B.T + v0).view(T, H, W, heads, d)
    q = torch.randn(T, H, W, heads, d, generator=g, dtype=F64)
    dout = torch.randn(T, H, W, heads, d, generator=g, dtype=F64)
    off = (torch.rand(T, H, W, heads, 27, 3, generator=g, dtype=F64) - 0.5) * 1.8   # |off| < 0.9
    out, lse, dq, dk, dv, doff = run_oracle(q, k, v, off, window, dout)
    disp = torch.tensor(displacements(window), dtype=F64)
    scale = 1 / math.sqrt(d)
    checked = 0
    for (t, y, x) in itertools.product(range(2, 5), repeat=3):    # all samples stay interior
        pos = torch.tensor([t, y, x], dtype=F64) + disp + off[t, y, x, 0]          # [P,3]
        kp, vp = pos @ A.T + k0, pos @ B.T + v0
        s = kp @ q[t, y, x, 0] * scale
        a = torch.softmax(s, 0)
        assert torch.allclose(out[t, y, x, 0], a @ vp, rtol=0, atol=1e-12)
        assert torch.allclose(lse[t, y, x, 0], torch.logsumexp(s, 0), rtol=0, atol=1e-12)
        gp = vp @ dout[t, y, x, 0]
        dS = a * (gp - a @ gp)
        assert torch.allclose(dq[t, y, x, 0], scale * dS @ kp, rtol=0, atol=1e-12)
        ref_doff = scale * dS[:, None] * (q[t, y, x, 0] @ A)[None] + a[:, None] * (dout[t, y, x, 0] @ B)[None]
        assert torch.allclose(doff[t, y, x, 0], ref_doff, rtol=0, atol=1e-12)
        checked += 1
    assert checked == 27


def test_one_dimensional_linear_interpolation_and_partition_of_unity():
    T, H, W, heads, d, window = 1, 1, 6, 1, 2, (1, 1, 1)
    k = torch.arange(12, dtype=F64).view(T, H, W, heads, d) ** 2
    v = torch.ones(T, H, W, heads, d, dtype=F64) * 3.5          # constant field
    q = torch.ones(T, H, W, heads, d, dtype=F64)
    off = torch.zeros(T, H, W, heads, 1, 3, dtype=F64)
    off[0, 0, 2, 0, 0, 2] = 1.25                                 # x = 3.25
    out, lse = run_oracle(q, k, v, off, window)
    assert torch.allclose(out[0, 0, 2, 0], torch.full((2,), 3.5, dtype=F64), atol=1e-15)   # sum w = 1
    kp = 0.75 * k[0, 0, 3, 0] + 0.25 * k[0, 0, 4, 0]
    assert abs(lse[0, 0, 2, 0] - kp.sum() / math.sqrt(2)) < 1e-13


@pytest.mark.parametrize("window,sigma", [((3, 3, 3), 1.0), ((2, 2, 2), 2.5), ((1, 3, 3), 0.7)])
def test_matches_grid_sample_softmax_autograd(window, sigma):
    """The composition the paper describes (grid_sample for K and V, softmax, weighted sum)
    and autograd through it, including partly and fully out-of-range samples."""
    q, k, v, off, dout = rand_problem(3, 4, 5, 2, 4, window, sigma, seed=5)
    out, lse, dq, dk, dv, doff = run_oracle(q, k, v, off, window, dout)
    tq, tk, tv, toff = (z.clone().requires_grad_(True) for z in (q, k, v, off))
    ref_out, ref_lse = torch_grid_sample_dsa(tq, tk, tv, toff, window)
    (ref_out * dout).sum().backward()
    assert torch.allclose(out, ref_out.detach(), rtol=0, atol=1e-12)
    assert torch.allclose(lse, ref_lse.detach(), rtol=0, atol=1e-12)
    assert torch.allclose(dq, tq.grad, rtol=0, atol=1e-11)
    assert torch.allclose(dk, tk.grad, rtol=0, atol=1e-11)
    assert torch.allclose(dv, tv.grad, rtol=0, atol=1e-11)
    assert torch.allclose(doff, toff.grad, rtol=0, atol=1e-11)
    assert float(doff.abs().max()) > 1e-3          # the comparison is not vacuous


@pytest.mark.parametrize("dtype", [F64, torch.float32])
def test_grid_sample_on_exact_lattice_and_boundary_positions(dtype):
    """Sizes with size-1 a power of two make the normalisation exact, so positions exactly
    on integers, at -1 and at size agree with grid_sample including its one-sided
    derivative convention at the kinks."""
    T, H, W, heads, d, window = 3, 5, 9, 1, 2, (1, 1, 1)
    g = torch.Generator().manual_seed(6)
    q, k, v, _, dout = rand_problem(T, H, W, heads, d, window, 0.0, seed=6)
    pos = torch.stack([torch.randint(-8, 8 * (s + 1), (T, H, W, heads, 1), generator=g).to(F64) / 8
                       for s in (T, H, W)], -1)                     # multiples of 1/8 in [-1, size]
    coords = torch.tensor(tokens(T, H, W), dtype=F64).view(T, H, W, 1, 1, 3)
    off = pos - coords
    q, k, v, off, dout = (z.to(dtype) for z in (q, k, v, off, dout))    # all exactly representable
    out, lse, dq, dk, dv, doff = run_oracle(q, k, v, off, window, dout)
    q, k, v, off, dout = (z.to(F64) for z in (q, k, v, off, dout))
    tk, tv, toff = (z.clone().requires_grad_(True) for z in (k, v, off))
    ref_out, ref_lse = torch_grid_sample_dsa(q, tk, tv, toff, window)
    (ref_out * dout).sum().backward()
    assert torch.allclose(out, ref_out.detach(), rtol=0, atol=1e-13)
    assert torch.allclose(dk, tk.grad, rtol=0, atol=1e-13)
    assert torch.allclose(dv, tv.grad, rtol=0, atol=1e-13)
    assert torch.allclose(doff, toff.grad, rtol=0, atol=1e-12)


def test_zero_padding_hand_cases():
    T, H, W, heads, d, window = 1, 1, 4, 1, 2, (1, 1, 1)
    k = torch.tensor([[1.0, 2.0], [3.0, 5.0], [7.0, 11.0], [13.0, 17.0]], dtype=F64).view(T, H, W, heads, d)
    v = k * 2 + 1
    q = torch.ones(T, H, W, heads, d, dtype=F64)
    off = torch.zeros(T, H, W, heads, 1, 3, dtype=F64)
    off[0, 0, 0, 0, 0, 2] = -0.25          # x = -0.25: 0.75 * row 0, the other corner is outside
    off[0, 0, 1, 0, 0, 2] = -2.0           # x = -1 exactly: weight 0 on row 0
    off[0, 0, 2, 0, 0, 2] = 2.0            # x = size: nothing
    off[0, 0, 3, 0, 0, 2] = 0.5            # x = 3.5: 0.5 * row 3 (no renormalisation)
    out, lse = run_oracle(q, k, v, off, window)
    assert torch.allclose(out[0, 0, 0, 0], 0.75 * v[0, 0, 0, 0], atol=1e-15)
    assert torch.allclose(out[0, 0, 1, 0], torch.zeros(2, dtype=F64), atol=0)
    assert torch.allclose(out[0, 0, 2, 0], torch.zeros(2, dtype=F64), atol=0)
    assert torch.allclose(out[0, 0, 3, 0], 0.5 * v[0, 0, 3, 0], atol=1e-15)
    assert abs(lse[0, 0, 0, 0] - 0.75 * 3.0 / math.sqrt(2)) < 1e-14
    assert abs(lse[0, 0, 2, 0]) < 1e-15


def test_all_samples_outside_grid_gives_uniform_softmax_and_zero_output():
    window = (3, 3, 3)
    q, k, v, off, dout = rand_problem(2, 3, 3, 2, 4, window, 0.0, seed=8)
    off = torch.full_like(off, 50.0)
    off[0, 0, 0] = float("nan")
    off[0, 0, 1] = float("inf")
    off[0, 0, 2] = -1e30
    out, lse, dq, dk, dv, doff = run_oracle(q, k, v, off, window, dout)
    assert torch.equal(out, torch.zeros_like(out))
    assert torch.allclose(lse, torch.full_like(lse, math.log(27)), atol=1e-15)
    for z in (dq, dk, dv, doff):
        assert torch.equal(z, torch.zeros_like(z))


def test_dead_samples_stay_in_the_softmax():
    """One live sample among P: its weight is exp(s)/(exp(s) + P - 1), not 1."""
    T, H, W, heads, d, window = 1, 1, 2, 1, 2, (1, 1, 3)
    q, k, v, off, _ = rand_problem(T, H, W, heads, d, window, 0.0, seed=9)
    off = torch.zeros_like(off)
    off[..., 0, 2] = -40.0
    off[..., 2, 2] = 40.0
    out, lse = run_oracle(q, k, v, off, window)
    for x in range(2):
        s = float(q[0, 0, x, 0] @ k[0, 0, x, 0]) / math.sqrt(d)
        a = math.exp(s) / (math.exp(s) + 2.0)
        assert torch.allclose(out[0, 0, x, 0], a * v[0, 0, x, 0], atol=1e-14)
        assert abs(float(lse[0, 0, x, 0]) - math.log(math.exp(s) + 2.0)) < 1e-14


def test_single_cell_window_returns_sampled_value():
    window = (1, 1, 1)
    q, k, v, off, dout = rand_problem(3, 3, 3, 2, 4, window, 0.4, seed=10)
    out, lse, dq, dk, dv, doff = run_oracle(q, k, v, off, window, dout)
    tv, toff = v.clone().requires_grad_(True), off.clone().requires_grad_(True)
    vs, _ = torch_grid_sample_dsa(q, k, tv, toff, window)       # softmax over one sample is 1
    (vs * dout).sum().backward()
    assert torch.allclose(out, vs.detach(), atol=1e-13)
    assert torch.equal(dq, torch.zeros_like(dq))
    assert torch.equal(dk, torch.zeros_like(dk))
    assert torch.allclose(dv, tv.grad, atol=1e-13)
    assert torch.allclose(doff, toff.grad, atol=1e-12)


def test_softmax_sums_to_one_and_shift_invariances():
    T, H, W, heads, d, window = 6, 6, 6, 2, 4, (3, 3, 3)
    q, k, v, off, _ = rand_problem(T, H, W, heads, d, window, 0.3, seed=11)
    off = off.clamp(-0.9, 0.9)
    out, lse, alpha = oracle.forward(q, k, v, off, T, H, W, heads, d, window, return_alpha=True)
    assert torch.allclose(alpha.sum(-1), torch.ones(T * H * W, heads, dtype=F64), atol=1e-14)
    cv, ck = torch.randn(d, dtype=F64), torch.randn(d, dtype=F64)
    out_v, _ = oracle.forward(q, k, v + cv, off, T, H, W, heads, d, window)
    out_k, _, alpha_k = oracle.forward(q, k + ck, v, off, T, H, W, heads, d, window, return_alpha=True)
    inner = torch.zeros(T, H, W, dtype=torch.bool)
    inner[2:4, 2:4, 2:4] = True                      # every corner of every sample is inside
    inner = inner.view(-1)
    assert torch.allclose(out_v[inner], out[inner] + cv, atol=1e-13)
    assert torch.allclose(alpha_k[inner], alpha[inner], atol=1e-13)
    assert torch.allclose(out_k[inner], out[inner], atol=1e-13)
    assert not torch.allclose(out_v[~inner], out[~inner] + cv, atol=1e-6)   # padding breaks it


@pytest.mark.parametrize("window,sigma", [((3, 3, 3), 1.0), ((2, 2, 2), 0.6)])
def test_backward_matches_central_finite_differences(window, sigma):
    T, H, W, heads, d = 3, 4, 5, 2, 4
    q, k, v, off, dout = rand_problem(T, H, W, heads, d, window, sigma, seed=12)
    _, _, dq, dk, dv, doff = run_oracle(q, k, v, off, window, dout)

    def loss(q_, k_, v_, off_):
        o, _ = oracle.forward(q_, k_, v_, off_, T, H, W, heads, d, window)
        return float((o.view_as(dout) * dout).sum())

    g = torch.Generator().manual_seed(13)
    eps = 1e-6
    args = [q, k, v, off]
    for which, grad in enumerate([dq, dk, dv, doff]):
        flat = args[which].reshape(-1)
        for idx in torch.randint(0, flat.numel(), (12,), generator=g).tolist():
            plus, minus = [a.clone() for a in args], [a.clone() for a in args]
            plus[which].view(-1)[idx] += eps
            minus[which].view(-1)[idx] -= eps
            fd = (loss(*plus) - loss(*minus)) / (2 * eps)
            assert abs(fd - float(grad.reshape(-1)[idx])) < 2e-8, (which, idx)


def test_bilinearity_invariants():
    """sum <q, dQ> = sum <K, dK> (logits are bilinear in q and K); sum <V, dV> = sum <out, dO>
    (the output is linear in V).  Hold per head for any offsets, padding included."""
    window = (3, 3, 3)
    q, k, v, off, dout = rand_problem(4, 5, 5, 3, 8, window, 1.5, seed=14)
    out, _, dq, dk, dv, _ = run_oracle(q, k, v, off, window, dout)
    for m in range(3):
        i1a, i1b = (q[..., m, :] * dq[..., m, :]).sum(), (k[..., m, :] * dk[..., m, :]).sum()
        i2a, i2b = (v[..., m, :] * dv[..., m, :]).sum(), (out[..., m, :] * dout[..., m, :]).sum()
        assert abs(i1a - i1b) < 1e-11 * max(1.0, abs(i1a))
        assert abs(i2a - i2b) < 1e-11 * max(1.0, abs(i2a))


def test_translation_equivariance_in_the_interior():
    T, H, W, heads, d, window = 8, 8, 8, 1, 3, (3, 3, 3)
    q, k, v, off, _ = rand_problem(T, H, W, heads, d, window, 0.3, seed=15)
    off = off.clamp(-0.9, 0.9)
    out, lse = run_oracle(q, k, v, off, window)
    sh = (1, 2, -1)
    rolled = [torch.roll(z, sh, (0, 1, 2)) for z in (q, k, v, off)]
    out2, lse2 = run_oracle(*rolled, window)
    # queries whose samples stay clear of the wrap-around seam in both versions
    a = out[2:4, 2:4, 3:5]
    b = out2[2 + sh[0]:4 + sh[0], 2 + sh[1]:4 + sh[1], 3 + sh[2]:5 + sh[2]]
    assert torch.allclose(a, b, atol=1e-13)


def test_fp32_position_rounding_decides_the_cell():
    """With fp32 offsets the position is rounded to fp32 before the floor: 200 + 1e-6
    is exactly 200 in fp32, so the sample is an exact gather; in fp64 it is not."""
    T, H, W, heads, d, window = 1, 1, 256, 1, 2, (1, 1, 1)
    g = torch.Generator().manual_seed(16)
    k64 = torch.randn(T, H, W, heads, d, generator=g, dtype=F64)
    q64 = torch.ones(T, H, W, heads, d, dtype=F64)
    off64 = torch.zeros(T, H, W, heads, 1, 3, dtype=F64)
    off64[0, 0, 200, 0, 0, 2] = -1e-6
    out32, _ = oracle.forward(q64.float(), k64.float(), k64.float(), off64.float(), T, H, W, heads, d, window)
    out64, _ = oracle.forward(q64, k64, k64, off64, T, H, W, heads, d, window)
    assert torch.equal(out32[200, 0], k64.float().to(F64)[0, 0, 200, 0])
    expect = (1 - 1e-6) * k64[0, 0, 200, 0] + 1e-6 * k64[0, 0, 199, 0]
    assert torch.allclose(out64[200, 0], expect, atol=1e-15)
    assert not torch.equal(out64[200, 0], k64[0, 0, 200, 0])


def test_bf16_storage_is_read_exactly():
    window = (2, 2, 2)
    q, k, v, off, dout = rand_problem(3, 3, 3, 2, 8, window, 1.0, dtype=torch.bfloat16, seed=17)
    res_bf = run_oracle(q, k, v, off, window, dout)
    res_f32 = run_oracle(q.float(), k.float(), v.float(), off, window, dout.float())
    for a, b in zip(res_bf, res_f32):
        assert torch.equal(a, b)


def test_query_and_key_subsets_match_the_full_result():
    window = (3, 3, 3)
    T, H, W, heads, d = 4, 5, 6, 2, 4
    q, k, v, off, dout = rand_problem(T, H, W, heads, d, window, 1.2, dtype=torch.float32, seed=18)
    N = T * H * W
    out, lse = oracle.forward(q, k, v, off, T, H, W, heads, d, window)
    dq, dk, dv, doff = oracle.backward(q, k, v, off, dout, T, H, W, heads, d, window)
    qtok = torch.tensor([5, 0, N - 1, 37, 64])
    rows = lambda z, width: z.reshape(N, heads, *width)[qtok]
    o2, l2 = oracle.forward(rows(q, (d,)), k, v, rows(off, (27, 3)), T, H, W, heads, d, window, qtok=qtok)
    assert torch.equal(o2, out[qtok]) and torch.equal(l2, lse[qtok])
    ktok = torch.tensor([3, 77, N - 1, 0])
    dq2, dk2, dv2, doff2 = oracle.backward(q, k, v, off, dout, T, H, W, heads, d, window, ktok=ktok)
    assert torch.equal(dq2, dq) and torch.equal(doff2, doff)
    assert torch.equal(dk2, dk[ktok]) and torch.equal(dv2, dv[ktok])
    dq3, dk3, _, doff3 = oracle.backward(rows(q, (d,)), k, v, rows(off, (27, 3)), rows(dout, (d,)),
                                         T, H, W, heads, d, window, qtok=qtok)
    assert torch.equal(dq3, dq[qtok]) and torch.equal(doff3, doff[qtok])
    assert float(dk3.abs().sum()) < float(dk.abs().sum())       # only these queries contribute
