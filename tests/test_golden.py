"""The stored small case (tests/golden/dsa3d_small_case.json, written by
tests/golden/make_golden.py from the oracle alone): the oracle must reproduce it (to 1e-12
relative: the last bit of exp/log may differ between C libraries), and the CUDA path must match
it within the fp32 tolerances."""
import json
import os

import pytest
import torch

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def _load():
    with open(os.path.join(HERE, "golden", "dsa3d_small_case.json")) as f:
        case = json.load(f)
    T, H, W, heads, d = case["dims"]
    P = case["window"][0] * case["window"][1] * case["window"][2]
    f32 = lambda name, shape: torch.tensor(case["inputs"][name], dtype=torch.float32).view(shape)
    t = {n: f32(n, (T, H, W, heads, d)) for n in ("q", "k", "v", "dout")}
    t["offsets"] = f32("offsets", (T, H, W, heads, P, 3))
    exp = {n: torch.tensor(vals, dtype=torch.float64) for n, vals in case["expected_fp64"].items()}
    return case, t, exp


def test_oracle_reproduces_the_stored_case():
    case, t, exp = _load()
    T, H, W, heads, d = case["dims"]
    window = tuple(case["window"])
    P = window[0] * window[1] * window[2]
    out, lse = oracle.forward(t["q"].view(-1, heads, d), t["k"], t["v"], t["offsets"].view(-1, heads, P, 3),
                              T, H, W, heads, d, window)
    grads = oracle.backward(t["q"].view(-1, heads, d), t["k"], t["v"], t["offsets"].view(-1, heads, P, 3),
                            t["dout"].view(-1, heads, d), T, H, W, heads, d, window)
    for name, got in zip(("out", "lse", "dq", "dk", "dv", "doffsets"), (out, lse) + tuple(grads)):
        got = got.reshape(-1).double()
        assert bool(((got - exp[name]).abs() <= 1e-12 * exp[name].abs().clamp_min(1.0)).all()), name
    # the case was built to contain a dead sample: its offset gradient is exactly zero
    assert torch.equal(exp["doffsets"].view(T, H, W, heads, P, 3)[1, 1, 2, 0, 7], torch.zeros(3, dtype=torch.float64))


@pytest.mark.gpu
def test_cuda_path_matches_the_stored_case():
    from paper_2607_22696_b200 import binding
    case, t, exp = _load()
    T, H, W, heads, d = case["dims"]
    window = tuple(case["window"])
    dev = {n: z.cuda() for n, z in t.items()}
    out = torch.empty_like(dev["q"])
    lse = torch.empty((T, H, W, heads), dtype=torch.float32, device="cuda")
    binding.dsa3d_forward(dev["q"], dev["k"], dev["v"], dev["offsets"], T, H, W, heads, d, window, out, lse)
    dq, dk, dv = (torch.empty_like(dev["q"]) for _ in range(3))
    doff = torch.empty_like(dev["offsets"])
    binding.dsa3d_backward(dev["q"], dev["k"], dev["v"], dev["offsets"], lse, dev["dout"], T, H, W, heads, d, window,
                           dq, dk, dv, doff, None)
    torch.cuda.synchronize()
    for name, got, tol in (("out", out, 1e-5), ("lse", lse, 1e-5), ("dq", dq, 1e-4), ("dk", dk, 1e-4), ("dv", dv, 1e-4),
                           ("doffsets", doff, 1e-4)):
        err = float((got.cpu().double().reshape(-1) - exp[name]).abs().max())
        assert err <= tol, (name, err)
