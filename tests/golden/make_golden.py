"""Writes tests/golden/dsa3d_small_case.json: a tiny 3D-DSA problem (inputs stored, so the file
does not depend on any generator) and the oracle's forward and backward results for it.

Run from the repository root:  python tests/golden/make_golden.py
Calls only the CPU oracle.  The stored values guard the oracle against silent drift (a CPU test
recomputes them exactly) and give the CUDA path a fixed target (a GPU test compares within the
fp32 tolerances).  The problem: grid 2 x 2 x 3, one head of 32 channels, window 2 x 2 x 2, fp32,
offsets of about one grid unit, so that samples fall outside the grid on every side.
"""
import json
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402


def main():
    T, H, W, heads, d, window = 2, 2, 3, 1, 32, (2, 2, 2)
    P = 8
    g = torch.Generator().manual_seed(20260725)
    shape = (T, H, W, heads, d)
    q, k, v, dout = (torch.randn(shape, generator=g, dtype=torch.float32) for _ in range(4))
    off = torch.randn((T, H, W, heads, P, 3), generator=g, dtype=torch.float32)
    off[0, 0, 0, 0, 0] = torch.tensor([0.0, 0.0, 0.0])          # a sample exactly on a grid position
    off[1, 1, 2, 0, 7] = torch.tensor([5.0, 0.25, -0.5])        # a dead sample (beyond the last frame)
    out, lse = oracle.forward(q.view(-1, heads, d), k, v, off.view(-1, heads, P, 3), T, H, W, heads, d, window)
    dq, dk, dv, doff = oracle.backward(q.view(-1, heads, d), k, v, off.view(-1, heads, P, 3), dout.view(-1, heads, d),
                                       T, H, W, heads, d, window)
    flat = lambda z: [float(x) for x in z.reshape(-1).tolist()]
    # fp32 inputs: nine significant digits identify a float32 exactly
    flat32 = lambda z: [float(f"{float(x):.9g}") for x in z.reshape(-1).tolist()]
    case = {"dims": [T, H, W, heads, d], "window": list(window), "dtype": "float32",
            "inputs": {"q": flat32(q), "k": flat32(k), "v": flat32(v), "dout": flat32(dout), "offsets": flat32(off)},
            "expected_fp64": {"out": flat(out), "lse": flat(lse), "dq": flat(dq), "dk": flat(dk), "dv": flat(dv),
                              "doffsets": flat(doff)}}
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "dsa3d_small_case.json")
    with open(path, "w") as f:
        json.dump(case, f)
    print(path, os.path.getsize(path), "bytes")


if __name__ == "__main__":
    main()
