"""dsa3d_backward_noalloc: the backward for callers that cannot give the library scratch
memory (pre-planned memory regions, plug-ins without access to the host's allocator,
loops that must not hit cudaMalloc's device-wide synchronisation).  Its accumulators sit in
a fixed array inside the library, shared by all calls, so the test calls it twice in a row
(the second call must not see the first call's sums) and compares both against the
workspace variant through the C ABI.

This file sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import ctypes

import pytest
import torch

from paper_2607_22696_b200 import binding, inputs


def _problem(seed, dims, window, device):
    T, H, W, heads, d = dims
    wl = inputs.Workload("noalloc", T, H, W, heads, d, window, torch.bfloat16, 1.2, seed)
    return {n: z.to(device) for n, z in inputs.make_inputs(wl, "cpu", with_dout=True).items()}


def _raw_backward(lib, fn_name, t, lse, dims, window, with_workspace):
    """Call the C entry point directly with device addresses."""
    T, H, W, heads, d = dims
    outs = [torch.full_like(t["q"], float("nan")) for _ in range(3)] + [torch.full_like(t["offsets"], float("nan"))]
    win = (ctypes.c_int * 3)(*window)
    args = [t["q"].data_ptr(), t["k"].data_ptr(), t["v"].data_ptr(), t["offsets"].data_ptr(), lse.data_ptr(),
            t["dout"].data_ptr(), T, H, W, heads, d, win] + [o.data_ptr() for o in outs]
    ws = None
    if with_workspace:
        nbytes = lib.dsa3d_backward_workspace_bytes(T, H, W, heads, d, win, binding.DSA3D_BF16)
        ws = torch.empty(nbytes, dtype=torch.uint8, device=t["q"].device)
        args += [ws.data_ptr(), nbytes]
    args += [binding.DSA3D_BF16, torch.cuda.current_stream().cuda_stream or None]
    status = getattr(lib, fn_name)(*args)
    torch.cuda.synchronize()
    return status, outs


def _close(a, b):
    a, b = a.float(), b.float()
    rms = float(b.pow(2).mean().sqrt())
    return bool(((a - b).abs() <= 2e-2 * torch.clamp(b.abs(), min=rms) + 1e-4).all())


@pytest.mark.gpu
def test_noalloc_backward_matches_workspace_backward_twice_in_a_row():
    lib = binding.load()
    window = (3, 3, 3)
    for seed, dims in ((101, (6, 12, 14, 4, 128)), (102, (5, 9, 11, 3, 64))):    # two different problems
        t = _problem(seed, dims, window, "cuda")
        out = torch.empty_like(t["q"])
        lse = torch.empty(dims[:4], dtype=torch.float32, device="cuda")
        binding.dsa3d_forward(t["q"], t["k"], t["v"], t["offsets"], *dims, window, out, lse)
        status, ref = _raw_backward(lib, "dsa3d_backward", t, lse, dims, window, with_workspace=True)
        assert status == 0
        for attempt in range(2):
            status, got = _raw_backward(lib, "dsa3d_backward_noalloc", t, lse, dims, window, with_workspace=False)
            assert status == 0, lib.dsa3d_status_string(status)
            assert torch.equal(got[0], ref[0]) and torch.equal(got[3], ref[3])     # dq, doffsets: deterministic
            assert _close(got[1], ref[1]) and _close(got[2], ref[2]), (seed, attempt)  # dk, dv: atomic order
            assert float(got[1].float().abs().max()) > 0


@pytest.mark.gpu
def test_noalloc_backward_matches_the_oracle():
    """All four gradients of the no-allocation entry point against the CPU oracle directly (not
    only against dsa3d_backward), at the tolerances of the parity tests."""
    import oracle
    import parity_util as pu
    lib = binding.load()
    window, dims = (3, 3, 3), (4, 7, 9, 3, 128)
    T, H, W, heads, d = dims
    wl = inputs.Workload("noalloc_oracle", T, H, W, heads, d, window, torch.bfloat16, 1.2, 103)
    host = inputs.make_inputs(wl, "cpu", with_dout=True)
    t = {n: z.cuda() for n, z in host.items()}
    out = torch.empty_like(t["q"])
    lse = torch.empty(dims[:4], dtype=torch.float32, device="cuda")
    binding.dsa3d_forward(t["q"], t["k"], t["v"], t["offsets"], *dims, window, out, lse)
    status, got = _raw_backward(lib, "dsa3d_backward_noalloc", t, lse, dims, window, with_workspace=False)
    assert status == 0
    refs = oracle.backward(host["q"], host["k"], host["v"], host["offsets"], host["dout"], T, H, W, heads, d, window)
    for name, g, r in zip(("dq", "dk", "dv", "doffsets"), got, refs):
        pu.assert_close(name, g, r, torch.bfloat16, backward=True)


@pytest.mark.gpu
def test_noalloc_backward_rejects_problems_beyond_its_fixed_array():
    lib = binding.load()
    limit = lib.dsa3d_backward_noalloc_max_elements()
    assert limit == 8 * 1024 * 1024
    win = (ctypes.c_int * 3)(3, 3, 3)
    a = 4096                                              # never dereferenced: the size check comes first
    too_big = [a] * 6 + [64, 64, 64, 4, 128, win] + [a] * 4 + [binding.DSA3D_BF16, None]
    assert 64 * 64 * 64 * 4 * 128 > limit
    assert lib.dsa3d_backward_noalloc(*too_big) == 5
    assert b"workspace" in lib.dsa3d_status_string(5)


def test_noalloc_size_check_needs_no_gpu():
    """Host-only: the limit is enforced before any CUDA call, and bad shapes still get the
    ordinary status."""
    lib = binding.load()
    win = (ctypes.c_int * 3)(3, 3, 3)
    a = 4096
    assert lib.dsa3d_backward_noalloc(*([a] * 6 + [1 << 20, 1 << 20, 1 << 20, 1 << 20, 128, win] + [a] * 4 + [1, None])) == 5
    assert lib.dsa3d_backward_noalloc(*([a] * 6 + [0, 8, 8, 2, 32, win] + [a] * 4 + [1, None])) == 2
    assert lib.dsa3d_backward_noalloc(*([a] * 6 + [4, 8, 8, 2, 32, None] + [a] * 4 + [1, None])) == 1
