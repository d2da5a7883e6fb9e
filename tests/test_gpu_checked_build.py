"""The bounds-checked build of the library (compiled with -DDSA3D_DEBUG into libdsa3d_debug.so).

In that build every K/V row a sample is about to gather, every dK/dV row a contribution is about
to be added to and every bin and scratch slot of the dK/dV pre-reduction is tested against the
extent of its tensor first; a violation would be recorded in a device word (and the access
skipped: nothing traps).  The small parity cases run once through it: the results must match the
oracle as in the normal build and the record must stay empty - on problems whose offsets reach far
outside the grid, are NaN or infinite, on grids with extents of one, and through both dK/dV paths."""
import ctypes

import pytest
import torch

import oracle
import parity_util as pu
from paper_2607_22696_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _win(window):
    return (ctypes.c_int * 3)(*window)


def _run_checked(lib, host, dims, window, dtype):
    T, H, W, heads, d = dims
    code = binding.DSA3D_BF16 if dtype == torch.bfloat16 else binding.DSA3D_F32
    dev = {n: z.cuda() for n, z in host.items()}
    out = torch.full_like(dev["q"], float("nan"))
    lse = torch.full((T, H, W, heads), float("nan"), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream or None
    assert lib.dsa3d_forward(dev["q"].data_ptr(), dev["k"].data_ptr(), dev["v"].data_ptr(), dev["offsets"].data_ptr(),
                             T, H, W, heads, d, _win(window), out.data_ptr(), lse.data_ptr(), code, stream) == 0
    grads = [torch.full_like(dev["q"], float("nan")) for _ in range(3)] + [torch.full_like(dev["offsets"], float("nan"))]
    nbytes = lib.dsa3d_backward_workspace_bytes(T, H, W, heads, d, _win(window), code)
    ws = torch.full((max(nbytes, 16),), 0xFF, dtype=torch.uint8, device="cuda")
    assert lib.dsa3d_backward(dev["q"].data_ptr(), dev["k"].data_ptr(), dev["v"].data_ptr(), dev["offsets"].data_ptr(),
                              lse.data_ptr(), dev["dout"].data_ptr(), T, H, W, heads, d, _win(window),
                              *[g.data_ptr() for g in grads], ws.data_ptr(), nbytes, code, stream) == 0
    torch.cuda.synchronize()
    return out, lse, grads


def _violation(lib):
    code, off = ctypes.c_int(-1), ctypes.c_longlong(-1)
    assert lib.dsa3d_debug_first_violation(ctypes.byref(code), ctypes.byref(off)) == 0
    return code.value, off.value


CASES = [
    # (T, H, W, heads, d), window, dtype, sigma, what the offsets are made of
    ((4, 8, 8, 2, 32), (3, 3, 3), torch.float32, 0.5, "normal"),
    ((5, 7, 9, 3, 128), (3, 3, 3), torch.bfloat16, 2.5, "normal"),       # the tile pre-reduction of dK/dV
    ((4, 9, 10, 2, 64), (3, 5, 5), torch.bfloat16, 1.5, "normal"),
    ((1, 1, 40, 2, 128), (3, 3, 3), torch.bfloat16, 0.7, "normal"),      # extents of one
    ((4, 5, 6, 2, 32), (3, 3, 3), torch.float32, 1.0, "wild"),           # NaN, +-inf, 3e38, far outside
    ((5, 6, 7, 2, 64), (3, 3, 3), torch.bfloat16, 0.0, "integer"),       # positions exactly at -1 and at size
]


@pytest.mark.parametrize("key_blocks", [False, True])
@pytest.mark.parametrize("dims,window,dtype,sigma,kind", CASES)
def test_parity_cases_leave_no_violation_in_the_checked_build(dims, window, dtype, sigma, kind, key_blocks, monkeypatch):
    if key_blocks:
        if dtype != torch.bfloat16 or dims[4] < 64:
            pytest.skip("the key-block kernel takes bf16 rows of 64 or 128 channels")
        monkeypatch.setenv("DSA3D_KEY_BLOCKS", "1")       # dK/dV on the tensor cores instead of the tile kernel
    lib = binding.load_checked_build()
    assert lib.dsa3d_debug_build() == 1 and binding.load().dsa3d_debug_build() == 0
    assert lib.dsa3d_debug_clear() == 0
    T, H, W, heads, d = dims
    wl = inputs.Workload("checked", T, H, W, heads, d, window, dtype, max(sigma, 0.1), 500 + T * H)
    host = inputs.make_inputs(wl, "cpu", with_dout=True)
    off = host["offsets"]
    if kind == "wild":
        flat = off.view(-1, 3)
        flat[0::7, 0] = float("nan")
        flat[1::7, 1] = float("inf")
        flat[2::7, 2] = -float("inf")
        flat[3::7, 0] = 3e38
        flat[4::7, 1] = -1e30
        flat[5::7, 2] = 1000.0
    elif kind == "integer":
        host["offsets"] = inputs.uniform_int(off.shape, 501, 3, -3, 3, torch.float32)
    out, lse, grads = _run_checked(lib, host, dims, window, dtype)
    assert _violation(lib) == (0, 0)
    o_ref, l_ref = oracle.forward(host["q"], host["k"], host["v"], host["offsets"], T, H, W, heads, d, window)
    refs = oracle.backward(host["q"], host["k"], host["v"], host["offsets"], host["dout"], T, H, W, heads, d, window)
    pu.assert_close("out", out, o_ref, dtype)
    pu.assert_close("lse", lse, l_ref, dtype)
    for name, got, ref in zip(("dq", "dk", "dv", "doffsets"), grads, refs):
        pu.assert_close(name, got, ref, dtype, backward=True)


def test_the_normal_build_reports_no_checks():
    lib = binding.load()
    assert lib.dsa3d_debug_build() == 0
    assert _violation(lib) == (0, 0)
    assert lib.dsa3d_debug_clear() == 0
