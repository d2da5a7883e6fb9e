"""Host-side checks of the C ABI: the library loads, exports every symbol the header
declares, and rejects bad arguments with the documented status before launching."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2607_22696_b200 import build, binding
    build.build()
    return binding.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dsa3d.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dsa3d_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_expected_entry_points():
    syms = declared_symbols()
    for name in ["dsa3d_forward", "dsa3d_backward", "dsa3d_backward_workspace_bytes",
                 "dsa3d_status_string", "dsa3d_last_cuda_error"]:
        assert name in syms


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert lib.dsa3d_status_string(0) == b"success"
    for code in range(1, 8):
        s = lib.dsa3d_status_string(code)
        assert s and s != b"unknown status"
    assert lib.dsa3d_status_string(99) == b"unknown status"


def test_workspace_size(lib):
    win = (ctypes.c_int * 3)(3, 3, 3)
    assert lib.dsa3d_backward_workspace_bytes(4, 8, 8, 2, 32, win, 0) == 0
    # bf16: fp32 dK/dV accumulators + two fp32 coefficients per sample (section rounded up to
    # 256 bytes) + the tile bins, whose size depends on the tiling only
    up = lambda x: (x + 255) // 256 * 256
    small = lib.dsa3d_backward_workspace_bytes(4, 8, 8, 2, 32, win, 1)
    small_fixed = 256 * 2 * 32 * 4 * 2 + up(256 * 2 * 27 * 8)
    assert small > small_fixed
    big = lib.dsa3d_backward_workspace_bytes(256, 68, 120, 16, 128, win, 1)
    items = 2088960 * 16
    assert big - (items * 128 * 4 * 2 + up(items * 27 * 8)) == small - small_fixed
    assert big < 45 * 10**9
    odd = lib.dsa3d_backward_workspace_bytes(5, 7, 9, 3, 32, win, 1)       # 945 items: unaligned sizes
    assert (odd - (small - small_fixed)) % 256 == 0
    assert lib.dsa3d_backward_workspace_bytes(4, 8, 8, 2, 48, win, 1) == 0      # rejected shape


def test_forward_rejects_bad_arguments_without_launching(lib):
    win = (ctypes.c_int * 3)(3, 3, 3)
    a = 4096                                     # fake, aligned, never dereferenced
    ok = [a, a, a, a, 4, 8, 8, 2, 32, win, a, a, 0, None]

    def call(**kw):
        args = list(ok)
        for idx, val in kw.items():
            args[int(idx[1:])] = val
        return lib.dsa3d_forward(*args)

    assert call(_0=None) == 1
    assert call(_10=None) == 1
    assert call(_9=None) == 1
    assert call(_4=0) == 2
    assert call(_7=-1) == 2
    assert call(_9=(ctypes.c_int * 3)(3, 0, 3)) == 2
    assert call(_4=1 << 15, _5=1 << 15, _6=4) == 2           # 2^32 tokens
    assert call(_8=48) == 3
    assert call(_12=7) == 3
    assert call(_9=(ctypes.c_int * 3)(7, 7, 7)) == 3         # P = 343 > 256
    assert call(_1=a + 8) == 4
    assert call(_11=a + 4) == 4


def test_backward_rejects_bad_arguments_without_launching(lib):
    win = (ctypes.c_int * 3)(3, 3, 3)
    a = 4096
    ok = [a, a, a, a, a, a, 4, 8, 8, 2, 32, win, a, a, a, a, a, 1 << 30, 1, None]

    def call(**kw):
        args = list(ok)
        for idx, val in kw.items():
            args[int(idx[1:])] = val
        return lib.dsa3d_backward(*args)

    assert call(_5=None) == 1
    assert call(_15=None) == 1
    assert call(_10=100) == 3
    assert call(_16=None) == 5
    assert call(_17=1024) == 5
    assert call(_16=a + 4) == 4
    assert call(_13=a + 2) == 4


def test_binding_refuses_cpu_tensors():
    import torch
    from paper_2607_22696_b200 import binding
    z = torch.zeros(4 * 8 * 8 * 2 * 32)
    off = torch.zeros(4 * 8 * 8 * 2 * 27 * 3)
    lse = torch.zeros(4 * 8 * 8 * 2)
    with pytest.raises(ValueError, match="CUDA tensor"):
        binding.dsa3d_forward(z, z, z, off, 4, 8, 8, 2, 32, (3, 3, 3), z, lse, stream=0)


def test_producer_entry_points_reject_bad_arguments_without_launching(lib):
    """The convolution, the linear layer and the forward with the convolution term validate
    their arguments before touching the device (fake aligned addresses, never dereferenced)."""
    a = 4096
    win = (ctypes.c_int * 3)(3, 3, 3)
    lib.dsa3d_dwconv3d_forward.restype = ctypes.c_int
    lib.dsa3d_dwconv3d_forward.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int] * 4 + \
        [ctypes.POINTER(ctypes.c_int), ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
    conv = lambda *args: lib.dsa3d_dwconv3d_forward(*args)
    assert conv(None, a, None, 2, 2, 2, 8, win, a, 1, None) == 1          # null x
    assert conv(a, a, None, 2, 2, 2, 12, win, a, 1, None) == 2            # channels not a multiple of 8
    assert conv(a, a, None, 0, 2, 2, 8, win, a, 1, None) == 2             # empty grid
    assert conv(a, a, None, 2, 2, 2, 8, (ctypes.c_int * 3)(3, 3, 9), a, 1, None) == 2   # kernel too wide
    assert conv(a, a, None, 2, 2, 2, 8, win, a, 5, None) == 3             # unknown dtype
    assert conv(a + 4, a, None, 2, 2, 2, 8, win, a, 1, None) == 4         # misaligned x

    lib.dsa3d_offsets_linear_forward.restype = ctypes.c_int
    lib.dsa3d_offsets_linear_forward.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_longlong, ctypes.c_int, ctypes.c_int,
                                                                        ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
    lin = lambda *args: lib.dsa3d_offsets_linear_forward(*args)
    assert lin(a, a, None, 16, 64, 81, a, 1, None) == 1                   # bias is required
    assert lin(a, a, a, 0, 64, 81, a, 1, None) == 2                       # no tokens
    assert lin(a, a, a, 16, 60, 81, a, 1, None) == 2                      # channels not a multiple of 8
    assert lin(a, a, a, 1 << 31, 64, 81, a, 1, None) == 2                 # too many tokens for the tile maps
    assert lin(a, a, a, 16, 64, 81, a, 7, None) == 3
    assert lin(a, a + 8, a, 16, 64, 81, a, 1, None) == 4

    lib.dsa3d_forward_residual.restype = ctypes.c_int
    lib.dsa3d_forward_residual.argtypes = [ctypes.c_void_p] * 5 + [ctypes.c_int] * 5 + \
        [ctypes.POINTER(ctypes.c_int), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
    res = lambda *args: lib.dsa3d_forward_residual(*args)
    assert res(a, a, a, a, None, 4, 8, 8, 2, 32, win, a, a, 0, None) == 1  # the term itself is required
    assert res(a, a, a, a, a + 2, 4, 8, 8, 2, 32, win, a, a, 0, None) == 4
    assert res(a, a, a, a, a, 4, 8, 8, 2, 48, win, a, a, 0, None) == 3     # head size not supported


def test_producer_backward_entry_points_reject_bad_arguments_without_launching(lib):
    """Gradients of the convolution and of the linear layer: every check runs before the first
    launch or copy (fake aligned addresses, never dereferenced), and the workspace queries need
    no device."""
    a = 4096
    win = (ctypes.c_int * 3)(3, 3, 3)
    vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.dsa3d_dwconv3d_backward_workspace_bytes.restype = sz
    lib.dsa3d_dwconv3d_backward_workspace_bytes.argtypes = [ci, ctypes.POINTER(ci)]
    assert lib.dsa3d_dwconv3d_backward_workspace_bytes(64, win) >= 27 * 64 * 4
    assert lib.dsa3d_dwconv3d_backward_workspace_bytes(0, win) == 0
    lib.dsa3d_dwconv3d_backward.restype = ci
    lib.dsa3d_dwconv3d_backward.argtypes = [vp, vp, vp, ci, ci, ci, ci, ctypes.POINTER(ci), vp, vp, vp, vp, sz, ci, vp]
    conv = lambda *args: lib.dsa3d_dwconv3d_backward(*args)
    assert conv(a, a, None, 2, 2, 2, 8, win, a, a, None, a, 1 << 20, 1, None) == 1      # dy is required
    assert conv(a, a, a, 2, 2, 2, 8, win, a, None, None, None, 0, 1, None) == 1         # dx needs a workspace
    assert conv(a, a, a, 2, 2, 2, 8, win, None, None, a, None, 0, 1, None) == 1         # dbias needs dweight
    assert conv(None, a, a, 2, 2, 2, 8, win, None, a, None, None, 0, 1, None) == 1      # dweight needs x
    assert conv(a, a, a, 2, 2, 2, 12, win, a, a, None, a, 1 << 20, 1, None) == 2        # channels
    assert conv(a, a, a, 2, 2, 2, 8, (ctypes.c_int * 3)(3, 16, 3), a, a, None, a, 1 << 20, 1, None) == 2
    assert conv(a, a, a, 2, 2, 2, 8, win, a, a, None, a, 1 << 20, 9, None) == 3         # dtype
    assert conv(a, a, a + 8, 2, 2, 2, 8, win, a, a, None, a, 1 << 20, 1, None) == 4     # misaligned dy
    assert conv(a, a, a, 2, 2, 2, 8, win, None, a, a + 4, None, 0, 1, None) == 4        # misaligned dbias
    assert conv(a, a, a, 2, 2, 2, 8, win, a, None, None, a, 16, 1, None) == 5           # workspace too small

    lib.dsa3d_offsets_linear_backward_workspace_bytes.restype = sz
    lib.dsa3d_offsets_linear_backward_workspace_bytes.argtypes = [ctypes.c_longlong, ci, ci, ci]
    need = lib.dsa3d_offsets_linear_backward_workspace_bytes(1000, 64, 81, 1)
    assert need >= 64 * 88 * 2 + 1000 * 88 * 2            # w^T and the bf16 copy, rows padded to 8 columns
    assert lib.dsa3d_offsets_linear_backward_workspace_bytes(1000, 64, 81, 0) == 0      # fp32 needs none
    # the slab bounds the workspace: beyond 262144 tokens it no longer grows
    assert lib.dsa3d_offsets_linear_backward_workspace_bytes(10 ** 7, 64, 81, 1) == \
        lib.dsa3d_offsets_linear_backward_workspace_bytes(262144, 64, 81, 1)
    lib.dsa3d_offsets_linear_backward.restype = ci
    lib.dsa3d_offsets_linear_backward.argtypes = [vp, vp, vp, ctypes.c_longlong, ci, ci, vp, vp, vp, vp, sz, ci, vp]
    lin = lambda *args: lib.dsa3d_offsets_linear_backward(*args)
    assert lin(a, a, None, 16, 64, 81, a, a, a, a, need, 1, None) == 1                  # doffsets is required
    assert lin(a, None, a, 16, 64, 81, a, None, None, a, need, 1, None) == 1            # du needs w
    assert lin(None, a, a, 16, 64, 81, None, a, None, a, need, 1, None) == 1            # dw needs u
    assert lin(a, a, a, 0, 64, 81, a, a, a, a, need, 1, None) == 2
    assert lin(a, a, a, 16, 60, 81, a, a, a, a, need, 1, None) == 2
    assert lin(a, a, a, 16, 64, 81, a, a, a, a, need, 4, None) == 3
    assert lin(a, a, a + 4, 16, 64, 81, a, a, a, a, need, 1, None) == 4
    assert lin(a, a, a, 16, 64, 81, a, a, a, None, 0, 1, None) == 1                     # bf16 needs its workspace
    assert lin(a, a, a, 16, 64, 81, a, a, a, a, 64, 1, None) == 5                       # too small
