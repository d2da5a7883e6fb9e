"""Thin ctypes binding of libdsa3d.so: same names and argument order as include/dsa3d.h.

Only argument marshalling happens here (tensor -> device pointer, window -> int[3],
status -> exception).  Every step of the operator runs in the library's CUDA kernels; there
is no fallback: if the shared library is missing or a tensor is not on a CUDA device the
call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdsa3d.so")

DSA3D_F32, DSA3D_BF16 = 0, 1
_DTYPES = {torch.float32: DSA3D_F32, torch.bfloat16: DSA3D_BF16}

_lib = None


class Dsa3dError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"dsa3d status {status}: {message}")
        self.status = status


def load():
    """Load libdsa3d.so (built by paper_2607_22696_b200.build) and declare its prototypes."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2607_22696_b200.build`; "
            "there is no CPU or PyTorch fallback for this operator")
    lib = ctypes.CDLL(LIB_PATH)
    _declare(lib)
    _lib = lib
    return lib


def load_checked_build():
    """The bounds-checked build of the library (libdsa3d_debug.so, see include/dsa3d.h) as a ctypes
    handle of its own with the same prototypes; the functions of this module keep using the normal
    build.  Built on first use."""
    from . import build as _build
    lib = ctypes.CDLL(_build.build(debug=True))
    _declare(lib)
    return lib


def _declare(lib) -> None:
    p, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    win = ctypes.POINTER(ctypes.c_int)
    lib.dsa3d_forward.restype = i
    lib.dsa3d_forward.argtypes = [p, p, p, p, i, i, i, i, i, win, p, p, i, p]
    lib.dsa3d_backward.restype = i
    lib.dsa3d_backward.argtypes = [p, p, p, p, p, p, i, i, i, i, i, win, p, p, p, p, p, sz, i, p]
    lib.dsa3d_backward_workspace_bytes.restype = sz
    lib.dsa3d_backward_workspace_bytes.argtypes = [i, i, i, i, i, win, i]
    lib.dsa3d_backward_bounded_offsets.restype = i
    lib.dsa3d_backward_bounded_offsets.argtypes = [p, p, p, p, p, p, i, i, i, i, i, win, p, p, p, p, p, sz, i, p]
    lib.dsa3d_backward_bounded_offsets_workspace_bytes.restype = sz
    lib.dsa3d_backward_bounded_offsets_workspace_bytes.argtypes = [i, i, i, i, i, win, i]
    lib.dsa3d_step_host.restype = i
    lib.dsa3d_step_host.argtypes = [p, p, p, p, p, i, i, i, i, i, win, p, p, p, p, p, p, p, sz, i, p]
    lib.dsa3d_step_host_pipelined.restype = i
    lib.dsa3d_step_host_pipelined.argtypes = [p, p, p, p, p, i, i, i, i, i, win, p, p, p, p, p, p, p, sz, i, p]
    lib.dsa3d_step_host_flush.restype = i
    lib.dsa3d_step_host_flush.argtypes = [p]
    lib.dsa3d_step_host_arena_bytes.restype = sz
    lib.dsa3d_step_host_arena_bytes.argtypes = [i, i, i, i, i, win, i]
    lib.dsa3d_set_profile_events.restype = i
    lib.dsa3d_set_profile_events.argtypes = [p, p, p, p, p, p]
    lib.dsa3d_backward_noalloc.restype = i
    lib.dsa3d_backward_noalloc.argtypes = [p, p, p, p, p, p, i, i, i, i, i, win, p, p, p, p, i, p]
    lib.dsa3d_backward_noalloc_max_elements.restype = sz
    lib.dsa3d_backward_noalloc_max_elements.argtypes = []
    lib.dsa3d_backward_noalloc_last_cuda_error.restype = i
    lib.dsa3d_backward_noalloc_last_cuda_error.argtypes = []
    dptr = ctypes.POINTER(ctypes.c_double)
    lib.dsa3d_probe_gather.restype = i
    lib.dsa3d_probe_gather.argtypes = [p, sz, i, dptr, p]
    lib.dsa3d_probe_red.restype = i
    lib.dsa3d_probe_red.argtypes = [p, sz, i, dptr, p]
    lib.dsa3d_probe_fma.restype = i
    lib.dsa3d_probe_fma.argtypes = [p, i, i, dptr, p]
    lib.dsa3d_forward_batch.restype = i
    lib.dsa3d_forward_batch.argtypes = [p, p, p, p, i, i, i, i, i, i, win, p, p, i, p]
    lib.dsa3d_backward_batch.restype = i
    lib.dsa3d_backward_batch.argtypes = [p, p, p, p, p, p, i, i, i, i, i, i, win, p, p, p, p, p, sz, i, p]
    lib.dsa3d_dwconv3d_forward.restype = i
    lib.dsa3d_dwconv3d_forward.argtypes = [p, p, p, i, i, i, i, win, p, i, p]
    lib.dsa3d_offsets_linear_forward.restype = i
    lib.dsa3d_offsets_linear_forward.argtypes = [p, p, p, ctypes.c_longlong, i, i, p, i, p]
    lib.dsa3d_dwconv3d_backward.restype = i
    lib.dsa3d_dwconv3d_backward.argtypes = [p, p, p, i, i, i, i, win, p, p, p, p, sz, i, p]
    lib.dsa3d_dwconv3d_backward_workspace_bytes.restype = sz
    lib.dsa3d_dwconv3d_backward_workspace_bytes.argtypes = [i, win]
    lib.dsa3d_offsets_linear_backward.restype = i
    lib.dsa3d_offsets_linear_backward.argtypes = [p, p, p, ctypes.c_longlong, i, i, p, p, p, p, sz, i, p]
    lib.dsa3d_offsets_linear_backward_workspace_bytes.restype = sz
    lib.dsa3d_offsets_linear_backward_workspace_bytes.argtypes = [ctypes.c_longlong, i, i, i]
    lib.dsa3d_device_timeout_flag.restype = i
    lib.dsa3d_device_timeout_flag.argtypes = []
    lib.dsa3d_check_device_timeout.restype = i
    lib.dsa3d_check_device_timeout.argtypes = []
    lib.dsa3d_clear_device_timeout.restype = i
    lib.dsa3d_clear_device_timeout.argtypes = []
    lib.dsa3d_test_wait_timeout.restype = i
    lib.dsa3d_test_wait_timeout.argtypes = [ctypes.c_uint, p]
    lib.dsa3d_forward_residual.restype = i
    lib.dsa3d_forward_residual.argtypes = [p, p, p, p, p, i, i, i, i, i, win, p, p, i, p]
    lib.dsa3d_forward_bounded_offsets.restype = i
    lib.dsa3d_forward_bounded_offsets.argtypes = [p, p, p, p, i, i, i, i, i, win, p, p, i, p]
    lib.dsa3d_forward_fixed_window.restype = i
    lib.dsa3d_forward_fixed_window.argtypes = [p, p, p, i, i, i, i, i, win, p, p, i, p]
    lib.dsa3d_backward_fixed_window.restype = i
    lib.dsa3d_backward_fixed_window.argtypes = [p, p, p, p, p, i, i, i, i, i, win, p, p, p, p, p, sz, i, p]
    lib.dsa3d_backward_fixed_window_workspace_bytes.restype = sz
    lib.dsa3d_backward_fixed_window_workspace_bytes.argtypes = [i, i, i, i, i, win, i]
    lib.dsa3d_forward_host.restype = i
    lib.dsa3d_forward_host.argtypes = [p, p, p, p, i, i, i, i, i, win, p, p, p, sz, i, p]
    lib.dsa3d_forward_host_arena_bytes.restype = sz
    lib.dsa3d_forward_host_arena_bytes.argtypes = [i, i, i, i, i, win, i]
    lib.dsa3d_status_string.restype = ctypes.c_char_p
    lib.dsa3d_status_string.argtypes = [i]
    lib.dsa3d_last_cuda_error.restype = i
    lib.dsa3d_last_cuda_error.argtypes = []
    lib.dsa3d_debug_build.restype = i
    lib.dsa3d_debug_build.argtypes = []
    lib.dsa3d_debug_first_violation.restype = i
    lib.dsa3d_debug_first_violation.argtypes = [ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_longlong)]
    lib.dsa3d_debug_clear.restype = i
    lib.dsa3d_debug_clear.argtypes = []


def _window(window: Sequence[int]):
    if len(window) != 3:
        raise ValueError("window must be (kt, kh, kw)")
    return (ctypes.c_int * 3)(int(window[0]), int(window[1]), int(window[2]))


def _ptr(t: Optional[torch.Tensor], name: str, numel: Optional[int] = None, dtype=None) -> Optional[int]:
    if t is None:
        return None
    if not isinstance(t, torch.Tensor):
        return int(t)                        # a raw device address
    if t.device.type != "cuda":
        raise ValueError(f"{name} must be a CUDA tensor (the library takes device pointers)")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    if numel is not None and t.numel() != numel:
        raise ValueError(f"{name} has {t.numel()} elements, expected {numel}")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream or None
    return int(stream) or None


def _check(status: int) -> None:
    if status != 0:
        lib = load()
        msg = lib.dsa3d_status_string(status).decode()
        if status == 6:
            msg += f" (cudaError {lib.dsa3d_last_cuda_error()})"
        raise Dsa3dError(status, msg)


def dsa3d_status_string(status: int) -> str:
    return load().dsa3d_status_string(int(status)).decode()


def dsa3d_last_cuda_error() -> int:
    return int(load().dsa3d_last_cuda_error())


def dsa3d_backward_workspace_bytes(T, H, W, heads, d, window, dtype) -> int:
    code = _DTYPES[dtype] if isinstance(dtype, torch.dtype) else int(dtype)
    return int(load().dsa3d_backward_workspace_bytes(T, H, W, heads, d, _window(window), code))


def dsa3d_forward(q, k, v, offsets, T, H, W, heads, d, window, out, lse, dtype=None, stream=None) -> None:
    """out, lse <- 3D-DSA forward of (q, k, v, offsets); see include/dsa3d.h.  `dtype`
    defaults to q's dtype; `stream` to torch's current stream."""
    lib = load()
    dt = q.dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    n = T * H * W * heads
    P = int(window[0]) * int(window[1]) * int(window[2])
    _check(lib.dsa3d_forward(
        _ptr(q, "q", n * d), _ptr(k, "k", n * d), _ptr(v, "v", n * d),
        _ptr(offsets, "offsets", n * P * 3, torch.float32), T, H, W, heads, d, _window(window),
        _ptr(out, "out", n * d), _ptr(lse, "lse", n, torch.float32), code, _stream(stream)))


def dsa3d_forward_bounded_offsets(q, k, v, offsets, T, H, W, heads, d, window, out, lse, dtype=None, stream=None) -> None:
    """dsa3d_forward for offsets that are small perturbations of the window: tensor-core tile kernel when
    every |offset| < 1 (decided on the device), the general kernel otherwise; see include/dsa3d.h."""
    lib = load()
    dt = q.dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    n = T * H * W * heads
    P = int(window[0]) * int(window[1]) * int(window[2])
    _check(lib.dsa3d_forward_bounded_offsets(
        _ptr(q, "q", n * d), _ptr(k, "k", n * d), _ptr(v, "v", n * d),
        _ptr(offsets, "offsets", n * P * 3, torch.float32), T, H, W, heads, d, _window(window),
        _ptr(out, "out", n * d), _ptr(lse, "lse", n, torch.float32), code, _stream(stream)))


def dsa3d_forward_residual(q, k, v, offsets, residual, T, H, W, heads, d, window, out, lse, dtype=None,
                           stream=None) -> None:
    """out, lse <- residual + 3D-DSA forward (Eq. 1 with its first term); see include/dsa3d.h."""
    lib = load()
    dt = q.dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    n = T * H * W * heads
    P = int(window[0]) * int(window[1]) * int(window[2])
    _check(lib.dsa3d_forward_residual(
        _ptr(q, "q", n * d), _ptr(k, "k", n * d), _ptr(v, "v", n * d),
        _ptr(offsets, "offsets", n * P * 3, torch.float32), _ptr(residual, "residual", n * d), T, H, W, heads, d,
        _window(window), _ptr(out, "out", n * d), _ptr(lse, "lse", n, torch.float32), code, _stream(stream)))


def dsa3d_forward_fixed_window(q, k, v, T, H, W, heads, d, window, out, lse, dtype=None, stream=None) -> None:
    """out, lse <- 3D-DSA forward with all offsets zero (no offsets tensor); see include/dsa3d.h."""
    lib = load()
    dt = q.dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    n = T * H * W * heads
    _check(lib.dsa3d_forward_fixed_window(
        _ptr(q, "q", n * d), _ptr(k, "k", n * d), _ptr(v, "v", n * d), T, H, W, heads, d, _window(window),
        _ptr(out, "out", n * d), _ptr(lse, "lse", n, torch.float32), code, _stream(stream)))


def dsa3d_backward_fixed_window_workspace_bytes(T, H, W, heads, d, window, dtype) -> int:
    code = _DTYPES[dtype] if isinstance(dtype, torch.dtype) else int(dtype)
    return int(load().dsa3d_backward_fixed_window_workspace_bytes(T, H, W, heads, d, _window(window), code))


def dsa3d_backward_fixed_window(q, k, v, lse, dout, T, H, W, heads, d, window, dq, dk, dv, doffsets, workspace,
                                dtype=None, stream=None) -> None:
    """dq, dk, dv (and doffsets unless None) <- backward with all offsets zero; see include/dsa3d.h."""
    lib = load()
    dt = q.dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    n = T * H * W * heads
    P = int(window[0]) * int(window[1]) * int(window[2])
    _check(lib.dsa3d_backward_fixed_window(
        _ptr(q, "q", n * d), _ptr(k, "k", n * d), _ptr(v, "v", n * d), _ptr(lse, "lse", n, torch.float32),
        _ptr(dout, "dout", n * d), T, H, W, heads, d, _window(window), _ptr(dq, "dq", n * d), _ptr(dk, "dk", n * d),
        _ptr(dv, "dv", n * d), _ptr(doffsets, "doffsets", n * P * 3, torch.float32), _ptr(workspace, "workspace"),
        workspace.numel() * workspace.element_size(), code, _stream(stream)))


def dsa3d_dwconv3d_forward(x, weight, bias, T, H, W, C, kernel, y, dtype=None, stream=None) -> None:
    """y <- depthwise 3-D convolution of x (channels-last); see include/dsa3d.h."""
    lib = load()
    dt = x.dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    taps = int(kernel[0]) * int(kernel[1]) * int(kernel[2])
    _check(lib.dsa3d_dwconv3d_forward(
        _ptr(x, "x", T * H * W * C), _ptr(weight, "weight", taps * C, torch.float32),
        _ptr(bias, "bias", C, torch.float32), T, H, W, C, _window(kernel), _ptr(y, "y", T * H * W * C), code,
        _stream(stream)))


def dsa3d_offsets_linear_forward(u, w, bias, tokens, C, O, offsets, dtype=None, stream=None) -> None:
    """offsets <- u . w^T + bias (the linear layer of the offset predictor); see include/dsa3d.h."""
    lib = load()
    dt = u.dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    _check(lib.dsa3d_offsets_linear_forward(
        _ptr(u, "u", tokens * C), _ptr(w, "w", O * C), _ptr(bias, "bias", O, torch.float32), tokens, C, O,
        _ptr(offsets, "offsets", tokens * O, torch.float32), code, _stream(stream)))


def _nbytes(t: Optional[torch.Tensor]) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def dsa3d_dwconv3d_backward_workspace_bytes(C, kernel) -> int:
    return int(load().dsa3d_dwconv3d_backward_workspace_bytes(C, _window(kernel)))


def dsa3d_dwconv3d_backward(x, weight, dy, T, H, W, C, kernel, dx, dweight, dbias, workspace, dtype=None,
                            stream=None) -> None:
    """dx, dweight, dbias <- gradients of the depthwise convolution (each may be None); see
    include/dsa3d.h."""
    lib = load()
    dt = dy.dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    taps = int(kernel[0]) * int(kernel[1]) * int(kernel[2])
    n = T * H * W * C
    _check(lib.dsa3d_dwconv3d_backward(
        _ptr(x, "x", n), _ptr(weight, "weight", taps * C, torch.float32), _ptr(dy, "dy", n), T, H, W, C,
        _window(kernel), _ptr(dx, "dx", n), _ptr(dweight, "dweight", taps * C, torch.float32),
        _ptr(dbias, "dbias", C, torch.float32), _ptr(workspace, "workspace"), _nbytes(workspace), code,
        _stream(stream)))


def dsa3d_offsets_linear_backward_workspace_bytes(tokens, C, O, dtype) -> int:
    code = _DTYPES[dtype] if isinstance(dtype, torch.dtype) else int(dtype)
    return int(load().dsa3d_offsets_linear_backward_workspace_bytes(tokens, C, O, code))


def dsa3d_offsets_linear_backward(u, w, doffsets, tokens, C, O, du, dw, dbias, workspace, dtype=None,
                                  stream=None) -> None:
    """du, dw, dbias <- gradients of the offset-producing linear layer (each may be None);
    see include/dsa3d.h."""
    lib = load()
    dt = (u if u is not None else w).dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    _check(lib.dsa3d_offsets_linear_backward(
        _ptr(u, "u", tokens * C), _ptr(w, "w", O * C), _ptr(doffsets, "doffsets", tokens * O, torch.float32),
        tokens, C, O, _ptr(du, "du", tokens * C), _ptr(dw, "dw", O * C, torch.float32),
        _ptr(dbias, "dbias", O, torch.float32), _ptr(workspace, "workspace"), _nbytes(workspace), code,
        _stream(stream)))


def dsa3d_device_timeout_flag() -> int:
    return int(load().dsa3d_device_timeout_flag())


def dsa3d_check_device_timeout() -> None:
    """Raises Dsa3dError (status 7) if a kernel of the library gave up a bounded wait."""
    _check(load().dsa3d_check_device_timeout())


def dsa3d_clear_device_timeout() -> None:
    """Resets the (sticky) timeout flag."""
    _check(load().dsa3d_clear_device_timeout())


def dsa3d_test_wait_timeout(polls: int, stream=None) -> None:
    """Test aid: one thread waits `polls` polls on a barrier nobody arrives at, gives up and raises
    the timeout flag; see include/dsa3d.h."""
    _check(load().dsa3d_test_wait_timeout(int(polls), _stream(stream)))


def dsa3d_backward(q, k, v, offsets, lse, dout, T, H, W, heads, d, window, dq, dk, dv, doffsets,
                   workspace=None, workspace_bytes=None, dtype=None, stream=None) -> None:
    """dq, dk, dv, doffsets <- 3D-DSA backward; see include/dsa3d.h.  `workspace` is a CUDA
    tensor (any dtype) of at least dsa3d_backward_workspace_bytes(...) bytes."""
    lib = load()
    dt = q.dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    n = T * H * W * heads
    P = int(window[0]) * int(window[1]) * int(window[2])
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.dsa3d_backward(
        _ptr(q, "q", n * d), _ptr(k, "k", n * d), _ptr(v, "v", n * d),
        _ptr(offsets, "offsets", n * P * 3, torch.float32), _ptr(lse, "lse", n, torch.float32),
        _ptr(dout, "dout", n * d), T, H, W, heads, d, _window(window),
        _ptr(dq, "dq", n * d), _ptr(dk, "dk", n * d), _ptr(dv, "dv", n * d),
        _ptr(doffsets, "doffsets", n * P * 3, torch.float32),
        _ptr(workspace, "workspace"), int(workspace_bytes), code, _stream(stream)))


def dsa3d_backward_bounded_offsets_workspace_bytes(T, H, W, heads, d, window, dtype) -> int:
    code = _DTYPES[dtype] if isinstance(dtype, torch.dtype) else int(dtype)
    return int(load().dsa3d_backward_bounded_offsets_workspace_bytes(T, H, W, heads, d, _window(window), code))


def dsa3d_backward_bounded_offsets(q, k, v, offsets, lse, dout, T, H, W, heads, d, window, dq, dk, dv, doffsets,
                                   workspace=None, workspace_bytes=None, dtype=None, stream=None) -> None:
    """dsa3d_backward for offsets that are small perturbations of the window: tensor-core tile kernels when
    every |offset| < 1 (decided on the device), the general kernels otherwise; see include/dsa3d.h."""
    lib = load()
    dt = q.dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    n = T * H * W * heads
    P = int(window[0]) * int(window[1]) * int(window[2])
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.dsa3d_backward_bounded_offsets(
        _ptr(q, "q", n * d), _ptr(k, "k", n * d), _ptr(v, "v", n * d),
        _ptr(offsets, "offsets", n * P * 3, torch.float32), _ptr(lse, "lse", n, torch.float32),
        _ptr(dout, "dout", n * d), T, H, W, heads, d, _window(window),
        _ptr(dq, "dq", n * d), _ptr(dk, "dk", n * d), _ptr(dv, "dv", n * d),
        _ptr(doffsets, "doffsets", n * P * 3, torch.float32),
        _ptr(workspace, "workspace"), int(workspace_bytes), code, _stream(stream)))


def _host_ptr(t: torch.Tensor, name: str, numel: int, dtype) -> int:
    if t.device.type != "cpu" or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CPU tensor")
    if t.dtype != dtype or t.numel() != numel:
        raise ValueError(f"{name}: expected {numel} elements of {dtype}")
    return t.data_ptr()


def dsa3d_step_host_arena_bytes(T, H, W, heads, d, window, dtype) -> int:
    code = _DTYPES[dtype] if isinstance(dtype, torch.dtype) else int(dtype)
    return int(load().dsa3d_step_host_arena_bytes(T, H, W, heads, d, _window(window), code))


def _step_host(fn, q_h, k_h, v_h, offsets_h, dout_h, T, H, W, heads, d, window,
               out_h, lse_h, dq_h, dk_h, dv_h, doffsets_h, arena, stream) -> None:
    dt = q_h.dtype
    n = T * H * W * heads
    P = int(window[0]) * int(window[1]) * int(window[2])
    f32 = torch.float32
    _check(fn(
        _host_ptr(q_h, "q_h", n * d, dt), _host_ptr(k_h, "k_h", n * d, dt), _host_ptr(v_h, "v_h", n * d, dt),
        _host_ptr(offsets_h, "offsets_h", n * P * 3, f32), _host_ptr(dout_h, "dout_h", n * d, dt),
        T, H, W, heads, d, _window(window),
        _host_ptr(out_h, "out_h", n * d, dt), _host_ptr(lse_h, "lse_h", n, f32),
        _host_ptr(dq_h, "dq_h", n * d, dt), _host_ptr(dk_h, "dk_h", n * d, dt),
        _host_ptr(dv_h, "dv_h", n * d, dt), _host_ptr(doffsets_h, "doffsets_h", n * P * 3, f32),
        _ptr(arena, "arena"), arena.numel() * arena.element_size(), _DTYPES[dt], _stream(stream)))


def dsa3d_step_host(q_h, k_h, v_h, offsets_h, dout_h, T, H, W, heads, d, window,
                    out_h, lse_h, dq_h, dk_h, dv_h, doffsets_h, arena, stream=None) -> None:
    """Forward + backward from HOST tensors (pinned for speed) through a caller-owned
    device arena (a CUDA uint8 tensor); see include/dsa3d.h.  Asynchronous on `stream`."""
    _step_host(load().dsa3d_step_host, q_h, k_h, v_h, offsets_h, dout_h, T, H, W, heads, d, window,
               out_h, lse_h, dq_h, dk_h, dv_h, doffsets_h, arena, stream)


def dsa3d_step_host_pipelined(q_h, k_h, v_h, offsets_h, dout_h, T, H, W, heads, d, window,
                              out_h, lse_h, dq_h, dk_h, dv_h, doffsets_h, arena, stream=None) -> None:
    """The same step for a sequence of steps on one arena: transfers overlap the neighbouring
    calls' kernels; results are final after dsa3d_step_host_flush + stream completion."""
    _step_host(load().dsa3d_step_host_pipelined, q_h, k_h, v_h, offsets_h, dout_h, T, H, W, heads, d, window,
               out_h, lse_h, dq_h, dk_h, dv_h, doffsets_h, arena, stream)


def dsa3d_step_host_flush(stream=None) -> None:
    _check(load().dsa3d_step_host_flush(_stream(stream)))


def dsa3d_forward_host_arena_bytes(T, H, W, heads, d, window, dtype) -> int:
    code = _DTYPES[dtype] if isinstance(dtype, torch.dtype) else int(dtype)
    return int(load().dsa3d_forward_host_arena_bytes(T, H, W, heads, d, _window(window), code))


def dsa3d_forward_host(q_h, k_h, v_h, offsets_h, T, H, W, heads, d, window, out_h, lse_h, arena, stream=None) -> None:
    """Forward from HOST tensors (pinned for speed) through a caller-owned device arena; see
    include/dsa3d.h.  Asynchronous on `stream`."""
    lib = load()
    dt = q_h.dtype
    n = T * H * W * heads
    P = int(window[0]) * int(window[1]) * int(window[2])
    f32 = torch.float32
    _check(lib.dsa3d_forward_host(
        _host_ptr(q_h, "q_h", n * d, dt), _host_ptr(k_h, "k_h", n * d, dt), _host_ptr(v_h, "v_h", n * d, dt),
        _host_ptr(offsets_h, "offsets_h", n * P * 3, f32), T, H, W, heads, d, _window(window),
        _host_ptr(out_h, "out_h", n * d, dt), _host_ptr(lse_h, "lse_h", n, f32),
        _ptr(arena, "arena"), arena.numel() * arena.element_size(), _DTYPES[dt], _stream(stream)))


def dsa3d_set_profile_events(fwd_start=None, fwd_stop=None, bwd_start=None, bwd_stop=None,
                             scatter_start=None, scatter_stop=None) -> None:
    """Timing hook: torch.cuda.Event objects (created with enable_timing=True and already
    recorded once so that their handles exist) or None."""
    def handle(ev):
        return None if ev is None else ev.cuda_event
    _check(load().dsa3d_set_profile_events(handle(fwd_start), handle(fwd_stop), handle(bwd_start),
                                           handle(bwd_stop), handle(scatter_start), handle(scatter_stop)))


def dsa3d_backward_noalloc_max_elements() -> int:
    return int(load().dsa3d_backward_noalloc_max_elements())


def dsa3d_backward_noalloc(q, k, v, offsets, lse, dout, T, H, W, heads, d, window, dq, dk, dv, doffsets,
                           dtype=None, stream=None) -> None:
    """Backward for callers that cannot supply scratch memory: same results as
    dsa3d_backward, accumulators in a fixed array inside the library (problems up to
    dsa3d_backward_noalloc_max_elements() = T*H*W*heads*d elements).  Calls on one device
    must not overlap; see include/dsa3d.h."""
    lib = load()
    dt = q.dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    n = T * H * W * heads
    P = int(window[0]) * int(window[1]) * int(window[2])
    _check(lib.dsa3d_backward_noalloc(
        _ptr(q, "q", n * d), _ptr(k, "k", n * d), _ptr(v, "v", n * d),
        _ptr(offsets, "offsets", n * P * 3, torch.float32), _ptr(lse, "lse", n, torch.float32),
        _ptr(dout, "dout", n * d), T, H, W, heads, d, _window(window),
        _ptr(dq, "dq", n * d), _ptr(dk, "dk", n * d), _ptr(dv, "dv", n * d),
        _ptr(doffsets, "doffsets", n * P * 3, torch.float32), code, _stream(stream)))


def _timed(launch, reps: int = 3) -> float:
    """Best CUDA-event time (ms) of `launch()` over `reps` runs after one warm-up."""
    launch()
    torch.cuda.synchronize()
    best = float("inf")
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        launch()
        b.record()
        b.synchronize()
        best = min(best, a.elapsed_time(b))
    return best


def dsa3d_probe_gather(buffer: torch.Tensor, working_set_bytes: int, iters: int = 2048) -> float:
    """GB/s of random 256-byte-row reads spread over the first `working_set_bytes` of `buffer`."""
    lib, work = load(), ctypes.c_double()
    def launch():
        _check(lib.dsa3d_probe_gather(_ptr(buffer, "buffer"), working_set_bytes, iters, ctypes.byref(work), _stream(None)))
    ms = _timed(launch)
    return work.value / ms / 1e6


def dsa3d_probe_red(buffer: torch.Tensor, working_set_bytes: int, iters: int = 512) -> float:
    """GB/s of fp32 vector-reduction operands onto random 512-byte rows of `buffer`."""
    lib, work = load(), ctypes.c_double()
    def launch():
        _check(lib.dsa3d_probe_red(_ptr(buffer, "buffer"), working_set_bytes, iters, ctypes.byref(work), _stream(None)))
    ms = _timed(launch)
    return work.value / ms / 1e6


def dsa3d_probe_fma(seed: torch.Tensor, kind: int, iters: int = 4096) -> float:
    """TFMA/s of register-resident FMAs: kind 0 fp32, kind 1 bf16 x bf16 -> fp32."""
    lib, work = load(), ctypes.c_double()
    def launch():
        _check(lib.dsa3d_probe_fma(_ptr(seed, "seed"), iters, kind, ctypes.byref(work), _stream(None)))
    ms = _timed(launch)
    return work.value / ms / 1e9


def dsa3d_forward_batch(q, k, v, offsets, batch, T, H, W, heads, d, window, out, lse, dtype=None,
                        stream=None) -> None:
    """Forward of `batch` independent videos stored back to back; see include/dsa3d.h."""
    lib = load()
    dt = q.dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    n = batch * T * H * W * heads
    P = int(window[0]) * int(window[1]) * int(window[2])
    _check(lib.dsa3d_forward_batch(
        _ptr(q, "q", n * d), _ptr(k, "k", n * d), _ptr(v, "v", n * d),
        _ptr(offsets, "offsets", n * P * 3, torch.float32), batch, T, H, W, heads, d, _window(window),
        _ptr(out, "out", n * d), _ptr(lse, "lse", n, torch.float32), code, _stream(stream)))


def dsa3d_backward_batch(q, k, v, offsets, lse, dout, batch, T, H, W, heads, d, window, dq, dk, dv, doffsets,
                         workspace=None, dtype=None, stream=None) -> None:
    """Backward of `batch` independent videos stored back to back; see include/dsa3d.h."""
    lib = load()
    dt = q.dtype if dtype is None else dtype
    code = _DTYPES[dt] if isinstance(dt, torch.dtype) else int(dt)
    n = batch * T * H * W * heads
    P = int(window[0]) * int(window[1]) * int(window[2])
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.dsa3d_backward_batch(
        _ptr(q, "q", n * d), _ptr(k, "k", n * d), _ptr(v, "v", n * d),
        _ptr(offsets, "offsets", n * P * 3, torch.float32), _ptr(lse, "lse", n, torch.float32),
        _ptr(dout, "dout", n * d), batch, T, H, W, heads, d, _window(window),
        _ptr(dq, "dq", n * d), _ptr(dk, "dk", n * d), _ptr(dv, "dv", n * d),
        _ptr(doffsets, "doffsets", n * P * 3, torch.float32), _ptr(workspace, "workspace"), nbytes, code,
        _stream(stream)))
