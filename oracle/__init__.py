"""CPU oracle for 3D Deformable Slide Attention: ctypes wrapper around dsa3d_oracle.c.

TEST INFRASTRUCTURE ONLY.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA library and its binding never do, and
this package imports nothing from them.

The arithmetic lives in ``dsa3d_oracle.c`` (fp64, plain loops, written from the paper's
Formulation section, Eq. 1 and the softmax definition under it).  This module only builds
that file with gcc and marshals CPU tensors into it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dsa3d_oracle.c")
_LIB = os.path.join(_HERE, "libdsa3d_oracle.so")
_lock = threading.Lock()
_lib = None

_DTYPE_CODE = {torch.float32: 0, torch.bfloat16: 1, torch.float64: 2}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no contraction) and return the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True, capture_output=True, text=True)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            vp, i64p, dp, ip = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
            lib.dsa3d_oracle_forward.restype = ctypes.c_int
            lib.dsa3d_oracle_forward.argtypes = [vp, vp, vp, vp, i64p, ctypes.c_int64] + \
                [ctypes.c_int] * 5 + [ip, ctypes.c_int, dp, dp, dp]
            lib.dsa3d_oracle_backward.restype = ctypes.c_int
            lib.dsa3d_oracle_backward.argtypes = [vp, vp, vp, vp, vp, i64p, ctypes.c_int64] + \
                [ctypes.c_int] * 5 + [ip, ctypes.c_int, i64p, dp, dp, dp, dp]
            lib.dsa3d_oracle_last_threads.restype = ctypes.c_int
            lib.dsa3d_oracle_max_threads.restype = ctypes.c_int
            _lib = lib
    return _lib


def last_threads() -> int:
    """Number of host threads the most recent oracle call could use."""
    return int(_load().dsa3d_oracle_last_threads())


def max_threads() -> int:
    return int(_load().dsa3d_oracle_max_threads())


def _prep(x: torch.Tensor, dtype: torch.dtype) -> torch.Tensor:
    if x.device.type != "cpu":
        raise ValueError("the oracle takes CPU tensors")
    if x.dtype != dtype:
        raise ValueError(f"expected {dtype}, got {x.dtype}")
    return x.contiguous()


def _common(q_rows, k, v, off_rows, qtok, T, H, W, heads, d, window):
    dtype = k.dtype
    if dtype not in _DTYPE_CODE:
        raise ValueError(f"unsupported dtype {dtype}")
    off_dtype = torch.float64 if dtype == torch.float64 else torch.float32
    P = int(window[0]) * int(window[1]) * int(window[2])
    N = T * H * W
    k = _prep(k, dtype)
    v = _prep(v, dtype)
    if k.numel() != N * heads * d or v.numel() != N * heads * d:
        raise ValueError("k/v must hold the full grid [T,H,W,heads,d]")
    q_rows = _prep(q_rows, dtype)
    nq = q_rows.numel() // (heads * d)
    off_rows = _prep(off_rows, off_dtype)
    if off_rows.numel() != nq * heads * P * 3:
        raise ValueError("offsets must be [nq,heads,P,3]")
    if qtok is not None:
        qtok = _prep(torch.as_tensor(qtok, dtype=torch.int64), torch.int64)
        if qtok.numel() != nq:
            raise ValueError("qtok must have one entry per query row")
        if nq and (int(qtok.min()) < 0 or int(qtok.max()) >= N):
            raise ValueError("qtok out of range")
    elif nq != N:
        raise ValueError("without qtok the query rows must be the full grid")
    win = (ctypes.c_int * 3)(int(window[0]), int(window[1]), int(window[2]))
    return dtype, P, N, nq, q_rows, k, v, off_rows, qtok, win


def forward(q_rows, k, v, off_rows, T, H, W, heads, d, window, qtok=None, return_alpha=False):
    """Forward of the operator for the given query rows.

    q_rows [nq,heads,d], k/v [T,H,W,heads,d] (one of fp32, bf16, fp64), off_rows
    [nq,heads,P,3] (fp32, or fp64 when the values are fp64), qtok [nq] token index of each
    row (None: the rows are the whole grid in order).  Returns (out [nq,heads,d] fp64,
    lse [nq,heads] fp64[, alpha [nq,heads,P] fp64]).
    """
    dtype, P, N, nq, q_rows, k, v, off_rows, qtok, win = _common(
        q_rows, k, v, off_rows, qtok, T, H, W, heads, d, window)
    out = torch.zeros(nq, heads, d, dtype=torch.float64)
    lse = torch.zeros(nq, heads, dtype=torch.float64)
    alpha = torch.zeros(nq, heads, P, dtype=torch.float64) if return_alpha else None
    rc = _load().dsa3d_oracle_forward(
        q_rows.data_ptr(), k.data_ptr(), v.data_ptr(), off_rows.data_ptr(),
        qtok.data_ptr() if qtok is not None else None, nq, T, H, W, heads, d, win,
        _DTYPE_CODE[dtype], out.data_ptr(), lse.data_ptr(),
        alpha.data_ptr() if alpha is not None else None)
    if rc != 0:
        raise RuntimeError(f"oracle forward failed with code {rc}")
    return (out, lse, alpha) if return_alpha else (out, lse)


def backward(q_rows, k, v, off_rows, dout_rows, T, H, W, heads, d, window, qtok=None, ktok=None):
    """Backward of the operator for the given query rows.

    Same inputs as ``forward`` plus dout_rows [nq,heads,d].  Returns (dq [nq,heads,d],
    dk, dv, doff [nq,heads,P,3]) in fp64.  dk/dv hold the contribution of THESE query rows
    only: [T*H*W,heads,d] when ktok is None, else [len(ktok),heads,d] for the listed key
    tokens.
    """
    dtype, P, N, nq, q_rows, k, v, off_rows, qtok, win = _common(
        q_rows, k, v, off_rows, qtok, T, H, W, heads, d, window)
    dout_rows = _prep(dout_rows, dtype)
    if dout_rows.numel() != nq * heads * d:
        raise ValueError("dout must be [nq,heads,d]")
    if ktok is None:
        nk, kslot = N, None
    else:
        ktok = torch.as_tensor(ktok, dtype=torch.int64).contiguous()
        nk = ktok.numel()
        kslot = torch.full((N,), -1, dtype=torch.int64)
        kslot[ktok] = torch.arange(nk, dtype=torch.int64)
    dq = torch.zeros(nq, heads, d, dtype=torch.float64)
    dk = torch.zeros(nk, heads, d, dtype=torch.float64)
    dv = torch.zeros(nk, heads, d, dtype=torch.float64)
    doff = torch.zeros(nq, heads, P, 3, dtype=torch.float64)
    rc = _load().dsa3d_oracle_backward(
        q_rows.data_ptr(), k.data_ptr(), v.data_ptr(), off_rows.data_ptr(), dout_rows.data_ptr(),
        qtok.data_ptr() if qtok is not None else None, nq, T, H, W, heads, d, win,
        _DTYPE_CODE[dtype], kslot.data_ptr() if kslot is not None else None,
        dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), doff.data_ptr())
    if rc != 0:
        raise RuntimeError(f"oracle backward failed with code {rc}")
    return dq, dk, dv, doff
