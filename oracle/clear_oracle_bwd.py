"""ctypes binding of the fp64 CPU oracle of the backward pass (``clear_oracle_bwd.c``).

TEST INFRASTRUCTURE ONLY: only the tests use it; the CUDA library never does.  It imports nothing from
the CUDA package and shares no code with it (nor with the forward oracle: the readings of Eq. 3 are
restated in its C file).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "clear_oracle_bwd.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_SO = os.path.join(_OUT_DIR, "libclear_oracle_bwd.so")
_lock = threading.Lock()
_lib = None

BF16, F32, F64 = 0, 1, 2


def build(force: bool = False) -> str:
    os.makedirs(_OUT_DIR, exist_ok=True)
    stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.run(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-o", tmp, _SRC, "-lm"],
                       check=True)
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            i32, f64, vp = ctypes.c_int, ctypes.c_double, ctypes.c_void_p
            lib.clear_oracle_attn_bwd.restype = i32
            lib.clear_oracle_attn_bwd.argtypes = [vp, vp, vp, i32, vp, i32, i32, i32, i32, i32, i32, f64, f64, vp, vp, vp]
            _lib = lib
    return _lib


def _as_input(x):
    try:
        import torch
        if isinstance(x, torch.Tensor):
            x = x.detach().cpu().contiguous()
            if x.dtype == torch.bfloat16:
                return x.view(torch.int16).numpy().view(np.uint16), BF16
            if x.dtype == torch.float32:
                return x.numpy(), F32
            if x.dtype == torch.float64:
                return x.numpy(), F64
            raise TypeError(f"unsupported tensor dtype {x.dtype}")
    except ImportError:
        pass
    a = np.ascontiguousarray(x)
    if a.dtype == np.uint16:
        return a, BF16
    if a.dtype == np.float32:
        return a, F32
    if a.dtype == np.float64:
        return a, F64
    raise TypeError(f"unsupported array dtype {a.dtype}")


def attn_bwd(q, k, v, d_out, grid_h: int, grid_w: int, n_text: int, radius: float, scale: float):
    """(dq, dk, dv), each [B, H, N, d] float64, for the upstream gradient ``d_out`` of the attention output."""
    qa, dt = _as_input(q)
    ka, dtk = _as_input(k)
    va, dtv = _as_input(v)
    if not (dt == dtk == dtv) or qa.shape != ka.shape or qa.shape != va.shape or qa.ndim != 4:
        raise ValueError("q, k, v must share dtype and a [B, H, N, d] shape")
    B, H, N, d = qa.shape
    if N != n_text + grid_h * grid_w:
        raise ValueError("token axis does not match n_text + grid_h*grid_w")
    try:
        import torch
        if isinstance(d_out, torch.Tensor):
            d_out = d_out.detach().cpu().double().numpy()
    except ImportError:
        pass
    go = np.ascontiguousarray(np.asarray(d_out, dtype=np.float64))
    if go.shape != qa.shape:
        raise ValueError("d_out must have the shape of the output")
    dq, dk, dv = (np.empty(qa.shape, dtype=np.float64) for _ in range(3))
    rc = _load().clear_oracle_attn_bwd(qa.ctypes.data, ka.ctypes.data, va.ctypes.data, dt, go.ctypes.data, B, H,
                                       grid_h, grid_w, n_text, d, float(radius), float(scale),
                                       dq.ctypes.data, dk.ctypes.data, dv.ctypes.data)
    if rc != 0:
        raise ValueError(f"oracle rejected its arguments (status {rc})")
    return dq, dk, dv
