"""ctypes binding of the fp64 CPU oracle of the other window kinds (``clear_oracle_windows.c``).

TEST INFRASTRUCTURE ONLY: only the tests use it.  It imports nothing from the CUDA package and shares no code
with it or with the other oracle files.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "clear_oracle_windows.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_SO = os.path.join(_OUT_DIR, "libclear_oracle_windows.so")
_lock = threading.Lock()
_lib = None

DISC, SQUARE, WINDOWS, STRIDED = 0, 1, 2, 3


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
            i64, i32, f64, vp = ctypes.c_int64, ctypes.c_int, ctypes.c_double, ctypes.c_void_p
            lib.clear_oracle_window_row.restype = i64
            lib.clear_oracle_window_row.argtypes = [i32, f64, f64, i64, i32, i32, i32, vp]
            lib.clear_oracle_window_counts.restype = i64
            lib.clear_oracle_window_counts.argtypes = [i32, f64, f64, i32, i32, i32, vp]
            lib.clear_oracle_window_attn.restype = i32
            lib.clear_oracle_window_attn.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i32, f64, f64, f64, vp]
            _lib = lib
    return _lib


def mask_row(kind, a, b, i, grid_h, grid_w, n_text) -> np.ndarray:
    row = np.empty(n_text + grid_h * grid_w, dtype=np.uint8)
    if _load().clear_oracle_window_row(kind, float(a), float(b), i, grid_h, grid_w, n_text, row.ctypes.data) < 0:
        raise ValueError("oracle rejected its arguments")
    return row


def mask_counts(kind, a, b, grid_h, grid_w, n_text):
    counts = np.empty(n_text + grid_h * grid_w, dtype=np.int64)
    total = _load().clear_oracle_window_counts(kind, float(a), float(b), grid_h, grid_w, n_text, counts.ctypes.data)
    if total < 0:
        raise ValueError("oracle rejected its arguments")
    return int(total), counts


def _as_input(x):
    import torch
    if isinstance(x, torch.Tensor):
        x = x.detach().cpu().contiguous()
        if x.dtype == torch.bfloat16:
            return x.view(torch.int16).numpy().view(np.uint16), 0
        if x.dtype == torch.float32:
            return x.numpy(), 1
        if x.dtype == torch.float64:
            return x.numpy(), 2
        raise TypeError(f"unsupported tensor dtype {x.dtype}")
    a = np.ascontiguousarray(x)
    return a, {np.dtype(np.uint16): 0, np.dtype(np.float32): 1, np.dtype(np.float64): 2}[a.dtype]


def attn(q, k, v, grid_h, grid_w, n_text, kind, a, b, scale) -> np.ndarray:
    """[B, H, N, d] float64 output of Eq. 1 under the mask of the given kind."""
    qa, dt = _as_input(q)
    ka, dtk = _as_input(k)
    va, dtv = _as_input(v)
    if not (dt == dtk == dtv) or qa.shape != ka.shape or qa.shape != va.shape or qa.ndim != 4:
        raise ValueError("q, k, v must share dtype and a [B, H, N, d] shape")
    B, H, N, d = qa.shape
    if N != n_text + grid_h * grid_w:
        raise ValueError("token axis does not match n_text + grid_h*grid_w")
    out = np.empty(qa.shape, dtype=np.float64)
    rc = _load().clear_oracle_window_attn(qa.ctypes.data, ka.ctypes.data, va.ctypes.data, dt, B, H, grid_h, grid_w,
                                          n_text, d, kind, float(a), float(b), float(scale), out.ctypes.data)
    if rc != 0:
        raise ValueError(f"oracle rejected its arguments (status {rc})")
    return out
