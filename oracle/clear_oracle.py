"""ctypes binding of the fp64 CPU oracle (``clear_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the bench's
cpu-baseline leg use it; the CUDA library never does.  It imports nothing from
the CUDA package and shares no code with it.

The C file is compiled on first use with gcc (OpenMP) into
``oracle/_build/libclear_oracle.so``; ``build()`` can be called directly.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "clear_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_SO = os.path.join(_OUT_DIR, "libclear_oracle.so")
_lock = threading.Lock()
_lib = None

BF16, F32, F64 = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _SO + f".{os.getpid()}.tmp"
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            i64, i32, f64, vp = ctypes.c_int64, ctypes.c_int, ctypes.c_double, ctypes.c_void_p
            lib.clear_oracle_mask_row.restype = i64
            lib.clear_oracle_mask_row.argtypes = [i64, i32, i32, i32, f64, vp]
            lib.clear_oracle_mask_counts.restype = i64
            lib.clear_oracle_mask_counts.argtypes = [i32, i32, i32, f64, vp]
            lib.clear_oracle_attn_rows.restype = i32
            lib.clear_oracle_attn_rows.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32,
                                                   f64, f64, vp, i64, vp]
            lib.clear_oracle_attn.restype = i32
            lib.clear_oracle_attn.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32,
                                              f64, f64, vp]
            lib.clear_oracle_num_threads.restype = i32
            lib.clear_oracle_num_threads.argtypes = []
            _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().clear_oracle_num_threads())


def mask_row(i: int, grid_h: int, grid_w: int, n_text: int, radius: float) -> np.ndarray:
    """Row i of the Eq. 3 mask as a uint8 vector of length N."""
    N = n_text + grid_h * grid_w
    row = np.empty(N, dtype=np.uint8)
    _load().clear_oracle_mask_row(i, grid_h, grid_w, n_text, float(radius), row.ctypes.data)
    return row


def mask_counts(grid_h: int, grid_w: int, n_text: int, radius: float, want_counts: bool = True):
    """(sum(M), per-query counts) from visiting every (i, j) pair of Eq. 3."""
    N = n_text + grid_h * grid_w
    counts = np.empty(N, dtype=np.int64) if want_counts else None
    total = _load().clear_oracle_mask_counts(grid_h, grid_w, n_text, float(radius),
                                             counts.ctypes.data if want_counts else None)
    return int(total), counts


def _as_input(x):
    """Accept numpy (uint16 = bf16 bits, float32, float64) or torch CPU tensors."""
    try:
        import torch
        if isinstance(x, torch.Tensor):
            x = x.detach().cpu().contiguous()
            if x.dtype == torch.bfloat16:
                return x.view(torch.int16).numpy().view(np.uint16), BF16
            x = x.numpy()
    except ImportError:  # numpy-only use
        pass
    x = np.ascontiguousarray(x)
    if x.dtype == np.uint16:
        return x, BF16
    if x.dtype == np.float32:
        return x, F32
    if x.dtype == np.float64:
        return x, F64
    raise TypeError(f"unsupported oracle input dtype {x.dtype}")


def _prep(q, k, v):
    qa, dt = _as_input(q)
    ka, dk = _as_input(k)
    va, dv = _as_input(v)
    if not (dt == dk == dv):
        raise TypeError("q, k, v must share one dtype")
    if qa.ndim != 4 or qa.shape != ka.shape or qa.shape != va.shape:
        raise ValueError("q, k, v must be [B, H, N, d] and equal in shape")
    return qa, ka, va, dt


def attn(q, k, v, grid_h: int, grid_w: int, n_text: int, radius: float, scale: float) -> np.ndarray:
    """Full [B, H, N, d] float64 output."""
    qa, ka, va, dt = _prep(q, k, v)
    B, H, N, d = qa.shape
    if N != n_text + grid_h * grid_w:
        raise ValueError("token axis does not match n_text + grid_h*grid_w")
    out = np.empty((B, H, N, d), dtype=np.float64)
    rc = _load().clear_oracle_attn(qa.ctypes.data, ka.ctypes.data, va.ctypes.data, dt, B, H,
                                   grid_h, grid_w, n_text, d, float(radius), float(scale),
                                   out.ctypes.data)
    if rc != 0:
        raise ValueError(f"oracle rejected its arguments (status {rc})")
    return out


def attn_rows(q, k, v, grid_h: int, grid_w: int, n_text: int, radius: float, scale: float,
              rows) -> np.ndarray:
    """Output rows for the (b, h, i) triples in ``rows`` ([n_rows, 3] ints): [n_rows, d] float64."""
    qa, ka, va, dt = _prep(q, k, v)
    B, H, N, d = qa.shape
    if N != n_text + grid_h * grid_w:
        raise ValueError("token axis does not match n_text + grid_h*grid_w")
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64).reshape(-1, 3))
    out = np.empty((rows.shape[0], d), dtype=np.float64)
    rc = _load().clear_oracle_attn_rows(qa.ctypes.data, ka.ctypes.data, va.ctypes.data, dt, B, H,
                                        grid_h, grid_w, n_text, d, float(radius), float(scale),
                                        rows.ctypes.data, rows.shape[0], out.ctypes.data)
    if rc != 0:
        raise ValueError(f"oracle rejected its arguments (status {rc})")
    return out
