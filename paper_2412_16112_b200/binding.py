"""ctypes binding of ``libclear_attn.so``: same names as the C ABI, argument marshalling only.

Every step of the attention path runs in the library's CUDA kernels; PyTorch appears here only
as the owner of device memory and streams (``data_ptr()``, ``current_stream()``).  There is no
fallback: if the library cannot be loaded, or a call fails, a ``ClearError`` is raised.
"""
from __future__ import annotations

import ctypes
import os
import threading
from typing import Optional

from . import build as _build

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_MISALIGNED, ERR_PLAN_MISMATCH = -1, -2, -3, -4
ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_NO_MEMORY, ERR_TOO_LARGE = -5, -6, -7, -8
BF16, F32 = 0, 1
KERNEL_AUTO, KERNEL_SIMT, KERNEL_TCGEN05, KERNEL_TCGEN05_WS = 0, 1, 2, 3
MASK_DISC, MASK_SQUARE, MASK_WINDOWS, MASK_STRIDED = 0, 1, 2, 3
PART_ALL, PART_BAND_IMAGE, PART_BAND_TEXT = 0, 1, 2
TEXT_MERGE_EXACT, TEXT_MERGE_AVERAGE = 0, 1
TILE_LINEAR, TILE_MASKED = 1, 2
STEP_USE0, STEP_USE1, STEP_SHARED, STEP_LINEAR, STEP_MASKED0, STEP_MASKED1 = 1, 2, 4, 8, 16, 32
STEP_CLIP0, STEP_CLIP1 = 64, 128

EXPORTS = [
    "clear_attn_fwd", "clear_attn_fwd_f32", "clear_plan_create", "clear_plan_create_host",
    "clear_plan_tables", "clear_attn_fwd_planned", "clear_attn_fwd_host", "clear_plan_info",
    "clear_plan_check", "clear_plan_destroy", "clear_cache_clear", "clear_status_string",
    "clear_last_cuda_error", "clear_attn_fwd_static", "clear_plan_pair_tables",
    "clear_last_device_status", "clear_plan_mask_table", "clear_cache_check", "clear_plan_trim", "clear_attn_bwd_f32", "clear_plan_create_ex",
    "clear_qk_norm_rope", "clear_log_scale_factor",
    "clear_band_geometry", "clear_plan_create_band", "clear_attn_text_partial", "clear_text_merge",
    "clear_plan_create_mask", "clear_attn_bwd_bf16", "clear_attn_bwd_bf16_tc",
]


class ClearError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        detail = f", device status {last_device_status()}" if status == ERR_DEVICE_TIMEOUT else ""
        super().__init__(f"{what}: {status_string(status)} (status {status}, cuda error {last_cuda_error()}{detail})")


class PlanInfo(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "H", "grid_h", "grid_w", "n_text", "head_dim", "dtype", "kernel", "radius_sq_ceil",
                 "tile_h", "tile_w", "n_work_items", "n_text_splits", "max_item_tiles")] + \
               [("sum_mask", ctypes.c_int64), ("executed_pairs", ctypes.c_int64),
                ("workspace_bytes", ctypes.c_int64), ("flops", ctypes.c_double)]


class KvTile(ctypes.Structure):
    _fields_ = [("x", ctypes.c_int32), ("y", ctypes.c_int32), ("flags", ctypes.c_int32),
                ("n_valid", ctypes.c_int32)]


class WorkItem(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("kind", "qx", "qy", "n_rows", "tile_begin", "tile_count", "partial_slot", "reserved")]


class PairStep(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("x0", "y0", "x1", "y1", "flags", "n_valid0", "n_valid1", "load_base")]


class PairItem(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("kind", "n_sides", "qx", "qy0", "qy1", "n_rows0", "n_rows1", "step_begin", "step_count",
                 "n_loads", "partial_slot0", "partial_slot1")]


_lock = threading.Lock()
_lib: Optional[ctypes.CDLL] = None


def library_path() -> str:
    return _build.LIB


def load() -> ctypes.CDLL:
    """Load the shared library (building it with nvcc first if it is missing or stale)."""
    global _lib
    with _lock:
        if _lib is not None:
            return _lib
        path = _build.LIB
        if not os.path.exists(path) or os.environ.get("CLEAR_REBUILD") == "1":
            path = _build.build()
        lib = ctypes.CDLL(path)
        vp, i32, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
        fwd_args = [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, f32, f32, vp]
        lib.clear_attn_fwd.argtypes = fwd_args
        lib.clear_attn_fwd_f32.argtypes = fwd_args
        lib.clear_attn_fwd_static.argtypes = fwd_args
        lib.clear_attn_bwd_f32.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, f32, f32, vp]
        lib.clear_attn_bwd_bf16.argtypes = lib.clear_attn_bwd_f32.argtypes
        lib.clear_attn_bwd_bf16_tc.argtypes = lib.clear_attn_bwd_f32.argtypes
        lib.clear_qk_norm_rope.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i32, i32, i32,
                                           f32, f32, f32, f32, vp]
        pi32 = ctypes.POINTER(ctypes.c_int32)
        lib.clear_band_geometry.argtypes = [i32, f32, i32, i32, i32, pi32, pi32, pi32, pi32]
        lib.clear_plan_create_band.argtypes = [ctypes.POINTER(vp), i32, i32, i32, i32, i32, i32, f32, i32, i32, i32, i32,
                                               i32, i32]
        lib.clear_attn_text_partial.argtypes = [vp, vp, vp, vp, vp, f32, vp]
        lib.clear_plan_create_mask.argtypes = [ctypes.POINTER(vp), i32, i32, i32, i32, i32, i32, i32, i32, f32, i32, i32]
        lib.clear_text_merge.argtypes = [vp, i32, i32, i32, i32, i32, i32, vp, ctypes.c_longlong, vp]
        lib.clear_log_scale_factor.argtypes = [ctypes.c_longlong, ctypes.c_longlong]
        lib.clear_log_scale_factor.restype = f32
        plan_args = [ctypes.POINTER(vp), i32, i32, i32, i32, i32, i32, f32, i32, i32]
        lib.clear_plan_create.argtypes = plan_args
        lib.clear_plan_create_host.argtypes = plan_args
        lib.clear_plan_create_ex.argtypes = plan_args + [i32, i32]
        lib.clear_plan_tables.argtypes = [vp, ctypes.POINTER(ctypes.POINTER(WorkItem)), ctypes.POINTER(ctypes.c_int32),
                                          ctypes.POINTER(ctypes.POINTER(KvTile)), ctypes.POINTER(ctypes.c_int32),
                                          ctypes.POINTER(ctypes.POINTER(ctypes.c_int32)),
                                          ctypes.POINTER(ctypes.c_int32)]
        lib.clear_plan_pair_tables.argtypes = [vp, ctypes.POINTER(ctypes.POINTER(PairItem)),
                                               ctypes.POINTER(ctypes.c_int32),
                                               ctypes.POINTER(ctypes.POINTER(PairStep)),
                                               ctypes.POINTER(ctypes.c_int32)]
        lib.clear_plan_mask_table.argtypes = [vp, ctypes.POINTER(ctypes.POINTER(ctypes.c_uint32)),
                                              ctypes.POINTER(ctypes.c_int32)]
        lib.clear_attn_fwd_planned.argtypes = [vp, vp, vp, vp, vp, f32, vp]
        lib.clear_attn_fwd_host.argtypes = [vp, vp, vp, vp, vp, f32, vp]
        lib.clear_plan_info.argtypes = [vp, ctypes.POINTER(PlanInfo)]
        lib.clear_plan_check.argtypes = [vp, vp]
        lib.clear_plan_destroy.argtypes = [vp]
        lib.clear_cache_clear.argtypes = []
        lib.clear_cache_check.argtypes = [vp]
        lib.clear_plan_trim.argtypes = [vp]
        lib.clear_status_string.argtypes = [i32]
        lib.clear_status_string.restype = ctypes.c_char_p
        lib.clear_last_cuda_error.argtypes = []
        lib.clear_last_device_status.argtypes = []
        for name in EXPORTS:
            if name not in ("clear_status_string", "clear_log_scale_factor"):
                getattr(lib, name).restype = i32
        _lib = lib
        return lib


def status_string(status: int) -> str:
    return load().clear_status_string(int(status)).decode()


def last_cuda_error() -> int:
    return int(load().clear_last_cuda_error())


def last_device_status() -> int:
    """Kernel-internal code of the wait that expired in the last DEVICE_TIMEOUT seen by this thread."""
    return int(load().clear_last_device_status())


def _check(status: int, what: str) -> None:
    if status != OK:
        raise ClearError(status, what)


def _stream_ptr(stream) -> int:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _tensor_args(q, k, v, out, dtype_code):
    import torch
    want = torch.bfloat16 if dtype_code == BF16 else torch.float32
    for name, t in (("q", q), ("k", k), ("v", v), ("out", out)):
        if not t.is_cuda:
            raise ValueError(f"{name} must be a CUDA tensor")
        if t.dtype != want:
            raise TypeError(f"{name} must be {want}")
        if not t.is_contiguous():
            raise ValueError(f"{name} must be contiguous [B, H, N, d]")
    if not (q.shape == k.shape == v.shape == out.shape) or q.dim() != 4:
        raise ValueError("q, k, v, out must share one [B, H, N, d] shape")
    return q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr()


def clear_attn_fwd(q, k, v, out, grid_h, grid_w, n_text, radius, scale, stream=None):
    """bf16 CLEAR attention forward into ``out``; tensors are [B, H, n_text + grid_h*grid_w, d]."""
    ptrs = _tensor_args(q, k, v, out, BF16)
    B, H, _, d = q.shape
    _check(load().clear_attn_fwd(*ptrs, B, H, grid_h, grid_w, n_text, d, float(radius), float(scale),
                                 _stream_ptr(stream)), "clear_attn_fwd")
    return out


def _backward(fn_name, dtype, q, k, v, d_out, dq, dk, dv, grid_h, grid_w, n_text, radius, scale, stream):
    for t in (q, k, v, d_out, dq, dk, dv):
        if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype and t.shape == q.shape):
            raise ValueError(f"backward tensors must be contiguous {dtype} CUDA tensors of one [B, H, N, d] shape")
    B, H, _, d = q.shape
    _check(getattr(load(), fn_name)(q.data_ptr(), k.data_ptr(), v.data_ptr(), d_out.data_ptr(), dq.data_ptr(),
                                    dk.data_ptr(), dv.data_ptr(), B, H, grid_h, grid_w, n_text, d, float(radius),
                                    float(scale), _stream_ptr(stream)), fn_name)
    return dq, dk, dv


def clear_attn_bwd_f32(q, k, v, d_out, dq, dk, dv, grid_h, grid_w, n_text, radius, scale, stream=None):
    """fp32 backward pass: gradients of q, k, v into ``dq``, ``dk``, ``dv`` for the upstream gradient ``d_out``."""
    import torch
    return _backward("clear_attn_bwd_f32", torch.float32, q, k, v, d_out, dq, dk, dv, grid_h, grid_w, n_text, radius,
                     scale, stream)


def clear_attn_bwd_bf16(q, k, v, d_out, dq, dk, dv, grid_h, grid_w, n_text, radius, scale, stream=None):
    """The same for bf16 tensors (fp32 arithmetic, gradients rounded to bf16)."""
    import torch
    return _backward("clear_attn_bwd_bf16", torch.bfloat16, q, k, v, d_out, dq, dk, dv, grid_h, grid_w, n_text, radius,
                     scale, stream)


def clear_attn_bwd_bf16_tc(q, k, v, d_out, dq, dk, dv, grid_h, grid_w, n_text, radius, scale, stream=None):
    """bf16 backward pass on the tensor cores (head size 64 or 128)."""
    import torch
    return _backward("clear_attn_bwd_bf16_tc", torch.bfloat16, q, k, v, d_out, dq, dk, dv, grid_h, grid_w, n_text,
                     radius, scale, stream)


def clear_qk_norm_rope(q, k, q_out, k_out, grid_h, grid_w, n_text, axes_dim, gain_q=None, gain_k=None, theta=10000.0,
                       ntk_factor=1.0, eps=1e-6, q_factor=1.0, stream=None):
    """RMS normalisation, two-axis rotary embedding and the factor on Q, from ``q``, ``k`` into ``q_out``, ``k_out``
    (bf16 or fp32 CUDA tensors of one [B, H, N, d] shape; an output may be its own input)."""
    import torch
    for t in (q, k, q_out, k_out):
        if not (t.is_cuda and t.is_contiguous() and t.dtype == q.dtype and t.shape == q.shape):
            raise ValueError("q, k and the outputs must be contiguous CUDA tensors of one dtype and [B, H, N, d] shape")
    if q.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("bf16 or fp32 tensors")
    for g in (gain_q, gain_k):
        if g is not None and not (g.is_cuda and g.is_contiguous() and g.dtype == torch.float32 and g.numel() == q.shape[-1]):
            raise ValueError("a gain is a contiguous fp32 CUDA tensor of head_dim values")
    B, H, _, d = q.shape
    a0, a1, a2 = (int(a) for a in axes_dim)
    _check(load().clear_qk_norm_rope(q.data_ptr(), k.data_ptr(), q_out.data_ptr(), k_out.data_ptr(),
                                     gain_q.data_ptr() if gain_q is not None else None,
                                     gain_k.data_ptr() if gain_k is not None else None,
                                     B, H, grid_h, grid_w, n_text, d, BF16 if q.dtype == torch.bfloat16 else F32,
                                     a0, a1, a2, float(theta), float(ntk_factor), float(eps), float(q_factor),
                                     _stream_ptr(stream)), "clear_qk_norm_rope")
    return q_out, k_out


def clear_log_scale_factor(n_tokens: int, n_train_tokens: int) -> float:
    return float(load().clear_log_scale_factor(int(n_tokens), int(n_train_tokens)))


def clear_attn_fwd_f32(q, k, v, out, grid_h, grid_w, n_text, radius, scale, stream=None):
    """fp32 CLEAR attention forward into ``out``."""
    ptrs = _tensor_args(q, k, v, out, F32)
    B, H, _, d = q.shape
    _check(load().clear_attn_fwd_f32(*ptrs, B, H, grid_h, grid_w, n_text, d, float(radius), float(scale),
                                     _stream_ptr(stream)), "clear_attn_fwd_f32")
    return out


def clear_attn_fwd_static(q, k, v, out, grid_h, grid_w, n_text, radius, scale, stream=None):
    """bf16 forward pass that allocates no device memory: its tables and split-KV scratch live in a
    fixed-size array inside the library.  Meant for callers that cannot call cudaMalloc where attention
    runs (fixed memory budgets, plug-ins, processes whose caching allocator already owns the device).
    Shapes beyond the fixed capacities raise ``ClearError`` with status ``ERR_TOO_LARGE``; calls on one
    device share the array, so do not let two of them overlap on the GPU."""
    ptrs = _tensor_args(q, k, v, out, BF16)
    B, H, _, d = q.shape
    _check(load().clear_attn_fwd_static(*ptrs, B, H, grid_h, grid_w, n_text, d, float(radius), float(scale),
                                        _stream_ptr(stream)), "clear_attn_fwd_static")
    return out


class Plan:
    """Owner of a ``clear_plan_t``."""

    def __init__(self, B, H, grid_h, grid_w, n_text, head_dim, radius, dtype=BF16, kernel=KERNEL_AUTO,
                 host_only=False, mask_kind=MASK_DISC, mask_param=0):
        """``radius``: r of the disc / square window, the window size of ``MASK_WINDOWS``, the stride of
        ``MASK_STRIDED``; ``mask_param``: the shift of the window grid / the layer index of the strided mask."""
        self._h = ctypes.c_void_p()
        if mask_kind in (MASK_WINDOWS, MASK_STRIDED) or mask_param != 0:
            if kernel not in (KERNEL_AUTO, KERNEL_SIMT):
                raise ClearError(ERR_UNSUPPORTED, "clear_plan_create_mask")
            _check(load().clear_plan_create_mask(ctypes.byref(self._h), B, H, grid_h, grid_w, n_text, head_dim, dtype,
                                                 mask_kind, float(radius), mask_param, 1 if host_only else 0),
                   "clear_plan_create_mask")
        elif mask_kind != MASK_DISC:
            _check(load().clear_plan_create_ex(ctypes.byref(self._h), B, H, grid_h, grid_w, n_text, head_dim,
                                               float(radius), dtype, kernel, mask_kind, 1 if host_only else 0),
                   "clear_plan_create_ex")
        else:
            fn = load().clear_plan_create_host if host_only else load().clear_plan_create
            _check(fn(ctypes.byref(self._h), B, H, grid_h, grid_w, n_text, head_dim, float(radius), dtype, kernel),
                   "clear_plan_create_host" if host_only else "clear_plan_create")
        self.dtype = dtype

    @property
    def handle(self):
        return self._h

    def info(self) -> PlanInfo:
        out = PlanInfo()
        _check(load().clear_plan_info(self._h, ctypes.byref(out)), "clear_plan_info")
        return out

    def tables(self):
        """(items, tiles, half_width) as lists of ctypes structs / ints (copies)."""
        items, tiles, hw = ctypes.POINTER(WorkItem)(), ctypes.POINTER(KvTile)(), ctypes.POINTER(ctypes.c_int32)()
        ni, nt, nh = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
        _check(load().clear_plan_tables(self._h, ctypes.byref(items), ctypes.byref(ni), ctypes.byref(tiles),
                                        ctypes.byref(nt), ctypes.byref(hw), ctypes.byref(nh)), "clear_plan_tables")
        return ([items[i] for i in range(ni.value)], [tiles[i] for i in range(nt.value)],
                [hw[i] for i in range(nh.value)])

    def pair_tables(self):
        """(pair items, steps) of a TCGEN05_WS plan as lists of ctypes structs (copies)."""
        items, steps = ctypes.POINTER(PairItem)(), ctypes.POINTER(PairStep)()
        ni, ns = ctypes.c_int32(), ctypes.c_int32()
        _check(load().clear_plan_pair_tables(self._h, ctypes.byref(items), ctypes.byref(ni), ctypes.byref(steps),
                                             ctypes.byref(ns)), "clear_plan_pair_tables")
        return [items[i] for i in range(ni.value)], [steps[i] for i in range(ns.value)]

    def mask_table(self):
        """Mask table of a TCGEN05_WS plan as a numpy array [n_entries, 128, 4] of uint32 (a copy)."""
        import numpy as np
        words, n = ctypes.POINTER(ctypes.c_uint32)(), ctypes.c_int32()
        _check(load().clear_plan_mask_table(self._h, ctypes.byref(words), ctypes.byref(n)), "clear_plan_mask_table")
        if n.value == 0:
            return np.zeros((0, 128, 4), dtype=np.uint32)
        return np.ctypeslib.as_array(words, shape=(n.value, 128, 4)).copy()

    def forward(self, q, k, v, out, scale, stream=None):
        ptrs = _tensor_args(q, k, v, out, self.dtype)
        _check(load().clear_attn_fwd_planned(self._h, *ptrs, float(scale), _stream_ptr(stream)),
               "clear_attn_fwd_planned")
        return out

    def forward_host(self, q, k, v, out, scale, stream=None):
        """Host (CPU, ideally pinned) tensors in, host tensor out; returns after the stream is idle."""
        for t in (q, k, v, out):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("forward_host takes contiguous CPU tensors")
        _check(load().clear_attn_fwd_host(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                          float(scale), _stream_ptr(stream)), "clear_attn_fwd_host")
        return out

    def check(self, stream=None) -> None:
        _check(load().clear_plan_check(self._h, _stream_ptr(stream)), "clear_plan_check")

    def trim(self) -> None:
        _check(load().clear_plan_trim(self._h), "clear_plan_trim")

    def destroy(self) -> None:
        if self._h:
            load().clear_plan_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class BandPlan(Plan):
    """Plan of one part (``PART_BAND_IMAGE`` or ``PART_BAND_TEXT``) of a row band over its local grid."""

    def __init__(self, B, H, local_rows, grid_w, n_text, head_dim, radius, part, q_row_begin, q_row_end,
                 text_keys=True, mask_kind=MASK_DISC, host_only=False):
        self._h = ctypes.c_void_p()
        _check(load().clear_plan_create_band(ctypes.byref(self._h), B, H, local_rows, grid_w, n_text, head_dim,
                                             float(radius), mask_kind, part, q_row_begin, q_row_end,
                                             1 if text_keys else 0, 1 if host_only else 0), "clear_plan_create_band")
        self.dtype = BF16
        self.part = part

    def text_partial(self, q, k, v, records, scale, stream=None):
        """Records [B * H, n_text, d + 2] (fp32) of the text queries over this band's keys."""
        import torch
        ptrs = _tensor_args(q, k, v, q, BF16)
        if not (records.is_cuda and records.is_contiguous() and records.dtype == torch.float32):
            raise ValueError("records must be a contiguous fp32 CUDA tensor")
        _check(load().clear_attn_text_partial(self._h, ptrs[0], ptrs[1], ptrs[2], records.data_ptr(), float(scale),
                                              _stream_ptr(stream)), "clear_attn_text_partial")
        return records


def band_geometry(grid_h, radius, n_bands, band, mask_kind=MASK_DISC):
    """(y0, y1, halo_lo, halo_hi) of one band."""
    vals = [ctypes.c_int32() for _ in range(4)]
    _check(load().clear_band_geometry(grid_h, float(radius), mask_kind, n_bands, band, *[ctypes.byref(x) for x in vals]),
           "clear_band_geometry")
    return tuple(x.value for x in vals)


def clear_text_merge(records, out, n_text, mode=TEXT_MERGE_EXACT, stream=None):
    """Merge the bands' records [n_parts, B * H, n_text, d + 2] into the first n_text rows of ``out`` [B, H, N, d]."""
    import torch
    if not (records.is_cuda and records.is_contiguous() and records.dtype == torch.float32 and records.dim() == 4):
        raise ValueError("records must be a contiguous fp32 CUDA tensor [n_parts, B * H, n_text, d + 2]")
    if not (out.is_cuda and out.is_contiguous() and out.dtype == torch.bfloat16 and out.dim() == 4):
        raise ValueError("out must be a contiguous bf16 CUDA tensor [B, H, N, d]")
    B, H, N, d = out.shape
    if records.shape[1:] != (B * H, n_text, d + 2):
        raise ValueError("records do not match out")
    _check(load().clear_text_merge(records.data_ptr(), records.shape[0], B, H, n_text, d, mode, out.data_ptr(), N,
                                   _stream_ptr(stream)), "clear_text_merge")
    return out


def clear_cache_clear() -> None:
    _check(load().clear_cache_clear(), "clear_cache_clear")


def clear_cache_check(stream=None) -> None:
    _check(load().clear_cache_check(_stream_ptr(stream)), "clear_cache_check")
