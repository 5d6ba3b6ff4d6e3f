"""ctypes binding: argument marshalling only.  Names match include/bigbird.h."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import numpy as np
import torch

BIGBIRD_ITC, BIGBIRD_ETC = 0, 1
BIGBIRD_FP32, BIGBIRD_BF16 = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
# BIGBIRD_LIB selects another build of the same library (the checked build libbigbird_debug.so, say)
_LIB_PATH = os.environ.get("BIGBIRD_LIB") or os.path.join(_HERE, "libbigbird.so")
_lib: Optional[C.CDLL] = None


class BigBirdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().bigbird_strerror(code).decode()
        extra = ""
        if code == -3:
            extra = f" (cudaError {lib().bigbird_last_cuda_error()})"
        super().__init__(f"{where}: {msg}{extra} [{code}]")


def library_path() -> str:
    return _LIB_PATH


def lib() -> C.CDLL:
    """Loads libbigbird.so (built by paper_2007_14062_b200/build.py).  Raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2007_14062_b200.build` "
            "(needs nvcc).  This package has no CPU or PyTorch fallback.")
    L = C.CDLL(_LIB_PATH)
    vp, i32, i64, u64, f32 = C.c_void_p, C.c_int, C.c_int64, C.c_uint64, C.c_float
    L.bigbird_build_layout.argtypes = [i64, i32, i32, i32, i32, u64, i32, i32, C.POINTER(vp)]
    L.bigbird_layout_nnz.argtypes = [vp, C.POINTER(i64)]
    L.bigbird_layout_export.argtypes = [vp, vp, vp]
    L.bigbird_layout_export_transposed.argtypes = [vp, vp, vp]
    L.bigbird_layout_schedule.argtypes = [vp, vp, vp, vp, vp]
    L.bigbird_layout_destroy.argtypes = [vp]
    fwd = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i64, i32, i32, f32, i32, vp]
    L.bigbird_attn_fwd.argtypes = fwd
    L.bigbird_attn_fwd_simt.argtypes = fwd
    L.bigbird_attn_fwd_static.argtypes = fwd
    L.bigbird_attn_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i64, i32, i32, f32, i32, vp]
    L.bigbird_last_status.argtypes = [vp, C.POINTER(i32), C.POINTER(i32)]
    L.bigbird_last_status_static.argtypes = [vp, C.POINTER(i32), C.POINTER(i32)]
    L.bigbird_last_cuda_error.argtypes = []
    L.bigbird_selftest_wait_expiry.argtypes = [vp]
    L.bigbird_last_launch_count.argtypes = []
    L.bigbird_strerror.argtypes = [i32]
    L.bigbird_strerror.restype = C.c_char_p
    for name in ("bigbird_build_layout", "bigbird_layout_nnz", "bigbird_layout_export", "bigbird_layout_export_transposed", "bigbird_layout_schedule", "bigbird_attn_bwd",
                 "bigbird_layout_destroy", "bigbird_attn_fwd", "bigbird_attn_fwd_simt", "bigbird_attn_fwd_static", "bigbird_last_status", "bigbird_last_status_static",
                 "bigbird_last_cuda_error", "bigbird_last_launch_count", "bigbird_selftest_wait_expiry"):
        getattr(L, name).restype = i32
    _lib = L
    return L


def _check(code: int, where: str) -> None:
    if code != 0:
        raise BigBirdError(code, where)


class Layout:
    """Owns a bigbird_layout handle."""

    def __init__(self, handle: int, N: int, b: int, w: int, g: int, r: int, seed: int, H: int, mode: int):
        self.handle = C.c_void_p(handle)
        self.N, self.b, self.w, self.g, self.r, self.seed, self.H, self.mode = N, b, w, g, r, seed, H, mode
        self.nb = N // b

    @property
    def nnz(self) -> int:
        n = C.c_int64(0)
        _check(lib().bigbird_layout_nnz(self.handle, C.byref(n)), "bigbird_layout_nnz")
        return n.value

    def export(self) -> Tuple[np.ndarray, np.ndarray]:
        """CSR (row_ptr int32[H*nb+1], col_idx int32[nnz]) over rows h*nb + j."""
        row_ptr = np.empty(self.H * self.nb + 1, dtype=np.int32)
        col_idx = np.empty(max(self.nnz, 1), dtype=np.int32)
        _check(lib().bigbird_layout_export(self.handle, row_ptr.ctypes.data, col_idx.ctypes.data),
               "bigbird_layout_export")
        return row_ptr, col_idx[: self.nnz]

    def export_transposed(self) -> Tuple[np.ndarray, np.ndarray]:
        """The graph by key block: (col_ptr int32[H*nb+1], row_idx int32[nnz]) over rows h*nb + c."""
        col_ptr = np.empty(self.H * self.nb + 1, dtype=np.int32)
        row_idx = np.empty(max(self.nnz, 1), dtype=np.int32)
        _check(lib().bigbird_layout_export_transposed(self.handle, col_ptr.ctypes.data, row_idx.ctypes.data),
               "bigbird_layout_export_transposed")
        return col_ptr, row_idx[: self.nnz]

    def schedule(self):
        """(sizes, items int32[H*ipH, 8], step_base int32[H], steps int32[S, 2]) of the tile schedule."""
        sizes = np.zeros(4, dtype=np.int32)
        _check(lib().bigbird_layout_schedule(self.handle, sizes.ctypes.data, None, None, None), "bigbird_layout_schedule")
        items = np.zeros((self.H * int(sizes[0]), 8), dtype=np.int32)
        base = np.zeros(self.H, dtype=np.int32)
        steps = np.zeros((max(int(sizes[2]), 1), 2), dtype=np.int32)
        _check(lib().bigbird_layout_schedule(self.handle, sizes.ctypes.data, items.ctypes.data, base.ctypes.data,
                                             steps.ctypes.data), "bigbird_layout_schedule")
        return sizes, items, base, steps[: int(sizes[2])]

    def close(self) -> None:
        if self.handle:
            lib().bigbird_layout_destroy(self.handle)
            self.handle = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def bigbird_build_layout(N: int, b: int, w: int, g: int, r: int, seed: int, H: int, mode: int = BIGBIRD_ITC) -> Layout:
    h = C.c_void_p(None)
    _check(lib().bigbird_build_layout(N, b, w, g, r, seed, H, mode, C.byref(h)), "bigbird_build_layout")
    return Layout(h.value, N, b, w, g, r, seed, H, mode)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _fwd(fn_name: str, q, k, v, layout: Layout, key_padding_mask, out, lse, scale: float, stream) -> None:
    if not (q.is_cuda and k.is_cuda and v.is_cuda and out.is_cuda):
        raise ValueError("q, k, v, out must be CUDA tensors (there is no CPU path)")
    for t in (q, k, v, out):
        if not t.is_contiguous() or t.shape != q.shape or t.dtype != q.dtype:
            raise ValueError("q, k, v, out must be contiguous [B, H, N, D] tensors of one dtype")
    B, H, N, D = q.shape
    dtype = {torch.float32: BIGBIRD_FP32, torch.bfloat16: BIGBIRD_BF16}.get(q.dtype)
    if dtype is None:
        raise ValueError("dtype must be float32 or bfloat16")
    if key_padding_mask is not None:
        if key_padding_mask.dtype != torch.uint8 or tuple(key_padding_mask.shape) != (B, N) or \
                not key_padding_mask.is_cuda or not key_padding_mask.is_contiguous():
            raise ValueError("key_padding_mask must be a contiguous CUDA uint8 [B, N] tensor")
    if lse is not None:
        if lse.dtype != torch.float32 or tuple(lse.shape) != (B, H, N) or not lse.is_cuda or not lse.is_contiguous():
            raise ValueError("lse must be a contiguous CUDA float32 [B, H, N] tensor")
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    with torch.cuda.device(q.device):
        code = getattr(lib(), fn_name)(_ptr(q), _ptr(k), _ptr(v), layout.handle, _ptr(key_padding_mask), _ptr(out),
                                       _ptr(lse), B, H, N, D, layout.b, float(scale), dtype, C.c_void_p(stream))
    _check(code, fn_name)


def bigbird_attn_fwd(q, k, v, layout: Layout, key_padding_mask, out, lse, scale: float, stream: Optional[int] = None) -> None:
    """Enqueues the forward pass on `stream` (default: torch's current stream).  B, H, N, D are read off q."""
    _fwd("bigbird_attn_fwd", q, k, v, layout, key_padding_mask, out, lse, scale, stream)


def bigbird_attn_fwd_simt(q, k, v, layout: Layout, key_padding_mask, out, lse, scale: float, stream: Optional[int] = None) -> None:
    _fwd("bigbird_attn_fwd_simt", q, k, v, layout, key_padding_mask, out, lse, scale, stream)


def bigbird_attn_fwd_static(q, k, v, layout: Layout, key_padding_mask, out, lse, scale: float, stream: Optional[int] = None) -> None:
    """bigbird_attn_fwd for callers that must not allocate device memory: the library's scratch is a fixed array
    inside the loaded module.  bf16, D == 64, b == 64 only; BigBirdError(-6) if the problem exceeds the array.
    Calls on one device must not overlap on the GPU; make the first call on a device outside stream capture."""
    _fwd("bigbird_attn_fwd_static", q, k, v, layout, key_padding_mask, out, lse, scale, stream)


def bigbird_attn_bwd(q, k, v, out, lse, dout, layout: Layout, key_padding_mask, dq, dk, dv, scale: float,
                     stream: Optional[int] = None) -> None:
    """Enqueues the gradient kernels: dq, dk, dv from dout and the forward pass's out and lse."""
    ts = (q, k, v, out, dout, dq, dk, dv)
    if not all(t.is_cuda for t in ts):
        raise ValueError("all tensors must be CUDA tensors (there is no CPU path)")
    for t in ts:
        if not t.is_contiguous() or t.shape != q.shape or t.dtype != q.dtype:
            raise ValueError("q, k, v, out, dout, dq, dk, dv must be contiguous [B, H, N, D] tensors of one dtype")
    B, H, N, D = q.shape
    dtype = {torch.float32: BIGBIRD_FP32, torch.bfloat16: BIGBIRD_BF16}.get(q.dtype)
    if dtype is None:
        raise ValueError("dtype must be float32 or bfloat16")
    if lse.dtype != torch.float32 or tuple(lse.shape) != (B, H, N) or not lse.is_cuda or not lse.is_contiguous():
        raise ValueError("lse must be a contiguous CUDA float32 [B, H, N] tensor")
    if key_padding_mask is not None:
        if key_padding_mask.dtype != torch.uint8 or tuple(key_padding_mask.shape) != (B, N) or \
                not key_padding_mask.is_cuda or not key_padding_mask.is_contiguous():
            raise ValueError("key_padding_mask must be a contiguous CUDA uint8 [B, N] tensor")
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    with torch.cuda.device(q.device):
        code = lib().bigbird_attn_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), _ptr(dout), layout.handle,
                                      _ptr(key_padding_mask), _ptr(dq), _ptr(dk), _ptr(dv), B, H, N, D, layout.b,
                                      float(scale), dtype, C.c_void_p(stream))
    _check(code, "bigbird_attn_bwd")


def bigbird_last_status(stream: Optional[int] = None) -> Tuple[int, int]:
    st, det = C.c_int(0), C.c_int(0)
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().bigbird_last_status(C.c_void_p(stream), C.byref(st), C.byref(det)), "bigbird_last_status")
    return st.value, det.value


def bigbird_last_status_static(stream: Optional[int] = None) -> Tuple[int, int]:
    """(status, detail) of the last bigbird_attn_fwd_static call on the current device; allocates nothing."""
    st, det = C.c_int(0), C.c_int(0)
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().bigbird_last_status_static(C.c_void_p(stream), C.byref(st), C.byref(det)), "bigbird_last_status_static")
    return st.value, det.value


def bigbird_selftest_wait_expiry(stream: Optional[int] = None) -> None:
    """Enqueues the bounded-wait self-test kernel (it gives up after about two seconds)."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().bigbird_selftest_wait_expiry(C.c_void_p(stream)), "bigbird_selftest_wait_expiry")


def bigbird_last_launch_count() -> int:
    return lib().bigbird_last_launch_count()


def bigbird_strerror(code: int) -> str:
    return lib().bigbird_strerror(code).decode()
