"""Thin ctypes binding of libmxfp8.so: argument marshalling only.

Every function has the name and argument order of its C entry point in ``include/mxfp8.h``
and takes torch tensors (device memory) where C takes device pointers.  Nothing here
computes: a missing library or a non-zero status raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

FP32, BF16 = 0, 1
ROW, COL, BOTH = 1, 2, 3
RULE_PAPER, RULE_OCP = 0, 1
E4M3, E5M2 = 0, 1
E2M3, E3M2, E2M1 = 3, 4, 5          # MXFP6 / MXFP4 elements: conversion kernels only
SF_LINEAR, SF_SWIZZLED = 0, 1
K_MAJOR, MN_MAJOR = 0, 1
ERR_NULL, ERR_ENUM, ERR_SHAPE, ERR_ALIGN, ERR_UNSUPPORTED, ERR_CUDA = -1, -2, -3, -4, -5, -6
ERR_DEVICE_TIMEOUT, ERR_WORKSPACE, ERR_DEVICE_ARGS = -7, -8, -9
ACT_NONE, ACT_RELU, ACT_RELU2, ACT_SILU, ACT_GELU_TANH = 0, 1, 2, 3, 4

EXPORTS = (
    "mxfp8_quantize", "mxfp8_dequantize", "mxfp8_gemm", "mxfp8_scale_bytes", "mxfp8_sf_offset",
    "mxfp8_gemm_workspace_bytes", "mxfp8_device_status", "mxfp8_status_string",
    "mxfp8_launch_count", "mxfp8_quantize_host_ws_bytes", "mxfp8_quantize_host",
    "mxfp8_linear_host_ws_bytes", "mxfp8_linear_host", "mxfp8_fake_quantize", "mxfp8_linear_ws_bytes",
    "mxfp8_linear", "mxfp8_grouped_gemm", "mxfp8_quantize_multi", "mxfp8_gemm_multi", "mxfp8_act_quantize", "mxfp8_rmsnorm_quantize",
    "mxfp8_rmsnorm_quantize_static", "mxfp8_rmsnorm_quantize_static_max_rows", "mxfp8_glu_quantize",
    "mxfp8_sf_concat_k", "mxfp8_gemm_reduce_scatter", "mxfp8_enable_peer_access", "mxfp8_gemm_last_clock", "mxfp8_layernorm_quantize", "mxfp8_act_grad_quantize",
)


class Mxfp8Error(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__("%s failed: %d (%s)" % (what, status, status_string(status)))
        self.status = status


class _QuantizeItem(ctypes.Structure):
    _fields_ = [("src", ctypes.c_void_p), ("rows", ctypes.c_int64), ("cols", ctypes.c_int64),
                ("q_row", ctypes.c_void_p), ("s_row", ctypes.c_void_p),
                ("q_col", ctypes.c_void_p), ("s_col", ctypes.c_void_p)]


class _GemmProblem(ctypes.Structure):
    _fields_ = [("Aq", ctypes.c_void_p), ("As", ctypes.c_void_p), ("Bq", ctypes.c_void_p), ("Bs", ctypes.c_void_p),
                ("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("a_major", ctypes.c_int), ("b_major", ctypes.c_int), ("a_elem", ctypes.c_int), ("b_elem", ctypes.c_int),
                ("D", ctypes.c_void_p)]


class _Epilogue(ctypes.Structure):
    _fields_ = [("orientation", ctypes.c_int), ("scale_rule", ctypes.c_int), ("elem", ctypes.c_int),
                ("q_row", ctypes.c_void_p), ("s_row", ctypes.c_void_p),
                ("q_col", ctypes.c_void_p), ("s_col", ctypes.c_void_p)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load (building first if the sources are newer) the CUDA library; fail loudly."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if os.environ.get("MXFP8_NO_BUILD") != "1":
            path = _build.build()
        if not os.path.exists(path):
            raise ImportError("libmxfp8.so is missing: run `python -m paper_2506_08027_b200.build`")
        _lib = load_library(path)
    return _lib


def load_library(path: str) -> ctypes.CDLL:
    """dlopen a build of the library and declare every entry point's signature."""
    L = ctypes.CDLL(path)
    i, i64, p, sz = ctypes.c_int, ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t
    L.mxfp8_quantize.restype = i
    L.mxfp8_quantize.argtypes = [p, i, i64, i64, i, i, i, p, p, p, p, i, p]
    L.mxfp8_dequantize.restype = i
    L.mxfp8_dequantize.argtypes = [p, p, i64, i64, i, i, i, p, i, p]
    L.mxfp8_gemm.restype = i
    L.mxfp8_gemm.argtypes = [p, p, p, p, i64, i64, i64, i, i, i, i, p, i, ctypes.POINTER(_Epilogue), p, sz, p]
    L.mxfp8_scale_bytes.restype = sz
    L.mxfp8_scale_bytes.argtypes = [i64, i64, i, i]
    L.mxfp8_sf_offset.restype = i64
    L.mxfp8_sf_offset.argtypes = [i64, i64, i64, i]
    L.mxfp8_gemm_workspace_bytes.restype = sz
    L.mxfp8_gemm_workspace_bytes.argtypes = [i64, i64, i64, i, i]
    L.mxfp8_device_status.restype = i
    L.mxfp8_device_status.argtypes = [p]
    L.mxfp8_status_string.restype = ctypes.c_char_p
    L.mxfp8_status_string.argtypes = [i]
    L.mxfp8_launch_count.restype = i64
    L.mxfp8_launch_count.argtypes = []
    L.mxfp8_quantize_host_ws_bytes.restype = sz
    L.mxfp8_quantize_host_ws_bytes.argtypes = [i, i64, i64, i]
    L.mxfp8_quantize_host.restype = i
    L.mxfp8_quantize_host.argtypes = [p, i, i64, i64, i, i, i, p, p, p, p, i, p, sz, p]
    L.mxfp8_fake_quantize.restype = i
    L.mxfp8_fake_quantize.argtypes = [p, i, i64, i64, i, i, i, p, p, p]
    L.mxfp8_rmsnorm_quantize.restype = i
    L.mxfp8_rmsnorm_quantize.argtypes = [p, i, i64, i64, p, ctypes.c_float, p, i, i, i, p, p, p, p, i, p]
    L.mxfp8_layernorm_quantize.restype = i
    L.mxfp8_layernorm_quantize.argtypes = [p, i, i64, i64, p, p, ctypes.c_float, p, p, i, i, i, p, p, p, p, i, p]
    L.mxfp8_rmsnorm_quantize_static.restype = i
    L.mxfp8_rmsnorm_quantize_static.argtypes = [p, i, i64, i64, p, ctypes.c_float, i, i, i, p, p, p, p, i, p]
    L.mxfp8_rmsnorm_quantize_static_max_rows.restype = i64
    L.mxfp8_rmsnorm_quantize_static_max_rows.argtypes = []
    L.mxfp8_glu_quantize.restype = i
    L.mxfp8_glu_quantize.argtypes = [p, i, i64, i64, i, i, i, i, p, p, p, p, i, p]
    L.mxfp8_act_grad_quantize.restype = i
    L.mxfp8_act_grad_quantize.argtypes = [p, p, i, i64, i64, i, i, i, i, p, p, p, p, i, p]
    L.mxfp8_act_quantize.restype = i
    L.mxfp8_act_quantize.argtypes = [p, i, i64, i64, i, i, i, i, p, p, p, p, i, p]
    L.mxfp8_gemm_multi.restype = i
    L.mxfp8_gemm_multi.argtypes = [ctypes.POINTER(_GemmProblem), i, i, p]
    L.mxfp8_quantize_multi.restype = i
    L.mxfp8_quantize_multi.argtypes = [ctypes.POINTER(_QuantizeItem), i, i, i, i, i, i, p]
    L.mxfp8_grouped_gemm.restype = i
    L.mxfp8_grouped_gemm.argtypes = [p, p, p, p, p, i, i, i64, i64, i64, i, i, i, p, i, p]
    L.mxfp8_gemm_last_clock.restype = i
    L.mxfp8_gemm_last_clock.argtypes = [p, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    L.mxfp8_enable_peer_access.restype = i
    L.mxfp8_enable_peer_access.argtypes = [i]
    L.mxfp8_sf_concat_k.restype = i
    L.mxfp8_sf_concat_k.argtypes = [p, i, i64, i64, p, p]
    L.mxfp8_gemm_reduce_scatter.restype = i
    L.mxfp8_gemm_reduce_scatter.argtypes = [p, p, p, p, i64, i64, i64, i, i, i, i, ctypes.POINTER(ctypes.c_void_p), i, i, p]
    L.mxfp8_linear_ws_bytes.restype = sz
    L.mxfp8_linear_ws_bytes.argtypes = [i64, i64, i64]
    L.mxfp8_linear.restype = i
    L.mxfp8_linear.argtypes = [p, p, p, i64, i64, i64, i, p, p, p, p, sz, p]
    L.mxfp8_linear_host_ws_bytes.restype = sz
    L.mxfp8_linear_host_ws_bytes.argtypes = [i64, i64, i64]
    L.mxfp8_linear_host.restype = i
    L.mxfp8_linear_host.argtypes = [p, p, p, i64, i64, i64, i, p, p, p, p, sz, p]
    return L


def status_string(status: int) -> str:
    return lib().mxfp8_status_string(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != 0:
        raise Mxfp8Error(status, what)


def _ptr(t):
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("the C entry points take dense row-major buffers: pass a contiguous tensor")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return FP32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("source must be float32 or bfloat16")


def mxfp8_scale_bytes(rows: int, cols: int, orientation: int, sf_layout: int) -> int:
    return int(lib().mxfp8_scale_bytes(rows, cols, orientation, sf_layout))


def mxfp8_sf_offset(mn: int, kblock: int, n_kblocks: int, sf_layout: int) -> int:
    return int(lib().mxfp8_sf_offset(mn, kblock, n_kblocks, sf_layout))


def mxfp8_gemm_workspace_bytes(M: int, N: int, K: int, out_dtype: int, has_epilogue: bool) -> int:
    return int(lib().mxfp8_gemm_workspace_bytes(M, N, K, out_dtype, int(has_epilogue)))


def mxfp8_device_status(stream=None) -> int:
    return int(lib().mxfp8_device_status(_stream(stream)))


def mxfp8_launch_count() -> int:
    return int(lib().mxfp8_launch_count())


def alloc_quantize_outputs(rows: int, cols: int, orientation: int, sf_layout: int, device="cuda"):
    """Caller-side allocation helper: (q_row, s_row, q_col, s_col), None where unused."""
    out = []
    for o in (ROW, COL):
        if orientation & o:
            out.append(torch.empty((rows, cols), dtype=torch.uint8, device=device))
            out.append(torch.empty(mxfp8_scale_bytes(rows, cols, o, sf_layout), dtype=torch.uint8, device=device))
        else:
            out += [None, None]
    return tuple(out)


def mxfp8_quantize(src: torch.Tensor, orientation: int, scale_rule: int, elem: int,
                   q_row, s_row, q_col, s_col, sf_layout: int, stream=None) -> None:
    rows, cols = src.shape
    assert src.is_contiguous()
    _check(lib().mxfp8_quantize(_ptr(src), _dtype_code(src), rows, cols, orientation, scale_rule, elem,
                                _ptr(q_row), _ptr(s_row), _ptr(q_col), _ptr(s_col), sf_layout,
                                _stream(stream)), "mxfp8_quantize")


def mxfp8_dequantize(q: torch.Tensor, s: torch.Tensor, orientation: int, elem: int, sf_layout: int,
                     dst: torch.Tensor, stream=None) -> None:
    rows, cols = q.shape
    _check(lib().mxfp8_dequantize(_ptr(q), _ptr(s), rows, cols, orientation, elem, sf_layout,
                                  _ptr(dst), _dtype_code(dst), _stream(stream)), "mxfp8_dequantize")


def make_epilogue(orientation: int, scale_rule: int, elem: int, q_row=None, s_row=None, q_col=None, s_col=None):
    e = _Epilogue()
    e.orientation, e.scale_rule, e.elem = orientation, scale_rule, elem
    e.q_row = None if q_row is None else q_row.data_ptr()
    e.s_row = None if s_row is None else s_row.data_ptr()
    e.q_col = None if q_col is None else q_col.data_ptr()
    e.s_col = None if s_col is None else s_col.data_ptr()
    e._keep = (q_row, s_row, q_col, s_col)
    return e


def mxfp8_gemm(Aq, As, Bq, Bs, M: int, N: int, K: int, a_major: int, b_major: int, a_elem: int,
               b_elem: int, D, epi=None, workspace=None, stream=None) -> None:
    out_dtype = FP32 if D is None else _dtype_code(D)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().mxfp8_gemm(_ptr(Aq), _ptr(As), _ptr(Bq), _ptr(Bs), M, N, K, a_major, b_major,
                            a_elem, b_elem, _ptr(D), out_dtype,
                            None if epi is None else ctypes.byref(epi),
                            _ptr(workspace), ws_bytes, _stream(stream)), "mxfp8_gemm")


def mxfp8_quantize_host_ws_bytes(src_dtype: int, rows: int, cols: int, orientation: int) -> int:
    return int(lib().mxfp8_quantize_host_ws_bytes(src_dtype, rows, cols, orientation))


def mxfp8_quantize_host(src_host: torch.Tensor, orientation: int, scale_rule: int, elem: int,
                        q_row_host, s_row_host, q_col_host, s_col_host, sf_layout: int,
                        dev_ws: torch.Tensor, stream=None) -> None:
    rows, cols = src_host.shape
    _check(lib().mxfp8_quantize_host(_ptr(src_host), _dtype_code(src_host), rows, cols, orientation,
                                     scale_rule, elem, _ptr(q_row_host), _ptr(s_row_host),
                                     _ptr(q_col_host), _ptr(s_col_host), sf_layout, _ptr(dev_ws),
                                     dev_ws.numel() * dev_ws.element_size(), _stream(stream)),
           "mxfp8_quantize_host")


def mxfp8_linear_host_ws_bytes(T: int, H: int, F: int) -> int:
    return int(lib().mxfp8_linear_host_ws_bytes(T, H, F))


def mxfp8_linear_host(x_host, w_host, dy_host, scale_rule: int, y_host, dx_host, dw_host,
                      dev_ws: torch.Tensor, stream=None) -> None:
    T, H = x_host.shape
    F = w_host.shape[0]
    _check(lib().mxfp8_linear_host(_ptr(x_host), _ptr(w_host), _ptr(dy_host), T, H, F, scale_rule,
                                   _ptr(y_host), _ptr(dx_host), _ptr(dw_host), _ptr(dev_ws),
                                   dev_ws.numel() * dev_ws.element_size(), _stream(stream)),
           "mxfp8_linear_host")


def mxfp8_fake_quantize(src: torch.Tensor, orientation: int, scale_rule: int, elem: int,
                        dst_row, dst_col, stream=None) -> None:
    rows, cols = src.shape
    _check(lib().mxfp8_fake_quantize(_ptr(src), _dtype_code(src), rows, cols, orientation, scale_rule, elem,
                                     _ptr(dst_row), _ptr(dst_col), _stream(stream)), "mxfp8_fake_quantize")


def mxfp8_linear_ws_bytes(T: int, H: int, F: int) -> int:
    return int(lib().mxfp8_linear_ws_bytes(T, H, F))


def mxfp8_linear(x, w, dy, scale_rule: int, y, dx, dw, ws, stream=None) -> None:
    T, H = x.shape
    F = w.shape[0]
    _check(lib().mxfp8_linear(_ptr(x), _ptr(w), _ptr(dy), T, H, F, scale_rule, _ptr(y), _ptr(dx), _ptr(dw),
                              _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)), "mxfp8_linear")


GROUP_M, GROUP_K = 1, 2


def mxfp8_grouped_gemm(aq, a_s, bq, b_s, group_offsets: torch.Tensor, mode: int, M: int, N: int, K: int,
                       b_major: int, a_elem: int, b_elem: int, D: torch.Tensor, stream=None) -> None:
    assert group_offsets.dtype == torch.int32 and group_offsets.is_cuda
    _check(lib().mxfp8_grouped_gemm(_ptr(aq), _ptr(a_s), _ptr(bq), _ptr(b_s), _ptr(group_offsets),
                                    group_offsets.numel() - 1, mode, M, N, K, b_major, a_elem, b_elem,
                                    _ptr(D), _dtype_code(D), _stream(stream)), "mxfp8_grouped_gemm")


def mxfp8_sf_concat_k(parts: torch.Tensor, num_parts: int, mn: int, k_part: int, dst: torch.Tensor, stream=None) -> None:
    _check(lib().mxfp8_sf_concat_k(_ptr(parts), num_parts, mn, k_part, _ptr(dst), _stream(stream)), "mxfp8_sf_concat_k")


def mxfp8_gemm_last_clock(stream=None):
    """(SM MHz, microseconds) of the most recent GEMM launch, measured by the kernel itself; waits for the stream."""
    mhz, us = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(lib().mxfp8_gemm_last_clock(_stream(stream), ctypes.byref(mhz), ctypes.byref(us)), "mxfp8_gemm_last_clock")
    return mhz.value, us.value


def mxfp8_enable_peer_access(peer_device: int) -> None:
    _check(lib().mxfp8_enable_peer_access(peer_device), "mxfp8_enable_peer_access")


def make_owner_pointers(addresses):
    """addresses: one device address per owner (int, or a tensor whose data_ptr() is taken).  Returns the
    host pointer array mxfp8_gemm_reduce_scatter takes; build it once per set of buffers."""
    arr = (ctypes.c_void_p * len(addresses))()
    for k, a in enumerate(addresses):
        arr[k] = a.data_ptr() if isinstance(a, torch.Tensor) else int(a)
    return arr


def mxfp8_gemm_reduce_scatter(aq, a_s, bq, b_s, M: int, N: int, K: int, a_major: int, b_major: int, a_elem: int, b_elem: int,
                              owners, first_owner: int, stream=None) -> None:
    _check(lib().mxfp8_gemm_reduce_scatter(_ptr(aq), _ptr(a_s), _ptr(bq), _ptr(b_s), M, N, K, a_major, b_major, a_elem, b_elem,
                                           owners, len(owners), first_owner, _stream(stream)), "mxfp8_gemm_reduce_scatter")


def make_quantize_items(entries):
    """entries: sequence of (src, q_row, s_row, q_col, s_col) tensors (None where unused).  Returns the
    ctypes array mxfp8_quantize_multi takes; build it once and reuse it while the tensors live."""
    arr = (_QuantizeItem * len(entries))()
    for k, (src, q_row, s_row, q_col, s_col) in enumerate(entries):
        assert src.is_contiguous()
        arr[k].src = src.data_ptr()
        arr[k].rows, arr[k].cols = src.shape
        arr[k].q_row, arr[k].s_row, arr[k].q_col, arr[k].s_col = _ptr(q_row), _ptr(s_row), _ptr(q_col), _ptr(s_col)
    return arr


def mxfp8_quantize_multi(items, src_dtype: int, orientation: int, scale_rule: int, elem: int, sf_layout: int,
                         stream=None) -> None:
    _check(lib().mxfp8_quantize_multi(items, len(items), src_dtype, orientation, scale_rule, elem, sf_layout,
                                      _stream(stream)), "mxfp8_quantize_multi")


def make_gemm_problems(entries):
    """entries: sequence of (Aq, As, Bq, Bs, M, N, K, a_major, b_major, a_elem, b_elem, D).  Returns the ctypes
    array mxfp8_gemm_multi takes; build it once and reuse it while the tensors live."""
    arr = (_GemmProblem * len(entries))()
    for k, (aq, a_s, bq, b_s, M, N, K, a_major, b_major, a_elem, b_elem, D) in enumerate(entries):
        arr[k].Aq, arr[k].As, arr[k].Bq, arr[k].Bs = aq.data_ptr(), a_s.data_ptr(), bq.data_ptr(), b_s.data_ptr()
        arr[k].M, arr[k].N, arr[k].K = M, N, K
        arr[k].a_major, arr[k].b_major, arr[k].a_elem, arr[k].b_elem = a_major, b_major, a_elem, b_elem
        arr[k].D = D.data_ptr()
    return arr


def mxfp8_gemm_multi(problems, out_dtype: int, stream=None) -> None:
    _check(lib().mxfp8_gemm_multi(problems, len(problems), out_dtype, _stream(stream)), "mxfp8_gemm_multi")


def mxfp8_act_grad_quantize(dh: torch.Tensor, z: torch.Tensor, act: int, orientation: int, scale_rule: int, elem: int,
                            q_row, s_row, q_col, s_col, sf_layout: int, stream=None) -> None:
    rows, cols = z.shape
    assert z.is_contiguous() and dh.is_contiguous() and dh.shape == z.shape and dh.dtype == z.dtype
    _check(lib().mxfp8_act_grad_quantize(_ptr(dh), _ptr(z), _dtype_code(z), rows, cols, act, orientation, scale_rule, elem,
                                         _ptr(q_row), _ptr(s_row), _ptr(q_col), _ptr(s_col), sf_layout,
                                         _stream(stream)), "mxfp8_act_grad_quantize")


def mxfp8_act_quantize(src: torch.Tensor, act: int, orientation: int, scale_rule: int, elem: int,
                       q_row, s_row, q_col, s_col, sf_layout: int, stream=None) -> None:
    rows, cols = src.shape
    assert src.is_contiguous()
    _check(lib().mxfp8_act_quantize(_ptr(src), _dtype_code(src), rows, cols, act, orientation, scale_rule, elem,
                                    _ptr(q_row), _ptr(s_row), _ptr(q_col), _ptr(s_col), sf_layout,
                                    _stream(stream)), "mxfp8_act_quantize")


def mxfp8_layernorm_quantize(src: torch.Tensor, gamma: torch.Tensor, beta: torch.Tensor, eps: float, mean: torch.Tensor, rstd: torch.Tensor,
                             orientation: int, scale_rule: int, elem: int,
                             q_row, s_row, q_col, s_col, sf_layout: int, stream=None) -> None:
    rows, cols = src.shape
    assert src.is_contiguous() and gamma.dtype == src.dtype and beta.dtype == src.dtype
    assert mean.dtype == torch.float32 and rstd.dtype == torch.float32
    _check(lib().mxfp8_layernorm_quantize(_ptr(src), _dtype_code(src), rows, cols, _ptr(gamma), _ptr(beta), eps, _ptr(mean), _ptr(rstd),
                                          orientation, scale_rule, elem, _ptr(q_row), _ptr(s_row), _ptr(q_col), _ptr(s_col), sf_layout,
                                          _stream(stream)), "mxfp8_layernorm_quantize")


def mxfp8_rmsnorm_quantize(src: torch.Tensor, gamma: torch.Tensor, eps: float, rstd: torch.Tensor,
                           orientation: int, scale_rule: int, elem: int,
                           q_row, s_row, q_col, s_col, sf_layout: int, stream=None) -> None:
    rows, cols = src.shape
    assert src.is_contiguous() and gamma.dtype == src.dtype and gamma.numel() == cols
    assert rstd.dtype == torch.float32 and rstd.numel() == rows
    _check(lib().mxfp8_rmsnorm_quantize(_ptr(src), _dtype_code(src), rows, cols, _ptr(gamma), eps, _ptr(rstd),
                                        orientation, scale_rule, elem, _ptr(q_row), _ptr(s_row), _ptr(q_col), _ptr(s_col),
                                        sf_layout, _stream(stream)), "mxfp8_rmsnorm_quantize")


def mxfp8_rmsnorm_quantize_static_max_rows() -> int:
    return int(lib().mxfp8_rmsnorm_quantize_static_max_rows())


def mxfp8_rmsnorm_quantize_static(src: torch.Tensor, gamma: torch.Tensor, eps: float,
                                  orientation: int, scale_rule: int, elem: int,
                                  q_row, s_row, q_col, s_col, sf_layout: int, stream=None) -> None:
    rows, cols = src.shape
    assert src.is_contiguous() and gamma.dtype == src.dtype and gamma.numel() == cols
    _check(lib().mxfp8_rmsnorm_quantize_static(_ptr(src), _dtype_code(src), rows, cols, _ptr(gamma), eps,
                                               orientation, scale_rule, elem, _ptr(q_row), _ptr(s_row), _ptr(q_col),
                                               _ptr(s_col), sf_layout, _stream(stream)), "mxfp8_rmsnorm_quantize_static")


def mxfp8_glu_quantize(src: torch.Tensor, act: int, orientation: int, scale_rule: int, elem: int,
                       q_row, s_row, q_col, s_col, sf_layout: int, stream=None) -> None:
    """src: [rows, 2 * cols] = (gate | up); the outputs have shape [rows, cols]."""
    rows, two_cols = src.shape
    assert src.is_contiguous() and two_cols % 2 == 0
    _check(lib().mxfp8_glu_quantize(_ptr(src), _dtype_code(src), rows, two_cols // 2, act, orientation, scale_rule, elem,
                                    _ptr(q_row), _ptr(s_row), _ptr(q_col), _ptr(s_col), sf_layout,
                                    _stream(stream)), "mxfp8_glu_quantize")
