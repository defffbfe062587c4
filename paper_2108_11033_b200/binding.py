"""Thin ctypes binding of libgrim.so: argument marshalling only.

Function names mirror the C ABI (include/grim.h).  Host arrays are NumPy arrays, device
buffers are torch CUDA tensors (torch is used for device memory and streams only).  There
is no fallback: if the shared library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libgrim.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} not found: build it with `python -m paper_2108_11033_b200.build` "
        "(there is no CPU or PyTorch fallback for the CUDA library)")

lib = C.CDLL(LIB_PATH)

GRIM_OK = 0
GRIM_ERR_INVALID_ARG, GRIM_ERR_SHAPE, GRIM_ERR_DTYPE, GRIM_ERR_NOT_BCR = 1, 2, 3, 4
GRIM_ERR_ALLOC, GRIM_ERR_CUDA, GRIM_ERR_UNSUPPORTED, GRIM_ERR_TIMEOUT = 5, 6, 7, 8
GRIM_F32, GRIM_BF16 = 0, 1
GRIM_PACK_REORDER, GRIM_PACK_HOST_ONLY, GRIM_PACK_NARROW_ONLY, GRIM_PACK_WIDE_ONLY = 1, 2, 4, 8
GRIM_CONV_RELU, GRIM_CONV_PAIRED, GRIM_CONV_SINGLE = 1, 2, 4

EXPORTED = [
    "grim_bcr_pack", "grim_bcr_destroy", "grim_bcr_info", "grim_bcr_export", "grim_bcr_unpack_dense",
    "grim_bcr_spmm", "grim_bcr_spmm_ex", "grim_bcr_status", "grim_bcr_tune", "grim_bcr_conv2d", "grim_maxpool2x2",
    "grim_gru_create", "grim_gru_seq", "grim_gru_status", "grim_gru_destroy", "grim_gru_debug_barrier",
    "grim_gru_profile", "grim_gru_profile_read", "grim_gru_seq_static", "grim_gru_set_pipeline",
    "grim_launch_count", "grim_launch_count_reset", "grim_status_string", "grim_version", "grim_measure_ffma_peak", "grim_bcr_reserve", "grim_bcr_export_bcrc", "grim_bcr_project", "grim_gru_step",
]


class GrimError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class grim_mat_t(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64), ("dtype", C.c_int)]


class grim_bcr_info_t(C.Structure):
    _fields_ = [("M", C.c_int64), ("K", C.c_int64), ("bh", C.c_int32), ("bw", C.c_int32), ("nbr", C.c_int64),
                ("nbc", C.c_int64), ("nnz", C.c_int64), ("nonempty_blocks", C.c_int64), ("k_used", C.c_int64),
                ("dtype", C.c_int32), ("flags", C.c_uint32), ("on_device", C.c_int32), ("reserved", C.c_int32),
                ("value_bytes", C.c_int64), ("index_bytes_spmm", C.c_int64), ("index_bytes_gemv", C.c_int64),
                ("export_bytes", C.c_int64), ("index_bytes_tc", C.c_int64)]


class grim_bcrc_sizes_t(C.Structure):
    _fields_ = [("M", C.c_int64), ("K", C.c_int64), ("nnz", C.c_int64), ("groups", C.c_int64), ("compact_columns", C.c_int64)]


class grim_tune_t(C.Structure):
    _fields_ = [("tile_n", C.c_int32), ("path", C.c_int32), ("reserved", C.c_int32 * 6)]


class grim_conv_desc_t(C.Structure):
    _fields_ = [("N", C.c_int64), ("C", C.c_int64), ("H", C.c_int64), ("W", C.c_int64), ("KH", C.c_int32),
                ("KW", C.c_int32), ("stride", C.c_int32), ("pad", C.c_int32), ("bias_dev", C.c_void_p),
                ("flags", C.c_uint32), ("in_dtype", C.c_int), ("out_dtype", C.c_int)]


_vp = C.c_void_p
lib.grim_bcr_pack.argtypes = [_vp, C.c_int64, _vp, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_int,
                              C.c_uint32, C.POINTER(_vp)]
lib.grim_bcr_destroy.argtypes = [_vp]
lib.grim_bcr_status.argtypes = [_vp]
lib.grim_bcr_reserve.argtypes = [_vp, C.c_int64]
lib.grim_bcr_info.argtypes = [_vp, C.POINTER(grim_bcr_info_t)]
lib.grim_bcr_export.argtypes = [_vp, _vp, C.c_int64, C.POINTER(C.c_int64)]
lib.grim_bcr_unpack_dense.argtypes = [_vp, _vp, C.c_int64]
lib.grim_bcr_project.argtypes = [_vp, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_double, _vp, C.c_int64, C.POINTER(C.c_int64)]
lib.grim_bcr_export_bcrc.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, C.POINTER(grim_bcrc_sizes_t)]
lib.grim_bcr_spmm.argtypes = [_vp, C.POINTER(grim_mat_t), C.POINTER(grim_mat_t), _vp]
lib.grim_bcr_spmm_ex.argtypes = [_vp, C.POINTER(grim_mat_t), C.POINTER(grim_mat_t), C.POINTER(grim_tune_t), _vp]
lib.grim_bcr_tune.argtypes = [_vp, C.POINTER(grim_mat_t), C.POINTER(grim_mat_t), C.c_int, C.POINTER(grim_tune_t),
                              C.POINTER(C.c_float), _vp]
lib.grim_bcr_conv2d.argtypes = [_vp, C.POINTER(grim_conv_desc_t), _vp, _vp, _vp]
lib.grim_maxpool2x2.argtypes = [_vp, _vp, C.c_int64, C.c_int64, C.c_int64, C.c_int64, C.c_int, _vp]
lib.grim_gru_create.argtypes = [C.c_int, C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp), C.c_int64,
                                C.POINTER(_vp)]
lib.grim_gru_seq.argtypes = [_vp, _vp, C.c_int64, _vp, _vp, _vp, _vp]
lib.grim_gru_seq_static.argtypes = [_vp, _vp, C.c_int64, _vp, _vp, _vp, _vp]
lib.grim_gru_status.argtypes = [_vp]
lib.grim_gru_step.argtypes = [_vp, _vp, C.c_int64, _vp, _vp, _vp]
lib.grim_gru_destroy.argtypes = [_vp]
lib.grim_gru_debug_barrier.argtypes = [_vp, C.c_int, C.c_uint]
lib.grim_gru_profile.argtypes = [_vp, C.c_int]
lib.grim_gru_set_pipeline.argtypes = [_vp, C.c_int]
lib.grim_gru_profile_read.argtypes = [_vp, C.POINTER(C.c_float), C.POINTER(C.c_float)]
lib.grim_measure_ffma_peak.argtypes = [C.POINTER(C.c_double), _vp]
lib.grim_launch_count.restype = C.c_int64
lib.grim_launch_count_reset.restype = None
lib.grim_status_string.argtypes = [C.c_int]
lib.grim_status_string.restype = C.c_char_p
lib.grim_version.restype = C.c_char_p


def status_string(s: int) -> str:
    return lib.grim_status_string(int(s)).decode()


def grim_version() -> str:
    return lib.grim_version().decode()


def _check(st: int, where: str):
    if st != GRIM_OK:
        raise GrimError(st, where)


def _stream_ptr(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _torch_dtype_code(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return GRIM_F32
    if t.dtype == torch.bfloat16:
        return GRIM_BF16
    raise TypeError(f"unsupported tensor dtype {t.dtype}")


def _mat(t) -> grim_mat_t:
    if t.dim() == 1:
        t = t.unsqueeze(1)
    assert t.is_cuda and t.dim() == 2 and t.stride(1) == 1
    return grim_mat_t(t.data_ptr(), t.shape[0], t.shape[1], t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1]),
                      _torch_dtype_code(t))


# ------------------------------------------------------------------------------------------ packing


def grim_bcr_pack(W: np.ndarray, mask: np.ndarray, bh: int, bw: int, dtype: int = GRIM_F32, flags: int = 0) -> int:
    W = np.ascontiguousarray(W, dtype=np.float32)
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    assert W.ndim == 2 and W.shape == mask.shape
    h = _vp()
    st = lib.grim_bcr_pack(W.ctypes.data, W.shape[1], mask.ctypes.data, mask.shape[1], W.shape[0], W.shape[1], bh, bw,
                           dtype, flags, C.byref(h))
    _check(st, "grim_bcr_pack")
    return h.value


def grim_bcr_destroy(h: int):
    _check(lib.grim_bcr_destroy(h), "grim_bcr_destroy")


def grim_bcr_info(h: int) -> grim_bcr_info_t:
    info = grim_bcr_info_t()
    _check(lib.grim_bcr_info(h, C.byref(info)), "grim_bcr_info")
    return info


def grim_bcr_export(h: int) -> bytes:
    n = grim_bcr_info(h).export_bytes
    buf = np.empty(n, dtype=np.uint8)
    written = C.c_int64(0)
    _check(lib.grim_bcr_export(h, buf.ctypes.data, n, C.byref(written)), "grim_bcr_export")
    return buf[:written.value].tobytes()


def grim_bcr_export_bcrc(h: int) -> dict:
    sz = grim_bcrc_sizes_t()
    _check(lib.grim_bcr_export_bcrc(h, None, None, None, None, None, None, C.byref(sz)), "grim_bcr_export_bcrc")
    out = dict(reorder=np.empty(sz.M, np.int32), row_offset=np.empty(sz.M + 1, np.int64),
               occurrence=np.empty(sz.groups + 1, np.int32), column_stride=np.empty(sz.groups + 1, np.int64),
               compact_column=np.empty(sz.compact_columns, np.int32), weights=np.empty(sz.nnz, np.float32))
    _check(lib.grim_bcr_export_bcrc(h, out["reorder"].ctypes.data, out["row_offset"].ctypes.data, out["occurrence"].ctypes.data,
                                    out["column_stride"].ctypes.data, out["compact_column"].ctypes.data,
                                    out["weights"].ctypes.data, C.byref(sz)), "grim_bcr_export_bcrc")
    return out


def grim_bcr_project(V: np.ndarray, bh: int, bw: int, sparsity: float) -> np.ndarray:
    V = np.ascontiguousarray(V, dtype=np.float32)
    M, K = V.shape
    mask = np.empty((M, K), np.uint8)
    kept = C.c_int64(0)
    _check(lib.grim_bcr_project(V.ctypes.data, K, M, K, bh, bw, float(sparsity), mask.ctypes.data, K, C.byref(kept)),
           "grim_bcr_project")
    assert int(mask.sum()) == kept.value
    return mask


def grim_bcr_unpack_dense(h: int) -> np.ndarray:
    info = grim_bcr_info(h)
    W = np.empty((info.M, info.K), dtype=np.float32)
    _check(lib.grim_bcr_unpack_dense(h, W.ctypes.data, info.K), "grim_bcr_unpack_dense")
    return W


# ------------------------------------------------------------------------------------------ multiply


def grim_bcr_spmm(h: int, X, Y, stream=None):
    mx, my = _mat(X), _mat(Y)
    _check(lib.grim_bcr_spmm(h, C.byref(mx), C.byref(my), _stream_ptr(stream)), "grim_bcr_spmm")


def grim_bcr_reserve(h: int, max_ncols: int):
    _check(lib.grim_bcr_reserve(h, int(max_ncols)), "grim_bcr_reserve")


def grim_bcr_status(h: int) -> int:
    return lib.grim_bcr_status(h)


def grim_bcr_spmm_ex(h: int, X, Y, tile_n: int = 0, path: int = 0, stream=None):
    mx, my = _mat(X), _mat(Y)
    tune = grim_tune_t(tile_n, path)
    _check(lib.grim_bcr_spmm_ex(h, C.byref(mx), C.byref(my), C.byref(tune), _stream_ptr(stream)), "grim_bcr_spmm_ex")


def grim_bcr_tune(h: int, X, Y, reps: int = 5, stream=None):
    mx, my = _mat(X), _mat(Y)
    best = grim_tune_t()
    ms = C.c_float(0)
    _check(lib.grim_bcr_tune(h, C.byref(mx), C.byref(my), reps, C.byref(best), C.byref(ms), _stream_ptr(stream)),
           "grim_bcr_tune")
    return dict(tile_n=best.tile_n, path=best.path, ms=ms.value)


def grim_bcr_conv2d(h: int, x, out, ksize: int, stride: int = 1, pad: int = 0, bias=None, relu: bool = False,
                    stream=None, kernel_flags: int = 0):
    assert x.is_cuda and out.is_cuda and x.is_contiguous() and out.is_contiguous() and x.dim() == 4
    d = grim_conv_desc_t(x.shape[0], x.shape[1], x.shape[2], x.shape[3], ksize, ksize, stride, pad,
                         bias.data_ptr() if bias is not None else None, (GRIM_CONV_RELU if relu else 0) | kernel_flags,
                         _torch_dtype_code(x), _torch_dtype_code(out))
    _check(lib.grim_bcr_conv2d(h, C.byref(d), x.data_ptr(), out.data_ptr(), _stream_ptr(stream)), "grim_bcr_conv2d")


def grim_maxpool2x2(x, out, stream=None):
    assert x.is_cuda and out.is_cuda and x.is_contiguous() and out.is_contiguous()
    n, c, hh, ww = x.shape
    _check(lib.grim_maxpool2x2(x.data_ptr(), out.data_ptr(), n, c, hh, ww, _torch_dtype_code(x), _stream_ptr(stream)),
           "grim_maxpool2x2")


# ------------------------------------------------------------------------------------------ GRU


def grim_gru_create(W_ih, W_hh, b_ih, b_hh, max_T: int) -> int:
    L = len(W_ih)
    keep = [np.ascontiguousarray(b, dtype=np.float32) for b in list(b_ih) + list(b_hh)]
    arr = lambda xs: (_vp * L)(*xs)
    g = _vp()
    st = lib.grim_gru_create(L, arr(W_ih), arr(W_hh), arr([k.ctypes.data for k in keep[:L]]),
                             arr([k.ctypes.data for k in keep[L:]]), max_T, C.byref(g))
    _check(st, "grim_gru_create")
    return g.value


def grim_gru_seq(g: int, x, y, h0=None, hT=None, stream=None):
    assert x.is_cuda and y.is_cuda and x.is_contiguous() and y.is_contiguous()
    _check(lib.grim_gru_seq(g, x.data_ptr(), x.shape[0], h0.data_ptr() if h0 is not None else None, y.data_ptr(),
                            hT.data_ptr() if hT is not None else None, _stream_ptr(stream)), "grim_gru_seq")


def grim_gru_seq_static(g: int, x, y, h0=None, hT=None, stream=None):
    """grim_gru_seq for callers that may not allocate device memory: scratch comes from a fixed 8 MiB
    array inside the library (shared by all calls; see include/grim.h for the size limit)."""
    assert x.is_cuda and y.is_cuda and x.is_contiguous() and y.is_contiguous()
    _check(lib.grim_gru_seq_static(g, x.data_ptr(), x.shape[0], h0.data_ptr() if h0 is not None else None,
                                   y.data_ptr(), hT.data_ptr() if hT is not None else None, _stream_ptr(stream)),
           "grim_gru_seq_static")


def grim_gru_step(g: int, x, h, y=None, stream=None):
    assert x.is_cuda and h.is_cuda and x.is_contiguous() and h.is_contiguous() and x.dim() == 2 and h.dim() == 3
    _check(lib.grim_gru_step(g, x.data_ptr(), x.shape[0], h.data_ptr(), y.data_ptr() if y is not None else None,
                             _stream_ptr(stream)), "grim_gru_step")


def grim_gru_status(g: int) -> int:
    return lib.grim_gru_status(g)


def grim_gru_debug_barrier(g: int, skip_cta: int, spin_limit: int):
    _check(lib.grim_gru_debug_barrier(g, skip_cta, spin_limit), "grim_gru_debug_barrier")


def grim_gru_set_pipeline(g: int, chunks: int):
    _check(lib.grim_gru_set_pipeline(g, chunks), "grim_gru_set_pipeline")


def grim_gru_profile(g: int, enable: bool):
    _check(lib.grim_gru_profile(g, int(enable)), "grim_gru_profile")


def grim_gru_profile_read(g: int):
    a, b = C.c_float(0), C.c_float(0)
    _check(lib.grim_gru_profile_read(g, C.byref(a), C.byref(b)), "grim_gru_profile_read")
    return a.value, b.value


def grim_gru_destroy(g: int):
    _check(lib.grim_gru_destroy(g), "grim_gru_destroy")


def grim_measure_ffma_peak(stream=None) -> float:
    v = C.c_double(0.0)
    _check(lib.grim_measure_ffma_peak(C.byref(v), _stream_ptr(stream)), "grim_measure_ffma_peak")
    return float(v.value)


def grim_launch_count() -> int:
    return lib.grim_launch_count()


def grim_launch_count_reset():
    lib.grim_launch_count_reset()
