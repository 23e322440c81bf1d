"""ctypes binding of libspdp (include/spdp.h): same entry points, argument marshalling only.

Tensors are torch CUDA tensors (their data_ptr() is handed to the library); the stream is
torch's current stream unless given.  There is no fallback: if libspdp.so is missing the
first call raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspdp.so")

SPDP_OK = 0
SPDP_ERR_INVALID_ARG = -1
SPDP_ERR_UNSUPPORTED_SHAPE = -2
SPDP_ERR_ALLOC = -3
SPDP_ERR_CUDA = -4
SPDP_ERR_OVERFLOW = -5
SPDP_ERR_TIMEOUT = -6

SPDP_DP_NONE, SPDP_DP_ABS_GT, SPDP_DP_MASK = 0, 1, 2
SPDP_Y_F16, SPDP_Y_F32 = 0, 1

EXPORTS = (
    "spdp_pack_tiled_cbc", "spdp_pack_tiled_cbc_ex", "spdp_import_tiled_cbc", "spdp_spmspv",
    "spdp_spmspv_host", "spdp_spmspv_noalloc", "spdp_spmspv_batch", "spdp_free", "spdp_get_info", "spdp_export", "spdp_unpack",
    "spdp_active_columns", "spdp_last_device_status", "spdp_set_num_ctas", "spdp_last_cuda_error",
    "spdp_status_string", "spdp_probe_stream_read", "spdp_probe_gather", "spdp_spmm", "spdp_pack_tiled_cbc_q4", "spdp_export_q4", "spdp_row_shard", "spdp_swiglu_dp",
)


class spdp_info(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in ("M", "K", "R", "C", "NGT", "pad_elems", "nnz", "values_len",
                                              "packed_bytes", "workspace_bytes")] + \
               [(n, ctypes.c_void_p) for n in ("tileoffset_dev", "colinfo_dev", "bitmap_dev", "values_dev")] + \
               [("num_ctas", ctypes.c_int32), ("device", ctypes.c_int32)]


class SpdpError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().spdp_status_string(status).decode()
        detail = lib().spdp_last_cuda_error().decode()
        super().__init__(f"{where}: {msg}" + (f" [{detail}]" if detail and status in (-3, -4) else ""))


_lib = None


def lib():
    """Loads libspdp.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_21985_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, ci, cf = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float
        L.spdp_pack_tiled_cbc.argtypes = [vp, i64, i64, i64, ci, ci, vp, ctypes.POINTER(vp)]
        L.spdp_pack_tiled_cbc_ex.argtypes = [vp, i64, i64, i64, ci, ci, ci, vp, ctypes.POINTER(vp)]
        L.spdp_import_tiled_cbc.argtypes = [i64, i64, ci, vp, vp, vp, vp, i64, ctypes.POINTER(vp)]
        L.spdp_spmspv.argtypes = [vp, vp, ci, cf, vp, vp, ci, vp]
        L.spdp_spmspv_host.argtypes = [vp, vp, ci, cf, vp, vp, ci, vp]
        L.spdp_spmspv_noalloc.argtypes = [vp, vp, vp, vp, i64, i64, vp, ci, cf, vp, vp, ci, vp]
        L.spdp_spmspv_batch.argtypes = [vp, vp, i64, ci, ci, cf, vp, i64, vp, i64, ci, vp]
        L.spdp_free.argtypes = [vp]
        L.spdp_get_info.argtypes = [vp, ctypes.POINTER(spdp_info)]
        L.spdp_export.argtypes = [vp, vp, vp, vp, vp]
        L.spdp_unpack.argtypes = [vp, vp, i64, vp]
        L.spdp_active_columns.argtypes = [vp, vp, ci, cf, vp, vp, vp, vp]
        L.spdp_last_device_status.argtypes = [vp, ctypes.POINTER(ci)]
        L.spdp_set_num_ctas.argtypes = [vp, ci]
        L.spdp_spmm.argtypes = [vp, vp, i64, i64, vp, i64, ci, vp]
        L.spdp_pack_tiled_cbc_q4.argtypes = [vp, i64, i64, i64, ci, ci, vp, ctypes.POINTER(vp)]
        L.spdp_export_q4.argtypes = [vp, vp, vp, vp, vp, vp]
        L.spdp_swiglu_dp.argtypes = [vp, vp, i64, cf, vp, vp, vp, vp]
        L.spdp_row_shard.argtypes = [i64, ci, ci, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.spdp_probe_stream_read.argtypes = [vp, vp]
        L.spdp_probe_gather.argtypes = [vp, vp, ci, cf, vp, vp]
        for name in EXPORTS:
            getattr(L, name).restype = ci
        L.spdp_last_cuda_error.restype = ctypes.c_char_p
        L.spdp_last_cuda_error.argtypes = []
        L.spdp_status_string.restype = ctypes.c_char_p
        L.spdp_status_string.argtypes = [ci]
        _lib = L
    return _lib


def _check(st: int, where: str):
    if st != SPDP_OK:
        raise SpdpError(st, where)


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


def _dev_ptr(t, name, allow_none=False):
    if t is None:
        if allow_none:
            return None
        raise ValueError(f"{name} is required")
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor")
    return t.data_ptr()


def _host_ptr(a, name, allow_none=False):
    if a is None:
        if allow_none:
            return None
        raise ValueError(f"{name} is required")
    if isinstance(a, np.ndarray):
        if not a.flags["C_CONTIGUOUS"]:
            raise ValueError(f"{name} must be C-contiguous")
        return a.ctypes.data
    if a.is_cuda or not a.is_contiguous():       # torch CPU tensor (e.g. pinned)
        raise ValueError(f"{name} must be a contiguous host tensor")
    return a.data_ptr()


# ---- the entry points, named as in spdp.h --------------------------------------------------
def spdp_pack_tiled_cbc(W, tile_m: int = 256, tile_k: int = 16, stream=None, pad_elems: int | None = None) -> int:
    """W: fp16 CUDA tensor [M, K] (row stride = ldw, unit column stride).  Returns the handle."""
    import torch
    if W.dtype != torch.float16 or W.dim() != 2 or not W.is_cuda or W.stride(1) != 1:
        raise ValueError("W must be a 2-D fp16 CUDA tensor with unit column stride")
    M, K = W.shape
    h = ctypes.c_void_p()
    if pad_elems is None:
        st = lib().spdp_pack_tiled_cbc(W.data_ptr(), M, K, W.stride(0), tile_m, tile_k, _stream(stream), ctypes.byref(h))
    else:
        st = lib().spdp_pack_tiled_cbc_ex(W.data_ptr(), M, K, W.stride(0), tile_m, tile_k, pad_elems,
                                          _stream(stream), ctypes.byref(h))
    _check(st, "spdp_pack_tiled_cbc")
    return h.value


def spdp_pack_tiled_cbc_q4(W, stream=None) -> int:
    """W: fp16 CUDA tensor [M, K] -> handle of the 4-bit variant (codes + one fp16 scale per column tile)."""
    import torch
    if W.dtype != torch.float16 or W.dim() != 2 or not W.is_cuda or W.stride(1) != 1:
        raise ValueError("W must be a 2-D fp16 CUDA tensor with unit column stride")
    M, K = W.shape
    h = ctypes.c_void_p()
    st = lib().spdp_pack_tiled_cbc_q4(W.data_ptr(), M, K, W.stride(0), 256, 16, _stream(stream), ctypes.byref(h))
    _check(st, "spdp_pack_tiled_cbc_q4")
    return h.value


def spdp_export_q4(h: int) -> dict:
    """The arrays of a 4-bit handle as NumPy arrays (synchronous device-to-host copies)."""
    info = spdp_get_info(h)
    to = np.empty(info.NGT + 1, np.uint32)
    ci = np.empty(info.NGT * 16, np.uint32)
    bm = np.empty(info.NGT * 64, np.uint64)
    codes = np.empty(info.values_len // 2, np.uint8)
    scales = np.empty(info.NGT * 16, np.uint16)
    st = lib().spdp_export_q4(h, to.ctypes.data, ci.ctypes.data, bm.ctypes.data, codes.ctypes.data if codes.size else None,
                              scales.ctypes.data)
    _check(st, "spdp_export_q4")
    return dict(M=info.M, K=info.K, pad_elems=info.pad_elems, tileoffset=to, colinfo=ci, bitmap=bm, codes=codes,
                scales=scales, nnz=info.nnz)


def spdp_import_tiled_cbc(M: int, K: int, tileoffset, colinfo, bitmap, values, pad_elems: int = 8) -> int:
    """Host arrays (NumPy: uint32, uint32, uint64, uint16/float16) -> handle."""
    to = np.ascontiguousarray(tileoffset, dtype=np.uint32)
    ci = np.ascontiguousarray(colinfo, dtype=np.uint32)
    bm = np.ascontiguousarray(bitmap, dtype=np.uint64)
    va = np.ascontiguousarray(values)
    if va.dtype == np.float16:
        va = va.view(np.uint16)
    if va.dtype != np.uint16:
        raise ValueError("values must be uint16 bit patterns or float16")
    h = ctypes.c_void_p()
    st = lib().spdp_import_tiled_cbc(M, K, pad_elems, to.ctypes.data, ci.ctypes.data, bm.ctypes.data,
                                     va.ctypes.data if va.size else None, va.size, ctypes.byref(h))
    _check(st, "spdp_import_tiled_cbc")
    return h.value


def spdp_spmspv(h: int, x, rule: int, thr: float, y, mask=None, stream=None) -> None:
    """x: fp16 CUDA [K]; y: fp16 or fp32 CUDA [M] (its dtype selects the output type)."""
    import torch
    ydt = SPDP_Y_F32 if y.dtype == torch.float32 else SPDP_Y_F16
    if y.dtype not in (torch.float16, torch.float32) or x.dtype != torch.float16:
        raise ValueError("x must be fp16 and y fp16 or fp32")
    st = lib().spdp_spmspv(h, _dev_ptr(x, "x"), rule, float(thr), _dev_ptr(mask, "mask", True), _dev_ptr(y, "y"),
                           ydt, _stream(stream))
    _check(st, "spdp_spmspv")


def spdp_spmspv_host(h: int, x_host, rule: int, thr: float, y_host, mask_host=None, stream=None) -> None:
    """x_host / y_host: host arrays (NumPy or pinned torch CPU tensors); blocks until y_host is filled."""
    ydt = SPDP_Y_F32 if str(y_host.dtype).endswith("float32") else SPDP_Y_F16
    st = lib().spdp_spmspv_host(h, _host_ptr(x_host, "x_host"), rule, float(thr),
                                _host_ptr(mask_host, "mask_host", True), _host_ptr(y_host, "y_host"), ydt,
                                _stream(stream))
    _check(st, "spdp_spmspv_host")


def spdp_spmspv_noalloc(tileoffset, colinfo, bitmap, values, M: int, K: int, x, rule: int, thr: float, y,
                        mask=None, stream=None) -> None:
    """The allocation-free call: the four packed arrays are CUDA tensors (or raw device addresses)
    owned by the caller; scratch lives in a fixed array inside the library.  For callers that
    cannot let the library allocate device memory; see spdp.h for the limits and the sharing rule."""
    import torch
    ydt = SPDP_Y_F32 if y.dtype == torch.float32 else SPDP_Y_F16
    if y.dtype not in (torch.float16, torch.float32) or x.dtype != torch.float16:
        raise ValueError("x must be fp16 and y fp16 or fp32")
    ptr = lambda t, n: t if isinstance(t, int) else _dev_ptr(t, n)
    st = lib().spdp_spmspv_noalloc(ptr(tileoffset, "tileoffset"), ptr(colinfo, "colinfo"), ptr(bitmap, "bitmap"),
                                   ptr(values, "values"), M, K, _dev_ptr(x, "x"), rule, float(thr),
                                   _dev_ptr(mask, "mask", True), _dev_ptr(y, "y"), ydt, _stream(stream))
    _check(st, "spdp_spmspv_noalloc")


def spdp_spmspv_batch(h: int, X, rule: int, thr: float, Y, mask=None, stream=None) -> None:
    """Small-batch call: X fp16 CUDA [B][K] (rows may be strided), Y fp16 or fp32 CUDA [B][M], 1 <= B <= 8;
    mask (SPDP_DP_MASK only) int32/uint32 CUDA [B][>= ceil(K/32)] words."""
    import torch
    if X.dim() != 2 or Y.dim() != 2 or X.shape[0] != Y.shape[0]:
        raise ValueError("X must be [B][K] and Y [B][M]")
    if Y.dtype not in (torch.float16, torch.float32) or X.dtype != torch.float16:
        raise ValueError("X must be fp16 and Y fp16 or fp32")
    if X.stride(1) != 1 or Y.stride(1) != 1 or (mask is not None and (mask.dim() != 2 or mask.stride(1) != 1)):
        raise ValueError("the last dimension of X, Y and mask must be contiguous")
    ydt = SPDP_Y_F32 if Y.dtype == torch.float32 else SPDP_Y_F16
    B = int(X.shape[0])
    ldx = int(X.stride(0)) if B > 1 else int(X.shape[1])
    ldy = int(Y.stride(0)) if B > 1 else int(Y.shape[1])
    mstride = 0 if mask is None else (int(mask.stride(0)) if B > 1 else int(mask.shape[1]))
    if not X.is_cuda or not Y.is_cuda or (mask is not None and not mask.is_cuda):
        raise ValueError("X, Y and mask must be CUDA tensors")
    st = lib().spdp_spmspv_batch(h, X.data_ptr(), ldx, B, rule, float(thr),
                                 None if mask is None else mask.data_ptr(), mstride, Y.data_ptr(), ldy, ydt,
                                 _stream(stream))
    _check(st, "spdp_spmspv_batch")


def spdp_spmm(h: int, X, Y, stream=None) -> None:
    """Prefill call: X fp16 CUDA [N][K] (rows may be strided), Y fp16 or fp32 CUDA [N][M]."""
    import torch
    if X.dim() != 2 or Y.dim() != 2 or X.shape[0] != Y.shape[0] or not X.is_cuda or not Y.is_cuda:
        raise ValueError("X must be CUDA [N][K] and Y CUDA [N][M]")
    if Y.dtype not in (torch.float16, torch.float32) or X.dtype != torch.float16:
        raise ValueError("X must be fp16 and Y fp16 or fp32")
    if X.stride(1) != 1 or Y.stride(1) != 1:
        raise ValueError("the last dimension of X and Y must be contiguous")
    N = int(X.shape[0])
    ldx = int(X.stride(0)) if N > 1 else max(int(X.shape[1]), int(X.stride(0)))
    ldy = int(Y.stride(0)) if N > 1 else max(int(Y.shape[1]), int(Y.stride(0)))
    ydt = SPDP_Y_F32 if Y.dtype == torch.float32 else SPDP_Y_F16
    _check(lib().spdp_spmm(h, X.data_ptr(), N, ldx, Y.data_ptr(), ldy, ydt, _stream(stream)), "spdp_spmm")


def spdp_swiglu_dp(gate, up, thr: float, x_out, mask_out, count_out=None, stream=None) -> None:
    """x_out = silu(gate) * up (fp16 CUDA [K]) and the K-bit keep-mask of its columns in one pass."""
    K = int(gate.shape[0])
    st = lib().spdp_swiglu_dp(_dev_ptr(gate, "gate"), _dev_ptr(up, "up"), K, float(thr), _dev_ptr(x_out, "x_out"),
                              _dev_ptr(mask_out, "mask_out"), _dev_ptr(count_out, "count_out", True), _stream(stream))
    _check(st, "spdp_swiglu_dp")


def spdp_row_shard(M: int, world: int, rank: int):
    """(first_row, rows) of `rank` in the row-tile split of an M-row matrix over `world` ranks."""
    first, rows = ctypes.c_int64(0), ctypes.c_int64(0)
    _check(lib().spdp_row_shard(M, world, rank, ctypes.byref(first), ctypes.byref(rows)), "spdp_row_shard")
    return first.value, rows.value


def spdp_free(h) -> None:
    _check(lib().spdp_free(h), "spdp_free")


def spdp_get_info(h: int) -> spdp_info:
    info = spdp_info()
    _check(lib().spdp_get_info(h, ctypes.byref(info)), "spdp_get_info")
    return info


def spdp_export(h: int) -> dict:
    """The four packed arrays as NumPy arrays (synchronous device-to-host copies)."""
    info = spdp_get_info(h)
    to = np.empty(info.NGT + 1, np.uint32)
    ci = np.empty(info.NGT * 16, np.uint32)
    bm = np.empty(info.NGT * 64, np.uint64)
    va = np.empty(info.values_len, np.uint16)
    st = lib().spdp_export(h, to.ctypes.data, ci.ctypes.data, bm.ctypes.data, va.ctypes.data if va.size else None)
    _check(st, "spdp_export")
    return dict(M=info.M, K=info.K, pad_elems=info.pad_elems, tileoffset=to, colinfo=ci, bitmap=bm, values=va,
                nnz=info.nnz)


def spdp_unpack(h: int, W_out, stream=None) -> None:
    """W_out: fp16 CUDA tensor [M, K] with unit column stride (row stride = ldw)."""
    if not W_out.is_cuda or W_out.dim() != 2 or W_out.stride(1) != 1:
        raise ValueError("W_out must be a 2-D fp16 CUDA tensor with unit column stride")
    _check(lib().spdp_unpack(h, W_out.data_ptr(), W_out.stride(0), _stream(stream)), "spdp_unpack")


def spdp_active_columns(h: int, x, rule: int, thr: float, bitmask_out, count_out=None, mask=None, stream=None) -> None:
    st = lib().spdp_active_columns(h, _dev_ptr(x, "x"), rule, float(thr), _dev_ptr(mask, "mask", True),
                                   _dev_ptr(bitmask_out, "bitmask_out"), _dev_ptr(count_out, "count_out", True),
                                   _stream(stream))
    _check(st, "spdp_active_columns")


def spdp_last_device_status(h: int) -> int:
    v = ctypes.c_int(0)
    _check(lib().spdp_last_device_status(h, ctypes.byref(v)), "spdp_last_device_status")
    return v.value


def spdp_set_num_ctas(h: int, num_ctas: int) -> None:
    _check(lib().spdp_set_num_ctas(h, num_ctas), "spdp_set_num_ctas")


def spdp_probe_stream_read(h: int, stream=None) -> None:
    """Benchmark context: one contiguous read of the handle's Values array."""
    _check(lib().spdp_probe_stream_read(h, _stream(stream)), "spdp_probe_stream_read")


def spdp_probe_gather(h: int, x, rule: int, thr: float, mask=None, stream=None) -> None:
    """Benchmark context: fetch what spdp_spmspv would fetch for this x, with plain loads and no decode."""
    _check(lib().spdp_probe_gather(h, _dev_ptr(x, "x"), rule, float(thr), _dev_ptr(mask, "mask", True), _stream(stream)),
           "spdp_probe_gather")


def spdp_status_string(status: int) -> str:
    return lib().spdp_status_string(status).decode()
