"""ctypes front end of the C oracle (oracle/spdp_oracle.c) and its build step.

TEST INFRASTRUCTURE ONLY: for the test-suite, the smoke check and the benchmark's CPU-baseline
leg.  Nothing here touches the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spdp_oracle.c")
_LIB = os.path.join(_HERE, "libspdp_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile spdp_oracle.c with gcc -O2 -fopenmp into oracle/libspdp_oracle.so."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, p = ctypes.c_int64, ctypes.c_void_p
        L.oracle_half_to_double.restype = ctypes.c_double
        L.oracle_half_to_double.argtypes = [ctypes.c_uint16]
        L.oracle_pack.restype = i64
        L.oracle_pack.argtypes = [p, i64, i64, i64, i64, p, p, p, p]
        L.oracle_unpack.restype = None
        L.oracle_unpack.argtypes = [i64, i64, p, p, p, p, p, i64]
        L.oracle_active.restype = i64
        L.oracle_active.argtypes = [p, i64, ctypes.c_int, ctypes.c_float, p, p]
        L.oracle_spmspv.restype = ctypes.c_int
        L.oracle_spmspv.argtypes = [p, i64, i64, i64, p, p, p, p, ctypes.c_int]
        L.oracle_active_bytes.restype = i64
        L.oracle_active_bytes.argtypes = [i64, i64, i64, p, p, i64]
        L.oracle_max_threads.restype = ctypes.c_int
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _bits(a):
    a = np.ascontiguousarray(a)
    return a.view(np.uint16) if a.dtype == np.float16 else a


def half_to_double(h: int) -> float:
    return lib().oracle_half_to_double(int(h))


def pack(W, pad_elems: int = 8) -> dict:
    Wb = _bits(W)
    assert Wb.dtype == np.uint16 and Wb.ndim == 2
    M, K = Wb.shape
    R, C = (M + 255) // 256, (K + 15) // 16
    NGT = R * C
    to = np.zeros(NGT + 1, np.uint32)
    ci = np.zeros(NGT * 16, np.uint32)
    bm = np.zeros(NGT * 64, np.uint64)
    n = lib().oracle_pack(_ptr(Wb), M, K, K, pad_elems, _ptr(to), _ptr(ci), _ptr(bm), None)
    if n < 0:
        raise OverflowError("TileOffset does not fit 32 bits")
    vals = np.zeros(n, np.uint16)
    lib().oracle_pack(_ptr(Wb), M, K, K, pad_elems, _ptr(to), _ptr(ci), _ptr(bm), _ptr(vals))
    nnz = int((ci & np.uint32(0xFFFF)).astype(np.int64).sum())
    return dict(M=M, K=K, pad_elems=pad_elems, tileoffset=to, colinfo=ci, bitmap=bm, values=vals, nnz=nnz)


def unpack(p: dict) -> np.ndarray:
    W = np.empty((p["M"], p["K"]), np.uint16)
    lib().oracle_unpack(p["M"], p["K"], _ptr(p["tileoffset"]), _ptr(p["colinfo"]), _ptr(p["bitmap"]),
                        _ptr(p["values"]), _ptr(W), p["K"])
    return W


def active(x, rule: int, thr: float = 0.0, mask_words=None) -> np.ndarray:
    xb = _bits(x)
    a = np.zeros(xb.shape[0], np.uint8)
    mw = None if mask_words is None else np.ascontiguousarray(mask_words, dtype=np.uint32)
    lib().oracle_active(_ptr(xb), xb.shape[0], rule, float(np.float32(thr)), _ptr(mw), _ptr(a))
    return a.astype(bool)


def spmspv(W, x, active_mask, threads: int = 0, want_scale: bool = True):
    """Returns (y, S, threads_used); S is None when want_scale is False."""
    Wb, xb = _bits(W), _bits(x)
    M, K = Wb.shape
    a = np.ascontiguousarray(np.asarray(active_mask, dtype=np.uint8))
    y = np.empty(M, np.float64)
    S = np.empty(M, np.float64) if want_scale else None
    used = lib().oracle_spmspv(_ptr(Wb), M, K, K, _ptr(xb), _ptr(a), _ptr(y), _ptr(S), threads)
    return y, S, used


def active_bytes(p: dict, active_mask, y_bytes_per_elem: int = 2) -> int:
    a = np.ascontiguousarray(np.asarray(active_mask, dtype=np.uint8))
    return int(lib().oracle_active_bytes(p["M"], p["K"], p["pad_elems"], _ptr(p["colinfo"]), _ptr(a),
                                         y_bytes_per_elem))


def max_threads() -> int:
    return int(lib().oracle_max_threads())


if __name__ == "__main__":
    print(build(force=True))
