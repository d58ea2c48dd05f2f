"""ctypes access to the plain-C oracle (slim_oracle.c).  Test infrastructure only."""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "slim_oracle.c")
_LIB = os.path.join(_HERE, "libslim_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile slim_oracle.c with gcc (OpenMP over output rows) into this folder."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True, capture_output=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        L.slim_oracle_packed_bytes.restype = ctypes.c_size_t
        L.slim_oracle_packed_bytes.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
        for name in ("slim_oracle_pack", "slim_oracle_unpack"):
            getattr(L, name).restype = ctypes.c_int
            getattr(L, name).argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int]
        L.slim_oracle_dequant_f16.restype = None
        L.slim_oracle_dequant_f16.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int] * 2
        L.slim_oracle_linear_f64.restype = ctypes.c_int
        L.slim_oracle_linear_f64.argtypes = [ctypes.c_void_p] * 5 + [ctypes.c_int] * 4
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def packed_bytes(N, K, bits) -> int:
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    return int(lib().slim_oracle_packed_bytes(N, K, _p(bits)))


def pack(codes, bits) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    N, K = codes.shape
    out = np.empty(packed_bytes(N, K, bits), dtype=np.uint8)
    rc = lib().slim_oracle_pack(_p(codes), _p(bits), _p(out), N, K)
    if rc:
        raise ValueError(f"slim_oracle_pack failed: {rc}")
    return out


def unpack(packed, N, K, bits) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    codes = np.empty((N, K), dtype=np.uint8)
    rc = lib().slim_oracle_unpack(_p(packed), _p(bits), _p(codes), N, K)
    if rc:
        raise ValueError(f"slim_oracle_unpack failed: {rc}")
    return codes


def dequant_f16(codes, scales, zeros) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.float16)
    zeros = np.ascontiguousarray(zeros, dtype=np.float16)
    N, K = codes.shape
    W = np.empty((N, K), dtype=np.float16)
    lib().slim_oracle_dequant_f16(_p(codes), _p(scales), _p(zeros), _p(W), N, K)
    return W


def linear_f64(x16, codes, scales, zeros, threads: int = 0):
    """Returns (y fp64 [M][N], threads used)."""
    x16 = np.ascontiguousarray(x16, dtype=np.float16)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.float16)
    zeros = np.ascontiguousarray(zeros, dtype=np.float16)
    M, K = x16.shape
    N = codes.shape[0]
    y = np.empty((M, N), dtype=np.float64)
    used = lib().slim_oracle_linear_f64(_p(x16), _p(codes), _p(scales), _p(zeros), _p(y), M, N, K, threads)
    return y, int(used)
