"""CPU oracle for the FluxBin decode linear layer (test infrastructure only).

Thin ctypes wrapper over oracle/fluxbin_oracle.c (plain fp64 C, compiled with gcc on first
use) plus the paper's analytic cost models in oracle/models.py.  Nothing here is part of the
product path and nothing here imports the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "fluxbin_oracle.c")
_LIB = os.path.join(_DIR, "_build", "libfluxbin_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc -O2 -fopenmp; returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        os.makedirs(os.path.dirname(_LIB), exist_ok=True)
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.fbo_half_to_double.restype = ctypes.c_double
        _lib.fbo_half_to_double.argtypes = [ctypes.c_uint16]
        _lib.fbo_num_threads.restype = ctypes.c_int
    return _lib


def _p(a):
    return None if a is None or a.size == 0 else a.ctypes.data_as(ctypes.c_void_p)


def _layer_args(L):
    keep = [np.ascontiguousarray(a) for a in (L.bits, L.row_scale, L.col_scale, L.sal_idx, L.sal_bits,
                                              L.sal_row_scale, L.sal_col_scale)]
    assert keep[0].dtype == np.uint32 and keep[1].dtype == np.uint16 and keep[3].dtype == np.int32
    args = [ctypes.c_int(L.M), ctypes.c_int(L.N), ctypes.c_int(L.Kb), ctypes.c_int(L.Ks), ctypes.c_int(L.g),
            ctypes.c_int(L.n_sal)]
    return args, [_p(a) for a in keep], keep


def num_threads() -> int:
    return int(_load().fbo_num_threads())


def half_to_double(h: int) -> float:
    return float(_load().fbo_half_to_double(ctypes.c_uint16(h)))


def dense_weight(L) -> np.ndarray:
    """What[M][N] in fp64 by brute force."""
    lib = _load()
    W = np.empty((L.M, L.N), np.float64)
    args, ptrs, keep = _layer_args(L)
    lib.fbo_dense_weight(*args, *ptrs, _p(W))
    return W


def dense_linear(L, x: np.ndarray) -> np.ndarray:
    """y[B][M] via the materialised matrix (brute force; tiny shapes)."""
    lib = _load()
    x = np.ascontiguousarray(x, dtype=np.uint16)
    B = x.shape[0]
    W = dense_weight(L)
    y = np.empty((B, L.M), np.float64)
    lib.fbo_dense_linear(ctypes.c_int(L.M), ctypes.c_int(L.N), ctypes.c_int(B), _p(W), _p(x),
                         ctypes.c_int64(x.shape[1]), _p(y))
    return y


def linear_direct(L, x: np.ndarray) -> np.ndarray:
    """THE oracle: y[B][M] in fp64, direct sum over bases (x: uint16 fp16 bit patterns [B][>=N])."""
    lib = _load()
    x = np.ascontiguousarray(x, dtype=np.uint16)
    B = x.shape[0]
    y = np.empty((B, L.M), np.float64)
    args, ptrs, keep = _layer_args(L)
    lib.fbo_linear_direct(*args, *ptrs, _p(x), ctypes.c_int(B), ctypes.c_int64(x.shape[1]), _p(y))
    return y


def lut_tables(a: np.ndarray, mu: int) -> np.ndarray:
    """Eq. 14 tables [len(a)/mu][2^mu] for fused activations a (fp64)."""
    lib = _load()
    a = np.ascontiguousarray(a, dtype=np.float64)
    assert a.size % mu == 0
    t = np.empty((a.size // mu, 1 << mu), np.float64)
    lib.fbo_lut_tables(ctypes.c_int(a.size), ctypes.c_int(mu), _p(a), _p(t))
    return t


def lut_linear(L, x: np.ndarray, mu: int = 8) -> np.ndarray:
    """y[B][M] the LUT way in fp64 (Eq. 11, 13-15)."""
    lib = _load()
    assert L.g % mu == 0
    x = np.ascontiguousarray(x, dtype=np.uint16)
    B = x.shape[0]
    y = np.empty((B, L.M), np.float64)
    args, ptrs, keep = _layer_args(L)
    lib.fbo_lut_linear(*args, ctypes.c_int(mu), *ptrs, _p(x), ctypes.c_int(B), ctypes.c_int64(x.shape[1]), _p(y))
    return y
