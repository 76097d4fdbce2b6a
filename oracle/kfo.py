"""ctypes front end of the fp64 CPU oracle (``oracle/kfo.c``).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the bench's CPU-baseline / reference legs
may import this module; the product package never does, and this module never imports the
product package.  It compiles ``kfo.c`` with gcc on first use (``-O2 -fopenmp``, no fast-math)
and passes numpy arrays through unchanged: float32 arrays as fp32, uint16 arrays as bf16 bit
patterns, float64 arrays as fp64.  Results are float64 arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "kfo.c"
_LIB = _HERE / "libkfo.so"

ACT = {"none": 0, "gelu_erf": 1, "gelu_tanh": 2, "silu": 3, "relu": 4, "sigmoid": 5}
NORM = {"none": 0, "softmax": 1, "layernorm": 2, "rmsnorm": 3}

_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle's C source into ``libkfo.so`` next to it (no-op when up to date)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=gnu11", "-o", str(tmp), str(_SRC), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        c_long, c_int, c_float, vp = ctypes.c_long, ctypes.c_int, ctypes.c_float, ctypes.c_void_p
        lib.kfo_linear_epilogue_rownorm.restype = c_int
        lib.kfo_linear_epilogue_rownorm.argtypes = [
            vp, c_long, vp, c_long, vp, c_int, c_float, vp, c_long, c_int, vp, vp, c_float,
            vp, c_long, c_long, c_long, c_long, c_int]
        lib.kfo_row_norm.restype = c_int
        lib.kfo_row_norm.argtypes = [vp, c_long, c_int, vp, vp, c_float, vp, c_long, c_long, c_long, c_int]
        lib.kfo_act.restype = ctypes.c_double
        lib.kfo_act.argtypes = [c_int, ctypes.c_double]
        lib.kfo_threads.restype = c_int
        lib.kfo_threads.argtypes = []
        _lib = lib
    return _lib


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return 0
    if a.dtype == np.uint16:
        return 1
    if a.dtype == np.float64:
        return 2
    raise TypeError(f"oracle takes float32, uint16 (bf16 bits) or float64 arrays, got {a.dtype}")


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check2d(a: np.ndarray, name: str):
    if a.ndim != 2:
        raise ValueError(f"{name} must be 2-D")
    if a.shape[0] <= 1 or a.shape[1] == 0:
        if a.shape[0] == 1 and a.shape[1] > 1 and a.strides[1] != a.itemsize:
            raise ValueError(f"{name} must have unit inner stride")
        return max(a.shape[1], 1)
    if (a.shape[1] > 1 and a.strides[1] != a.itemsize) or a.strides[0] % a.itemsize:
        raise ValueError(f"{name} must be 2-D with unit inner stride")
    return a.strides[0] // a.itemsize


def threads() -> int:
    """Host threads OpenMP will use for the row loop."""
    return int(_load().kfo_threads())


def act(name: str, z: float) -> float:
    """The activation alone, in double."""
    return float(_load().kfo_act(ACT[name], float(z)))


def linear_epilogue_rownorm(X, W, bias=None, act="none", scale=1.0, residual=None, norm="none",
                            gamma=None, beta=None, eps=1e-5) -> np.ndarray:
    """Row op(act(X W^T + bias) * scale + residual) in double.  X [M,K], W [N,K]."""
    lib = _load()
    dt = _dtype_code(X)
    for name, arr in (("W", W), ("bias", bias), ("residual", residual), ("gamma", gamma), ("beta", beta)):
        if arr is not None and _dtype_code(arr) != dt:
            raise TypeError(f"{name} dtype differs from X")
    M, K = X.shape
    N, K2 = W.shape
    if K2 != K:
        raise ValueError("X and W disagree on K")
    ldx, ldw = _check2d(X, "X"), _check2d(W, "W")
    ldr = _check2d(residual, "residual") if residual is not None else 0
    if residual is not None and residual.shape != (M, N):
        raise ValueError("residual must be [M,N]")
    for name, arr in (("bias", bias), ("gamma", gamma), ("beta", beta)):
        if arr is not None and (arr.shape != (N,) or not arr.flags.c_contiguous):
            raise ValueError(f"{name} must be a contiguous [N] vector")
    Y = np.empty((M, N), dtype=np.float64)
    rc = lib.kfo_linear_epilogue_rownorm(
        _ptr(X), ldx, _ptr(W), ldw, _ptr(bias), ACT[act], float(scale), _ptr(residual), ldr,
        NORM[norm], _ptr(gamma), _ptr(beta), float(np.float32(eps)), _ptr(Y), max(N, 1), M, N, K, dt)
    if rc != 0:
        raise RuntimeError(f"oracle returned {rc}")
    return Y


def linear_epilogue(X, W, bias=None, act="none", scale=1.0, residual=None) -> np.ndarray:
    return linear_epilogue_rownorm(X, W, bias, act, scale, residual, "none")


def row_norm(X, norm, gamma=None, beta=None, eps=1e-5) -> np.ndarray:
    lib = _load()
    dt = _dtype_code(X)
    M, N = X.shape
    ldx = _check2d(X, "X")
    for name, arr in (("gamma", gamma), ("beta", beta)):
        if arr is not None and (_dtype_code(arr) != dt or arr.shape != (N,) or not arr.flags.c_contiguous):
            raise ValueError(f"{name} must be a contiguous [N] vector of X's dtype")
    Y = np.empty((M, N), dtype=np.float64)
    rc = lib.kfo_row_norm(_ptr(X), ldx, NORM[norm], _ptr(gamma), _ptr(beta), float(np.float32(eps)),
                          _ptr(Y), max(N, 1), M, N, dt)
    if rc != 0:
        raise RuntimeError(f"oracle returned {rc}")
    return Y


def row_softmax(X) -> np.ndarray:
    return row_norm(X, "softmax")


def row_layernorm(X, gamma=None, beta=None, eps=1e-5) -> np.ndarray:
    return row_norm(X, "layernorm", gamma, beta, eps)


def row_rmsnorm(X, gamma=None, eps=1e-5) -> np.ndarray:
    return row_norm(X, "rmsnorm", gamma, None, eps)
