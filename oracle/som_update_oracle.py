"""ctypes front end of the CPU update oracle (``som_update_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/`` to check the CUDA update path (Section 3.4 of
the paper: scatter onto the lattice, factorised box blur of numerator and denominator, divide).
It shares no code with the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "som_update_oracle.c")
_LIB = os.path.join(_HERE, "libsom_update_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        P, I64, INT = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        lib.som_oracle_blur.argtypes = [P, P, I64, I64, I64, INT]
        lib.som_oracle_blur.restype = None
        lib.som_oracle_update.argtypes = [P, I64, I64, I64, P, P, I64, P, I64, INT, P]
        lib.som_oracle_update.restype = INT
        _lib = lib
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def blur(field, rows: int, cols: int, radius: int, passes: int = 3) -> np.ndarray:
    """`passes` box passes per axis of half-width `radius`, unnormalised, truncated at the edge."""
    f = np.ascontiguousarray(field, dtype=np.float64).reshape(rows * cols).copy()
    tmp = np.empty(rows * cols, np.float64)
    _load().som_oracle_blur(_p(f), _p(tmp), rows, cols, radius, passes)
    return f.reshape(rows, cols)


def update(W_old, V: int, rows: int, cols: int, indptr, indices, bmu, radius: int, passes: int = 3) -> np.ndarray:
    """New feature-major codebook as fp64 [V*M] (unrounded)."""
    W_old = np.ascontiguousarray(W_old, dtype=np.float32).reshape(-1)
    M = rows * cols
    assert W_old.size == V * M
    indptr = np.ascontiguousarray(indptr, dtype=np.int32)
    indices = np.ascontiguousarray(indices, dtype=np.int32)
    bmu = np.ascontiguousarray(bmu, dtype=np.int32)
    n = indptr.size - 1
    assert bmu.size == n and (n == 0 or (bmu.min() >= 0 and bmu.max() < M))
    out = np.empty(V * M, np.float64)
    rc = _load().som_oracle_update(_p(W_old), V, rows, cols, _p(indptr), _p(indices), n, _p(bmu), radius,
                                   passes, _p(out))
    if rc != 0:
        raise MemoryError("update oracle: out of memory")
    return out
