"""ctypes front end of the CPU oracle (``som_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, the smoke check and the CPU-baseline /
reference legs of ``bench.py``.  The CUDA library and its Python binding never import it.

The oracle states Eq. 1 of the paper in fp64 and scans for the argmin with the
lowest-index tie rule of Section 3.1; see the header of ``som_oracle.c``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "som_oracle.c")
_LIB = os.path.join(_HERE, "libsom_oracle.so")

FEATURE_MAJOR = 0
NODE_MAJOR = 1

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        P = ctypes.c_void_p
        I64 = ctypes.c_int64
        lib.som_oracle_threads.restype = ctypes.c_int
        lib.som_oracle_norms.argtypes = [P, ctypes.c_int, I64, I64, P]
        lib.som_oracle_bmu.argtypes = [P, ctypes.c_int, I64, I64, P, P, P, I64, I64, ctypes.c_int,
                                       P, P, P, P]
        lib.som_oracle_dist_at.argtypes = [P, ctypes.c_int, I64, I64, P, P, P, I64, P, P]
        lib.som_oracle_all_distances.argtypes = [P, ctypes.c_int, I64, I64, P, P, P, I64, P]
        lib.som_oracle_bmu_values.argtypes = [P, ctypes.c_int, I64, I64, P, P, P, P, I64, P, P, P, P]
        lib.som_oracle_dist_at_values.argtypes = [P, ctypes.c_int, I64, I64, P, P, P, P, I64, P, P]
        for f in (lib.som_oracle_norms, lib.som_oracle_bmu, lib.som_oracle_dist_at,
                  lib.som_oracle_all_distances, lib.som_oracle_bmu_values, lib.som_oracle_dist_at_values):
            f.restype = None
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().som_oracle_threads())


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def norms(W, V: int, M: int, layout: int = FEATURE_MAJOR) -> np.ndarray:
    """fp64 squared norms of the M prototypes of a flat fp32 codebook."""
    W = _f32(W).reshape(-1)
    assert W.size == V * M
    out = np.empty(M, dtype=np.float64)
    _load().som_oracle_norms(_p(W), layout, V, M, _p(out))
    return out


@dataclass
class Top2:
    b1: np.ndarray  # int64 [n] best unit
    d1: np.ndarray  # float64 [n] its squared distance
    b2: np.ndarray  # int64 [n] second-best unit (-1 if M == 1)
    d2: np.ndarray  # float64 [n]


def bmu(W, V: int, M: int, indptr, indices, layout: int = FEATURE_MAJOR, norms_=None,
        m_offset: int = 0, running: Top2 | None = None) -> Top2:
    """Best and second-best unit per sample over this codebook (or codebook slab).

    ``running`` merges the slab into an earlier result (slabs in ascending neuron order).
    """
    W = _f32(W).reshape(-1)
    assert W.size == V * M
    indptr = _i32(indptr)
    indices = _i32(indices)
    n = indptr.size - 1
    if norms_ is None:
        norms_ = norms(W, V, M, layout)
    norms_ = np.ascontiguousarray(norms_, dtype=np.float64)
    if running is None:
        out = Top2(np.empty(n, np.int64), np.empty(n, np.float64),
                   np.empty(n, np.int64), np.empty(n, np.float64))
        merge = 0
    else:
        out = running
        merge = 1
    _load().som_oracle_bmu(_p(W), layout, V, M, _p(norms_), _p(indptr), _p(indices), n,
                           m_offset, merge, _p(out.b1), _p(out.d1), _p(out.b2), _p(out.d2))
    return out


def bmu_values(W, V: int, M: int, indptr, indices, values, layout: int = FEATURE_MAJOR, norms_=None) -> Top2:
    """Best and second-best unit per sparse real-valued sample (``values`` parallel to ``indices``)."""
    W = _f32(W).reshape(-1)
    assert W.size == V * M
    indptr, indices, values = _i32(indptr), _i32(indices), _f32(values)
    assert values.size == indices.size
    n = indptr.size - 1
    if norms_ is None:
        norms_ = norms(W, V, M, layout)
    norms_ = np.ascontiguousarray(norms_, dtype=np.float64)
    out = Top2(np.empty(n, np.int64), np.empty(n, np.float64), np.empty(n, np.int64), np.empty(n, np.float64))
    _load().som_oracle_bmu_values(_p(W), layout, V, M, _p(norms_), _p(indptr), _p(indices), _p(values), n,
                                  _p(out.b1), _p(out.d1), _p(out.b2), _p(out.d2))
    return out


def dist_at_values(W, V: int, M: int, indptr, indices, values, neuron, layout: int = FEATURE_MAJOR,
                   norms_=None) -> np.ndarray:
    """fp64 squared distance of real-valued sample n to neuron[n]."""
    W = _f32(W).reshape(-1)
    indptr, indices, values = _i32(indptr), _i32(indices), _f32(values)
    n = indptr.size - 1
    neuron = np.ascontiguousarray(neuron, dtype=np.int64)
    if norms_ is None:
        norms_ = norms(W, V, M, layout)
    norms_ = np.ascontiguousarray(norms_, dtype=np.float64)
    out = np.empty(n, np.float64)
    _load().som_oracle_dist_at_values(_p(W), layout, V, M, _p(norms_), _p(indptr), _p(indices), _p(values), n,
                                      _p(neuron), _p(out))
    return out


def dist_at(W, V: int, M: int, indptr, indices, neuron, layout: int = FEATURE_MAJOR,
            norms_=None) -> np.ndarray:
    """fp64 squared distance of sample n to neuron[n]."""
    W = _f32(W).reshape(-1)
    indptr = _i32(indptr)
    indices = _i32(indices)
    n = indptr.size - 1
    neuron = np.ascontiguousarray(neuron, dtype=np.int64)
    assert neuron.size == n
    if norms_ is None:
        norms_ = norms(W, V, M, layout)
    norms_ = np.ascontiguousarray(norms_, dtype=np.float64)
    out = np.empty(n, np.float64)
    _load().som_oracle_dist_at(_p(W), layout, V, M, _p(norms_), _p(indptr), _p(indices), n,
                               _p(neuron), _p(out))
    return out


def all_distances(W, V: int, M: int, indptr, indices, layout: int = FEATURE_MAJOR) -> np.ndarray:
    """Full [n, M] fp64 distance matrix; tiny inputs only."""
    W = _f32(W).reshape(-1)
    indptr = _i32(indptr)
    indices = _i32(indices)
    n = indptr.size - 1
    nn = norms(W, V, M, layout)
    out = np.empty((n, M), np.float64)
    _load().som_oracle_all_distances(_p(W), layout, V, M, _p(nn), _p(indptr), _p(indices), n, _p(out))
    return out
