"""ctypes access to the plain-C fp64 oracle (harp_oracle.c) -- TEST INFRASTRUCTURE.

Builds ``libharp_oracle.so`` next to the source with gcc on first use.  Used where
the numpy oracle is too slow: sampled rows of the full-size configurations and
the benchmark's timed CPU baseline.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "harp_oracle.c")
_LIB = os.path.join(_HERE, "libharp_oracle.so")
_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", _LIB, _SRC])
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.harp_oracle_apply.restype = ctypes.c_int
        lib.harp_oracle_apply.argtypes = [
            ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int]
        lib.harp_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().harp_oracle_threads())


class CPlan:
    """Flat fp64 arrays of one processor, laid out for harp_oracle_apply."""

    def __init__(self, spec):
        self.d = int(spec.d)
        self.radices = np.asarray(spec.radices, dtype=np.int32)
        self.perm = None if spec.perm is None else np.ascontiguousarray(spec.perm, dtype=np.int64)
        self.signs = None if spec.signs is None else np.ascontiguousarray(spec.signs, dtype=np.float64)
        self.blocks = np.concatenate([np.asarray(k, dtype=np.float64).ravel() for k in spec.blocks])


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def apply(plan: CPlan, x: np.ndarray, transposed: bool = False) -> np.ndarray:
    """Returns forward (or transpose) of the rows x[B, d]; x is not modified."""
    y = np.array(x, dtype=np.float64, ndmin=2, order="C", copy=True)
    assert y.shape[1] == plan.d
    rc = _load().harp_oracle_apply(plan.d, len(plan.radices), _ptr(plan.radices), _ptr(plan.perm),
                                   _ptr(plan.signs), _ptr(plan.blocks), _ptr(y), y.shape[0],
                                   1 if transposed else 0)
    if rc != 0:
        raise MemoryError("harp_oracle_apply failed")
    return y


def forward(plan: CPlan, x: np.ndarray) -> np.ndarray:
    return apply(plan, x, False)


def transpose(plan: CPlan, y: np.ndarray) -> np.ndarray:
    return apply(plan, y, True)


def two_sided(plan_out: CPlan, plan_in: CPlan, w: np.ndarray) -> np.ndarray:
    """W~ = Q_out^T W Q_in: rows through Q_in, then columns through Q_out."""
    r = apply(plan_in, w, False)
    return np.ascontiguousarray(apply(plan_out, np.ascontiguousarray(r.T), False).T)
