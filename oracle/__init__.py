"""CPU oracle for the SpMM hot path.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; the product (the CUDA library and its binding) never
does, and this package imports nothing from the product.

* ``spmm_ref``      -- fp64 C = A x B straight from CSR (Sec. 2.3 problem
                       statement), implemented in plain C (spmm_ref.c).
* ``formats``       -- BCSR / WCSR / split-plan definitions (Sec. 2.3,
                       Sec. 3.3) written out with numpy.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spmm_ref.c")
_LIB = os.path.join(_HERE, "libspmm_ref.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile spmm_ref.c with gcc into a shared object next to it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.spmm_csr_ref.restype = None
        lib.spmm_csr_ref.argtypes = [
            ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_int64,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
        ]
        _lib = lib
    return _lib


def spmm_ref(row_ptr, col_idx, vals, B, rows=None, want_abs=True):
    """fp64 reference C = A x B and S = |A| x |B| from CSR (Sec. 2.3).

    row_ptr int64 [m+1], col_idx int32 [nnz], vals any float dtype [nnz]
    (widened exactly to float64 here), B [k, n] any float dtype (widened
    exactly).  ``rows=(r0, r1)`` restricts the computation to a row range;
    the returned arrays still have m rows and rows outside the range are 0.
    Returns (C, S) as float64 arrays of shape [m, n] (S is None when
    want_abs is False).  Single-threaded.
    """
    lib = _load()
    row_ptr = np.ascontiguousarray(row_ptr, dtype=np.int64)
    col_idx = np.ascontiguousarray(col_idx, dtype=np.int32)
    vals64 = np.ascontiguousarray(vals, dtype=np.float64)
    B64 = np.ascontiguousarray(B, dtype=np.float64)
    m = row_ptr.shape[0] - 1
    k, n = B64.shape
    if col_idx.size and (col_idx.min() < 0 or col_idx.max() >= k):
        raise ValueError("column index outside B")
    r0, r1 = (0, m) if rows is None else rows
    C = np.zeros((m, n), dtype=np.float64)
    S = np.zeros((m, n), dtype=np.float64) if want_abs else None
    lib.spmm_csr_ref(
        r0, r1, n,
        row_ptr.ctypes.data, col_idx.ctypes.data, vals64.ctypes.data,
        B64.ctypes.data, n,
        C.ctypes.data, S.ctypes.data if want_abs else None, n,
    )
    return C, S
