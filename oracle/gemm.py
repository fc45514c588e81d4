"""ctypes front end of ``gemm_oracle.c`` -- TEST INFRASTRUCTURE ONLY.

The C file is the oracle; this module only compiles it (gcc, OpenMP) and
marshals numpy arrays.  Inputs and outputs are raw 16-bit words (``uint16``)
so that both sides of a parity test see the same bits.

Definition implemented (paper Section 4.1 and the paragraph around Eq. 2):
``C64[i][j] = sum_k double(A[i][k]) * double(B[k][j])`` in ascending k, and
``C16 = RN-even_16(C64)`` rounded once, directly from binary64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

F16 = 0
BF16 = 1
ROW_MAJOR = 0
COL_MAJOR = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gemm_oracle.c")
_LIB = os.path.join(_HERE, "build", "libgemm_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".{os.getpid()}.tmp"
    cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fno-fast-math", "-ffp-contract=off",
           "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is not None:
            return _lib
        lib = ctypes.CDLL(build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        f64p = ctypes.POINTER(ctypes.c_double)
        i64p = ctypes.POINTER(ctypes.c_int64)
        lib.oracle_gemm_rows.restype = ctypes.c_int
        lib.oracle_gemm_rows.argtypes = [ctypes.c_int64] * 3 + [ctypes.c_int] * 3 + [
            u16p, u16p, i64p, ctypes.c_int64, f64p, u16p, ctypes.c_int]
        lib.oracle_addmm_rows.restype = ctypes.c_int
        lib.oracle_addmm_rows.argtypes = [ctypes.c_int64] * 3 + [ctypes.c_int] * 3 + [
            u16p, u16p, u16p, ctypes.c_int, ctypes.c_double, ctypes.c_double, i64p, ctypes.c_int64, f64p, u16p, ctypes.c_int]
        lib.oracle_decode16_array.argtypes = [u16p, f64p, ctypes.c_size_t, ctypes.c_int]
        lib.oracle_encode16_array.argtypes = [f64p, u16p, ctypes.c_size_t, ctypes.c_int]
        lib.oracle_fro_accumulate.argtypes = [u16p, f64p, ctypes.c_size_t, ctypes.c_int,
                                              f64p, f64p, i64p]
        lib.oracle_max_threads.restype = ctypes.c_int
        _lib = lib
        return lib


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("oracle inputs are raw 16-bit words (uint16)")
    return a


def _ptr(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def decode16(bits, dtype: int) -> np.ndarray:
    """Exact value of each 16-bit word as float64."""
    b = _u16(bits)
    out = np.empty(b.shape, dtype=np.float64)
    _load().oracle_decode16_array(_ptr(b, ctypes.c_uint16), _ptr(out, ctypes.c_double), b.size, dtype)
    return out


def encode16(x, dtype: int) -> np.ndarray:
    """Round float64 values once, to nearest even, to the 16-bit type."""
    v = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.uint16)
    _load().oracle_encode16_array(_ptr(v, ctypes.c_double), _ptr(out, ctypes.c_uint16), v.size, dtype)
    return out


def gemm_rows(A_bits, B_bits, M: int, N: int, K: int, dtype: int,
              layoutA: int = ROW_MAJOR, layoutB: int = ROW_MAJOR,
              rows=None, want16: bool = True, nthreads: int = 0):
    """Rows ``rows`` (default: all) of C = A*B.  Returns (C64, C16-or-None)."""
    A = _u16(A_bits).reshape(-1)
    B = _u16(B_bits).reshape(-1)
    if A.size != M * K or B.size != K * N:
        raise ValueError("operand size does not match (M, N, K)")
    if rows is None:
        rows_arr = None
        nrows = M
    else:
        rows_arr = np.ascontiguousarray(rows, dtype=np.int64)
        nrows = rows_arr.size
    C64 = np.zeros((nrows, N), dtype=np.float64)
    C16 = np.zeros((nrows, N), dtype=np.uint16) if want16 else None
    rc = _load().oracle_gemm_rows(
        M, N, K, dtype, layoutA, layoutB,
        _ptr(A, ctypes.c_uint16), _ptr(B, ctypes.c_uint16),
        _ptr(rows_arr, ctypes.c_int64) if rows_arr is not None else None, nrows,
        _ptr(C64, ctypes.c_double),
        _ptr(C16, ctypes.c_uint16) if C16 is not None else None, nthreads)
    if rc != 0:
        raise ValueError("oracle_gemm_rows rejected its arguments")
    return C64, C16


def gemm(A_bits, B_bits, M, N, K, dtype, layoutA=ROW_MAJOR, layoutB=ROW_MAJOR, nthreads=0):
    """Whole product.  Returns (C64, C16)."""
    return gemm_rows(A_bits, B_bits, M, N, K, dtype, layoutA, layoutB, None, True, nthreads)


def addmm_rows(A_bits, B_bits, D_bits, M: int, N: int, K: int, dtype: int, alpha: float, beta: float,
               layoutA: int = ROW_MAJOR, layoutB: int = ROW_MAJOR, rows=None, nthreads: int = 0):
    """Rows ``rows`` (default: all) of alpha * (A*B) + beta * D (Section 6.5's AddMM operator), D either M x N
    or a row of N values (a bias, recognised by its size).  alpha and beta are taken at their binary32 values.
    Returns (O64, O16)."""
    A = _u16(A_bits).reshape(-1)
    B = _u16(B_bits).reshape(-1)
    D = _u16(D_bits).reshape(-1)
    if A.size != M * K or B.size != K * N or D.size not in (N, M * N):
        raise ValueError("operand size does not match (M, N, K)")
    is_vec = 1 if D.size == N else 0      # with M == 1 the two readings coincide
    if rows is None:
        rows_arr, nrows = None, M
    else:
        rows_arr = np.ascontiguousarray(rows, dtype=np.int64)
        nrows = rows_arr.size
    O64 = np.zeros((nrows, N), dtype=np.float64)
    O16 = np.zeros((nrows, N), dtype=np.uint16)
    rc = _load().oracle_addmm_rows(
        M, N, K, dtype, layoutA, layoutB, _ptr(A, ctypes.c_uint16), _ptr(B, ctypes.c_uint16), _ptr(D, ctypes.c_uint16), is_vec,
        float(np.float32(alpha)), float(np.float32(beta)),
        _ptr(rows_arr, ctypes.c_int64) if rows_arr is not None else None, nrows,
        _ptr(O64, ctypes.c_double), _ptr(O16, ctypes.c_uint16), nthreads)
    if rc != 0:
        raise ValueError("oracle_addmm_rows rejected its arguments")
    return O64, O16


def rel_fro_error(C_got_bits, C_ref64, dtype: int):
    """(||C_got - C_ref||_F / ||C_ref||_F, count of non-finite differences), norms in fp64."""
    g = _u16(C_got_bits).reshape(-1)
    r = np.ascontiguousarray(C_ref64, dtype=np.float64).reshape(-1)
    if g.size != r.size:
        raise ValueError("size mismatch")
    num = ctypes.c_double(0.0)
    den = ctypes.c_double(0.0)
    bad = ctypes.c_int64(0)
    _load().oracle_fro_accumulate(_ptr(g, ctypes.c_uint16), _ptr(r, ctypes.c_double), g.size, dtype,
                                  ctypes.byref(num), ctypes.byref(den), ctypes.byref(bad))
    if den.value == 0.0:
        return (0.0 if num.value == 0.0 else float("inf")), int(bad.value)
    return float(np.sqrt(num.value / den.value)), int(bad.value)
