"""ctypes binding of the CPU oracle (``atb_oracle.cpp``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's ``cpu_baseline`` / reference
arm import this package.  It shares nothing with the CUDA library: it is built
from its own single C++ file with g++ and works on plain numpy arrays.

Logical layouts: ``mant[M][K]`` int8, ``exp[M][K/8]`` uint8 (both row-major),
``B[K][N]`` bf16 bit patterns as uint16.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "atb_oracle.cpp")
_LIB = os.path.join(_HERE, "libatb_oracle.so")
_lib = None


def _host_has_avx2() -> bool:
    try:
        with open("/proc/cpuinfo") as f:
            return " avx2 " in f.read().replace("\n", " ")
    except OSError:
        return False


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (OpenMP).  Returns the path of the library."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["g++", "-std=c++17", "-O3", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off"]
    if _host_has_avx2():
        cmd += ["-mavx2"]
    cmd += [_SRC, "-o", _LIB]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = ctypes.CDLL(_LIB)
    i64, vp = ctypes.c_int64, ctypes.c_void_p
    lib.oracle_num_threads.restype = ctypes.c_int
    lib.oracle_quantize_bfp16.restype = ctypes.c_int
    lib.oracle_quantize_bfp16.argtypes = [vp, i64, i64, i64, vp, vp]
    lib.oracle_dequantize_f64.restype = None
    lib.oracle_dequantize_f64.argtypes = [vp, vp, i64, i64, vp]
    lib.oracle_gemm_rows_f64.restype = None
    lib.oracle_gemm_rows_f64.argtypes = [i64, i64, vp, vp, vp, i64, vp, i64, vp, vp]
    lib.oracle_gemm_f64.restype = None
    lib.oracle_gemm_f64.argtypes = [i64, i64, i64, vp, vp, vp, i64, vp, vp]
    lib.oracle_check_tolerance.restype = i64
    lib.oracle_check_tolerance.argtypes = [vp, i64, vp, vp, i64, i64, vp]
    _lib = lib
    return lib


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def quantize_bfp16(A: np.ndarray):
    """fp32 ``A[M][K]`` -> (``mant`` int8 [M][K], ``exp`` uint8 [M][K/8])."""
    A = np.ascontiguousarray(A, dtype=np.float32)
    M, K = A.shape
    if K % 8:
        raise ValueError("K must be a multiple of 8")
    mant = np.empty((M, K), np.int8)
    exp = np.empty((M, K // 8), np.uint8)
    rc = _load().oracle_quantize_bfp16(_ptr(A), M, K, K, _ptr(mant), _ptr(exp))
    if rc:
        raise ValueError("oracle_quantize_bfp16 rejected the shape")
    return mant, exp


def dequantize(mant: np.ndarray, exp: np.ndarray) -> np.ndarray:
    """(mant, exp) -> FP64 values ``m * 2^(E-133)``."""
    mant = np.ascontiguousarray(mant, dtype=np.int8)
    exp = np.ascontiguousarray(exp, dtype=np.uint8)
    M, K = mant.shape
    assert exp.shape == (M, K // 8)
    out = np.empty((M, K), np.float64)
    _load().oracle_dequantize_f64(_ptr(mant), _ptr(exp), M, K, _ptr(out))
    return out


def gemm(mant: np.ndarray, exp: np.ndarray, B_bits: np.ndarray, rows=None):
    """FP64 ``C = dequant(A) @ B`` and ``S = sum_k |a b|``.

    ``rows`` (optional int64 index array) restricts the result to those rows of
    C, in the given order.  Returns ``(C, S)`` of shape ``[len(rows) or M][N]``.
    """
    mant = np.ascontiguousarray(mant, dtype=np.int8)
    exp = np.ascontiguousarray(exp, dtype=np.uint8)
    B_bits = np.ascontiguousarray(B_bits, dtype=np.uint16)
    M, K = mant.shape
    K2, N = B_bits.shape
    assert K2 == K and exp.shape == (M, K // 8)
    if rows is None:
        n_rows, rows_p = M, ctypes.c_void_p(0)
    else:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        assert rows.ndim == 1 and (rows.size == 0 or (rows.min() >= 0 and rows.max() < M))
        n_rows, rows_p = rows.size, _ptr(rows)
    C = np.empty((n_rows, N), np.float64)
    S = np.empty((n_rows, N), np.float64)
    _load().oracle_gemm_rows_f64(N, K, _ptr(mant), _ptr(exp), _ptr(B_bits), N, rows_p, n_rows,
                                 _ptr(C), _ptr(S))
    return C, S


def check_tolerance(C_gpu_bits: np.ndarray, C_ref: np.ndarray, S: np.ndarray):
    """Per-element test ``|C_gpu - C_ref| <= 2^-7 |C_ref| + 2^-12 S``.

    ``C_gpu_bits``: bf16 bit patterns (uint16) with the same shape as ``C_ref``.
    Returns ``(n_failing, max_error_over_bound)``.
    """
    C_gpu_bits = np.ascontiguousarray(C_gpu_bits, dtype=np.uint16)
    C_ref = np.ascontiguousarray(C_ref, dtype=np.float64)
    S = np.ascontiguousarray(S, dtype=np.float64)
    assert C_gpu_bits.shape == C_ref.shape == S.shape
    n_rows, N = C_ref.shape
    worst = ctypes.c_double(0.0)
    bad = _load().oracle_check_tolerance(_ptr(C_gpu_bits), N, _ptr(C_ref), _ptr(S), n_rows, N,
                                         ctypes.byref(worst))
    return int(bad), float(worst.value)
