"""Python face of the CPU oracle (``oracle_gemm.c``).

TEST INFRASTRUCTURE ONLY.  Only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may import this module; the product package
never does, and this module never imports the product package.

The oracle is the plain definition of the matrix product with exact bf16
products and fp64 accumulation in ascending k (see the header of
``oracle_gemm.c``).  The paper's GEMM workload (Evaluation, Table 2: GEMM,
BF16) fixes neither tolerance nor layouts; the acceptance bound used with
this oracle is

    |C - C_ref|_ij <= K * 2^-23 * S_ij ,   S = |A| . |B|

for fp32 outputs (standard running-error bound with unit roundoff 2^-23),
bit equality on small-integer inputs, and for bf16 outputs the same bound
widened by one bf16 rounding (unit roundoff 2^-8).

Pins (see tests/test_oracle_pins.py): exact rational brute force on tiny
shapes, identity and permutation matrices, the rank-1 closed form, int64
matmul on integer inputs, a hand-worked example, fp64 library matmul, layout
and leading-dimension invariance.  No function here is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "oracle_gemm.c"
_LIB = _HERE / "liboracle_gemm.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (OpenMP over rows, no fast-math)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        cmd = ["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off",
               "-shared", "-fPIC", "-o", str(_LIB), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        i64, p = ctypes.c_int64, ctypes.c_void_p
        lib.oracle_gemm_bf16.restype = ctypes.c_int
        lib.oracle_gemm_bf16.argtypes = [i64, i64, i64, p, i64, p, i64, ctypes.c_int,
                                         p, p, i64, i64, i64, ctypes.c_int]
        lib.oracle_round_to_bf16_array.restype = None
        lib.oracle_round_to_bf16_array.argtypes = [p, p, i64]
        _lib = lib
    return _lib


def _as_bits(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x)
    if x.dtype != np.uint16:
        raise TypeError("bf16 operands are passed as uint16 bit patterns")
    return x


def gemm(M: int, N: int, K: int, A_bits: np.ndarray, lda: int, B_bits: np.ndarray, ldb: int,
         b_col_major: bool = False, rows=None, want_S: bool = True, nthreads: int = 0):
    """C_ref (fp64) and S = |A|.|B| (fp64), each of shape (M, N).

    ``A_bits`` / ``B_bits`` are flat (or any-shape, C-contiguous) uint16 buffers
    holding bf16 bit patterns laid out with leading dimensions ``lda`` / ``ldb``
    in elements.  ``rows`` = (row_begin, row_end) restricts the computed rows;
    other rows of the returned arrays are NaN so that a stray read shows.
    """
    lib = _load()
    A_bits, B_bits = _as_bits(A_bits), _as_bits(B_bits)
    if K > 0 and M > 0 and N > 0:
        need_a = (M - 1) * lda + K
        need_b = ((N - 1) * ldb + K) if b_col_major else ((K - 1) * ldb + N)
        if A_bits.size < need_a or B_bits.size < need_b:
            raise ValueError("operand buffer smaller than its leading dimension implies")
    r0, r1 = (0, M) if rows is None else rows
    C = np.full((M, N), np.nan, dtype=np.float64)
    S = np.full((M, N), np.nan, dtype=np.float64) if want_S else None
    rc = lib.oracle_gemm_bf16(M, N, K, A_bits.ctypes.data, lda, B_bits.ctypes.data, ldb,
                              1 if b_col_major else 0, C.ctypes.data,
                              S.ctypes.data if want_S else None, N, r0, r1, nthreads)
    if rc != 0:
        raise ValueError(f"oracle_gemm_bf16 rejected its arguments (rc={rc})")
    return C, S


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp64 -> fp32 -> bf16 bit patterns, round-to-nearest-even (uint16)."""
    lib = _load()
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.uint16)
    lib.oracle_round_to_bf16_array(x.ctypes.data, out.ctypes.data, x.size)
    return out


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact decode of bf16 bit patterns (uint16) to fp64."""
    w = bits.astype(np.uint32) << np.uint32(16)
    return w.view(np.float32).astype(np.float64)


def bound_f32(K: int, S: np.ndarray) -> np.ndarray:
    """Elementwise acceptance bound for an fp32 result: K * 2^-23 * S."""
    return float(K) * 2.0 ** -23 * S


def bound_bf16(K: int, S: np.ndarray, C_ref: np.ndarray) -> np.ndarray:
    """Bound for a bf16 result: the fp32 bound plus one bf16 rounding (2^-8 relative)."""
    tol = bound_f32(K, S)
    return tol + 2.0 ** -8 * (np.abs(C_ref) + tol)


def host_threads() -> int:
    return len(os.sched_getaffinity(0))
