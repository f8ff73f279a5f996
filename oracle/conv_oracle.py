"""Python face of the Conv2d CPU oracle (``oracle_conv.c``).

TEST INFRASTRUCTURE ONLY: only the test-suite and the smoke check import this module; the product
package never does, and this module never imports the product package.

The oracle is the plain definition of the channels-last 2-D cross-correlation with zero padding
(paper, Evaluation, Table 2: Conv2d N=8, C=64, 56x56, F=128, 3x3, FP16), fp16 operands decoded exactly to
fp64, fp64 products and sums in ascending (r, s, c).  The paper prints neither layout, padding, stride nor
a tolerance for it; the readings (channels-last, "same" padding 1, stride 1 for the benchmark shape; any
padding and stride in the interface) and the acceptance bound

    |y - y_ref| <= K * 2^-23 * S ,   K = R*S*C,  S = sum |x| |w|       (fp32 output)
    the same widened by one fp16 rounding, 2^-11 * (|y_ref| + tol)      (fp16 output)

mirror those of the GEMM oracle.  Pins (tests/test_oracle_pins.py): torch's fp64 conv2d, the fp64 matrix
product for 1x1 filters, a shifted-delta filter (index order of r, s and of the padding), all-ones operands
(the count of in-range taps), exact rational brute force on tiny shapes, a hand-worked example.
No function here is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "oracle_conv.c"
_LIB = _HERE / "liboracle_conv.so"
_lib = None


def build(force: bool = False) -> Path:
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        cmd = ["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC", "-o", str(_LIB),
               str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        i64, p = ctypes.c_int64, ctypes.c_void_p
        lib.oracle_conv2d.restype = ctypes.c_int
        lib.oracle_conv2d.argtypes = [i64] * 11 + [p, p, p, p, ctypes.c_int]
        _lib = lib
    return _lib


def out_size(H: int, W: int, R: int, S: int, pad, stride):
    return (H + 2 * pad[0] - R) // stride[0] + 1, (W + 2 * pad[1] - S) // stride[1] + 1


def f16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact decode of fp16 bit patterns (uint16) to fp64."""
    return np.ascontiguousarray(bits, dtype=np.uint16).view(np.float16).astype(np.float64)


def round_to_f16(y: np.ndarray) -> np.ndarray:
    """fp64 -> fp16 bit patterns, round to nearest even (one rounding)."""
    with np.errstate(over="ignore"):
        return np.ascontiguousarray(y, dtype=np.float64).astype(np.float16).view(np.uint16)


def conv2d(x_bits: np.ndarray, w_bits: np.ndarray, pad=(1, 1), stride=(1, 1), want_S: bool = True, nthreads: int = 0):
    """y_ref and S, fp64, shape (N, P, Q, F), for x (N, H, W, C) and w (F, R, S, C) given as fp16 bit patterns."""
    lib = _load()
    N, H, W, C = x_bits.shape
    F, R, S_, C2 = w_bits.shape
    if C2 != C:
        raise ValueError("channel counts differ")
    P, Q = out_size(H, W, R, S_, pad, stride)
    x = f16_bits_to_f64(x_bits)
    w = f16_bits_to_f64(w_bits)
    y = np.full((N, P, Q, F), np.nan, dtype=np.float64)
    s = np.full((N, P, Q, F), np.nan, dtype=np.float64) if want_S else None
    rc = lib.oracle_conv2d(N, H, W, C, F, R, S_, pad[0], pad[1], stride[0], stride[1], x.ctypes.data, w.ctypes.data,
                           y.ctypes.data, s.ctypes.data if want_S else None, nthreads)
    if rc != 0:
        raise ValueError(f"oracle_conv2d rejected its arguments (rc={rc})")
    return y, s


def bound_f32(K: int, S: np.ndarray) -> np.ndarray:
    return float(K) * 2.0 ** -23 * S


def bound_f16(K: int, S: np.ndarray, y_ref: np.ndarray) -> np.ndarray:
    tol = bound_f32(K, S)
    return tol + 2.0 ** -11 * (np.abs(y_ref) + tol)
