"""Seeded synthetic inputs for the bf16 GEMM lineage.

This module holds no GEMM arithmetic: it only draws numbers, rounds them to
bf16 and lays them out with leading dimensions.  It is the one module the
tests hand to both the CUDA path and the CPU oracle.

The paper's GEMM workload is one synthetic shape (Evaluation, Table 2: GEMM,
M=N=K=4096, BF16) whose value distribution is not stated, plus plain-MM shapes
in its held-out appendix (8192^3 among them); the five configurations below
stand in for those and take their shapes and dtype.  bf16 values are carried
as uint16 bit patterns in numpy arrays.

Recipe: numpy Philox keyed by (seed, tensor id).  uniform: u in [0,1) in fp64,
value 2u-1 -> fp32 -> bf16 (round to nearest even).  normal: standard_normal in
fp64 times sigma -> fp32 -> bf16.  integer: integers in {-4..4}.  Padding
between the logical width and the leading dimension is filled with NaN bit
patterns so that any read of padding that reaches C shows up.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Tuple

import numpy as np

BF16_NAN_BITS = np.uint16(0x7FC1)  # a NaN payload distinct from the canonical 0x7FC0


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest, ties to even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    w = x.view(np.uint32).astype(np.uint64)
    lsb = (w >> np.uint64(16)) & np.uint64(1)
    r = (w + np.uint64(0x7FFF) + lsb) >> np.uint64(16)
    out = r.astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> fp32, exact."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(tensor_id)]))


def draw(shape: Tuple[int, int], dist: str, seed: int, tensor_id: int, sigma: float = 1.0) -> np.ndarray:
    """A (rows, cols) array of bf16 bit patterns drawn from ``dist``."""
    g = _rng(seed, tensor_id)
    if dist == "uniform":
        v = (2.0 * g.random(shape) - 1.0).astype(np.float32)
    elif dist == "normal":
        v = (g.standard_normal(shape) * sigma).astype(np.float32)
    elif dist == "integer":
        v = g.integers(-4, 5, size=shape).astype(np.float32)
    else:
        raise ValueError(dist)
    return f32_to_bf16_bits(v)


def with_ld(bits2d: np.ndarray, ld: int) -> np.ndarray:
    """Copy a (rows, cols) array into a (rows, ld) buffer whose padding is NaN."""
    rows, cols = bits2d.shape
    if ld < cols:
        raise ValueError("leading dimension smaller than the row length")
    out = np.full((rows, ld), BF16_NAN_BITS, dtype=np.uint16)
    out[:, :cols] = bits2d
    return out


@dataclass
class GemmCase:
    """One GEMM problem: bf16 bit patterns laid out as the C ABI expects them."""
    name: str
    M: int
    N: int
    K: int
    lda: int
    ldb: int
    ldc: int
    b_col_major: bool
    c_bf16: bool
    A: np.ndarray = field(repr=False)   # (M, lda) uint16
    B: np.ndarray = field(repr=False)   # (K, ldb) row-major  |  (N, ldb) column-major
    seed: int = 0
    dist: str = ""

    @property
    def flops(self) -> float:
        return 2.0 * self.M * self.N * self.K

    @property
    def algorithmic_bytes(self) -> int:
        """A and B read once, C written once."""
        return 2 * self.M * self.K + 2 * self.K * self.N + (2 if self.c_bf16 else 4) * self.M * self.N


# name -> (M, N, K, lda, ldb, ldc, b_col_major, c_bf16, distA, sigmaA, distB, sigmaB)
_CONFIGS = {
    "c1": (256, 256, 256, 256, 256, 256, False, False, "uniform", 1.0, "uniform", 1.0),
    "c2": (1000, 1001, 999, 999, 1001, 1001, False, False, "uniform", 1.0, "uniform", 1.0),
    "c2pad": (1000, 1001, 999, 1008, 1008, 1004, False, False, "uniform", 1.0, "uniform", 1.0),
    "c3": (4096, 4096, 4096, 4096, 4096, 4096, True, True, "normal", 1.0, "normal", 1.0),
    "c4": (8192, 8192, 8192, 8192, 8192, 8192, False, True, "normal", 8192 ** -0.5, "normal", 8192 ** -0.5),
    "c5": (16, 8192, 8192, 8192, 8192, 8192, False, False, "normal", 1.0, "normal", 0.02),
}
CONFIG_NAMES = ("c1", "c2", "c3", "c4", "c5")


def make_case(M: int, N: int, K: int, seed: int, dist_a: str = "uniform", dist_b: str = "uniform",
              sigma_a: float = 1.0, sigma_b: float = 1.0, lda: Optional[int] = None,
              ldb: Optional[int] = None, ldc: Optional[int] = None, b_col_major: bool = False,
              c_bf16: bool = False, name: str = "custom") -> GemmCase:
    lda = K if lda is None else lda
    ldb = (K if b_col_major else N) if ldb is None else ldb
    ldc = N if ldc is None else ldc
    a = draw((M, K), dist_a, seed, 0, sigma_a)
    b_logical = draw((K, N), dist_b, seed, 1, sigma_b)          # always drawn as K x N
    b_store = np.ascontiguousarray(b_logical.T) if b_col_major else b_logical
    return GemmCase(name=name, M=M, N=N, K=K, lda=lda, ldb=ldb, ldc=ldc, b_col_major=b_col_major,
                    c_bf16=c_bf16, A=with_ld(a, lda), B=with_ld(b_store, ldb), seed=seed,
                    dist=f"{dist_a}/{dist_b}")


def make_config(name: str, seed: int, integer: bool = False, c_bf16: Optional[bool] = None) -> GemmCase:
    """One of the named configurations; ``integer`` swaps in entries from {-4..4}."""
    M, N, K, lda, ldb, ldc, col, cb, da, sa, db, sb = _CONFIGS[name]
    if integer:
        da = db = "integer"
    if c_bf16 is not None:
        cb = c_bf16
    return make_case(M, N, K, seed, da, db, sa, sb, lda, ldb, ldc, col, cb, name + ("-int" if integer else ""))


def config_shape(name: str):
    M, N, K, lda, ldb, ldc, col, cb = _CONFIGS[name][:8]
    return dict(M=M, N=N, K=K, lda=lda, ldb=ldb, ldc=ldc, b_col_major=col, c_bf16=cb)


# ---------------------------------------------------------------------------- Conv2d inputs (fp16)
@dataclass
class ConvCase:
    """A channels-last Conv2d problem: x (N, H, W, C) and w (F, R, S, C) as fp16 bit patterns (uint16)."""
    name: str
    N: int
    H: int
    W: int
    C: int
    F: int
    R: int
    S: int
    pad: Tuple[int, int]
    stride: Tuple[int, int]
    y_f16: bool
    x: np.ndarray = field(repr=False)
    w: np.ndarray = field(repr=False)

    @property
    def P(self) -> int:
        return (self.H + 2 * self.pad[0] - self.R) // self.stride[0] + 1

    @property
    def Q(self) -> int:
        return (self.W + 2 * self.pad[1] - self.S) // self.stride[1] + 1

    @property
    def K(self) -> int:
        return self.R * self.S * self.C

    @property
    def flops(self) -> float:
        return 2.0 * self.N * self.P * self.Q * self.F * self.K


def draw_f16(shape, dist: str, seed: int, tensor_id: int, sigma: float = 1.0) -> np.ndarray:
    """fp16 bit patterns drawn as in ``draw`` (fp64 -> fp32 -> fp16, round to nearest even)."""
    g = _rng(seed, tensor_id)
    if dist == "uniform":
        v = (2.0 * g.random(shape) - 1.0).astype(np.float32)
    elif dist == "normal":
        v = (g.standard_normal(shape) * sigma).astype(np.float32)
    elif dist == "integer":
        v = g.integers(-4, 5, size=shape).astype(np.float32)
    else:
        raise ValueError(f"unknown distribution {dist!r}")
    return v.astype(np.float16).view(np.uint16)


def make_conv_case(N: int, H: int, W: int, C: int, F: int, R: int, S: int, seed: int, pad=(1, 1), stride=(1, 1),
                   dist: str = "normal", y_f16: bool = True, name: str = "") -> ConvCase:
    """x ~ dist (sigma 1), w ~ dist with sigma 1/sqrt(R*S*C) for "normal" (outputs of order 1)."""
    sig_w = 1.0 / np.sqrt(max(R * S * C, 1)) if dist == "normal" else 1.0
    x = draw_f16((N, H, W, C), dist, seed, 10)
    w = draw_f16((F, R, S, C), dist, seed, 11, sig_w)
    return ConvCase(name or f"conv{N}x{H}x{W}x{C}-f{F}-{R}x{S}", N, H, W, C, F, R, S, tuple(pad), tuple(stride), y_f16,
                    x, w)


def conv_benchmark_case(seed: int, integer: bool = False) -> ConvCase:
    """The paper's Conv2d shape: N=8, C=64, 56x56, F=128, 3x3, fp16; read as padding 1, stride 1."""
    return make_conv_case(8, 56, 56, 64, 128, 3, 3, seed, dist="integer" if integer else "normal", name="conv_t2")
