"""ctypes face of ``libklineage_gemm.so``: argument marshalling only.

Names mirror the C ABI (``include/klineage_gemm.h``).  PyTorch appears only as
the owner of device memory and streams.  There is no fallback of any kind: if
the CUDA library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path
from typing import Optional

PKG = Path(__file__).resolve().parent
LIB_PATH = PKG / "libklineage_gemm.so"

KLINEAGE_OK = 0
KLINEAGE_ERR_INVALID_ARG = 1
KLINEAGE_ERR_BAD_VARIANT = 2
KLINEAGE_ERR_UNSUPPORTED_DEVICE = 3
KLINEAGE_ERR_ALLOC = 4
KLINEAGE_ERR_LAUNCH = 5
KLINEAGE_ERR_TIMEOUT = 6
KLINEAGE_ERR_INTERNAL = 7
KLINEAGE_ERR_SCRATCH_LIMIT = 8

KLINEAGE_B_ROW_MAJOR, KLINEAGE_B_COL_MAJOR = 0, 1
KLINEAGE_C_F32, KLINEAGE_C_BF16, KLINEAGE_C_F16 = 0, 1, 2
KLINEAGE_FLAG_STATIC_B = 1
KLINEAGE_FLAG_TEST_GIVE_UP = 2
KLINEAGE_NAIVE, KLINEAGE_TILED, KLINEAGE_VECTORIZED, KLINEAGE_PIPELINED, KLINEAGE_TCGEN05, KLINEAGE_MMA_SYNC = range(6)
# the five-step ladder, then the intermediate legacy tensor-core rung ("3.5")
VARIANTS = (KLINEAGE_NAIVE, KLINEAGE_TILED, KLINEAGE_VECTORIZED, KLINEAGE_PIPELINED, KLINEAGE_TCGEN05,
            KLINEAGE_MMA_SYNC)

EXPORTED_SYMBOLS = (
    "klineage_gemm_create", "klineage_gemm_run", "klineage_gemm_destroy", "klineage_gemm_check_args",
    "klineage_gemm_get_device_status", "klineage_gemm_last_kernel_id", "klineage_status_string",
    "klineage_variant_name", "klineage_gemm_run_noalloc", "klineage_gemm_run_addmm",
    "klineage_gemm_run_batched", "klineage_gemm_run_grouped", "klineage_gemm_last_launch_count",
    "klineage_gemm_run_multi_dst", "klineage_conv2d_run", "klineage_conv2d_check_args",
    "klineage_gemm_plan_candidates", "klineage_gemm_set_plan", "klineage_gemm_get_plan", "klineage_gemm_autotune",
    "klineage_gemm_host_scratch_bytes", "klineage_gemm_run_host", "klineage_gemm_last_give_up",
)


class klineage_gemm_config_t(ctypes.Structure):
    _fields_ = [("device", ctypes.c_int), ("b_layout", ctypes.c_int), ("c_dtype", ctypes.c_int),
                ("workspace_bytes", ctypes.c_size_t), ("flags", ctypes.c_uint)]


class KlineageError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {klineage_status_string(status)} (status {status})")


if not LIB_PATH.exists():
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2605_28213_b200.build` "
        "(nvcc, sm_100a).  This package has no CPU or PyTorch fallback.")

_lib = ctypes.CDLL(str(LIB_PATH))
_i64, _p, _int = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int

_lib.klineage_gemm_create.restype = _int
_lib.klineage_gemm_create.argtypes = [ctypes.POINTER(_p), ctypes.POINTER(klineage_gemm_config_t)]
_lib.klineage_gemm_run.restype = _int
_lib.klineage_gemm_run.argtypes = [_p, _i64, _i64, _i64, _p, _i64, _p, _i64, _p, _i64, _int, _p]
_lib.klineage_gemm_destroy.restype = _int
_lib.klineage_gemm_destroy.argtypes = [_p]
_lib.klineage_gemm_check_args.restype = _int
_lib.klineage_gemm_check_args.argtypes = [_int, _int, _i64, _i64, _i64, _p, _i64, _p, _i64, _p, _i64, _int]
_lib.klineage_gemm_get_device_status.restype = _int
_lib.klineage_gemm_get_device_status.argtypes = [_p, ctypes.POINTER(_int), ctypes.POINTER(_int)]
_lib.klineage_gemm_last_kernel_id.restype = _int
_lib.klineage_gemm_last_kernel_id.argtypes = [_p]
_lib.klineage_status_string.restype = ctypes.c_char_p
_lib.klineage_status_string.argtypes = [_int]
_lib.klineage_variant_name.restype = ctypes.c_char_p
_lib.klineage_variant_name.argtypes = [_int]


_lib.klineage_gemm_run_noalloc.restype = _int
_lib.klineage_gemm_run_noalloc.argtypes = [_int, _int, _i64, _i64, _i64, _p, _i64, _p, _i64, _p, _i64, _p]


def klineage_gemm_run_noalloc(b_layout, c_dtype, M, N, K, A, lda, B, ldb, C, ldc, stream=None) -> int:
    """Raw status of the allocation-free tcgen05 call (no handle; fixed in-library scratch).

    For callers that may not allocate device memory.  Pointers are integer device
    addresses on the current device; see the header for the scratch limit and the
    one-stream-at-a-time rule.
    """
    return _lib.klineage_gemm_run_noalloc(b_layout, c_dtype, M, N, K, A, lda, B, ldb, C, ldc, stream)


_lib.klineage_gemm_host_scratch_bytes.restype = ctypes.c_size_t
_lib.klineage_gemm_host_scratch_bytes.argtypes = [_int, _int, _i64, _i64, _i64]
_lib.klineage_gemm_run_host.restype = _int
_lib.klineage_gemm_run_host.argtypes = [_p, _i64, _i64, _i64, _p, _i64, _p, _i64, _p, _i64, _p, ctypes.c_size_t, _int, _p]


def klineage_gemm_host_scratch_bytes(b_layout, c_dtype, M, N, K) -> int:
    """Device scratch (bytes) that klineage_gemm_run_host needs for this shape; 0 for an empty or invalid one."""
    return int(_lib.klineage_gemm_host_scratch_bytes(b_layout, c_dtype, M, N, K))


def klineage_gemm_run_host_raw(h, M, N, K, A_host, lda, B_host, ldb, C_host, ldc, scratch, scratch_bytes, variant,
                               stream) -> int:
    """Raw status of C = A.B with A, B, C in HOST memory (integer addresses) and a device scratch buffer."""
    return _lib.klineage_gemm_run_host(h, M, N, K, A_host, lda, B_host, ldb, C_host, ldc, scratch, scratch_bytes,
                                       variant, stream)


_lib.klineage_gemm_run_addmm.restype = _int
_lib.klineage_gemm_run_addmm.argtypes = [_p, _i64, _i64, _i64, _p, _i64, _p, _i64, _p, _p, _i64, _int, _p]


def klineage_gemm_run_addmm_raw(h, M, N, K, A, lda, B, ldb, bias, C, ldc, variant, stream) -> int:
    """Raw status of C <- A.B + bias (bias: N bf16 values on the device)."""
    return _lib.klineage_gemm_run_addmm(h, M, N, K, A, lda, B, ldb, bias, C, ldc, variant, stream)


_lib.klineage_gemm_last_launch_count.restype = _int
_lib.klineage_gemm_last_launch_count.argtypes = [_p]
_lib.klineage_gemm_run_batched.restype = _int
_lib.klineage_gemm_run_batched.argtypes = [_p, _i64, _i64, _i64, _i64, _p, _i64, _i64, _p, _i64, _i64, _p, _i64, _i64,
                                           _int, _p]
_lib.klineage_gemm_run_grouped.restype = _int
_lib.klineage_gemm_run_grouped.argtypes = [_p, _int] + [ctypes.POINTER(_i64)] * 3 + [
    ctypes.POINTER(_p), ctypes.POINTER(_i64), ctypes.POINTER(_p), ctypes.POINTER(_i64), ctypes.POINTER(_p),
    ctypes.POINTER(_i64), _int, _p]


def klineage_gemm_run_batched_raw(h, batch, M, N, K, A, lda, stride_a, B, ldb, stride_b, C, ldc, stride_c, variant,
                                  stream) -> int:
    """Raw status of C_b <- A_b . B_b, b < batch (strides in elements)."""
    return _lib.klineage_gemm_run_batched(h, batch, M, N, K, A, lda, stride_a, B, ldb, stride_b, C, ldc, stride_c,
                                          variant, stream)


_lib.klineage_gemm_run_multi_dst.restype = _int
_lib.klineage_gemm_run_multi_dst.argtypes = [_p, _i64, _i64, _i64, _p, _i64, _p, _i64, _int, ctypes.POINTER(_p),
                                             ctypes.POINTER(_i64), _int, _p]


def klineage_gemm_run_multi_dst_raw(h, M, N, K, A, lda, B, ldb, C, ldc, variant, stream) -> int:
    """Raw status of C_d <- A . B for every destination (C, ldc: sequences of device pointers / pitches)."""
    n = len(C)
    assert len(ldc) == n
    return _lib.klineage_gemm_run_multi_dst(h, M, N, K, A, lda, B, ldb, n, (_p * n)(*[int(x) for x in C]),
                                            (_i64 * n)(*[int(x) for x in ldc]), variant, stream)


def klineage_gemm_run_grouped_raw(h, M, N, K, A, lda, B, ldb, C, ldc, variant, stream) -> int:
    """Raw status of C_i <- A_i . B_i over groups; every argument up to ldc is a sequence with one entry per group."""
    n = len(M)
    assert all(len(x) == n for x in (N, K, A, lda, B, ldb, C, ldc))
    i64s = lambda xs: (_i64 * n)(*[int(x) for x in xs])
    ptrs = lambda xs: (_p * n)(*[None if x is None else int(x) for x in xs])
    return _lib.klineage_gemm_run_grouped(h, n, i64s(M), i64s(N), i64s(K), ptrs(A), i64s(lda), ptrs(B), i64s(ldb),
                                          ptrs(C), i64s(ldc), variant, stream)


_lib.klineage_conv2d_run.restype = _int
_lib.klineage_conv2d_run.argtypes = [_p] + [_i64] * 11 + [_p, _p, _p, _int, _p]
_lib.klineage_conv2d_check_args.restype = _int
_lib.klineage_conv2d_check_args.argtypes = [_int] + [_i64] * 11 + [_p, _p, _p, _int]


def klineage_conv2d_run_raw(h, N, H, W, C, F, R, S, pad_h, pad_w, stride_h, stride_w, x, w, y, variant, stream) -> int:
    """Raw status of the channels-last fp16 Conv2d (x, w, y: device addresses)."""
    return _lib.klineage_conv2d_run(h, N, H, W, C, F, R, S, pad_h, pad_w, stride_h, stride_w, x, w, y, variant, stream)


def klineage_conv2d_check_args(y_dtype, N, H, W, C, F, R, S, pad_h, pad_w, stride_h, stride_w, x, w, y, variant) -> int:
    return _lib.klineage_conv2d_check_args(y_dtype, N, H, W, C, F, R, S, pad_h, pad_w, stride_h, stride_w, x, w, y,
                                           variant)


class klineage_gemm_plan_t(ctypes.Structure):
    """Launch plan of the tcgen05 rung (0 in a field = the rung's heuristic)."""
    _fields_ = [("kernel", _int), ("splits", _int), ("split_via", _int), ("group_m", _int), ("half_tail", _int),
                ("tile_n", _int), ("tail_n", _int), ("stages", _int)]
    FIELDS = ("kernel", "splits", "split_via", "group_m", "half_tail", "tile_n", "tail_n", "stages")

    def as_tuple(self):
        return tuple(getattr(self, f) for f in self.FIELDS)

    def as_dict(self):
        return dict(zip(self.FIELDS, self.as_tuple()))

    def __repr__(self):
        return "plan(" + ", ".join("%s=%d" % kv for kv in self.as_dict().items()) + ")"


KLINEAGE_MAX_PLANS = 48
_shape_args = [_p, _i64, _i64, _i64, _p, _i64, _p, _i64, _p, _i64]
_lib.klineage_gemm_plan_candidates.restype = _int
_lib.klineage_gemm_plan_candidates.argtypes = _shape_args + [ctypes.POINTER(klineage_gemm_plan_t), _int,
                                                             ctypes.POINTER(_int)]
_lib.klineage_gemm_set_plan.restype = _int
_lib.klineage_gemm_set_plan.argtypes = _shape_args + [ctypes.POINTER(klineage_gemm_plan_t)]
_lib.klineage_gemm_get_plan.restype = _int
_lib.klineage_gemm_get_plan.argtypes = _shape_args + [ctypes.POINTER(klineage_gemm_plan_t), ctypes.POINTER(_int)]
_lib.klineage_gemm_autotune.restype = _int
_lib.klineage_gemm_autotune.argtypes = _shape_args + [_int, _p, ctypes.POINTER(klineage_gemm_plan_t),
                                                      ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float)]


def klineage_gemm_plan_candidates(h, M, N, K, A, lda, B, ldb, C, ldc):
    """List of candidate plans (klineage_gemm_plan_t); the first is the all-zero heuristic plan."""
    arr = (klineage_gemm_plan_t * KLINEAGE_MAX_PLANS)()
    n = _int(0)
    st = _lib.klineage_gemm_plan_candidates(h, M, N, K, A, lda, B, ldb, C, ldc, arr, KLINEAGE_MAX_PLANS,
                                            ctypes.byref(n))
    if st != KLINEAGE_OK:
        raise KlineageError(st, "klineage_gemm_plan_candidates")
    return [klineage_gemm_plan_t(*arr[i].as_tuple()) for i in range(n.value)]


def klineage_gemm_set_plan_raw(h, M, N, K, A, lda, B, ldb, C, ldc, plan) -> int:
    """Raw status of pinning `plan` (None removes the pin)."""
    ref = None if plan is None else ctypes.byref(plan)
    return _lib.klineage_gemm_set_plan(h, M, N, K, A, lda, B, ldb, C, ldc, ref)


def klineage_gemm_get_plan(h, M, N, K, A, lda, B, ldb, C, ldc):
    """(plan, pinned?) for the shape."""
    plan, pinned = klineage_gemm_plan_t(), _int(0)
    st = _lib.klineage_gemm_get_plan(h, M, N, K, A, lda, B, ldb, C, ldc, ctypes.byref(plan), ctypes.byref(pinned))
    if st != KLINEAGE_OK:
        raise KlineageError(st, "klineage_gemm_get_plan")
    return plan, bool(pinned.value)


def klineage_gemm_autotune(h, M, N, K, A, lda, B, ldb, C, ldc, iters, stream):
    """(pinned plan, its microseconds per launch, the heuristic plan's microseconds)."""
    plan = klineage_gemm_plan_t()
    best, heur = ctypes.c_float(0), ctypes.c_float(0)
    st = _lib.klineage_gemm_autotune(h, M, N, K, A, lda, B, ldb, C, ldc, iters, stream, ctypes.byref(plan),
                                     ctypes.byref(best), ctypes.byref(heur))
    if st != KLINEAGE_OK:
        raise KlineageError(st, "klineage_gemm_autotune")
    return plan, best.value, heur.value


def klineage_status_string(status: int) -> str:
    return _lib.klineage_status_string(int(status)).decode()


def klineage_variant_name(variant: int) -> str:
    return _lib.klineage_variant_name(int(variant)).decode()


def klineage_gemm_check_args(b_layout, c_dtype, M, N, K, A, lda, B, ldb, C, ldc, variant) -> int:
    """Raw status of the host-side argument checks (pointers are integers or None)."""
    return _lib.klineage_gemm_check_args(b_layout, c_dtype, M, N, K, A, lda, B, ldb, C, ldc, variant)


def klineage_gemm_create(device: int, b_layout: int, c_dtype: int, workspace_bytes: int = 0,
                         flags: int = 0) -> int:
    """Returns the opaque handle (an integer); raises KlineageError on failure."""
    cfg = klineage_gemm_config_t(device, b_layout, c_dtype, workspace_bytes, flags)
    h = _p()
    st = _lib.klineage_gemm_create(ctypes.byref(h), ctypes.byref(cfg))
    if st != KLINEAGE_OK:
        raise KlineageError(st, "klineage_gemm_create")
    return h.value


def klineage_gemm_run_raw(h, M, N, K, A, lda, B, ldb, C, ldc, variant, stream) -> int:
    """Raw status code; pointers are integers (device addresses) or None."""
    return _lib.klineage_gemm_run(h, M, N, K, A, lda, B, ldb, C, ldc, variant, stream)


def klineage_gemm_run(h, M, N, K, A, lda, B, ldb, C, ldc, variant, stream=None) -> None:
    st = klineage_gemm_run_raw(h, M, N, K, A, lda, B, ldb, C, ldc, variant, stream)
    if st != KLINEAGE_OK:
        raise KlineageError(st, "klineage_gemm_run")


def klineage_gemm_destroy(h) -> None:
    _lib.klineage_gemm_destroy(h)


def klineage_gemm_get_device_status(h):
    """(status code, id of the kernel that last ran on the device)."""
    code, kid = _int(0), _int(0)
    st = _lib.klineage_gemm_get_device_status(h, ctypes.byref(code), ctypes.byref(kid))
    if st != KLINEAGE_OK:
        raise KlineageError(st, "klineage_gemm_get_device_status")
    return code.value, kid.value


def klineage_gemm_last_kernel_id(h) -> int:
    return _lib.klineage_gemm_last_kernel_id(h)


_lib.klineage_gemm_last_give_up.restype = _int
_lib.klineage_gemm_last_give_up.argtypes = [_p, ctypes.POINTER(ctypes.c_uint), ctypes.POINTER(ctypes.c_uint)]


def klineage_gemm_last_give_up(h):
    """(CTA, role-and-barrier code) of the last device-side give-up read through get_device_status; (0, 0) if none."""
    block, where = ctypes.c_uint(0), ctypes.c_uint(0)
    st = _lib.klineage_gemm_last_give_up(h, ctypes.byref(block), ctypes.byref(where))
    if st != KLINEAGE_OK:
        raise KlineageError(st, "klineage_gemm_last_give_up")
    return block.value, where.value


class Gemm:
    """Handle wrapper: ``Gemm(device, b_col_major, c_bf16).run(A, B, C, M, N, K, lda, ldb, ldc, variant)``.

    ``A``, ``B``, ``C`` are torch CUDA tensors (any shape; only ``data_ptr()`` is
    used) or integer device addresses.  The launch goes to torch's current stream
    unless ``stream`` (a ``torch.cuda.Stream`` or raw pointer) is given.
    """

    def __init__(self, device: int = 0, b_col_major: bool = False, c_bf16: bool = False,
                 workspace_bytes: int = 0, static_b: bool = False, test_give_up: bool = False):
        self.device = int(device)
        self.b_col_major = bool(b_col_major)
        self.c_bf16 = bool(c_bf16)
        self._h: Optional[int] = klineage_gemm_create(
            self.device, KLINEAGE_B_COL_MAJOR if b_col_major else KLINEAGE_B_ROW_MAJOR,
            KLINEAGE_C_BF16 if c_bf16 else KLINEAGE_C_F32, workspace_bytes,
            (KLINEAGE_FLAG_STATIC_B if static_b else 0) | (KLINEAGE_FLAG_TEST_GIVE_UP if test_give_up else 0))

    @staticmethod
    def _ptr(x):
        if x is None or isinstance(x, int):
            return x
        return x.data_ptr()

    @staticmethod
    def _stream(stream):
        if stream is None:
            import torch
            return torch.cuda.current_stream().cuda_stream
        if isinstance(stream, int):
            return stream
        return stream.cuda_stream

    def run(self, A, B, C, M, N, K, lda, ldb, ldc, variant, stream=None) -> None:
        klineage_gemm_run(self._h, M, N, K, self._ptr(A), lda, self._ptr(B), ldb, self._ptr(C), ldc,
                          int(variant), self._stream(stream))

    def host_scratch_bytes(self, M, N, K) -> int:
        return klineage_gemm_host_scratch_bytes(KLINEAGE_B_COL_MAJOR if self.b_col_major else KLINEAGE_B_ROW_MAJOR,
                                                KLINEAGE_C_BF16 if self.c_bf16 else KLINEAGE_C_F32, M, N, K)

    def run_host(self, A_host, B_host, C_host, M, N, K, lda, ldb, ldc, scratch, scratch_bytes, variant,
                 stream=None) -> None:
        """A_host, B_host, C_host: CPU tensors (pinned for overlap) or integer host addresses; scratch: device."""
        st = klineage_gemm_run_host_raw(self._h, M, N, K, self._ptr(A_host), lda, self._ptr(B_host), ldb,
                                        self._ptr(C_host), ldc, self._ptr(scratch), int(scratch_bytes), int(variant),
                                        self._stream(stream))
        if st != KLINEAGE_OK:
            raise KlineageError(st, "klineage_gemm_run_host")

    def run_addmm(self, A, B, bias, C, M, N, K, lda, ldb, ldc, variant, stream=None) -> None:
        st = klineage_gemm_run_addmm_raw(self._h, M, N, K, self._ptr(A), lda, self._ptr(B), ldb, self._ptr(bias),
                                         self._ptr(C), ldc, int(variant), self._stream(stream))
        if st != KLINEAGE_OK:
            raise KlineageError(st, "klineage_gemm_run_addmm")

    def run_batched(self, batch, A, B, C, M, N, K, lda, ldb, ldc, stride_a, stride_b, stride_c, variant,
                    stream=None) -> None:
        st = klineage_gemm_run_batched_raw(self._h, batch, M, N, K, self._ptr(A), lda, stride_a, self._ptr(B), ldb,
                                           stride_b, self._ptr(C), ldc, stride_c, int(variant), self._stream(stream))
        if st != KLINEAGE_OK:
            raise KlineageError(st, "klineage_gemm_run_batched")

    def run_grouped(self, A, B, C, M, N, K, lda, ldb, ldc, variant, stream=None) -> None:
        st = klineage_gemm_run_grouped_raw(self._h, M, N, K, [self._ptr(x) for x in A], lda,
                                           [self._ptr(x) for x in B], ldb, [self._ptr(x) for x in C], ldc,
                                           int(variant), self._stream(stream))
        if st != KLINEAGE_OK:
            raise KlineageError(st, "klineage_gemm_run_grouped")

    def run_multi_dst(self, A, B, Cs, M, N, K, lda, ldb, ldcs, variant, stream=None) -> None:
        st = klineage_gemm_run_multi_dst_raw(self._h, M, N, K, self._ptr(A), lda, self._ptr(B), ldb,
                                             [self._ptr(c) for c in Cs], ldcs, int(variant), self._stream(stream))
        if st != KLINEAGE_OK:
            raise KlineageError(st, "klineage_gemm_run_multi_dst")

    def run_raw(self, A, B, C, M, N, K, lda, ldb, ldc, variant, stream=None) -> int:
        return klineage_gemm_run_raw(self._h, M, N, K, self._ptr(A), lda, self._ptr(B), ldb, self._ptr(C),
                                     ldc, int(variant), self._stream(stream))

    def plan_candidates(self, A, B, C, M, N, K, lda, ldb, ldc):
        return klineage_gemm_plan_candidates(self._h, M, N, K, self._ptr(A), lda, self._ptr(B), ldb, self._ptr(C), ldc)

    def set_plan(self, plan, A, B, C, M, N, K, lda, ldb, ldc) -> None:
        st = klineage_gemm_set_plan_raw(self._h, M, N, K, self._ptr(A), lda, self._ptr(B), ldb, self._ptr(C), ldc,
                                        plan)
        if st != KLINEAGE_OK:
            raise KlineageError(st, "klineage_gemm_set_plan")

    def get_plan(self, A, B, C, M, N, K, lda, ldb, ldc):
        return klineage_gemm_get_plan(self._h, M, N, K, self._ptr(A), lda, self._ptr(B), ldb, self._ptr(C), ldc)

    def autotune(self, A, B, C, M, N, K, lda, ldb, ldc, iters: int = 10, stream=None):
        return klineage_gemm_autotune(self._h, M, N, K, self._ptr(A), lda, self._ptr(B), ldb, self._ptr(C), ldc,
                                      int(iters), self._stream(stream))

    def device_status(self):
        return klineage_gemm_get_device_status(self._h)

    def last_kernel_id(self) -> int:
        return klineage_gemm_last_kernel_id(self._h)

    def last_give_up(self):
        return klineage_gemm_last_give_up(self._h)

    def last_launch_count(self) -> int:
        return _lib.klineage_gemm_last_launch_count(self._h)

    def close(self) -> None:
        if self._h is not None:
            klineage_gemm_destroy(self._h)
            self._h = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Conv2d:
    """Handle wrapper of the fp16 channels-last Conv2d: ``Conv2d(device, y_f16).run(x, w, y, N, H, W, C, F, R, S, ...)``.

    ``x`` (N, H, W, C), ``w`` (F, R, S, C) hold fp16 values, ``y`` (N, P, Q, F) fp16 or fp32; torch CUDA tensors (only
    ``data_ptr()`` is used) or integer device addresses.  variant 0 = direct convolution, 4 = implicit GEMM on tcgen05.
    """

    def __init__(self, device: int = 0, y_f16: bool = True):
        self.device, self.y_f16 = int(device), bool(y_f16)
        self._h: Optional[int] = klineage_gemm_create(self.device, KLINEAGE_B_COL_MAJOR,
                                                      KLINEAGE_C_F16 if y_f16 else KLINEAGE_C_F32, 0)

    def run(self, x, w, y, N, H, W, C, F, R, S, pad=(1, 1), stride=(1, 1), variant=4, stream=None) -> None:
        st = klineage_conv2d_run_raw(self._h, N, H, W, C, F, R, S, pad[0], pad[1], stride[0], stride[1], Gemm._ptr(x),
                                     Gemm._ptr(w), Gemm._ptr(y), int(variant), Gemm._stream(stream))
        if st != KLINEAGE_OK:
            raise KlineageError(st, "klineage_conv2d_run")

    def device_status(self):
        return klineage_gemm_get_device_status(self._h)

    def last_kernel_id(self) -> int:
        return klineage_gemm_last_kernel_id(self._h)

    def close(self) -> None:
        if self._h is not None:
            klineage_gemm_destroy(self._h)
            self._h = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
