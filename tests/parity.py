"""Helpers of the GPU parity tests: upload with guard bands, run through the C ABI, compare with the oracle."""
from __future__ import annotations

import functools

import numpy as np

from oracle import gemm_oracle as orc
from paper_2605_28213_b200 import inputs as gen

GUARD = 4096          # bytes of 0xA5 before and after every device buffer
POISON = 0xA5


def sample_rows(M: int) -> np.ndarray:
    """All rows for small M; otherwise two rows of every 128-row tile, residues spread."""
    if M <= 1024:
        return np.arange(M)
    rows = []
    for t in range((M + 127) // 128):
        for s in (0, 64):
            r = 128 * t + ((37 * t + s) % 128)
            if r < M:
                rows.append(r)
    return np.array(sorted(set(rows)))


def oracle_rows(case: gen.GemmCase, rows: np.ndarray):
    """Oracle C_ref and S for the given rows (same arithmetic per row as a full run)."""
    A_sub = np.ascontiguousarray(case.A[rows])
    return orc.gemm(len(rows), case.N, case.K, A_sub, case.lda, case.B, case.ldb, case.b_col_major)


@functools.lru_cache(maxsize=6)
def cached_reference(name: str, seed: int, integer: bool):
    """(case, rows, C_ref, S) for a named configuration; cached across the rungs."""
    case = gen.make_config(name, seed, integer=integer)
    rows = sample_rows(case.M)
    C_ref, S = oracle_rows(case, rows)
    return case, rows, C_ref, S


class DeviceBuffer:
    """A byte buffer on the GPU with 0xA5 guard bands; ``ptr`` points ``offset`` bytes past the front guard."""

    def __init__(self, nbytes: int, offset: int = 0, align: int = 256):
        import torch
        self.nbytes, self.offset = int(nbytes), int(offset)
        self.raw = torch.full((GUARD + align + self.offset + self.nbytes + GUARD,), POISON, dtype=torch.uint8,
                              device="cuda")
        base = self.raw.data_ptr() + GUARD
        self.start = GUARD + ((-base) % align) + self.offset      # index into raw of the payload
        self.ptr = self.raw.data_ptr() + self.start

    def upload(self, arr: np.ndarray):
        import torch
        b = np.ascontiguousarray(arr).view(np.uint8).reshape(-1)
        assert b.size <= self.nbytes
        self.raw[self.start:self.start + b.size] = torch.from_numpy(b).cuda()
        return self

    def download(self) -> np.ndarray:
        return self.raw[self.start:self.start + self.nbytes].cpu().numpy()

    def guards_intact(self) -> bool:
        head = self.raw[:self.start]
        tail = self.raw[self.start + self.nbytes:]
        return bool((head == POISON).all().item()) and bool((tail == POISON).all().item())


class DeviceCase:
    """A GemmCase resident on the GPU; offsets (in elements) shift each base pointer."""

    def __init__(self, case: gen.GemmCase, off_a: int = 0, off_b: int = 0, off_c: int = 0):
        self.case = case
        self.celt = 2 if case.c_bf16 else 4
        self.a = DeviceBuffer(case.A.size * 2, off_a * 2).upload(case.A)
        self.b = DeviceBuffer(case.B.size * 2, off_b * 2).upload(case.B)
        self.c_bytes = (max(case.M - 1, 0) * case.ldc + case.N) * self.celt if case.M and case.N else 0
        self.c = DeviceBuffer(max(self.c_bytes, 4), off_c * self.celt)

    def run(self, gemm, variant: int, check: bool = True):
        import torch
        c = self.case
        gemm.run(self.a.ptr, self.b.ptr, self.c.ptr, c.M, c.N, c.K, c.lda, c.ldb, c.ldc, variant)
        torch.cuda.synchronize()
        if check:
            code, _ = gemm.device_status()
            assert code == 0, f"device status {code}"

    def result(self):
        """(values as fp32 (M,N), raw bits (M,N)); asserts guards and row padding untouched."""
        c = self.case
        assert self.a.guards_intact() and self.b.guards_intact() and self.c.guards_intact(), "guard band overwritten"
        if c.M == 0 or c.N == 0:
            return np.zeros((c.M, c.N), np.float32), np.zeros((c.M, c.N), np.uint32)
        raw = self.c.download()[:self.c_bytes]
        full = np.full(c.M * c.ldc * self.celt, POISON, dtype=np.uint8)
        full[:raw.size] = raw
        dt = np.uint16 if c.c_bf16 else np.uint32
        grid = full.view(dt).reshape(c.M, c.ldc)
        pad = grid[:, c.N:]
        poison = dt(0xA5A5) if c.c_bf16 else dt(0xA5A5A5A5)
        assert np.all(pad == poison), "padding between N and ldc was written"
        bits = np.ascontiguousarray(grid[:, :c.N])
        vals = gen.bf16_bits_to_f32(bits) if c.c_bf16 else bits.view(np.float32)
        return vals, bits


def assert_matches_oracle(case: gen.GemmCase, vals: np.ndarray, bits: np.ndarray, C_ref: np.ndarray, S: np.ndarray,
                          exact: bool, what: str = ""):
    """The parity gate.  exact: bit equality (integer-valued inputs).  Otherwise the error bound."""
    assert not np.isnan(vals).any(), f"{what}: NaN in C (padding or out-of-range data was consumed)"
    if exact:
        if case.c_bf16:
            want = orc.round_to_bf16(C_ref)
            bad = np.argwhere(bits != want)
        else:
            want = C_ref.astype(np.float32)
            assert np.array_equal(want.astype(np.float64), C_ref), "reference not exact in fp32"
            bad = np.argwhere(bits != want.view(np.uint32))
        assert bad.size == 0, f"{what}: {len(bad)} elements differ, first at {bad[0]}: " \
                              f"got {vals[tuple(bad[0])]} want {C_ref[tuple(bad[0])]}"
        return
    err = np.abs(vals.astype(np.float64) - C_ref)
    bound = orc.bound_bf16(case.K, S, C_ref) if case.c_bf16 else orc.bound_f32(case.K, S)
    bad = np.argwhere(err > bound)
    assert bad.size == 0, f"{what}: {len(bad)} elements outside the bound, first at {bad[0]}: " \
                          f"err {err[tuple(bad[0])]:.3e} bound {bound[tuple(bad[0])]:.3e}"


def integer_checksums_match(case: gen.GemmCase, vals: np.ndarray) -> bool:
    """Full-matrix property on integer inputs: 1^T C = (1^T A) B and C 1 = A (B 1), exact in int64."""
    a = gen.bf16_bits_to_f32(case.A[:, :case.K]).astype(np.int64)
    bs = gen.bf16_bits_to_f32(case.B[:, :(case.K if case.b_col_major else case.N)]).astype(np.int64)
    b = bs.T if case.b_col_major else bs                      # logical K x N
    c = np.rint(vals.astype(np.float64)).astype(np.int64)
    if not np.array_equal(c.astype(np.float64), vals.astype(np.float64)):
        return False
    col = a.sum(axis=0) @ b
    row = a @ b.sum(axis=1)
    return bool(np.array_equal(c.sum(axis=0), col) and np.array_equal(c.sum(axis=1), row))
