"""klineage_gemm_run_host: the product with A, B and C in HOST memory, copies and row-slab kernels overlapped inside the
library.  Same parity gate as the device call (bit-exact on integer inputs, the error bound on random ones), on every
rung; the device scratch starts as NaN patterns and the host C as poison, so a pad column consumed or a byte outside
the M x N block written shows up."""
import numpy as np
import pytest

from paper_2605_28213_b200 import inputs as gen
from tests import parity as P

pytestmark = pytest.mark.gpu

POISON16, POISON32 = 0xA5A5, 0xA5A5A5A5


@pytest.fixture(scope="module")
def kb():
    from paper_2605_28213_b200 import binding
    return binding


def run_host(kb, case, variant, pinned=True, extra_scratch=0):
    """Returns (vals, bits, launches, kernel id) of one run_host call on freshly poisoned buffers."""
    import torch
    dt = torch.int16 if case.c_bf16 else torch.int32
    hA = torch.from_numpy(case.A.view(np.int16).copy())
    hB = torch.from_numpy(case.B.view(np.int16).copy())
    hC = torch.full((case.M, case.ldc), POISON16 - 65536 if case.c_bf16 else POISON32 - (1 << 32), dtype=dt)
    if pinned:
        hA, hB, hC = hA.pin_memory(), hB.pin_memory(), hC.pin_memory()
    with kb.Gemm(0, b_col_major=case.b_col_major, c_bf16=case.c_bf16) as g:
        need = g.host_scratch_bytes(case.M, case.N, case.K)
        scratch = torch.full((need + extra_scratch,), 0xFF, dtype=torch.uint8, device="cuda")     # bf16 0xFFFF = NaN
        assert scratch.data_ptr() % 256 == 0
        a_before, b_before = hA.clone(), hB.clone()
        g.run_host(hA, hB, hC, case.M, case.N, case.K, case.lda, case.ldb, case.ldc, scratch, need + extra_scratch,
                   variant)
        torch.cuda.current_stream().synchronize()         # the call's own stream: everything must be done by now
        code, _ = g.device_status()
        assert code == 0
        launches, kid = g.last_launch_count(), g.last_kernel_id()
    assert torch.equal(hA, a_before) and torch.equal(hB, b_before), "a host operand was modified"
    grid = hC.numpy().view(np.uint16 if case.c_bf16 else np.uint32)
    assert np.all(grid[:, case.N:] == (POISON16 if case.c_bf16 else POISON32)), "host padding of C was written"
    bits = np.ascontiguousarray(grid[:, :case.N])
    vals = gen.bf16_bits_to_f32(bits) if case.c_bf16 else bits.view(np.float32)
    return vals, bits, launches, kid


CASES = [  # M, N, K, col, bf16, pads (a, b, c)
    (300, 520, 200, False, False, (0, 0, 0)),      # one slab
    (1300, 333, 257, False, True, (3, 5, 1)),      # 3 slabs (512, 512, 276), odd pitches on the host
    (1300, 333, 257, True, False, (1, 0, 7)),      # column-major B
    (2100, 264, 72, False, True, (0, 0, 0)),       # 5 slabs of 512 rows (last: 52)
    (64, 1000, 999, True, True, (0, 2, 0)),        # a single short slab
]


@pytest.mark.parametrize("variant", [0, 1, 2, 3, 5, 4], ids=["naive", "tiled", "vectorized", "pipelined", "mma_sync",
                                                              "tcgen05"])
def test_host_operands_every_rung(kb, variant):
    for idx, (M, N, K, col, bf, (pa, pb, pc)) in enumerate(CASES):
        for dist, exact in (("integer", True), ("normal", False)):
            case = gen.make_case(M, N, K, seed=600 + idx, dist_a=dist, dist_b=dist, b_col_major=col, c_bf16=bf,
                                 lda=K + pa, ldb=(K if col else N) + pb, ldc=N + pc, name=f"host{M}x{N}x{K}-{dist}")
            C_ref, S = P.oracle_rows(case, np.arange(M))
            vals, bits, launches, kid = run_host(kb, case, variant)
            P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=exact, what=f"{case.name} v{variant}")
            assert launches == -(-M // 512) and kid // 100 == variant, (launches, kid)


def test_pageable_memory_and_larger_scratch(kb):
    case = gen.make_case(1100, 400, 300, seed=610, dist_a="integer", dist_b="integer", c_bf16=True, name="host-pageable")
    C_ref, S = P.oracle_rows(case, np.arange(case.M))
    vals, bits, _, _ = run_host(kb, case, 4, pinned=False, extra_scratch=4096)
    P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=True, what=case.name)


def test_many_rows_use_sixteen_slabs(kb):
    # 16 x 640 rows would be 10240: slabs grow beyond 512 rows once M > 8192
    case = gen.make_case(9000, 136, 72, seed=611, dist_a="integer", dist_b="integer", c_bf16=False, name="host-tall")
    rows = P.sample_rows(case.M)
    C_ref, S = P.oracle_rows(case, rows)
    vals, bits, launches, _ = run_host(kb, case, 4)
    assert launches == -(-9000 // 640)               # 640-row slabs: 15 of them
    P.assert_matches_oracle(case, vals[rows], bits[rows], C_ref, S, exact=True, what=case.name)
    assert P.integer_checksums_match(case, vals)


def test_k_zero_clears_the_host_matrix_and_empty_shapes_do_nothing(kb):
    import torch
    with kb.Gemm(0) as g:
        hC = torch.full((70, 33), 7.0).pin_memory()
        need = g.host_scratch_bytes(70, 33, 0)
        scratch = torch.empty(need, dtype=torch.uint8, device="cuda")
        g.run_host(None, None, hC, 70, 33, 0, 8, 33, 33, scratch, need, 4)
        torch.cuda.synchronize()
        assert torch.count_nonzero(hC) == 0
        hC.fill_(7.0)
        g.run_host(None, None, hC, 0, 33, 5, 5, 33, 33, None, 0, 4)
        g.run_host(None, None, hC, 70, 0, 5, 5, 1, 1, None, 0, 4)
        torch.cuda.synchronize()
        assert torch.all(hC == 7.0) and g.last_launch_count() == 0


def test_scratch_rules(kb):
    import torch
    M, N, K = 200, 96, 64
    a = torch.zeros((M, K), dtype=torch.int16).pin_memory()
    b = torch.zeros((K, N), dtype=torch.int16).pin_memory()
    c = torch.zeros((M, N), dtype=torch.float32).pin_memory()
    with kb.Gemm(0) as g:
        need = g.host_scratch_bytes(M, N, K)
        scratch = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
        raw = lambda ptr, nbytes, variant=4: kb.klineage_gemm_run_host_raw(
            g._h, M, N, K, a.data_ptr(), K, b.data_ptr(), N, c.data_ptr(), N, ptr, nbytes, variant, None)
        assert raw(None, need) == kb.KLINEAGE_ERR_INVALID_ARG
        assert raw(scratch.data_ptr(), need - 1) == kb.KLINEAGE_ERR_INVALID_ARG
        assert raw(scratch.data_ptr() + 16, need) == kb.KLINEAGE_ERR_INVALID_ARG        # 256-byte alignment
        assert raw(scratch.data_ptr(), need, 9) == kb.KLINEAGE_ERR_BAD_VARIANT
        assert kb.klineage_gemm_run_host_raw(g._h, M, N, K, a.data_ptr(), K - 1, b.data_ptr(), N, c.data_ptr(), N,
                                             scratch.data_ptr(), need, 4, None) == kb.KLINEAGE_ERR_INVALID_ARG
        assert kb.klineage_gemm_run_host_raw(g._h, M, N, K, a.data_ptr(), K, b.data_ptr(), N, a.data_ptr(), N,
                                             scratch.data_ptr(), need, 4, None) == kb.KLINEAGE_ERR_INVALID_ARG  # C over A
        assert raw(scratch.data_ptr(), need) == kb.KLINEAGE_OK
        torch.cuda.synchronize()
        assert g.device_status()[0] == 0


def test_back_to_back_calls_share_scratch_in_stream_order(kb):
    # two different products through ONE scratch buffer on one stream, no host synchronisation in between: the
    # second call's copies must wait for the first call's last copy back
    import torch
    c1 = gen.make_case(700, 264, 136, seed=620, dist_a="integer", dist_b="integer", c_bf16=False, name="host-seq1")
    c2 = gen.make_case(640, 200, 264, seed=621, dist_a="integer", dist_b="integer", c_bf16=False, name="host-seq2")
    with kb.Gemm(0) as g:
        need = max(g.host_scratch_bytes(c.M, c.N, c.K) for c in (c1, c2))
        scratch = torch.empty(need, dtype=torch.uint8, device="cuda")
        host = []
        for c in (c1, c2):
            host.append((torch.from_numpy(c.A.view(np.int16).copy()).pin_memory(),
                         torch.from_numpy(c.B.view(np.int16).copy()).pin_memory(),
                         torch.zeros((c.M, c.ldc), dtype=torch.float32).pin_memory()))
        for _ in range(3):
            for c, (hA, hB, hC) in zip((c1, c2), host):
                g.run_host(hA, hB, hC, c.M, c.N, c.K, c.lda, c.ldb, c.ldc, scratch, need, 4)
        torch.cuda.current_stream().synchronize()
        assert g.device_status()[0] == 0
    for c, (_, _, hC) in zip((c1, c2), host):
        C_ref, S = P.oracle_rows(c, np.arange(c.M))
        vals = hC.numpy()[:, :c.N]
        P.assert_matches_oracle(c, vals, np.ascontiguousarray(vals).view(np.uint32), C_ref, S, exact=True, what=c.name)
