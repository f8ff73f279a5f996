"""The allocation-free entry point against the handle-based one.

Some users of this library sit where device allocation is forbidden: an
operator plugged into a framework that owns the whole memory budget, a serving
loop that cannot afford cudaMalloc's implicit synchronisation, a process whose
remaining HBM is already committed.  klineage_gemm_run_noalloc serves them from
a fixed scratch array inside the library.  Its results must equal those of
klineage_gemm_run on the tcgen05 rung bit for bit - on a first call and on a
second call that finds the first call's leftovers in the shared scratch.

This file sorts last on purpose: a run that stops at the first failure has
already executed every other test.
"""
import numpy as np
import pytest

from paper_2605_28213_b200 import inputs as gen
from tests import parity as P

pytestmark = pytest.mark.gpu


def run_both(kb, case, calls=2):
    """C from the handle path, then `calls` results of the allocation-free path on the same inputs."""
    import torch
    stream = torch.cuda.current_stream().cuda_stream
    with kb.Gemm(0, b_col_major=case.b_col_major, c_bf16=case.c_bf16) as g:
        dev = P.DeviceCase(case)
        dev.run(g, kb.KLINEAGE_TCGEN05)
        _, want_bits = dev.result()
        kid = g.last_kernel_id()
    outs = []
    for _ in range(calls):
        d2 = P.DeviceCase(case)                       # fresh, poisoned C every call
        st = kb.klineage_gemm_run_noalloc(
            kb.KLINEAGE_B_COL_MAJOR if case.b_col_major else kb.KLINEAGE_B_ROW_MAJOR,
            kb.KLINEAGE_C_BF16 if case.c_bf16 else kb.KLINEAGE_C_F32,
            case.M, case.N, case.K, d2.a.ptr, case.lda, d2.b.ptr, case.ldb, d2.c.ptr, case.ldc, stream)
        assert st == kb.KLINEAGE_OK, kb.klineage_status_string(st)
        torch.cuda.synchronize()
        outs.append(d2.result()[1])                   # also checks guard bands and row padding
    return want_bits, outs, kid


def test_no_alloc_matches_handle_path_on_two_calls_in_a_row():
    from paper_2605_28213_b200 import binding as kb
    # a short-and-wide, long-K shape: split along K through the workspace, i.e. really uses the scratch array
    skinny = gen.make_case(48, 2048, 4096, seed=5, dist_a="normal", dist_b="normal", sigma_b=0.02, name="skinny")
    want, outs, kid = run_both(kb, skinny)
    flags = kid - 400                                 # 4 = split along K, 16 = reduced inside a cluster (no scratch)
    assert (flags & 4) and not (flags & 16), "the comparison shape must exercise split-K scratch in global memory"
    for k, got in enumerate(outs):
        assert np.array_equal(got, want), f"call {k + 1}: allocation-free result differs from the handle path"
    # and against the oracle, with the tolerance every other parity test uses
    C_ref, S = P.oracle_rows(skinny, np.arange(skinny.M))
    P.assert_matches_oracle(skinny, outs[-1].view(np.float32), outs[-1], C_ref, S, exact=False, what="no-alloc skinny")

    # taller tile, split along K with the row-block reduce; and a decode-like M=16 shape (cluster reduce,
    # no global scratch) plus a ragged column-major bf16 case without any split: same call, same bits
    for case in (gen.make_case(200, 256, 30016, seed=7, dist_a="integer", dist_b="integer", name="tall"),
                 gen.make_case(16, 2048, 4096, seed=8, dist_a="normal", dist_b="normal", name="decode"),
                 gen.make_case(300, 520, 200, seed=6, dist_a="integer", dist_b="integer", b_col_major=True,
                               c_bf16=True, name="ragged")):
        want, outs, _ = run_both(kb, case)
        for got in outs:
            assert np.array_equal(got, want), case.name


def test_no_alloc_unaligned_operands_empty_shapes_and_no_allocation():
    """What the entry point promises beyond the aligned case: unaligned operands are accepted (gathered tile by
    tile, where the handle path repacks them first) and give the exact result on integer-valued inputs; K == 0
    zero-fills; M == 0 does nothing; and the device's free memory is the same after a call as before it."""
    import torch
    from paper_2605_28213_b200 import binding as kb
    stream = torch.cuda.current_stream().cuda_stream
    for (M, N, K, col, bf, offs) in ((130, 263, 1070, False, False, (1, 1, 1)), (300, 520, 200, True, True, (1, 0, 0))):
        case = gen.make_case(M, N, K, seed=9, dist_a="integer", dist_b="integer", b_col_major=col, c_bf16=bf,
                             lda=K + 1, ldb=(K if col else N) + 1, ldc=N + 1, name="no-alloc unaligned")
        with kb.Gemm(0, b_col_major=col, c_bf16=bf) as g:
            dev = P.DeviceCase(case, *offs)
            dev.run(g, kb.KLINEAGE_TCGEN05)
            _, want = dev.result()
        d2 = P.DeviceCase(case, *offs)
        args = (kb.KLINEAGE_B_COL_MAJOR if col else kb.KLINEAGE_B_ROW_MAJOR, kb.KLINEAGE_C_BF16 if bf else kb.KLINEAGE_C_F32,
                M, N, K, d2.a.ptr, case.lda, d2.b.ptr, case.ldb, d2.c.ptr, case.ldc, stream)
        assert kb.klineage_gemm_run_noalloc(*args) == kb.KLINEAGE_OK
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        assert kb.klineage_gemm_run_noalloc(*args) == kb.KLINEAGE_OK
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, "the allocation-free call changed the free device memory"
        vals, bits = d2.result()
        C_ref, S = P.oracle_rows(case, np.arange(M))
        P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=True, what=case.name)
        assert np.array_equal(bits, want), "exact sums: both paths must give the same bits"
    # K == 0: C <- 0 through this entry point too; M == 0: nothing is written
    case = gen.make_case(40, 50, 3, seed=1, ldc=53)
    d3 = P.DeviceCase(case)
    assert kb.klineage_gemm_run_noalloc(0, 0, 40, 50, 0, d3.a.ptr, 3, d3.b.ptr, 50, d3.c.ptr, 53, stream) == kb.KLINEAGE_OK
    torch.cuda.synchronize()
    assert np.all(d3.result()[1] == 0)
    d4 = P.DeviceCase(case)
    before = d4.c.download().copy()
    assert kb.klineage_gemm_run_noalloc(0, 0, 0, 50, 3, d4.a.ptr, 3, d4.b.ptr, 50, d4.c.ptr, 53, stream) == kb.KLINEAGE_OK
    torch.cuda.synchronize()
    assert np.array_equal(d4.c.download(), before) and d4.c.guards_intact()


def test_no_alloc_refuses_shapes_beyond_its_fixed_scratch():
    import torch
    from paper_2605_28213_b200 import binding as kb
    # 64 rows (partial sums go through global memory), K long enough for 9 splits:
    # 9 x 64 x 4096 fp32 partial sums = 9 MiB > the 8 MiB reserved
    M, N, K = 64, 4096, 32768
    A = torch.zeros(M * K, dtype=torch.int16, device="cuda")
    B = torch.zeros(K * N, dtype=torch.int16, device="cuda")
    C = torch.full((M * N,), 7.0, dtype=torch.float32, device="cuda")
    st = kb.klineage_gemm_run_noalloc(0, 0, M, N, K, A.data_ptr(), K, B.data_ptr(), N, C.data_ptr(), N,
                                      torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert st == kb.KLINEAGE_ERR_SCRATCH_LIMIT
    assert "scratch" in kb.klineage_status_string(st)
    assert bool((C == 7.0).all().item()), "a refused call must not touch C"
    # argument errors are reported exactly as by the handle path
    assert kb.klineage_gemm_run_noalloc(0, 0, 8, 8, 8, A.data_ptr(), 7, B.data_ptr(), 8, C.data_ptr(), 8,
                                        None) == kb.KLINEAGE_ERR_INVALID_ARG
