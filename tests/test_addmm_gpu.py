"""AddMM (C = A.B + bias, bias a bf16 row vector) through every rung, against the oracle plus the bias in fp64.

The paper's held-out plain-GEMM family (Appendix D) contains AddMM at 4096^3; here the fused bias epilogue is
checked on shapes that reach every epilogue of the library: direct, TMA store, swapped operands, cluster reduce,
split-K reduce, CTA pairs, repacked and gathered operands, K = 0.
"""
import dataclasses

import numpy as np
import pytest

from oracle import gemm_oracle as orc
from paper_2605_28213_b200 import inputs as gen
from tests import parity as P

pytestmark = pytest.mark.gpu

VARIANT_NAMES = ["naive", "tiled", "vectorized", "pipelined", "tcgen05", "mma_sync"]


@pytest.fixture(scope="module")
def kb():
    from paper_2605_28213_b200 import binding
    return binding


def run_addmm(kb, case, bias_bits, variant, workspace_bytes=0, pin=None):
    import torch
    dev = P.DeviceCase(case)
    bias = P.DeviceBuffer(bias_bits.size * 2, 2).upload(bias_bits)       # element-aligned only
    with kb.Gemm(0, b_col_major=case.b_col_major, c_bf16=case.c_bf16, workspace_bytes=workspace_bytes) as g:
        if pin is not None:
            g.set_plan(kb.klineage_gemm_plan_t(*pin), dev.a.ptr, dev.b.ptr, dev.c.ptr, case.M, case.N, case.K, case.lda,
                       case.ldb, case.ldc)
        g.run_addmm(dev.a.ptr, dev.b.ptr, bias.ptr, dev.c.ptr, case.M, case.N, case.K, case.lda, case.ldb,
                    case.ldc, variant)
        torch.cuda.synchronize()
        code, _ = g.device_status()
        kid = g.last_kernel_id()
    assert code == 0 and bias.guards_intact()
    vals, bits = dev.result()
    return vals, bits, kid


def reference(case, bias_bits, rows):
    C_ref, S = P.oracle_rows(case, rows)
    b = orc.bf16_bits_to_f64(bias_bits)[None, :]
    return C_ref + b, S + np.abs(b)


SHAPES = [  # (M, N, K, col, bf16 C, pads)
    (256, 256, 256, False, False, (0, 0, 0)),
    (300, 520, 200, True, True, (0, 0, 0)),
    (130, 263, 70, False, True, (1, 1, 1)),       # unaligned everything
    (16, 1024, 4096, False, False, (0, 0, 0)),    # skinny: cluster reduce on the tcgen05 rung
    (48, 700, 8192, True, False, (0, 0, 0)),      # swapped operands, split-K through the workspace
    (65, 520, 32768, False, True, (0, 0, 0)),     # 128-row tiles, split-K with row-block reduce
    (40, 50, 0, False, False, (0, 0, 3)),         # K == 0: C = bias
]


@pytest.mark.parametrize("variant", range(6), ids=VARIANT_NAMES)
def test_addmm_all_rungs(kb, variant):
    for idx, (M, N, K, col, bf, (pa, pb, pc)) in enumerate(SHAPES):
        if variant == 0 and K > 8192:
            continue
        Kg = max(K, 1)
        case = gen.make_case(M, N, Kg, seed=200 + idx, dist_a="integer", dist_b="integer", b_col_major=col, c_bf16=bf,
                             lda=Kg + pa, ldb=(Kg if col else N) + pb, ldc=N + pc, name=f"addmm{M}x{N}x{K}-int")
        case = dataclasses.replace(case, K=K)
        bias = gen.draw((1, N), "integer", 300 + idx, 2)[0]
        rows = np.arange(M)
        C_ref, S = reference(case, bias, rows)
        vals, bits, _ = run_addmm(kb, case, bias, variant)
        P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=True, what=f"{case.name} {VARIANT_NAMES[variant]}")
        if K == 0:
            continue
        case = gen.make_case(M, N, K, seed=200 + idx, dist_a="normal", dist_b="uniform", b_col_major=col, c_bf16=bf,
                             lda=K + pa, ldb=(K if col else N) + pb, ldc=N + pc, name=f"addmm{M}x{N}x{K}")
        bias = gen.draw((1, N), "normal", 300 + idx, 2, 3.0)[0]
        C_ref, S = reference(case, bias, rows)
        vals, bits, _ = run_addmm(kb, case, bias, variant)
        P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=False, what=f"{case.name} {VARIANT_NAMES[variant]}")


def test_addmm_large_tensor_core_paths(kb):
    """CTA-pair kernel, half-tile tail, gathered operands."""
    for idx, (M, N, K, variant, ws, flag) in enumerate([(2816, 2808, 2200, 4, 0, 32), (1500, 2100, 333, 4, 0, 0),
                                                        (1000, 1001, 999, 4, 4096, 1), (1000, 1001, 999, 5, 0, 0)]):
        for bf in (False, True):
            case = gen.make_case(M, N, K, seed=400 + idx, dist_a="integer", dist_b="integer", c_bf16=bf,
                                 lda=K, ldb=N, ldc=N, name=f"addmm-large{M}x{N}x{K}")
            bias = gen.draw((1, N), "integer", 500 + idx, 2)[0]
            rows = P.sample_rows(M)
            C_ref, S = reference(case, bias, rows)
            vals, bits, kid = run_addmm(kb, case, bias, variant, ws)
            P.assert_matches_oracle(case, vals[rows], bits[rows], C_ref, S, exact=True, what=case.name)
            if variant == 4 and flag:
                assert (kid - 400) & flag, (kid, flag)


@pytest.mark.parametrize("shape", [(256, 512, 8192, 0), (200, 700, 9000, 0), (130, 264, 12000, 1)],
                         ids=lambda s: "x".join(map(str, s[:3])))
def test_addmm_through_the_workspace_split(kb, shape):
    # few tiles, long K, K split through the workspace (pinned): the bias must be added once, by the
    # reduce - on its test-free path (whole rows of tiles inside an aligned C) and on the general one
    M, N, K, pad = shape
    for bf in (False, True):
        case = gen.make_case(M, N, K, seed=270, dist_a="integer", dist_b="integer", c_bf16=bf, ldc=N + pad,
                             name=f"addmm-split{M}x{N}x{K}")
        bias = gen.draw((1, N), "integer", 271, 2)[0]
        C_ref, S = reference(case, bias, np.arange(M))
        vals, bits, kid = run_addmm(kb, case, bias, 4, pin=(1, 6, 1))
        assert (kid - 400) & ~(3 | 64) == 4, kid
        P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=True, what=case.name)


@pytest.mark.parametrize("shape", [(256, 512, 8192, 0), (200, 700, 9000, 0), (130, 264, 12000, 1)],
                         ids=lambda s: "x".join(map(str, s[:3])))
def test_addmm_through_the_cluster_split(kb, shape):
    # the same shapes with the K splits of a tile as a cluster: the owner CTA of a block adds the bias once, after
    # the partial sums; TMA-stored and masked-store forms, the heuristic's own choice and pinned cluster sizes
    M, N, K, pad = shape
    for bf in (False, True):
        case = gen.make_case(M, N, K, seed=272, dist_a="integer", dist_b="integer", c_bf16=bf, ldc=N + pad,
                             name=f"addmm-csplit{M}x{N}x{K}")
        bias = gen.draw((1, N), "integer", 273, 2)[0]
        C_ref, S = reference(case, bias, np.arange(M))
        for pin in (None, (1, 2, 2), (1, 4, 2), (1, 8, 2)):
            vals, bits, kid = run_addmm(kb, case, bias, 4, pin=pin)
            assert (kid - 400) & ~(3 | 64) == (4 | 16), (kid, pin)
            P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=True, what=f"{case.name} {pin}")


def test_addmm_argument_errors(kb):
    import torch
    a = torch.zeros(64 * 64, dtype=torch.int16, device="cuda")
    c = torch.zeros(64 * 64, dtype=torch.float32, device="cuda")
    with kb.Gemm(0) as g:
        raw = lambda bias, cptr=c.data_ptr(): kb.klineage_gemm_run_addmm_raw(
            g._h, 64, 64, 64, a.data_ptr(), 64, a.data_ptr(), 64, bias, cptr, 64, 0, None)
        assert raw(None) == kb.KLINEAGE_ERR_INVALID_ARG
        assert raw(a.data_ptr() + 1) == kb.KLINEAGE_ERR_INVALID_ARG          # bf16 needs 2-byte alignment
        assert raw(c.data_ptr() + 8) == kb.KLINEAGE_ERR_INVALID_ARG          # bias overlaps C
        assert raw(a.data_ptr() + 2) == kb.KLINEAGE_OK
        torch.cuda.synchronize()


@pytest.mark.parametrize("bf", [False, True], ids=["f32", "bf16"])
@pytest.mark.parametrize("plan,shape", [((2, 1, 0, 0, 0), (600, 776, 136)),
                                        ((2, 1, 0, 0, 0, 0, 0, 3), (600, 776, 136)),        # 256-row tiles, one per pair
                                        ((2, 1, 0, 0, 0, 0, 0, 3), (2100, 2056, 200))],     # 81 of them: two for some pairs
                         ids=["512-row", "256-row", "256-row-two-rounds"])
def test_addmm_on_the_pair_kernel_full_width_tiles(kb, bf, plan, shape):
    # full-width tiles of the CTA-pair kernel hand the accumulator back before they stage and store, and a lane fetches
    # its bias values before the accumulator is complete: the bias must still reach every unit, for both output types
    # and both tile heights
    import torch
    M, N, K = shape
    for dist, exact in (("integer", True), ("normal", False)):
        case = gen.make_case(M, N, K, seed=260, dist_a=dist, dist_b=dist, c_bf16=bf, name=f"addmm-pair-{dist}")
        bias = gen.draw((1, N), dist, 261, 2)[0]
        C_ref, S = reference(case, bias, np.arange(M))
        dev = P.DeviceCase(case)
        bbuf = P.DeviceBuffer(bias.size * 2).upload(bias)
        with kb.Gemm(0, c_bf16=bf) as g:
            g.set_plan(kb.klineage_gemm_plan_t(*plan), dev.a.ptr, dev.b.ptr, dev.c.ptr, M, N, K, case.lda, case.ldb,
                       case.ldc)
            g.run_addmm(dev.a.ptr, dev.b.ptr, bbuf.ptr, dev.c.ptr, M, N, K, case.lda, case.ldb, case.ldc, 4)
            torch.cuda.synchronize()
            flags = g.last_kernel_id() - 400
            assert g.device_status()[0] == 0 and flags & 32 and bool(flags & 256) == (len(plan) == 8)
        vals, bits = dev.result()
        P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=exact, what=f"{case.name} bf16={bf}")
