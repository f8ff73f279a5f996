"""Launch plans and the autotuner of the tcgen05 rung (paper, Table 1: `templatize` / `autotune`).

Every candidate plan of a shape is pinned in turn and must reproduce the oracle: bit for bit on integer-valued
inputs, within the error bound on random ones; candidates that do not split K must also agree with one another bit
for bit on random inputs (same products, same summation order).  The autotuner must pin one of the candidates, the
pinned plan must be the one later calls run, and plans that cannot run a shape must be refused.
"""
import numpy as np
import pytest

from paper_2605_28213_b200 import inputs as gen
from tests import parity as P

pytestmark = pytest.mark.gpu

SHAPES = [  # (M, N, K, col, bf16 C)
    (1100, 1300, 520, False, True),      # pair kernel possible; ragged everywhere
    (640, 768, 1024, True, False),       # few tiles: K splits through the workspace are candidates
    (16, 2048, 4096, False, False),      # skinny: cluster and workspace splits
    (48, 1024, 4096, True, True),        # skinny without the cluster option (M > 32)
    (300, 2100, 260, False, False),      # pitch of A and B not a multiple of 8 elements: repacked operands
]


@pytest.fixture(scope="module")
def kb():
    from paper_2605_28213_b200 import binding
    return binding


def shape_args(case, dev):
    return (dev.a.ptr, dev.b.ptr, dev.c.ptr, case.M, case.N, case.K, case.lda, case.ldb, case.ldc)


def run_plan(kb, g, case, dev, plan):
    import torch
    g.set_plan(plan, *shape_args(case, dev))
    got, pinned = g.get_plan(*shape_args(case, dev))
    assert pinned and got.as_tuple() == plan.as_tuple()
    dev.run(g, kb.KLINEAGE_TCGEN05)
    torch.cuda.synchronize()
    kid = g.last_kernel_id()
    vals, bits = dev.result()
    g.set_plan(None, *shape_args(case, dev))
    assert g.get_plan(*shape_args(case, dev))[1] is False
    return vals, bits, kid


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s[:3])))
def test_every_candidate_plan_matches_the_oracle(kb, shape):
    M, N, K, col, bf = shape
    rows = np.arange(M)
    for integer in (True, False):
        dist = "integer" if integer else "normal"
        case = gen.make_case(M, N, K, seed=41, dist_a=dist, dist_b=dist, b_col_major=col, c_bf16=bf,
                             name=f"plan{M}x{N}x{K}-{dist}")
        C_ref, S = P.oracle_rows(case, rows)
        dev = P.DeviceCase(case)
        with kb.Gemm(0, b_col_major=col, c_bf16=bf) as g:
            plans = g.plan_candidates(*shape_args(case, dev))
            assert len(plans) >= 2 and not any(plans[0].as_tuple())
            assert len({p.as_tuple() for p in plans}) == len(plans), "duplicate candidates"
            unsplit = {}
            kernels = set()
            for plan in plans:
                vals, bits, kid = run_plan(kb, g, case, dev, plan)
                P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=integer, what=f"{case.name} {plan}")
                flags = kid - 400
                assert 0 <= flags < 512, kid
                kernels.add(bool(flags & 32))
                if plan.kernel == 2:
                    assert flags & 32, f"{plan} ran kernel {kid}"
                    assert bool(flags & 128) == (plan.split_via == 3), f"{plan} ran kernel {kid}"
                    assert bool(flags & 256) == (plan.stages == 3), f"{plan} ran kernel {kid}"
                if plan.kernel == 1:
                    assert not flags & 32, f"{plan} ran kernel {kid}"
                if plan.splits > 1:
                    assert flags & 4, f"{plan} ran kernel {kid}"
                    assert bool(flags & 16) == (plan.split_via == 2), f"{plan} ran kernel {kid}"
                if plan.splits == 1:
                    assert not flags & 4, f"{plan} ran kernel {kid}"
                    unsplit[plan.as_tuple()] = bits
            if not integer and len(unsplit) > 1:
                first = next(iter(unsplit.values()))
                for key, bits in unsplit.items():
                    assert np.array_equal(bits, first), f"unsplit plan {key} differs bitwise from another unsplit plan"
            if M > 128 and case.lda % 8 == 0 and case.ldb % 8 == 0:
                assert kernels == {True, False}, "both kernels must be among the candidates"


def test_autotune_pins_a_candidate_and_later_calls_use_it(kb):
    import torch
    M, N, K, col, bf = 1100, 1300, 520, False, True
    case = gen.make_case(M, N, K, seed=43, dist_a="integer", dist_b="integer", b_col_major=col, c_bf16=bf,
                         name="tune-int")
    C_ref, S = P.oracle_rows(case, np.arange(M))
    dev = P.DeviceCase(case)
    with kb.Gemm(0, b_col_major=col, c_bf16=bf) as g:
        args = shape_args(case, dev)
        plans = {p.as_tuple() for p in g.plan_candidates(*args)}
        best, best_us, heur_us = g.autotune(*args, iters=5)
        torch.cuda.synchronize()
        assert best.as_tuple() in plans
        assert 0.0 < best_us <= heur_us
        if any(best.as_tuple()):
            assert best_us <= 0.99 * heur_us, "a non-default plan must beat the heuristic by more than the noise"
        got, pinned = g.get_plan(*args)
        assert pinned and got.as_tuple() == best.as_tuple()
        vals, bits = dev.result()                  # autotune leaves C computed by the pinned plan
        P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=True, what="after autotune")
        kid_tuned = g.last_kernel_id()
        dev.run(g, kb.KLINEAGE_TCGEN05)
        assert g.last_kernel_id() == kid_tuned
        vals, bits = dev.result()
        P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=True, what="run after autotune")
        # another shape on the same handle is not affected by the pin
        other = gen.make_case(200, 264, 136, seed=44, dist_a="integer", dist_b="integer", b_col_major=col, c_bf16=bf,
                              name="tune-other")
        odev = P.DeviceCase(other)
        assert g.get_plan(*shape_args(other, odev))[1] is False
        odev.run(g, kb.KLINEAGE_TCGEN05)
        vals, bits = odev.result()
        C2, S2 = P.oracle_rows(other, np.arange(other.M))
        P.assert_matches_oracle(other, vals, bits, C2, S2, exact=True, what="other shape")


def test_plans_that_cannot_run_are_refused(kb):
    case = gen.make_case(300, 520, 260, seed=45, dist_a="integer", dist_b="integer", name="refuse")   # pitches 260, 520
    dev = P.DeviceCase(case)
    Plan = kb.klineage_gemm_plan_t
    with kb.Gemm(0) as g:
        args = shape_args(case, dev)
        raw = lambda plan: kb.klineage_gemm_set_plan_raw(g._h, case.M, case.N, case.K, dev.a.ptr, case.lda, dev.b.ptr,
                                                         case.ldb, dev.c.ptr, case.ldc, plan)
        bad = [Plan(2, 1, 0, 0, 0),      # pair kernel: pitch of A (260 elements) is not 16-byte aligned
               Plan(1, 9, 1, 0, 0),      # 9 splits of 5 k-blocks
               Plan(1, 3, 2, 0, 0),      # a cluster reduce runs in 2, 4 or 8 CTAs
               Plan(1, 1, 0, 0, 0, 96),  # tile widths are multiples of 64 columns
               Plan(1, 1, 0, 0, 0, 0, 0, 5),   # ring depths: 0 (automatic), 4 or 6
               Plan(3, 0, 0, 0, 0), Plan(0, -1, 0, 0, 0), Plan(0, 0, 3, 0, 0), Plan(0, 0, 0, 0, 3)]
        for plan in bad:
            assert raw(plan) == kb.KLINEAGE_ERR_INVALID_ARG, plan
            assert g.get_plan(*args)[1] is False
        assert raw(Plan(1, 2, 1, 8, 0)) == kb.KLINEAGE_OK
        dev.run(g, kb.KLINEAGE_TCGEN05)
        vals, bits = dev.result()
        C_ref, S = P.oracle_rows(case, np.arange(case.M))
        P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=True, what="2 splits pinned")
        assert (g.last_kernel_id() - 400) & 4
