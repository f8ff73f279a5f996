"""Multi-destination epilogue (fused all-gather of a column-partitioned GEMM), emulated on one GPU: every "rank" has
its own full-width C buffer on the same device, runs its column slice and stores it into all of them.  After all
ranks ran, every C must equal the oracle's A.B, and nothing outside the matrices may have been written."""
import numpy as np
import pytest

from paper_2605_28213_b200 import inputs as gen
from paper_2605_28213_b200 import npart
from tests import parity as P

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kb():
    from paper_2605_28213_b200 import binding
    return binding


def run_world(kb, case, world, variant, quantum=8, expect_one_launch=None, expect_pair=None):
    import torch
    celt = 2 if case.c_bf16 else 4
    a = P.DeviceBuffer(case.A.size * 2).upload(case.A)
    c_bytes = ((case.M - 1) * case.ldc + case.N) * celt
    cs = [P.DeviceBuffer(c_bytes) for _ in range(world)]
    with kb.Gemm(0, b_col_major=case.b_col_major, c_bf16=case.c_bf16) as g:
        for rank in range(world):
            part = npart.NPartitionedGemm(g, world, rank, case.N, [c.ptr for c in cs], case.ldc, quantum)
            if part.n_local == 0:
                continue
            if case.b_col_major:                    # B stored N x ldb: the slice is a row range
                Bs = np.ascontiguousarray(case.B[part.n0:part.n1])
                ldb = case.ldb
            else:                                   # B stored K x ldb: the slice is a column range, repitched
                ldb = (part.n_local + 7) // 8 * 8 if case.ldb % 8 == 0 else part.n_local
                Bs = np.full((case.K, ldb), 0x7FC0, np.uint16)
                Bs[:, :part.n_local] = case.B[:, part.n0:part.n1]
            b = P.DeviceBuffer(Bs.size * 2).upload(Bs)
            if expect_pair:             # pin the CTA-pair kernel for this rank's slice (short K would take the other kernel)
                g.set_plan(kb.klineage_gemm_plan_t(2, 1, 0, 0, 0), a.ptr, b.ptr, part.dst[0], case.M, part.n_local, case.K,
                           case.lda, ldb, case.ldc)
            part.run(a.ptr, b.ptr, case.M, case.K, case.lda, ldb, variant)
            torch.cuda.synchronize()
            code, _ = g.device_status()
            assert code == 0 and b.guards_intact()
            if expect_one_launch is not None:
                assert (g.last_launch_count() == 1) == expect_one_launch, g.last_launch_count()
            if expect_pair is not None:
                assert bool((g.last_kernel_id() - 400) & 32) == expect_pair, g.last_kernel_id()
    assert a.guards_intact()
    C_ref, S = P.oracle_rows(case, np.arange(case.M))
    dt = np.uint16 if case.c_bf16 else np.uint32
    poison = dt(0xA5A5) if case.c_bf16 else dt(0xA5A5A5A5)
    for k, c in enumerate(cs):
        assert c.guards_intact(), f"guard band of rank {k}'s C overwritten"
        raw = c.download()
        full = np.full(case.M * case.ldc * celt, P.POISON, np.uint8)
        full[:raw.size] = raw
        grid = full.view(dt).reshape(case.M, case.ldc)
        assert np.all(grid[:, case.N:] == poison), "row padding written"
        bits = np.ascontiguousarray(grid[:, :case.N])
        vals = gen.bf16_bits_to_f32(bits) if case.c_bf16 else bits.view(np.float32)
        yield k, vals, bits, C_ref, S


CASES = [  # (M, N, K, col, bf16, world, ldc pad, quantum, one launch?, pair?)
    (300, 2048, 136, False, True, 4, 0, 8, True, False),        # aligned slices: TMA stores to every destination
    (300, 1000, 136, False, False, 3, 0, 8, True, False),       # 336 / 336 / 328 columns: ragged tiles
    (260, 1001, 72, True, True, 3, 3, 1, True, False),          # unaligned slices and pitch: masked direct stores
    (2100, 8192, 72, False, True, 2, 8, 8, True, True),         # 5 x 16 tiles of 512 x 256 per rank: the pair kernel
    (16, 2048, 1024, False, False, 2, 0, 8, None, False),       # skinny orientation: compute into C_0, then copies
]


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: f"{c[0]}x{c[1]}x{c[2]}-w{c[5]}")
def test_every_rank_ends_with_the_full_product(kb, cfg):
    M, N, K, col, bf, world, pad, q, one, pair = cfg
    for dist, exact in (("integer", True), ("normal", False)):
        case = gen.make_case(M, N, K, seed=160, dist_a=dist, dist_b=dist, b_col_major=col, c_bf16=bf, ldc=N + pad,
                             name=f"npart{M}x{N}x{K}-{dist}")
        first = None
        for k, vals, bits, C_ref, S in run_world(kb, case, world, 4, q, one, pair):
            P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=exact, what=f"{case.name} C of rank {k}")
            if first is None:
                first = bits
            assert np.array_equal(bits, first), f"rank {k}'s C differs from rank 0's"


@pytest.mark.parametrize("variant", [0, 1, 2, 3, 5])
def test_lower_rungs_compute_once_and_copy(kb, variant):
    case = gen.make_case(140, 200, 72, seed=170, dist_a="integer", dist_b="integer", c_bf16=True, ldc=203,
                         name="npart-low")
    for k, vals, bits, C_ref, S in run_world(kb, case, 3, variant, 8, expect_one_launch=True):
        P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=True, what=f"variant {variant} C of rank {k}")


def test_multi_dst_argument_rules(kb):
    case = gen.make_case(64, 64, 64, seed=171, dist_a="integer", dist_b="integer", name="md-args")
    dev = P.DeviceCase(case)
    other = P.DeviceBuffer(64 * 64 * 4)
    with kb.Gemm(0) as g:
        raw = lambda Cs, ldcs: kb.klineage_gemm_run_multi_dst_raw(g._h, 64, 64, 64, dev.a.ptr, 64, dev.b.ptr, 64, Cs,
                                                                  ldcs, 4, None)
        assert raw([dev.c.ptr, dev.c.ptr + 64], [64, 64]) == kb.KLINEAGE_ERR_INVALID_ARG     # destinations overlap
        assert raw([dev.c.ptr, dev.a.ptr], [64, 64]) == kb.KLINEAGE_ERR_INVALID_ARG          # a destination aliases A
        assert raw([dev.c.ptr, other.ptr], [64, 63]) == kb.KLINEAGE_ERR_INVALID_ARG
        assert raw([dev.c.ptr] * 17, [64] * 17) == kb.KLINEAGE_ERR_INVALID_ARG
        assert raw([dev.c.ptr, other.ptr], [64, 64]) == kb.KLINEAGE_OK
        import torch
        torch.cuda.synchronize()
    vals, bits = dev.result()
    C_ref, S = P.oracle_rows(case, np.arange(64))
    P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=True, what="destination 0")
    assert np.array_equal(other.download().view(np.uint32).reshape(64, 64), bits) and other.guards_intact()
