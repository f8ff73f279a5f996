"""GPU parity: every lineage rung, through the C ABI, against the CPU oracle.

Bit-exact on integer-valued inputs; within K * 2^-23 * (|A|.|B|)_ij on random
bf16 inputs (fp32 C), widened by one bf16 rounding for bf16 C.  The paper's own
gate is a correctness check with three random seeds (Evaluation, Setup); seeds 1..3 are
used on the small configurations.
"""
import numpy as np
import pytest

from paper_2605_28213_b200 import inputs as gen
from tests import parity as P

pytestmark = pytest.mark.gpu

VARIANT_NAMES = ["naive", "tiled", "vectorized", "pipelined", "tcgen05", "mma_sync"]
VARIANTS = list(range(6))


@pytest.fixture(scope="module")
def kb():
    from paper_2605_28213_b200 import binding
    return binding


@pytest.fixture(scope="module")
def handles(kb):
    """One handle per (B layout, C dtype)."""
    hs = {(col, bf): kb.Gemm(0, b_col_major=col, c_bf16=bf) for col in (False, True) for bf in (False, True)}
    yield hs
    for h in hs.values():
        h.close()


@pytest.fixture(scope="module")
def handles_tiny_ws(kb):
    """Handles whose workspace is too small for operand repacking or split-K partials: on the tcgen05 rung
    unaligned operands then go through the generic-proxy producers."""
    hs = {(col, bf): kb.Gemm(0, b_col_major=col, c_bf16=bf, workspace_bytes=4096)
          for col in (False, True) for bf in (False, True)}
    yield hs
    for h in hs.values():
        h.close()


def run_and_check(handles, case, variant, C_ref=None, S=None, rows=None, exact=False, offsets=(0, 0, 0), pin=None):
    """pin: a launch plan (kernel, splits, split_via, group_m, half_tail) pinned for this shape during the call."""
    dev = P.DeviceCase(case, *offsets)
    g = handles[(case.b_col_major, case.c_bf16)]
    shape = (dev.a.ptr, dev.b.ptr, dev.c.ptr, case.M, case.N, case.K, case.lda, case.ldb, case.ldc)
    if pin is not None:
        from paper_2605_28213_b200 import binding as kb
        g.set_plan(kb.klineage_gemm_plan_t(*pin), *shape)
    try:
        dev.run(g, variant)
    finally:
        if pin is not None:
            g.set_plan(None, *shape)
    vals, bits = dev.result()
    if C_ref is None:
        rows = np.arange(case.M)
        C_ref, S = P.oracle_rows(case, rows)
    P.assert_matches_oracle(case, vals[rows], bits[rows], C_ref, S, exact,
                            f"{case.name} {VARIANT_NAMES[variant]}")
    return vals, bits


# ------------------------------------------------------------------ the five configurations
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_NAMES)
@pytest.mark.parametrize("name,seeds", [("c1", (1, 2, 3)), ("c2", (1, 2, 3)), ("c2pad", (1, 2, 3)), ("c5", (1, 2, 3)),
                                        ("c3", (1, 2, 3)), ("c4", (1, 2, 3))])
def test_config_random_within_bound(handles, variant, name, seeds):
    # three seeds everywhere (the paper's gate); at 4096^3 and 8192^3 the rungs without tensor cores, which take up to a
    # second per run there, keep to the first seed
    if name in ("c3", "c4") and variant not in (4, 5):
        seeds = seeds[:1]
    for seed in seeds:
        case, rows, C_ref, S = P.cached_reference(name, seed, False)
        run_and_check(handles, case, variant, C_ref, S, rows)


@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_NAMES)
@pytest.mark.parametrize("name", ["c1", "c2", "c2pad", "c5", "c3", "c4"])
def test_config_integer_bit_exact(handles, variant, name):
    case, rows, C_ref, S = P.cached_reference(name, 2, True)
    vals_a, _ = run_and_check(handles, case, variant, C_ref, S, rows, exact=True)
    # the other output dtype, plus the full-matrix checksum on whichever result is fp32
    import dataclasses
    other = dataclasses.replace(case, c_bf16=not case.c_bf16)
    vals_b, _ = run_and_check(handles, other, variant, C_ref, S, rows, exact=True)
    f32_vals = vals_b if case.c_bf16 else vals_a
    assert P.integer_checksums_match(case, f32_vals), "row/column checksums of the full matrix differ"


# ------------------------------------------------------------------ adversarial shapes
EDGE = [1, 2, 7, 8, 9, 15, 16, 17, 63, 64, 65, 127, 128, 129, 255, 257]
ADVERSARIAL = [(1, 1, 1), (1, 1, 257), (2, 7, 8), (7, 2, 9), (8, 9, 15), (9, 8, 16), (15, 17, 17), (16, 16, 63),
               (17, 15, 64), (63, 65, 65), (64, 64, 127), (65, 63, 128), (127, 129, 129), (128, 128, 255),
               (129, 127, 257), (255, 257, 1), (257, 255, 2), (1, 257, 129), (257, 1, 127), (130, 260, 70),
               (300, 520, 200), (16, 700, 1030), (5, 33, 4100)]


@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_NAMES)
@pytest.mark.parametrize("col", [False, True], ids=["Brow", "Bcol"])
def test_adversarial_shapes(handles, variant, col):
    assert all(d in EDGE or d > 257 for s in ADVERSARIAL[:19] for d in s)
    for idx, (M, N, K) in enumerate(ADVERSARIAL):
        for bf in (False, True):
            # integer values: bit-exact, catches any dropped / duplicated / mis-indexed product
            ci = gen.make_case(M, N, K, seed=idx, dist_a="integer", dist_b="integer", b_col_major=col, c_bf16=bf,
                               name=f"adv{M}x{N}x{K}-int")
            run_and_check(handles, ci, variant, exact=True)
        cr = gen.make_case(M, N, K, seed=idx, dist_a="normal", dist_b="uniform", b_col_major=col, c_bf16=False,
                           name=f"adv{M}x{N}x{K}")
        run_and_check(handles, cr, variant)


@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_NAMES)
@pytest.mark.parametrize("col", [False, True], ids=["Brow", "Bcol"])
def test_unaligned_bases_and_padded_leading_dimensions(handles, variant, col):
    shapes = [(130, 136, 72), (67, 250, 129), (256, 264, 64)]
    for idx, (M, N, K) in enumerate(shapes):
        for (pa, pb, pc), offs in [((0, 0, 0), (1, 1, 1)), ((8, 8, 8), (0, 0, 0)), ((3, 5, 7), (1, 3, 1)),
                                   ((8, 16, 4), (8, 8, 4)), ((8, 8, 8), (0, 1, 0)), ((8, 8, 8), (0, 0, 1))]:
            for bf in (False, True):
                case = gen.make_case(M, N, K, seed=100 + idx, dist_a="integer", dist_b="integer", lda=K + pa,
                                     ldb=(K if col else N) + pb, ldc=N + pc, b_col_major=col, c_bf16=bf,
                                     name=f"ld{M}x{N}x{K}+{pa},{pb},{pc}@{offs}")
                run_and_check(handles, case, variant, exact=True, offsets=offs)


@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_NAMES)
def test_random_small_shapes(handles, variant):
    rng = np.random.default_rng(1234 + variant)
    for it in range(24):
        M, N, K = (int(rng.integers(1, 400)) for _ in range(3))
        col, bf = bool(rng.integers(2)), bool(rng.integers(2))
        pa, pb, pc = (int(rng.integers(0, 9)) for _ in range(3))
        case = gen.make_case(M, N, K, seed=it, dist_a="uniform", dist_b="normal", lda=K + pa,
                             ldb=(K if col else N) + pb, ldc=N + pc, b_col_major=col, c_bf16=bf, name=f"rnd{it}")
        run_and_check(handles, case, variant, offsets=tuple(int(rng.integers(0, 3)) for _ in range(3)))


# ------------------------------------------------------------------ generic-proxy producers of the top rung
@pytest.mark.parametrize("col", [False, True], ids=["Brow", "Bcol"])
def test_tcgen05_generic_producers(handles_tiny_ws, col):
    """With no room to repack, unaligned operands are gathered tile by tile into the swizzled layout."""
    shapes = [(1000, 1001, 999, (0, 0, 0)), (130, 270, 100, (1, 1, 1)), (16, 1001, 2051, (1, 0, 1)),
              (300, 520, 200, (1, 1, 0)), (64, 64, 64, (1, 1, 1)), (257, 513, 129, (0, 1, 0))]
    for idx, (M, N, K, offs) in enumerate(shapes):
        for bf in (False, True):
            case = gen.make_case(M, N, K, seed=120 + idx, dist_a="integer", dist_b="integer", b_col_major=col,
                                 c_bf16=bf, lda=K + (K % 2 == 0), ldb=(K if col else N) + ((K if col else N) % 2 == 0),
                                 ldc=N + 1, name=f"generic{M}x{N}x{K}-int")
            run_and_check(handles_tiny_ws, case, 4, exact=True, offsets=offs)
            flags = handles_tiny_ws[(col, bf)].last_kernel_id() - 400
            assert (flags & 1) and not (flags & 64), (M, N, K, flags)
        case = gen.make_case(M, N, K, seed=120 + idx, dist_a="normal", dist_b="uniform", b_col_major=col,
                             lda=K + (K % 2 == 0), ldb=(K if col else N) + ((K if col else N) % 2 == 0),
                             name=f"generic{M}x{N}x{K}")
        run_and_check(handles_tiny_ws, case, 4, offsets=offs)


# ------------------------------------------------------------------ skinny shapes of the top rung
SKINNY = [  # (M, N, K, expected flags of kernel id - 400: 4 split-K, 8 swapped operands, 16 cluster reduce)
    (16, 1024, 8192, 4 | 8 | 16),      # 4 tiles: cluster of 8
    (16, 16384, 1024, 4 | 8 | 16),     # 64 tiles: cluster of 2
    (8, 2048, 2048, 4 | 8 | 16),       # cluster of 4, M below one MMA N step
    (32, 1000, 4096, 4 | 8 | 16),      # M = 32: largest cluster-reduced M, ragged N
    (33, 1000, 4096, 4 | 8),           # M = 33: swapped, split through the global workspace
    (64, 520, 2048, 4 | 8),            # M = 64: last swapped M
    (65, 520, 32768, 4 | 16),          # M = 65: regular orientation, K long enough for a split: cluster of 8, reduce through the rings
    (16, 256, 64, 8),                  # one tile, one k-block: no split
    (1, 8192, 8192, 4 | 8 | 16),       # GEMV
]


@pytest.mark.parametrize("col", [False, True], ids=["Brow", "Bcol"])
def test_tcgen05_skinny_modes(handles, col):
    for idx, (M, N, K, flags) in enumerate(SKINNY):
        for bf in (False, True):
            case = gen.make_case(M, N, K, seed=40 + idx, dist_a="integer", dist_b="integer", b_col_major=col,
                                 c_bf16=bf, name=f"skinny{M}x{N}x{K}-int")
            run_and_check(handles, case, 4, exact=True)
            got = handles[(col, bf)].last_kernel_id() - 400
            assert got & ~3 == flags, (M, N, K, got, flags)
        case = gen.make_case(M, N, K, seed=40 + idx, dist_a="normal", dist_b="normal", sigma_b=0.02, b_col_major=col,
                             name=f"skinny{M}x{N}x{K}")
        run_and_check(handles, case, 4)
    # unaligned operands: the generic-proxy producers feed the swapped and the cluster paths too
    case = gen.make_case(16, 1001, 4099, seed=77, dist_a="integer", dist_b="integer", b_col_major=col, lda=4101,
                         ldb=(4099 if col else 1001) + 2, ldc=1003, name="skinny-unaligned")
    run_and_check(handles, case, 4, exact=True, offsets=(1, 1, 1))
    assert (handles[(col, False)].last_kernel_id() - 400) & 64, "unaligned operands that fit are repacked"


# ------------------------------------------------------------------ K splits of 128-row tiles
REGULAR_SPLIT = [  # (M, N, K, (pad of lda, ldb, ldc)): few 128-row tiles, K long enough to split
    (256, 256, 8192, (0, 0, 0)),       # two whole tiles, C stored by TMA
    (384, 512, 1536, (0, 0, 0)),       # six tiles
    (130, 300, 1000, (0, 0, 0)),       # ragged M, N and K; a bf16 row ends inside a 16-byte unit: masked stores
    (200, 700, 3000, (8, 8, 1)),       # odd pitch of C: masked stores for both C types
    (65, 520, 4096, (0, 0, 0)),        # first M of the regular orientation: three of four row blocks empty
    (128, 256, 16384, (0, 0, 0)),      # one tile, very long K
]


@pytest.mark.parametrize("col", [False, True], ids=["Brow", "Bcol"])
def test_tcgen05_regular_split_routes(handles, handles_tiny_ws, col):
    """The K splits of a 128-row tile as a cluster (partials exchanged through the operand rings, owner CTAs reduce
    in rank order) in 2, 4 and 8 CTAs, and through the global workspace; every route bit-exact on integers."""
    for idx, (M, N, K, (pa, pb, pc)) in enumerate(REGULAR_SPLIT):
        for bf in (False, True):
            case = gen.make_case(M, N, K, seed=300 + idx, dist_a="integer", dist_b="integer", b_col_major=col,
                                 c_bf16=bf, lda=K + pa, ldb=(K if col else N) + pb, ldc=N + pc,
                                 name=f"rsplit{M}x{N}x{K}-int")
            C_ref, S = P.oracle_rows(case, np.arange(M))
            for splits, via in ((2, 2), (4, 2), (8, 2), (3, 1), (4, 1)):
                run_and_check(handles, case, 4, C_ref, S, np.arange(M), exact=True, pin=(1, splits, via))
                got = (handles[(col, bf)].last_kernel_id() - 400) & ~(3 | 64)
                assert got == (4 | (16 if via == 2 else 0)), (M, N, K, splits, via, got)
        # random values: inside the bound, and two runs of the cluster route agree bit for bit
        case = gen.make_case(M, N, K, seed=300 + idx, dist_a="normal", dist_b="uniform", b_col_major=col,
                             lda=K + pa, ldb=(K if col else N) + pb, ldc=N + pc, name=f"rsplit{M}x{N}x{K}")
        C_ref, S = P.oracle_rows(case, np.arange(M))
        _, b1 = run_and_check(handles, case, 4, C_ref, S, np.arange(M), pin=(1, 4, 2))
        _, b2 = run_and_check(handles, case, 4, C_ref, S, np.arange(M), pin=(1, 4, 2))
        assert np.array_equal(b1, b2), "two runs of the cluster reduce differ"
    # unpinned: the heuristic takes the cluster route for few tiles and long K
    case = gen.make_case(256, 256, 8192, seed=310, dist_a="integer", dist_b="integer", b_col_major=col, c_bf16=True)
    run_and_check(handles, case, 4, exact=True)
    assert (handles[(col, True)].last_kernel_id() - 400) & ~3 == (4 | 16)
    # unaligned operands and no room to repack them: the gathering producers feed the cluster route too
    case = gen.make_case(130, 270, 2100, seed=311, dist_a="integer", dist_b="integer", b_col_major=col, lda=2101,
                         ldb=(2101 if col else 271), ldc=271, name="rsplit-generic")
    run_and_check(handles_tiny_ws, case, 4, exact=True, offsets=(1, 1, 1), pin=(1, 4, 2))
    assert (handles_tiny_ws[(col, False)].last_kernel_id() - 400) == (1 | 2 | 4 | 16)


# ------------------------------------------------------------------ CTA-pair form of the top rung
PAIR = (2, 1, 0, 0, 0)      # launch plan: the CTA-pair kernel, no K split
@pytest.mark.parametrize("col", [False, True], ids=["Brow", "Bcol"])
def test_tcgen05_cta_pair_ragged(handles, col):
    """Large aligned shapes run on tcgen05.mma.cta_group::2 (512 x 256 pair tiles); tails in M, N and K."""
    # aligned pitch but a row length that ends inside a 16-byte unit: C padding must stay untouched
    for bf in (False, True):
        case = gen.make_case(4608, 4350 + (0 if bf else 1), 64, seed=59, dist_a="integer", dist_b="integer",
                             b_col_major=col, c_bf16=bf, lda=64, ldb=(64 if col else 4352), ldc=4352,
                             name="pair-ragged-row-end")
        rows = P.sample_rows(case.M)
        C_ref, S = P.oracle_rows(case, rows)
        run_and_check(handles, case, 4, C_ref, S, rows, exact=True, pin=PAIR)
        assert (handles[(col, bf)].last_kernel_id() - 400) & 32
    # (the pair kernel is pinned: for short K the dispatch prefers the single-CTA kernel, whose epilogue is hidden)
    for idx, (M, N, K) in enumerate([(5000, 5200, 1000), (4608, 4352, 72), (4200, 4352, 136)]):
        for bf in (False, True):
            case = gen.make_case(M, N, K, seed=60 + idx, dist_a="integer", dist_b="integer", b_col_major=col,
                                 c_bf16=bf, name=f"pair{M}x{N}x{K}-int")
            rows = P.sample_rows(M)
            C_ref, S = P.oracle_rows(case, rows)
            vals, _ = run_and_check(handles, case, 4, C_ref, S, rows, exact=True, pin=PAIR)
            assert (handles[(col, bf)].last_kernel_id() - 400) & 32, "expected the CTA-pair kernel"
            if not bf:
                assert P.integer_checksums_match(case, vals)
        case = gen.make_case(M, N, K, seed=60 + idx, dist_a="normal", dist_b="uniform", b_col_major=col,
                             name=f"pair{M}x{N}x{K}")
        rows = P.sample_rows(M)
        C_ref, S = P.oracle_rows(case, rows)
        run_and_check(handles, case, 4, C_ref, S, rows, pin=PAIR)


STREAMED = (2, 1, 3)        # launch plan: the CTA-pair kernel, last wave streamed along K
@pytest.mark.parametrize("col", [False, True], ids=["Brow", "Bcol"])
def test_tcgen05_cta_pair_streamed_last_wave(handles, col):
    """The under-filled last wave of pair tiles cut along K: pieces without a tile's first k-block leave their fp32
    partial tile in the workspace, the piece with it adds them in k order.  Bit-exact on integers, identical to the
    whole-tile schedule, for fewer tiles than pairs, for one and for several full rounds before the streamed wave."""
    for idx, (M, N, K) in enumerate([(2048, 4096, 2048),     # 64 tiles on 74 pairs: everything is streamed
                                     (4096, 4096, 1024),     # 128 tiles: one full round, then 54 streamed tiles
                                     (5000, 5200, 1104),     # 10 x 21 = 210 tiles: two rounds + 62 tiles, ragged M, N, K
                                     (1536, 2048, 4096),     # 24 tiles: every tile cut into three or four pieces
                                     (2500, 2120, 1104)]):   # 5 x 9 = 45 tiles, all streamed, ragged M, N and K
        for bf in (False, True):
            case = gen.make_case(M, N, K, seed=320 + idx, dist_a="integer", dist_b="integer", b_col_major=col,
                                 c_bf16=bf, name=f"streamed{M}x{N}x{K}-int")
            rows = P.sample_rows(M)
            C_ref, S = P.oracle_rows(case, rows)
            vals, bits = run_and_check(handles, case, 4, C_ref, S, rows, exact=True, pin=STREAMED)
            flags = handles[(col, bf)].last_kernel_id() - 400
            assert (flags & 32) and (flags & 128), (M, N, K, flags)
            _, whole = run_and_check(handles, case, 4, C_ref, S, rows, exact=True, pin=(2, 1, 1))
            assert not ((handles[(col, bf)].last_kernel_id() - 400) & 128)
            assert np.array_equal(bits, whole), "streamed and whole-tile schedules differ"
            if not bf:
                assert P.integer_checksums_match(case, vals)
        case = gen.make_case(M, N, K, seed=320 + idx, dist_a="normal", dist_b="uniform", b_col_major=col,
                             name=f"streamed{M}x{N}x{K}")
        rows = P.sample_rows(M)
        C_ref, S = P.oracle_rows(case, rows)
        _, b1 = run_and_check(handles, case, 4, C_ref, S, rows, pin=STREAMED)
        _, b2 = run_and_check(handles, case, 4, C_ref, S, rows, pin=STREAMED)
        assert np.array_equal(b1, b2), "two streamed runs differ"
    # a shape whose streamed pieces would be too short: the plan is refused
    case = gen.make_case(4200, 4352, 136, seed=330, dist_a="integer", dist_b="integer", b_col_major=col)
    dev = P.DeviceCase(case)
    g = handles[(col, False)]
    from paper_2605_28213_b200 import binding as kb
    assert kb.klineage_gemm_set_plan_raw(g._h, case.M, case.N, case.K, dev.a.ptr, case.lda, dev.b.ptr, case.ldb, dev.c.ptr,
                                         case.ldc, kb.klineage_gemm_plan_t(*STREAMED)) == kb.KLINEAGE_ERR_INVALID_ARG


K_PAIRED = (2, 1, 0, 0, 0, 0, 0, 3)     # launch plan: the CTA-pair kernel on 256-row tiles, two k-blocks per stage
@pytest.mark.parametrize("col", [False, True], ids=["Brow", "Bcol"])
def test_tcgen05_cta_pair_k_paired_tiles(handles, col):
    """256 x 256 pair tiles on a ring of three two-k-block stages, the TMEM accumulators alternating between a pair's
    consecutive tiles.  Bit-exact on integers and identical to the 512-row schedule: one round, several rounds (both
    accumulators in flight), an odd number of k-blocks (the last stage's second half lies past K), ragged M and N,
    a tile row with at most 128 live rows (the odd CTA has none)."""
    for idx, (M, N, K) in enumerate([(2048, 2048, 4096),     # 64 tiles on 74 pairs, one round
                                     (4096, 4096, 320),      # 256 tiles: 3.5 rounds, five k-blocks
                                     (2500, 2120, 1104),     # 10 x 9 tiles, ragged M, N and K (17.25 k-blocks)
                                     (2100, 1304, 72),       # two k-blocks, the second one 8 deep; last tile row 52 rows
                                     (300, 520, 64)]):       # one k-block: every stage's second half is empty
        for bf in (False, True):
            case = gen.make_case(M, N, K, seed=340 + idx, dist_a="integer", dist_b="integer", b_col_major=col,
                                 c_bf16=bf, name=f"kpaired{M}x{N}x{K}-int")
            rows = P.sample_rows(M)
            C_ref, S = P.oracle_rows(case, rows)
            vals, bits = run_and_check(handles, case, 4, C_ref, S, rows, exact=True, pin=K_PAIRED)
            flags = handles[(col, bf)].last_kernel_id() - 400
            assert (flags & 32) and (flags & 256), (M, N, K, flags)
            _, whole = run_and_check(handles, case, 4, C_ref, S, rows, exact=True, pin=(2, 1, 1))
            assert not ((handles[(col, bf)].last_kernel_id() - 400) & 256)
            assert np.array_equal(bits, whole), "256-row and 512-row schedules differ"
            if not bf:
                assert P.integer_checksums_match(case, vals)
        case = gen.make_case(M, N, K, seed=340 + idx, dist_a="normal", dist_b="uniform", b_col_major=col,
                             name=f"kpaired{M}x{N}x{K}")
        rows = P.sample_rows(M)
        C_ref, S = P.oracle_rows(case, rows)
        run_and_check(handles, case, 4, C_ref, S, rows, pin=K_PAIRED)
    # the form is the pair kernel's and 256 columns wide: other combinations are refused
    case = gen.make_case(2048, 2048, 4096, seed=350, dist_a="integer", dist_b="integer", b_col_major=col)
    dev = P.DeviceCase(case)
    g = handles[(col, False)]
    from paper_2605_28213_b200 import binding as kb
    for bad in ((2, 1, 0, 0, 0, 192, 0, 3), (2, 1, 3, 0, 0, 0, 0, 3), (2, 1, 0, 0, 0, 0, 0, 4), (1, 1, 0, 0, 0, 0, 0, 3)):
        assert kb.klineage_gemm_set_plan_raw(g._h, case.M, case.N, case.K, dev.a.ptr, case.lda, dev.b.ptr, case.ldb,
                                             dev.c.ptr, case.ldc, kb.klineage_gemm_plan_t(*bad)) == kb.KLINEAGE_ERR_INVALID_ARG


def test_dispatch_between_the_two_kernels(handles):
    """Long K and enough 512 x 256 (or 256 x 256) tiles: the pair kernel; short K or few tiles: the single-CTA kernel."""
    for (M, N, K), want_pair in (((2048, 4096, 4096), True), ((3072, 2048, 8192), True), ((2816, 2816, 2816), True),
                                 ((2048, 2048, 1024), False), ((1536, 3072, 1024), False), ((3584, 3584, 3584), True),    # (three rounds of 256-row tiles)
                                 ((2304, 2304, 2304), True), ((1536, 1536, 1536), False), ((4096, 4096, 512), True),
                                 ((2048, 2048, 8192), True),       # one round of 64 k-paired 256-row tiles
                                 ((1024, 2048, 8192), False)):     # 32 such tiles: the single-CTA kernel's cluster split
        case = gen.make_case(M, N, K, seed=70, dist_a="integer", dist_b="integer", c_bf16=True, name=f"disp{M}x{N}x{K}")
        rows = P.sample_rows(M)[::8]
        C_ref, S = P.oracle_rows(case, rows)
        run_and_check(handles, case, 4, C_ref, S, rows, exact=True)
        kid = handles[(False, True)].last_kernel_id()
        assert bool((kid - 400) & 32) == want_pair, (M, N, K, kid)


# ------------------------------------------------------------------ mid-size shapes: every scheduling mode of the top rung
MIDSIZE = [  # (M, N, K): what the shape exercises on the tcgen05 rung
    (1500, 2100, 333),    # 12 x 9 tiles on 148 SMs: single under-filled wave cut into half tiles, N tail inside a half
    (2304, 5120, 200),    # 360 tiles: two full waves + a 64-tile tail cut into half tiles
    (3000, 2900, 150),    # 24 x 12 = 288 tiles: 140-tile tail, too full for half tiles
    (200, 700, 30000),    # 2 x 3 tiles, very long K: split along K (a cluster per tile), M tail
    (130, 8192, 1024),    # 2 x 32 tiles of 128 rows, half tiles
    (4200, 4352, 136),    # CTA pairs: last 512-row tile has 104 rows (second row block and odd CTA empty)
    (1024, 9000, 96),     # wide N with a tail, K tail
]


@pytest.mark.parametrize("variant", [4, 5], ids=["tcgen05", "mma_sync"])
def test_midsize_shapes(handles, variant):
    rng = np.random.default_rng(99)
    for idx, (M, N, K) in enumerate(MIDSIZE):
        col, bf = bool(idx & 1), bool(rng.integers(2))
        case = gen.make_case(M, N, K, seed=80 + idx, dist_a="integer", dist_b="integer", b_col_major=col, c_bf16=False,
                             name=f"mid{M}x{N}x{K}-int")
        rows = P.sample_rows(M)
        C_ref, S = P.oracle_rows(case, rows)
        vals, _ = run_and_check(handles, case, variant, C_ref, S, rows, exact=True)
        assert P.integer_checksums_match(case, vals), case.name
        if variant == 4:
            # the schedule named above is the single-CTA kernel's: run it there whatever the dispatch rule prefers
            run_and_check(handles, case, variant, C_ref, S, rows, exact=True, pin=(1, 0, 0, 0, 0))
            assert not (handles[(col, False)].last_kernel_id() - 400) & 32
        case = gen.make_case(M, N, K, seed=80 + idx, dist_a="normal", dist_b="uniform", b_col_major=not col, c_bf16=bf,
                             name=f"mid{M}x{N}x{K}")
        C_ref, S = P.oracle_rows(case, rows)
        run_and_check(handles, case, variant, C_ref, S, rows)


# ------------------------------------------------------------------ degenerate sizes
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_NAMES)
def test_degenerate_sizes(handles, kb, variant):
    for bf in (False, True):
        case = gen.make_case(40, 50, 3, seed=1, c_bf16=bf, ldc=53)
        import dataclasses
        k0 = dataclasses.replace(case, K=0)
        dev = P.DeviceCase(k0)
        g = handles[(False, bf)]
        dev.run(g, variant)
        vals, bits = dev.result()
        assert np.all(bits == 0), "K == 0 must give +0 everywhere"
        assert g.last_kernel_id() == 900
        for (M, N) in [(0, 50), (40, 0), (0, 0)]:
            e = dataclasses.replace(case, M=M, N=N)
            d2 = P.DeviceCase(e)
            d2.run(g, variant)
            d2.result()                      # guards intact, nothing written
            assert g.last_kernel_id() == -1


# ------------------------------------------------------------------ closed forms and invariants on the GPU
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_NAMES)
def test_rank_one_closed_form_and_identity(handles, variant):
    rng = np.random.default_rng(5)
    vals8 = np.array([1.0, 1.125, 1.25, 1.375, 1.5, 1.625, 1.75, 1.875])
    for (M, N, K) in [(130, 270, 999), (16, 300, 8192)]:
        u = rng.choice(vals8, M) * rng.choice([-1, 1], M) * np.exp2(rng.integers(-3, 4, M))
        v = rng.choice(vals8, N) * rng.choice([-1, 1], N) * np.exp2(rng.integers(-3, 4, N))
        for col in (False, True):
            A = gen.f32_to_bf16_bits(np.repeat(u[:, None], K, axis=1).astype(np.float32))
            Bl = gen.f32_to_bf16_bits(np.repeat(v[None, :], K, axis=0).astype(np.float32))
            Bs = np.ascontiguousarray(Bl.T) if col else Bl
            case = gen.GemmCase("rank1", M, N, K, K, Bs.shape[1], N, col, False, A, Bs)
            dev = P.DeviceCase(case)
            dev.run(handles[(col, False)], variant)
            got, _ = dev.result()
            assert np.array_equal(got.astype(np.float64), K * np.outer(u, v)), "C_ij = K u_i v_j must be exact"
    # identity: C = B exactly, bf16 output round-trips the bits
    n = 200
    B = gen.draw((n, 333), "normal", 3, 1)
    I = gen.f32_to_bf16_bits(np.eye(n, dtype=np.float32))
    case = gen.GemmCase("identity", n, 333, n, n, 333, 333, False, True, I, B)
    dev = P.DeviceCase(case)
    dev.run(handles[(False, True)], variant)
    _, bits = dev.result()
    assert np.array_equal(bits, B)


@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_NAMES)
def test_deterministic_and_bf16_is_rounded_fp32(handles, variant):
    import dataclasses
    for name in ("c2", "c5"):
        case = gen.make_config(name, 3)
        dev = P.DeviceCase(case)
        dev.run(handles[(case.b_col_major, False)], variant)
        v1, b1 = dev.result()
        dev.run(handles[(case.b_col_major, False)], variant)
        v2, b2 = dev.result()
        assert np.array_equal(b1, b2), "two runs differ"
        cb = dataclasses.replace(case, c_bf16=True)
        devb = P.DeviceCase(cb)
        devb.run(handles[(case.b_col_major, True)], variant)
        _, bb = devb.result()
        assert np.array_equal(bb, gen.f32_to_bf16_bits(v1)), "bf16 C must be RNE of the fp32 C"


# ------------------------------------------------------------------ no fallback: each rung runs its own kernel
def test_each_variant_reports_its_own_kernel(handles, kb):
    aligned = gen.make_config("c1", 1)
    ragged = gen.make_config("c2", 1)
    padded = gen.make_config("c2pad", 1)
    g = handles[(False, False)]
    expect = {("c1", 0): 0, ("c1", 1): 100, ("c1", 2): 207, ("c1", 3): 300, ("c1", 5): 500,
              ("c2", 0): 0, ("c2", 1): 100, ("c2", 2): 200, ("c2", 3): 301, ("c2", 5): 501,
              ("c2pad", 2): 207, ("c2pad", 3): 300, ("c2pad", 5): 500}
    for case in (aligned, ragged, padded):
        dev = P.DeviceCase(case)
        for v in VARIANTS:
            dev.run(g, v)
            code, dev_id = g.device_status()
            assert code == 0 and dev_id == g.last_kernel_id()
            if v == 4:
                assert 400 <= dev_id < 656
                # unaligned operands are repacked into the workspace (flag 64), never gathered, when they fit
                assert ((dev_id - 400) & 1) == 0 and bool((dev_id - 400) & 64) == (case.name == "c2")
            else:
                want = expect.get((case.name, v))
                if want is not None:
                    assert dev_id == want, (case.name, v, dev_id)
    skinny = P.DeviceCase(gen.make_config("c5", 1))
    skinny.run(g, 4)
    flags = g.last_kernel_id() - 400
    assert (flags & 4) and (flags & 8) and (flags & 16), "the skinny shape must run swapped, split along K, cluster-reduced"


def test_error_codes(handles, kb):
    g = handles[(False, False)]
    case = gen.make_case(64, 64, 64, seed=1)
    dev = P.DeviceCase(case)
    a, b, c = dev.a.ptr, dev.b.ptr, dev.c.ptr
    run = lambda *args: g.run_raw(*args)
    assert run(a, b, c, 64, 64, 64, 64, 64, 64, 6) == kb.KLINEAGE_ERR_BAD_VARIANT
    assert run(a, b, c, 64, 64, 64, 64, 64, 64, -1) == kb.KLINEAGE_ERR_BAD_VARIANT
    assert run(a, b, c, 64, 64, 64, 63, 64, 64, 0) == kb.KLINEAGE_ERR_INVALID_ARG
    assert run(a, b, c, 64, 64, 64, 64, 63, 64, 1) == kb.KLINEAGE_ERR_INVALID_ARG
    assert run(a, b, c, 64, 64, 64, 64, 64, 63, 2) == kb.KLINEAGE_ERR_INVALID_ARG
    assert run(None, b, c, 64, 64, 64, 64, 64, 64, 3) == kb.KLINEAGE_ERR_INVALID_ARG
    assert run(a, b, None, 64, 64, 64, 64, 64, 64, 4) == kb.KLINEAGE_ERR_INVALID_ARG
    assert run(a, b, a, 64, 64, 64, 64, 64, 64, 4) == kb.KLINEAGE_ERR_INVALID_ARG     # C aliases A
    assert run(a, b, c, -1, 64, 64, 64, 64, 64, 0) == kb.KLINEAGE_ERR_INVALID_ARG
    assert run(a, b, c + 2, 64, 64, 64, 64, 64, 64, 0) == kb.KLINEAGE_ERR_INVALID_ARG  # fp32 C needs 4-byte alignment
    with pytest.raises(kb.KlineageError):
        kb.klineage_gemm_create(0, 7, 0)
    with pytest.raises(kb.KlineageError):
        kb.klineage_gemm_create(999, 0, 0)
    dev.run(g, 4)
    dev.result()


# ------------------------------------------------------------------ paired k-blocks of narrow tiles
# (kernel, splits, split_via, group_m, half_tail, tile_n, tail_n, stages): 64 columns x 8 stages and 128 columns x 6
# stages run two 64-deep k-blocks per stage.  K below: one k-block (the stage's second half lies wholly past K), an odd
# number of k-blocks, a ragged last k-block, many pairs; with a cluster split, K ranges counted in pairs.
PAIRED_K = [((1, 1, 0, 0, 0, 64, 0, 8), 40), ((1, 1, 0, 0, 0, 64, 0, 8), 200), ((1, 1, 0, 0, 0, 64, 0, 8), 328),
            ((1, 1, 0, 0, 0, 128, 0, 6), 64), ((1, 1, 0, 0, 0, 128, 0, 6), 456), ((1, 1, 0, 0, 0, 128, 0, 6), 1096),
            ((1, 2, 2, 0, 0, 128, 0, 6), 1096), ((1, 4, 2, 0, 0, 128, 0, 6), 2056)]


@pytest.mark.parametrize("col", [False, True], ids=["Brow", "Bcol"])
@pytest.mark.parametrize("pin,K", PAIRED_K, ids=lambda v: "x".join(map(str, v)) if isinstance(v, tuple) else f"K{v}")
def test_tcgen05_paired_k_blocks(handles, pin, K, col):
    for bf in (False, True):
        case = gen.make_case(300, 264, K, seed=77, dist_a="integer", dist_b="integer", b_col_major=col, c_bf16=bf,
                             name=f"paired {pin} K={K}")
        run_and_check(handles, case, 4, exact=True, pin=pin)
        g = handles[(col, bf)]
        flags = g.last_kernel_id() - 400
        assert flags >= 0 and not (flags & 32), "the single-CTA kernel must have run"
        assert bool(flags & 16) == (pin[1] > 1), "cluster split exactly when the plan asks for one"
