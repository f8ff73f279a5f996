"""Batched and grouped GEMM (paper, Appendix D: BMM and GroupedGEMM are held-out members of the GEMM family).

Every problem of a batch / group is checked against the oracle (bit for bit on integer-valued inputs, within the
error bound on random ones) and, where the single-problem call does not split K, bit for bit against separate
klineage_gemm_run calls.  Shapes are chosen so that the one-launch path of the tcgen05 rung (CTA-pair kernel over
3-D tensor maps / a table of per-group tensor maps) and the problem-by-problem path are both reached; gaps between
batches, row padding and guard bands must stay untouched.
"""
import numpy as np
import pytest

from paper_2605_28213_b200 import inputs as gen
from tests import parity as P

pytestmark = pytest.mark.gpu

VARIANT_NAMES = ["naive", "tiled", "vectorized", "pipelined", "tcgen05", "mma_sync"]
NAN_BITS = np.uint16(0x7FC0)


@pytest.fixture(scope="module")
def kb():
    from paper_2605_28213_b200 import binding
    return binding


class Batch:
    """`batch` cases of one shape laid out with element strides; the gaps hold NaN (A, B) or poison (C)."""

    def __init__(self, batch, M, N, K, col, bf, dist, seed, pad=(0, 0, 0), gap=(0, 0, 0), share_a=False):
        self.cases = [gen.make_case(M, N, K, seed=seed + b, dist_a=dist, dist_b=dist, b_col_major=col, c_bf16=bf,
                                    lda=K + pad[0], ldb=(K if col else N) + pad[1], ldc=N + pad[2],
                                    name=f"bmm{b}-{M}x{N}x{K}-{dist}") for b in range(batch)]
        c0 = self.cases[0]
        self.batch, self.celt = batch, 2 if bf else 4
        self.stride_a = 0 if share_a else c0.A.size + gap[0]
        self.stride_b = c0.B.size + gap[1]
        self.stride_c = M * c0.ldc + gap[2]
        if share_a:
            for c in self.cases[1:]:
                c.A[...] = c0.A
        a_all = np.full(max(self.stride_a * (batch - 1), 0) + c0.A.size, NAN_BITS, np.uint16)
        b_all = np.full(self.stride_b * (batch - 1) + c0.B.size, NAN_BITS, np.uint16)
        for b, c in enumerate(self.cases):
            a_all[b * self.stride_a: b * self.stride_a + c.A.size] = c.A.reshape(-1)
            b_all[b * self.stride_b: b * self.stride_b + c.B.size] = c.B.reshape(-1)
        self.a = P.DeviceBuffer(a_all.size * 2).upload(a_all)
        self.b = P.DeviceBuffer(b_all.size * 2).upload(b_all)
        self.c_elems = self.stride_c * (batch - 1) + (M - 1) * c0.ldc + N
        self.c = P.DeviceBuffer(self.c_elems * self.celt)

    def run(self, g, variant):
        import torch
        c = self.cases[0]
        g.run_batched(self.batch, self.a.ptr, self.b.ptr, self.c.ptr, c.M, c.N, c.K, c.lda, c.ldb, c.ldc,
                      self.stride_a, self.stride_b, self.stride_c, variant)
        torch.cuda.synchronize()
        code, _ = g.device_status()
        assert code == 0

    def results(self):
        """Per batch (vals, bits); asserts guards, row padding and inter-batch gaps untouched."""
        assert self.a.guards_intact() and self.b.guards_intact() and self.c.guards_intact(), "guard band overwritten"
        c0 = self.cases[0]
        dt = np.uint16 if c0.c_bf16 else np.uint32
        poison = dt(0xA5A5) if c0.c_bf16 else dt(0xA5A5A5A5)
        flat = self.c.download().view(dt)
        touched = np.zeros(flat.size, bool)
        out = []
        for b in range(self.batch):
            idx = b * self.stride_c + np.arange(c0.M)[:, None] * c0.ldc + np.arange(c0.N)[None, :]
            touched[idx.reshape(-1)] = True
            bits = flat[idx]
            vals = gen.bf16_bits_to_f32(bits) if c0.c_bf16 else bits.view(np.float32)
            out.append((vals, bits))
        assert np.all(flat[~touched] == poison), "row padding or a gap between batches was written"
        return out


def plan_of(kernel):
    """A kernel number (1 single-CTA, 2 CTA pair) or a whole plan as a tuple."""
    return kernel if isinstance(kernel, tuple) else (kernel, 1, 0, 0, 0)


K_PAIRED = (2, 1, 0, 0, 0, 0, 0, 3)     # the CTA-pair kernel on 256-row tiles, two k-blocks per stage


def check_batch(kb, bt, variant, exact, want_pair=None, one_launch=None, kernel=0, want_k_paired=None):
    """kernel: 1 / 2 pins the single-CTA / CTA-pair kernel for the per-problem shape first (a tuple: that plan)."""
    c0 = bt.cases[0]
    with kb.Gemm(0, b_col_major=c0.b_col_major, c_bf16=c0.c_bf16) as g:
        if kernel:
            g.set_plan(kb.klineage_gemm_plan_t(*plan_of(kernel)), bt.a.ptr, bt.b.ptr, bt.c.ptr, c0.M, c0.N, c0.K,
                       c0.lda, c0.ldb, c0.ldc)
        bt.run(g, variant)
        kid = g.last_kernel_id()
        if one_launch is not None:
            assert (g.last_launch_count() == 1) == one_launch, g.last_launch_count()
        res = bt.results()
        for b, case in enumerate(bt.cases):
            C_ref, S = P.oracle_rows(case, np.arange(case.M))
            P.assert_matches_oracle(case, res[b][0], res[b][1], C_ref, S, exact=exact,
                                    what=f"{case.name} {VARIANT_NAMES[variant]} batch {b}")
        if want_pair is not None:
            assert bool((kid - 400) & 32) == want_pair, kid
        if want_k_paired is not None:
            assert bool((kid - 400) & 256) == want_k_paired, kid
        # the same problems one by one through klineage_gemm_run
        for b, case in enumerate(bt.cases):
            dev = P.DeviceCase(case)
            dev.run(g, variant)
            kid1 = g.last_kernel_id()
            _, bits1 = dev.result()
            if variant != 4 or not (kid1 - 400) & 4:
                assert np.array_equal(bits1, res[b][1]), f"batch {b} differs bitwise from the single-problem call"


# (batch, M, N, K, col, bf16, pad, gap): at least 74 tiles of 512 x 256 in the batch, so that both kernels qualify
ONE_LAUNCH = [
    (7, 1100, 1104, 136, False, True, (0, 8, 8), (8, 16, 24)),      # ragged tiles, bf16 C through the 3-D TMA store
    (5, 600, 2100, 200, True, False, (8, 8, 4), (0, 0, 0)),         # column-major B, fp32 C through the TMA store
    (7, 520, 1301, 72, False, False, (0, 3, 1), (0, 0, 5)),         # odd N (pitch of B 1304): masked direct stores
    (5, 1100, 1104, 2056, False, True, (0, 0, 0), (0, 0, 0)),       # K >= 2048: the pair kernel by default
]


@pytest.mark.parametrize("cfg", ONE_LAUNCH, ids=lambda c: f"b{c[0]}-{c[1]}x{c[2]}x{c[3]}")
@pytest.mark.parametrize("kernel", [0, 1, 2], ids=["default", "single", "pair"])
def test_bmm_one_launch(kb, cfg, kernel):
    batch, M, N, K, col, bf, pad, gap = cfg
    # unpinned: the cycle estimate of the schedules decides - rounds of 512 x 256 or 256 x 256 pair tiles beat the waves
    # of 128 x 256 tiles at all four shapes (measured: 15.4 against 17.4 us at 5 x 600 x 2104 x 200, 39.8 against 43.0 at
    # 5 x 1100 x 1104 x 2056)
    pair = True if kernel == 0 else (kernel == 2)
    for dist, exact in (("integer", True), ("normal", False)):
        if kernel and dist == "normal" and K >= 2048:
            continue                      # (the long-K case costs the oracle most; integers cover the pinned kernels)
        bt = Batch(batch, M, N, K, col, bf, dist, seed=70, pad=pad, gap=gap)
        check_batch(kb, bt, 4, exact, want_pair=pair, one_launch=True, kernel=kernel)


@pytest.mark.parametrize("cfg", [ONE_LAUNCH[0], ONE_LAUNCH[1], ONE_LAUNCH[3]], ids=lambda c: f"b{c[0]}-{c[1]}x{c[2]}x{c[3]}")
def test_bmm_k_paired_tiles(kb, cfg):
    """The batched launch on 256 x 256 pair tiles, two k-blocks per stage: pinned, against the oracle and bit-equal to
    the problems one by one; K = 136 / 200 / 2056 give an odd number of k-blocks and a ragged last one."""
    batch, M, N, K, col, bf, pad, gap = cfg
    for dist, exact in (("integer", True),) + ((("normal", False),) if K < 2048 else ()):
        bt = Batch(batch, M, N, K, col, bf, dist, seed=75, pad=pad, gap=gap)
        check_batch(kb, bt, 4, exact, want_pair=True, one_launch=True, kernel=K_PAIRED, want_k_paired=True)


def test_bmm_k_paired_tiles_by_default(kb):
    """Twice the tiles in fewer than twice the rounds: 5 x (1100 x 1104 x 2056) is 75 tiles of 512 x 256 (two rounds on
    74 CTA pairs) or 125 of 256 x 256 (two rounds as well) - the launch takes the 256-row tiles on its own."""
    bt = Batch(5, 1100, 1104, 2056, False, True, "integer", seed=76)
    check_batch(kb, bt, 4, True, want_pair=True, one_launch=True, want_k_paired=True)
    # a pinned pair kernel without the stage count keeps the 512-row tiles
    bt = Batch(5, 1100, 1104, 2056, False, True, "integer", seed=76)
    check_batch(kb, bt, 4, True, want_pair=True, one_launch=True, kernel=2, want_k_paired=False)


def test_bmm_problem_by_problem_paths(kb):
    # batch strides that are not multiples of 16 bytes, a shared A, small and skinny problems, few tiles
    cfgs = [dict(batch=3, M=300, N=264, K=136, col=False, bf=True, gap=(3, 5, 1)),
            dict(batch=4, M=16, N=520, K=1024, col=True, bf=False, gap=(0, 0, 0)),
            dict(batch=3, M=700, N=520, K=72, col=False, bf=False, gap=(0, 0, 0), share_a=True),
            dict(batch=2, M=130, N=70, K=50, col=False, bf=True, pad=(1, 1, 1), gap=(1, 0, 3))]
    for cfg in cfgs:
        for dist, exact in (("integer", True), ("uniform", False)):
            bt = Batch(cfg["batch"], cfg["M"], cfg["N"], cfg["K"], cfg["col"], cfg["bf"], dist, seed=80,
                       pad=cfg.get("pad", (0, 0, 0)), gap=cfg["gap"], share_a=cfg.get("share_a", False))
            check_batch(kb, bt, 4, exact, want_pair=False if cfg["M"] <= 256 or cfg["gap"][0] % 8 else None,
                        one_launch=False)


@pytest.mark.parametrize("variant", [0, 1, 2, 3, 5], ids=lambda v: VARIANT_NAMES[v])
def test_bmm_lower_rungs(kb, variant):
    bt = Batch(3, 140, 200, 72, False, True, "integer", seed=90, pad=(0, 0, 2), gap=(8, 0, 6))
    check_batch(kb, bt, variant, True)
    bt = Batch(2, 65, 130, 264, True, False, "normal", seed=91, gap=(0, 8, 0))
    check_batch(kb, bt, variant, False)


def test_bmm_argument_rules(kb):
    bt = Batch(2, 64, 64, 64, False, False, "integer", seed=95)
    c = bt.cases[0]
    with kb.Gemm(0) as g:
        raw = lambda batch, sa, sb, sc: kb.klineage_gemm_run_batched_raw(
            g._h, batch, c.M, c.N, c.K, bt.a.ptr, c.lda, sa, bt.b.ptr, c.ldb, sb, bt.c.ptr, c.ldc, sc, 4, None)
        assert raw(0, 0, 0, 0) == kb.KLINEAGE_OK                                  # empty batch: no-op
        assert raw(2, bt.stride_a, bt.stride_b, c.M * c.ldc - 1) == kb.KLINEAGE_ERR_INVALID_ARG   # C matrices overlap
        assert raw(2, -1, bt.stride_b, bt.stride_c) == kb.KLINEAGE_ERR_INVALID_ARG
        assert raw(70000, bt.stride_a, bt.stride_b, bt.stride_c) == kb.KLINEAGE_ERR_INVALID_ARG
        assert raw(-1, bt.stride_a, bt.stride_b, bt.stride_c) == kb.KLINEAGE_ERR_INVALID_ARG
        import torch
        torch.cuda.synchronize()
    assert bt.c.guards_intact()


# ---------------------------------------------------------------------------- grouped
def run_grouped(kb, cases, variant, exact, want_pair=None, one_launch=None, kernel=0, want_k_paired=None):
    import torch
    c0 = cases[0]
    devs = [P.DeviceCase(c) for c in cases]
    with kb.Gemm(0, b_col_major=c0.b_col_major, c_bf16=c0.c_bf16) as g:
        if kernel:
            first = next(i for i, c in enumerate(cases) if c.M and c.N)
            c, d = cases[first], devs[first]
            g.set_plan(kb.klineage_gemm_plan_t(*plan_of(kernel)), d.a.ptr, d.b.ptr, d.c.ptr, c.M, c.N, c.K, c.lda,
                       c.ldb, c.ldc)
        g.run_grouped([d.a.ptr for d in devs], [d.b.ptr for d in devs], [d.c.ptr for d in devs],
                      [c.M for c in cases], [c.N for c in cases], [c.K for c in cases],
                      [c.lda for c in cases], [c.ldb for c in cases], [c.ldc for c in cases], variant)
        torch.cuda.synchronize()
        code, _ = g.device_status()
        assert code == 0
        kid = g.last_kernel_id()
        if one_launch is not None:
            assert (g.last_launch_count() == 1) == one_launch, g.last_launch_count()
        if want_pair is not None:
            assert bool((kid - 400) & 32) == want_pair, kid
        if want_k_paired is not None:
            assert bool((kid - 400) & 256) == want_k_paired, kid
        got = [d.result() for d in devs]
        for case, (vals, bits) in zip(cases, got):
            if case.M == 0 or case.N == 0:
                continue
            if case.K == 0:
                assert not bits.any(), "K == 0 must give zeros"
                continue
            C_ref, S = P.oracle_rows(case, np.arange(case.M))
            P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=exact, what=f"group {case.name}")
        for case, (vals, bits) in zip(cases, got):
            if case.M == 0 or case.N == 0 or case.K == 0:
                continue
            dev = P.DeviceCase(case)
            dev.run(g, variant)
            if variant != 4 or not (g.last_kernel_id() - 400) & 4:
                assert np.array_equal(dev.result()[1], bits), f"group {case.name} differs from the single-problem call"


GROUP_SHAPES = [(300, 2048, 136), (1100, 1304, 200), (513, 2000, 64), (700, 1528, 520), (1025, 1304, 72),
                (600, 520, 328)]      # 8 + 18 + 16 + 12 + 18 + 6 = 78 pair tiles


@pytest.mark.parametrize("col,bf", [(False, True), (True, False)], ids=["row-bf16", "col-f32"])
@pytest.mark.parametrize("kernel", [0, 1, 2], ids=["default", "single", "pair"])
def test_grouped_one_launch(kb, col, bf, kernel):
    for dist, exact in (("integer", True), ("normal", False)):
        cases = [gen.make_case(M, N, K, seed=100 + i, dist_a=dist, dist_b=dist, b_col_major=col, c_bf16=bf,
                               ldc=N + (4 if i % 2 else 0), name=f"g{i}-{M}x{N}x{K}-{dist}")
                 for i, (M, N, K) in enumerate(GROUP_SHAPES)]
        # every group has more than 256 rows, so the pair kernel qualifies, and the cycle estimate prefers it (two rounds
        # of 256 x 256 tiles against two waves of 128 x 256 tiles)
        run_grouped(kb, cases, 4, exact, want_pair=kernel != 1, one_launch=True, kernel=kernel)


def test_grouped_long_k_takes_the_pair_kernel_and_small_groups_the_single_one(kb):
    shapes = [(520, 2048, 2056), (300, 1304, 2048), (1030, 1528, 2120), (700, 2560, 2048)]      # 16 + 6 + 18 + 20
    shapes += [(600, 2048, 2048), (513, 1024, 2048)]                                             # + 16 + 8 = 84 tiles of 512 x 256
    cases = [gen.make_case(M, N, K, seed=140 + i, dist_a="integer", dist_b="integer", c_bf16=True, name=f"gk{i}")
             for i, (M, N, K) in enumerate(shapes)]
    run_grouped(kb, cases, 4, True, want_pair=True, one_launch=True)
    # one group of 40 rows among them: the pair kernel no longer qualifies, the single-CTA kernel takes all groups
    small = [(40, 2048, 136), (1100, 1304, 200), (64, 2000, 64), (700, 1528, 520), (129, 1304, 72), (600, 520, 328),
             (1, 264, 8), (900, 2048, 264)]
    cases = [gen.make_case(M, N, K, seed=150 + i, dist_a="integer", dist_b="integer", c_bf16=False, name=f"gs{i}")
             for i, (M, N, K) in enumerate(small)]
    run_grouped(kb, cases, 4, True, want_pair=False, one_launch=True)


def test_grouped_with_an_odd_width_group_uses_masked_stores_for_it(kb):
    shapes = list(GROUP_SHAPES)
    shapes[2] = (513, 1999, 64)          # pitch of B would be 1999: give it an aligned pitch, keep N odd
    cases = []
    for i, (M, N, K) in enumerate(shapes):
        cases.append(gen.make_case(M, N, K, seed=110 + i, dist_a="integer", dist_b="integer", c_bf16=True,
                                   ldb=(N + 7) // 8 * 8, ldc=N + 3, name=f"godd{i}"))
    run_grouped(kb, cases, 4, True, want_pair=False, one_launch=True, kernel=1)
    run_grouped(kb, cases, 4, True, want_pair=True, one_launch=True, kernel=2)
    run_grouped(kb, cases, 4, True, one_launch=True)


def test_grouped_problem_by_problem_paths(kb):
    # a skinny group, an empty one and a K == 0 group force the ordinary path; every rung takes it
    shapes = [(16, 520, 1024), (0, 64, 64), (300, 264, 136), (40, 72, 0), (130, 70, 50)]
    for variant in range(6):
        cases = []
        for i, (M, N, K) in enumerate(shapes):
            c = gen.make_case(max(M, 1), N, max(K, 1), seed=120 + i, dist_a="integer", dist_b="integer",
                              name=f"gl{i}-{M}x{N}x{K}")
            import dataclasses
            cases.append(dataclasses.replace(c, M=M, K=K))
        run_grouped(kb, cases, variant, True, want_pair=False if variant == 4 else None, one_launch=False)


def test_grouped_argument_rules(kb):
    cases = [gen.make_case(64, 64, 64, seed=130 + i, dist_a="integer", dist_b="integer", name=f"ga{i}") for i in range(2)]
    devs = [P.DeviceCase(c) for c in cases]
    with kb.Gemm(0) as g:
        def raw(C_ptrs, ldc=None, variant=4):
            return kb.klineage_gemm_run_grouped_raw(
                g._h, [64, 64], [64, 64], [64, 64], [d.a.ptr for d in devs], [64, 64], [d.b.ptr for d in devs],
                [64, 64], C_ptrs, ldc or [64, 64], variant, None)
        assert raw([devs[0].c.ptr, devs[0].c.ptr]) == kb.KLINEAGE_ERR_INVALID_ARG          # two groups write one C
        assert raw([devs[0].c.ptr, devs[1].a.ptr]) == kb.KLINEAGE_ERR_INVALID_ARG          # C aliases an A
        assert raw([devs[0].c.ptr, devs[1].c.ptr], ldc=[64, 63]) == kb.KLINEAGE_ERR_INVALID_ARG
        assert raw([devs[0].c.ptr, devs[1].c.ptr], variant=9) == kb.KLINEAGE_ERR_BAD_VARIANT
        assert raw([devs[0].c.ptr, devs[1].c.ptr]) == kb.KLINEAGE_OK
        import torch
        torch.cuda.synchronize()
    for d, c in zip(devs, cases):
        vals, bits = d.result()
        C_ref, S = P.oracle_rows(c, np.arange(c.M))
        P.assert_matches_oracle(c, vals, bits, C_ref, S, exact=True, what=c.name)


def test_grouped_ragged_rows_on_the_pair_kernel(kb):
    """Groups whose last tile row has at most 256 live rows: those tile rows become table entries of their own at the
    end of the schedule (their second row block issues no MMAs) - the result must not notice.  Heights: a multiple of
    512, at most 256 in all, exactly 256 and 257 over a multiple, one row over."""
    shapes = [(1024, 1304, 200), (64, 2048, 136), (256, 520, 72), (768, 1528, 328), (769, 1024, 64), (513, 2000, 264),
              (1536, 2048, 72), (1200, 776, 136), (2, 304, 520)]       # 97 pair tiles: at least one per CTA pair
    for col, bf in ((False, True), (True, False)):
        cases = [gen.make_case(M, N, K, seed=170 + i, dist_a="integer", dist_b="integer", b_col_major=col, c_bf16=bf,
                               ldc=N + (8 if i % 3 == 0 else 0), name=f"gr{i}-{M}x{N}x{K}")
                 for i, (M, N, K) in enumerate(shapes)]
        run_grouped(kb, cases, 4, True, want_pair=True, one_launch=True, kernel=2, want_k_paired=False)
        # the same groups on 256-row tiles (no tile row is split off: every tile is one row block)
        run_grouped(kb, cases, 4, True, want_pair=True, one_launch=True, kernel=K_PAIRED, want_k_paired=True)
