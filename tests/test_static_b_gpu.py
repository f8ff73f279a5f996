"""KLINEAGE_FLAG_STATIC_B (the caller promises that no in-flight GPU work writes B): the tcgen05 rung then issues the
first B loads of a short launch before it waits for the previous kernel.  The arithmetic must not change: results are
bit-identical to a handle without the flag, also when the calls run back to back on one stream with A produced by the
call before (the case the remaining wait protects)."""
import numpy as np
import pytest

from paper_2605_28213_b200 import inputs as gen
from tests import parity as P

pytestmark = pytest.mark.gpu

SHAPES = [  # M, N, K, col, bf16, (pad of lda, ldb, ldc)
    (16, 2048, 4096, False, False, (0, 0, 0)),     # skinny, cluster reduce, single wave
    (48, 1024, 8192, True, True, (0, 0, 0)),       # skinny, workspace split
    (300, 520, 1024, False, True, (0, 0, 0)),      # single wave of 128 x 256 tiles
    (1100, 2100, 264, True, False, (0, 0, 0)),     # more tiles than SMs would take in one wave? (45 tiles: one wave)
    (2100, 4200, 136, False, True, (0, 0, 0)),     # multi-wave: the flag changes nothing there
    (130, 263, 70, False, False, (1, 1, 1)),       # unaligned: repacked operands (the repack kernels precede the GEMM)
    # only B unaligned, K long enough for the early first ring fill, one wave: the library's own aligned copy of B
    # is written by the repack kernel just ahead of the GEMM, so the early loads must not run ahead of it
    (16, 2047, 4096, False, False, (0, 2, 0)),
    (200, 519, 1024, True, True, (0, 3, 0)),
]


@pytest.fixture(scope="module")
def kb():
    from paper_2605_28213_b200 import binding
    return binding


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s[:3])))
def test_static_b_changes_no_bit(kb, shape):
    M, N, K, col, bf, (pa, pb, pc) = shape
    case = gen.make_case(M, N, K, seed=190, dist_a="normal", dist_b="normal", b_col_major=col, c_bf16=bf,
                         lda=K + pa, ldb=(K if col else N) + pb, ldc=N + pc, name=f"static{M}x{N}x{K}")
    C_ref, S = P.oracle_rows(case, np.arange(M))
    out = []
    for static in (False, True):
        dev = P.DeviceCase(case)
        with kb.Gemm(0, b_col_major=col, c_bf16=bf, static_b=static) as g:
            for _ in range(3):                      # back to back: the later calls start while the earlier ones drain
                dev.run(g, kb.KLINEAGE_TCGEN05, check=False)
            dev.run(g, kb.KLINEAGE_TCGEN05)
            vals, bits = dev.result()
            if pb:
                assert (g.last_kernel_id() - 400) & 64, "the unaligned B must have been repacked for this test to bite"
        P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=False, what=f"{case.name} static_b={static}")
        out.append(bits)
    assert np.array_equal(out[0], out[1])


def test_a_produced_by_the_previous_call_is_waited_for(kb):
    # chain: Y = X . W1 (bf16), then Z = Y . W2 on the same stream, no synchronisation in between; with static B the
    # second call streams W2 early but must still read the finished Y
    import torch
    M, K1, N1, N2 = 16, 4096, 2048, 1024
    c1 = gen.make_case(M, N1, K1, seed=191, dist_a="integer", dist_b="integer", c_bf16=True, name="chain1")
    a = P.DeviceBuffer(c1.A.size * 2).upload(c1.A)
    w1 = P.DeviceBuffer(c1.B.size * 2).upload(c1.B)
    c2 = gen.make_case(M, N2, N1, seed=192, dist_a="integer", dist_b="integer", c_bf16=False, name="chain2")
    w2 = P.DeviceBuffer(c2.B.size * 2).upload(c2.B)
    y = P.DeviceBuffer(M * N1 * 2)
    z = P.DeviceBuffer(M * N2 * 4)
    # reference: Y exactly (small integers: bf16 rounding of the exact sums), then Z from that Y in fp64
    from oracle import gemm_oracle as orc
    Y_ref, _ = orc.gemm(M, N1, K1, c1.A, c1.lda, c1.B, c1.ldb, False)
    y_bits = orc.round_to_bf16(Y_ref)
    Z_ref, S = orc.gemm(M, N2, N1, y_bits, N1, c2.B, c2.ldb, False)
    with kb.Gemm(0, c_bf16=True, static_b=True) as g1, kb.Gemm(0, c_bf16=False, static_b=True) as g2:
        for _ in range(5):
            g1.run(a.ptr, w1.ptr, y.ptr, M, N1, K1, K1, N1, N1, kb.KLINEAGE_TCGEN05)
            g2.run(y.ptr, w2.ptr, z.ptr, M, N2, N1, N1, N2, N2, kb.KLINEAGE_TCGEN05)
        torch.cuda.synchronize()
        assert g1.device_status()[0] == 0 and g2.device_status()[0] == 0
    got_y = y.download().view(np.uint16).reshape(M, N1)
    assert np.array_equal(got_y, y_bits)
    got_z = z.download().view(np.float32).reshape(M, N2).astype(np.float64)
    assert np.all(np.abs(got_z - Z_ref) <= orc.bound_f32(N1, S))
    assert all(b.guards_intact() for b in (a, w1, w2, y, z))


def test_unknown_flag_bits_are_refused(kb):
    with pytest.raises(kb.KlineageError):
        kb.klineage_gemm_create(0, kb.KLINEAGE_B_ROW_MAJOR, kb.KLINEAGE_C_F32, 0, 4)
