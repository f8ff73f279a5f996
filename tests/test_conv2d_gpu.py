"""Conv2d (paper, Evaluation, Table 2: N=8, C=64, 56x56, F=128, 3x3, FP16) against the fp64 oracle: the direct kernel
and the implicit GEMM on the tcgen05 rung, bit for bit on integer-valued inputs, within K*2^-23*S (widened by one fp16
rounding for fp16 outputs) on random ones; paddings, strides, ragged channel counts, unaligned bases, guard bands."""
import numpy as np
import pytest

from oracle import conv_oracle as co
from paper_2605_28213_b200 import inputs as gen
from tests import parity as P

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kb():
    from paper_2605_28213_b200 import binding
    return binding


def run_conv(kb, c, variant, off=(0, 0, 0)):
    import torch
    yelt = 2 if c.y_f16 else 4
    x = P.DeviceBuffer(c.x.size * 2, off[0] * 2).upload(c.x)
    w = P.DeviceBuffer(c.w.size * 2, off[1] * 2).upload(c.w)
    n_out = c.N * c.P * c.Q * c.F
    y = P.DeviceBuffer(max(n_out * yelt, 4), off[2] * yelt)
    with kb.Conv2d(0, y_f16=c.y_f16) as conv:
        conv.run(x.ptr, w.ptr, y.ptr, c.N, c.H, c.W, c.C, c.F, c.R, c.S, c.pad, c.stride, variant)
        torch.cuda.synchronize()
        code, _ = conv.device_status()
        kid = conv.last_kernel_id()
    assert code == 0
    assert x.guards_intact() and w.guards_intact() and y.guards_intact(), "guard band overwritten"
    raw = y.download()[:n_out * yelt]
    if c.y_f16:
        bits = raw.view(np.uint16).reshape(c.N, c.P, c.Q, c.F)
        vals = bits.view(np.float16).astype(np.float64)
    else:
        bits = raw.view(np.uint32).reshape(c.N, c.P, c.Q, c.F)
        vals = bits.view(np.float32).astype(np.float64)
    return vals, bits, kid


def check(c, vals, bits, exact, what):
    y_ref, S = co.conv2d(c.x, c.w, c.pad, c.stride)
    assert not np.isnan(vals).any(), f"{what}: NaN in y"
    if exact:
        if c.y_f16:
            want = co.round_to_f16(y_ref)
        else:
            want = y_ref.astype(np.float32)
            assert np.array_equal(want.astype(np.float64), y_ref)
            want = want.view(np.uint32)
        bad = np.argwhere(bits != want)
        assert bad.size == 0, f"{what}: {len(bad)} values differ, first at {bad[0]}: got {vals[tuple(bad[0])]} want {y_ref[tuple(bad[0])]}"
        return
    bound = co.bound_f16(c.K, S, y_ref) if c.y_f16 else co.bound_f32(c.K, S)
    err = np.abs(vals - y_ref)
    bad = np.argwhere(err > bound)
    assert bad.size == 0, f"{what}: {len(bad)} values outside the bound, first at {bad[0]}"


SHAPES = [  # N, H, W, C, F, R, S, pad, stride
    (2, 12, 10, 64, 128, 3, 3, (1, 1), (1, 1)),      # the benchmark's channel / filter counts; Q = 10: gathered patches
    (3, 9, 16, 64, 136, 3, 3, (1, 1), (1, 1)),       # Q = 16: patches by TMA; 432 pixels (ragged last tile), F > 128
    (1, 11, 24, 128, 72, 5, 3, (2, 0), (1, 1)),      # two 64-channel groups per tap, Q = 22 ... no: W - 2 = 22 -> gathered
    (2, 10, 26, 128, 72, 5, 3, (2, 0), (1, 1)),      # two 64-channel groups per tap, Q = 24: patches by TMA
    (1, 9, 7, 16, 40, 3, 2, (1, 0), (2, 1)),         # strides, asymmetric padding, ragged F
    (3, 5, 6, 8, 130, 1, 1, (0, 0), (1, 2)),         # 1x1 filter: a plain GEMM with strided rows; F > 128
    (1, 7, 7, 24, 3, 5, 5, (2, 2), (3, 3)),          # K = 600: ragged last k-block
    (2, 6, 5, 5, 9, 2, 3, (0, 2), (1, 1)),           # C % 8 != 0: element-wise patch gather
    (1, 20, 20, 32, 300, 3, 3, (1, 1), (1, 1)),      # more than one column tile, half-tile tail
    (1, 3, 3, 8, 8, 3, 3, (0, 0), (1, 1)),           # a single output pixel
    (2, 13, 21, 64, 100, 3, 3, (1, 1), (1, 1)),      # patch tiling, P and Q ragged; F * 2 % 16 != 0: masked stores by pixel
    (1, 17, 35, 64, 328, 3, 3, (0, 2), (1, 1)),      # patch tiling, two column tiles (one a half tile), asymmetric padding
    (3, 8, 16, 192, 64, 1, 1, (0, 0), (1, 1)),       # patch tiling, 1x1 filter over three 64-channel groups, exact patches
]


@pytest.mark.parametrize("variant", [0, 4], ids=["naive", "tcgen05"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s[:7])))
def test_conv2d_matches_the_oracle(kb, variant, shape):
    N, H, W, C, F, R, S, pad, stride = shape
    for y_f16 in (True, False):
        for dist, exact in (("integer", True), ("normal", False)):
            c = gen.make_conv_case(N, H, W, C, F, R, S, seed=180, pad=pad, stride=stride, dist=dist, y_f16=y_f16)
            vals, bits, kid = run_conv(kb, c, variant)
            assert kid == 600 if variant == 0 else 700 <= kid <= 708, kid
            check(c, vals, bits, exact, f"{c.name} variant {variant} f16={y_f16} {dist}")


def test_benchmark_shape_both_rungs(kb):
    for dist, exact in (("integer", True), ("normal", False)):
        c = gen.conv_benchmark_case(1, integer=exact)
        for variant in (0, 4):
            vals, bits, kid = run_conv(kb, c, variant)
            check(c, vals, bits, exact, f"conv_t2 variant {variant} {dist}")
            if variant == 4:
                assert kid == 708, kid          # patches and filters by TMA, transposed orientation (F <= 128)


@pytest.mark.parametrize("shape", [(3, 8, 16, 192, 64, 1, 1, (0, 0)),       # 3 patch tiles: the last unit's second tile lies past the images
                                   (2, 10, 26, 128, 72, 5, 3, (2, 0)),      # F = 72: the third warp's filter box is clipped, the fourth idles
                                   (5, 20, 33, 64, 128, 3, 3, (1, 1)),      # 3 x 3 patch tiles per image, ragged in P and Q, 45 tiles
                                   (1, 9, 16, 64, 8, 3, 3, (1, 1))],        # 8 filters; 2 patch tiles (the second: one pixel row)
                         ids=lambda s: "x".join(map(str, s[:7])))
def test_at_most_128_filters_run_transposed(kb, shape):
    # fp16 y with at most 128 filters: filters are the 128-row MMA operand, a unit is two patch tiles (kernel id 708);
    # fp32 y keeps the pixel-row orientation (700)
    N, H, W, C, F, R, S, pad = shape
    for y_f16, want_kid in ((True, 708), (False, 700)):
        for dist, exact in (("integer", True), ("normal", False)):
            c = gen.make_conv_case(N, H, W, C, F, R, S, seed=185, pad=pad, dist=dist, y_f16=y_f16)
            vals, bits, kid = run_conv(kb, c, 4)
            assert kid == want_kid, kid
            check(c, vals, bits, exact, f"{c.name} f16={y_f16} {dist}")


def test_unaligned_bases_take_the_slow_gather_and_direct_stores(kb):
    c = gen.make_conv_case(2, 8, 9, 16, 24, 3, 3, seed=181, dist="integer", y_f16=True)
    vals, bits, kid = run_conv(kb, c, 4, off=(1, 1, 1))
    assert kid == 707, kid
    check(c, vals, bits, True, "unaligned bases")
    vals, bits, _ = run_conv(kb, c, 0, off=(1, 1, 1))
    check(c, vals, bits, True, "unaligned bases, naive")


def test_conv2d_argument_rules(kb):
    chk = kb.klineage_conv2d_check_args
    X, Wt, Y = 0x100000, 0x200000, 0x400000
    ok = lambda **kw: chk(kw.get("dt", 2), kw.get("N", 1), kw.get("H", 8), kw.get("W", 8), kw.get("C", 8), kw.get("F", 8),
                          kw.get("R", 3), kw.get("S", 3), kw.get("ph", 1), kw.get("pw", 1), kw.get("sh", 1), kw.get("sw", 1),
                          kw.get("x", X), kw.get("w", Wt), kw.get("y", Y), kw.get("v", 4))
    assert ok() == kb.KLINEAGE_OK
    assert ok(dt=1) == kb.KLINEAGE_ERR_INVALID_ARG          # bf16 is not a Conv2d output type
    assert ok(v=3) == kb.KLINEAGE_ERR_BAD_VARIANT
    assert ok(R=0) == kb.KLINEAGE_ERR_INVALID_ARG
    assert ok(H=1, ph=0) == kb.KLINEAGE_ERR_INVALID_ARG     # filter larger than the padded image
    assert ok(sh=0) == kb.KLINEAGE_ERR_INVALID_ARG
    assert ok(y=None) == kb.KLINEAGE_ERR_INVALID_ARG
    assert ok(y=X) == kb.KLINEAGE_ERR_INVALID_ARG           # y aliases x
    assert ok(N=0, y=None) == kb.KLINEAGE_OK                # nothing to compute
    with kb.Gemm(0, c_bf16=True) as g:                      # a bf16 GEMM handle is refused by the Conv2d call
        assert kb.klineage_conv2d_run_raw(g._h, 1, 8, 8, 8, 8, 3, 3, 1, 1, 1, 1, X, Wt, Y, 4, None) == kb.KLINEAGE_ERR_INVALID_ARG
    with kb.Conv2d(0, y_f16=True) as cv:                    # and an fp16 Conv2d handle by the GEMM call
        assert kb.klineage_gemm_run_raw(cv._h, 8, 8, 8, X, 8, Wt, 8, Y, 8, 4, None) == kb.KLINEAGE_ERR_INVALID_ARG
