"""Pins of the Conv2d oracle against things other than itself (CPU only)."""
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest

from oracle import conv_oracle as co
from paper_2605_28213_b200 import inputs as gen

GOLDEN = Path(__file__).resolve().parent / "golden"


def f16(vals) -> np.ndarray:
    return np.asarray(vals, dtype=np.float64).astype(np.float16).view(np.uint16)


def test_hand_worked_example():
    rows = {}
    for line in (GOLDEN / "conv_hand_worked_1x3x3x1.txt").read_text().splitlines():
        if line and not line.startswith("#"):
            key, *vals = line.split()
            rows[key] = [float(v) for v in vals]
    x = f16(rows["x"]).reshape(1, 3, 3, 1)
    w = f16(rows["w"]).reshape(1, 2, 2, 1)
    y, s = co.conv2d(x, w, pad=(1, 0), stride=(1, 1))
    assert y.shape == (1, 4, 2, 1)
    assert np.array_equal(y.reshape(-1), np.array(rows["y"]))
    assert s[0, 1, 0, 0] == 1 + 4 + 2 + 15


@pytest.mark.parametrize("cfg", [(2, 9, 7, 5, 4, 3, 2, (1, 0), (2, 1)), (1, 8, 8, 16, 8, 3, 3, (1, 1), (1, 1)),
                                 (3, 5, 6, 3, 2, 1, 1, (0, 0), (1, 2)), (1, 7, 7, 4, 3, 5, 5, (2, 2), (3, 3)),
                                 (2, 6, 5, 8, 5, 2, 3, (0, 2), (1, 1))])
def test_against_the_library_convolution_in_fp64(cfg):
    import torch
    N, H, W, C, F, R, S, pad, stride = cfg
    c = gen.make_conv_case(N, H, W, C, F, R, S, seed=3, pad=pad, stride=stride)
    y, _ = co.conv2d(c.x, c.w, pad, stride)
    xt = torch.from_numpy(co.f16_bits_to_f64(c.x)).permute(0, 3, 1, 2)
    wt = torch.from_numpy(co.f16_bits_to_f64(c.w)).permute(0, 3, 1, 2)
    ref = torch.nn.functional.conv2d(xt, wt, stride=stride, padding=pad).permute(0, 2, 3, 1).numpy()
    assert y.shape == ref.shape == (N, c.P, c.Q, F)
    assert np.allclose(y, ref, rtol=1e-13, atol=1e-13)


def test_one_by_one_filter_is_a_matrix_product():
    c = gen.make_conv_case(2, 5, 4, 24, 7, 1, 1, seed=4, pad=(0, 0), stride=(1, 1))
    y, s = co.conv2d(c.x, c.w, (0, 0), (1, 1))
    X = co.f16_bits_to_f64(c.x).reshape(-1, 24)
    Wm = co.f16_bits_to_f64(c.w).reshape(7, 24)
    assert np.allclose(y.reshape(-1, 7), X @ Wm.T, rtol=1e-14, atol=1e-14)
    assert np.allclose(s.reshape(-1, 7), np.abs(X) @ np.abs(Wm).T, rtol=1e-14, atol=1e-14)


def test_delta_filter_shifts_the_input():
    # w[f][r0][s0][c] = (c == f): y[n][p][q][f] = x[n][p + r0 - pad][q + s0 - pad][f], zero outside
    N, H, W, C, R, S = 1, 6, 7, 3, 3, 3
    c = gen.make_conv_case(N, H, W, C, C, R, S, seed=5, dist="integer")
    x = co.f16_bits_to_f64(c.x)
    for r0 in range(R):
        for s0 in range(S):
            w = np.zeros((C, R, S, C))
            for f in range(C):
                w[f, r0, s0, f] = 1.0
            y, _ = co.conv2d(c.x, f16(w), (1, 1), (1, 1))
            want = np.zeros_like(y)
            for p in range(H):
                for q in range(W):
                    h, ww = p + r0 - 1, q + s0 - 1
                    if 0 <= h < H and 0 <= ww < W:
                        want[0, p, q] = x[0, h, ww]
            assert np.array_equal(y, want), (r0, s0)


def test_all_ones_counts_the_taps_in_range():
    N, H, W, C, F, R, S = 1, 5, 4, 6, 2, 3, 3
    x = f16(np.ones((N, H, W, C)))
    w = f16(np.ones((F, R, S, C)))
    for pad, stride in (((1, 1), (1, 1)), ((2, 0), (2, 1)), ((0, 1), (1, 2))):
        y, _ = co.conv2d(x, w, pad, stride)
        P, Q = co.out_size(H, W, R, S, pad, stride)
        for p in range(P):
            for q in range(Q):
                nh = sum(0 <= p * stride[0] + r - pad[0] < H for r in range(R))
                nw = sum(0 <= q * stride[1] + s - pad[1] < W for s in range(S))
                assert np.all(y[0, p, q] == nh * nw * C)


def test_exact_rational_brute_force_on_tiny_shapes():
    def frac(bits):
        return Fraction(float(np.uint16(bits).view(np.float16)))
    for seed, (N, H, W, C, F, R, S, pad, stride) in enumerate([(1, 3, 3, 2, 2, 2, 2, (1, 1), (1, 1)),
                                                               (2, 4, 3, 1, 1, 3, 1, (0, 0), (1, 2)),
                                                               (1, 2, 5, 3, 2, 1, 3, (0, 1), (2, 2))]):
        c = gen.make_conv_case(N, H, W, C, F, R, S, seed=20 + seed, pad=pad, stride=stride, dist="uniform")
        y, s = co.conv2d(c.x, c.w, pad, stride)
        K = R * S * C
        for n in range(N):
            for p in range(c.P):
                for q in range(c.Q):
                    for f in range(F):
                        acc, sab = Fraction(0), Fraction(0)
                        for r in range(R):
                            for ss in range(S):
                                h, ww = p * stride[0] + r - pad[0], q * stride[1] + ss - pad[1]
                                if 0 <= h < H and 0 <= ww < W:
                                    for ch in range(C):
                                        a, b = frac(c.x[n, h, ww, ch]), frac(c.w[f, r, ss, ch])
                                        acc += a * b
                                        sab += abs(a * b)
                        assert abs(Fraction(float(y[n, p, q, f])) - acc) <= Fraction(K) * Fraction(1, 2 ** 52) * sab
                        assert abs(Fraction(float(s[n, p, q, f])) - sab) <= Fraction(K) * Fraction(1, 2 ** 52) * sab


def test_fp16_rounding_is_to_nearest_even():
    # 2049 lies between 2048 and 2050 (spacing 2 above 2048): tie -> even mantissa (2048); 2051 -> 2052
    got = co.round_to_f16(np.array([2049.0, 2051.0, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 65520.0, -0.0]))
    want = f16([2048.0, 2052.0, 1.0, 1.0 + 2.0 ** -9, np.inf, -0.0])
    assert np.array_equal(got, want)


def test_bad_geometry_is_rejected():
    c = gen.make_conv_case(1, 2, 2, 1, 1, 3, 3, seed=1, pad=(0, 0))
    with pytest.raises(ValueError):
        co.conv2d(c.x, c.w, (0, 0), (1, 1))
