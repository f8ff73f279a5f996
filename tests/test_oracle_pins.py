"""Pins for the CPU oracle: each test fixes it to something other than itself.

The paper (Evaluation, Setup) says only that correctness is checked with three
random seeds against a vendor reference and prints no GEMM values, so the
pins are mathematics: exact rational arithmetic, closed forms, invariants, a
hand-worked example and library routines used as cross-checks.
"""
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest

from oracle import gemm_oracle as orc
from paper_2605_28213_b200 import inputs as gen

GOLDEN = Path(__file__).resolve().parent / "golden"


def bits_of(values) -> np.ndarray:
    """bf16 bit patterns of values that are exactly representable in bf16."""
    v = np.asarray(values, dtype=np.float32)
    bits = (v.view(np.uint32) >> np.uint32(16)).astype(np.uint16)
    assert np.array_equal(gen.bf16_bits_to_f32(bits), v), "test value not exact in bf16"
    return bits


def frac_of_bits(b: int) -> Fraction:
    """Exact rational value of one bf16 bit pattern, decoded by hand (not via numpy)."""
    sign = -1 if (b >> 15) & 1 else 1
    e = (b >> 7) & 0xFF
    m = b & 0x7F
    assert e != 0xFF
    if e == 0:
        return sign * Fraction(m, 1 << 7) * Fraction(1, 1 << 126)
    mant = Fraction((1 << 7) + m, 1 << 7)
    return sign * mant * (Fraction(2) ** (e - 127))


def exact_product(A, B, absolute=False):
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    out = [[Fraction(0)] * N for _ in range(M)]
    for i in range(M):
        for j in range(N):
            acc = Fraction(0)
            for k in range(K):
                t = frac_of_bits(int(A[i, k])) * frac_of_bits(int(B[k, j]))
                acc += abs(t) if absolute else t
            out[i][j] = acc
    return out


def run_oracle(A, B, b_col_major=False, lda=None, ldb=None, **kw):
    """A: (M,K) bits, B: logical (K,N) bits."""
    M, K = A.shape
    N = B.shape[1]
    lda = K if lda is None else lda
    Bs = np.ascontiguousarray(B.T) if b_col_major else B
    ldb = Bs.shape[1] if ldb is None else ldb
    return orc.gemm(M, N, K, gen.with_ld(A, lda), lda, gen.with_ld(Bs, ldb), ldb, b_col_major, **kw)


# ---------------------------------------------------------------- brute force
def narrow_bits(rng, shape):
    """bf16 values +-(128..255) * 2^e, e in [-15, 1]: any K<=8 sum of products fits 53 bits."""
    mant = rng.integers(128, 256, size=shape).astype(np.float64)
    e = rng.integers(-15, 2, size=shape)
    sign = rng.choice([-1.0, 1.0], size=shape)
    return bits_of(sign * mant * np.exp2(e.astype(np.float64)))


SMALL_SHAPES = [(m, n, k) for m in range(1, 5) for n in range(1, 5) for k in range(1, 5)] + \
               [(8, 8, 8), (5, 7, 6), (1, 8, 7), (7, 1, 8), (3, 2, 8)]


@pytest.mark.parametrize("col", [False, True])
def test_brute_force_exact_rational(col):
    """With a 53-bit-safe exponent range the fp64 sum is exact: oracle == rational value."""
    rng = np.random.default_rng(11)
    for (M, N, K) in SMALL_SHAPES:
        A, B = narrow_bits(rng, (M, K)), narrow_bits(rng, (K, N))
        C, S = run_oracle(A, B, b_col_major=col)
        exC, exS = exact_product(A, B), exact_product(A, B, absolute=True)
        for i in range(M):
            for j in range(N):
                assert Fraction(float(C[i, j])) == exC[i][j], (M, N, K, i, j)
                assert Fraction(float(S[i, j])) == exS[i][j], (M, N, K, i, j)


def test_brute_force_general_values_within_fp64_bound():
    """Uniform bf16 draws (wide exponents): |oracle - exact| <= K * 2^-53 * S_exact."""
    for seed, (M, N, K) in enumerate([(4, 4, 4), (3, 5, 8), (8, 8, 8), (2, 3, 7)]):
        A = gen.draw((M, K), "uniform", seed, 0)
        B = gen.draw((K, N), "normal", seed, 1, 3.0)
        C, S = run_oracle(A, B)
        exC, exS = exact_product(A, B), exact_product(A, B, absolute=True)
        for i in range(M):
            for j in range(N):
                bound = Fraction(K, 1 << 53) * exS[i][j]
                assert abs(Fraction(float(C[i, j])) - exC[i][j]) <= bound
                assert abs(Fraction(float(S[i, j])) - exS[i][j]) <= bound


def test_hand_worked_example():
    rows = {}
    for line in (GOLDEN / "hand_worked_2x3x2.txt").read_text().splitlines():
        if line and not line.startswith("#"):
            key, *vals = line.split()
            rows[key] = np.array([float(v) for v in vals])
    A = bits_of(rows["A"].reshape(2, 3))
    B = bits_of(rows["B"].reshape(3, 2))
    for col in (False, True):
        C, S = run_oracle(A, B, b_col_major=col)
        assert np.array_equal(C.ravel(), rows["C"])
        assert np.array_equal(S.ravel(), rows["S"])
        got = gen.bf16_bits_to_f32(orc.round_to_bf16(C)).ravel()
        assert np.array_equal(got, rows["C_BF16"].astype(np.float32))


def test_addmm_reference_is_product_plus_row_bias():
    """The AddMM reference used by the GPU tests: oracle product + bias broadcast along rows, in fp64."""
    rows = {}
    for line in (GOLDEN / "hand_worked_2x3x2.txt").read_text().splitlines():
        if line and not line.startswith("#"):
            key, *vals = line.split()
            rows[key] = np.array([float(v) for v in vals])
    A, B = bits_of(rows["A"].reshape(2, 3)), bits_of(rows["B"].reshape(3, 2))
    bias = bits_of([0.5, -2.0])
    C, S = run_oracle(A, B)
    got = C + orc.bf16_bits_to_f64(bias)[None, :]
    # by hand: C = [[0, -4.71875], [-139.5, 3.5]]  ->  [[0.5, -6.71875], [-139, 1.5]]
    assert np.array_equal(got, np.array([[0.5, -6.71875], [-139.0, 1.5]]))


# ------------------------------------------------------------- index / layout
def test_identity_left_and_right():
    B = gen.draw((37, 53), "normal", 5, 1)
    I = bits_of(np.eye(37))
    C, S = run_oracle(I, B)
    assert np.array_equal(C, orc.bf16_bits_to_f64(B))
    assert np.array_equal(S, np.abs(orc.bf16_bits_to_f64(B)))
    A = gen.draw((29, 41), "uniform", 5, 0)
    C, _ = run_oracle(A, bits_of(np.eye(41)), b_col_major=True)
    assert np.array_equal(C, orc.bf16_bits_to_f64(A))
    # bf16 output of an identity product round-trips the bits
    assert np.array_equal(orc.round_to_bf16(C), A)


def test_permutation_rows_and_columns():
    rng = np.random.default_rng(3)
    n = 23
    perm = rng.permutation(n)
    P = np.zeros((n, n))
    P[np.arange(n), perm] = 1.0           # (P.B)[i] = B[perm[i]]
    B = gen.draw((n, 17), "normal", 9, 1)
    C, _ = run_oracle(bits_of(P), B)
    assert np.array_equal(C, orc.bf16_bits_to_f64(B)[perm])
    A = gen.draw((19, n), "uniform", 9, 0)
    for col in (False, True):
        C, _ = run_oracle(A, bits_of(P), b_col_major=col)   # (A.P)[:, perm[i]] = A[:, i]
        expect = np.zeros((19, n))
        expect[:, perm] = orc.bf16_bits_to_f64(A)
        assert np.array_equal(C, expect)


def test_single_nonzero_picks_the_right_indices():
    """A = e_i e_k^T, B arbitrary: C has row i equal to row k of B, zeros elsewhere."""
    M, N, K = 5, 6, 7
    B = gen.draw((K, N), "uniform", 2, 1)
    for (i, k) in [(0, 6), (4, 0), (2, 3)]:
        A = np.zeros((M, K))
        A[i, k] = -2.0
        for col in (False, True):
            C, _ = run_oracle(bits_of(A), B, b_col_major=col)
            expect = np.zeros((M, N))
            expect[i] = -2.0 * orc.bf16_bits_to_f64(B)[k]
            assert np.array_equal(C, expect)


def test_layout_and_leading_dimension_invariance():
    A = gen.draw((31, 45), "uniform", 4, 0)
    B = gen.draw((45, 27), "uniform", 4, 1)
    C0, S0 = run_oracle(A, B)
    for col in (False, True):
        for pad in (0, 1, 8, 13):
            C, S = run_oracle(A, B, b_col_major=col, lda=45 + pad,
                              ldb=(45 if col else 27) + pad)
            assert np.array_equal(C, C0) and np.array_equal(S, S0)
            assert not np.isnan(C).any()     # NaN padding never read


def test_not_symmetric_in_operands():
    """A transposed-operand mistake cannot hide: A.B != (B^T.A^T) laid out the same way."""
    A = gen.draw((6, 6), "integer", 1, 0)
    B = gen.draw((6, 6), "integer", 1, 1)
    Cab, _ = run_oracle(A, B)
    Cba, _ = run_oracle(B, A)
    a, b = orc.bf16_bits_to_f64(A), orc.bf16_bits_to_f64(B)
    assert np.array_equal(Cab, a @ b) and np.array_equal(Cba, b @ a)
    assert not np.array_equal(Cab, Cba)


# ------------------------------------------------------------ reduction over k
RANK1_SET = np.array([1.0, 1.125, 1.25, 1.375, 1.5, 1.625, 1.75, 1.875])


@pytest.mark.parametrize("K", [1, 7, 64, 999, 8192])
def test_rank_one_closed_form(K):
    """A_ik = u_i, B_kj = v_j with 4-bit significands: C_ij = K u_i v_j exactly."""
    rng = np.random.default_rng(K)
    M, N = 9, 11
    u = rng.choice(RANK1_SET, M) * rng.choice([-1, 1], M) * np.exp2(rng.integers(-3, 4, M))
    v = rng.choice(RANK1_SET, N) * rng.choice([-1, 1], N) * np.exp2(rng.integers(-3, 4, N))
    A = bits_of(np.repeat(u[:, None], K, axis=1))
    B = bits_of(np.repeat(v[None, :], K, axis=0))
    for col in (False, True):
        C, S = run_oracle(A, B, b_col_major=col)
        assert np.array_equal(C, K * np.outer(u, v))
        assert np.array_equal(S, K * np.abs(np.outer(u, v)))


@pytest.mark.parametrize("shape", [(16, 16, 16), (33, 65, 129), (100, 101, 999)])
def test_integer_inputs_match_int64_matmul(shape):
    M, N, K = shape
    A = gen.draw((M, K), "integer", 7, 0)
    B = gen.draw((K, N), "integer", 7, 1)
    ai = gen.bf16_bits_to_f32(A).astype(np.int64)
    bi = gen.bf16_bits_to_f32(B).astype(np.int64)
    assert ai.min() >= -4 and ai.max() <= 4
    for col in (False, True):
        C, S = run_oracle(A, B, b_col_major=col)
        assert np.array_equal(C, (ai @ bi).astype(np.float64))
        assert np.array_equal(S, (np.abs(ai) @ np.abs(bi)).astype(np.float64))


@pytest.mark.parametrize("shape", [(64, 48, 300), (17, 130, 1025)])
def test_against_fp64_library_matmul(shape):
    M, N, K = shape
    A = gen.draw((M, K), "normal", 21, 0)
    B = gen.draw((K, N), "normal", 21, 1, 0.02)
    C, S = run_oracle(A, B)
    a, b = orc.bf16_bits_to_f64(A), orc.bf16_bits_to_f64(B)
    assert np.all(np.abs(C - a @ b) <= 4 * K * 2.0 ** -53 * S)
    assert np.all(np.abs(S - np.abs(a) @ np.abs(b)) <= 4 * K * 2.0 ** -53 * S)
    assert np.all(S >= np.abs(C))


def test_scaling_by_powers_of_two_is_exact():
    A = gen.draw((12, 40), "uniform", 8, 0)
    B = gen.draw((40, 10), "uniform", 8, 1)
    C, _ = run_oracle(A, B)
    a4 = bits_of(gen.bf16_bits_to_f32(A) * 4.0)
    C4, _ = run_oracle(a4, B)
    assert np.array_equal(C4, 4.0 * C)


def test_zero_rows_and_columns_give_exact_zero_and_zero_bound():
    A = gen.draw((6, 20), "uniform", 8, 0)
    B = gen.draw((20, 5), "uniform", 8, 1)
    A[2, :] = 0
    B[:, 3] = 0
    C, S = run_oracle(A, B)
    assert np.all(C[2] == 0) and np.all(C[:, 3] == 0)
    assert np.all(S[2] == 0) and np.all(S[:, 3] == 0)


# ---------------------------------------------------------------- edges / slab
def test_degenerate_sizes():
    A = gen.draw((3, 4), "uniform", 1, 0)
    B = gen.draw((4, 5), "uniform", 1, 1)
    C, S = orc.gemm(3, 5, 0, A, 4, B, 5)          # K = 0 -> zeros
    assert C.shape == (3, 5) and np.all(C == 0) and np.all(S == 0)
    C, _ = orc.gemm(0, 5, 4, A, 4, B, 5)
    assert C.shape == (0, 5)
    C, _ = orc.gemm(3, 0, 4, A, 4, B, 5)
    assert C.shape == (3, 0)
    with pytest.raises(ValueError):
        orc.gemm(3, 5, 4, A, 3, B, 5)             # lda < K


def test_row_slab_equals_full_and_leaves_other_rows_nan():
    A = gen.draw((40, 33), "uniform", 6, 0)
    B = gen.draw((33, 21), "uniform", 6, 1)
    C, S = run_oracle(A, B)
    Cs, Ss = run_oracle(A, B, rows=(7, 19))
    assert np.array_equal(Cs[7:19], C[7:19]) and np.array_equal(Ss[7:19], S[7:19])
    assert np.isnan(Cs[:7]).all() and np.isnan(Cs[19:]).all()


def test_thread_count_does_not_change_bits():
    A = gen.draw((64, 200), "normal", 6, 0)
    B = gen.draw((200, 64), "normal", 6, 1)
    C1, S1 = run_oracle(A, B, nthreads=1)
    C4, S4 = run_oracle(A, B, nthreads=4)
    assert np.array_equal(C1, C4) and np.array_equal(S1, S4)


# -------------------------------------------------------------- bf16 rounding
def test_round_to_bf16_hand_listed_cases():
    cases = [
        (1.0, 0x3F80), (-1.0, 0xBF80), (0.0, 0x0000),
        (1.0 + 2.0 ** -8, 0x3F80),            # tie, even significand below
        (1.0 + 3 * 2.0 ** -8, 0x3F82),        # tie, even significand above
        (1.0 + 2.0 ** -8 + 2.0 ** -20, 0x3F81),   # just above the tie
        (1.0 + 2.0 ** -7, 0x3F81),            # exact
        (255.5, 0x4380),                      # 255.5 -> 256 (tie to even carries)
        (131072.0, 0x4800), (-139.5, 0xC30C),
        (3.3895313892515355e38, 0x7F7F),      # largest finite bf16
    ]
    for x, bits in cases:
        assert int(orc.round_to_bf16(np.array([x]))[0]) == bits, x


def test_round_to_bf16_matches_torch_conversion():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000) * 37.0, rng.uniform(-1, 1, 20000) * 1e-3,
                        np.arange(-300, 300) / 2.0]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.round_to_bf16(x.astype(np.float64)), ref)


# ------------------------------------------------------------------ tolerance
def test_bounds_have_the_stated_constants():
    S = np.array([[1.0, 4.0]])
    assert np.array_equal(orc.bound_f32(256, S), np.array([[256 * 2.0 ** -23, 4 * 256 * 2.0 ** -23]]))
    assert orc.bound_f32(8192, np.array([1.0]))[0] == 2.0 ** -10
    Cref = np.array([[2.0, -8.0]])
    tol = orc.bound_f32(256, S)
    assert np.array_equal(orc.bound_bf16(256, S, Cref), tol + 2.0 ** -8 * (np.abs(Cref) + tol))


def test_bound_is_tight_enough_to_catch_a_dropped_term_on_integer_inputs():
    """Integer inputs are compared bit-exactly: dropping one product changes the value."""
    A = gen.draw((8, 64), "integer", 3, 0)
    B = gen.draw((64, 8), "integer", 3, 1)
    A[A == 0] = bits_of([1.0])[0]
    B[B == 0] = bits_of([1.0])[0]
    C, _ = run_oracle(A, B)
    C_drop, _ = run_oracle(A[:, :-1].copy(), B[:-1].copy())
    assert np.all(C != C_drop)
