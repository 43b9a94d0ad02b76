"""Pins for the FP16-input GEMM oracle (Listing 2 data types; C += A*B of Sec. 2).

The conversion is pinned over all 65536 bit patterns against the format's
definition evaluated in exact rational arithmetic and against numpy's
independent float16 type; the product against exact special cases, hand-worked
values and exact rationals; the accumulate form against cases where the prior
C alone, or the product alone, fixes the result.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2503_14985_b200 import inputs

h = inputs.f64_to_f16_bits


def hval(b):
    return np.asarray(b, dtype=np.uint16).view(np.float16).astype(np.float64)


def test_conversion_matches_numpy_for_every_pattern():
    allbits = np.arange(65536, dtype=np.uint16)
    got = oracle.f16_to_double(allbits)
    want = allbits.view(np.float16).astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))      # -0.0 keeps its sign


def test_conversion_landmarks_from_the_format_definition():
    # binary16: smallest subnormal 2^-24, smallest normal 2^-14, largest 65504, 1 + 2^-10 after 1
    cases = {0x0001: Fraction(1, 2 ** 24), 0x03FF: Fraction(1023, 2 ** 24), 0x0400: Fraction(1, 2 ** 14),
             0x3C00: Fraction(1), 0x3C01: Fraction(1025, 1024), 0x7BFF: Fraction(65504), 0xC000: Fraction(-2),
             0x3555: Fraction(1024 + 0x155, 1024) / 4, 0xB800: Fraction(-1, 2)}
    got = oracle.f16_to_double(np.array(list(cases), dtype=np.uint16))
    for g, w in zip(got, cases.values()):
        assert Fraction(float(g)) == w
    inf = oracle.f16_to_double(np.array([0x7C00, 0xFC00], dtype=np.uint16))
    assert inf[0] == np.inf and inf[1] == -np.inf


def test_a_bf16_reading_of_the_bits_would_fail():
    # 0x3C00 is 1.0 in binary16 but 2^-7 in BF16; 0x4000 is 2.0 but 2.0 in both -- use the first
    A = np.full((1, 1), 0x3C00, dtype=np.uint16)
    B = np.full((1, 1), 0x4200, dtype=np.uint16)                              # binary16 3.0
    assert oracle.gemm_f16(A, B, 1, 1, 1)[0, 0] == 3.0


def test_identity_and_permutation():
    _, B, _ = inputs.gemm_f16_inputs(48, 40, 48, seed=21)
    assert np.array_equal(oracle.gemm_f16(h(np.eye(48)), B, 48, 40, 48), hval(B))
    rng = np.random.default_rng(1)
    perm = rng.permutation(48)
    P = np.zeros((48, 48)); P[np.arange(48), perm] = 1.0
    assert np.array_equal(oracle.gemm_f16(h(P), B, 48, 40, 48), hval(B)[perm])
    A, _, _ = inputs.gemm_f16_inputs(17, 23, 23, seed=22)
    perm = rng.permutation(23)
    P = np.zeros((23, 23)); P[perm, np.arange(23)] = 1.0
    assert np.array_equal(oracle.gemm_f16(A, h(P), 17, 23, 23), hval(A)[:, perm])


def test_hand_worked_nonsymmetric_product_and_accumulate():
    A = h(np.array([[1., 2., 0.], [0., 1., 3.], [4., 0., 1.]]))
    B = h(np.array([[1., 0., 2.], [3., 1., 0.], [0., 5., 1.]]))
    want = np.array([[7., 2., 2.], [3., 16., 3.], [4., 5., 9.]])               # worked by hand
    assert np.array_equal(oracle.gemm_f16(A, B, 3, 3, 3), want)
    C0 = np.array([[10., -1., 0.5], [0., 0., -16.], [100., 0.25, -9.]], dtype=np.float32)
    want_acc = np.array([[17., 1., 2.5], [3., 16., -13.], [104., 5.25, 0.]])   # worked by hand
    assert np.array_equal(oracle.gemm_f16(A, B, 3, 3, 3, C_in=C0), want_acc)


@pytest.mark.parametrize("K", [1, 7, 512, 4096])
def test_all_ones_gives_K_plus_prior(K):
    A = h(np.ones((5, K))); B = h(np.ones((K, 9)))
    assert np.array_equal(oracle.gemm_f16(A, B, 5, 9, K), np.full((5, 9), float(K)))
    C0 = np.full((5, 9), -3.0, dtype=np.float32)
    assert np.array_equal(oracle.gemm_f16(A, B, 5, 9, K, C_in=C0), np.full((5, 9), float(K) - 3.0))


def test_accumulate_with_zero_operand_or_k0_returns_prior_c():
    M, N, K = 9, 14, 11
    A, B, C0 = inputs.gemm_f16_inputs(M, N, K, seed=23, ldc=16)
    Z = np.zeros_like(A)
    assert np.array_equal(oracle.gemm_f16(Z, B, M, N, K, C_in=C0), C0[:, :N].astype(np.float64))
    assert np.array_equal(oracle.gemm_f16(A[:, :0], B[:0], M, N, 0, C_in=C0), C0[:, :N].astype(np.float64))
    assert np.array_equal(oracle.gemm_f16(A[:, :0], B[:0], M, N, 0), np.zeros((M, N)))


def test_accumulate_is_product_plus_prior_and_reads_the_right_pitch():
    M, N, K = 12, 10, 33
    A, B, C0 = inputs.gemm_f16_inputs(M, N, K, seed=24, lda=40, ldb=16, ldc=12)   # NaN in every padding column
    plain = oracle.gemm_f16(A, B, M, N, K)
    acc = oracle.gemm_f16(A, B, M, N, K, C_in=C0)
    assert np.isfinite(acc).all()
    np.testing.assert_allclose(acc - plain, C0[:, :N].astype(np.float64), rtol=0, atol=1e-14)
    rows = [11, 0, 5]
    assert np.array_equal(oracle.gemm_f16(A, B, M, N, K, C_in=C0, rows=rows), acc[rows])


def test_exact_rational_brute_force():
    M, N, K = 4, 5, 6
    A, B, C0 = inputs.gemm_f16_inputs(M, N, K, seed=25, kind="uniform")
    a, b = hval(A), hval(B)
    C = oracle.gemm_f16(A, B, M, N, K, C_in=C0)
    for i in range(M):
        for j in range(N):
            exact = sum((Fraction(float(a[i, k])) * Fraction(float(b[k, j])) for k in range(K)), Fraction(0))
            exact += Fraction(float(C0[i, j]))
            assert abs(Fraction(float(C[i, j])) - exact) <= Fraction(1, 2 ** 48)


def test_agrees_with_the_bf16_oracle_on_values_both_formats_hold():
    # small integers are exact in both encodings: the two oracles must give the same product
    M, N, K = 14, 19, 50
    A16, B16 = inputs.gemm_inputs(M, N, K, seed=26, kind="ternary")
    v = inputs.bf16_bits_to_f64
    got = oracle.gemm_f16(h(v(A16)), h(v(B16)), M, N, K)
    assert np.array_equal(got, oracle.gemm(A16, B16, M, N, K))


def test_generator_rounds_to_nearest_even_binary16():
    # 1 + 2^-11 is a tie between 1 and 1 + 2^-10 (even: 1); 1 + 3*2^-11 ties to 1 + 2^-9
    assert list(h(np.array([1 + 2.0 ** -11, 1 + 3 * 2.0 ** -11, 65520.0, 2.0 ** -25]))) == [0x3C00, 0x3C02, 0x7C00, 0]
    A, B, C = inputs.gemm_f16_inputs(6, 7, 5, seed=27, lda=8, ldb=8, ldc=8)
    assert np.all(A[:, 5:] == 0x7E00) and np.all(B[:, 7:] == 0x7E00) and np.isnan(C[:, 7:]).all()
    Abf, _ = inputs.gemm_inputs(6, 7, 5, seed=27, lda=8)
    # same underlying values as the BF16 generator (binary16 keeps 3 more fraction bits)
    assert np.allclose(hval(A[:, :5]), inputs.bf16_bits_to_f64(Abf[:, :5]), rtol=2.0 ** -8, atol=2.0 ** -14)
