"""Pins for the FP64 GEMM oracle (C = A*B; Sec. 2 problem statement, Listing 2).

None of these re-types the oracle's loop: each fixes the result by a closed
form, an exact special case, an identity, or exact rational arithmetic.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2503_14985_b200 import inputs

bits = inputs.f64_to_bf16_bits
f64 = inputs.bf16_bits_to_f64


def test_identity_left_and_right():
    _, B = inputs.gemm_inputs(48, 40, 48, seed=11)
    eye = bits(np.eye(48))
    assert np.array_equal(oracle.gemm(eye, B, 48, 40, 48), f64(B))
    A, _ = inputs.gemm_inputs(33, 40, 40, seed=12)
    eye = bits(np.eye(40))
    assert np.array_equal(oracle.gemm(A, eye, 33, 40, 40), f64(A))


def test_permutation_matrices_move_rows_and_columns():
    rng = np.random.default_rng(0)
    _, B = inputs.gemm_inputs(31, 29, 31, seed=13)
    perm = rng.permutation(31)
    P = np.zeros((31, 31)); P[np.arange(31), perm] = 1.0     # row i of P*B = row perm[i] of B
    assert np.array_equal(oracle.gemm(bits(P), B, 31, 29, 31), f64(B)[perm])
    A, _ = inputs.gemm_inputs(17, 23, 23, seed=14)
    perm = rng.permutation(23)
    P = np.zeros((23, 23)); P[perm, np.arange(23)] = 1.0     # column j of A*P = column perm[j] of A
    assert np.array_equal(oracle.gemm(A, bits(P), 17, 23, 23), f64(A)[:, perm])


@pytest.mark.parametrize("K", [1, 7, 512, 4096])
def test_all_ones_gives_K(K):
    A = bits(np.ones((5, K))); B = bits(np.ones((K, 9)))
    assert np.array_equal(oracle.gemm(A, B, 5, 9, K), np.full((5, 9), float(K)))


def test_single_nonzero_with_padded_pitch():
    # padding holds NaN patterns: any read of it would poison the result
    M, N, K, lda, ldb = 20, 27, 19, 24, 32
    _, B = inputs.gemm_inputs(M, N, K, seed=15, ldb=ldb)
    for (i0, k0) in [(0, 0), (19, 18), (7, 11)]:
        A = np.full((M, lda), 0x7FC0, dtype=np.uint16)
        A[:, :K] = 0
        A[i0, k0] = bits(np.array([-1.5]))[0]
        C = oracle.gemm(A, B, M, N, K)
        want = np.zeros((M, N)); want[i0] = -1.5 * f64(B)[k0, :N]
        assert np.array_equal(C, want)


def test_transposed_operand_would_fail():
    # non-symmetric small integers: (A*B) != (A^T*B), (A*B^T), (B*A)
    A = bits(np.array([[1., 2., 0.], [0., 1., 3.], [4., 0., 1.]]))
    B = bits(np.array([[1., 0., 2.], [3., 1., 0.], [0., 5., 1.]]))
    want = np.array([[7., 2., 2.], [3., 16., 3.], [4., 5., 9.]])   # worked by hand
    assert np.array_equal(oracle.gemm(A, B, 3, 3, 3), want)


def test_k_split_additivity():
    M, N, K1, K2 = 13, 21, 37, 64
    A, B = inputs.gemm_inputs(M, N, K1 + K2, seed=16)
    whole = oracle.gemm(A, B, M, N, K1 + K2)
    first = oracle.gemm(np.ascontiguousarray(A[:, :K1]), B[:K1], M, N, K1)
    second = oracle.gemm(np.ascontiguousarray(A[:, K1:]), B[K1:], M, N, K2)
    np.testing.assert_allclose(whole, first + second, rtol=0, atol=1e-14)


def test_exact_rational_brute_force():
    M, N, K = 5, 6, 7
    A, B = inputs.gemm_inputs(M, N, K, seed=17, kind="uniform")
    a, b = f64(A), f64(B)
    C = oracle.gemm(A, B, M, N, K)
    for i in range(M):
        for j in range(N):
            exact = sum((Fraction(a[i, k]) * Fraction(b[k, j]) for k in range(K)), Fraction(0))
            assert abs(Fraction(C[i, j]) - exact) <= Fraction(1, 2 ** 48) * max(abs(exact), Fraction(1))


def test_row_subset_matches_full_and_numpy_matmul():
    M, N, K = 70, 45, 130
    A, B = inputs.gemm_inputs(M, N, K, seed=18, lda=136, ldb=48)
    full = oracle.gemm(A, B, M, N, K)
    rows = [0, 69, 5, 5, 33]
    assert np.array_equal(oracle.gemm(A, B, M, N, K, rows=rows), full[rows])
    # reduces to a library routine
    np.testing.assert_allclose(full, f64(A)[:, :K] @ f64(B)[:, :N], rtol=1e-13, atol=1e-13)
    # thread count does not change a single bit (rows are independent)
    assert np.array_equal(oracle.gemm(A, B, M, N, K, nthreads=1), oracle.gemm(A, B, M, N, K, nthreads=3))


def test_degenerate_sizes():
    A, B = inputs.gemm_inputs(4, 6, 0, seed=19)
    assert np.array_equal(oracle.gemm(A, B, 4, 6, 0), np.zeros((4, 6)))     # K = 0 -> zeros
    assert oracle.gemm(np.zeros((0, 8), np.uint16), np.zeros((8, 3), np.uint16), 0, 3, 8).shape == (0, 3)
