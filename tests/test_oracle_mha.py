"""Pins for the FP64 attention oracle (Algorithm 1: FlashAttention-2 forward
computes exact softmax attention; scale, causal mask, 1/l and LSE as the
benchmark configuration states them).

Each test fixes the result by a closed form, an invariant of softmax attention,
or an independently written brute-force evaluation.
"""
import math

import numpy as np
import pytest

import oracle
from paper_2503_14985_b200 import inputs

bits = inputs.f64_to_bf16_bits
f64 = inputs.bf16_bits_to_f64


def _qkv(B, H, Nq, Nk, D, seed, **kw):
    return inputs.mha_inputs(B, H, Nq, Nk, D, seed=seed, **kw)


def test_constant_keys_give_mean_of_values():
    B, H, N, D = 1, 2, 37, 8
    Q, K, V = _qkv(B, H, N, N, D, 21)
    K[:] = K[:, :, :1, :]                      # every key equal to key 0
    q, k, v = f64(Q), f64(K), f64(V)
    scale = np.float32(0.3)
    O, L = oracle.mha_fwd(Q, K, V, causal=False, scale=scale)
    O = O.reshape(B, H, N, D); L = L.reshape(B, H, N)
    s = float(scale) * np.einsum("bhid,bhd->bhi", q, k[:, :, 0])
    np.testing.assert_allclose(O, np.broadcast_to(v.mean(axis=2, keepdims=True), O.shape), atol=1e-13)
    np.testing.assert_allclose(L, s + math.log(N), atol=1e-12)
    Oc, Lc = oracle.mha_fwd(Q, K, V, causal=True, scale=scale)
    Oc = Oc.reshape(B, H, N, D); Lc = Lc.reshape(B, H, N)
    prefix_mean = np.cumsum(v, axis=2) / np.arange(1, N + 1)[None, None, :, None]
    np.testing.assert_allclose(Oc, prefix_mean, atol=1e-13)
    np.testing.assert_allclose(Lc, s + np.log(np.arange(1, N + 1)), atol=1e-12)


def test_zero_keys_lse_is_log_count():
    Q, K, V = _qkv(1, 1, 9, 9, 4, 22)
    K[:] = 0
    _, L = oracle.mha_fwd(Q, K, V, causal=True, scale=1.0)
    np.testing.assert_allclose(L, np.log(np.arange(1, 10)), atol=1e-15)


def test_causal_row0_is_value0():
    Q, K, V = _qkv(2, 3, 16, 16, 8, 23)
    scale = np.float32(1 / math.sqrt(8))
    O, L = oracle.mha_fwd(Q, K, V, causal=True, scale=scale)
    O = O.reshape(2, 3, 16, 8); L = L.reshape(2, 3, 16)
    assert np.array_equal(O[:, :, 0], f64(V)[:, :, 0])
    s00 = float(scale) * np.einsum("bhd,bhd->bh", f64(Q)[:, :, 0], f64(K)[:, :, 0])
    np.testing.assert_allclose(L[:, :, 0], s00, atol=1e-14)


def test_single_key_and_constant_value():
    Q, K, V = _qkv(1, 2, 5, 1, 8, 24)
    O, _ = oracle.mha_fwd(Q, K, V, causal=False, scale=0.7)
    assert np.array_equal(O.reshape(1, 2, 5, 8), np.broadcast_to(f64(V), (1, 2, 5, 8)))
    Q, K, V = _qkv(1, 1, 6, 11, 4, 25)
    V[:] = bits(np.array([0.75]))[0]
    O, _ = oracle.mha_fwd(Q, K, V, causal=False, scale=0.7)
    np.testing.assert_allclose(O, 0.75, atol=1e-15)


def test_probabilities_sum_to_one_and_respect_mask():
    Q, K, V = _qkv(1, 2, 7, 10, 4, 26)
    for causal in (False, True):
        O, L, P = oracle.mha_fwd(Q, K, V, causal=causal, scale=0.5, return_probs=True)
        np.testing.assert_allclose(P.sum(axis=1), 1.0, atol=1e-15)
        assert (P >= 0).all()
        P = P.reshape(1, 2, 7, 10)
        if causal:                              # bottom-right aligned: j <= i + (Nk - Nq)
            for i in range(7):
                assert (P[:, :, i, i + 4:] == 0).all() and (P[:, :, i, :i + 4] > 0).all()
        np.testing.assert_allclose(np.einsum("bhij,bhjd->bhid", P, f64(V)).reshape(-1, 4), O, atol=1e-14)


def test_key_permutation_invariance():
    Q, K, V = _qkv(1, 2, 12, 33, 8, 27)
    perm = np.random.default_rng(1).permutation(33)
    O1, L1 = oracle.mha_fwd(Q, K, V, causal=False, scale=0.4)
    O2, L2 = oracle.mha_fwd(Q, np.ascontiguousarray(K[:, :, perm]), np.ascontiguousarray(V[:, :, perm]),
                            causal=False, scale=0.4)
    np.testing.assert_allclose(O1, O2, atol=1e-13)
    np.testing.assert_allclose(L1, L2, atol=1e-13)


def test_split_merge_identity_pins_natural_log_lse():
    Q, K, V = _qkv(1, 1, 9, 40, 8, 28)
    O, L = oracle.mha_fwd(Q, K, V, causal=False, scale=0.35)
    O1, L1 = oracle.mha_fwd(Q, np.ascontiguousarray(K[:, :, :13]), np.ascontiguousarray(V[:, :, :13]),
                            causal=False, scale=0.35)
    O2, L2 = oracle.mha_fwd(Q, np.ascontiguousarray(K[:, :, 13:]), np.ascontiguousarray(V[:, :, 13:]),
                            causal=False, scale=0.35)
    w1, w2 = np.exp(L1), np.exp(L2)
    np.testing.assert_allclose(L, np.log(w1 + w2), atol=1e-13)
    np.testing.assert_allclose(O, (w1[:, None] * O1 + w2[:, None] * O2) / (w1 + w2)[:, None], atol=1e-13)


def test_key_shift_invariance():
    # adding the same vector c to every key adds scale*q.c to LSE and leaves O unchanged;
    # small dyadic values keep the shifted keys exactly representable in BF16
    rng = np.random.default_rng(2)
    B, H, Nq, Nk, D = 1, 1, 6, 9, 4
    q = rng.integers(-4, 5, (B, H, Nq, D)) / 4.0
    k = rng.integers(-4, 5, (B, H, Nk, D)) / 4.0
    v = rng.integers(-8, 9, (B, H, Nk, D)) / 8.0
    c = np.array([0.5, -1.0, 0.25, 2.0])
    O1, L1 = oracle.mha_fwd(bits(q), bits(k), bits(v), causal=False, scale=0.5)
    O2, L2 = oracle.mha_fwd(bits(q), bits(k + c), bits(v), causal=False, scale=0.5)
    np.testing.assert_allclose(O1, O2, atol=1e-14)
    np.testing.assert_allclose(L2 - L1, 0.5 * (q.reshape(-1, D) @ c), atol=1e-13)


def test_dominant_key_selects_its_value():
    B, H, N, D = 1, 1, 20, 8
    Q, K, V = _qkv(B, H, N, N, D, 29)
    q, k = f64(Q), f64(K)
    j0 = 13
    qhat = q[0, 0, 4] / np.linalg.norm(q[0, 0, 4])
    k[0, 0, j0] = 64.0 * qhat
    K = bits(k); k = f64(K)
    O, L = oracle.mha_fwd(Q, K, V, causal=False, scale=1.0)
    np.testing.assert_allclose(O[4], f64(V)[0, 0, j0], atol=1e-9)
    np.testing.assert_allclose(L[4], q[0, 0, 4] @ k[0, 0, j0], atol=1e-9)


def _brute(q, k, v, scale, causal):
    """Independent evaluation with Python floats and math.fsum; masked keys get -inf."""
    Nq, D = q.shape; Nk = k.shape[0]
    O = np.zeros((Nq, D)); L = np.zeros(Nq)
    for i in range(Nq):
        s = []
        for j in range(Nk):
            masked = causal and j > i + (Nk - Nq)
            s.append(-math.inf if masked else scale * math.fsum(float(q[i, d]) * float(k[j, d]) for d in range(D)))
        denom = math.fsum(math.exp(x) for x in s)      # no max subtraction: tiny scores
        for d in range(D):
            O[i, d] = math.fsum(math.exp(s[j]) * float(v[j, d]) for j in range(Nk)) / denom
        L[i] = math.log(denom)
    return O, L


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("Nq,Nk,D", [(1, 1, 1), (3, 3, 2), (5, 8, 4), (8, 8, 3)])
def test_brute_force_tiny(Nq, Nk, D, causal):
    Q, K, V = _qkv(1, 1, Nq, Nk, D, 30 + Nq)
    scale = np.float32(0.37)
    O, L = oracle.mha_fwd(Q, K, V, causal=causal, scale=scale)
    Ob, Lb = _brute(f64(Q)[0, 0], f64(K)[0, 0], f64(V)[0, 0], float(scale), causal)
    np.testing.assert_allclose(O, Ob, atol=1e-13)
    np.testing.assert_allclose(L, Lb, atol=1e-13)


def test_numpy_softmax_third_opinion_and_row_subset():
    B, H, Nq, Nk, D = 2, 2, 19, 27, 16
    Q, K, V = _qkv(B, H, Nq, Nk, D, 40)
    scale = np.float32(0.25)
    q, k, v = f64(Q), f64(K), f64(V)
    S = float(scale) * np.einsum("bhid,bhjd->bhij", q, k)
    mask = np.arange(Nk)[None, :] > np.arange(Nq)[:, None] + (Nk - Nq)
    Sm = np.where(mask, -np.inf, S)
    P = np.exp(Sm - Sm.max(-1, keepdims=True)); P /= P.sum(-1, keepdims=True)
    want = np.einsum("bhij,bhjd->bhid", P, v).reshape(-1, D)
    O, L = oracle.mha_fwd(Q, K, V, causal=True, scale=scale)
    np.testing.assert_allclose(O, want, atol=1e-13)
    rows = [0, 75, 18, 19, 37]
    Or, Lr = oracle.mha_fwd(Q, K, V, causal=True, scale=scale, qrows=rows)
    assert np.array_equal(Or, O[rows]) and np.array_equal(Lr, L[rows])
    assert np.array_equal(oracle.mha_fwd(Q, K, V, causal=True, scale=scale, nthreads=1)[0], O)


def test_scale_is_taken_in_fp32():
    # 1/sqrt(128) is not an FP32 value: the oracle must use the rounded one, as the GPU entry point does
    Q, K, V = _qkv(1, 1, 4, 4, 128, 41)
    s64 = 1.0 / math.sqrt(128.0)
    _, L = oracle.mha_fwd(Q, K, V, causal=False, scale=s64)
    Ob, Lb = _brute(f64(Q)[0, 0], f64(K)[0, 0], f64(V)[0, 0], float(np.float32(s64)), False)
    np.testing.assert_allclose(L, Lb, atol=1e-13)


def test_rejects_causal_with_more_queries_than_keys():
    Q, K, V = _qkv(1, 1, 5, 3, 4, 42)
    with pytest.raises(ValueError):
        oracle.mha_fwd(Q, K, V, causal=True, scale=1.0)
