"""Pins for the paged-attention decode oracle (Sec. 3.2 / 4.3: one query token per sequence, keys and values
reached through a block table).  Each fixes the result by reduction to the already pinned dense attention oracle,
by an invariance, by a closed form, or by an independent brute force."""
import math

import numpy as np
import pytest

import oracle
from paper_2503_14985_b200 import inputs

f64 = inputs.bf16_bits_to_f64


def gather(cache, table, lens, s, kvh, bs):
    rows = [cache[table[s, i // bs], kvh, i % bs] for i in range(int(lens[s]))]
    return np.stack(rows) if rows else np.zeros((0, cache.shape[-1]), np.uint16)


def test_reduces_to_dense_attention_with_one_query_row():
    S, H, Hkv, D, bs = 5, 4, 2, 16, 4
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, Hkv, D, bs, seed=51, min_len=1, max_len=23)
    O, L = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=0.3)
    for s in range(S):
        for h in range(H):
            k = gather(Kc, table, lens, s, h // (H // Hkv), bs)[None, None]
            v = gather(Vc, table, lens, s, h // (H // Hkv), bs)[None, None]
            o_ref, l_ref = oracle.mha_fwd(Q[s, h][None, None, None], k, v, causal=False, scale=0.3)
            np.testing.assert_allclose(O[s, h], o_ref[0], atol=1e-14)
            np.testing.assert_allclose(L[s, h], l_ref[0], atol=1e-14)


def test_physical_block_placement_does_not_matter():
    S, H, D, bs = 3, 2, 8, 4
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, H, D, bs, seed=52, min_len=5, max_len=19)
    O1, L1 = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=0.5)
    perm = np.random.default_rng(3).permutation(Kc.shape[0])          # new home of every physical block
    Kc2 = np.empty_like(Kc); Vc2 = np.empty_like(Vc)
    Kc2[perm] = Kc; Vc2[perm] = Vc
    table2 = np.where(table >= 0, perm[np.maximum(table, 0)], -1).astype(np.int32)
    O2, L2 = oracle.paged_attn_decode(Q, Kc2, Vc2, table2, lens, scale=0.5)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)


def test_length_one_returns_the_single_value_and_tokens_beyond_len_are_ignored():
    S, H, D, bs = 2, 3, 8, 4
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, H, D, bs, seed=53, min_len=6, max_len=6)
    lens1 = np.ones_like(lens)
    O, L = oracle.paged_attn_decode(Q, Kc, Vc, table, lens1, scale=0.7)
    for s in range(S):
        for h in range(H):
            assert np.array_equal(O[s, h], f64(Vc[table[s, 0], h, 0]))
            np.testing.assert_allclose(L[s, h], float(np.float32(0.7)) * (f64(Q[s, h]) @ f64(Kc[table[s, 0], h, 0])),
                                       atol=1e-13)
    # poisoning everything past the length (rest of the last block, unused blocks) changes nothing
    O6, L6 = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=0.7)
    Kp, Vp = Kc.copy(), Vc.copy()
    for s in range(S):
        Kp[table[s, 1], :, 2:] = 0x7FC0; Vp[table[s, 1], :, 2:] = 0x7FC0      # tokens 6, 7 of block 1
    O6p, L6p = oracle.paged_attn_decode(Q, Kp, Vp, table, lens, scale=0.7)
    assert np.array_equal(O6, O6p) and np.array_equal(L6, L6p)


def test_constant_keys_give_mean_value_and_log_count():
    S, H, D, bs = 2, 2, 8, 4
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, H, D, bs, seed=54, min_len=9, max_len=14)
    Kc[:] = Kc[0, 0, 0]
    O, L = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=0.25)
    for s in range(S):
        for h in range(H):
            v = f64(gather(Vc, table, lens, s, h, bs))
            np.testing.assert_allclose(O[s, h], v.mean(axis=0), atol=1e-13)
            np.testing.assert_allclose(L[s, h], 0.25 * (f64(Q[s, h]) @ f64(Kc[0, 0, 0])) + math.log(lens[s]), atol=1e-12)


def test_brute_force_and_grouped_heads():
    S, H, Hkv, D, bs = 2, 4, 2, 4, 2
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, Hkv, D, bs, seed=55, min_len=3, max_len=7)
    scale = float(np.float32(0.37))
    O, L = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=scale)
    for s in range(S):
        for h in range(H):
            kvh = h // 2
            w = []
            for i in range(int(lens[s])):
                k = f64(Kc[table[s, i // bs], kvh, i % bs])
                w.append(math.exp(scale * math.fsum(float(a) * float(b) for a, b in zip(f64(Q[s, h]), k))))
            den = math.fsum(w)
            for d in range(D):
                num = math.fsum(w[i] * float(f64(Vc[table[s, i // bs], kvh, i % bs])[d]) for i in range(int(lens[s])))
                assert abs(O[s, h, d] - num / den) < 1e-13
            assert abs(L[s, h] - math.log(den)) < 1e-13


def test_empty_sequence_and_bad_table():
    S, H, D, bs = 2, 1, 4, 2
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, H, D, bs, seed=56, min_len=3, max_len=5)
    lens0 = lens.copy(); lens0[1] = 0
    O, L = oracle.paged_attn_decode(Q, Kc, Vc, table, lens0, scale=1.0)
    assert np.array_equal(O[1], np.zeros((H, D))) and np.isneginf(L[1]).all()
    bad = table.copy(); bad[0, 0] = Kc.shape[0]
    with pytest.raises(ValueError):
        oracle.paged_attn_decode(Q, Kc, Vc, bad, lens, scale=1.0)


def test_generator_mixes_lengths_and_scatters_blocks():
    name = "paged_s16h8d128_len1k-8k"
    S, H, Hkv, D, bs, lo, hi, seed = inputs.PAGED_CONFIGS[name]
    u = inputs.hash_u01(seed, inputs.TENSOR_PAGED_Q, 9, np.arange(S, dtype=np.uint64))
    lens = lo + np.floor(u * (hi - lo + 1))
    assert lens.min() >= lo and lens.max() <= hi and lens.std() > 1000 and S >= 8
    _, _, _, table, l2 = inputs.paged_inputs(4, 2, 2, 8, 4, seed=seed, min_len=10, max_len=40)
    used = table[table >= 0]
    assert len(np.unique(used)) == len(used)                       # every physical block used once
    assert not np.array_equal(np.sort(table[0][table[0] >= 0]), table[0][table[0] >= 0])   # scattered, not ascending
