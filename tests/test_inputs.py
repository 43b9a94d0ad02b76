"""The seeded generators: determinism, BF16 rounding, distribution sanity."""
import numpy as np

from paper_2503_14985_b200 import inputs


def test_bf16_round_trip_and_rne():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0, 3.0e38, 1e-40], dtype=np.float32)
    bits = inputs.f32_to_bf16_bits(x)
    back = inputs.bf16_bits_to_f64(bits)
    # ties go to even mantissa: 1 + 2^-8 -> 1.0 ; 1 + 3*2^-8 -> 1 + 2^-6
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == 1.0 + 2.0 ** -6
    assert back[3] == -2.5 and back[4] == 0.0
    # every BF16 value survives bits -> f64 -> bits
    allbits = np.arange(0, 0x7F80, dtype=np.uint16)
    assert np.array_equal(inputs.f64_to_bf16_bits(inputs.bf16_bits_to_f64(allbits)), allbits)


def test_elements_do_not_depend_on_padding_or_chunking():
    a = inputs.matrix_bf16(37, 53, seed=3, tensor_id=1, kind="normal", scale=0.5)
    b = inputs.matrix_bf16(37, 53, seed=3, tensor_id=1, kind="normal", scale=0.5, ld=64, chunk_rows=5)
    assert np.array_equal(a, b[:, :53])
    assert np.all(b[:, 53:] == 0x7FC0)
    c = inputs.matrix_bf16(37, 53, seed=4, tensor_id=1, kind="normal", scale=0.5)
    assert not np.array_equal(a, c)


def test_distributions():
    u = inputs.bf16_bits_to_f64(inputs.matrix_bf16(512, 512, seed=0, tensor_id=0, kind="uniform"))
    assert u.min() >= -1.0 and u.max() <= 1.0
    assert abs(u.mean()) < 5e-3 and abs(u.var() - 1.0 / 3.0) < 5e-3
    n = inputs.bf16_bits_to_f64(inputs.matrix_bf16(512, 512, seed=5, tensor_id=2, kind="normal"))
    assert abs(n.mean()) < 1e-2 and abs(n.std() - 1.0) < 1e-2
    assert abs(np.mean(n ** 4) - 3.0) < 0.1
    t = inputs.bf16_bits_to_f64(inputs.matrix_bf16(64, 64, seed=5, tensor_id=2, kind="ternary"))
    assert set(np.unique(t)) == {-1.0, 0.0, 1.0}


def test_outlier_rows_fraction_and_effect():
    mask = inputs.outlier_rows(6, inputs.TENSOR_Q, 16 * 16384, 1)
    assert 0.008 < mask.mean() < 0.012
    q0, k0, v0 = inputs.mha_inputs(1, 2, 256, 256, 64, seed=6)
    q1, k1, v1 = inputs.mha_inputs(1, 2, 256, 256, 64, seed=6, outlier_percent=10)
    assert np.array_equal(v0, v1)
    mq = inputs.outlier_rows(6, inputs.TENSOR_Q, 512, 10).reshape(1, 2, 256)
    f0, f1 = inputs.bf16_bits_to_f64(q0), inputs.bf16_bits_to_f64(q1)
    assert np.array_equal(f1[mq], 8.0 * f0[mq]) and np.array_equal(f1[~mq], f0[~mq])
    assert not np.array_equal(k0, k1)
