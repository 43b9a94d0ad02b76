"""GPU parity of mlt_gemm_f16 (FP16 operands, FP32 result, optional C += A*B) against the FP64 oracle.

Tolerances.  The result is not rounded to 16 bits, so the only error is the FP32 accumulation over K.  With unit
roundoff u = 2^-23 (the tensor core may truncate rather than round), K / 16 dependent additions per element and
partial sums no larger than a few times the final RMS, a systematic drift is bounded by about (K / 16) * u * rms
= 2e-4 * rms at K = 28672 and the typical error is the square root of that count times u.  The tests take
rel_fro <= 1e-4 and max_abs / rms <= 1e-3, fifty times tighter than the BF16-output bounds.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
import paper_2503_14985_b200 as mlt  # noqa: E402
from paper_2503_14985_b200 import inputs  # noqa: E402

from gpu_util import assert_device_healthy  # noqa: E402
from parity import errors  # noqa: E402

REL_FRO_F32 = 1e-4
MAX_ABS_F32 = 1e-3
SENTINEL = np.uint32(0x7FC00123)  # a NaN pattern: unwritten or over-written elements are detected exactly


def dev16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()


def check(c, ref, what):
    rms = float(np.sqrt(np.mean(ref ** 2))) if ref.size else 1.0
    rel, mx = errors(c, ref, unit=rms if rms > 0 else 1.0)
    assert rel <= REL_FRO_F32, f"{what}: rel_fro {rel:.3e}"
    assert mx <= MAX_ABS_F32, f"{what}: max_abs/rms {mx:.3e}"
    return rel, mx


def run(A, B, M, N, K, ldc, C0=None, guard_rows=3):
    """Runs mlt_gemm_f16; C0 (M x ldc float32) switches the accumulate form on.  Returns C (M, N) float64."""
    buf = np.full((M + guard_rows, max(ldc, 4)), SENTINEL, dtype=np.uint32)
    if C0 is not None:
        buf[:M, :N] = np.ascontiguousarray(C0[:, :N]).view(np.uint32)
    d = torch.from_numpy(buf.view(np.int32)).cuda()
    dA, dB = dev16(A), dev16(B)
    rc = mlt.gemm_f16_raw(dA.data_ptr() if A.size else 0, dB.data_ptr() if B.size else 0, d.data_ptr(), M, N, K,
                          A.shape[1] if A.ndim == 2 and A.shape[1] else max(K, 8),
                          B.shape[1] if B.ndim == 2 and B.shape[1] else max(N, 8), max(ldc, 4),
                          0 if C0 is None else 1, torch.cuda.current_stream().cuda_stream)
    assert rc == 0, mlt.status_string(rc)
    assert_device_healthy()
    out = d.cpu().numpy().view(np.uint32)
    assert (out[M:] == SENTINEL).all(), "rows beyond M were written"
    assert (out[:M, N:] == SENTINEL).all(), "padding columns were written"
    assert not (out[:M, :N] == SENTINEL).any(), "unwritten output elements"
    return out[:M, :N].view(np.float32).astype(np.float64)


def ld8(width, extra):
    return (width + 7) // 8 * 8 + extra


def ld4(width, extra):
    return (width + 3) // 4 * 4 + extra


SHAPES = [(128, 256, 64), (1, 4, 8), (8, 8, 16), (129, 257, 72), (300, 518, 1000), (512, 512, 512),
          (130, 2500, 200), (2100, 2300, 520), (1281, 6150, 72)]


@pytest.mark.parametrize("accumulate", [False, True])
@pytest.mark.parametrize("extra", [0, 12])
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_parity_small_and_ragged(M, N, K, extra, accumulate):
    ldc = ld4(N, extra)
    A, B, C0 = inputs.gemm_f16_inputs(M, N, K, seed=300 + M + N + K, kind="uniform", lda=ld8(K, 8 if extra else 0),
                                      ldb=ld8(N, 8 if extra else 0), ldc=ldc)
    C = run(A, B, M, N, K, ldc, C0 if accumulate else None)
    ref = oracle.gemm_f16(A, B, M, N, K, C_in=C0 if accumulate else None)
    check(C, ref, f"{M}x{N}x{K}+{extra} acc={accumulate}")


@pytest.mark.parametrize("M,N,K", [(256, 512, 256), (129, 257, 200), (2176, 2312, 200)])
def test_bit_exact_on_small_integers(M, N, K):
    # entries in {-1,0,1}, prior C a small integer: every partial sum is an exact FP32 integer
    A16, B16 = inputs.gemm_inputs(M, N, K, seed=7, kind="ternary")
    v = inputs.bf16_bits_to_f64
    A, B = inputs.f64_to_f16_bits(v(A16)), inputs.f64_to_f16_bits(v(B16))
    A = np.pad(A, ((0, 0), (0, ld8(K, 0) - K))); B = np.pad(B, ((0, 0), (0, ld8(N, 0) - N)))
    C0 = np.round(4 * inputs.gemm_f16_inputs(M, N, 0, seed=8, ldc=ld4(N, 4))[2]).astype(np.float32)
    assert np.array_equal(run(A, B, M, N, K, ld4(N, 4)), oracle.gemm_f16(A, B, M, N, K))
    assert np.array_equal(run(A, B, M, N, K, ld4(N, 4), C0), oracle.gemm_f16(A, B, M, N, K, C_in=C0))


def test_fp16_bits_are_not_read_as_bf16():
    # 0x3C00 is 1.0 in binary16 and 2^-7 in BF16
    K = 64
    A = np.full((128, K), 0x3C00, np.uint16); B = np.full((K, 128), 0x3C00, np.uint16)
    assert np.array_equal(run(A, B, 128, 128, K, 128), np.full((128, 128), float(K)))


def test_result_keeps_fp32_precision():
    # 1 + 2^-10 squared summed 8 times = 8 + 2^-6 + 2^-17: needs 21 significant bits (BF16 or FP16 output would lose it)
    A = np.zeros((128, 8), np.uint16); B = np.zeros((8, 128), np.uint16)
    A[:] = 0x3C01; B[:] = 0x3C01
    want = 8 * (1 + 2.0 ** -10) ** 2
    assert np.array_equal(run(A, B, 128, 128, 8, 128), np.full((128, 128), want))


def test_k_zero_and_empty():
    A = np.zeros((16, 8), np.uint16); B = np.zeros((0, 24), np.uint16)
    _, _, C0 = inputs.gemm_f16_inputs(16, 24, 0, seed=5, ldc=32)
    assert np.array_equal(run(A, B, 16, 24, 0, 32), np.zeros((16, 24)))
    assert np.array_equal(run(A, B, 16, 24, 0, 32, C0), C0[:, :24].astype(np.float64))       # C += 0
    assert mlt.gemm_f16_raw(0, 0, 0, 0, 5, 5, 8, 8, 8, 0) == 0


def test_accumulating_twice_adds_twice():
    M, N, K = 384, 520, 264
    A, B, C0 = inputs.gemm_f16_inputs(M, N, K, seed=31, ldc=N)
    dA, dB = dev16(A), dev16(B)
    dC = torch.from_numpy(C0.copy()).cuda()
    for _ in range(2):
        assert mlt.gemm_f16_raw(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, K, N, N, 1) == 0
    assert_device_healthy()
    ref = 2 * oracle.gemm_f16(A, B, M, N, K) + C0.astype(np.float64)
    check(dC.cpu().numpy().astype(np.float64), ref, "two accumulations")


@pytest.mark.parametrize("name", ["gemm_4096", "gemm_8192x28672x4096", "gemm_8192x4096x28672"])
@pytest.mark.parametrize("accumulate", [False, True])
def test_benchmark_shapes_sampled_rows(name, accumulate):
    M, N, K, kind, seed = inputs.GEMM_CONFIGS[name]
    A, B, C0 = inputs.gemm_f16_inputs(M, N, K, seed=seed, kind=kind)
    dA, dB = dev16(A), dev16(B)
    dC = torch.from_numpy(C0).cuda() if accumulate else torch.full((M, N), float("nan"), device="cuda")
    rc = mlt.gemm_f16_raw(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, K, N, N, int(accumulate))
    assert rc == 0
    assert_device_healthy()
    assert torch.isfinite(dC).all()
    rng = np.random.default_rng(M + N)
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, M - 1], rng.integers(0, M, 40)])).astype(np.int64)
    ref = oracle.gemm_f16(A, B, M, N, K, C_in=C0 if accumulate else None, rows=rows)
    got = dC[torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.float64)
    rel, mx = check(got, ref, name)
    print(f"{name} acc={accumulate}: rel_fro={rel:.3e} max_abs/rms={mx:.3e}")


def test_argument_errors_do_not_launch():
    x = torch.zeros(64, 64, dtype=torch.float32, device="cuda")
    p = x.data_ptr()
    assert mlt.gemm_f16_raw(p, p, p + 4, 8, 8, 8, 64, 64, 64, 0) == 3      # C not 16-byte aligned
    assert mlt.gemm_f16_raw(p, p, p, 8, 8, 8, 64, 64, 10, 0) == 3          # ldc not a multiple of 4
    assert mlt.gemm_f16_raw(p, p, p, 8, 8, 8, 64, 64, 4, 0) == 1           # ldc < N
    assert mlt.gemm_f16_raw(p, p, 0, 8, 8, 8, 64, 64, 64, 1) == 1          # NULL C
