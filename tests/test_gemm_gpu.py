"""GPU parity of mlt_gemm (through the C ABI) against the FP64 oracle."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
import paper_2503_14985_b200 as mlt  # noqa: E402
from paper_2503_14985_b200 import inputs  # noqa: E402

from gpu_util import assert_device_healthy, to_bits, to_dev, to_f64  # noqa: E402
from parity import MAX_ABS_TOL, REL_FRO_TOL, RunningErrors, check_gemm, log_line  # noqa: E402

SENTINEL = 0x7FC1  # a NaN pattern: unwritten or over-written elements are detected exactly


def run_gemm(A, B, M, N, K, ldc=None, guard_rows=3):
    """Runs mlt_gemm on BF16 bit arrays; returns C (M, N) float64 and checks guard bands."""
    ldc = N if ldc is None else ldc
    Cbuf = torch.from_numpy(np.full((M + guard_rows, max(ldc, 1)), SENTINEL, dtype=np.uint16).view(np.int16)).cuda()
    Cbuf = Cbuf.view(torch.bfloat16)
    dA, dB = to_dev(A), to_dev(B)
    rc = mlt.gemm_raw(dA.data_ptr() if A.size else 0, dB.data_ptr() if B.size else 0, Cbuf.data_ptr(), M, N, K,
                      A.shape[1] if A.ndim == 2 and A.shape[1] else max(K, 8),
                      B.shape[1] if B.ndim == 2 and B.shape[1] else max(N, 8), ldc,
                      torch.cuda.current_stream().cuda_stream)
    assert rc == 0, mlt.status_string(rc)
    assert_device_healthy()
    bits = to_bits(Cbuf)
    assert (bits[M:] == SENTINEL).all(), "rows beyond M were written"
    assert (bits[:M, N:] == SENTINEL).all(), "padding columns were written"
    assert not (bits[:M, :N] == SENTINEL).any(), "unwritten output elements"
    return inputs.bf16_bits_to_f64(bits[:M, :N]).reshape(M, N)


def ld_for(width, extra):
    return (width + 7) // 8 * 8 + extra


# the last three are large enough for the CTA-pair (256 x 256) kernel, with ragged edges in M, N and K
SHAPES = [(128, 256, 64), (1, 8, 8), (8, 8, 16), (129, 257, 72), (300, 520, 1000), (512, 512, 512),
          (2048, 1024, 8), (130, 2500, 200), (4100, 300, 136), (2100, 2300, 520), (1281, 6152, 72), (19000, 264, 136)]


@pytest.mark.parametrize("extra", [0, 8, 64])
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_parity_small_and_ragged(M, N, K, extra):
    lda, ldb, ldc = ld_for(K, extra), ld_for(N, extra), ld_for(N, extra)
    A, B = inputs.gemm_inputs(M, N, K, seed=100 + M + N + K, kind="uniform", lda=lda, ldb=ldb)
    C = run_gemm(A, B, M, N, K, ldc=ldc)
    ref = oracle.gemm(A, B, M, N, K)
    check_gemm(C, ref, f"{M}x{N}x{K}+{extra}")


@pytest.mark.parametrize("M,N,K", [(256, 512, 256), (129, 257, 200), (384, 640, 1024), (2176, 2312, 200), (4096, 4096, 256)])
def test_bit_exact_on_small_integers(M, N, K):
    # entries in {-1,0,1}: every partial sum is an exact small integer; |c| <= 256 is BF16-representable
    A, B = inputs.gemm_inputs(M, N, K, seed=7, kind="ternary", lda=ld_for(K, 0), ldb=ld_for(N, 0))
    C = run_gemm(A, B, M, N, K, ldc=ld_for(N, 8))
    ref = oracle.gemm(A, B, M, N, K)
    assert np.abs(ref).max() <= 256
    assert np.array_equal(C, ref)


@pytest.mark.parametrize("K", [512, 4096])
def test_all_ones_is_exactly_K(K):
    A = np.full((128, K), 0x3F80, np.uint16); B = np.full((K, 256), 0x3F80, np.uint16)
    assert np.array_equal(run_gemm(A, B, 128, 256, K), np.full((128, 256), float(K)))


def test_single_nonzero_moves_one_row_of_B():
    M, N, K = 260, 264, 130
    _, B = inputs.gemm_inputs(M, N, K, seed=9, kind="uniform")
    for (i0, k0) in [(0, 0), (127, 63), (128, 64), (259, 129)]:
        A = np.zeros((M, 136), np.uint16); A[:, K:] = 0x7FC0
        A[i0, k0] = 0xC000  # -2.0
        C = run_gemm(A, B, M, N, K)
        want = np.zeros((M, N)); want[i0] = -2.0 * inputs.bf16_bits_to_f64(B)[k0]
        assert np.array_equal(C, want)


def test_k_zero_fills_zeros_and_empty_is_noop():
    A = np.zeros((16, 8), np.uint16); B = np.zeros((0, 24), np.uint16)
    C = run_gemm(A, B, 16, 24, 0, ldc=32)
    assert np.array_equal(C, np.zeros((16, 24)))
    assert mlt.gemm_raw(0, 0, 0, 0, 5, 5, 8, 8, 8) == 0


def test_deterministic_across_runs():
    M, N, K = 640, 768, 520
    A, B = inputs.gemm_inputs(M, N, K, seed=11, lda=ld_for(K, 0))
    dA, dB = to_dev(A), to_dev(B)
    C1 = mlt.gemm(dA, dB, M=M, N=N, K=K); C2 = mlt.gemm(dA, dB, M=M, N=N, K=K)
    torch.cuda.synchronize()
    assert torch.equal(C1.view(torch.int16), C2.view(torch.int16))


@pytest.mark.parametrize("name", list(inputs.GEMM_CONFIGS))
def test_benchmark_configs_every_element(name):
    # Every element of C against the FP64 oracle, in chunks of rows (the largest outputs would not fit twice in
    # float64), launched exactly as bench.py launches it; the figures go to the parity log.
    import time
    M, N, K, kind, seed = inputs.GEMM_CONFIGS[name]
    A, B = inputs.gemm_inputs(M, N, K, seed=seed, kind=kind)
    dA, dB = to_dev(A), to_dev(B)
    C = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    rc = mlt.gemm_raw(dA.data_ptr(), dB.data_ptr(), C.data_ptr(), M, N, K, K, N, N, torch.cuda.current_stream().cuda_stream)
    assert rc == 0, mlt.status_string(rc)
    assert_device_healthy()
    acc = RunningErrors()
    t0 = time.perf_counter()
    chunk = max(1, min(M, (1 << 25) // N))
    for r0 in range(0, M, chunk):
        rows = np.arange(r0, min(M, r0 + chunk), dtype=np.int64)
        acc.add(to_f64(C[r0:r0 + len(rows)]), oracle.gemm(A, B, M, N, K, rows=rows))
    secs = time.perf_counter() - t0
    rel, mx = acc.rel_fro(), acc.max_abs / acc.rms_ref()
    log_line(f"{name}: all {M}x{N} elements, rel_fro={rel:.3e} max_abs/rms={mx:.3e} "
             f"(limits {REL_FRO_TOL:.0e} / {MAX_ABS_TOL:.0e}); oracle {secs:.1f} s on {oracle.hardware_threads()} threads")
    assert rel <= REL_FRO_TOL, f"{name}: rel_fro {rel:.3e}"
    assert mx <= MAX_ABS_TOL, f"{name}: max_abs/rms {mx:.3e}"


def test_argument_errors_do_not_launch():
    x = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    p = x.data_ptr()
    assert mlt.gemm_raw(p, p, p + 2, 8, 8, 8, 64, 64, 64) == 3          # C not 16-byte aligned
    assert mlt.gemm_raw(p, p, p, 8, 8, 8, 257, 64, 64) == 3     # lda = 257: not a multiple of 8
    assert mlt.gemm_raw(p, p, p, 8, 8, 16, 8, 64, 64) == 1              # lda < K
    assert mlt.gemm_raw(0, p, p, 8, 8, 8, 64, 64, 64) == 1              # NULL A
    assert mlt.gemm_raw(p, p, p, -1, 8, 8, 64, 64, 64) == 1
