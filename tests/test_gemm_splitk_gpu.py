"""GPU parity of the K-cutting GEMM paths for the memory-bound shapes of Sec. 4.1 against the oracle: slices through
caller scratch (mlt_gemm_ex) and slices inside thread-block clusters (no scratch; mlt_gemm and mlt_gemm_ex)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
import paper_2503_14985_b200 as mlt  # noqa: E402
from paper_2503_14985_b200 import inputs  # noqa: E402

from gpu_util import assert_device_healthy, to_bits, to_dev  # noqa: E402
from parity import check_gemm  # noqa: E402

SENTINEL = 0x7FC1


def run_ex(A, B, M, N, K, ldc, workspace_bytes):
    Cbuf = torch.from_numpy(np.full((M + 2, ldc), SENTINEL, dtype=np.uint16).view(np.int16)).cuda().view(torch.bfloat16)
    # scratch prefilled with NaN patterns: a partial tile that is read without having been written shows in the result
    ws = torch.full((workspace_bytes + 64,), 0xFF, dtype=torch.uint8, device="cuda") if workspace_bytes else None
    dA, dB = to_dev(A), to_dev(B)
    rc = mlt.gemm_ex_raw(dA.data_ptr(), dB.data_ptr(), Cbuf.data_ptr(), M, N, K, A.shape[1], B.shape[1], ldc,
                         ws.data_ptr() if ws is not None else 0, workspace_bytes, torch.cuda.current_stream().cuda_stream)
    assert rc == 0, mlt.status_string(rc)
    assert_device_healthy()
    bits = to_bits(Cbuf)
    assert (bits[M:] == SENTINEL).all() and (bits[:M, N:] == SENTINEL).all(), "wrote outside C"
    assert not (bits[:M, :N] == SENTINEL).any(), "unwritten output elements"
    if ws is not None:
        assert (ws[workspace_bytes:].cpu().numpy() == 0xFF).all(), "workspace overrun"
    return inputs.bf16_bits_to_f64(bits[:M, :N]).reshape(M, N)


def plan(M, N, K, workspace_bytes=0):
    return mlt.gemm_plan(M, N, K, workspace_bytes, 0)          # the plan of the device the test runs on


# the last three have more than one 128 x 128 tile per two SMs: with scratch they take the two-kernel path
SHAPES = [(1, 4096, 4096), (16, 4096, 4096), (7, 1000, 2056), (64, 520, 8192), (130, 264, 4100), (16, 4096, 520),
          (512, 512, 512), (33, 6, 1024), (16, 9600, 2048), (40, 10008, 2064), (200, 5000, 4100)]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_parity_skinny_and_ragged(M, N, K):
    lda, ldb, ldc = (K + 7) // 8 * 8, (N + 7) // 8 * 8 + 8, (N + 7) // 8 * 8
    A, B = inputs.gemm_inputs(M, N, K, seed=500 + M + N, kind="uniform", lda=lda, ldb=ldb)
    need = mlt.gemm_workspace_bytes(M, N, K)
    C = run_ex(A, B, M, N, K, ldc, need)
    check_gemm(C, oracle.gemm(A, B, M, N, K), f"{M}x{N}x{K}")


@pytest.mark.parametrize("M,N,K", [(16, 1024, 4096), (16, 9600, 4096)])     # clusters / scratch
@pytest.mark.parametrize("fraction", [0.0, 0.13, 0.26, 1.0])   # 0.13: room for two uniform slices only
def test_any_workspace_size_is_correct(fraction, M, N, K):
    A, B = inputs.gemm_inputs(M, N, K, seed=510)
    need = mlt.gemm_workspace_bytes(M, N, K)
    assert need == 16 * M * N * 4           # 64 blocks of 64 -> at most 16 slices of 4
    given = int(need * fraction) // 16 * 16
    if N == 9600:
        assert plan(M, N, K, need)["split_k"] > 1 and plan(M, N, K, need)["split_k"] * M * N * 4 <= need
        assert plan(M, N, K, given)["split_k"] * M * N * 4 <= max(given, M * N * 4)
    C = run_ex(A, B, M, N, K, N, given)
    check_gemm(C, oracle.gemm(A, B, M, N, K), f"fraction {fraction}")


@pytest.mark.parametrize("M,N,K", [(24, 776, 2048), (24, 9736, 2048)])       # clusters / many tiles
def test_bit_exact_on_small_integers_and_deterministic(M, N, K):
    A, B = inputs.gemm_inputs(M, N, K, seed=7, kind="ternary")
    need = mlt.gemm_workspace_bytes(M, N, K)
    pl = plan(M, N, K, need)
    if N == 776:
        assert pl["cluster"] > 1
    C1 = run_ex(A, B, M, N, K, N, need)
    ref = oracle.gemm(A, B, M, N, K)
    assert np.abs(ref).max() <= 256 and np.array_equal(C1, ref)      # exact partial sums, exact final sum
    assert np.array_equal(C1, run_ex(A, B, M, N, K, N, need))


# Clusters of 2, 4 and 8 CTAs per tile (on 148 SMs), ragged M, N and K, one and two tile rows, a last slice shorter
# than the others, a K tail that is not a whole block; no scratch is given
CLUSTER_SHAPES = [(16, 8192, 4096, 2), (48, 8000, 4104, 2), (16, 4096, 4096, 4), (5, 2056, 3000, 8),
                  (16, 1024, 4096, 8), (130, 264, 4100, 8), (256, 520, 2048 + 24, 4), (1, 128, 4096, 8),
                  (128, 136, 36 * 64, 8)]


@pytest.mark.parametrize("M,N,K,S148", CLUSTER_SHAPES)
def test_cluster_split_parity(M, N, K, S148):
    pl = plan(M, N, K)
    assert pl["cluster"] > 1 and pl["split_k"] == 1
    print(f"{M}x{N}x{K}: {pl}")
    assert pl == mlt.gemm_plan(M, N, K, 0, 148) or pl["cluster"] < S148   # fewer resident clusters than SMs / S allow
    lda, ldb, ldc = (K + 7) // 8 * 8, (N + 7) // 8 * 8 + 8, (N + 7) // 8 * 8 + 16
    A, B = inputs.gemm_inputs(M, N, K, seed=900 + M + N, kind="uniform", lda=lda, ldb=ldb)
    C = run_ex(A, B, M, N, K, ldc, 0)
    ref = oracle.gemm(A, B, M, N, K)
    check_gemm(C, ref, f"cluster {M}x{N}x{K}")
    assert np.array_equal(C, run_ex(A, B, M, N, K, ldc, 0))          # fixed summation order
    # the public entry point without scratch takes the same path and gives the same bits
    dA, dB = to_dev(A), to_dev(B)
    out = torch.empty((M, ldc), dtype=torch.bfloat16, device="cuda")
    rc = mlt.gemm_raw(dA.data_ptr(), dB.data_ptr(), out.data_ptr(), M, N, K, lda, ldb, ldc,
                      torch.cuda.current_stream().cuda_stream)
    assert rc == 0
    assert np.array_equal(inputs.bf16_bits_to_f64(to_bits(out)[:, :N]).reshape(M, N), C)


@pytest.mark.parametrize("name", list(inputs.GEMM_DECODE_CONFIGS))
def test_decode_configs(name):
    M, N, K, kind, seed = inputs.GEMM_DECODE_CONFIGS[name]
    A, B = inputs.gemm_inputs(M, N, K, seed=seed, kind=kind)
    C = run_ex(A, B, M, N, K, N, mlt.gemm_workspace_bytes(M, N, K))
    rows = np.unique(np.linspace(0, M - 1, 8).astype(np.int64))
    rel, mx = check_gemm(C[rows], oracle.gemm(A, B, M, N, K, rows=rows), name)
    print(f"{name}: rel_fro={rel:.3e} max_abs/rms={mx:.3e}")


def test_argument_errors():
    x = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    p = x.data_ptr()
    assert mlt.gemm_ex_raw(p, p, p, 8, 8, 8, 8, 8, 8, p + 4, 1024) == 3       # misaligned workspace
    assert mlt.gemm_workspace_bytes(8192, 8192, 8192) == 0                     # plenty of tiles: no split
    assert mlt.gemm_workspace_bytes(16, 4096, 256) == 0                        # K too short to cut


# 129 to 640 rows: 128 x 256 tiles with K cut inside clusters (two tile rows and more, ragged edges, a short last slice)
WIDE_CLUSTER_SHAPES = [(384, 4096, 14336), (160, 4104, 28672 + 40), (256, 8192, 8192), (300, 2056, 16000), (640, 1000, 12000 + 8)]


@pytest.mark.parametrize("M,N,K", WIDE_CLUSTER_SHAPES)
def test_wide_tiles_in_clusters(M, N, K):
    pl = plan(M, N, K)
    print(f"{M}x{N}x{K}: {pl}")
    if mlt.gemm_plan(M, N, K, 0, 148)["variant"] == 1:   # what a device of 148 SMs with every SM usable would do
        assert mlt.gemm_plan(M, N, K, 0, 148)["cluster"] > 1
    lda, ldb, ldc = (K + 7) // 8 * 8, (N + 7) // 8 * 8 + 8, (N + 7) // 8 * 8 + 8
    A, B = inputs.gemm_inputs(M, N, K, seed=950 + M, kind="uniform", lda=lda, ldb=ldb)
    C = run_ex(A, B, M, N, K, ldc, 0)
    rows = np.unique(np.concatenate([np.arange(0, M, 37), [0, 127, 128, M - 1]])).astype(np.int64)
    check_gemm(C[rows], oracle.gemm(A, B, M, N, K, rows=rows), f"wide cluster {M}x{N}x{K}")
    assert np.array_equal(C, run_ex(A, B, M, N, K, ldc, 0))          # fixed summation order

