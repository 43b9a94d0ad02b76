"""GPU parity of mlt_gemm / mlt_gemm_ex on seeded random shapes: whatever path the launch plan picks for a shape
(tile variant, K slices through scratch, K cut inside clusters), the result must match the oracle (Sec. 2 problem
statement, Listing 2) and nothing outside C may be written."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
import paper_2503_14985_b200 as mlt  # noqa: E402
from paper_2503_14985_b200 import inputs  # noqa: E402

from parity import check_gemm  # noqa: E402
from test_gemm_splitk_gpu import run_ex  # noqa: E402


def random_shapes(count, seed):
    rng = np.random.default_rng(seed)
    shapes = []
    for _ in range(count):
        kind = rng.integers(0, 4)
        if kind == 0:    # skinny: next-token shapes
            M, N, K = int(rng.integers(1, 130)), int(rng.integers(1, 40)) * 128 + int(rng.integers(0, 128)), int(rng.integers(4, 80)) * 64 + int(rng.integers(0, 64))
        elif kind == 1:  # few tiles, long K
            M, N, K = int(rng.integers(100, 600)), int(rng.integers(8, 1200)), int(rng.integers(500, 6000))
        elif kind == 2:  # many tiles, short K
            M, N, K = int(rng.integers(300, 1500)), int(rng.integers(500, 3000)), int(rng.integers(1, 600))
        else:            # anything small
            M, N, K = int(rng.integers(1, 300)), int(rng.integers(1, 300)), int(rng.integers(1, 300))
        shapes.append((M, N, K, bool(rng.integers(0, 2)), int(rng.integers(0, 3))))
    return shapes


@pytest.mark.parametrize("M,N,K,scratch,pad", random_shapes(48, seed=20250314))
def test_random_shapes(M, N, K, scratch, pad):
    lda = (K + 7) // 8 * 8 + 8 * pad
    ldb = (N + 7) // 8 * 8 + 8 * pad
    ldc = (N + 7) // 8 * 8 + 8 * (2 - pad)
    A, B = inputs.gemm_inputs(M, N, K, seed=M * 7 + N * 3 + K, kind="uniform", lda=lda, ldb=ldb)
    ws = mlt.gemm_workspace_bytes(M, N, K) if scratch else 0
    C = run_ex(A, B, M, N, K, ldc, ws)
    check_gemm(C, oracle.gemm(A, B, M, N, K), f"{M}x{N}x{K} scratch={scratch} plan={mlt.gemm_plan(M, N, K, ws, 0)}")
