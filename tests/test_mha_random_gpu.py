"""GPU parity of mlt_mha_fwd (Sec. 2.5, Algorithm 1) on seeded random shapes: ragged query and key counts, both head
sizes, causal (bottom-right aligned) and not, one to several hundred work items."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
from paper_2503_14985_b200 import inputs  # noqa: E402

from parity import check_mha  # noqa: E402
from test_mha_gpu import run_mha, scale_for  # noqa: E402


def random_cases(count, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for _ in range(count):
        D = int(rng.choice([64, 128]))
        B, H = int(rng.integers(1, 4)), int(rng.integers(1, 60))
        Nq = int(rng.integers(1, 700))
        causal = int(rng.integers(0, 2))
        Nk = int(rng.integers(Nq, Nq + 400)) if causal else int(rng.integers(1, 900))  # causal: at least one visible key per row
        cases.append((B, H, Nq, Nk, D, causal))
    return cases


@pytest.mark.parametrize("B,H,Nq,Nk,D,causal", random_cases(32, seed=20250315))
def test_random_cases(B, H, Nq, Nk, D, causal):
    Q, K, V = inputs.mha_inputs(B, H, Nq, Nk, D, seed=B * 1000 + H * 17 + Nq + Nk)
    o, lse = run_mha(Q, K, V, causal, scale_for(D))
    o_ref, lse_ref = oracle.mha_fwd(Q, K, V, causal=bool(causal), scale=scale_for(D))
    check_mha(o, lse, o_ref, lse_ref, f"{(B, H, Nq, Nk, D, causal)}")
