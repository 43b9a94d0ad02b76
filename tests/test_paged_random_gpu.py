"""GPU parity of mlt_paged_attn_decode (Sec. 3.2 / 4.3) on seeded random shapes: every group size (1, 2, 4, 8 query
heads per KV head), head size and block size, length mixes from empty-ish to several thousand tokens, with the full
workspace, a part of it, or none; cache positions no sequence may read are poisoned."""
import math

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
import paper_2503_14985_b200 as mlt  # noqa: E402
from paper_2503_14985_b200 import inputs  # noqa: E402

from parity import check_mha  # noqa: E402
from test_paged_gpu import poison_unused, run_paged  # noqa: E402


def random_cases(count, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for _ in range(count):
        group = int(rng.choice([1, 2, 4, 8]))
        Hkv = int(rng.choice([1, 2, 4]))
        D = int(rng.choice([64, 128]))
        bs = int(rng.choice([8, 16, 32]))
        S = int(rng.integers(1, 12))
        hi = int(rng.choice([40, 300, 1500, 5000]))
        lo = int(rng.integers(1, hi + 1))
        cases.append((S, Hkv * group, Hkv, D, bs, lo, hi, int(rng.integers(0, 3))))
    return cases


@pytest.mark.parametrize("S,H,Hkv,D,bs,lo,hi,ws_kind", random_cases(36, seed=20250316))
def test_random_cases(S, H, Hkv, D, bs, lo, hi, ws_kind):
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, Hkv, D, bs, seed=S * 31 + H + hi + bs, min_len=lo, max_len=hi)
    Kc, Vc = poison_unused(Kc, Vc, table, lens, bs)
    scale = np.float32(1 / math.sqrt(D))
    full = mlt.paged_attn_workspace_bytes(S, H, D)
    ws = [None, 0, full // 3 // 16 * 16][ws_kind]
    o, lse = run_paged(Q, Kc, Vc, table, lens, scale, workspace_bytes=ws)
    o_ref, l_ref = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=scale)
    check_mha(o, lse, o_ref.reshape(-1, D), l_ref.reshape(-1), f"{(S, H, Hkv, D, bs, lo, hi, ws_kind)}")
