"""Host logic of the GEMM launch plan (no GPU): which tile shape a problem gets and how K is cut for the memory-bound
shapes of Sec. 4.1.  The plan is plain integer arithmetic behind mlt_debug_gemm_plan."""
import itertools

import pytest

import paper_2503_14985_b200 as mlt


def kb(K):
    return (K + 63) // 64


@pytest.mark.parametrize("sm_count", [148, 132, 64, 2])
def test_plan_invariants(sm_count):
    Ms = [1, 16, 100, 130, 300, 511, 512, 640, 2000]
    Ns = [8, 128, 520, 4096, 9600, 28672]
    Ks = [8, 64, 520, 2048, 4100, 28672]
    for M, N, K in itertools.product(Ms, Ns, Ks):
        need = mlt.gemm_workspace_bytes(M, N, K)
        for ws in {0, need // 3 // 16 * 16, need}:
            pl = mlt.gemm_plan(M, N, K, ws, sm_count)
            what = f"{M}x{N}x{K} ws={ws} sms={sm_count}: {pl}"
            assert pl["variant"] in (0, 1, 2, 3), what
            if pl["variant"] == 3:   # even K hand-out: shares cover all units, the partial tiles fit the scratch
                tiles = ((M + 127) // 128) * ((N + 127) // 128)
                assert pl["cluster"] == 1 and M < 512 and ws > 0, what
                assert pl["kb_per_split"] * sm_count >= tiles * kb(K) > pl["kb_per_split"] * (sm_count - 1) - sm_count, what
                assert pl["split_k"] == -(-kb(K) // pl["kb_per_split"]) + 1 and pl["split_k"] * M * N * 4 <= ws, what
                continue
            assert pl["cluster"] in (1, 2, 4, 8) and pl["split_k"] >= 1, what
            assert pl["cluster"] == 1 or pl["split_k"] == 1, what
            slices = max(pl["cluster"], pl["split_k"])
            if slices == 1:
                assert pl["kb_per_split"] == kb(K), what
                continue
            assert pl["variant"] == 2 or (pl["variant"] == 1 and pl["cluster"] > 1 and 128 < M <= 640), what
            # every slice has work, the slices cover K, none is shorter than 4 blocks by design of the cut
            assert pl["kb_per_split"] * (slices - 1) < kb(K) <= pl["kb_per_split"] * slices, what
            assert kb(K) // slices >= 4, what
            if pl["split_k"] > 1:
                assert pl["split_k"] * M * N * 4 <= ws, what
            elif pl["variant"] == 2:
                tiles = ((M + 127) // 128) * ((N + 127) // 128)
                assert 2 * tiles <= sm_count, what


def test_plan_known_cases_on_148_sms():
    full = lambda M, N, K: mlt.gemm_plan(M, N, K, mlt.gemm_workspace_bytes(M, N, K), 148)
    assert mlt.gemm_plan(8192, 8192, 8192)["variant"] == 0 and full(8192, 28672, 4096)["variant"] == 0
    assert full(8192, 8192, 8192)["split_k"] == 1 and full(8192, 8192, 8192)["cluster"] == 1
    # next-token shapes: 32 tiles -> 4 CTAs per tile; 64 tiles -> 2; 8 tiles -> 8
    assert full(16, 4096, 4096)["cluster"] == 4 and mlt.gemm_plan(16, 4096, 4096)["cluster"] == 4
    assert full(16, 4096, 28672)["cluster"] == 4 and full(16, 4096, 28672)["kb_per_split"] == 112
    assert full(16, 8192, 4096)["cluster"] == 2
    assert full(16, 1024, 4096)["cluster"] == 8
    # 224 tiles: clusters would need more than one round; with scratch K goes through the workspace, without it whole
    # one tile row, many tiles: the time model.  112 tiles of 128 x 256 in one round keep HBM busy without any cut ...
    assert full(16, 28672, 4096) == mlt.gemm_plan(16, 28672, 4096) == {"variant": 1, "split_k": 1, "cluster": 1, "kb_per_split": 64}
    # ... 160 of them would be a round and a bit: the even hand-out through scratch (320 x 64 units / 148), else small tiles
    assert full(16, 40960, 4096) == {"variant": 3, "split_k": 2, "cluster": 1, "kb_per_split": 139}
    assert mlt.gemm_plan(16, 40960, 4096)["variant"] == 2
    # a short K is not cut
    assert full(16, 4096, 192)["cluster"] == 1 and full(16, 4096, 192)["split_k"] == 1
    assert full(512, 512, 512)["cluster"] == 1
    # 129 to 640 rows: 128 x 256 tiles with K cut in clusters when that moves clearly fewer bytes per SM
    assert mlt.gemm_plan(256, 8192, 8192) == {"variant": 1, "split_k": 1, "cluster": 2, "kb_per_split": 64}
    assert mlt.gemm_plan(128, 8192, 8192)["variant"] == 2


def test_plan_rejects_bad_arguments():
    with pytest.raises(mlt.MltError):
        mlt.gemm_plan(0, 8, 8)
    with pytest.raises(mlt.MltError):
        mlt.gemm_plan(8, 8, 8, 0, 1)


def test_even_hand_out_slots_fit_the_plan():
    """Even K hand-out (plan variant 3): CTA c takes units [c U, (c + 1) U) of all tiles x K blocks in tile order and
    writes, per tile it touches, partial slot c - (first CTA of the tile).  The plan's split_k is the number of partial
    tiles the scratch must hold per output tile: no slot may reach it, and the reduce kernel's count formula must be
    the number of CTAs that really touch the tile."""
    seen = 0
    for sm_count in (148, 132, 64):
        for M, N, K in [(16, 40960, 4096), (16, 9600, 4096), (200, 5000, 4100), (1, 9600, 4100), (100, 20000, 1700),
                        (300, 12000, 3000), (511, 9000, 2500), (64, 30000, 8192)]:
            pl = mlt.gemm_plan(M, N, K, mlt.gemm_workspace_bytes(M, N, K), sm_count)
            if pl["variant"] != 3:
                continue
            seen += 1
            U, nkb = pl["kb_per_split"], kb(K)
            tiles = ((M + 127) // 128) * ((N + 127) // 128)
            total = tiles * nkb
            ctas = -(-total // U)
            assert ctas <= sm_count
            touched = {}
            for c in range(ctas):
                for t in range(c * U // nkb, (min(total, (c + 1) * U) - 1) // nkb + 1):
                    touched.setdefault(t, []).append(c)
            assert sorted(touched) == list(range(tiles))
            for t, cs in touched.items():
                assert cs == list(range(cs[0], cs[-1] + 1)) and cs[0] == t * nkb // U      # slot = c - cs[0]
                assert len(cs) == ((t + 1) * nkb - 1) // U - t * nkb // U + 1               # the reduce kernel's count
                assert len(cs) <= pl["split_k"], (M, N, K, sm_count, pl, t, cs)
    assert seen >= 6
