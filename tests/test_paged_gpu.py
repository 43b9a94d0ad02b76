"""GPU parity of mlt_paged_attn_decode (through the C ABI) against the FP64 oracle."""
import math

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
import paper_2503_14985_b200 as mlt  # noqa: E402
from paper_2503_14985_b200 import inputs  # noqa: E402

from gpu_util import assert_device_healthy, to_dev  # noqa: E402
from parity import check_mha  # noqa: E402

SENTINEL = 0x7FC1


def run_paged(Q, Kc, Vc, table, lens, scale, workspace_bytes=None, with_lse=True):
    """Runs the entry point on BF16 bit arrays with guard bands; returns (O [S*H, D] f64, LSE [S*H] f64)."""
    S, H, D = Q.shape
    NB, Hkv, bs, _ = Kc.shape
    guard = 256
    Obuf = torch.from_numpy(np.full((S * H * D + 2 * guard,), SENTINEL, np.uint16).view(np.int16)).cuda()
    Lbuf = torch.full((S * H + 2 * guard,), float("nan"), dtype=torch.float32, device="cuda")
    O = Obuf[guard:guard + S * H * D]
    L = Lbuf[guard:guard + S * H]
    if workspace_bytes is None:
        workspace_bytes = mlt.paged_attn_workspace_bytes(S, H, D)
    ws = torch.full((workspace_bytes + 64,), 0xFF, dtype=torch.uint8, device="cuda") if workspace_bytes else None  # NaN patterns: an unwritten partial that is read shows
    dQ, dK, dV = to_dev(Q), to_dev(Kc), to_dev(Vc)
    dT = torch.from_numpy(np.ascontiguousarray(table, dtype=np.int32)).cuda()
    dL = torch.from_numpy(np.ascontiguousarray(lens, dtype=np.int32)).cuda()
    rc = mlt.paged_attn_decode_raw(dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), dT.data_ptr(), dL.data_ptr(),
                                   O.data_ptr(), L.data_ptr() if with_lse else 0, S, H, Hkv, D, bs, table.shape[1], NB,
                                   float(np.float32(scale)), ws.data_ptr() if ws is not None else 0, workspace_bytes,
                                   torch.cuda.current_stream().cuda_stream)
    assert rc == 0, mlt.status_string(rc)
    assert_device_healthy()
    ob = Obuf.cpu().numpy().view(np.uint16)
    assert (ob[:guard] == SENTINEL).all() and (ob[-guard:] == SENTINEL).all(), "O guard band was written"
    lb = Lbuf.cpu().numpy()
    assert np.isnan(lb[:guard]).all() and np.isnan(lb[-guard:]).all(), "LSE guard band was written"
    if ws is not None:
        assert (ws[workspace_bytes:].cpu().numpy() == 0xFF).all(), "workspace overrun"
    body = ob[guard:-guard]
    assert not (body == SENTINEL).any(), "unwritten O elements"
    return inputs.bf16_bits_to_f64(body).reshape(S * H, D), (lb[guard:-guard].astype(np.float64) if with_lse else None)


def poison_unused(Kc, Vc, table, lens, bs):
    """NaN patterns in every cache position no sequence may read: tails of last blocks and unreferenced blocks."""
    used = np.zeros(Kc.shape[0], bool)
    Kp, Vp = Kc.copy(), Vc.copy()
    for s in range(table.shape[0]):
        n = (int(lens[s]) + bs - 1) // bs
        used[table[s, :n]] = True
        if n and lens[s] % bs:
            Kp[table[s, n - 1], :, lens[s] % bs:] = 0x7FC0
            Vp[table[s, n - 1], :, lens[s] % bs:] = 0x7FC0
    Kp[~used] = 0x7FC0
    Vp[~used] = 0x7FC0
    return Kp, Vp


CASES = [  # S, H, H_kv, D, block_size, min_len, max_len
    (3, 4, 4, 128, 16, 1, 100), (2, 8, 8, 64, 16, 17, 300), (5, 8, 2, 128, 16, 50, 700), (4, 8, 1, 64, 8, 1, 90),
    (2, 4, 2, 128, 32, 200, 1500), (1, 2, 2, 128, 16, 5000, 5000), (7, 16, 8, 64, 32, 1, 2000), (3, 2, 2, 64, 8, 1, 7),
    # 4 or 8 query heads per KV head (the tensor-core kernel), every block size and head dimension, lengths that end
    # inside a 16-token unit, and (8-token blocks) splits that must start at an even block
    (3, 16, 2, 128, 32, 100, 3000), (4, 8, 2, 64, 8, 1, 500), (2, 32, 4, 128, 8, 700, 2900), (5, 16, 4, 64, 16, 1, 1100),
    (2, 8, 1, 128, 16, 4000, 6000), (6, 4, 1, 64, 32, 1, 40),
]


@pytest.mark.parametrize("S,H,Hkv,D,bs,lo,hi", CASES)
def test_parity_with_length_mix_and_scattered_blocks(S, H, Hkv, D, bs, lo, hi):
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, Hkv, D, bs, seed=300 + S + H + hi, min_len=lo, max_len=hi)
    Kc, Vc = poison_unused(Kc, Vc, table, lens, bs)
    scale = np.float32(1 / math.sqrt(D))
    o, lse = run_paged(Q, Kc, Vc, table, lens, scale)
    o_ref, l_ref = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=scale)
    rel, mx, dl = check_mha(o, lse, o_ref.reshape(-1, D), l_ref.reshape(-1), f"{(S, H, Hkv, D, bs, lo, hi)}")
    print(f"rel_fro={rel:.3e} max_abs={mx:.3e} lse={dl:.3e}")


@pytest.mark.parametrize("workspace_bytes", [0, 4096, None])
def test_any_workspace_size_gives_the_same_answer(workspace_bytes):
    S, H, Hkv, D, bs = 2, 4, 4, 128, 16
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, Hkv, D, bs, seed=310, min_len=900, max_len=1200)
    scale = np.float32(1 / math.sqrt(D))
    o, lse = run_paged(Q, Kc, Vc, table, lens, scale, workspace_bytes=workspace_bytes)
    o_ref, l_ref = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=scale)
    check_mha(o, lse, o_ref.reshape(-1, D), l_ref.reshape(-1), f"workspace {workspace_bytes}")


@pytest.mark.parametrize("workspace_bytes", [0, 20000, None])
def test_grouped_heads_any_workspace_size(workspace_bytes):
    # 8 query heads per KV head: with the full workspace the CTAs get equal shares of the live tokens, with less the
    # sequences are cut into as many fixed pieces as the scratch allows, with none there is one CTA per sequence and head
    S, H, Hkv, D, bs = 3, 16, 2, 128, 16
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, Hkv, D, bs, seed=315, min_len=700, max_len=2100)
    scale = np.float32(1 / math.sqrt(D))
    o, lse = run_paged(Q, Kc, Vc, table, lens, scale, workspace_bytes=workspace_bytes)
    o_ref, l_ref = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=scale)
    check_mha(o, lse, o_ref.reshape(-1, D), l_ref.reshape(-1), f"grouped heads, workspace {workspace_bytes}")


def test_grouped_heads_empty_short_and_long_sequences_together():
    # equal shares of work per CTA: rows without any token, rows shorter than a chunk, and one row much longer
    # than all others together (it bounds the share size: no row may need more than 32 partial results)
    S, H, Hkv, D, bs = 9, 16, 2, 64, 16
    Q, Kc, Vc, table, _ = inputs.paged_inputs(S, H, Hkv, D, bs, seed=316, min_len=9000, max_len=9000)
    lens = np.array([0, 1, 9000, 0, 17, 300, 128, 129, 0], dtype=np.int32)
    o, lse = run_paged(Q, Kc, Vc, table, lens, 0.125)
    o_ref, l_ref = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=0.125)
    o = o.reshape(S, H, D); lse = lse.reshape(S, H)
    for s_ in (0, 3, 8):
        assert (o[s_] == 0).all() and np.isneginf(lse[s_]).all()
    live = lens > 0
    check_mha(o[live].reshape(-1, D), lse[live].reshape(-1), o_ref[live].reshape(-1, D), l_ref[live].reshape(-1), "mixed rows")


def test_grouped_heads_more_sequences_than_the_balancing_table():
    # beyond 1024 sequences the grouped-head kernel falls back to fixed pieces per sequence
    S, H, Hkv, D, bs = 1100, 8, 2, 64, 16
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, Hkv, D, bs, seed=317, min_len=1, max_len=1100)
    o, lse = run_paged(Q, Kc, Vc, table, lens, 0.125)
    o_ref, l_ref = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=0.125)
    check_mha(o, lse, o_ref.reshape(-1, D), l_ref.reshape(-1), "1100 sequences")


def test_empty_and_single_token_sequences():
    S, H, D, bs = 4, 2, 64, 16
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, H, D, bs, seed=311, min_len=40, max_len=40)
    lens = np.array([0, 1, 16, 40], dtype=np.int32)
    o, lse = run_paged(Q, Kc, Vc, table, lens, 0.125)
    o = o.reshape(S, H, D); lse = lse.reshape(S, H)
    assert (o[0] == 0).all() and np.isneginf(lse[0]).all()
    assert np.array_equal(o[1], inputs.bf16_bits_to_f64(Vc[table[1, 0], :, 0]))     # one token: exactly its value
    o_ref, l_ref = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=0.125)
    check_mha(o[2:].reshape(-1, D), lse[2:].reshape(-1), o_ref[2:].reshape(-1, D), l_ref[2:].reshape(-1), "16 and 40")


def test_length_beyond_the_table_is_cut_at_the_table_end():
    # 75 table entries per sequence, split over CTAs of 8 blocks each (10 x 8 = 80 > 75): a stated length that the
    # table cannot reach must not make any CTA read past the sequence's row (for the last sequence: past the table)
    S, H, D, bs = 3, 4, 128, 16
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, H, D, bs, seed=314, min_len=1200, max_len=1200)
    assert table.shape[1] == 75 and (table >= 0).all()
    too_long = lens.copy(); too_long[0] += 37; too_long[-1] += 500
    scale = np.float32(1 / math.sqrt(D))
    o, lse = run_paged(Q, Kc, Vc, table, too_long, scale)
    o_ref, l_ref = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=scale)
    check_mha(o, lse, o_ref.reshape(-1, D), l_ref.reshape(-1), "over-long lengths")


def test_bad_block_table_entry_is_reported_not_dereferenced():
    S, H, D, bs = 1, 2, 64, 16
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, H, D, bs, seed=312, min_len=64, max_len=64)
    bad = table.copy(); bad[0, 2] = Kc.shape[0] + 1000
    dQ, dK, dV = to_dev(Q), to_dev(Kc), to_dev(Vc)
    dT = torch.from_numpy(bad).cuda(); dL = torch.from_numpy(lens).cuda()
    O = torch.empty(S * H * D, dtype=torch.int16, device="cuda")
    rc = mlt.paged_attn_decode_raw(dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), dT.data_ptr(), dL.data_ptr(), O.data_ptr(),
                                   0, S, H, H, D, bs, table.shape[1], Kc.shape[0], 0.125)
    assert rc == 0
    status, detail = mlt.last_device_error()
    assert status == 7 and detail[0] == 7 and detail[1] == 2 and detail[2] == 0
    assert mlt.last_device_error()[0] == 0      # cleared


def test_bad_entry_with_grouped_heads_leaves_the_pipeline_in_step():
    # the tensor-core kernel leaves out the 16-token unit of a bad entry; its shared-memory ring must stay in step
    # (a wrong barrier parity would show as a timeout), and the next call must be clean
    S, H, Hkv, D, bs = 2, 8, 2, 128, 16
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, Hkv, D, bs, seed=318, min_len=1500, max_len=1500)
    bad = table.copy(); bad[1, 5] = -7; bad[0, 40] = Kc.shape[0]
    o, _ = None, None
    dQ, dK, dV = to_dev(Q), to_dev(Kc), to_dev(Vc)
    dL = torch.from_numpy(lens).cuda()
    O = torch.empty(S * H * D, dtype=torch.int16, device="cuda")
    ws = torch.empty(mlt.paged_attn_workspace_bytes(S, H, D), dtype=torch.uint8, device="cuda")
    for tab, want in ((bad, 7), (table, 0)):
        dT = torch.from_numpy(tab).cuda()
        rc = mlt.paged_attn_decode_raw(dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), dT.data_ptr(), dL.data_ptr(), O.data_ptr(),
                                       0, S, H, Hkv, D, bs, tab.shape[1], Kc.shape[0], 0.09, ws.data_ptr(), ws.numel())
        assert rc == 0
        status, detail = mlt.last_device_error()
        assert status == want, (status, detail)
        assert torch.isfinite(O.view(torch.bfloat16).float()).all()
    o_ref, _ = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=0.09)
    got = inputs.bf16_bits_to_f64(O.cpu().numpy().view(np.uint16)).reshape(-1, D)
    check_mha(got, np.zeros(0), o_ref.reshape(-1, D), np.zeros(0), "after a bad entry")


def test_deterministic_across_runs():
    S, H, Hkv, D, bs = 6, 8, 2, 128, 16
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, Hkv, D, bs, seed=313, min_len=100, max_len=3000)
    a = run_paged(Q, Kc, Vc, table, lens, 0.09)
    b = run_paged(Q, Kc, Vc, table, lens, 0.09)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


@pytest.mark.parametrize("name", list(inputs.PAGED_CONFIGS))
def test_benchmark_configs(name):
    S, H, Hkv, D, bs, lo, hi, seed = inputs.PAGED_CONFIGS[name]
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, Hkv, D, bs, seed=seed, min_len=lo, max_len=hi)
    scale = np.float32(1 / math.sqrt(D))
    ws = torch.empty(mlt.paged_attn_workspace_bytes(S, H, D), dtype=torch.uint8, device="cuda")
    dT = torch.from_numpy(table).cuda(); dL = torch.from_numpy(lens).cuda()
    O, LSE = mlt.paged_attn_decode(to_dev(Q), to_dev(Kc), to_dev(Vc), dT, dL, scale=float(scale), workspace=ws)
    assert_device_healthy()
    assert torch.isfinite(O.float()).all() and torch.isfinite(LSE).all()
    # the oracle on a sample of sequences (all heads): shortest, longest and a few others
    order = np.argsort(lens)
    pick = sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2]), 0, S - 1})[:4]
    sub = np.array(pick)
    o_ref, l_ref = oracle.paged_attn_decode(Q[sub], Kc, Vc, table[sub], lens[sub], scale=scale)
    got_o = inputs.bf16_bits_to_f64(O[torch.from_numpy(sub).cuda()].contiguous().view(torch.int16).cpu().numpy().view(np.uint16))
    got_l = LSE[torch.from_numpy(sub).cuda()].cpu().numpy().astype(np.float64)
    rel, mx, dl = check_mha(got_o.reshape(-1, D), got_l.reshape(-1), o_ref.reshape(-1, D), l_ref.reshape(-1), name)
    print(f"{name}: rel_fro={rel:.3e} max_abs={mx:.3e} lse={dl:.3e}")
