"""GPU parity of mlt_mha_fwd (through the C ABI) against the FP64 three-pass oracle."""
import math

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
import paper_2503_14985_b200 as mlt  # noqa: E402
from paper_2503_14985_b200 import inputs  # noqa: E402

from gpu_util import assert_device_healthy, to_bits, to_dev, to_f64  # noqa: E402
from parity import LSE_TOL, MAX_ABS_TOL, REL_FRO_TOL, RunningErrors, check_mha, log_line  # noqa: E402

SENTINEL = 0x7FC1


def run_mha(Q, K, V, causal, scale, with_lse=True):
    """Runs mlt_mha_fwd on BF16 bit arrays with guard bands around O and LSE."""
    Bn, H, Nq, D = Q.shape
    Nk = K.shape[2]
    guard = 256
    Obuf = torch.from_numpy(np.full((Bn * H * Nq * D + 2 * guard,), SENTINEL, np.uint16).view(np.int16)).cuda()
    Lbuf = torch.full((Bn * H * Nq + 2 * guard,), float("nan"), dtype=torch.float32, device="cuda")
    O = Obuf[guard:guard + Bn * H * Nq * D].view(torch.bfloat16)
    L = Lbuf[guard:guard + Bn * H * Nq]
    dQ, dK, dV = to_dev(Q), to_dev(K), to_dev(V)
    rc = mlt.mha_fwd_raw(dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), O.data_ptr(), L.data_ptr() if with_lse else 0,
                         Bn, H, Nq, Nk, D, int(causal), float(np.float32(scale)),
                         torch.cuda.current_stream().cuda_stream)
    assert rc == 0, mlt.status_string(rc)
    assert_device_healthy()
    ob = Obuf.cpu().numpy().view(np.uint16)
    assert (ob[:guard] == SENTINEL).all() and (ob[-guard:] == SENTINEL).all(), "O guard band was written"
    lb = Lbuf.cpu().numpy()
    assert np.isnan(lb[:guard]).all() and np.isnan(lb[-guard:]).all(), "LSE guard band was written"
    body = ob[guard:-guard]
    assert not (body == SENTINEL).any(), "unwritten O elements"
    o = inputs.bf16_bits_to_f64(body).reshape(Bn * H * Nq, D)
    return o, (lb[guard:-guard].astype(np.float64) if with_lse else None)


def scale_for(D):
    return np.float32(1.0 / math.sqrt(D))


CASES = [(1, 1, 128, 128, 64, 0), (1, 1, 128, 128, 128, 1), (1, 2, 1, 1, 64, 0), (2, 3, 200, 333, 128, 0),
         (1, 1, 77, 200, 64, 1), (1, 1, 129, 129, 128, 1), (1, 4, 1024, 1024, 64, 1), (1, 2, 256, 256, 128, 0),
         (1, 3, 300, 300, 64, 0), (2, 2, 257, 640, 128, 1), (1, 1, 512, 384 + 1, 64, 0), (1, 9, 384, 384, 64, 1),
         (1, 1, 1, 700, 128, 1),
         # more work items than SMs: a CTA runs several items one after another (ragged last pairs among them)
         (3, 70, 300, 300, 64, 1), (2, 80, 300, 420, 128, 1), (5, 40, 520, 260, 128, 0), (2, 90, 257, 257, 64, 0),
         # ... with a single K/V block per item, and with the second 128-row tile absent in every item
         (2, 100, 256, 128, 64, 0), (2, 100, 256, 100, 128, 0), (3, 60, 128, 128, 64, 1), (3, 60, 100, 228, 128, 1),
         # a last round of at most half the CTAs (on 148 SMs: 2, 8 and 52 items left over), handed out as single tiles
         (1, 150, 256, 300, 128, 1), (1, 75, 512, 512, 64, 1), (2, 76, 512, 640, 64, 0), (1, 100, 512, 384, 128, 0)]


@pytest.mark.parametrize("B,H,Nq,Nk,D,causal", CASES)
def test_parity_small_and_ragged(B, H, Nq, Nk, D, causal):
    Q, K, V = inputs.mha_inputs(B, H, Nq, Nk, D, seed=200 + Nq + Nk + D)
    o, lse = run_mha(Q, K, V, causal, scale_for(D))
    o_ref, lse_ref = oracle.mha_fwd(Q, K, V, causal=bool(causal), scale=scale_for(D))
    rel, mx, dl = check_mha(o, lse, o_ref, lse_ref, f"{(B, H, Nq, Nk, D, causal)}")
    print(f"rel_fro={rel:.3e} max_abs={mx:.3e} lse={dl:.3e}")


def test_one_long_head_causal_d128():
    B, H, N, D = 1, 1, 4096, 128
    Q, K, V = inputs.mha_inputs(B, H, N, N, D, seed=250)
    o, lse = run_mha(Q, K, V, 1, scale_for(D))
    rows = np.unique(np.concatenate([np.arange(0, N, 97), [0, 127, 128, 255, 256, N - 1]])).astype(np.int64)
    o_ref, lse_ref = oracle.mha_fwd(Q, K, V, causal=True, scale=scale_for(D), qrows=rows)
    check_mha(o[rows], lse[rows], o_ref, lse_ref, "4096 causal")


def test_lse_pointer_may_be_null():
    Q, K, V = inputs.mha_inputs(1, 2, 130, 130, 64, seed=260)
    o, _ = run_mha(Q, K, V, 0, 0.125, with_lse=False)
    o_ref, _ = oracle.mha_fwd(Q, K, V, causal=False, scale=0.125)
    check_mha(o, np.zeros(0), o_ref, np.zeros(0), "no lse")


def test_closed_forms_constant_keys_and_constant_values():
    B, H, N, D = 1, 2, 300, 64
    Q, K, V = inputs.mha_inputs(B, H, N, N, D, seed=261)
    K[:] = K[:, :, :1, :]
    v = inputs.bf16_bits_to_f64(V)
    o, lse = run_mha(Q, K, V, 1, 0.125)
    prefix_mean = (np.cumsum(v, axis=2) / np.arange(1, N + 1)[None, None, :, None]).reshape(-1, D)
    s = 0.125 * np.einsum("bhid,bhd->bhi", inputs.bf16_bits_to_f64(Q), inputs.bf16_bits_to_f64(K)[:, :, 0])
    check_mha(o, lse, prefix_mean, (s + np.log(np.arange(1, N + 1))).reshape(-1), "constant keys")
    # causal row 0 returns V[0] exactly (P = 1 exactly, one product, BF16 output of a BF16 value)
    assert np.array_equal(o.reshape(B, H, N, D)[:, :, 0], v[:, :, 0])
    Q, K, V = inputs.mha_inputs(B, H, N, N, D, seed=262)
    V[:] = 0x3F40  # 0.75
    o, _ = run_mha(Q, K, V, 0, 0.125)
    np.testing.assert_allclose(o, 0.75, atol=4e-3)


def test_key_permutation_invariance_across_blocks():
    B, H, Nq, Nk, D = 1, 1, 128, 512, 128
    Q, K, V = inputs.mha_inputs(B, H, Nq, Nk, D, seed=263)
    perm = np.random.default_rng(5).permutation(Nk)
    o1, l1 = run_mha(Q, K, V, 0, scale_for(D))
    o2, l2 = run_mha(Q, np.ascontiguousarray(K[:, :, perm]), np.ascontiguousarray(V[:, :, perm]), 0, scale_for(D))
    np.testing.assert_allclose(o1, o2, atol=2e-2)
    np.testing.assert_allclose(l1, l2, atol=1e-4)


@pytest.mark.parametrize("D", [128, 64])
def test_dominant_key_and_outlier_rows(D):
    # rows scaled x8 make the row max jump far above the reference max of the row's first block: the kernel has to
    # notice (a block sum at or above 2^64), take the true max, rescale O and l and repeat the pass
    B, H, N = 1, 2, 640
    sc = scale_for(D)
    Q, K, V = inputs.mha_inputs(B, H, N, N, D, seed=264, outlier_percent=5)
    for causal in (0, 1):
        o, lse = run_mha(Q, K, V, causal, sc)
        o_ref, lse_ref = oracle.mha_fwd(Q, K, V, causal=bool(causal), scale=sc)
        check_mha(o, lse, o_ref, lse_ref, f"outliers D={D} causal={causal}")
    # One key of the last block dominates query row 5 by `gap` nats: every earlier block's contribution must be
    # rescaled away.  2^64 = e^44.4, so a gap of 60 nats is sure to take the rescale branch; 120 nats (173 in
    # base 2) is beyond the range a single-precision 2^x can hold.  Key positions 626 and 635 are 2 and 11 modulo
    # 16: at D = 64 those exponentials are evaluated by the polynomial on the FMA pipe, 639 by the MUFU path.
    q = inputs.bf16_bits_to_f64(Q); k0 = inputs.bf16_bits_to_f64(K)
    for pos in (N - 1, 626, 635):
        for gap in (60.0, 120.0):
            k = k0.copy()
            k[0, 0, pos] = (gap / float(sc)) * q[0, 0, 5] / np.dot(q[0, 0, 5], q[0, 0, 5])
            K2 = inputs.f64_to_bf16_bits(k)
            # the jump as the kernel sees it: the dominant score against the best score of the row's first block
            s_row = float(sc) * inputs.bf16_bits_to_f64(K2)[0, 0] @ q[0, 0, 5]
            assert s_row[pos] - s_row[:128].max() > 45.0, "the test input does not force the rescale branch"
            o, lse = run_mha(Q, K2, V, 0, sc)
            o_ref, lse_ref = oracle.mha_fwd(Q, K2, V, causal=False, scale=sc)
            check_mha(o, lse, o_ref, lse_ref, f"dominant key at {pos}, gap {gap}, D={D}")


def test_all_three_tensors_with_outlier_rows():
    # The long-sequence recipe with the x8 rows in V as well (the other reading of "1 % of rows scaled x8"): outputs
    # are no longer unit scale, so the max-abs bound is applied relative to s = max(1, max|O_ref|).  Reported
    # separately from the benchmark configurations.
    for (B, H, N, D, causal) in [(1, 4, 2048, 128, 1), (1, 4, 2048, 128, 0), (1, 4, 1024, 64, 1)]:
        Q, K, V = inputs.mha_inputs(B, H, N, N, D, seed=266, outlier_percent=1, outlier_v=True)
        assert inputs.outlier_rows(266, inputs.TENSOR_V, B * H * N, 1).any()
        o, lse = run_mha(Q, K, V, causal, scale_for(D))
        o_ref, lse_ref = oracle.mha_fwd(Q, K, V, causal=bool(causal), scale=scale_for(D))
        unit = max(1.0, float(np.abs(o_ref).max()))
        rel, mx, dl = check_mha(o, lse, o_ref, lse_ref, f"Q/K/V outliers {(B, H, N, D, causal)}", unit=unit)
        log_line(f"Q/K/V-all-scaled variant B{B} H{H} N{N} D{D} causal={causal}: every element, rel_fro={rel:.3e} "
                 f"max_abs/s={mx:.3e} (s = max(1, max|O_ref|) = {unit:.2f}) lse={dl:.3e}")


@pytest.mark.parametrize("B,H,N,D,causal", [(1, 4, 512, 128, True), (3, 70, 300, 64, True), (2, 90, 600, 128, False)])
def test_deterministic_across_runs(B, H, N, D, causal):
    # the second and third shapes have more work items than SMs (several items per persistent CTA)
    Q, K, V = inputs.mha_inputs(B, H, N, N, D, seed=265)
    dQ, dK, dV = to_dev(Q), to_dev(K), to_dev(V)
    runs = [mlt.mha_fwd(dQ, dK, dV, causal=causal, scale=scale_for(D)) for _ in range(4)]
    torch.cuda.synchronize()
    for o, l in runs[1:]:
        assert torch.equal(runs[0][0].view(torch.int16), o.view(torch.int16)) and torch.equal(runs[0][1], l)


def _compare_by_heads(O, LSE, Q, K, V, causal, sc, heads_per_chunk=4, rows_of_head=None):
    """Every query row (or rows_of_head, the same row indices in every head) of O and LSE against the oracle, a few
    heads at a time; returns (rel_fro, max_abs, max LSE error, rows compared)."""
    Bn, H, Nq, D = Q.shape
    acc = RunningErrors()
    dl = 0.0
    nrows = 0
    O2 = O.reshape(Bn * H, Nq, D)
    L2 = LSE.reshape(Bn * H, Nq)
    for h0 in range(0, Bn * H, heads_per_chunk):
        h1 = min(Bn * H, h0 + heads_per_chunk)
        if rows_of_head is None:
            rows = np.arange(h0 * Nq, h1 * Nq, dtype=np.int64)
            got_o, got_l = to_f64(O2[h0:h1]).reshape(-1, D), L2[h0:h1].reshape(-1).cpu().numpy().astype(np.float64)
        else:
            rows = (np.arange(h0, h1, dtype=np.int64)[:, None] * Nq + rows_of_head[None, :]).reshape(-1)
            idx = torch.from_numpy(rows_of_head).cuda()
            got_o = to_f64(O2[h0:h1][:, idx]).reshape(-1, D)
            got_l = L2[h0:h1][:, idx].reshape(-1).cpu().numpy().astype(np.float64)
        o_ref, l_ref = oracle.mha_fwd(Q, K, V, causal=bool(causal), scale=sc, qrows=rows)
        acc.add(got_o, o_ref)
        assert np.isfinite(got_l).all()
        dl = max(dl, float(np.abs(got_l - l_ref).max()))
        nrows += len(rows)
    return acc.rel_fro(), acc.max_abs, dl, nrows


@pytest.mark.parametrize("name", list(inputs.MHA_CONFIGS))
def test_benchmark_configs_every_element(name):
    # Every element of O and LSE against the FP64 oracle, launched exactly as bench.py launches it; the figures go
    # to the parity log.
    import time
    B, H, Nq, Nk, D, causal, seed, outl = inputs.MHA_CONFIGS[name]
    Q, K, V = inputs.mha_inputs(B, H, Nq, Nk, D, seed=seed, outlier_percent=outl)
    dQ, dK, dV = to_dev(Q), to_dev(K), to_dev(V)
    O = torch.empty_like(dQ)
    LSE = torch.empty((B, H, Nq), dtype=torch.float32, device="cuda")
    rc = mlt.mha_fwd_raw(dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), O.data_ptr(), LSE.data_ptr(), B, H, Nq, Nk, D,
                         causal, float(scale_for(D)), torch.cuda.current_stream().cuda_stream)
    assert rc == 0, mlt.status_string(rc)
    assert_device_healthy()
    t0 = time.perf_counter()
    rel, mx, dl, nrows = _compare_by_heads(O, LSE, Q, K, V, causal, scale_for(D))
    secs = time.perf_counter() - t0
    log_line(f"{name}: all {nrows} query rows x {D}, rel_fro={rel:.3e} max_abs={mx:.3e} lse={dl:.3e} "
             f"(limits {REL_FRO_TOL:.0e} / {MAX_ABS_TOL:.0e} / {LSE_TOL:.0e}); oracle {secs:.1f} s on "
             f"{oracle.hardware_threads()} threads")
    assert rel <= REL_FRO_TOL and mx <= MAX_ABS_TOL and dl <= LSE_TOL, (name, rel, mx, dl)


# Sec. 4.2's benchmark shapes: 32k tokens in all, hidden size 2048 as 32 heads of 64 or 16 heads of 128, sequence
# length up to 32k; the shapes below are the ones no other test reaches (D = 64 beyond 1k tokens, 32k tokens).
SWEEP_SHAPES = [(4, 32, 8192, 64), (2, 32, 16384, 64), (1, 32, 32768, 64), (1, 16, 32768, 128)]


@pytest.mark.parametrize("causal", [0, 1])
@pytest.mark.parametrize("B,H,N,D", SWEEP_SHAPES)
def test_paper_sweep_shapes_sampled_rows(B, H, N, D, causal):
    Q, K, V = inputs.mha_inputs(B, H, N, N, D, seed=300 + N // 1024 + D)
    dQ, dK, dV = to_dev(Q), to_dev(K), to_dev(V)
    O, LSE = mlt.mha_fwd(dQ, dK, dV, causal=bool(causal), scale=scale_for(D))
    assert_device_healthy()
    assert torch.isfinite(O.float()).all() and torch.isfinite(LSE).all()
    # the same rows in every head: both ends, both sides of tile and 256-row item edges, and seeded interior rows
    rng = np.random.default_rng(N + D + causal)
    t0 = int(rng.integers(1, N // 256 - 1)) * 256
    rows = np.unique(np.concatenate([[0, 1, 127, 128, 255, 256, t0 - 1, t0, t0 + 127, t0 + 128, N - 257, N - 256,
                                      N - 129, N - 128, N - 1], rng.integers(0, N, 9)])).astype(np.int64)
    rel, mx, dl, nrows = _compare_by_heads(O, LSE, Q, K, V, causal, scale_for(D), heads_per_chunk=B * H,
                                           rows_of_head=rows)
    log_line(f"sweep shape B{B} H{H} N{N} D{D} causal={causal}: {nrows} sampled query rows ({len(rows)} per head), "
             f"rel_fro={rel:.3e} max_abs={mx:.3e} lse={dl:.3e}")
    assert rel <= REL_FRO_TOL and mx <= MAX_ABS_TOL and dl <= LSE_TOL, (rel, mx, dl)


@pytest.mark.parametrize("B,H,Nq,Nk,D,causal", [(2, 80, 16384, 128, 64, 0), (70, 148, 129, 129, 128, 1)])
def test_more_items_than_the_decoded_table_holds(B, H, Nq, Nk, D, causal):
    # A persistent CTA decodes its first 64 work items into shared memory ahead of time and the later ones on the
    # fly, in the loader, the issuer and every softmax warp: these launches give every CTA more than 64 items.
    props = torch.cuda.get_device_properties(0)
    items = B * H * ((Nq + 255) // 256)
    assert items > 64 * props.multi_processor_count
    Q, K, V = inputs.mha_inputs(B, H, Nq, Nk, D, seed=270 + D)
    dQ, dK, dV = to_dev(Q), to_dev(K), to_dev(V)
    O, LSE = mlt.mha_fwd(dQ, dK, dV, causal=bool(causal), scale=scale_for(D))
    assert_device_healthy()
    rel, mx, dl, nrows = _compare_by_heads(O, LSE, Q, K, V, causal, scale_for(D), heads_per_chunk=16)
    log_line(f"{items} work items (B{B} H{H} Nq{Nq} Nk{Nk} D{D} causal={causal}): all {nrows} query rows, "
             f"rel_fro={rel:.3e} max_abs={mx:.3e} lse={dl:.3e}")
    assert rel <= REL_FRO_TOL and mx <= MAX_ABS_TOL and dl <= LSE_TOL, (rel, mx, dl)


def test_argument_errors_do_not_launch():
    x = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    p = x.data_ptr()
    assert mlt.mha_fwd_raw(p, p, p, p, 0, 1, 1, 8, 8, 96, 0, 1.0) == 2      # head dimension
    assert mlt.mha_fwd_raw(p, p, p, p, 0, 1, 1, 9, 8, 64, 1, 1.0) == 1      # causal with Nq > Nk
    assert mlt.mha_fwd_raw(p, p, p, p, 0, 1, 1, 8, 0, 64, 0, 1.0) == 1      # no keys
    assert mlt.mha_fwd_raw(p, p, p + 2, p, 0, 1, 1, 8, 8, 64, 0, 1.0) == 3  # misaligned V
    assert mlt.mha_fwd_raw(p, p, p, p, 0, 1, 1, 8, 8, 64, 0, -1.0) == 1     # scale
    assert mlt.mha_fwd_raw(p, p, p, p, 0, 1, 0, 8, 8, 64, 0, 1.0) == 0      # empty batch
