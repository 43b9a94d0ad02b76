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
from parity import check_mha  # noqa: E402

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
         (2, 100, 256, 128, 64, 0), (2, 100, 256, 100, 128, 0), (3, 60, 128, 128, 64, 1), (3, 60, 100, 228, 128, 1)]


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


def test_dominant_key_and_outlier_rows():
    # rows scaled x8 make the running max jump by far more than the lazy-rescale threshold
    B, H, N, D = 1, 2, 640, 128
    Q, K, V = inputs.mha_inputs(B, H, N, N, D, seed=264, outlier_percent=5)
    for causal in (0, 1):
        o, lse = run_mha(Q, K, V, causal, scale_for(D))
        o_ref, lse_ref = oracle.mha_fwd(Q, K, V, causal=bool(causal), scale=scale_for(D))
        check_mha(o, lse, o_ref, lse_ref, f"outliers causal={causal}")
    # the largest key comes last: every earlier block's contribution must be rescaled away
    q = inputs.bf16_bits_to_f64(Q); k = inputs.bf16_bits_to_f64(K)
    k[0, 0, N - 1] = 40.0 * q[0, 0, 5] / np.linalg.norm(q[0, 0, 5])
    K2 = inputs.f64_to_bf16_bits(k)
    o, lse = run_mha(Q, K2, V, 0, scale_for(D))
    o_ref, lse_ref = oracle.mha_fwd(Q, K2, V, causal=False, scale=scale_for(D))
    check_mha(o, lse, o_ref, lse_ref, "dominant last key")


@pytest.mark.parametrize("B,H,N,D,causal", [(1, 4, 512, 128, True), (3, 70, 300, 64, True), (2, 90, 600, 128, False)])
def test_deterministic_across_runs(B, H, N, D, causal):
    # the second and third shapes have more work items than SMs (several items per persistent CTA)
    Q, K, V = inputs.mha_inputs(B, H, N, N, D, seed=265)
    dQ, dK, dV = to_dev(Q), to_dev(K), to_dev(V)
    runs = [mlt.mha_fwd(dQ, dK, dV, causal=causal, scale=scale_for(D)) for _ in range(4)]
    torch.cuda.synchronize()
    for o, l in runs[1:]:
        assert torch.equal(runs[0][0].view(torch.int16), o.view(torch.int16)) and torch.equal(runs[0][1], l)


@pytest.mark.parametrize("name", list(inputs.MHA_CONFIGS))
def test_benchmark_configs(name):
    B, H, Nq, Nk, D, causal, seed, outl = inputs.MHA_CONFIGS[name]
    Q, K, V = inputs.mha_inputs(B, H, Nq, Nk, D, seed=seed, outlier_percent=outl)
    dQ, dK, dV = to_dev(Q), to_dev(K), to_dev(V)
    O, LSE = mlt.mha_fwd(dQ, dK, dV, causal=bool(causal), scale=scale_for(D))
    assert_device_healthy()
    assert torch.isfinite(O.float()).all() and torch.isfinite(LSE).all()
    # sampled query rows: tile edges and interior rows in every head
    rng = np.random.default_rng(seed)
    per_head = 12 if Nq > 2048 else 24
    rows = []
    for bh in range(B * H):
        pick = set(rng.integers(0, Nq, per_head).tolist()) | {0, Nq - 1}
        t0 = int(rng.integers(0, Nq // 128)) * 128
        pick |= {t0, t0 + 127}
        rows += [bh * Nq + i for i in sorted(pick)]
    rows = np.array(rows, dtype=np.int64)
    o_ref, lse_ref = oracle.mha_fwd(Q, K, V, causal=bool(causal), scale=scale_for(D), qrows=rows)
    idx = torch.from_numpy(rows).cuda()
    got_o = to_f64(O.reshape(-1, D)[idx])
    got_l = LSE.reshape(-1)[idx].cpu().numpy().astype(np.float64)
    rel, mx, dl = check_mha(got_o, got_l, o_ref, lse_ref, name)
    print(f"{name}: rel_fro={rel:.3e} max_abs={mx:.3e} lse={dl:.3e}")


def test_argument_errors_do_not_launch():
    x = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    p = x.data_ptr()
    assert mlt.mha_fwd_raw(p, p, p, p, 0, 1, 1, 8, 8, 96, 0, 1.0) == 2      # head dimension
    assert mlt.mha_fwd_raw(p, p, p, p, 0, 1, 1, 9, 8, 64, 1, 1.0) == 1      # causal with Nq > Nk
    assert mlt.mha_fwd_raw(p, p, p, p, 0, 1, 1, 8, 0, 64, 0, 1.0) == 1      # no keys
    assert mlt.mha_fwd_raw(p, p, p + 2, p, 0, 1, 1, 8, 8, 64, 0, 1.0) == 3  # misaligned V
    assert mlt.mha_fwd_raw(p, p, p, p, 0, 1, 1, 8, 8, 64, 0, -1.0) == 1     # scale
    assert mlt.mha_fwd_raw(p, p, p, p, 0, 1, 0, 8, 8, 64, 0, 1.0) == 0      # empty batch
