"""mlt_paged_attn_decode_static: the decode entry point for callers that cannot hand over scratch memory
(an engine whose pool owns the whole device, a plug-in without an allocator, a loop where cudaMalloc is ruled
out).  Its scratch is an array inside the library.  Checked here against mlt_paged_attn_decode, which takes the
caller's workspace, on two calls in a row with different sequences (the array keeps the first call's contents),
against the CPU oracle, and for the claim itself: the amount of free device memory does not move across a call.

This file is named to be collected last, so that a run that stops at the first failure has already run every
other test."""
import math

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
import paper_2503_14985_b200 as mlt  # noqa: E402
from paper_2503_14985_b200 import inputs  # noqa: E402

from gpu_util import assert_device_healthy, to_dev  # noqa: E402
from parity import LSE_TOL, MAX_ABS_TOL, REL_FRO_TOL, errors  # noqa: E402


def _run_both(S, H, Hkv, D, bs, lo, hi, seed):
    Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, Hkv, D, bs, seed=seed, min_len=lo, max_len=hi)
    dQ, dK, dV = to_dev(Q), to_dev(Kc), to_dev(Vc)
    dT = torch.from_numpy(table).cuda(); dL = torch.from_numpy(lens).cuda()
    scale = float(np.float32(1 / math.sqrt(D)))
    sp = torch.cuda.current_stream().cuda_stream
    # reference: the entry point that takes the caller's workspace
    ws = torch.empty(mlt.paged_attn_workspace_bytes(S, H, D), dtype=torch.uint8, device="cuda")
    O_ref = torch.empty(S, H, D, dtype=torch.bfloat16, device="cuda"); L_ref = torch.empty(S, H, device="cuda")
    rc = mlt.paged_attn_decode_raw(dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), dT.data_ptr(), dL.data_ptr(),
                                   O_ref.data_ptr(), L_ref.data_ptr(), S, H, Hkv, D, bs, table.shape[1], Kc.shape[0],
                                   scale, ws.data_ptr(), ws.numel(), sp)
    assert rc == 0, mlt.status_string(rc)
    # under test: no workspace argument at all; outputs start as NaN so unwritten elements show
    O = torch.full((S, H, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    L = torch.full((S, H), float("nan"), device="cuda")
    rc = mlt.paged_attn_decode_static_raw(dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), dT.data_ptr(), dL.data_ptr(),
                                          O.data_ptr(), L.data_ptr(), S, H, Hkv, D, bs, table.shape[1], Kc.shape[0],
                                          scale, sp)
    assert rc == 0, mlt.status_string(rc)
    assert_device_healthy()
    o, o_ref = O.float().cpu().numpy().astype(np.float64), O_ref.float().cpu().numpy().astype(np.float64)
    rel, mx = errors(o.reshape(-1, D), o_ref.reshape(-1, D))
    assert rel <= REL_FRO_TOL and mx <= MAX_ABS_TOL, (rel, mx)
    assert float((L - L_ref).abs().max()) <= LSE_TOL
    # ... and against the oracle, so that the two CUDA entry points cannot be wrong in the same way unnoticed
    o_cpu, l_cpu = oracle.paged_attn_decode(Q, Kc, Vc, table, lens, scale=scale)
    rel, mx = errors(o.reshape(-1, D), o_cpu.reshape(-1, D))
    assert rel <= REL_FRO_TOL and mx <= MAX_ABS_TOL, (rel, mx)
    assert float(np.abs(L.cpu().numpy().astype(np.float64) - l_cpu).max()) <= LSE_TOL
    # The claim itself.  The first call on a device has looked the array's address up; a further call must leave
    # the device's free memory exactly where it was (outputs exist already, nothing is created in between).
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    rc = mlt.paged_attn_decode_static_raw(dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), dT.data_ptr(), dL.data_ptr(),
                                          O.data_ptr(), L.data_ptr(), S, H, Hkv, D, bs, table.shape[1], Kc.shape[0],
                                          scale, sp)
    assert rc == 0, mlt.status_string(rc)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "the entry point that allocates nothing changed the free device memory"
    return bool(torch.equal(O.view(torch.int16), O_ref.view(torch.int16)))


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # both shapes split every sequence over several CTAs, so the built-in scratch array is really used; the second
    # call has fewer, shorter sequences, so stale partials of the first call lie beside the ones it writes
    same1 = _run_both(6, 8, 8, 128, 16, 300, 3000, seed=401)
    same2 = _run_both(3, 8, 2, 64, 16, 40, 900, seed=402)
    # same kernels, same split: in fact the bits agree
    assert same1 and same2


def test_need_beyond_the_built_in_array_is_refused_without_a_launch():
    S, H, D, bs, max_blocks = 64, 32, 128, 16, 512          # 64 * 32 * 32 splits * 520 B = 34 MB > 16 MiB
    assert S * H * 32 * (4 * D + 8) > mlt.binding.PAGED_STATIC_SCRATCH_BYTES
    x = torch.zeros(1024, dtype=torch.int32, device="cuda")
    p = x.data_ptr()
    rc = mlt.paged_attn_decode_static_raw(p, p, p, p, p, p, 0, S, H, H, D, bs, max_blocks, 10, 0.1)
    assert rc == 8 and "scratch" in mlt.status_string(rc)
    assert mlt.last_device_error()[0] == 0
