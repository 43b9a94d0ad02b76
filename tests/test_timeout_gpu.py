"""The bounded device-side waits: a wait that nothing satisfies runs out, is reported, and leaves the context usable.

No fault, trap or hang is involved: the self-test kernel waits on a barrier with a budget of about a millisecond,
gives up, records the event in the device status word and returns like any other kernel.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
import paper_2503_14985_b200 as mlt  # noqa: E402
from paper_2503_14985_b200 import inputs  # noqa: E402

from gpu_util import to_dev, to_f64  # noqa: E402
from parity import check_gemm  # noqa: E402


def test_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    assert mlt.last_device_error()[0] == 0                       # clean start
    assert mlt.debug_wait_timeout_selftest(2_000_000) == 0       # about 1 ms of SM clocks
    rc, detail = mlt.last_device_error()                         # synchronises, reads and clears the status word
    assert rc == 6 and mlt.status_string(rc).startswith("a bounded device-side wait")
    assert detail[0] != 0 and detail[1] == 0x7E57 and detail[2] == 0 and detail[3] == 0
    assert mlt.last_device_error()[0] == 0                       # cleared by the read
    # the same context goes on computing
    M, N, K = 256, 384, 192
    A, B = inputs.gemm_inputs(M, N, K, seed=77)
    C = mlt.gemm(to_dev(A), to_dev(B))
    check_gemm(to_f64(C), oracle.gemm(A, B, M, N, K), "after the timeout self-test")
    assert mlt.last_device_error()[0] == 0


def test_budget_outside_the_range_is_refused_without_a_launch():
    assert mlt.debug_wait_timeout_selftest(0) == 1
    assert mlt.debug_wait_timeout_selftest(2_000_000_000) == 1
    assert mlt.last_device_error()[0] == 0


def test_kernels_report_the_clock_they_ran_at():
    # CTA 0 of the GEMM and attention kernels notes the SM cycle counter and the nanosecond timer at both ends
    import numpy as np
    from paper_2503_14985_b200 import inputs
    A, B = inputs.gemm_inputs(2048, 2048, 2048, seed=3)
    dA = torch.from_numpy(A.view(np.int16)).cuda().view(torch.bfloat16)
    dB = torch.from_numpy(B.view(np.int16)).cuda().view(torch.bfloat16)
    mlt.gemm(dA, dB)
    q = torch.randn(1, 8, 2048, 128, device="cuda").to(torch.bfloat16)
    mlt.mha_fwd(q, q, q, causal=True, scale=0.088)
    for which in (0, 1):
        mhz = mlt.last_clock_mhz(which)
        assert 300.0 < mhz < 2500.0, (which, mhz)
    assert mlt.binding.load().mlt_debug_last_clock_mhz(2, None) == 1
