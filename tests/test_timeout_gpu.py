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
