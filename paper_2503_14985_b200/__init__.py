"""B200 (sm_100a) dense hot path: BF16 GEMM and FlashAttention-2 style MHA forward.

`binding` wraps the C ABI of include/mlt.h (libmlt.so, built by `build`);
`inputs` holds the seeded synthetic workloads.  Nothing here computes on the CPU.
"""
from . import inputs  # noqa: F401
from .binding import (MltError, debug_wait_timeout_selftest, gemm, gemm_ex_raw, gemm_f16_raw, gemm_plan, gemm_raw, gemm_workspace_bytes, last_clock_mhz, last_device_error, load, mha_fwd, mha_fwd_raw,  # noqa: F401
                      paged_attn_decode, paged_attn_decode_raw, paged_attn_decode_static_raw,
                      paged_attn_workspace_bytes, status_string, version)
