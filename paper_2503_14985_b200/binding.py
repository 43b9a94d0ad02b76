"""Thin ctypes binding over the C ABI of include/mlt.h.

Argument marshalling only: every step of the GEMM and of the attention forward
runs inside the CUDA kernels of libmlt.so.  There is no fallback: if the library
is missing or the device is not sm_100, calls raise.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmlt.so")

MLT_OK = 0
STATUS_NAMES = {0: "MLT_OK", 1: "MLT_ERR_INVALID_ARG", 2: "MLT_ERR_UNSUPPORTED", 3: "MLT_ERR_ALIGNMENT",
                4: "MLT_ERR_CUDA", 5: "MLT_ERR_ARCH", 6: "MLT_ERR_TIMEOUT", 7: "MLT_ERR_BAD_BLOCK",
                8: "MLT_ERR_SCRATCH_LIMIT"}
PAGED_STATIC_SCRATCH_BYTES = 16 * 1024 * 1024

EXPORTS = ("mlt_gemm", "mlt_gemm_f16", "mlt_gemm_ex", "mlt_gemm_workspace_bytes", "mlt_mha_fwd", "mlt_paged_attn_decode", "mlt_paged_attn_decode_static",
           "mlt_paged_attn_workspace_bytes",
           "mlt_last_device_error", "mlt_debug_wait_timeout_selftest", "mlt_debug_last_clock_mhz", "mlt_debug_gemm_plan", "mlt_status_string",
           "mlt_version")

_lib = None


class MltError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {STATUS_NAMES.get(status, status)} ({status_string(status)})")


def load() -> ctypes.CDLL:
    """Load libmlt.so (built in-tree by paper_2503_14985_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} not found: build it with `python -m paper_2503_14985_b200.build`")
        lib = ctypes.CDLL(LIB_PATH)
        i64, p, i32 = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        lib.mlt_gemm.argtypes = [p, p, p, i64, i64, i64, i64, i64, i64, p]
        lib.mlt_gemm.restype = i32
        lib.mlt_debug_wait_timeout_selftest.argtypes = [ctypes.c_uint64, p]
        lib.mlt_debug_wait_timeout_selftest.restype = i32
        lib.mlt_debug_last_clock_mhz.argtypes = [i32, ctypes.POINTER(ctypes.c_double)]
        lib.mlt_debug_last_clock_mhz.restype = i32
        lib.mlt_debug_gemm_plan.argtypes = [i64, i64, i64, ctypes.c_size_t, i32, ctypes.POINTER(ctypes.c_int)]
        lib.mlt_debug_gemm_plan.restype = i32
        lib.mlt_gemm_f16.argtypes = [p, p, p, i64, i64, i64, i64, i64, i64, i32, p]
        lib.mlt_gemm_f16.restype = i32
        lib.mlt_gemm_ex.argtypes = [p, p, p, i64, i64, i64, i64, i64, i64, p, ctypes.c_size_t, p]
        lib.mlt_gemm_ex.restype = i32
        lib.mlt_gemm_workspace_bytes.argtypes = [i64, i64, i64]
        lib.mlt_gemm_workspace_bytes.restype = ctypes.c_size_t
        lib.mlt_mha_fwd.argtypes = [p, p, p, p, p, i32, i32, i32, i32, i32, i32, ctypes.c_float, p]
        lib.mlt_mha_fwd.restype = i32
        lib.mlt_paged_attn_workspace_bytes.argtypes = [i32, i32, i32]
        lib.mlt_paged_attn_workspace_bytes.restype = ctypes.c_size_t
        lib.mlt_paged_attn_decode.argtypes = [p, p, p, p, p, p, p, i32, i32, i32, i32, i32, i32, i32, ctypes.c_float,
                                              p, ctypes.c_size_t, p]
        lib.mlt_paged_attn_decode.restype = i32
        lib.mlt_paged_attn_decode_static.argtypes = [p, p, p, p, p, p, p, i32, i32, i32, i32, i32, i32, i32,
                                                     ctypes.c_float, p]
        lib.mlt_paged_attn_decode_static.restype = i32
        lib.mlt_last_device_error.argtypes = [p]
        lib.mlt_last_device_error.restype = i32
        lib.mlt_status_string.argtypes = [i32]
        lib.mlt_status_string.restype = ctypes.c_char_p
        lib.mlt_version.restype = i32
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load().mlt_status_string(int(status)).decode()


def version() -> int:
    return int(load().mlt_version())


def gemm_raw(A: int, B: int, C: int, M: int, N: int, K: int, lda: int, ldb: int, ldc: int, stream: int = 0) -> int:
    """mlt_gemm with raw device addresses; returns the status code."""
    return int(load().mlt_gemm(A, B, C, M, N, K, lda, ldb, ldc, stream))


def debug_wait_timeout_selftest(budget_cycles: int, stream: int = 0) -> int:
    """Launches the bounded-wait self-test (a wait that runs out after `budget_cycles` SM clocks); returns the status."""
    return int(load().mlt_debug_wait_timeout_selftest(budget_cycles, stream))


def gemm_f16_raw(A: int, B: int, C: int, M: int, N: int, K: int, lda: int, ldb: int, ldc: int, accumulate: int,
                 stream: int = 0) -> int:
    """mlt_gemm_f16 (FP16 operands, FP32 result, optional C += A*B) with raw device addresses."""
    return int(load().mlt_gemm_f16(A, B, C, M, N, K, lda, ldb, ldc, accumulate, stream))


def gemm_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(load().mlt_gemm_workspace_bytes(M, N, K))


def gemm_ex_raw(A: int, B: int, C: int, M: int, N: int, K: int, lda: int, ldb: int, ldc: int, workspace: int = 0,
                workspace_bytes: int = 0, stream: int = 0) -> int:
    """mlt_gemm_ex (split-K with caller scratch for skinny problems) with raw device addresses."""
    return int(load().mlt_gemm_ex(A, B, C, M, N, K, lda, ldb, ldc, workspace, workspace_bytes, stream))


def mha_fwd_raw(Q: int, K: int, V: int, O: int, LSE: int, B: int, H: int, Nq: int, Nk: int, D: int, causal: int,
                scale: float, stream: int = 0) -> int:
    """mlt_mha_fwd with raw device addresses; returns the status code."""
    return int(load().mlt_mha_fwd(Q, K, V, O, LSE, B, H, Nq, Nk, D, causal, scale, stream))


def paged_attn_workspace_bytes(num_seqs: int, H: int, D: int) -> int:
    return int(load().mlt_paged_attn_workspace_bytes(num_seqs, H, D))


def paged_attn_decode_raw(Q: int, K_cache: int, V_cache: int, block_table: int, seq_lens: int, O: int, LSE: int,
                          num_seqs: int, H: int, H_kv: int, D: int, block_size: int, max_blocks: int, num_blocks: int,
                          scale: float, workspace: int = 0, workspace_bytes: int = 0, stream: int = 0) -> int:
    """mlt_paged_attn_decode with raw device addresses; returns the status code."""
    return int(load().mlt_paged_attn_decode(Q, K_cache, V_cache, block_table, seq_lens, O, LSE, num_seqs, H, H_kv, D,
                                            block_size, max_blocks, num_blocks, scale, workspace, workspace_bytes,
                                            stream))


def paged_attn_decode_static_raw(Q: int, K_cache: int, V_cache: int, block_table: int, seq_lens: int, O: int, LSE: int,
                                 num_seqs: int, H: int, H_kv: int, D: int, block_size: int, max_blocks: int,
                                 num_blocks: int, scale: float, stream: int = 0) -> int:
    """mlt_paged_attn_decode_static (scratch inside the library, nothing allocated) with raw device addresses."""
    return int(load().mlt_paged_attn_decode_static(Q, K_cache, V_cache, block_table, seq_lens, O, LSE, num_seqs, H,
                                                   H_kv, D, block_size, max_blocks, num_blocks, scale, stream))


def last_device_error():
    """Synchronise, read and clear the device status word: (status, [code, barrier, block, aux])."""
    detail = (ctypes.c_uint32 * 4)()
    rc = int(load().mlt_last_device_error(ctypes.cast(detail, ctypes.c_void_p)))
    return rc, list(detail)


def last_clock_mhz(which: int) -> float:
    """SM clock in MHz that the last GEMM (which = 0) or attention (which = 1) launch ran at; 0.0 if none has run."""
    mhz = ctypes.c_double(0.0)
    rc = int(load().mlt_debug_last_clock_mhz(which, ctypes.byref(mhz)))
    if rc != MLT_OK:
        raise MltError(rc, "mlt_debug_last_clock_mhz")
    return float(mhz.value)


def gemm_plan(M: int, N: int, K: int, workspace_bytes: int = 0, sm_count: int = 148) -> dict:
    """Launch plan of gemm / gemm_ex for a shape: tile variant, K slices through the workspace, CTAs per K-cutting
    cluster, K blocks of 64 per slice.  sm_count >= 2: host arithmetic for such a device, no GPU; 0: the current device."""
    out = (ctypes.c_int * 4)()
    rc = int(load().mlt_debug_gemm_plan(M, N, K, workspace_bytes, sm_count, out))
    if rc != MLT_OK:
        raise MltError(rc, "mlt_debug_gemm_plan")
    return {"variant": out[0], "split_k": out[1], "cluster": out[2], "kb_per_split": out[3]}


def _stream(stream) -> int:
    import torch
    if stream is None:
        return int(torch.cuda.current_stream().cuda_stream)
    return int(getattr(stream, "cuda_stream", stream))


def gemm(A, B, C=None, *, M=None, N=None, K=None, stream=None):
    """C = A @ B for torch.bfloat16 CUDA tensors: A (M, K), B (K, N), row-major with unit inner stride.

    Row pitches are taken from the tensors' strides, so padded views work.  Returns C.
    """
    import torch
    if A.dtype != torch.bfloat16 or B.dtype != torch.bfloat16 or not A.is_cuda or not B.is_cuda:
        raise TypeError("A and B must be CUDA bfloat16 tensors")
    M = A.shape[0] if M is None else M
    K = A.shape[1] if K is None else K
    N = B.shape[1] if N is None else N
    if C is None:
        C = torch.empty((M, N), dtype=torch.bfloat16, device=A.device)
    for t in (A, B, C):
        if t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
            raise ValueError("operands must be 2-D with unit inner stride")
    lda = A.stride(0) if A.shape[0] > 1 else max(A.stride(0), K)
    ldb = B.stride(0) if B.shape[0] > 1 else max(B.stride(0), N)
    ldc = C.stride(0) if C.shape[0] > 1 else max(C.stride(0), N)
    rc = gemm_raw(A.data_ptr(), B.data_ptr(), C.data_ptr(), M, N, K, lda, ldb, ldc, _stream(stream))
    if rc != MLT_OK:
        raise MltError(rc, "mlt_gemm")
    return C


def mha_fwd(Q, K, V, *, causal: bool, scale: float, O=None, LSE=None, return_lse: bool = True, stream=None):
    """Attention forward for contiguous torch.bfloat16 CUDA tensors Q [B,H,Nq,D], K,V [B,H,Nk,D].

    Returns (O [B,H,Nq,D] bfloat16, LSE [B,H,Nq] float32 or None).
    """
    import torch
    for t in (Q, K, V):
        if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous() or t.dim() != 4:
            raise TypeError("Q, K, V must be contiguous 4-D CUDA bfloat16 tensors")
    Bn, H, Nq, D = Q.shape
    Nk = K.shape[2]
    if tuple(K.shape) != (Bn, H, Nk, D) or K.shape != V.shape:
        raise ValueError("shape mismatch")
    if O is None:
        O = torch.empty_like(Q)
    if LSE is None and return_lse:
        LSE = torch.empty((Bn, H, Nq), dtype=torch.float32, device=Q.device)
    rc = mha_fwd_raw(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr() if LSE is not None else 0,
                     Bn, H, Nq, Nk, D, int(bool(causal)), float(scale), _stream(stream))
    if rc != MLT_OK:
        raise MltError(rc, "mlt_mha_fwd")
    return O, LSE


def paged_attn_decode(Q, K_cache, V_cache, block_table, seq_lens, *, scale: float, workspace=None, O=None, LSE=None,
                      return_lse: bool = True, stream=None):
    """Paged-attention decode for CUDA tensors: Q [S,H,D] bfloat16, caches [num_blocks,H_kv,block_size,D] bfloat16,
    block_table [S,max_blocks] int32, seq_lens [S] int32.  `workspace` is an optional uint8 CUDA tensor (see
    paged_attn_workspace_bytes).  Returns (O [S,H,D] bfloat16, LSE [S,H] float32 or None).
    """
    import torch
    for t in (Q, K_cache, V_cache):
        if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous():
            raise TypeError("Q and the caches must be contiguous CUDA bfloat16 tensors")
    for t in (block_table, seq_lens):
        if t.dtype != torch.int32 or not t.is_cuda or not t.is_contiguous():
            raise TypeError("block_table and seq_lens must be contiguous CUDA int32 tensors")
    S, H, D = Q.shape
    NB, H_kv, bs, _ = K_cache.shape
    if O is None:
        O = torch.empty_like(Q)
    if LSE is None and return_lse:
        LSE = torch.empty((S, H), dtype=torch.float32, device=Q.device)
    rc = paged_attn_decode_raw(Q.data_ptr(), K_cache.data_ptr(), V_cache.data_ptr(), block_table.data_ptr(),
                               seq_lens.data_ptr(), O.data_ptr(), LSE.data_ptr() if LSE is not None else 0, S, H, H_kv, D,
                               bs, block_table.shape[1], NB, float(scale),
                               workspace.data_ptr() if workspace is not None else 0,
                               workspace.numel() * workspace.element_size() if workspace is not None else 0,
                               _stream(stream))
    if rc != MLT_OK:
        raise MltError(rc, "mlt_paged_attn_decode")
    return O, LSE
