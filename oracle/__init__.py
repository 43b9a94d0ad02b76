"""CPU oracle (FP64) for the GEMM and MHA-forward hot path -- TEST INFRASTRUCTURE.

Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s cpu_baseline /
reference legs may import this package.  The product package never does, and
this package imports nothing from the product.

The arithmetic lives in ``oracle.cpp`` (plain C++, threads over output rows);
this file only compiles it with g++ and marshals numpy arrays through ctypes.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile oracle.cpp into liboracle.so next to it (if stale) and return the path."""
    with _lock:
        stale = force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["g++", "-O3", "-march=native", "-std=c++17", "-fPIC", "-shared", "-pthread",
                   "-fno-fast-math", "-ffp-contract=off", "-o", tmp, _SRC]
            try:
                subprocess.run(cmd, check=True, capture_output=True, text=True)
            except subprocess.CalledProcessError as e:  # pragma: no cover
                raise RuntimeError(f"oracle build failed:\n{e.stderr}") from e
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, p, i32 = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        lib.oracle_gemm.argtypes = [p, p, p, i64, i64, i64, i64, i64, p, i64, i32]
        lib.oracle_gemm.restype = i32
        lib.oracle_gemm_f16.argtypes = [p, p, p, p, i64, i64, i64, i64, i64, i64, p, i64, i32]
        lib.oracle_gemm_f16.restype = i32
        lib.oracle_f16_to_double.argtypes = [p, p, i64]
        lib.oracle_f16_to_double.restype = i32
        lib.oracle_mha_fwd.argtypes = [p, p, p, p, p, p, i32, i32, i32, i32, i32, i32, ctypes.c_float, p, i64, i32]
        lib.oracle_mha_fwd.restype = i32
        lib.oracle_hardware_threads.restype = i32
        lib.oracle_paged_attn_decode.argtypes = [p, p, p, p, p, p, p, i32, i32, i32, i32, i32, i32, i32,
                                                 ctypes.c_float, i32]
        lib.oracle_paged_attn_decode.restype = i32
        _lib = lib
    return _lib


def hardware_threads() -> int:
    return int(_load().oracle_hardware_threads())


def _u16(x: np.ndarray) -> np.ndarray:
    if x.dtype != np.uint16:
        raise TypeError("oracle inputs are BF16 bit patterns (uint16)")
    return x


def gemm(A: np.ndarray, B: np.ndarray, M: int, N: int, K: int, *, rows=None, nthreads: int = 0) -> np.ndarray:
    """C = A @ B in FP64 over BF16 inputs (Sec. 2, Listing 2).

    A: (M, lda) uint16, B: (K, ldb) uint16 (row-major, padded pitch allowed).
    rows: optional 1-D list of output rows; returns (len(rows) or M, N) float64.
    """
    A = np.ascontiguousarray(_u16(A))
    B = np.ascontiguousarray(_u16(B))
    lda = A.shape[1] if A.ndim == 2 and A.shape[0] > 0 else max(K, 1)
    ldb = B.shape[1] if B.ndim == 2 and B.shape[0] > 0 else max(N, 1)
    if A.size and A.shape[0] < M or B.size and B.shape[0] < K:
        raise ValueError("array smaller than the stated shape")
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        R, rp = len(rows), rows.ctypes.data
    else:
        R, rp = M, None
    out = np.empty((R, N), dtype=np.float64)
    if R == 0 or N == 0:
        return out
    rc = _load().oracle_gemm(A.ctypes.data if A.size else None, B.ctypes.data if B.size else None,
                             out.ctypes.data, M, N, K, lda, ldb, rp, R, nthreads)
    if rc != 0:
        raise ValueError("oracle_gemm: invalid argument")
    return out


def f16_to_double(bits: np.ndarray) -> np.ndarray:
    """Values of binary16 bit patterns, by the oracle's own field-by-field conversion."""
    bits = np.ascontiguousarray(_u16(bits)).ravel()
    out = np.empty(bits.size, dtype=np.float64)
    if bits.size and _load().oracle_f16_to_double(bits.ctypes.data, out.ctypes.data, bits.size) != 0:
        raise ValueError("oracle_f16_to_double: invalid argument")
    return out


def gemm_f16(A: np.ndarray, B: np.ndarray, M: int, N: int, K: int, *, C_in=None, rows=None,
             nthreads: int = 0) -> np.ndarray:
    """C = [C_in +] A @ B in FP64 over FP16 inputs (Listing 2 data types; Sec. 2 accumulate form).

    A: (M, lda) uint16 binary16 patterns, B: (K, ldb) uint16; C_in: None or (M, ldc) float32.
    rows: optional 1-D list of output rows; returns (len(rows) or M, N) float64.
    """
    A = np.ascontiguousarray(_u16(A))
    B = np.ascontiguousarray(_u16(B))
    lda = A.shape[1] if A.ndim == 2 and A.shape[0] > 0 else max(K, 1)
    ldb = B.shape[1] if B.ndim == 2 and B.shape[0] > 0 else max(N, 1)
    if A.size and A.shape[0] < M or B.size and B.shape[0] < K:
        raise ValueError("array smaller than the stated shape")
    cp, ldc = None, max(N, 1)
    if C_in is not None:
        C_in = np.ascontiguousarray(C_in, dtype=np.float32)
        if C_in.ndim != 2 or C_in.shape[0] < M or C_in.shape[1] < N:
            raise ValueError("C_in smaller than the stated shape")
        cp, ldc = (C_in.ctypes.data if C_in.size else None), max(C_in.shape[1], 1)
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        R, rp = len(rows), rows.ctypes.data
    else:
        R, rp = M, None
    out = np.empty((R, N), dtype=np.float64)
    if R == 0 or N == 0:
        return out
    rc = _load().oracle_gemm_f16(A.ctypes.data if A.size else None, B.ctypes.data if B.size else None, cp,
                                 out.ctypes.data, M, N, K, lda, ldb, ldc, rp, R, nthreads)
    if rc != 0:
        raise ValueError("oracle_gemm_f16: invalid argument")
    return out


def mha_fwd(Q: np.ndarray, K: np.ndarray, V: np.ndarray, *, causal: bool, scale, qrows=None,
            return_probs: bool = False, nthreads: int = 0):
    """Exact softmax attention in FP64 (Algorithm 1 as the definition it reaches).

    Q: [B,H,Nq,D], K,V: [B,H,Nk,D] uint16 BF16 bits.  `scale` is narrowed to
    float32 first (the value the GPU entry point receives).  qrows: optional
    flat query indices (b*H + h)*Nq + i.  Returns (O [R,D], LSE [R]) or, with
    return_probs, (O, LSE, P [R,Nk]); R = len(qrows) or B*H*Nq.
    """
    Q = np.ascontiguousarray(_u16(Q))
    K = np.ascontiguousarray(_u16(K))
    V = np.ascontiguousarray(_u16(V))
    Bn, H, Nq, D = Q.shape
    Nk = K.shape[2]
    if K.shape != (Bn, H, Nk, D) or V.shape != K.shape:
        raise ValueError("shape mismatch")
    if qrows is not None:
        qrows = np.ascontiguousarray(qrows, dtype=np.int64)
        R, rp = len(qrows), qrows.ctypes.data
    else:
        R, rp = Bn * H * Nq, None
    O = np.empty((R, D), dtype=np.float64)
    LSE = np.empty((R,), dtype=np.float64)
    P = np.empty((R, Nk), dtype=np.float64) if return_probs else None
    if R > 0:
        rc = _load().oracle_mha_fwd(Q.ctypes.data, K.ctypes.data, V.ctypes.data, O.ctypes.data, LSE.ctypes.data,
                                    P.ctypes.data if return_probs else None, Bn, H, Nq, Nk, D, int(bool(causal)),
                                    float(np.float32(scale)), rp, R, nthreads)
        if rc != 0:
            raise ValueError("oracle_mha_fwd: invalid argument")
    return (O, LSE, P) if return_probs else (O, LSE)


def paged_attn_decode(Q: np.ndarray, K_cache: np.ndarray, V_cache: np.ndarray, block_table: np.ndarray,
                      seq_lens: np.ndarray, *, scale, nthreads: int = 0):
    """Paged-attention decode in FP64 (Sec. 3.2 / 4.3): softmax attention of one query token per sequence over
    the keys and values its block table points to.

    Q: [num_seqs, H, D]; K_cache, V_cache: [num_blocks, H_kv, block_size, D] uint16 BF16 bits;
    block_table: [num_seqs, max_blocks] int32; seq_lens: [num_seqs] int32.  Returns (O [num_seqs, H, D], LSE [num_seqs, H]).
    """
    Q = np.ascontiguousarray(_u16(Q))
    K_cache = np.ascontiguousarray(_u16(K_cache))
    V_cache = np.ascontiguousarray(_u16(V_cache))
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    S, H, D = Q.shape
    NB, H_kv, bs, D2 = K_cache.shape
    if D2 != D or V_cache.shape != K_cache.shape or block_table.shape[0] != S or seq_lens.shape != (S,):
        raise ValueError("shape mismatch")
    O = np.empty((S, H, D), dtype=np.float64)
    LSE = np.empty((S, H), dtype=np.float64)
    if S > 0:
        rc = _load().oracle_paged_attn_decode(Q.ctypes.data, K_cache.ctypes.data, V_cache.ctypes.data,
                                              block_table.ctypes.data, seq_lens.ctypes.data, O.ctypes.data,
                                              LSE.ctypes.data, S, H, H_kv, D, bs, block_table.shape[1], NB,
                                              float(np.float32(scale)), nthreads)
        if rc != 0:
            raise ValueError("oracle_paged_attn_decode: invalid argument")
    return O, LSE
