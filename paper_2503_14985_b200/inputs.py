"""Seeded synthetic inputs for the GEMM and MHA-forward workloads.

This module produces *data only*.  It contains none of the arithmetic of the
GEMM or of attention, imports nothing from the rest of the package, and is the
one piece both the CUDA path's tests and the CPU oracle's tests may share.

Recipe (stateless, counter based, so any element can be regenerated alone):

* ``h = mix64(seed, tensor_id, stream, index)`` -- a splitmix64-style finaliser
  applied to a 64-bit combination of the four integers.
* ``u = (h >> 11 + 0.5) * 2**-53`` lies strictly inside (0, 1).
* uniform value ``2u - 1``; normal value by Box-Muller from two independent
  streams of the same index.
* the value is multiplied by the workload's scale in float64, narrowed to
  float32 (round to nearest even) and then to BF16 (round to nearest even);
  both the oracle and the GPU kernels only ever see the BF16 bit patterns
  (``uint16``).
* the logical element index is ``row * ncols + col`` and does not depend on
  any leading-dimension padding.

The workloads stand in for the paper's LLM-derived GEMM shapes (Sec. 4.1) and
its FlashAttention-2 forward benchmark (Sec. 4.2); the paper does not state
the values it timed, so the value distributions are the benchmark
configuration's (uniform[-1,1], N(0,1)/sqrt(K), N(0,1) with 1 % outlier rows).
"""
from __future__ import annotations

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)

TENSOR_A, TENSOR_B = 0, 1
TENSOR_Q, TENSOR_K, TENSOR_V = 0, 1, 2


def _mix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on a uint64 array (wraps modulo 2**64)."""
    x = x.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        x += np.uint64(0x9E3779B97F4A7C15)
        x ^= x >> np.uint64(30)
        x *= np.uint64(0xBF58476D1CE4E5B9)
        x ^= x >> np.uint64(27)
        x *= np.uint64(0x94D049BB133111EB)
        x ^= x >> np.uint64(31)
    return x


def _key(seed: int, tensor_id: int, stream: int) -> np.uint64:
    k = (seed * 0x100000001B3 + tensor_id * 0x9E3779B1 + stream * 0x85EBCA77 + 0x1234567) & 0xFFFFFFFFFFFFFFFF
    return _mix64(np.array([k], dtype=np.uint64))[0]


def hash_u01(seed: int, tensor_id: int, stream: int, index: np.ndarray) -> np.ndarray:
    """u in (0,1), 53 bits, for each logical element index."""
    idx = np.asarray(index, dtype=np.uint64)
    with np.errstate(over="ignore"):
        h = _mix64(idx * np.uint64(0xD1342543DE82EF95) + _key(seed, tensor_id, stream))
    return ((h >> np.uint64(11)).astype(np.float64) + 0.5) * (2.0 ** -53)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> BF16 bit pattern (uint16), round to nearest even."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    out = ((b + rounding) >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out = np.where(nan, np.uint16(0x7FC0), out)
    return out


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """BF16 bit pattern (uint16) -> float64, exact."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    return f32_to_bf16_bits(np.asarray(x, dtype=np.float64).astype(np.float32))


def _values(kind: str, seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    idx = np.arange(start, start + count, dtype=np.uint64)
    if kind == "uniform":
        return 2.0 * hash_u01(seed, tensor_id, 0, idx) - 1.0
    if kind == "normal":
        u1 = hash_u01(seed, tensor_id, 1, idx)
        u2 = hash_u01(seed, tensor_id, 2, idx)
        return np.sqrt(-2.0 * np.log(u1)) * np.cos((2.0 * np.pi) * u2)
    if kind == "ternary":  # exact small integers {-1, 0, 1}: bit-exact GEMM tests
        return np.floor(3.0 * hash_u01(seed, tensor_id, 3, idx)) - 1.0
    raise ValueError(f"unknown value kind {kind!r}")


def outlier_rows(seed: int, tensor_id: int, nrows: int, percent: int = 1) -> np.ndarray:
    """Boolean mask of rows scaled up (about `percent` % of rows, seeded)."""
    r = np.arange(nrows, dtype=np.uint64)
    with np.errstate(over="ignore"):
        h = _mix64(r * np.uint64(0xA24BAED4963EE407) + _key(seed, tensor_id, 7))
    return (h % np.uint64(100)) < np.uint64(percent)


def matrix_bf16(rows: int, cols: int, *, seed: int, tensor_id: int, kind: str = "normal",
                scale: float = 1.0, ld: int | None = None, pad_bits: int = 0x7FC0,
                row_scale: np.ndarray | None = None, chunk_rows: int | None = None,
                to_bits=None) -> np.ndarray:
    """rows x cols BF16 bit patterns in a (rows, ld) uint16 array.

    `to_bits` replaces the FP64 -> BF16 rounding by another 16-bit encoder (see matrix_f16).

    Padding columns (ld > cols) hold `pad_bits` (a NaN pattern by default) so
    that any read of padding poisons a result.
    """
    ld = cols if ld is None else ld
    if ld < cols:
        raise ValueError("ld < cols")
    out = np.full((rows, ld), pad_bits, dtype=np.uint16)
    if rows == 0 or cols == 0:
        return out
    if chunk_rows is None:
        chunk_rows = max(1, (1 << 20) // cols)

    def fill(r0: int) -> None:
        r1 = min(rows, r0 + chunk_rows)
        v = _values(kind, seed, tensor_id, r0 * cols, (r1 - r0) * cols).reshape(r1 - r0, cols)
        v = v * scale
        if row_scale is not None:
            v = v * row_scale[r0:r1, None]
        out[r0:r1, :cols] = (to_bits or f64_to_bf16_bits)(v)

    starts = range(0, rows, chunk_rows)
    if len(starts) > 4:  # every element depends only on its index: chunks can be filled by a few threads
        from concurrent.futures import ThreadPoolExecutor
        import os
        with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as pool:
            list(pool.map(fill, starts))
    else:
        for r0 in starts:
            fill(r0)
    return out


def f64_to_f16_bits(v: np.ndarray) -> np.ndarray:
    """FP64 values rounded to nearest-even binary16, as uint16 bit patterns."""
    with np.errstate(over="ignore"):  # beyond 65520 rounds to infinity, as the format says
        return np.asarray(v, dtype=np.float64).astype(np.float16).view(np.uint16)


def matrix_f16(rows: int, cols: int, *, seed: int, tensor_id: int, kind: str = "normal", scale: float = 1.0,
               ld: int | None = None) -> np.ndarray:
    """matrix_bf16's values (same generator, same indices) rounded to binary16 instead; padding holds a NaN."""
    return matrix_bf16(rows, cols, seed=seed, tensor_id=tensor_id, kind=kind, scale=scale, ld=ld, pad_bits=0x7E00,
                       to_bits=f64_to_f16_bits)


# --------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------

def gemm_inputs(M: int, N: int, K: int, *, seed: int, kind: str = "normal", scale: float | None = None,
                lda: int | None = None, ldb: int | None = None):
    """A (M x K, row-major, pitch lda) and B (K x N, row-major, pitch ldb) as uint16 BF16 bits."""
    if scale is None:
        scale = 1.0 / np.sqrt(max(K, 1)) if kind == "normal" else 1.0
    A = matrix_bf16(M, K, seed=seed, tensor_id=TENSOR_A, kind=kind, scale=scale, ld=lda)
    B = matrix_bf16(K, N, seed=seed, tensor_id=TENSOR_B, kind=kind, scale=scale, ld=ldb)
    return A, B


TENSOR_C = 6


def gemm_f16_inputs(M: int, N: int, K: int, *, seed: int, kind: str = "normal", scale: float | None = None,
                    lda: int | None = None, ldb: int | None = None, ldc: int | None = None, prior_c: bool = True):
    """A, B as binary16 bit patterns (layouts of gemm_inputs) and a prior C (M x ldc float32, N(0,1) values,
    NaN in padding columns; None if not `prior_c`) for the accumulate form."""
    if scale is None:
        scale = 1.0 / np.sqrt(max(K, 1)) if kind == "normal" else 1.0
    A = matrix_f16(M, K, seed=seed, tensor_id=TENSOR_A, kind=kind, scale=scale, ld=lda)
    B = matrix_f16(K, N, seed=seed, tensor_id=TENSOR_B, kind=kind, scale=scale, ld=ldb)
    if not prior_c:
        return A, B, None
    ldc = N if ldc is None else ldc
    C = np.full((M, ldc), np.nan, dtype=np.float32)
    step = max(1, (1 << 20) // max(N, 1))
    for r0 in range(0, M if N else 0, step):
        r1 = min(M, r0 + step)
        C[r0:r1, :N] = _values("normal", seed, TENSOR_C, r0 * N, (r1 - r0) * N).reshape(r1 - r0, N).astype(np.float32)
    return A, B, C


def mha_inputs(B: int, H: int, Nq: int, Nk: int, D: int, *, seed: int, outlier_percent: int = 0,
               outlier_factor: float = 8.0, outlier_v: bool = False):
    """Q [B,H,Nq,D], K and V [B,H,Nk,D] as uint16 BF16 bits, i.i.d. N(0,1).

    With `outlier_percent` > 0 about that percentage of the rows of Q and of K
    (chosen independently, seeded) is multiplied by `outlier_factor`; V rows
    too only if `outlier_v`.
    """
    def one(tensor_id: int, n: int, outliers: bool):
        rs = None
        if outliers and outlier_percent > 0:
            rs = np.where(outlier_rows(seed, tensor_id, B * H * n, outlier_percent), outlier_factor, 1.0)
        m = matrix_bf16(B * H * n, D, seed=seed, tensor_id=tensor_id, kind="normal", row_scale=rs)
        return m.reshape(B, H, n, D)
    return one(TENSOR_Q, Nq, True), one(TENSOR_K, Nk, True), one(TENSOR_V, Nk, outlier_v)


TENSOR_PAGED_Q, TENSOR_PAGED_K, TENSOR_PAGED_V = 3, 4, 5


def paged_inputs(num_seqs: int, H: int, H_kv: int, D: int, block_size: int, *, seed: int, min_len: int, max_len: int,
                 spare_blocks: int = 3):
    """A paged KV cache with a mix of sequence lengths, and one query token per sequence.

    Returns Q [num_seqs, H, D], K_cache and V_cache [num_blocks, H_kv, block_size, D] (uint16 BF16 bits, N(0,1)),
    block_table [num_seqs, max_blocks] int32 (a seeded permutation scatters the logical blocks over the physical
    pool; unused entries are -1) and seq_lens [num_seqs] int32 (seeded, uniform in [min_len, max_len]).
    """
    u = hash_u01(seed, TENSOR_PAGED_Q, 9, np.arange(num_seqs, dtype=np.uint64))
    seq_lens = (min_len + np.floor(u * (max_len - min_len + 1))).astype(np.int32)
    seq_lens = np.minimum(seq_lens, max_len)
    blocks_per_seq = (seq_lens + block_size - 1) // block_size
    max_blocks = int((max_len + block_size - 1) // block_size)
    total = int(blocks_per_seq.sum())
    num_blocks = total + spare_blocks
    # seeded permutation of the physical pool: order blocks by a hash
    order = np.argsort(hash_u01(seed, TENSOR_PAGED_K, 9, np.arange(num_blocks, dtype=np.uint64)), kind="stable")
    block_table = np.full((num_seqs, max_blocks), -1, dtype=np.int32)
    pos = 0
    for s in range(num_seqs):
        n = int(blocks_per_seq[s])
        block_table[s, :n] = order[pos:pos + n]
        pos += n
    Q = matrix_bf16(num_seqs * H, D, seed=seed, tensor_id=TENSOR_PAGED_Q, kind="normal").reshape(num_seqs, H, D)
    Kc = matrix_bf16(num_blocks * H_kv * block_size, D, seed=seed, tensor_id=TENSOR_PAGED_K, kind="normal")
    Vc = matrix_bf16(num_blocks * H_kv * block_size, D, seed=seed, tensor_id=TENSOR_PAGED_V, kind="normal")
    shape = (num_blocks, H_kv, block_size, D)
    return Q, Kc.reshape(shape), Vc.reshape(shape), block_table, seq_lens


PAGED_CONFIGS = {
    # name: (num_seqs, H, H_kv, D, block_size, min_len, max_len, seed); the paper lists no decode shapes
    # sized so that the visible KV (0.2-0.3 GB) is larger than L2 and the generator stays within tens of seconds
    "paged_s16h8d128_len1k-8k": (16, 8, 8, 128, 16, 1024, 8192, 7),
    "paged_s2h8d128_len32k": (2, 8, 8, 128, 16, 30000, 32768, 8),
    "paged_s32h32kv4d128_len2k-4k": (32, 32, 4, 128, 16, 2048, 4096, 9),
}


def paged_bytes(seq_lens, H_kv: int, D: int) -> float:
    """Algorithmic HBM bytes of a decode step: every visible key and value read once (BF16)."""
    return float(np.asarray(seq_lens, dtype=np.int64).sum()) * H_kv * D * 2 * 2


GEMM_CONFIGS = {
    # name: (M, N, K, value kind, seed)
    "gemm_512": (512, 512, 512, "uniform", 0),
    "gemm_4096": (4096, 4096, 4096, "normal", 1),
    "gemm_8192x28672x4096": (8192, 28672, 4096, "normal", 2),
    "gemm_8192x4096x28672": (8192, 4096, 28672, "normal", 3),
}

# Memory-bound GEMM shapes (Sec. 4.1: next-token prediction; "large k" and "large n" cases; the paper lists none)
GEMM_DECODE_CONFIGS = {
    # name: (M, N, K, value kind, seed)
    "gemm_decode_16x4096x4096": (16, 4096, 4096, "normal", 11),
    "gemm_decode_16x28672x4096": (16, 28672, 4096, "normal", 12),
    "gemm_decode_16x4096x28672": (16, 4096, 28672, "normal", 13),
    "gemm_decode_64x8192x8192": (64, 8192, 8192, "normal", 14),
}

MHA_CONFIGS = {
    # name: (B, H, Nq, Nk, D, causal, seed, outlier_percent)
    "mha_b4h32n1024d64": (4, 32, 1024, 1024, 64, 0, 4, 0),
    "mha_b2h32n4096d128_causal": (2, 32, 4096, 4096, 128, 1, 5, 0),
    "mha_b1h16n16384d128_causal": (1, 16, 16384, 16384, 128, 1, 6, 1),
    "mha_b1h16n16384d128": (1, 16, 16384, 16384, 128, 0, 6, 1),
}


def gemm_flops(M: int, N: int, K: int) -> float:
    return 2.0 * M * N * K


def mha_flops(B: int, H: int, Nq: int, Nk: int, D: int, causal: int) -> float:
    """Convention: 4*B*H*Nq*Nk*D, halved when causal."""
    f = 4.0 * B * H * Nq * Nk * D
    return f * 0.5 if causal else f
