/*
 * mlt.h -- C ABI of the B200 (sm_100a) dense hot path: BF16 GEMM with FP32
 * accumulation and a FlashAttention-2 style multi-head-attention forward.
 *
 * Every pointer named "device" must be device memory of the CUDA device that
 * is current on the calling thread.  `stream` is a cudaStream_t passed as
 * void* (NULL = the legacy default stream).  All calls are asynchronous on
 * `stream`, allocate no device memory, keep no pointer after returning, and
 * return an mlt_status (never throw, never exit).  Argument validation runs
 * before any CUDA call.  Outputs must not alias inputs.
 *
 * BF16 values are passed as their 16-bit patterns.
 */
#ifndef MLT_H_
#define MLT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MLT_OK = 0,
    MLT_ERR_INVALID_ARG = 1, /* NULL pointer, negative size, pitch < row width, causal with Nq > Nk, Nk == 0, scale <= 0 */
    MLT_ERR_UNSUPPORTED = 2, /* head dimension other than 64 or 128; size beyond a TMA descriptor's range */
    MLT_ERR_ALIGNMENT = 3,   /* base pointer not 16-byte aligned, or pitch not a multiple of 8 elements */
    MLT_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed */
    MLT_ERR_ARCH = 5,        /* current device is not compute capability 10.x */
    MLT_ERR_TIMEOUT = 6,     /* a bounded device-side wait expired (reported by mlt_last_device_error) */
    MLT_ERR_BAD_BLOCK = 7,   /* a block-table entry outside [0, num_blocks) was met (reported by mlt_last_device_error) */
    MLT_ERR_SCRATCH_LIMIT = 8 /* mlt_paged_attn_decode_static: the call needs more than MLT_PAGED_STATIC_SCRATCH_BYTES */
} mlt_status;

/*
 * C = A * B  (paper Sec. 2: A in R^{m x k}, B in R^{k x n}, C in R^{m x n};
 * Listing 2: zero-initialised accumulator, K loop of tile dots, one store).
 * Reading taken: C is overwritten, its prior contents are ignored.
 *
 *   A  device, BF16, M x K row-major, A[i*lda + k]
 *   B  device, BF16, K x N row-major, B[k*ldb + j]
 *   C  device, BF16 out, M x N row-major, C[i*ldc + j]; products accumulate in
 *      FP32 and are rounded once, to nearest even
 *   lda, ldb, ldc  row pitches in ELEMENTS, each >= the row width and a multiple
 *      of 8 (16-byte rows for the TMA descriptors); base pointers 16-byte aligned
 *
 * M == 0 or N == 0: MLT_OK, nothing launched.  K == 0: C is zero-filled.
 * Any M, N, K otherwise (ragged tiles are zero-filled on load, clipped on store).
 */
int mlt_gemm(const void* A, const void* B, void* C,
             int64_t M, int64_t N, int64_t K,
             int64_t lda, int64_t ldb, int64_t ldc,
             void* stream);

/*
 * The GEMM in the data types of the paper's Listing 2 (FP16 operands, FP32 accumulator and FP32 result), with
 * the accumulate form of the problem statement of Sec. 2 (C += A * B) as an option.
 *
 *   A, B   device, FP16 (bit patterns), layouts and pitches as for mlt_gemm
 *   C      device, FP32, M x N row-major, pitch ldc in ELEMENTS, a multiple of 4; 16-byte aligned
 *   accumulate  0: C = A * B (prior contents ignored);  non-zero: C = C + A * B, the product summed in FP32 first
 *               and added to the prior C once
 * K == 0: C is zero-filled, or left as it is when accumulating.  Errors as for mlt_gemm.
 */
int mlt_gemm_f16(const void* A, const void* B, float* C,
                 int64_t M, int64_t N, int64_t K,
                 int64_t lda, int64_t ldb, int64_t ldc,
                 int accumulate, void* stream);

/*
 * mlt_gemm with caller-provided scratch, for the memory-bound shapes of paper Sec. 4.1 (next-token prediction:
 * few rows of A against large weight matrices, "large k" and "large n" cases).  Such a problem has too few output
 * tiles to occupy the GPU, so K is cut into slices (split-K) and every SM streams a part of B.  With at most one
 * 128 x 128 tile per two SMs the slices of a tile run as a thread-block cluster that sums its FP32 partial tiles
 * through distributed shared memory; this needs no scratch and mlt_gemm does the same.  With more tiles than that
 * the FP32 partial tiles go to the workspace and a second small kernel sums them.  Either way the sum runs in a
 * fixed order and is rounded once to BF16.  Same operation, arguments, layouts and errors as mlt_gemm; the result
 * can differ from an uncut sum in the last BF16 bit (the FP32 partial sums are added in a different order).
 *
 *   workspace        device scratch, 16-byte aligned, or NULL (then this is mlt_gemm)
 *   workspace_bytes  its size; mlt_gemm_workspace_bytes(M, N, K) is always enough (0 when K would not be cut; an
 *                    upper bound that does not depend on the device); with less, fewer slices are used.  Calls
 *                    that overlap on the GPU must not share it.
 */
size_t mlt_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K);
int mlt_gemm_ex(const void* A, const void* B, void* C,
                int64_t M, int64_t N, int64_t K,
                int64_t lda, int64_t ldb, int64_t ldc,
                void* workspace, size_t workspace_bytes, void* stream);

/*
 * O = softmax(scale * Q K^T [+ causal mask]) V,  LSE = log-sum-exp of the
 * scaled, masked scores (natural log)  -- paper Sec. 2.5, Algorithm 1
 * (FlashAttention-2 forward: per Q block, loop over K/V blocks, S = Q K_j^T,
 * online softmax with running row max m and row sum l, O += P V_j, store O).
 * The scale, the mask, the final 1/l and the LSE output are the benchmark
 * configuration's; the algorithm box leaves them implicit.
 *
 *   Q      device, BF16, [B, H, Nq, D] contiguous (D fastest)
 *   K, V   device, BF16, [B, H, Nk, D] contiguous
 *   O      device, BF16 out, [B, H, Nq, D]
 *   LSE    device, FP32 out, [B, H, Nq], or NULL to skip it
 *   D      64 or 128
 *   causal non-zero: key j is visible to query i iff j <= i + (Nk - Nq)
 *          (bottom-right aligned; requires Nq <= Nk)
 *   scale  multiplies the raw dot products (typically 1/sqrt(D)); must be finite and > 0
 *
 * B*H*Nq == 0: MLT_OK, nothing launched.  Nk == 0: MLT_ERR_INVALID_ARG.
 * P is rounded to BF16 for the second product; S, m, l and O accumulate in FP32.
 */
int mlt_mha_fwd(const void* Q, const void* K, const void* V,
                void* O, float* LSE,
                int B, int H, int Nq, int Nk, int D,
                int causal, float scale, void* stream);

/*
 * Paged-attention decode: O[s,h,:] = softmax(scale * q[s,h] . K_s^T) V_s over the len[s] tokens of sequence s,
 * whose keys and values live in cache blocks reached through a block table -- paper Sec. 3.2 (Listings 6 and 7:
 * one query token per sequence, KV blocks split across warps, cross-warp max / sum / output reduction) and
 * Sec. 4.3.  The listings are schematic (they normalise per block); the operation is plain softmax attention.
 *
 *   Q            device, BF16, [num_seqs, H, D]
 *   K_cache, V_cache  device, BF16, [num_blocks, H_kv, block_size, D] (D fastest)
 *   block_table  device, int32, [num_seqs, max_blocks_per_seq]: physical block of each logical block; entries of
 *                logical blocks a sequence uses must lie in [0, num_blocks) (others are never read; a bad entry is
 *                skipped and reported through mlt_last_device_error, it is never dereferenced)
 *   seq_lens     device, int32, [num_seqs], 0 <= len <= max_blocks_per_seq * block_size; token i sits in logical
 *                block i / block_size at offset i % block_size (a length outside that range is cut to it: no
 *                table entry beyond a sequence's row is read)
 *   O            device, BF16 out, [num_seqs, H, D];  LSE device FP32 out [num_seqs, H] (natural log) or NULL
 *   H_kv         KV heads; H / H_kv in {1, 2, 4, 8}; query head h reads KV head h / (H / H_kv)
 *   D in {64, 128}; block_size in {8, 16, 32}; scale finite and > 0
 *   workspace    device scratch of workspace_bytes bytes (16-byte aligned) for the partial results when a
 *                sequence is split over several CTAs; mlt_paged_attn_workspace_bytes gives a size that is always
 *                enough.  With less (or NULL) fewer splits are used, down to one CTA per (sequence, KV head).
 *                Its contents are scratch; calls that overlap on the GPU must not share it.
 * A sequence of length 0 gives O = 0 and LSE = -inf.  num_seqs == 0: MLT_OK, nothing launched.
 */
size_t mlt_paged_attn_workspace_bytes(int num_seqs, int H, int D);
int mlt_paged_attn_decode(const void* Q, const void* K_cache, const void* V_cache,
                          const int32_t* block_table, const int32_t* seq_lens,
                          void* O, float* LSE,
                          int num_seqs, int H, int H_kv, int D,
                          int block_size, int max_blocks_per_seq, int num_blocks, float scale,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * mlt_paged_attn_decode for callers that cannot supply scratch memory.  (The paper has no counterpart: this is a
 * library addition.)  Who needs it: an engine whose own pool already owns all device memory, a plug-in that
 * receives tensors but no allocator, a decode loop in which cudaMalloc -- it synchronises the device -- is ruled
 * out once the loop is running.  The partial results of split sequences go into an array of
 * MLT_PAGED_STATIC_SCRATCH_BYTES bytes that is part of the library's device image (every GPU that loads the
 * library carries it until the process exits).  The call allocates nothing, on host or device.
 *
 * Arguments, layouts, results and errors are those of mlt_paged_attn_decode, without the workspace pair.  The
 * split over CTAs is the one mlt_paged_attn_decode makes with a full workspace, so the outputs are the same;
 * it needs num_seqs * H * splits * (4 * D + 8) bytes with splits <= 32 (splits = ceil(max_blocks_per_seq / 16), / 32
 * with 4 or 8 query heads per KV head, half as many blocks per split for few sequences), and a call that needs more
 * than the array holds returns MLT_ERR_SCRATCH_LIMIT
 * and launches nothing.
 *
 * The first call on each device looks up the array's device address (with that device current); make that first
 * call before any stream capture begins.  All calls on a device share the one array and it keeps the last call's
 * contents: nothing in it has to be cleared between calls, but two calls that overlap on the GPU (different
 * streams, or one thread per stream) race on it -- serialise them, or use mlt_paged_attn_decode with separate
 * workspaces.
 */
#define MLT_PAGED_STATIC_SCRATCH_BYTES (16 * 1024 * 1024)
int mlt_paged_attn_decode_static(const void* Q, const void* K_cache, const void* V_cache,
                                 const int32_t* block_table, const int32_t* seq_lens,
                                 void* O, float* LSE,
                                 int num_seqs, int H, int H_kv, int D,
                                 int block_size, int max_blocks_per_seq, int num_blocks, float scale,
                                 void* stream);

/*
 * The SM clock the last GEMM (which = 0) or attention (which = 1) launch on the current device really ran at, in
 * MHz: CTA 0 of those kernels notes the SM cycle counter and the nanosecond timer at its start and at its end.  (No
 * counterpart in the paper; a measurement aid: under tensor-core load this part runs well below the clock NVML
 * reports, and throughput is only comparable across runs together with it.)  Synchronises the device.  *mhz is 0
 * if no such kernel has run yet.  Concurrent launches of the same kind overwrite each other's notes.
 */
int mlt_debug_last_clock_mhz(int which, double* mhz);

/*
 * The launch plan of mlt_gemm / mlt_gemm_ex for an M x N x K problem with BF16 output (no counterpart in the paper;
 * lets tests pin which kernel a shape reaches).  sm_count >= 2: a device of that many SMs on which clusters can use
 * every SM (host arithmetic only, no CUDA call).  sm_count == 0: the current device, with the number of resident
 * clusters it reports (a cluster must fit one GPC); configures the device on first use like any other call.
 *   out4[0]  tile shape: 0 = CTA pairs on 256 x 256 tiles, 1 = 128 x 256 tiles, 2 = 128 x 128 tiles, 3 = 128 x 128
 *            tiles with the even K hand-out through the workspace (every CTA the same number of (tile, K block)
 *            units; then out4[1] = the most partial tiles one output tile can get, out4[3] = units per CTA)
 *   out4[1]  K slices through the workspace (1 = none);  workspace_bytes = 0 stands for no workspace
 *   out4[2]  CTAs per cluster that cut K for one tile (1 = none)
 *   out4[3]  K blocks of 64 per slice
 * MLT_ERR_INVALID_ARG for a null pointer, a non-positive size, sm_count 1 or negative.
 */
int mlt_debug_gemm_plan(int64_t M, int64_t N, int64_t K, size_t workspace_bytes, int sm_count, int* out4);

/*
 * Device-side health word.  Kernels never trap: a wait that exceeds its bound
 * records {code, barrier id, block} in a per-device status word and the kernel
 * drains and returns.  This call synchronises the current device, reads and
 * clears that word, and returns MLT_OK, MLT_ERR_TIMEOUT, MLT_ERR_BAD_BLOCK or MLT_ERR_CUDA.
 * detail (host, may be NULL) receives 4 words: code, barrier id, block, aux.
 * (Library addition; the paper has no counterpart.)
 */
int mlt_last_device_error(uint32_t* detail);

/*
 * Self-test of the bounded device-side waits (library addition; the paper has no counterpart).  Launches one warp
 * that waits, with a budget of `budget_cycles` SM clocks (1 .. 1e9, i.e. at most about half a second), on a barrier
 * that nothing completes.  The wait gives up, the kernel returns normally, and the next mlt_last_device_error
 * reports MLT_ERR_TIMEOUT with detail = {code, barrier id 0x7E57, block 0, parity 0}.  Nothing traps; the context
 * stays usable.  Returns MLT_OK when the launch was made, MLT_ERR_INVALID_ARG for a budget outside the range.
 */
int mlt_debug_wait_timeout_selftest(uint64_t budget_cycles, void* stream);

/* Text for an mlt_status value (static storage). */
const char* mlt_status_string(int status);

/* Library version: major*10000 + minor*100 + patch. */
int mlt_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MLT_H_ */
