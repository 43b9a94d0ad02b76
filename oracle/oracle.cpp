// CPU oracle for the dense hot path: plain FP64 GEMM and naive three-pass
// softmax attention over BF16-rounded inputs.
//
// THIS IS TEST INFRASTRUCTURE.  Only the tests, the smoke check and the
// benchmark's cpu_baseline / reference legs may build, link or call it.  It
// shares no code with the CUDA path and is deliberately slow and literal so a
// reader can check it against the paper by eye.
//
// What it follows:
//  * GEMM: the problem statement of Sec. 2 (A in R^{m x k}, B in R^{k x n},
//    C in R^{m x n}) and the loop of Listing 2 (zero accumulator, sum over k of
//    A-tile times B-tile, store).  Reading taken: C = A*B (the listing stores
//    the loop result; prior C contents are ignored).
//  * MHA forward: Algorithm 1 (FlashAttention-2 forward) computes exact softmax
//    attention; the oracle is that definition written out per query row in three
//    passes (scores and their max; exponentials and their sum; weighted sum of
//    V), with the scale, causal mask, 1/l normalisation and log-sum-exp output
//    the algorithm box leaves implicit.
//
// Inputs are BF16 bit patterns (uint16).  BF16 -> double is exact and every
// product of two BF16 values is exact in double, so the only rounding is in the
// FP64 summations.  Outputs stay in FP64 (never rounded to BF16).
//
// Paged-attention decode (Sec. 3.2 / 4.3) is the same definition over keys gathered through a block table.  The
// paper's Listings 6 and 7 are schematic (they normalise per block and state no shapes or layouts): that the
// operation is plain softmax attention of one query token, and the cache layout, are readings -- parity unpinned
// by the paper for them; the function is pinned to the attention oracle above on the gathered tokens.
//
// FP16-operand GEMM with optional prior C (Listing 2 data types; C += A*B of the Sec. 2 problem statement): the
// same sum over binary16 values (conversion written out field by field, checked against all 65536 patterns), the
// prior C added after the sum.
//
// Pins (see tests/test_oracle_*.py): identity / permutation / all-ones /
// single-non-zero / K-split additivity / exact rational brute force for GEMM;
// constant-K mean-of-V, causal row 0, Nk = 1, rows summing to one, key
// permutation invariance, split-merge identity, shift invariance, dominant key,
// independent brute force for attention.  The causal alignment for Nq != Nk
// (bottom-right) is a convention the paper does not state: parity unpinned by
// the paper for that case.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

inline double bf16_to_double(uint16_t bits) {
    uint32_t w = static_cast<uint32_t>(bits) << 16;
    float f;
    std::memcpy(&f, &w, sizeof f);
    return static_cast<double>(f);
}

// IEEE 754 binary16 -> double, from the bit fields: 1 sign, 5 exponent (bias 15), 10 fraction bits.
//   e = 0      : (-1)^s * f * 2^-24            (zero and subnormals)
//   e = 1..30  : (-1)^s * (1024 + f) * 2^(e-25)
//   e = 31     : infinity (f = 0) or NaN
inline double f16_to_double(uint16_t bits) {
    const int s = bits >> 15, e = (bits >> 10) & 31, f = bits & 1023;
    double v;
    if (e == 0) v = std::ldexp(static_cast<double>(f), -24);
    else if (e == 31) v = f ? std::numeric_limits<double>::quiet_NaN() : std::numeric_limits<double>::infinity();
    else v = std::ldexp(static_cast<double>(1024 + f), e - 25);
    return s ? -v : v;
}

template <class F>
void parallel_for(int64_t n, int nthreads, F&& body) {
    if (nthreads <= 0) nthreads = static_cast<int>(std::thread::hardware_concurrency());
    if (nthreads < 1) nthreads = 1;
    if (n < nthreads) nthreads = static_cast<int>(std::max<int64_t>(n, 1));
    if (nthreads == 1) {
        for (int64_t i = 0; i < n; ++i) body(i);
        return;
    }
    std::vector<std::thread> pool;
    pool.reserve(nthreads);
    for (int t = 0; t < nthreads; ++t)
        pool.emplace_back([&, t] {
            for (int64_t i = t; i < n; i += nthreads) body(i);
        });
    for (auto& th : pool) th.join();
}

}  // namespace

extern "C" {

int oracle_hardware_threads(void) {
    int n = static_cast<int>(std::thread::hardware_concurrency());
    return n < 1 ? 1 : n;
}

// C_out[r][j] = sum_{k<K} A[rows[r]][k] * B[k][j]      (Sec. 2, Listing 2)
//
// A: M x K row-major, pitch lda (elements); B: K x N row-major, pitch ldb.
// rows: nrows row indices of C to compute, or NULL for all M rows (nrows
// ignored).  C_out: dense (nrows or M) x N doubles.  Returns 0, or 1 on a bad
// argument.
int oracle_gemm(const uint16_t* A, const uint16_t* B, double* C_out,
                int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb,
                const int64_t* rows, int64_t nrows, int nthreads) {
    if (M < 0 || N < 0 || K < 0 || lda < K || ldb < N) return 1;
    const int64_t R = rows ? nrows : M;
    if (rows)
        for (int64_t r = 0; r < R; ++r)
            if (rows[r] < 0 || rows[r] >= M) return 1;
    parallel_for(R, nthreads, [&](int64_t r) {
        const int64_t i = rows ? rows[r] : r;
        double* c = C_out + r * N;
        for (int64_t j = 0; j < N; ++j) c[j] = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            const double a = bf16_to_double(A[i * lda + k]);
            const uint16_t* b = B + k * ldb;
            for (int64_t j = 0; j < N; ++j) c[j] += a * bf16_to_double(b[j]);
        }
    });
    return 0;
}

// out[i] = value of the binary16 pattern in[i]  (test access to the conversion the FP16 GEMM uses).
int oracle_f16_to_double(const uint16_t* in, double* out, int64_t n) {
    if (n < 0) return 1;
    for (int64_t i = 0; i < n; ++i) out[i] = f16_to_double(in[i]);
    return 0;
}

// C_out[r][j] = (C_in ? C_in[rows[r]][j] : 0) + sum_{k<K} A[rows[r]][k] * B[k][j]
//
// The GEMM in the data types of Listing 2 (FP16 operands) with the accumulate form of Sec. 2 (C += A * B).
// A, B: binary16 bit patterns, layouts as in oracle_gemm.  C_in: NULL, or the prior C as FP32, M x N row-major with
// pitch ldc.  The product is summed first (k ascending) and the prior C added last.  rows / C_out as in oracle_gemm.
int oracle_gemm_f16(const uint16_t* A, const uint16_t* B, const float* C_in, double* C_out,
                    int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb, int64_t ldc,
                    const int64_t* rows, int64_t nrows, int nthreads) {
    if (M < 0 || N < 0 || K < 0 || lda < K || ldb < N || (C_in && ldc < N)) return 1;
    const int64_t R = rows ? nrows : M;
    if (rows)
        for (int64_t r = 0; r < R; ++r)
            if (rows[r] < 0 || rows[r] >= M) return 1;
    parallel_for(R, nthreads, [&](int64_t r) {
        const int64_t i = rows ? rows[r] : r;
        double* c = C_out + r * N;
        for (int64_t j = 0; j < N; ++j) c[j] = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            const double a = f16_to_double(A[i * lda + k]);
            const uint16_t* b = B + k * ldb;
            for (int64_t j = 0; j < N; ++j) c[j] += a * f16_to_double(b[j]);
        }
        if (C_in)
            for (int64_t j = 0; j < N; ++j) c[j] += static_cast<double>(C_in[i * ldc + j]);
    });
    return 0;
}

// Exact softmax attention for selected query rows (Algorithm 1, written as the
// definition it reaches).
//
// Q: [B,H,Nq,D], K,V: [B,H,Nk,D], contiguous, D fastest, BF16 bits.
// qrows: nrows flat query indices (b*H + h)*Nq + i, or NULL for all B*H*Nq.
// O_out: nrows x D doubles; LSE_out: nrows doubles (natural log); P_out: NULL,
// or nrows x Nk doubles receiving the normalised probabilities (0 where masked).
// Key j is visible to query i iff j < Nk and (not causal or j <= i + (Nk - Nq)).
//   pass 1: s_j = scale * sum_d Q[i][d] K[j][d] for visible j;  m = max_j s_j
//   pass 2: e_j = exp(s_j - m);  l = sum_j e_j
//   pass 3: O[i][d] = sum_j (e_j / l) V[j][d];  LSE[i] = m + ln l
// `scale` is the FP32 value the GPU entry point receives, widened to double.
int oracle_mha_fwd(const uint16_t* Q, const uint16_t* K, const uint16_t* V,
                   double* O_out, double* LSE_out, double* P_out,
                   int B, int H, int Nq, int Nk, int D, int causal, float scale,
                   const int64_t* qrows, int64_t nrows, int nthreads) {
    if (B < 0 || H < 0 || Nq < 0 || Nk < 1 || D < 1) return 1;
    if (causal && Nq > Nk) return 1;
    const int64_t total = static_cast<int64_t>(B) * H * Nq;
    const int64_t R = qrows ? nrows : total;
    if (qrows)
        for (int64_t r = 0; r < R; ++r)
            if (qrows[r] < 0 || qrows[r] >= total) return 1;
    const double sc = static_cast<double>(scale);
    parallel_for(R, nthreads, [&](int64_t r) {
        const int64_t flat = qrows ? qrows[r] : r;
        const int64_t bh = flat / Nq;
        const int64_t i = flat % Nq;
        const uint16_t* q = Q + flat * D;
        const uint16_t* Kh = K + bh * Nk * D;
        const uint16_t* Vh = V + bh * Nk * D;
        const int64_t visible = causal ? std::min<int64_t>(Nk, i + (Nk - Nq) + 1) : Nk;
        std::vector<double> s(static_cast<size_t>(visible));
        std::vector<double> qd(static_cast<size_t>(D));
        for (int d = 0; d < D; ++d) qd[d] = bf16_to_double(q[d]);
        // pass 1
        double m = -std::numeric_limits<double>::infinity();
        for (int64_t j = 0; j < visible; ++j) {
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += qd[d] * bf16_to_double(Kh[j * D + d]);
            s[j] = sc * dot;
            m = std::max(m, s[j]);
        }
        // pass 2
        double l = 0.0;
        for (int64_t j = 0; j < visible; ++j) {
            s[j] = std::exp(s[j] - m);
            l += s[j];
        }
        // pass 3
        double* o = O_out + r * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        for (int64_t j = 0; j < visible; ++j) {
            const double p = s[j] / l;
            for (int d = 0; d < D; ++d) o[d] += p * bf16_to_double(Vh[j * D + d]);
        }
        LSE_out[r] = m + std::log(l);
        if (P_out) {
            double* p = P_out + r * Nk;
            for (int64_t j = 0; j < Nk; ++j) p[j] = j < visible ? s[j] / l : 0.0;
        }
    });
    return 0;
}

// Paged-attention decode (Sec. 3.2 and 4.3: one query token per sequence, the request's keys and values live
// in fixed-size cache blocks reached through a block table; Listing 6 gives the per-block loop, which reaches
// plain softmax attention over the sequence's tokens).  Written as the definition: gather the sequence's keys and
// values through the table, then the same three passes as oracle_mha_fwd with a single query row.
//
// Q: [num_seqs, H, D]; K_cache, V_cache: [num_blocks, H_kv, block_size, D] (D fastest), BF16 bits.
// block_table: [num_seqs, max_blocks] physical block of logical block b of a sequence; seq_lens: [num_seqs].
// Query head h reads KV head h / (H / H_kv).  Token i of a sequence sits in logical block i / block_size at
// offset i % block_size.  O_out: [num_seqs, H, D] doubles; LSE_out: [num_seqs, H] (natural log).
// A sequence of length 0 gives O = 0 and LSE = -inf.  Returns 0, or 1 on a bad argument.
int oracle_paged_attn_decode(const uint16_t* Q, const uint16_t* K_cache, const uint16_t* V_cache,
                             const int32_t* block_table, const int32_t* seq_lens, double* O_out, double* LSE_out,
                             int num_seqs, int H, int H_kv, int D, int block_size, int max_blocks, int num_blocks,
                             float scale, int nthreads) {
    if (num_seqs < 0 || H < 1 || H_kv < 1 || H % H_kv != 0 || D < 1 || block_size < 1 || max_blocks < 0) return 1;
    for (int s = 0; s < num_seqs; ++s) {
        if (seq_lens[s] < 0 || seq_lens[s] > static_cast<int64_t>(max_blocks) * block_size) return 1;
        const int used = (seq_lens[s] + block_size - 1) / block_size;
        for (int b = 0; b < used; ++b)
            if (block_table[static_cast<int64_t>(s) * max_blocks + b] < 0 ||
                block_table[static_cast<int64_t>(s) * max_blocks + b] >= num_blocks)
                return 1;
    }
    const double sc = static_cast<double>(scale);
    const int group = H / H_kv;
    parallel_for(static_cast<int64_t>(num_seqs) * H, nthreads, [&](int64_t r) {
        const int s = static_cast<int>(r / H), h = static_cast<int>(r % H), kvh = h / group;
        const int len = seq_lens[s];
        const uint16_t* q = Q + r * D;
        auto row = [&](const uint16_t* cache, int i) {
            const int64_t blk = block_table[static_cast<int64_t>(s) * max_blocks + i / block_size];
            return cache + ((blk * H_kv + kvh) * block_size + i % block_size) * D;
        };
        std::vector<double> e(static_cast<size_t>(len));
        double m = -std::numeric_limits<double>::infinity();
        for (int i = 0; i < len; ++i) {  // pass 1: scores and their max
            const uint16_t* k = row(K_cache, i);
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += bf16_to_double(q[d]) * bf16_to_double(k[d]);
            e[i] = sc * dot;
            m = std::max(m, e[i]);
        }
        double l = 0.0;
        for (int i = 0; i < len; ++i) {  // pass 2: exponentials and their sum
            e[i] = std::exp(e[i] - m);
            l += e[i];
        }
        double* o = O_out + r * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        for (int i = 0; i < len; ++i) {  // pass 3: weighted sum of the values
            const uint16_t* v = row(V_cache, i);
            const double p = e[i] / l;
            for (int d = 0; d < D; ++d) o[d] += p * bf16_to_double(v[d]);
        }
        LSE_out[r] = len > 0 ? m + std::log(l) : -std::numeric_limits<double>::infinity();
    });
    return 0;
}

}  // extern "C"
