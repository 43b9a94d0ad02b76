// Paged-attention decode (paper Sec. 3.2, Listings 6-7, and Sec. 4.3): one query token per sequence attends
// to the sequence's keys and values, which live in fixed-size cache blocks reached through a block table.  As in
// the paper's warp-level kernel the KV blocks of a sequence are split across warps (and here also across CTAs,
// flash-decoding style), each keeps a partial running max / sum / output, and the partials are reduced at the end.
//
// The work is bound by HBM: every visible key and value is read once (2 * len * H_kv * D * 2 bytes per sequence)
// and used for 2 * G multiply-adds per element, so there are no tensor cores here; the kernel is laid out for
// coalesced 16-byte loads with many loads in flight per warp.
//   grid  = (splits, H_kv, num_seqs), 128 threads (4 warps)
//   warp  = KV blocks b0 + w, b0 + w + 4, ... of its split; for one block it first issues all K and V loads
//           (16 bytes per lane, D/8 lanes per token, 32 / (D/8) tokens per load instruction), then the dot
//           products (shuffle reduction inside the D/8 lanes of a token), one online-softmax update per block,
//           and the P V accumulation; each lane keeps 8 output columns for each of the G query heads that
//           share the KV head
//   end   = lane groups merge by shuffles, warps merge through shared memory, and the CTA writes O and LSE
//           (single split) or an unnormalised partial {m, l, o[D]} to the workspace, which a second small
//           kernel combines.
#pragma once

#include <math.h>

#include <algorithm>

#include "ptx.cuh"

namespace mlt {

constexpr int kPagedThreads = 128;
constexpr int kPagedWarps = kPagedThreads / 32;
constexpr int kPagedMaxSplits = 32;
constexpr unsigned int kStatusBadBlock = 7;  // a block-table entry outside [0, num_blocks)

struct PagedParams {
    const __nv_bfloat16* Q;        // [num_seqs, H, D]
    const __nv_bfloat16* K_cache;  // [num_blocks, H_kv, block_size, D]
    const __nv_bfloat16* V_cache;
    const int* block_table;        // [num_seqs, max_blocks]
    const int* seq_lens;           // [num_seqs]
    __nv_bfloat16* O;              // [num_seqs, H, D]
    float* LSE;                    // [num_seqs, H] or null
    float* part_o;                 // [num_seqs, H, splits, D]   (splits > 1)
    float2* part_ml;               // [num_seqs, H, splits] {m in log2 units, l}
    int num_seqs, H, H_kv, block_size, max_blocks, num_blocks;
    int splits;            // CTAs per (sequence, KV head) = grid.x
    int blocks_per_split;  // KV blocks each of them covers: the same for every sequence, so CTAs do equal work and
                           // the CTAs beyond a short sequence's end exit at once
    float scale_log2e;
    int head_groups;       // CTAs per KV head (1, or 2 when 8 query heads per KV head run as two groups of 4)
    int balanced;          // grouped-head kernel: equal work per CTA (see paged_decode_mma_kernel); splits = kPagedMaxSplits
    int balanced_ctas;     // ... and the grid it is launched with (the combine kernel repeats the arithmetic)
};

__device__ __forceinline__ void bf16x8_to_f32(const uint4& v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

__device__ __forceinline__ void bf16x8_to_f32x2(const uint4& v, float2 (&f)[4]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) f[i] = make_float2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
}

// merge partial {m, l, o} states a and b (log2-domain maxima); -inf maxima stand for "nothing seen"
__device__ __forceinline__ void paged_merge_scale(float ma, float mb, float& m, float& sa, float& sb) {
    m = fmaxf(ma, mb);
    sa = (ma == -INFINITY) ? 0.0f : fast_exp2(ma - m);
    sb = (mb == -INFINITY) ? 0.0f : fast_exp2(mb - m);
}

// Sum over the LPT lanes of a token of G partial dot products, scattered: every stage halves the number of values
// a lane carries (lanes with the stage's bit clear keep the lower half of their list, the others the upper half)
// until one is left, so G heads cost G - 1 + log2(LPT / G) shuffles instead of G * log2(LPT).  Returns the complete
// sum of head paged_my_head(sub); lanes whose `sub` agree in the low log2(G) bits hold the same head.
template <int G, int LPT>
__device__ __forceinline__ float paged_reduce_scatter(float (&d)[G], int sub) {
    int n = G;
#pragma unroll
    for (int mask = 1; mask < LPT; mask <<= 1) {
        if (n > 1) {
            const int half = n / 2;
            const bool upper = (sub & mask) != 0;
#pragma unroll
            for (int j = 0; j < G / 2; ++j) {
                if (j < half) {
                    const float send = upper ? d[j] : d[j + half];
                    const float keep = upper ? d[j + half] : d[j];
                    d[j] = keep + __shfl_xor_sync(0xffffffffu, send, mask);
                }
            }
            n = half;
        } else {
            d[0] += __shfl_xor_sync(0xffffffffu, d[0], mask);
        }
    }
    return d[0];
}
template <int G>
__device__ __forceinline__ int paged_my_head(int sub) {  // the head whose sum paged_reduce_scatter leaves in this lane
    int g = 0, half = G / 2;
    for (int mask = 1; half > 0; mask <<= 1, half >>= 1)
        if (sub & mask) g += half;
    return g;
}
template <int G>
__device__ __forceinline__ int paged_head_sub(int g) {  // the lowest `sub` that holds head g
    int sub = 0, half = G / 2;
    for (int mask = 1; half > 0; mask <<= 1, half >>= 1)
        if (g & half) sub |= mask;
    return sub;
}

template <int D, int G, int BS>
__global__ void __launch_bounds__(kPagedThreads)
paged_decode_kernel(const PagedParams p) {
    pdl_launch_dependents();  // the combine kernel's CTAs take the slots this grid's CTAs leave, and do their prologue early
    constexpr int LPT = D / 8;         // lanes per token
    constexpr int TPS = 32 / LPT;      // tokens per load instruction of a warp
    constexpr int STEPS = BS / TPS;    // load instructions per block and tensor
    static_assert(BS % TPS == 0, "block size must be a multiple of the tokens per warp step");
    __shared__ float sm_o[kPagedWarps][G][D];
    __shared__ float2 sm_ml[kPagedWarps][G];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // blockIdx.y = KV head x head group: with more query heads per KV head than G, several CTAs share a KV head
    // (p.head_groups of them, G heads each; the second reads K and V from L2)
    const int sp = blockIdx.x, kvh = blockIdx.y / p.head_groups, s = blockIdx.z;
    const int head0 = kvh * (G * p.head_groups) + (blockIdx.y % p.head_groups) * G;  // first query head of this CTA
    const int sub = lane % LPT;   // which 8 columns of D this lane owns
    const int grp = lane / LPT;   // which token of a step
    // a length beyond what the block table can reach is cut at the table's end: no entry past the row is read
    const int len = max(0, min(p.seq_lens[s], p.max_blocks * BS));
    const int nblk = (len + BS - 1) / BS;
    const int b0 = sp * p.blocks_per_split;
    const int b1 = min(nblk, b0 + p.blocks_per_split);
    if (p.splits > 1 && b0 >= nblk && !(sp == 0)) return;  // nothing of this sequence here (split 0 reports an empty one)

    // this lane's 8 columns of the G query rows
    float2 q[G][4];  // pairs: the products below are packed (fma.rn.f32x2), two columns per instruction
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const uint4 v = *reinterpret_cast<const uint4*>(p.Q + (static_cast<int64_t>(s) * p.H + head0 + g) * D + sub * 8);
        bf16x8_to_f32x2(v, q[g]);
    }
    // Running max and sum are kept for one head per lane (the head whose scores the scattered reduction leaves
    // here); the output accumulators cover this lane's 8 columns of all G heads.
    const int my_g = paged_my_head<G>(sub);
    float m_own = -INFINITY, l_own = 0.0f;
    float2 o[G][4];
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int e = 0; e < 4; ++e) o[g][e] = make_float2(0.0f, 0.0f);
    }
    (void)my_g;

    const int* table = p.block_table + static_cast<int64_t>(s) * p.max_blocks;
    for (int b = b0 + warp; b < b1; b += kPagedWarps) {
        const int phys = table[b];
        if (phys < 0 || phys >= p.num_blocks) {  // never dereference a bad table entry: report and skip the block
            if (lane == 0 && atomicCAS(&g_status[0], 0u, kStatusBadBlock) == 0u) {
                g_status[1] = static_cast<unsigned int>(b);
                g_status[2] = static_cast<unsigned int>(s);
                g_status[3] = static_cast<unsigned int>(phys);
            }
            continue;
        }
        const int64_t base = ((static_cast<int64_t>(phys) * p.H_kv + kvh) * BS) * D + sub * 8;
        const __nv_bfloat16* kp = p.K_cache + base;
        const __nv_bfloat16* vp = p.V_cache + base;
        uint4 kr[STEPS], vr[STEPS];
#pragma unroll
        for (int i = 0; i < STEPS; ++i) kr[i] = *reinterpret_cast<const uint4*>(kp + (i * TPS + grp) * D);
#pragma unroll
        for (int i = 0; i < STEPS; ++i) vr[i] = *reinterpret_cast<const uint4*>(vp + (i * TPS + grp) * D);
        // score of this lane's head for each of the lane group's STEPS tokens (log2 domain), masked beyond the length
        float sc[STEPS];
#pragma unroll
        for (int i = 0; i < STEPS; ++i) {
            float2 kf[4];
            bf16x8_to_f32x2(kr[i], kf);
            const bool visible = b * BS + i * TPS + grp < len;
            float d[G];
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float2 d2 = make_float2(0.0f, 0.0f);
#pragma unroll
                for (int e = 0; e < 4; ++e) d2 = ffma2(q[g][e], kf[e], d2);
                d[g] = d2.x + d2.y;
            }
            const float dot = paged_reduce_scatter<G, LPT>(d, sub);
            sc[i] = visible ? dot * p.scale_log2e : -INFINITY;
        }
        // one online-softmax update per block, for this lane's head: one exponential per (head, token) and lane
        float pw[STEPS];
        float alpha;
        {
            float mb = sc[0];
#pragma unroll
            for (int i = 1; i < STEPS; ++i) mb = fmaxf(mb, sc[i]);
            const float mn = fmaxf(m_own, mb);
            alpha = (m_own == -INFINITY) ? 0.0f : fast_exp2(m_own - mn);
            const float ref = (mn == -INFINITY) ? 0.0f : mn;
            float sum = 0.0f;
#pragma unroll
            for (int i = 0; i < STEPS; ++i) {
                pw[i] = fast_exp2(sc[i] - ref);
                sum += pw[i];
            }
            m_own = mn;
            l_own = l_own * alpha + sum;
        }
        // rescale and accumulate all heads' outputs: the factors come from the lanes that hold each head
        const int lane0 = grp * LPT;  // first lane of this token group
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float ag = G == 1 ? alpha : __shfl_sync(0xffffffffu, alpha, lane0 + paged_head_sub<G>(g));
#pragma unroll
            for (int e = 0; e < 4; ++e) o[g][e] = make_float2(o[g][e].x * ag, o[g][e].y * ag);
        }
#pragma unroll
        for (int i = 0; i < STEPS; ++i) {
            float2 vf[4];
            // bytes past the sequence's last token are whatever the cache holds: weight 0 must not meet a NaN
            if (b * BS + i * TPS + grp >= len) vr[i] = make_uint4(0u, 0u, 0u, 0u);
            bf16x8_to_f32x2(vr[i], vf);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float pg = G == 1 ? pw[i] : __shfl_sync(0xffffffffu, pw[i], lane0 + paged_head_sub<G>(g));
                const float2 pg2 = make_float2(pg, pg);
#pragma unroll
                for (int e = 0; e < 4; ++e) o[g][e] = ffma2(pg2, vf[e], o[g][e]);
            }
        }
    }

    // every lane needs all heads' running max and sum for the merges below
    float m[G], l[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const int src = (lane / LPT) * LPT + paged_head_sub<G>(g);
        m[g] = G == 1 ? m_own : __shfl_sync(0xffffffffu, m_own, src);
        l[g] = G == 1 ? l_own : __shfl_sync(0xffffffffu, l_own, src);
    }

    // merge the TPS lane groups of the warp (lanes that own the same columns), then the warps through smem
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int w = LPT; w < 32; w <<= 1) {
            const float mo = __shfl_xor_sync(0xffffffffu, m[g], w);
            const float lo = __shfl_xor_sync(0xffffffffu, l[g], w);
            float mn, sa, sb;
            paged_merge_scale(m[g], mo, mn, sa, sb);
            l[g] = l[g] * sa + lo * sb;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float ox = __shfl_xor_sync(0xffffffffu, o[g][e].x, w);
                const float oy = __shfl_xor_sync(0xffffffffu, o[g][e].y, w);
                o[g][e] = make_float2(o[g][e].x * sa + ox * sb, o[g][e].y * sa + oy * sb);
            }
            m[g] = mn;
        }
        if (grp == 0) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                sm_o[warp][g][sub * 8 + 2 * e] = o[g][e].x;
                sm_o[warp][g][sub * 8 + 2 * e + 1] = o[g][e].y;
            }
            if (sub == 0) sm_ml[warp][g] = make_float2(m[g], l[g]);
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < G * D; idx += kPagedThreads) {
        const int g = idx / D, d = idx % D;
        float mt = -INFINITY;
#pragma unroll
        for (int w = 0; w < kPagedWarps; ++w) mt = fmaxf(mt, sm_ml[w][g].x);
        float lt = 0.0f, ot = 0.0f;
#pragma unroll
        for (int w = 0; w < kPagedWarps; ++w) {
            const float2 ml = sm_ml[w][g];
            const float sw = (ml.x == -INFINITY) ? 0.0f : fast_exp2(ml.x - mt);
            lt += ml.y * sw;
            ot += sm_o[w][g][d] * sw;
        }
        const int64_t row = static_cast<int64_t>(s) * p.H + head0 + g;
        if (p.splits == 1) {
            p.O[row * D + d] = __float2bfloat16(lt > 0.0f ? ot / lt : 0.0f);
            if (d == 0 && p.LSE) p.LSE[row] = lt > 0.0f ? (mt + log2f(lt)) * 0.6931471805599453f : -INFINITY;
        } else {
            p.part_o[(row * p.splits + sp) * D + d] = ot;
            if (d == 0) p.part_ml[row * p.splits + sp] = make_float2(mt, lt);
        }
    }
}

// ---------------------------------------------------------------------------------------------------------
// Grouped heads (4 or 8 query heads per KV head) on the tensor cores.
//
// With G query heads reading the same keys and values, the FP32-pipe kernel above spends G times the
// instructions per byte and runs out of issue slots long before HBM is busy (8 heads: 0.38 of the copy
// bandwidth).  Here the G heads are the rows of a warp-level MMA (mma.sync m16n8k16, rows G..15 are zero):
//   scores  S[16 x 16 tokens] = Q[16 x D] K^T   (2 column tiles of 8 tokens, D/16 steps)
//   output  O[16 x D]        += P[16 x 16 tokens] V   (D/8 column tiles, one step)
// per unit of 16 tokens and warp: 32 MMAs at D = 128 instead of about 500 packed FMAs.  K and V rows go from global
// memory into a per-warp shared-memory ring by bulk copies and from there into the B fragments as they are, with
// 16-byte loads and no transposes:
//  * the order of the summation index of an MMA is free as long as both operands use the same order, and so is
//    the order of its output columns.  For Q K^T the 16 index slots of two consecutive steps are mapped to the 8
//    consecutive elements of D a lane loads (lane (g, tg): elements pp*32 + tg*8 .. +7 of token column g), for Q and
//    K alike.  The 8 output columns of score tile e are mapped to tokens 4*(c/2) + c%2 + 2e, so that lane (g, tg)
//    ends up with the scores of head g for the 4 consecutive tokens 4 tg .. 4 tg + 3;
//  * for P V the index slots 2tg, 2tg+1, 2tg+8, 2tg+9 of a lane are exactly those 4 tokens, so the score
//    accumulators, exponentiated and packed, ARE the A fragment.  Output column n of tile (h, nt) is mapped to
//    element h*64 + n*8 + nt of D: lane (g, tg) loads 8 consecutive elements (16 bytes) of each of its 4 tokens and
//    pairs the same element of two tokens into one register with a byte permute.
// Splits, partial format and the combine kernel are those of the kernel above.
// ---------------------------------------------------------------------------------------------------------
// Units of 16 tokens per warp in the shared-memory ring (one being used, one in flight), and CTAs per SM the
// grouped-head kernel is compiled for (168 registers).  Measured (32 / 128 sequences, H = 32, H_kv = 4, 2k-4k
// tokens): ring 2 with 3 CTAs per SM 50 / 155 us; ring 3 with 2 CTAs 52 / 169; ring 4 with 2 CTAs 67 / 237; ring 2
// with 4 CTAs (128 registers) 56 / 171.
constexpr int kPagedRing = 2;
constexpr int kPagedMmaCtasPerSm = 3;
// A unit in shared memory: 16 K rows then 16 V rows of D BF16 each, as they lie in the cache (one bulk copy per
// tensor and cache block).  The fragment loads meet 2-way (K) and 4-way (V) bank conflicts; the load/store unit has
// the room (a quarter busy without them), and copies of single padded rows were far slower (256-byte bulk copies:
// 1.8-2.1 TB/s).
template <int D>
struct PagedRow {
    static constexpr int kPitch = D * 2;
};
template <int D>
constexpr size_t paged_mma_smem_bytes() {
    return static_cast<size_t>(kPagedWarps) * kPagedRing * 32 * PagedRow<D>::kPitch + 128;
}
// global -> shared bulk copy of `bytes` (a multiple of 16, both addresses 16-byte aligned), completion counted on `bar`
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Equal work per CTA (p.balanced): the live chunks of kPagedChunkTokens tokens of all (sequence, KV head) rows, in
// the order sequence, KV head, chunk, are numbered 0 .. n-1 and CTA c takes numbers c*q .. (c+1)*q - 1, whatever
// rows they belong to; it writes one partial per row it touches, into slot c - (first CTA of that row).  The numbers
// come from seq_lens, which only the device knows: every CTA scans them itself.  q is at least n / gridDim.x and at
// least a 30th of the longest row, so that no row has more than kPagedMaxSplits partials.
constexpr int kPagedChunkTokens = 128;
constexpr int kPagedBalanceMaxSeqs = 1024;  // the scan's shared-memory table; beyond it the static split is used
__device__ __forceinline__ int paged_chunks(const PagedParams& p, int s) {
    const int len = max(0, min(p.seq_lens[s], p.max_blocks * p.block_size));
    return (len + kPagedChunkTokens - 1) / kPagedChunkTokens;
}
__device__ __forceinline__ int paged_quota(long long n, int max_row, int ctas) {
    const long long q = max(max((n + ctas - 1) / ctas, static_cast<long long>((max_row + 29) / 30)), 1ll);
    return static_cast<int>(q);
}

template <int D, int G, int BS>
__global__ void __launch_bounds__(kPagedThreads, kPagedMmaCtasPerSm)
paged_decode_mma_kernel(const PagedParams p) {
    pdl_launch_dependents();  // the combine kernel's CTAs take the slots this grid's CTAs leave, and do their prologue early
    static_assert(G == 4 || G == 8, "rows of the MMA: 4 or 8 query heads");
    constexpr int PP = D / 32;  // pairs of 16-element steps of Q K^T
    constexpr int HV = D / 64;  // halves of D in the P V output mapping
    constexpr int NB = BS >= 16 ? 1 : 16 / BS;  // cache blocks per unit of 16 tokens
    __shared__ float2 sm_ml[kPagedWarps][G];
    __shared__ int sm_pre[kPagedBalanceMaxSeqs + 1];  // balanced: chunks of all sequences before s
    __shared__ int sm_red[2 * kPagedWarps];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tg = lane & 3;  // MMA fragment coordinates: row / column group, position in the group

    // K and V travel global -> shared by bulk copies (the TMA engine: no address generation, no load/store-unit
    // queue entries in the SM; with per-lane 16-byte cp.async the same ring streamed 4.3-4.6 TB/s at best), one copy
    // per tensor and cache block (a unit of 16 tokens is one block, half a block, or two blocks).  Each warp has its
    // own ring of kPagedRing units and one mbarrier per ring stage.
    constexpr int kPitch = PagedRow<D>::kPitch;
    constexpr int kUnitBytes = 32 * kPitch;
    extern __shared__ uint8_t paged_ring_raw[];
    uint8_t* ring_base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(paged_ring_raw) + 127) & ~uintptr_t(127));
    uint8_t* my_ring = ring_base + static_cast<size_t>(warp) * kPagedRing * kUnitBytes;
    __shared__ uint64_t ring_bar[kPagedWarps][kPagedRing];
    __shared__ uint32_t ring_abort;
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < kPagedRing; ++i) mbar_init(&ring_bar[warp][i], 1);
        if (warp == 0) ring_abort = 0;
        fence_mbar_init();
    }

    // ---- which segments (row, token range, partial slot) this CTA works on ----
    int seg_s, seg_kvh, seg_tok_begin, seg_tok_end, seg_slot;
    long long bal_i = 0, bal_hi = 0;  // balanced: next live chunk number, end of this CTA's numbers
    int bal_q = 1;
    if (!p.balanced) {
        seg_s = blockIdx.z;
        seg_kvh = blockIdx.y;
        const int len = max(0, min(p.seq_lens[seg_s], p.max_blocks * BS));
        const int nblk = (len + BS - 1) / BS;
        const int b0 = blockIdx.x * p.blocks_per_split;  // even for BS = 8 (the host sees to it): a multiple of 16 tokens
        const int b1 = min(nblk, b0 + p.blocks_per_split);
        if (p.splits > 1 && b0 >= nblk && blockIdx.x != 0) return;  // nothing of this sequence here (split 0 reports an empty one)
        seg_tok_begin = b0 * BS;
        seg_tok_end = min(len, b1 * BS);
        seg_slot = blockIdx.x;
        __syncthreads();  // the ring barriers are initialised
    } else {
        // inclusive scan of the sequences' chunk counts into sm_pre, and their maximum
        const int S = p.num_seqs;
        const int per = (S + kPagedThreads - 1) / kPagedThreads;
        const int s_lo = min(S, static_cast<int>(threadIdx.x) * per), s_hi = min(S, s_lo + per);
        int sum = 0, mx = 0;
        for (int s2 = s_lo; s2 < s_hi; ++s2) {
            const int c = paged_chunks(p, s2);
            sum += c;
            mx = max(mx, c);
        }
        int incl = sum;
#pragma unroll
        for (int w = 1; w < 32; w <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, w);
            if (lane >= w) incl += v;
            mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, w));
        }
        if (lane == 31) sm_red[warp] = incl;
        if (lane == 0) sm_red[kPagedWarps + warp] = mx;
        __syncthreads();  // also: the ring barriers are initialised
        int before = incl - sum;
        int total = 0, max_row = 0;
#pragma unroll
        for (int w = 0; w < kPagedWarps; ++w) {
            if (w < warp) before += sm_red[w];
            total += sm_red[w];
            max_row = max(max_row, sm_red[kPagedWarps + w]);
        }
        if (threadIdx.x == 0) sm_pre[0] = 0;
        for (int s2 = s_lo; s2 < s_hi; ++s2) {
            before += paged_chunks(p, s2);
            sm_pre[s2 + 1] = before;
        }
        __syncthreads();
        const long long n = static_cast<long long>(total) * p.H_kv;
        bal_q = paged_quota(n, max_row, static_cast<int>(gridDim.x));
        bal_i = static_cast<long long>(blockIdx.x) * bal_q;
        bal_hi = min(n, bal_i + bal_q);
        if (bal_i >= n) return;
        // the sequence that holds chunk number bal_i: the last s with H_kv * pre[s] <= bal_i
        int lo = 0, hi = S;  // invariant: H_kv * pre[lo] <= bal_i < H_kv * pre[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (static_cast<long long>(sm_pre[mid]) * p.H_kv <= bal_i) lo = mid; else hi = mid;
        }
        seg_s = lo;
        seg_kvh = 0; seg_tok_begin = 0; seg_tok_end = 0; seg_slot = 0;  // set by next_segment below
    }
    // balanced: the segment that starts at chunk number bal_i (inside sequence seg_s); false when the CTA is done
    auto next_segment = [&]() -> bool {
        if (bal_i >= bal_hi) return false;
        while (static_cast<long long>(sm_pre[seg_s + 1]) * p.H_kv <= bal_i) ++seg_s;  // skips empty sequences too
        const int n_s = sm_pre[seg_s + 1] - sm_pre[seg_s];
        const long long r = bal_i - static_cast<long long>(sm_pre[seg_s]) * p.H_kv;
        seg_kvh = static_cast<int>(r / n_s);
        const int ch0 = static_cast<int>(r % n_s);
        const int ch1 = static_cast<int>(min(static_cast<long long>(n_s), ch0 + (bal_hi - bal_i)));
        const int len = max(0, min(p.seq_lens[seg_s], p.max_blocks * BS));
        seg_tok_begin = ch0 * kPagedChunkTokens;
        seg_tok_end = min(len, ch1 * kPagedChunkTokens);
        const long long row_start = bal_i - ch0;
        seg_slot = static_cast<int>(blockIdx.x - row_start / bal_q);
        bal_i += ch1 - ch0;
        return true;
    };
    if (p.balanced && !next_segment()) return;

    uint32_t kbase = 0;        // units this warp has been through so far (the ring stage follows it)
    uint32_t ring_parity = 0;  // bit st: parity of the next completion of stage st's barrier
    bool ok = true;
    for (;;) {
    // =============================== one segment ===============================
    const int s = seg_s, kvh = seg_kvh, tok_begin = seg_tok_begin, tok_end = seg_tok_end;
    const int head0 = kvh * G;
    const int b1 = (tok_end + BS - 1) / BS;  // cache blocks of the sequence this segment may touch end here

    // Q as A fragments: rows g < G hold head head0 + g, the others are zero
    uint32_t qa[PP][4];
#pragma unroll
    for (int pp = 0; pp < PP; ++pp) {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (g < G) v = *reinterpret_cast<const uint4*>(p.Q + (static_cast<int64_t>(s) * p.H + head0 + g) * D + pp * 32 + tg * 8);
        qa[pp][0] = v.x; qa[pp][1] = v.y; qa[pp][2] = v.z; qa[pp][3] = v.w;
    }
    float oacc[HV][8][4];
#pragma unroll
    for (int h = 0; h < HV; ++h)
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) oacc[h][nt][i] = 0.0f;
    float m_run = -INFINITY, l_part = 0.0f;  // head g: running max (log2 units, equal in the 4 lanes of a group), this lane's share of the sum

    const int* table = p.block_table + static_cast<int64_t>(s) * p.max_blocks;
    const int64_t head_off = static_cast<int64_t>(kvh) * BS * D;
    const int64_t blk_stride = static_cast<int64_t>(p.H_kv) * BS * D;

    struct Unit {  // the K and V registers of one unit of 16 tokens
        uint4 kr[2][PP], vr[HV][4];
    };
    // Unit k of this warp starts at token first + k * kStep.  The table entries of 32 units at a time are read by
    // one coalesced load (lane i: unit tab_base + i) and handed out by shuffles: a table load in every unit's path
    // would put a second memory latency in front of its K/V loads.
    constexpr int kStep = kPagedWarps * 16;
    const int first = tok_begin + warp * 16;
    const int n_units = first < tok_end ? (tok_end - first + kStep - 1) / kStep : 0;
    int tab[NB];
    int tab_base = -64;
    auto issue_unit = [&](int stage, int k) -> bool {  // returns false if a bad table entry makes the unit unusable
        const int u0 = first + k * kStep;
        if (k >= tab_base + 32) {
            tab_base = k;
#pragma unroll
            for (int i = 0; i < NB; ++i) {
                const int b = (first + (k + lane) * kStep) / BS + i;
                tab[i] = (k + lane < n_units && b < b1) ? table[b] : 0;
            }
        }
        int phys[NB];
        bool usable = true;
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            const int b = u0 / BS + i;
            phys[i] = __shfl_sync(0xffffffffu, tab[i], k - tab_base);
            if (b < b1 && (phys[i] < 0 || phys[i] >= p.num_blocks)) {  // never dereference a bad table entry
                usable = false;
                if (lane == 0 && atomicCAS(&g_status[0], 0u, kStatusBadBlock) == 0u) {
                    g_status[1] = static_cast<unsigned int>(b);
                    g_status[2] = static_cast<unsigned int>(s);
                    g_status[3] = static_cast<unsigned int>(phys[i]);
                }
            }
        }
        if (!usable) return false;
        // every lane must be done reading the stage's previous contents before the copies overwrite them
        __syncwarp();
        const int rows_in = min(16, tok_end - u0);  // rows beyond the sequence's end are not copied but zeroed
        uint64_t* bar = &ring_bar[warp][stage];
        if (lane == 0) mbar_arrive_expect_tx(bar, 2u * rows_in * (D * 2));
        __syncwarp();
        uint8_t* dst = my_ring + stage * kUnitBytes;
        constexpr int kPieceRows = 16 / NB;  // token rows per bulk copy: a cache block, or the half of one that the unit covers
        if (lane < 2 * NB) {  // lanes 0 .. NB-1: the K pieces, lanes NB .. 2 NB - 1: the V pieces
            const int piece = lane % NB, is_v = lane / NB;
            const int rows = min(kPieceRows, rows_in - piece * kPieceRows);
            if (rows > 0) {
                const int t0 = u0 + piece * kPieceRows;
                const __nv_bfloat16* src = (is_v ? p.V_cache : p.K_cache) + static_cast<int64_t>(phys[piece]) * blk_stride + head_off +
                                           static_cast<int64_t>(t0 % BS) * D;
                bulk_load(dst + (is_v * 16 + piece * kPieceRows) * kPitch, src, rows * (D * 2), bar);
            }
        }
        if (rows_in < 16) {  // a weight of 0 must not meet whatever the cache holds beyond the sequence's end
            for (int i = lane; i < (16 - rows_in) * (kPitch / 16); i += 32) {
                reinterpret_cast<uint4*>(dst + rows_in * kPitch)[i] = make_uint4(0u, 0u, 0u, 0u);
                reinterpret_cast<uint4*>(dst + (16 + rows_in) * kPitch)[i] = make_uint4(0u, 0u, 0u, 0u);
            }
            __syncwarp();
        }
        return true;
    };
    auto fetch_unit = [&](Unit& un, int stage) {
        const uint8_t* src = my_ring + stage * kUnitBytes;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int tok = 4 * (g >> 1) + (g & 1) + 2 * e;
#pragma unroll
            for (int pp = 0; pp < PP; ++pp)
                un.kr[e][pp] = *reinterpret_cast<const uint4*>(src + tok * kPitch + (pp * 32 + tg * 8) * 2);
        }
#pragma unroll
        for (int h = 0; h < HV; ++h)
#pragma unroll
            for (int i = 0; i < 4; ++i)
                un.vr[h][i] = *reinterpret_cast<const uint4*>(src + (16 + 4 * tg + i) * kPitch + (h * 64 + g * 8) * 2);
    };
    auto compute_unit = [&](const Unit& un, int u0) {
        // ---- scores of head g for tokens 4 tg .. 4 tg + 3 ----
        float sc[2][4];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
#pragma unroll
            for (int i = 0; i < 4; ++i) sc[e][i] = 0.0f;
#pragma unroll
            for (int pp = 0; pp < PP; ++pp) {
                mma_bf16_16816(sc[e], qa[pp][0], 0u, qa[pp][1], 0u, un.kr[e][pp].x, un.kr[e][pp].y);
                mma_bf16_16816(sc[e], qa[pp][2], 0u, qa[pp][3], 0u, un.kr[e][pp].z, un.kr[e][pp].w);
            }
        }
        float x[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            x[i] = (u0 + 4 * tg + i < tok_end) ? sc[i >> 1][i & 1] * p.scale_log2e : -INFINITY;
        float mb = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
        mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, 1));
        mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, 2));
        const float mn = fmaxf(m_run, mb);  // finite: token u0 of this unit is inside the sequence
        const float alpha = fast_exp2(m_run - mn);  // 0 for the first unit (m_run = -inf)
        float pw[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) pw[i] = fast_exp2(x[i] - mn);
        l_part = l_part * alpha + (pw[0] + pw[1]) + (pw[2] + pw[3]);
        if (__any_sync(0xffffffffu, mn != m_run)) {  // the maximum rarely moves after the first units
#pragma unroll
            for (int h = 0; h < HV; ++h)
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) {
                    oacc[h][nt][0] *= alpha;
                    oacc[h][nt][1] *= alpha;
                }
        }
        m_run = mn;
        // ---- O += P V: the probabilities are the A fragment as they stand ----
        const uint32_t pa0 = pack_bf16x2(pw[0], pw[1]), pa2 = pack_bf16x2(pw[2], pw[3]);
#pragma unroll
        for (int h = 0; h < HV; ++h) {
            const uint32_t w0[4] = {un.vr[h][0].x, un.vr[h][0].y, un.vr[h][0].z, un.vr[h][0].w};
            const uint32_t w1[4] = {un.vr[h][1].x, un.vr[h][1].y, un.vr[h][1].z, un.vr[h][1].w};
            const uint32_t w2[4] = {un.vr[h][2].x, un.vr[h][2].y, un.vr[h][2].z, un.vr[h][2].w};
            const uint32_t w3[4] = {un.vr[h][3].x, un.vr[h][3].y, un.vr[h][3].z, un.vr[h][3].w};
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                const uint32_t sel = (nt & 1) ? 0x7632u : 0x5410u;  // the same element of D from two tokens
                const uint32_t vb0 = __byte_perm(w0[nt >> 1], w1[nt >> 1], sel);
                const uint32_t vb1 = __byte_perm(w2[nt >> 1], w3[nt >> 1], sel);
                mma_bf16_16816(oacc[h][nt], pa0, 0u, pa2, 0u, vb0, vb1);
            }
        }
    };
    // Unit k of the segment is the warp's unit kbase + k and uses ring stage (kbase + k) % kPagedRing.  A stage's
    // barrier completes once per use; a unit that is left out (bad table entry) does not use its stage, so the parity
    // to wait for is kept per stage (ring_parity) and flips with every wait.
    uint32_t usable = 0;  // bit (k % 32): unit k may be used
#pragma unroll
    for (int k = 0; k < kPagedRing - 1; ++k)
        if (k < n_units && issue_unit((kbase + k) % kPagedRing, k)) usable |= 1u << k;
    for (int k = 0; k < n_units && ok; ++k) {
        const int kk = k + kPagedRing - 1;
        if (kk < n_units) {
            if (issue_unit((kbase + kk) % kPagedRing, kk)) usable |= 1u << (kk & 31);
            else usable &= ~(1u << (kk & 31));
        }
        if (usable & (1u << (k & 31))) {
            const uint32_t st = (kbase + k) % kPagedRing;
            ok = __all_sync(0xffffffffu, mbar_wait(&ring_bar[warp][st], (ring_parity >> st) & 1, &ring_abort, 0x500 + warp)) != 0;
            if (!ok) break;
            ring_parity ^= 1u << st;
            Unit un;
            fetch_unit(un, st);
            compute_unit(un, first + k * kStep);
        }
    }
    kbase += n_units;

    // The warps' partial outputs go where the ring was (every warp's copies have landed and been read by now).
    __syncthreads();
    float (*sm_o)[G][D] = reinterpret_cast<float (*)[G][D]>(ring_base);
    static_assert(sizeof(float) * kPagedWarps * G * D <= kPagedWarps * kPagedRing * 32 * PagedRow<D>::kPitch, "partials fit the ring");
    // ---- warp result: sum of the group's shares of l; output element of (h, nt, column 2 tg + i) is h*64 + (2 tg + i)*8 + nt ----
    l_part += __shfl_xor_sync(0xffffffffu, l_part, 1);
    l_part += __shfl_xor_sync(0xffffffffu, l_part, 2);
    if (g < G) {
#pragma unroll
        for (int h = 0; h < HV; ++h)
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                sm_o[warp][g][h * 64 + (2 * tg) * 8 + nt] = oacc[h][nt][0];
                sm_o[warp][g][h * 64 + (2 * tg + 1) * 8 + nt] = oacc[h][nt][1];
            }
        if (tg == 0) sm_ml[warp][g] = make_float2(m_run, l_part);
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < G * D; idx += kPagedThreads) {
        const int gg = idx / D, d = idx % D;
        float mt = -INFINITY;
#pragma unroll
        for (int w = 0; w < kPagedWarps; ++w) mt = fmaxf(mt, sm_ml[w][gg].x);
        float lt = 0.0f, ot = 0.0f;
#pragma unroll
        for (int w = 0; w < kPagedWarps; ++w) {
            const float2 ml = sm_ml[w][gg];
            const float sw = (ml.x == -INFINITY) ? 0.0f : fast_exp2(ml.x - mt);
            lt += ml.y * sw;
            ot += sm_o[w][gg][d] * sw;
        }
        const int64_t row = static_cast<int64_t>(s) * p.H + head0 + gg;
        if (p.splits == 1) {
            p.O[row * D + d] = __float2bfloat16(lt > 0.0f ? ot / lt : 0.0f);
            if (d == 0 && p.LSE) p.LSE[row] = lt > 0.0f ? (mt + log2f(lt)) * 0.6931471805599453f : -INFINITY;
        } else {
            p.part_o[(row * p.splits + seg_slot) * D + d] = ot;
            if (d == 0) p.part_ml[row * p.splits + seg_slot] = make_float2(mt, lt);
        }
    }
    if (!p.balanced || !ok) break;
    __syncthreads();  // the partials have left shared memory: the ring may be filled again
    if (!next_segment()) break;
    }  // segments
}

// O[row] = sum over splits of the partials, rescaled to the common max; one CTA of D threads per (seq, head).
// The {m, l} pairs go through shared memory once, and the partial outputs are read with independent loads
// (eight in flight per thread), so the kernel is a few microseconds of latency rather than a chain of them.
template <int D>
__global__ void __launch_bounds__(D)
paged_combine_kernel(const PagedParams p) {
    __shared__ float sm_w[kPagedMaxSplits];  // 2^(m_sp - m) per split
    __shared__ float sm_stat[2];             // common max, total l
    const int64_t row = blockIdx.x;
    const int d = threadIdx.x;
    int used;  // partials the decode kernel wrote for this row
    if (!p.balanced) {
        const int len = max(0, min(p.seq_lens[row / p.H], p.max_blocks * p.block_size));  // as in the decode kernel
        const int nblk = (len + p.block_size - 1) / p.block_size;
        used = max(1, min(p.splits, (nblk + p.blocks_per_split - 1) / p.blocks_per_split));
    } else {
        // the decode kernel's arithmetic again: chunks before this row's sequence, in all, and the longest row's
        __shared__ int sm_bal[3][D / 32];
        const int s = static_cast<int>(row / p.H), kvh = static_cast<int>(row % p.H) / (p.H / p.H_kv);
        int below = 0, total = 0, mx = 0;
        for (int s2 = d; s2 < p.num_seqs; s2 += D) {
            const int c = paged_chunks(p, s2);
            total += c;
            mx = max(mx, c);
            if (s2 < s) below += c;
        }
#pragma unroll
        for (int w = 16; w > 0; w >>= 1) {
            below += __shfl_xor_sync(0xffffffffu, below, w);
            total += __shfl_xor_sync(0xffffffffu, total, w);
            mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, w));
        }
        if ((d & 31) == 0) { sm_bal[0][d >> 5] = below; sm_bal[1][d >> 5] = total; sm_bal[2][d >> 5] = mx; }
        __syncthreads();
        below = total = mx = 0;
#pragma unroll
        for (int w = 0; w < D / 32; ++w) { below += sm_bal[0][w]; total += sm_bal[1][w]; mx = max(mx, sm_bal[2][w]); }
        const int n_s = paged_chunks(p, s);
        const int q = paged_quota(static_cast<long long>(total) * p.H_kv, mx, p.balanced_ctas);
        const long long row_start = static_cast<long long>(below) * p.H_kv + static_cast<long long>(kvh) * n_s;
        used = n_s > 0 ? static_cast<int>((row_start + n_s - 1) / q - row_start / q + 1) : 0;
    }
    // Launched with programmatic stream serialisation: the CTAs may start while the decode kernel is still
    // running (which hides this kernel's launch latency) and wait here until all of its writes are visible.
    cudaGridDependencySynchronize();
    // the first 8 partial outputs are requested before the weights are known: one memory latency instead of two
    const float* po = p.part_o + row * p.splits * D + d;
    float v0[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v0[i] = i < used ? po[i * D] : 0.0f;
    if (d < 32) {
        const float2 ml = d < used ? p.part_ml[row * p.splits + d] : make_float2(-INFINITY, 0.0f);
        float mt = ml.x;
#pragma unroll
        for (int w = 16; w > 0; w >>= 1) mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, w));
        const float sw = (ml.x == -INFINITY) ? 0.0f : fast_exp2(ml.x - mt);
        float lt = ml.y * sw;
#pragma unroll
        for (int w = 16; w > 0; w >>= 1) lt += __shfl_xor_sync(0xffffffffu, lt, w);
        sm_w[d] = sw;
        if (d == 0) {
            sm_stat[0] = mt;
            sm_stat[1] = lt;
        }
    }
    __syncthreads();
    float ot = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) ot = fmaf(v0[i], sm_w[i], ot);  // slots beyond `used` have weight 0
    int sp = 8;
    for (; sp + 8 <= used; sp += 8) {
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = po[(sp + i) * D];
#pragma unroll
        for (int i = 0; i < 8; ++i) ot = fmaf(v[i], sm_w[sp + i], ot);
    }
    for (; sp < used; ++sp) ot = fmaf(po[sp * D], sm_w[sp], ot);
    const float mt = sm_stat[0], lt = sm_stat[1];
    p.O[row * D + d] = __float2bfloat16(lt > 0.0f ? ot / lt : 0.0f);
    if (d == 0 && p.LSE) p.LSE[row] = lt > 0.0f ? (mt + log2f(lt)) * 0.6931471805599453f : -INFINITY;
}

inline size_t paged_workspace_bytes(int num_seqs, int H, int D, int splits) {
    return splits <= 1 ? 0 : static_cast<size_t>(num_seqs) * H * splits * (static_cast<size_t>(D) * 4 + 8);
}

// How many CTAs share one (sequence, KV head).  Each covers the same number of KV blocks, so the CTAs beyond a
// short sequence's end are empty: aim at 16 blocks (256 tokens) per CTA, which leaves enough busy CTAs per SM to
// hide the HBM latency even when most sequences are shorter than the longest allowed; 8 blocks if that still
// leaves SMs idle; no split when there are already many (sequence, KV head) pairs per SM.
// With 4 or 8 query heads per KV head a CTA computes more per byte and writes a larger partial: 32 blocks per CTA.
inline int paged_choose_splits(int num_seqs, int H_kv, int group, int max_blocks, int sm_count) {
    const int64_t base = static_cast<int64_t>(num_seqs) * H_kv;
    if (base >= 16ll * sm_count) return 1;
    const int per_cta = group >= 4 ? 32 : 16;
    int splits = (max_blocks + per_cta - 1) / per_cta;
    if (base * splits < 4ll * sm_count) splits = (max_blocks + per_cta / 2 - 1) / (per_cta / 2);
    return std::max(1, std::min(splits, kPagedMaxSplits));
}

// Equal work per CTA is used by the grouped-head kernel whenever it would split sequences at all (and the
// sequences fit the scan's table): one CTA per slot the kernel can occupy, or fewer if there is not that much work.
inline bool paged_use_balanced(const PagedParams& p, int sm_count) {
    (void)sm_count;
    const int group = p.H / p.H_kv;
    return group >= 4 && p.splits > 1 && p.num_seqs <= kPagedBalanceMaxSeqs;
}
inline void paged_set_balanced(PagedParams* p, int sm_count) {
    const long long max_chunks = static_cast<long long>(p->num_seqs) * p->H_kv *
                                 ((static_cast<long long>(p->max_blocks) * p->block_size + kPagedChunkTokens - 1) / kPagedChunkTokens);
    p->balanced = 1;
    p->balanced_ctas = static_cast<int>(std::max<long long>(1, std::min<long long>(static_cast<long long>(kPagedMmaCtasPerSm) * sm_count, max_chunks)));
    p->splits = kPagedMaxSplits;  // partial slots per row
}

// KV blocks per CTA of a split sequence.  The grouped-head kernel works in units of 16 tokens, so with 8-token
// blocks every CTA starts at an even block.
inline int paged_blocks_per_split(int max_blocks, int splits, int block_size, int group) {
    int bps = (max_blocks + splits - 1) / splits;
    if (group >= 4 && block_size == 8) bps = (bps + 1) & ~1;
    return bps;
}

template <int D, int G>
int paged_launch_bs(const PagedParams& p, cudaStream_t st) {
    dim3 grid(p.splits, p.H_kv * p.head_groups, p.num_seqs);
    if (p.balanced) grid = dim3(p.balanced_ctas);
    if constexpr (G >= 4) {  // grouped heads: rows of a tensor-core MMA
        constexpr size_t smem = paged_mma_smem_bytes<D>();
        switch (p.block_size) {
            case 8: paged_decode_mma_kernel<D, G, 8><<<grid, kPagedThreads, smem, st>>>(p); break;
            case 16: paged_decode_mma_kernel<D, G, 16><<<grid, kPagedThreads, smem, st>>>(p); break;
            case 32: paged_decode_mma_kernel<D, G, 32><<<grid, kPagedThreads, smem, st>>>(p); break;
            default: return 2;
        }
    } else {
        switch (p.block_size) {
            case 8: paged_decode_kernel<D, G, 8><<<grid, kPagedThreads, 0, st>>>(p); break;
            case 16: paged_decode_kernel<D, G, 16><<<grid, kPagedThreads, 0, st>>>(p); break;
            case 32: paged_decode_kernel<D, G, 32><<<grid, kPagedThreads, 0, st>>>(p); break;
            default: return 2;
        }
    }
    if (cudaGetLastError() != cudaSuccess) return 4;
    if (p.splits > 1) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(p.num_seqs * p.H);
        cfg.blockDim = dim3(D);
        cfg.stream = st;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, paged_combine_kernel<D>, p) != cudaSuccess) return 4;
    }
    return 0;
}

template <int D>
int paged_launch_g(const PagedParams& p, cudaStream_t st) {
    switch (p.H / p.H_kv) {
        case 1: return paged_launch_bs<D, 1>(p, st);
        case 2: return paged_launch_bs<D, 2>(p, st);
        case 4: return paged_launch_bs<D, 4>(p, st);
        case 8: return paged_launch_bs<D, 8>(p, st);
        default: return 2;
    }
}

// Once per device: the grouped-head kernels' shared-memory ring is larger than the default limit.
template <int D, int G>
int paged_configure_one() {
    const int bytes = static_cast<int>(paged_mma_smem_bytes<D>());
    if (cudaFuncSetAttribute(paged_decode_mma_kernel<D, G, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess ||
        cudaFuncSetAttribute(paged_decode_mma_kernel<D, G, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess ||
        cudaFuncSetAttribute(paged_decode_mma_kernel<D, G, 32>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
        return 1;
    return 0;
}
inline int paged_configure() {
    return paged_configure_one<64, 4>() | paged_configure_one<64, 8>() | paged_configure_one<128, 4>() | paged_configure_one<128, 8>();
}

// workspace layout: part_o floats first, then part_ml pairs
inline int paged_launch(PagedParams p, int D, void* workspace, cudaStream_t st) {
    if (p.splits > 1) {
        p.part_o = static_cast<float*>(workspace);
        p.part_ml = reinterpret_cast<float2*>(p.part_o + static_cast<size_t>(p.num_seqs) * p.H * p.splits * D);
    } else {
        p.part_o = nullptr;
        p.part_ml = nullptr;
    }
    return D == 64 ? paged_launch_g<64>(p, st) : paged_launch_g<128>(p, st);
}

}  // namespace mlt
