// Multi-head attention forward in the FlashAttention-2 form (paper Sec. 2.5,
// Algorithm 1): per block of query rows, loop over K/V blocks; S = Q K_j^T on the
// tensor cores, online softmax with running row max m and row sum l, O += P V_j on
// the tensor cores, final O / l and LSE = m + ln l.
//
// A work item is 256 query rows of one (batch, head): two 128-row tiles that take turns on the tensor pipe, so
// the exponentials of one tile overlap the products of the other.  CTAs are persistent (one per SM): each runs
// the items at positions r * gridDim.x +/- blockIdx.x of a list sorted by length (direction alternating per
// round, which balances the CTAs' sums without a global counter); the loader prefetches the next item's K/V
// tiles, and its Q tiles once the current item's last Q K^T has completed.
//   warps 0-3   softmax / O-rescale / epilogue of tile 0 (one thread per query row)
//   warps 4-7   the same for tile 1
//   warp  8     UMMA issuer (the whole warp runs the loop, one elected lane issues) and owner of the
//               tensor-memory allocation; at D = 128 it serves both tiles in a fixed order, which keeps the two
//               softmax warpgroups half a period apart (one issuer per tile was tried there: the tiles fall into
//               step and D = 128 loses 18 %); at D = 64 it serves tile 0 only
//   warp  9     TMA loader (one lane): Q tiles, then K/V tiles through a ring; it also initialises the
//               barriers and issues the first loads before the CTA-wide sync
//   warp  10    D = 64: UMMA issuer of tile 1 (there S_t(j+1) does not wait for P_t(j) V, so a tile's products
//               follow its own softmax only; one warp serving both tiles in turn made each wait for the other's
//               softmax: 724 -> 760 TFLOP/s at 16k tokens); D = 128: idle
//   warp  11    idle (completes the third warpgroup for the register hand-over)
// One in eight of the exponentials of a D = 128 block (one in four at D = 64) is a cubic on the FMA pipe instead of
// a MUFU operation (exp2_poly2): the MUFU pipe is the longest leg of a tile's chain S -> softmax -> P -> P V -> S.
// Tensor memory (512 columns): S_0 | S_1 (128 FP32 columns each), O_0 | O_1 (D FP32 columns each).  D = 128:
// the BF16 P of a tile overwrites the first 64 columns of its S and is consumed from there as the A operand of
// P V.  D = 64: P_0 | P_1 have their own columns, and the next Q K^T of a tile is issued as soon as the softmax
// warps hold S in registers.
// Epilogue: O / l as BF16 into a 4 KB staging area per warp (128-byte swizzle), one TMA store per 32 x 64 box.
//
// Measured on B200 (what shaped this kernel):
//  * a UMMA of 128x128x16 takes 64 clocks, also with A from tensor memory; issuing one costs the issuing
//    thread about 46 clocks from a single divergent lane and about 20 from warp-uniform code with an elected
//    lane; a warp that shares its scheduler partition with busy warps is served rarely: a barrier wait costs
//    the issuer about 280 clocks even when the barrier completed long before, and a step of both tiles (four
//    waits, 32 products) takes about as long as the whole period -- the issuer is co-limiting;
//  * code that runs once per item (a separate copy of the first Q K^T, an unrolled epilogue, the item decode
//    with its divisions) is fetched cold every time and costs thousands of clocks on those starved warps: the
//    first products go through the loop body, the epilogue is a short loop, the decode is done once per CTA
//    into shared memory;
//  * per tile and K/V block the chain is: S ready -> TMEM load (125) -> softmax (about 1700: 1024 MUFU clocks
//    plus the packed FP32 work a single warp per partition cannot fully overlap) -> P V and next Q K^T
//    (about 1085) -> S ready; with two tiles half a period apart the period is about 3230 clocks, i.e. the
//    tensor pipe is busy about two thirds of the time;
//  * the SM clock under this kernel is 1.72-1.77 GHz (power management), not the 1.965 GHz maximum.
#pragma once

#include <math.h>

#include <cstdlib>

#include "ptx.cuh"

namespace mlt {

// In-kernel clock trace (development builds only, -DMLT_TRACE): CTA 0 records the SM clock at fixed points of K/V
// blocks 32..47 of its first work item; role 0 / 1 = first softmax warp of tile 0 / 1, role 2 = UMMA issuer.
#ifdef MLT_TRACE_ITEMS
// second form (-DMLT_TRACE -DMLT_TRACE_ITEMS): per work item r < 16 of CTA 0, the first 8 blocks' "S seen" and
// "P handed over" times (slots 2j, 2j + 1) and the item's start, "O complete seen" and "epilogue done" (18, 16, 17)
__device__ unsigned int g_mha_trace[3][16][24];
#define MLT_TR(role, j, ev)                                                                                  \
    do {                                                                                                     \
        if (blockIdx.x == 0 && r < 16 && (j) >= 0 && (j) < 8 && ((ev) == 1 || (ev) == 4))                     \
            g_mha_trace[role][r][(j) * 2 + ((ev) == 4)] = static_cast<unsigned int>(clock64());              \
    } while (0)
#define MLT_TRI(role, ev)                                                                                    \
    do {                                                                                                     \
        if (blockIdx.x == 0 && r < 16) g_mha_trace[role][r][ev] = static_cast<unsigned int>(clock64());      \
    } while (0)
#elif defined(MLT_TRACE)
__device__ unsigned int g_mha_trace[3][16][24];
#define MLT_TR(role, j, ev)                                                                                  \
    do {                                                                                                     \
        if (blockIdx.x == 0 && r == 0 && (j) >= 32 && (j) < 48) g_mha_trace[role][(j) - 32][ev] = static_cast<unsigned int>(clock64()); \
    } while (0)
#define MLT_TRI(role, ev) do { } while (0)
#else
#define MLT_TR(role, j, ev) do { } while (0)
#define MLT_TRI(role, ev) do { } while (0)
#endif

constexpr int kMhaBlock = 128;   // query rows per tile and keys per K/V block
constexpr int kMhaThreads = 384; // three warpgroups
#ifndef MLT_SOFTMAX_REGS
#define MLT_SOFTMAX_REGS 208
#endif
#ifndef MLT_OTHER_REGS
#define MLT_OTHER_REGS 88
#endif
constexpr int kMhaSoftmaxRegs = MLT_SOFTMAX_REGS;  // per thread of the 8 softmax warps after the hand-over
constexpr int kMhaOtherRegs = MLT_OTHER_REGS;      // per thread of the 4 other warps
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleLimit = 18446744073709551616.0f;  // 2^64: a block sum at or above it forces a new reference max

template <int D>
struct MhaSmem {
    static constexpr int kTileBytes = kMhaBlock * D * 2;  // one Q, K or V tile: D/64 chunks of 128 rows x 128 B
    static constexpr int kChunkBytes = kMhaBlock * 128;
    static constexpr int kStages = (D == 128) ? 4 : 8;
    static constexpr int kBarrierBytes = 512;
    static constexpr int kItemSlots = 64;       // work items decoded ahead of time (16 bytes each)
    static constexpr int kStageBytes = 8 * 4096;  // output staging: 4 KB per softmax warp
    static constexpr int kTotal =
        2 * kTileBytes + kStages * kTileBytes + kBarrierBytes + kItemSlots * 16 + kStageBytes + 1024;
};

struct MhaParams {
    float* LSE;  // may be null
    int BH, Nq, Nk;
    int causal;
    float scale;
    int num_pairs;   // 256-row query groups per head
    int head_group;  // heads that share a span of consecutive item indices
    int num_items;   // entries of the work list
    // Entries below full_items are whole items (both 128-row tiles of a 256-row group).  The entries after them are
    // single tiles, two entries per remaining item: a last round that would occupy at most half of the CTAs is
    // handed out tile by tile, so twice as many CTAs share it (a CTA with one tile runs its blocks in 0.8-0.9 of
    // the time of a CTA with two).
    int full_items;
};

// item index -> (pair, bh).  Heads are taken in groups; inside a group the query
// position is the slow index and runs from the last rows to the first, so under a
// causal mask the longest items are dispatched first, and the CTAs resident at any
// time read the K/V of few heads (L2 reuse).
__device__ __forceinline__ void mha_item(const MhaParams& p, int block, int& pair, int& bh) {
    const int per_group = p.num_pairs * p.head_group;
    const int g = block / per_group;
    const int first = g * p.head_group;
    const int heads = min(p.head_group, p.BH - first);
    const int r = block - g * per_group;
    pair = p.num_pairs - 1 - r / heads;
    bh = first + r % heads;
}

// 2^((s - m) * c) for a pair of scores on the FMA pipe (no MUFU).  The exponent x = (s - m) * c is clamped to
// [-125, 127] by a saturating FMA: u = sat((x + 125) / 252) in [0, 1], so x + 125 = 252 u.  Round-to-nearest split
// 252 u = N + f, |f| <= 0.5 (adding 1.5 * 2^23 leaves N in the low mantissa bits), a cubic for 2^f (relative error
// below 9e-5, far below the BF16 rounding of P), and N - 125 is added to the exponent field: the constant is
// folded into the magic number, whose low 9 mantissa bits then hold N - 125 in two's complement.
// 2^-125 ~ 2e-38 stands for 0 (masked scores are -inf and saturate to it); the upper end keeps the exponent add
// from carrying into the sign bit, and 2^127 is above the 2^64 limit, so a score that far above the reference max
// still forces the true-max repeat pass.  `cs` = c / 252, `ns` = (125 - m c) / 252.
constexpr float kPolySpan = 252.0f;
constexpr float kPolyLow = 125.0f;
__device__ __forceinline__ float fma_sat(float a, float b, float c) {
    float d;
    asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float2 exp2_poly2(float s0, float s1, float cs, float ns) {
    constexpr float kMagic = 12582912.0f - kPolyLow;  // 1.5 * 2^23 - 125
    const float2 u = make_float2(fma_sat(s0, cs, ns), fma_sat(s1, cs, ns));
    const float2 span = make_float2(kPolySpan, kPolySpan), magic = make_float2(kMagic, kMagic);
    const float2 t = ffma2(u, span, magic);  // N + magic, exact integer grid
    const float2 f = ffma2(u, span, fsub2(magic, t));
    float2 y = ffma2(f, make_float2(0.05508868396282196f, 0.05508868396282196f),
                     make_float2(0.24260404706001282f, 0.24260404706001282f));
    y = ffma2(y, f, make_float2(0.6932762265205383f, 0.6932762265205383f));
    y = ffma2(y, f, make_float2(0.9999289512634277f, 0.9999289512634277f));
    y.x = __int_as_float(__float_as_int(y.x) + (__float_as_int(t.x) << 23));
    y.y = __int_as_float(__float_as_int(y.y) + (__float_as_int(t.y) << 23));
    return y;
}

// Which of the 8 score pairs of every 16 keys take the FMA-pipe exponential (bit i = pair i).
#ifndef MLT_POLY_MASK_64
#define MLT_POLY_MASK_64 0x22
#endif
#ifndef MLT_POLY_MASK_128
#define MLT_POLY_MASK_128 0x10
#endif

template <int D>
__global__ void __launch_bounds__(kMhaThreads, 1)
mha_fwd_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_o,
               const MhaParams p) {
    using L = MhaSmem<D>;
    constexpr int kIssuers = (D == 64) ? 2 : 1;  // UMMA-issuing warps (see the role table)
    constexpr int kStages = L::kStages;
    constexpr int kChunks = D / 64;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* smem_q = smem;                        // [2][tile]
    uint8_t* smem_kv = smem + 2 * L::kTileBytes;   // [kStages][tile]
    uint8_t* smem_stage = smem_kv + kStages * L::kTileBytes;  // [8 warps][4 KB], 1024-byte aligned (TMA swizzle atoms)
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_stage + L::kStageBytes);
    uint64_t* q_full = bars;                  // [1]
    uint64_t* kv_full = bars + 1;             // [kStages]
    uint64_t* kv_empty = kv_full + kStages;   // [kStages]
    uint64_t* s_full = kv_empty + kStages;    // [2]  UMMA -> softmax: S_t(j) complete
    uint64_t* p_full = s_full + 2;            // [2]  softmax -> UMMA: P_t(j) in TMEM, O_t rescaled
    uint64_t* o_full = p_full + 2;            // [2]  UMMA -> epilogue: O_t complete
    uint64_t* q_empty = o_full + 2;           // [1]  UMMA -> loader: the item's last Q K^T has read the Q tiles
    uint64_t* s_free = q_empty + 1;           // [2]  softmax -> UMMA (D = 64): S_t(j) is in registers
    uint64_t* p_free = s_free + 2;            // [2]  UMMA -> softmax (D = 64): P_t(j) V has completed
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(p_free + 2);
    volatile uint32_t* abort_flag = tmem_base_slot + 1;

#ifndef MLT_ROLE_SHIFT
#define MLT_ROLE_SHIFT 0
#endif
    const int warp = ((threadIdx.x >> 5) + MLT_ROLE_SHIFT) % 12;  // role index (see the table above)
    const int lane = threadIdx.x & 31;
    if (blockIdx.x == 0 && threadIdx.x == 0) clock_probe(1, 0);

    // Work items of this CTA: item list position r * gridDim.x + (c or gridDim.x - 1 - c), the direction alternating
    // from round to round, so that with the list sorted by length the CTAs' sums stay within about one item.
    const int G = static_cast<int>(gridDim.x);
    const int rounds = (p.num_items + G - 1) / G;
    const int shift = p.Nk - p.Nq;  // bottom-right alignment of the causal mask
    struct Item {
        int q_base, bh, J[2], Jmax;
    };
    auto decode_item = [&](int r, Item& it) -> bool {
        const int idx = r * G + ((r & 1) ? G - 1 - static_cast<int>(blockIdx.x) : static_cast<int>(blockIdx.x));
        if (r >= rounds || idx >= p.num_items) return false;
        int pair, only = -1;  // only: the one tile a single-tile entry stands for
        int item = idx;
        if (idx >= p.full_items) {
            item = p.full_items + ((idx - p.full_items) >> 1);
            only = (idx - p.full_items) & 1;
        }
        mha_item(p, item, pair, it.bh);
        it.q_base = pair * 2 * kMhaBlock;
#pragma unroll
        for (int t = 0; t < 2; ++t) {  // number of K/V blocks each tile needs
            const int q0 = it.q_base + t * kMhaBlock;
            if (q0 >= p.Nq || (only >= 0 && t != only)) {
                it.J[t] = 0;
            } else {
                int last_key = p.Nk - 1;
                if (p.causal) last_key = min(last_key, min(q0 + kMhaBlock, p.Nq) - 1 + shift);
                it.J[t] = last_key / kMhaBlock + 1;
            }
        }
        it.Jmax = max(it.J[0], it.J[1]);
        return true;
    };
    // The first kItemSlots items of this CTA are decoded once, one per thread, into shared memory before the
    // CTA-wide sync: the issuing and loading warps share their scheduler partitions with the softmax warps and
    // get few issue slots, so the divisions of the decode would cost them thousands of clocks per item.
    int4* item_table = reinterpret_cast<int4*>(reinterpret_cast<uint8_t*>(bars) + L::kBarrierBytes);
    if (threadIdx.x < L::kItemSlots) {
        Item it;
        const bool have = decode_item(threadIdx.x, it);
        item_table[threadIdx.x] = have ? make_int4(it.q_base, it.bh, it.J[0], it.J[1]) : make_int4(0, 0, 0, 0);
    }
    auto item_at = [&](int r, Item& it) -> bool {  // valid after the CTA-wide sync
        if (r >= L::kItemSlots) return decode_item(r, it);
        const int4 e = item_table[r];
        it.q_base = e.x;
        it.bh = e.y;
        it.J[0] = e.z;
        it.J[1] = e.w;
        it.Jmax = max(e.z, e.w);
        return it.Jmax > 0;
    };

    // loader state: ring position and the number of Q loads so far
    int ld_stage = 0;
    uint32_t ld_phase = 0;
    auto load_q = [&](const Item& it) {
        mbar_arrive_expect_tx(q_full, 2 * L::kTileBytes);
#pragma unroll
        for (int t = 0; t < 2; ++t)
#pragma unroll
            for (int c = 0; c < kChunks; ++c)
                tma_load_3d(smem_q + t * L::kTileBytes + c * L::kChunkBytes, &tmap_q, q_full, c * 64,
                            it.q_base + t * kMhaBlock, it.bh);
    };
    // ring tile i of the item: K_0, V_0, K_1, V_1, ... (D = 128), or in the order the early Q K^T consumes them:
    // K_0, K_1, V_0, K_2, V_1, ..., K_{J-1}, V_{J-2}, V_{J-1} (D = 64)
    auto load_kv = [&](const Item& it, int i) {
        bool is_k = (i & 1) == 0;
        int blk = i >> 1;
        if (D == 64 && i > 0) {
            if (i == 2 * it.Jmax - 1) {
                is_k = false;
                blk = it.Jmax - 1;
            } else {
                is_k = (i & 1) == 1;
                blk = is_k ? (i + 1) >> 1 : (i >> 1) - 1;
            }
        }
        uint8_t* dst = smem_kv + ld_stage * L::kTileBytes;
        mbar_arrive_expect_tx(&kv_full[ld_stage], L::kTileBytes);
#pragma unroll
        for (int c = 0; c < kChunks; ++c)
            tma_load_3d(dst + c * L::kChunkBytes, is_k ? &tmap_k : &tmap_v, &kv_full[ld_stage], c * 64,
                        blk * kMhaBlock, it.bh);
        if (++ld_stage == kStages) { ld_stage = 0; ld_phase ^= 1; }
    };

    // The loader lane initialises the barriers and issues the first loads (Q and the first K/V tiles of the first
    // item: the ring is empty, nothing to wait for) before the CTA-wide sync, so they overlap the tensor-memory
    // allocation.
    int pre_tiles = 0;  // ring tiles of the first item already requested
    if (warp == 9 && lane == 0) {
        mbar_init(q_full, 1);
        // D = 64 has one issuing warp per query tile: each of them releases every K/V slot and the Q tiles
        mbar_init(q_empty, kIssuers);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&kv_full[s], 1);
            mbar_init(&kv_empty[s], kIssuers);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(&s_full[t], 1);
            mbar_init(&p_full[t], 4);  // one arrive per softmax warp
            mbar_init(&o_full[t], 1);
            mbar_init(&s_free[t], 4);
            mbar_init(&p_free[t], 1);
        }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_q);
        prefetch_tensormap(&tmap_k);
        prefetch_tensormap(&tmap_v);
        prefetch_tensormap(&tmap_o);
        Item it;
        if (decode_item(0, it)) {
            // K_0 first: with Q it is all the first product needs
            pre_tiles = min(2 * it.Jmax, kStages);
            for (int i = 0; i < pre_tiles; ++i) {
                if (i == 1) load_q(it);
                load_kv(it, i);
            }
        }
    }
    if (warp == 8) {
        tmem_alloc(tmem_base_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_slot;
    constexpr uint32_t kColS = 0;      // S_t at kColS + t*128
    constexpr uint32_t kColO = 256;    // O_t at kColO + t*D
    // D = 128 fills the 512 columns, so P_t (BF16) overwrites the first 64 columns of S_t and the next Q K^T of a
    // tile has to follow its P V.  D = 64 leaves 128 columns: P_t gets its own, and Q_t K_{j+1}^T is issued as soon
    // as the softmax warps hold S_t(j) in registers, so S_t(j+1) is ready when they come back for it.
    constexpr bool kEarlyQK = (D == 64);
    constexpr uint32_t kColP = kEarlyQK ? 384 : kColS;  // P_t at kColP + t*(kEarlyQK ? 64 : 128)
    constexpr uint32_t kStrideP = kEarlyQK ? 64 : kMhaBlock;

    // Register hand-over: setmaxnreg moves registers inside the CTA's launch allocation (384 threads x 168), it cannot
    // draw on the rest of the register file; if the two budgets together exceeded it, the increase below would wait
    // for ever.  208 / 88 measured best: the softmax code does not use more (232 / 40 was 3 % slower: the issuing
    // warp then spills).
    static_assert(8 * 32 * kMhaSoftmaxRegs + 4 * 32 * kMhaOtherRegs <= kMhaThreads * 168, "setmaxnreg budget exceeds the launch allocation");
    if (warp == 11 || (warp == 10 && kIssuers == 1)) {
        setmaxnreg_dec<kMhaOtherRegs>();  // only hand their registers over
#ifdef MLT_TRACE
        if (blockIdx.x == 0 && lane == 0) {  // spies: when do S_t(j) of the first item really complete?
            const int t = warp - 10;
            const int r = 0;
            for (int j = 0; j < 48; ++j) {
                int spins = 0;
                while (!mbar_test_wait(&s_full[t], j & 1) && ++spins < 4000000) {}
                MLT_TR(t, j, 8);
            }
        }
#endif
    } else if (warp == 9) {
        // ------------------------------- loader -------------------------------
        setmaxnreg_dec<kMhaOtherRegs>();
        if (lane == 0) {
            bool ok = true;
            Item it;
            for (int r = 0; ok && item_at(r, it); ++r) {
                for (int i = (r == 0 ? pre_tiles : 0); i < 2 * it.Jmax && ok; ++i) {
                    if (i == 1 && r > 0) {
                        // Q of the next item: the tiles are free once the previous item's last Q K^T has completed
                        ok = mbar_wait(q_empty, (r - 1) & 1, abort_flag, 0x110);
                        if (!ok) break;
                        load_q(it);
                    }
                    ok = mbar_wait(&kv_empty[ld_stage], ld_phase ^ 1, abort_flag, 0x100 + ld_stage);
                    if (!ok) break;
                    load_kv(it, i);
                }
            }
        }
    } else if (warp == 8 || warp == 10) {
        // ------------------------------- UMMA issuer -------------------------------
        // D = 128: warp 8 serves both tiles in a fixed order (which keeps them half a period apart).  D = 64: warp 8
        // serves tile 0 and warp 10 tile 1, each in its tile's own order (Q_t K_{j+1}^T when S_t(j) has been read,
        // P_t(j) V_j when P_t(j) is there), so that neither tile ever waits for the other's softmax; both walk
        // the same K/V ring and both release every slot.
        const int t_lo = (kIssuers == 2 && warp == 10) ? 1 : 0;
        const int t_hi = (kIssuers == 2 && warp == 8) ? 1 : 2;
        // The whole warp runs this code (uniform control flow keeps addresses and descriptors in the uniform
        // datapath: an issue costs about 20 clocks instead of about 46 from a single divergent lane); one
        // elected lane executes the tcgen05 instructions.
        setmaxnreg_dec<kMhaOtherRegs>();
        {
            const bool leader = elect_one();
            constexpr uint32_t idesc_qk = make_idesc_bf16(kMhaBlock, kMhaBlock, false, false);
            constexpr uint32_t idesc_pv = make_idesc_bf16(kMhaBlock, D, false, true);
            // descriptor low words: Q tiles fixed, K/V per ring slot; K steps add small constants
            const uint32_t q_lo0 = sdesc_lo(smem_u32(smem_q), 16);
            const uint32_t kv_lo0 = sdesc_lo(smem_u32(smem_kv), 16);
            const uint32_t v_lbo = (static_cast<uint32_t>(L::kChunkBytes) >> 4) << 16;  // V is MN-major: chunk pitch
            // S_t = Q_t K^T over the D/16 k-steps of the tile in ring slot `slot`
            auto issue_qk = [&](int t, int slot) {
                const uint32_t d = tmem_base + kColS + t * kMhaBlock;
                const uint32_t a0 = q_lo0 + t * (L::kTileBytes >> 4);
                const uint32_t b0 = kv_lo0 + slot * (L::kTileBytes >> 4);
                if (leader) {
                    umma_ss_lo<false>(d, a0, b0, idesc_qk);
#pragma unroll
                    for (int kk = 1; kk < D / 16; ++kk) {
                        const uint32_t off = ((kk / 4) * L::kChunkBytes + (kk % 4) * 32) >> 4;
                        umma_ss_lo<true>(d, a0 + off, b0 + off, idesc_qk);
                    }
                    umma_commit(&s_full[t]);
                }
                __syncwarp();
            };
            // O_t (+)= P_t V over the 8 k-steps (16 keys each) of the tile in ring slot `slot`
            auto issue_pv = [&](int t, int slot, bool first) {
                const uint32_t d = tmem_base + kColO + t * D;
                const uint32_t a0 = tmem_base + kColP + t * kStrideP;
                const uint32_t b0 = (kv_lo0 & 0xFFFFu) + slot * (L::kTileBytes >> 4) + v_lbo;
                if (leader) {
                    umma_ts_lo(d, a0, b0, idesc_pv, first ? 0u : 1u);
#pragma unroll
                    for (int kk = 1; kk < kMhaBlock / 16; ++kk)
                        umma_ts_lo(d, a0 + kk * 8, b0 + kk * (2048 >> 4), idesc_pv, 1u);
                }
                __syncwarp();
            };
            auto wait_all = [&](uint64_t* bar, uint32_t parity, uint32_t id) {
                return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, id)) != 0;
            };
            int stage = 0;
            uint32_t phase = 0;
            uint32_t n_p[2] = {0, 0};  // P tiles consumed so far, per query tile (parity of p_full)
            bool ok = true;
            Item it;
            uint32_t n_qk[2] = {0, 0};  // Q K^T products issued so far, per query tile (parity of s_free)
            if constexpr (kEarlyQK) {
                for (int r = 0; ok && item_at(r, it); ++r) {
                    const int Jmax = it.Jmax;
                    ok = wait_all(q_full, r & 1, 0x200);
                    // Step j: Q_t K_{j+1}^T as soon as S_t(j) has been read, then P_t(j) V_j, for this warp's tile(s).
                    // Step -1 issues the first Q K^T products only (same instructions, no cold copy).
#pragma unroll 1
                    for (int j = -1; j < Jmax && ok; ++j) {
                        if (leader && warp == 8) MLT_TR(2, j, 0);
                        if (j + 1 < Jmax) {
                            const int kslot = stage;
                            ok = wait_all(&kv_full[kslot], phase, 0x240 + kslot);
                            if (!ok) break;
                            if (leader && warp == 8) MLT_TR(2, j, 1);
                            if (++stage == kStages) { stage = 0; phase ^= 1; }
                            tc_fence_after();
                            for (int t = t_lo; t < t_hi && ok; ++t) {
                                if (j + 1 >= it.J[t]) continue;
                                if (n_qk[t] > 0) {  // S_t is free once the softmax warps hold its previous contents
                                    ok = wait_all(&s_free[t], (n_qk[t] - 1) & 1, 0x250 + t);
                                    if (!ok) break;
                                    tc_fence_after();
                                }
                                if (leader && warp == 8) MLT_TR(2, j, 2);
                                ++n_qk[t];
                                issue_qk(t, kslot);
                                if (leader && warp == 8) MLT_TR(2, j, 3);
                            }
                            if (!ok) break;
                            if (leader) {
                                umma_commit(&kv_empty[kslot]);
                                if (j + 2 == Jmax) umma_commit(q_empty);  // the item's last Q K^T products are issued
                            }
                            __syncwarp();
                        }
                        if (j >= 0) {
                            const int vslot = stage;
                            ok = wait_all(&kv_full[vslot], phase, 0x220 + vslot);
                            if (!ok) break;
                            if (++stage == kStages) { stage = 0; phase ^= 1; }
                            if (leader && warp == 8) MLT_TR(2, j, 4);
                            for (int t = t_lo; t < t_hi && ok; ++t) {
                                if (j >= it.J[t]) continue;
                                // P_t(0) of an item also tells that the softmax warps have read the previous O_t
                                ok = wait_all(&p_full[t], n_p[t] & 1, 0x230 + t);
                                if (!ok) break;
                                if (leader && warp == 8) MLT_TR(2, j, 5);
                                ++n_p[t];
                                tc_fence_after();
                                issue_pv(t, vslot, j == 0);
                                if (leader && warp == 8) MLT_TR(2, j, 6);
                                if (leader) {
                                    umma_commit(&p_free[t]);
                                    if (j == it.J[t] - 1) umma_commit(&o_full[t]);
                                }
                                __syncwarp();
                            }
                            if (!ok) break;
                            if (leader) umma_commit(&kv_empty[vslot]);
                            __syncwarp();
                        }
                    }
                }
            } else {
            for (int r = 0; ok && item_at(r, it); ++r) {
                const int Jmax = it.Jmax;
                ok = wait_all(q_full, r & 1, 0x200);
                // Step j issues P_t(j) V_j and then Q_t K_{j+1}^T for both tiles; step -1 issues only the first
                // Q K^T products, through the same instructions as every other step (code that runs once per item
                // would be fetched cold each time).  S_t(0) may overwrite P_t of the previous item: the tensor
                // pipe runs the products in issue order.
#pragma unroll 1
                for (int j = -1; j < Jmax && ok; ++j) {
                    int vslot = 0;
                    if (leader) MLT_TR(2, j, 0);
                    if (j >= 0) {
                        vslot = stage;
                        ok = wait_all(&kv_full[vslot], phase, 0x220 + vslot);
                        if (!ok) break;
                        if (++stage == kStages) { stage = 0; phase ^= 1; }
                    }
                    const int kslot = stage;  // K_{j+1}, if there is one
                    bool k_ready = false;
                    for (int t = 0; t < 2 && ok; ++t) {
                        if (j >= 0 && j < it.J[t]) {
                            // P_t(0) of an item also tells that the softmax warps have read the previous item's O_t
                            if (leader) MLT_TR(2, j, 1 + 4 * t);
                            ok = wait_all(&p_full[t], n_p[t] & 1, 0x230 + t);
                            if (!ok) break;
                            if (leader) MLT_TR(2, j, 2 + 4 * t);
                            ++n_p[t];
                            tc_fence_after();
                            issue_pv(t, vslot, j == 0);
                            if (leader) MLT_TR(2, j, 3 + 4 * t);
                            if (j == it.J[t] - 1 && leader) umma_commit(&o_full[t]);
                        }
                        if (j + 1 < it.J[t]) {
                            if (!k_ready) {
                                ok = wait_all(&kv_full[kslot], phase, 0x240 + kslot);
                                if (!ok) break;
                                tc_fence_after();
                                k_ready = true;
                            }
                            issue_qk(t, kslot);
                            if (leader) MLT_TR(2, j, 4 + 4 * t);
                        }
                    }
                    if (!ok) break;
                    if (leader) {
                        if (j >= 0) umma_commit(&kv_empty[vslot]);
                        if (j + 1 < Jmax) umma_commit(&kv_empty[kslot]);
                        if (j + 2 == Jmax) umma_commit(q_empty);  // the item's last Q K^T products are issued
                    }
                    __syncwarp();
                    if (j + 1 < Jmax) {
                        if (++stage == kStages) { stage = 0; phase ^= 1; }
                    }
                }
            }
            }  // !kEarlyQK
        }
    } else {
        // ------------------- softmax, O rescale and epilogue of tile t -------------------
        setmaxnreg_inc<kMhaSoftmaxRegs>();
        const int t = warp >> 2;
        const int quarter = warp & 3;
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const uint32_t s_addr = lane_addr + kColS + t * kMhaBlock;
        const uint32_t o_addr = lane_addr + kColO + t * D;
        const uint32_t p_addr = lane_addr + kColP + t * kStrideP;
        const float c = p.scale * kLog2e;
        uint32_t n_s = 0, n_o = 0;  // S tiles and O tiles taken so far (parities of s_full / o_full)
        bool ok = true;
        Item it;
        for (int r = 0; ok && item_at(r, it); ++r) {
        const int Jt = it.J[t];
        if (Jt == 0) continue;  // this tile lies beyond the last query row
        const int qi = it.q_base + t * kMhaBlock + row_in_tile;  // query index inside the head
        const int limit = p.causal ? min(p.Nk - 1, qi + shift) : p.Nk - 1;  // last visible key of this row
        float m_run = -INFINITY;  // reference max (raw score units), taken from the row's first block
        float l_run = 0.0f;
        if (quarter == 0 && lane == 0) MLT_TRI(t, 18);

        for (int j = 0; j < Jt; ++j) {
            if (quarter == 0 && lane == 0) MLT_TR(t, j, 0);
            ok = __all_sync(0xffffffffu, mbar_wait(&s_full[t], n_s & 1, abort_flag, 0x300 + t));
            if (!ok) break;
            if (quarter == 0 && lane == 0) MLT_TR(t, j, 1);
            ++n_s;
            tc_fence_after();
            uint32_t s[4][32];  // this thread's row of S: 4 chunks of 32 keys
#pragma unroll
            for (int q = 0; q < 4; ++q) tmem_ld_32x32b_x32(s_addr + q * 32, s[q]);
            tmem_wait_ld();
            if (quarter == 0 && lane == 0) MLT_TR(t, j, 2);
            if constexpr (kEarlyQK) {  // S_t is in registers: the next Q K^T of this tile may overwrite it
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_free[t]);
            }
            const int j0 = j * kMhaBlock;
            if (j0 + kMhaBlock - 1 > limit) {  // diagonal or tail block: mask keys beyond the row's last visible one
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (j0 + q * 32 + i > limit) s[q][i] = 0xFF800000u;  // -inf
            }
            // One pass: p = 2^((s - m_ref)*c) against a reference max m_ref taken from an earlier block.  Any
            // reference gives the same O / l and the same m_ref*scale + ln l as long as nothing overflows (FP32
            // and BF16 share the exponent range), so the row max is not taken at all on the fast path.  Only if
            // the block's sum reaches 2^64 (or is not finite) is the true row max taken, O and l rescaled to it
            // and the pass repeated; the first block of a row takes its max first.
            float2 acc0, acc1;
            auto row_max = [&]() {
                float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        mx[(i >> 2) & 3] = fmaxf(mx[(i >> 2) & 3],
                                                 fmaxf(fmaxf(__uint_as_float(s[q][i]), __uint_as_float(s[q][i + 1])),
                                                       fmaxf(__uint_as_float(s[q][i + 2]), __uint_as_float(s[q][i + 3]))));
                return fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
            };
            auto exp_pass = [&](float neg_mc) {
                constexpr int kPolyMask = (D == 64) ? MLT_POLY_MASK_64 : MLT_POLY_MASK_128;
                const float2 c2 = make_float2(c, c), n2 = make_float2(neg_mc, neg_mc);
                const float cs = c * (1.0f / kPolySpan), ns = (neg_mc + kPolyLow) * (1.0f / kPolySpan);
                acc0 = make_float2(0.0f, 0.0f);
                acc1 = make_float2(0.0f, 0.0f);
                uint32_t pk[16];
                auto exp_pair = [&](int k, bool poly) {  // keys k, k + 1 of the block
                    const float s0 = __uint_as_float(s[k >> 5][k & 31]), s1 = __uint_as_float(s[k >> 5][(k & 31) + 1]);
                    if (poly) return exp2_poly2(s0, s1, cs, ns);
                    float2 x = ffma2(make_float2(s0, s1), c2, n2);
                    x.x = fast_exp2(x.x);
                    x.y = fast_exp2(x.y);
                    return x;
                };
#pragma unroll
                for (int w = 0; w < 8; ++w) {  // waves of 16 keys
#pragma unroll
                    for (int i = 0; i < 8; i += 2) {
                        const int k = w * 16 + 2 * i;
                        const float2 x0 = exp_pair(k, (kPolyMask >> i) & 1);
                        const float2 x1 = exp_pair(k + 2, (kPolyMask >> (i + 1)) & 1);
                        acc0 = fadd2(acc0, x0);
                        acc1 = fadd2(acc1, x1);
                        pk[(w & 1) * 8 + i] = pack_bf16x2(x0.x, x0.y);
                        pk[(w & 1) * 8 + i + 1] = pack_bf16x2(x1.x, x1.y);
                    }
                    if (kEarlyQK && w == 1 && n_s > 1) {
                        // P_t has its own columns: the previous P_t V (P number n_s - 1) must have read them
                        if (!__all_sync(0xffffffffu, mbar_wait(&p_free[t], n_s & 1, abort_flag, 0x310 + t))) ok = false;
                        tc_fence_after();
                    }
                    if (w & 1) tmem_st_32x32b_x16(p_addr + (w >> 1) * 16, pk);
                }
            };
            // The first block of a row takes its max first and then runs the same pass as every other block.
            if (j == 0) m_run = row_max();
            exp_pass((m_run == -INFINITY) ? 0.0f : -m_run * c);
            if (quarter == 0 && lane == 0) MLT_TR(t, j, 3);
            if (j > 0) {
                const float blk = (acc0.x + acc0.y) + (acc1.x + acc1.y);
                const bool moved = !(blk < kRescaleLimit);  // also catches inf and NaN
                if (__any_sync(0xffffffffu, moved)) {
                    // rare: rescale O_t and l by 2^((m_old - m_new)*c) (1 for rows whose reference stays) and redo P.
                    // O_t may be rewritten in place because P_t(j-1) V has landed in it.  D = 128: S_t(j) complete
                    // implies every UMMA issued before Q_t K_j^T, P_t(j-1) V among them.  D = 64: Q_t K_j^T is
                    // issued BEFORE P_t(j-1) V, so s_full says nothing; the guarantee is the p_free[t] wait inside
                    // the first exp_pass (w == 1), which every path to this point has passed.
                    // (A single copy of the pass inside a retry loop was measured 7 % slower.)
                    float alpha = 1.0f;
                    if (moved) {
                        const float mxr = fmaxf(row_max(), m_run);
                        alpha = m_run == -INFINITY ? 0.0f : fast_exp2((m_run - mxr) * c);
                        m_run = mxr;
                    }
#pragma unroll 1
                    for (int q = 0; q < D / 16; ++q) {
                        uint32_t o[16];
                        tmem_ld_32x32b_x16(o_addr + q * 16, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st_32x32b_x16(o_addr + q * 16, o);
                    }
                    l_run *= alpha;
                    exp_pass((m_run == -INFINITY) ? 0.0f : -m_run * c);
                }
            }
            if (!ok) break;
            l_run += (acc0.x + acc0.y) + (acc1.x + acc1.y);
            if (quarter == 0 && lane == 0) MLT_TR(t, j, 5);
            tmem_wait_st();
            if (quarter == 0 && lane == 0) MLT_TR(t, j, 6);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&p_full[t]);
            if (quarter == 0 && lane == 0) MLT_TR(t, j, 4);
        }

        if (!ok) break;
        ok = __all_sync(0xffffffffu, mbar_wait(&o_full[t], n_o & 1, abort_flag, 0x400 + t));
        if (!ok) break;
        ++n_o;
        tc_fence_after();
        if (quarter == 0 && lane == 0) MLT_TRI(t, 16);
        {
            // Once the loads from tensor memory have completed the next item's first P V may overwrite O_t: the
            // softmax of that item, and with it P_t(0), comes after this point in program order.
            const float inv_l = __fdividef(1.0f, l_run);
            const bool valid = qi < p.Nq;
            // 64 columns at a time: BF16 into this warp's 4 KB staging area (32 rows x 128 B in the 128-byte
            // swizzle of the tensor map: 16-byte chunk k of row r sits at chunk k ^ (r & 7)), then one TMA store
            // of the 32 x 64 box; rows beyond Nq are clipped by the tensor map.
            uint8_t* stage_o = smem_stage + warp * 4096;
            const int row0 = it.q_base + t * kMhaBlock + quarter * 32;  // first query row of this warp
#pragma unroll 1
            for (int h = 0; h < D / 64; ++h) {  // a short loop, not unrolled: this code runs once per item
                uint32_t o[2][32];
                tmem_ld_32x32b_x32(o_addr + h * 64, o[0]);
                tmem_ld_32x32b_x32(o_addr + h * 64 + 32, o[1]);
                if (lane == 0) tma_store_wait_read<0>();  // the staging area's previous store has been read out
                __syncwarp();
                tmem_wait_ld();
#pragma unroll
                for (int k = 0; k < 8; ++k) {  // 16-byte chunks of the BF16 half row
                    const uint32_t* w = &o[k >> 2][(k & 3) * 8];
                    uint4 out;
                    out.x = pack_bf16x2(__uint_as_float(w[0]) * inv_l, __uint_as_float(w[1]) * inv_l);
                    out.y = pack_bf16x2(__uint_as_float(w[2]) * inv_l, __uint_as_float(w[3]) * inv_l);
                    out.z = pack_bf16x2(__uint_as_float(w[4]) * inv_l, __uint_as_float(w[5]) * inv_l);
                    out.w = pack_bf16x2(__uint_as_float(w[6]) * inv_l, __uint_as_float(w[7]) * inv_l);
                    *reinterpret_cast<uint4*>(stage_o + lane * 128 + ((k ^ (lane & 7)) * 16)) = out;
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0 && row0 < p.Nq) {
                    tma_store_3d(&tmap_o, stage_o, h * 64, row0, it.bh);
                    tma_store_commit();
                }
            }
            if (valid && p.LSE)
                p.LSE[static_cast<int64_t>(it.bh) * p.Nq + qi] = m_run * p.scale + __log2f(l_run) * 0.6931471805599453f;
        }
        if (quarter == 0 && lane == 0) MLT_TRI(t, 17);
        }  // items
        if (lane == 0) tma_store_wait_all<0>();  // shared memory must outlive the stores that read it
    }

    // common exit: every role reaches this, also after an aborted wait
    tc_fence_before();
    __syncthreads();
    if (blockIdx.x == 0 && threadIdx.x == 0) clock_probe(1, 1);
    if (warp == 8) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// Registers per thread the launch allocation must hold for the hand-over inside the kernel (8 softmax warps at
// 232, 4 other warps at 40): with fewer, setmaxnreg.inc would wait for registers that never come.
constexpr int kMhaMinRegsPerThread = (8 * 32 * kMhaSoftmaxRegs + 4 * 32 * kMhaOtherRegs + kMhaThreads - 1) / kMhaThreads;

// Returns 0, 1 (a CUDA call failed) or 2 (the compiled kernel's register count is below the hand-over budget, e.g.
// after a compiler or flag change: nothing may be launched).
inline int mha_configure() {
    if (cudaFuncSetAttribute(mha_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, MhaSmem<64>::kTotal) !=
        cudaSuccess)
        return 1;
    if (cudaFuncSetAttribute(mha_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, MhaSmem<128>::kTotal) !=
        cudaSuccess)
        return 1;
    cudaFuncAttributes a64, a128;
    if (cudaFuncGetAttributes(&a64, mha_fwd_kernel<64>) != cudaSuccess ||
        cudaFuncGetAttributes(&a128, mha_fwd_kernel<128>) != cudaSuccess)
        return 1;
    if (a64.numRegs < kMhaMinRegsPerThread || a128.numRegs < kMhaMinRegsPerThread) return 2;
    return 0;
}

// Development switch (environment variable MLT_MHA_NO_HALF_ITEMS): hand the last round out as whole items.
inline bool debug_no_half_items() {
    static const bool off = std::getenv("MLT_MHA_NO_HALF_ITEMS") != nullptr;
    return off;
}

inline int mha_launch(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to, float* LSE,
                      int B, int H, int Nq, int Nk, int D, bool causal, float scale, int sm_count, cudaStream_t st,
                      int head_group_override = 0, int grid_override = 0) {
    MhaParams p;
    p.LSE = LSE;
    p.BH = B * H;
    p.Nq = Nq;
    p.Nk = Nk;
    p.causal = causal ? 1 : 0;
    p.scale = scale;
    p.num_pairs = (Nq + 2 * kMhaBlock - 1) / (2 * kMhaBlock);
    const int64_t items = static_cast<int64_t>(p.num_pairs) * p.BH;
    if (items > INT32_MAX - 1024) return 2;
    p.num_items = p.full_items = static_cast<int>(items);
    // Items of equal length (no mask), or many short ones under a causal mask: persistent CTAs, one per SM, which
    // hide each item's fill and drain behind its neighbours.  Causal list order: all heads' last query rows first
    // (longest first over the whole problem), so that the static hand-out balances; otherwise heads go in groups
    // of 8, so that the CTAs running at any time read the K/V of few heads (L2 reuse).
    // Long causal items (more than about 24 K/V blocks on average) gain nothing from the overlap and lose 2-5 % to
    // the static hand-out: there one CTA per item, dispatched by the hardware in list order (longest first inside
    // each group of 8 heads).
    const int64_t avg_blocks = causal ? (Nk / kMhaBlock) / 2 + 1 : Nk / kMhaBlock;
    const bool persistent = !causal || avg_blocks <= 24;
    p.head_group = (causal && persistent) ? p.BH : 8;
    if (head_group_override > 0) p.head_group = head_group_override;
    int grid = static_cast<int>(persistent ? std::min<int64_t>(items, sm_count) : items);
    if (grid_override > 0) grid = static_cast<int>(std::min<int64_t>(items, grid_override));
    if (persistent) {
        // a last round of at most half the CTAs goes out tile by tile (only when every item has two real tiles, so
        // that no entry is empty)
        const int ctas = grid_override > 0 ? grid_override : sm_count;
        const int rem = static_cast<int>(items % ctas);
        const bool two_tiles_each = ((Nq + kMhaBlock - 1) / kMhaBlock) % 2 == 0;
        // (not when the whole problem is one round: 68 items ran 4 % slower as 136 single tiles)
        if (items > ctas && rem > 0 && 2 * rem <= ctas && two_tiles_each && !debug_no_half_items()) {
            p.full_items = static_cast<int>(items) - rem;
            p.num_items = static_cast<int>(items) + rem;
            grid = std::min(p.num_items, ctas);
        }
    }
    if (D == 64)
        mha_fwd_kernel<64><<<grid, kMhaThreads, MhaSmem<64>::kTotal, st>>>(tq, tk, tv, to, p);
    else
        mha_fwd_kernel<128><<<grid, kMhaThreads, MhaSmem<128>::kTotal, st>>>(tq, tk, tv, to, p);
    return cudaGetLastError() == cudaSuccess ? 0 : 4;
}

}  // namespace mlt
