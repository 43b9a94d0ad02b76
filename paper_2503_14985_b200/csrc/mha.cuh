// Multi-head attention forward in the FlashAttention-2 form (paper Sec. 2.5,
// Algorithm 1): per block of query rows, loop over K/V blocks; S = Q K_j^T on the
// tensor cores, online softmax with running row max m and row sum l, O += P V_j on
// the tensor cores, final O / l and LSE = m + ln l.
//
// A CTA owns 256 query rows of one (batch, head): two 128-row tiles that take turns
// on the tensor pipe, so the exponentials of one tile overlap the products of the other.
//   warps 0-3   softmax / O-rescale / epilogue of tile 0 (one thread per query row)
//   warps 4-7   the same for tile 1
//   warp  8     UMMA issuer (the whole warp runs the loop, one elected lane issues) and owner of the
//               tensor-memory allocation; it serves the tiles in a fixed order (P V of tile 0, next
//               Q K^T of tile 0, the same for tile 1), which keeps the two softmax warpgroups half a
//               period apart
//   warp  9     TMA loader (one lane): both Q tiles once, then K_0, V_0, K_1, V_1, ... through a ring;
//               it also initialises the barriers and issues the first loads before the CTA-wide sync
//   warps 10-11 idle (they complete the third warpgroup for the register hand-over)
// Tensor memory (512 columns): S_0 | S_1 (128 FP32 columns each; the BF16 P of a tile
// overwrites the first 64 columns of its S and is consumed from there as the A operand
// of P V), then O_0 | O_1 (D FP32 columns each).
//
// Measured on B200 (what shaped this kernel):
//  * a UMMA of 128x128x16 takes 64 clocks, also with A from tensor memory; issuing one costs the issuing
//    thread about 46 clocks from a single divergent lane and about 20 from warp-uniform code with an elected
//    lane; a warp that shares its scheduler partition with a busy warp is served much more rarely;
//  * per tile and K/V block the chain is: S ready -> TMEM load (125) -> softmax (about 1700: 1024 MUFU clocks
//    plus the packed FP32 work a single warp per partition cannot fully overlap) -> P V and next Q K^T
//    (about 1085) -> S ready; with two tiles half a period apart the period is about 3230 clocks, i.e. the
//    tensor pipe is busy about two thirds of the time.
#pragma once

#include <math.h>

#include "ptx.cuh"

namespace mlt {

constexpr int kMhaBlock = 128;   // query rows per tile and keys per K/V block
constexpr int kMhaThreads = 384; // three warpgroups
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleLimit = 18446744073709551616.0f;  // 2^64: a block sum at or above it forces a new reference max

template <int D>
struct MhaSmem {
    static constexpr int kTileBytes = kMhaBlock * D * 2;  // one Q, K or V tile: D/64 chunks of 128 rows x 128 B
    static constexpr int kChunkBytes = kMhaBlock * 128;
    static constexpr int kStages = (D == 128) ? 4 : 8;
    static constexpr int kBarrierBytes = 512;
    static constexpr int kTotal = 2 * kTileBytes + kStages * kTileBytes + kBarrierBytes + 1024;
};

struct MhaParams {
    __nv_bfloat16* O;
    float* LSE;  // may be null
    int BH, Nq, Nk;
    int causal;
    float scale;
    int num_pairs;   // 256-row query groups per head
    int head_group;  // heads that share a span of consecutive block indices
};

// block index -> (pair, bh).  Heads are taken in groups; inside a group the query
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

// 2^x for a pair of values on the FMA pipe (no MUFU): round-to-nearest split x = r + f, |f| <= 0.5, cubic for
// 2^f (relative error < 8e-5, far below the BF16 rounding of P), then r is added to the exponent field.
// x is clamped at -126 (2^x ~ 1e-38 stands for 0).
__device__ __forceinline__ float2 exp2_poly2(float2 x) {
    x.x = fmaxf(x.x, -126.0f);
    x.y = fmaxf(x.y, -126.0f);
    const float kMagic = 12582912.0f;  // 1.5 * 2^23: adding it leaves round(x) in the low mantissa bits
    const float2 t = fadd2(x, make_float2(kMagic, kMagic));
    const float2 r = fadd2(t, make_float2(-kMagic, -kMagic));
    const float2 f = ffma2(r, make_float2(-1.0f, -1.0f), x);
    float2 y = ffma2(f, make_float2(0.05508868396282196f, 0.05508868396282196f),
                     make_float2(0.24260404706001282f, 0.24260404706001282f));
    y = ffma2(y, f, make_float2(0.6932762265205383f, 0.6932762265205383f));
    y = ffma2(y, f, make_float2(0.9999289512634277f, 0.9999289512634277f));
    y.x = __int_as_float(__float_as_int(y.x) + (__float_as_int(t.x) << 23));
    y.y = __int_as_float(__float_as_int(y.y) + (__float_as_int(t.y) << 23));
    return y;
}

template <int D>
__global__ void __launch_bounds__(kMhaThreads, 1)
mha_fwd_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v, const MhaParams p) {
    using L = MhaSmem<D>;
    constexpr int kStages = L::kStages;
    constexpr int kChunks = D / 64;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* smem_q = smem;                        // [2][tile]
    uint8_t* smem_kv = smem + 2 * L::kTileBytes;   // [kStages][tile]
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_kv + kStages * L::kTileBytes);
    uint64_t* q_full = bars;                  // [1]
    uint64_t* kv_full = bars + 1;             // [kStages]
    uint64_t* kv_empty = kv_full + kStages;   // [kStages]
    uint64_t* s_full = kv_empty + kStages;    // [2]  UMMA -> softmax: S_t(j) complete
    uint64_t* p_full = s_full + 2;            // [2]  softmax -> UMMA: P_t(j) in TMEM, O_t rescaled
    uint64_t* o_full = p_full + 2;            // [2]  UMMA -> epilogue: O_t complete
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(o_full + 2);
    volatile uint32_t* abort_flag = tmem_base_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    int pair, bh;
    mha_item(p, blockIdx.x, pair, bh);
    const int q_base = pair * 2 * kMhaBlock;
    const int shift = p.Nk - p.Nq;  // bottom-right alignment of the causal mask
    // number of K/V blocks each tile needs
    int J[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int q0 = q_base + t * kMhaBlock;
        if (q0 >= p.Nq) {
            J[t] = 0;
        } else {
            int last_key = p.Nk - 1;
            if (p.causal) last_key = min(last_key, min(q0 + kMhaBlock, p.Nq) - 1 + shift);
            J[t] = last_key / kMhaBlock + 1;
        }
    }
    const int Jmax = max(J[0], J[1]);

    // The loader lane initialises the barriers and issues the first loads (Q and the first K/V tiles: the ring
    // is empty, nothing to wait for) before the CTA-wide sync, so they overlap the tensor-memory allocation.
    int pre_tiles = 0;  // ring tiles already requested (K_0, V_0, K_1, ...)
    if (warp == 9 && lane == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&kv_full[s], 1);
            mbar_init(&kv_empty[s], 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(&s_full[t], 1);
            mbar_init(&p_full[t], 4);  // one arrive per softmax warp
            mbar_init(&o_full[t], 1);
        }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_q);
        prefetch_tensormap(&tmap_k);
        prefetch_tensormap(&tmap_v);
        // K_0 first: with Q it is all the first product needs
        pre_tiles = min(2 * Jmax, kStages);
        for (int i = 0; i < pre_tiles; ++i) {
            if (i == 1) {
                mbar_arrive_expect_tx(q_full, 2 * L::kTileBytes);
#pragma unroll
                for (int t = 0; t < 2; ++t)
#pragma unroll
                    for (int c = 0; c < kChunks; ++c)
                        tma_load_3d(smem_q + t * L::kTileBytes + c * L::kChunkBytes, &tmap_q, q_full, c * 64,
                                    q_base + t * kMhaBlock, bh);
            }
            uint8_t* dst = smem_kv + i * L::kTileBytes;
            mbar_arrive_expect_tx(&kv_full[i], L::kTileBytes);
#pragma unroll
            for (int c = 0; c < kChunks; ++c)
                tma_load_3d(dst + c * L::kChunkBytes, (i & 1) == 0 ? &tmap_k : &tmap_v, &kv_full[i], c * 64,
                            (i >> 1) * kMhaBlock, bh);
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

    if (warp >= 10) {
        setmaxnreg_dec<40>();  // only hand their registers over
    } else if (warp == 9) {
        // ------------------------------- loader -------------------------------
        setmaxnreg_dec<40>();
        if (lane == 0) {
            int stage = pre_tiles == kStages ? 0 : pre_tiles;
            uint32_t phase = pre_tiles == kStages ? 1 : 0;
            bool ok = true;
            for (int i = pre_tiles; i < 2 * Jmax && ok; ++i) {
                ok = mbar_wait(&kv_empty[stage], phase ^ 1, abort_flag, 0x100 + stage);
                if (!ok) break;
                uint8_t* dst = smem_kv + stage * L::kTileBytes;
                mbar_arrive_expect_tx(&kv_full[stage], L::kTileBytes);
#pragma unroll
                for (int c = 0; c < kChunks; ++c)
                    tma_load_3d(dst + c * L::kChunkBytes, (i & 1) == 0 ? &tmap_k : &tmap_v, &kv_full[stage], c * 64,
                                (i >> 1) * kMhaBlock, bh);
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == 8) {
        // ------------------------------- UMMA issuer -------------------------------
        // The whole warp runs this code (uniform control flow keeps addresses and descriptors in the uniform
        // datapath: an issue costs about 20 clocks instead of about 46 from a single divergent lane); one
        // elected lane executes the tcgen05 instructions.
        setmaxnreg_dec<40>();
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
                const uint32_t a0 = tmem_base + kColS + t * kMhaBlock;
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
            bool ok = true;
            if (Jmax > 0) {
                ok = wait_all(q_full, 0, 0x200);
                if (ok) ok = wait_all(&kv_full[stage], phase, 0x210 + stage);
                if (ok) {
                    tc_fence_after();
                    for (int t = 0; t < 2; ++t)
                        if (J[t] > 0) issue_qk(t, stage);
                    if (leader) umma_commit(&kv_empty[stage]);
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
            }
            for (int j = 0; j < Jmax && ok; ++j) {
                const int vslot = stage;
                ok = wait_all(&kv_full[vslot], phase, 0x220 + vslot);
                if (!ok) break;
                if (++stage == kStages) { stage = 0; phase ^= 1; }
                const int kslot = stage;  // K_{j+1}, if there is one
                bool k_ready = false;
                for (int t = 0; t < 2 && ok; ++t) {
                    if (j >= J[t]) continue;
                    ok = wait_all(&p_full[t], j & 1, 0x230 + t);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(t, vslot, j == 0);
                    if (j == J[t] - 1 && leader) umma_commit(&o_full[t]);
                    if (j + 1 < J[t]) {
                        if (!k_ready) {
                            ok = wait_all(&kv_full[kslot], phase, 0x240 + kslot);
                            if (!ok) break;
                            tc_fence_after();
                            k_ready = true;
                        }
                        issue_qk(t, kslot);
                    }
                }
                if (!ok) break;
                if (leader) umma_commit(&kv_empty[vslot]);
                if (j + 1 < Jmax) {
                    if (leader) umma_commit(&kv_empty[kslot]);
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else {
        // ------------------- softmax, O rescale and epilogue of tile t -------------------
        setmaxnreg_inc<232>();
        const int t = warp >> 2;
        const int quarter = warp & 3;
        const int row_in_tile = quarter * 32 + lane;
        const int qi = q_base + t * kMhaBlock + row_in_tile;  // query index inside the head
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const uint32_t s_addr = lane_addr + kColS + t * kMhaBlock;
        const uint32_t o_addr = lane_addr + kColO + t * D;
        const float c = p.scale * kLog2e;
        const int Jt = J[t];
        const int limit = p.causal ? min(p.Nk - 1, qi + shift) : p.Nk - 1;  // last visible key of this row
        float m_run = -INFINITY;  // reference max (raw score units); may lag the true max by < 2^8 in exp2 units
        float l_run = 0.0f;
        bool ok = true;

        for (int j = 0; j < Jt; ++j) {
            ok = __all_sync(0xffffffffu, mbar_wait(&s_full[t], j & 1, abort_flag, 0x300 + t));
            if (!ok) break;
            tc_fence_after();
            uint32_t s[4][32];  // this thread's row of S: 4 chunks of 32 keys
#pragma unroll
            for (int q = 0; q < 4; ++q) tmem_ld_32x32b_x32(s_addr + q * 32, s[q]);
            tmem_wait_ld();
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
                const float2 c2 = make_float2(c, c), n2 = make_float2(neg_mc, neg_mc);
                acc0 = make_float2(0.0f, 0.0f);
                acc1 = make_float2(0.0f, 0.0f);
                uint32_t pk[16];
#pragma unroll
                for (int w = 0; w < 8; ++w) {  // waves of 16 keys
#pragma unroll
                    for (int i = 0; i < 8; i += 2) {
                        const int k = w * 16 + 2 * i;
                        float2 x0 = ffma2(make_float2(__uint_as_float(s[k >> 5][k & 31]), __uint_as_float(s[k >> 5][(k & 31) + 1])), c2, n2);
                        float2 x1 = ffma2(make_float2(__uint_as_float(s[k >> 5][(k & 31) + 2]), __uint_as_float(s[k >> 5][(k & 31) + 3])), c2, n2);
                        x0.x = fast_exp2(x0.x);
                        x0.y = fast_exp2(x0.y);
                        if (D == 64 && (i / 2) % 2 == 0) {  // D = 64 is MUFU-bound: a quarter of the exponentials go to the FMA pipe
                            x1 = exp2_poly2(x1);
                        } else {
                            x1.x = fast_exp2(x1.x);
                            x1.y = fast_exp2(x1.y);
                        }
                        acc0 = fadd2(acc0, x0);
                        acc1 = fadd2(acc1, x1);
                        pk[(w & 1) * 8 + i] = pack_bf16x2(x0.x, x0.y);
                        pk[(w & 1) * 8 + i + 1] = pack_bf16x2(x1.x, x1.y);
                    }
                    if (w & 1) tmem_st_32x32b_x16(s_addr + (w >> 1) * 16, pk);
                }
            };
            if (j == 0) {
                m_run = row_max();  // no reference yet
                exp_pass((m_run == -INFINITY) ? 0.0f : -m_run * c);
            } else {
                exp_pass((m_run == -INFINITY) ? 0.0f : -m_run * c);
                const float blk = (acc0.x + acc0.y) + (acc1.x + acc1.y);
                const bool moved = !(blk < kRescaleLimit);  // also catches inf and NaN
                if (__any_sync(0xffffffffu, moved)) {
                    // rare: rescale O_t and l by 2^((m_old - m_new)*c) (1 for rows whose reference stays) and redo P.
                    // S_t(j) complete implies every earlier UMMA, so P_t(j-1) V has landed in O_t.
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
            l_run += (acc0.x + acc0.y) + (acc1.x + acc1.y);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&p_full[t]);
        }

        if (ok && Jt > 0) {
            ok = __all_sync(0xffffffffu, mbar_wait(&o_full[t], 0, abort_flag, 0x400 + t));
            if (ok) {
                tc_fence_after();
                const float inv_l = 1.0f / l_run;
                const bool valid = qi < p.Nq;
                // O / l -> BF16 into the tile's Q region (no product reads it any more), 16-byte chunks XOR-swizzled
                // by row; then each warp writes its own 32 rows out row-major, 512 contiguous bytes per instruction.
                constexpr int kRowChunks = D / 8;  // 16-byte chunks per row
                uint8_t* stage_o = smem_q + t * L::kTileBytes;
                {
                    uint32_t o[D / 32][32];  // the whole row at once: one TMEM round trip instead of eight
#pragma unroll
                    for (int q = 0; q < D / 32; ++q) tmem_ld_32x32b_x32(o_addr + q * 32, o[q]);
                    tmem_wait_ld();
#pragma unroll
                    for (int k = 0; k < D / 8; ++k) {  // 16-byte chunks of the BF16 row
                        const uint32_t* w = &o[k >> 2][(k & 3) * 8];
                        uint4 out;
                        out.x = pack_bf16x2(__uint_as_float(w[0]) * inv_l, __uint_as_float(w[1]) * inv_l);
                        out.y = pack_bf16x2(__uint_as_float(w[2]) * inv_l, __uint_as_float(w[3]) * inv_l);
                        out.z = pack_bf16x2(__uint_as_float(w[4]) * inv_l, __uint_as_float(w[5]) * inv_l);
                        out.w = pack_bf16x2(__uint_as_float(w[6]) * inv_l, __uint_as_float(w[7]) * inv_l);
                        const int chunk = k ^ (row_in_tile & (kRowChunks - 1));
                        *reinterpret_cast<uint4*>(stage_o + row_in_tile * (D * 2) + chunk * 16) = out;
                    }
                }
                __syncwarp();
                constexpr int kRowsPerStore = 32 / kRowChunks;
                __nv_bfloat16* obase = p.O + (static_cast<int64_t>(bh) * p.Nq + q_base + t * kMhaBlock) * D;
#pragma unroll
                for (int r0 = 0; r0 < 32; r0 += kRowsPerStore) {
                    const int rr = quarter * 32 + r0 + lane / kRowChunks;
                    const int cc = lane % kRowChunks;
                    const uint4 v = *reinterpret_cast<const uint4*>(stage_o + rr * (D * 2) + ((cc ^ (rr & (kRowChunks - 1))) * 16));
                    if (q_base + t * kMhaBlock + rr < p.Nq) *reinterpret_cast<uint4*>(obase + rr * D + cc * 8) = v;
                }
                if (valid && p.LSE) p.LSE[static_cast<int64_t>(bh) * p.Nq + qi] = m_run * p.scale + logf(l_run);
            }
        }
    }

    // common exit: every role reaches this, also after an aborted wait
    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

inline int mha_configure() {
    if (cudaFuncSetAttribute(mha_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, MhaSmem<64>::kTotal) !=
        cudaSuccess)
        return 1;
    if (cudaFuncSetAttribute(mha_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, MhaSmem<128>::kTotal) !=
        cudaSuccess)
        return 1;
    return 0;
}

inline int mha_launch(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, __nv_bfloat16* O, float* LSE,
                      int B, int H, int Nq, int Nk, int D, bool causal, float scale, int sm_count, cudaStream_t st) {
    (void)sm_count;
    MhaParams p;
    p.O = O;
    p.LSE = LSE;
    p.BH = B * H;
    p.Nq = Nq;
    p.Nk = Nk;
    p.causal = causal ? 1 : 0;
    p.scale = scale;
    p.num_pairs = (Nq + 2 * kMhaBlock - 1) / (2 * kMhaBlock);
    p.head_group = 8;
    const int64_t items = static_cast<int64_t>(p.num_pairs) * p.BH;
    if (items > INT32_MAX) return 2;
    const int grid = static_cast<int>(items);
    if (D == 64)
        mha_fwd_kernel<64><<<grid, kMhaThreads, MhaSmem<64>::kTotal, st>>>(tq, tk, tv, p);
    else
        mha_fwd_kernel<128><<<grid, kMhaThreads, MhaSmem<128>::kTotal, st>>>(tq, tk, tv, p);
    return cudaGetLastError() == cudaSuccess ? 0 : 4;
}

}  // namespace mlt
