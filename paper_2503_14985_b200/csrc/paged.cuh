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
    const int len = max(0, min(p.seq_lens[row / p.H], p.max_blocks * p.block_size));  // as in the decode kernel
    const int nblk = (len + p.block_size - 1) / p.block_size;
    const int used = max(1, min(p.splits, (nblk + p.blocks_per_split - 1) / p.blocks_per_split));  // splits that wrote
    // Launched with programmatic stream serialisation: the CTAs may start while the decode kernel is still
    // running (which hides this kernel's launch latency) and wait here until all of its writes are visible.
    cudaGridDependencySynchronize();
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
    const float* po = p.part_o + row * p.splits * D + d;
    float ot = 0.0f;
    int sp = 0;
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

template <int D, int G>
int paged_launch_bs(const PagedParams& p, cudaStream_t st) {
    const dim3 grid(p.splits, p.H_kv * p.head_groups, p.num_seqs);
    switch (p.block_size) {
        case 8: paged_decode_kernel<D, G, 8><<<grid, kPagedThreads, 0, st>>>(p); break;
        case 16: paged_decode_kernel<D, G, 16><<<grid, kPagedThreads, 0, st>>>(p); break;
        case 32: paged_decode_kernel<D, G, 32><<<grid, kPagedThreads, 0, st>>>(p); break;
        default: return 2;
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
        case 8: {
            // 8 heads per CTA need 255 registers and leave two CTAs per SM; two CTAs of 4 heads run faster
            PagedParams p2 = p;
            p2.head_groups = 2;
            return paged_launch_bs<D, 4>(p2, st);
        }
        default: return 2;
    }
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
