// BF16 GEMM C = A * B with FP32 accumulation in tensor memory (paper Sec. 2,
// Listing 2: per output tile, a K loop of tile dots into a zero-initialised
// accumulator, then one store).
//
// One persistent CTA per SM, 6 warps with fixed roles:
//   warp 0      TMA producer: A tile (BM x 64, K-major) and B tile (64 x BN, N contiguous) per stage
//   warp 1      UMMA issuer (one elected lane) and owner of the tensor-memory allocation
//   warps 2-5   epilogue: TMEM -> registers -> BF16 -> global, overlapped with the next tile's main loop
// Tile 128 x BN x 64, kStages-deep smem ring guarded by full/empty mbarriers; two
// accumulators in TMEM (2 x BN columns) guarded by acc_full/acc_empty mbarriers.
// Large problems run on CTA pairs (256 x 256 tiles, tcgen05.mma.cta_group::2; see gemm_bf16_pair_kernel).
//
// The same kernels serve three destinations of the accumulators (gemm_store_chunk / gemm_store_chunk_tma):
//   BF16 C        one rounding to nearest even, 16-byte stores from the thread that owns the row
//   FP32 partial  split-K: work item = (tile, K slice), a second kernel sums the slices in a fixed order
//   FP32 C        FP16 or BF16 operands, result through a shared-memory box and a TMA store, or a TMA
//                 add-reduction for C += A * B (template parameter kCTma: its own instantiation, so the BF16
//                 path keeps its registers and code size)
#pragma once

#include "ptx.cuh"

namespace mlt {

constexpr int kGemmBM = 128;
constexpr int kGemmBK = 64;
constexpr int kGemmThreads = 192;

// FP32 output goes through shared memory and TMA: two 4 KB boxes (32 rows x 32 FP32 columns) per epilogue warp
constexpr int kGemmStagingBytes = 4 * 2 * 4096;

// BF16 output of the 128 x 128 kernel: each epilogue warp stages 32 rows x 64 columns (128 bytes per row, pitch 144:
// the 16-byte row writes of 8 lanes and the 128-byte row reads of 8 lanes both touch every bank once)
constexpr int kGemmBf16StagePitch = 144;

template <int BN, int kStages>
struct GemmSmem {
    static constexpr int kABytes = kGemmBM * kGemmBK * 2;  // 16 KB
    static constexpr int kBBytes = kGemmBK * BN * 2;       // 64 rows x BN, as BN/64 boxes of 64 x 64
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kBarrierBytes = 256;
    // stages | barriers (padded to 1 KB) | staging for FP32 output (only requested by launches that write FP32 C)
    static constexpr int kNoStaging = kStages * kStageBytes + 1024 + 1024;  // + alignment slack
    static constexpr int kTotal = kNoStaging + kGemmStagingBytes;
    // BF16 output of the 128-wide kernel goes through a small staging area (see gemm_store_half_coalesced)
    static constexpr int kBf16Staging = kNoStaging + 4 * 32 * kGemmBf16StagePitch;
};

struct GemmParams {
    __nv_bfloat16* C;
    int64_t ldc;
    int M, N, K;
    int tiles_m, tiles_n;
    int group_m;  // M-tiles per raster group
    // split-K (single-CTA kernel only): work item = (tile, K slice); a slice covers kb_per_split blocks of 64 and
    // its FP32 partial tile goes to partial[slice][M][N], which gemm_splitk_reduce_kernel sums and rounds.
    int split_k;       // 1: no split, the epilogue writes BF16 C
    int kb_per_split;
    float* partial;
    // Even K hand-out (single-CTA kernel, with scratch): all (tile, K block) units in tile order are cut into one
    // contiguous share of `even_units` per CTA, whatever tiles a share touches; a CTA writes one FP32 partial per tile
    // it touches, into slot (its index) - (index of the first CTA that touches the tile).  0: off.
    int even_units;
    // FP16-input / FP32-output variant (the dtypes of the paper's Listing 2) and its accumulate form C += A*B
    float* Cf;         // non-null: FP32 output with pitch ldcf instead of BF16 C
    int64_t ldcf;
    int accumulate;    // with Cf: add to the prior contents of C (the "C += A*B" of Sec. 2)
    // CTA-pair kernel: work items 0 .. full_items-1 are whole 256 x 256 tiles; the tiles after them (a last wave that
    // would occupy at most half of the SM pairs) are cut into two 256 x 128 halves, one item each
    int full_items, num_items;
    uint32_t f16_inputs;  // 0: BF16 operands, 1: FP16 operands (same tiles and descriptors, other format field)
};

// Instruction descriptor with the operand format chosen at run time (BF16: format 1, FP16: format 0).
__device__ __forceinline__ uint32_t gemm_idesc(uint32_t m, uint32_t n, uint32_t f16_inputs) {
    const uint32_t bf16 = make_idesc_bf16(m, n, /*a_mn_major=*/false, /*b_mn_major=*/true);
    return f16_inputs ? (bf16 & ~((7u << 7) | (7u << 10))) : bf16;
}

// One row segment of 32 accumulator columns (TMEM -> registers) to its destination: the split-K FP32 partial, the
// FP32 C (optionally added to what is there), or BF16 C.  Ragged right edges fall back to element stores.
__device__ __forceinline__ void gemm_store_chunk(const GemmParams& p, const uint32_t (&v)[32], int row, int col0, int slice) {
    if (row >= p.M) return;
    float* frow = p.partial ? p.partial + (static_cast<int64_t>(slice) * p.M + row) * p.N
                            : (p.Cf ? p.Cf + static_cast<int64_t>(row) * p.ldcf : nullptr);
    if (frow) {
        const bool add = !p.partial && p.accumulate;
        const bool vec_ok = p.partial ? (p.N & 3) == 0 : true;  // partial rows are N floats apart; C rows are aligned
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int col = col0 + q * 4;
            if (col + 4 <= p.N && vec_ok) {
                float4 o = make_float4(__uint_as_float(v[q * 4]), __uint_as_float(v[q * 4 + 1]), __uint_as_float(v[q * 4 + 2]),
                                       __uint_as_float(v[q * 4 + 3]));
                if (add) {
                    const float4 c = *reinterpret_cast<const float4*>(frow + col);
                    o.x += c.x; o.y += c.y; o.z += c.z; o.w += c.w;
                }
                *reinterpret_cast<float4*>(frow + col) = o;
            } else {
                for (int j = 0; j < 4 && col + j < p.N; ++j)
                    frow[col + j] = __uint_as_float(v[q * 4 + j]) + (add ? frow[col + j] : 0.0f);
            }
        }
        return;
    }
    __nv_bfloat16* crow = p.C + static_cast<int64_t>(row) * p.ldc;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const int col = col0 + q * 8;
        uint4 out;
        out.x = pack_bf16x2(__uint_as_float(v[q * 8 + 0]), __uint_as_float(v[q * 8 + 1]));
        out.y = pack_bf16x2(__uint_as_float(v[q * 8 + 2]), __uint_as_float(v[q * 8 + 3]));
        out.z = pack_bf16x2(__uint_as_float(v[q * 8 + 4]), __uint_as_float(v[q * 8 + 5]));
        out.w = pack_bf16x2(__uint_as_float(v[q * 8 + 6]), __uint_as_float(v[q * 8 + 7]));
        if (col + 8 <= p.N) {
            *reinterpret_cast<uint4*>(crow + col) = out;
        } else if (col < p.N) {
            const uint32_t w[4] = {out.x, out.y, out.z, out.w};
#pragma unroll
            for (int j = 0; j < 8; ++j)  // constant indices keep w in registers
                if (col + j < p.N)
                    crow[col + j] = __ushort_as_bfloat16(static_cast<unsigned short>(w[j >> 1] >> ((j & 1) * 16)));
        }
    }
}

// 32 rows x 64 accumulator columns of one epilogue warp to BF16 C through shared memory: lane = row writes its 128
// bytes into the staging row, then 8 lanes per row copy 4 rows per instruction to C, so a store instruction covers
// 4 lines of 128 bytes instead of 32 lines of 16 bytes (the per-row stores of gemm_store_chunk take about 2000
// clocks per 128 x 128 tile in the load/store unit, which shows when the epilogue is not hidden behind a next tile).
// Whole tiles only: the caller keeps ragged right edges on the per-row path.
__device__ __forceinline__ void gemm_store_half_coalesced(const GemmParams& p, uint8_t* stg, const uint32_t (&v)[2][32],
                                                          int lane, int row0, int col0) {
    uint4* mine = reinterpret_cast<uint4*>(stg + lane * kGemmBf16StagePitch);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const uint32_t* w = &v[q >> 2][(q & 3) * 8];
        mine[q] = make_uint4(pack_bf16x2(__uint_as_float(w[0]), __uint_as_float(w[1])),
                             pack_bf16x2(__uint_as_float(w[2]), __uint_as_float(w[3])),
                             pack_bf16x2(__uint_as_float(w[4]), __uint_as_float(w[5])),
                             pack_bf16x2(__uint_as_float(w[6]), __uint_as_float(w[7])));
    }
    __syncwarp();
    const int sub = lane >> 3, unit = lane & 7;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = i * 4 + sub;
        const uint4 x = *reinterpret_cast<const uint4*>(stg + r * kGemmBf16StagePitch + unit * 16);
        if (row0 + r < p.M)
            *reinterpret_cast<uint4*>(p.C + static_cast<int64_t>(row0 + r) * p.ldc + col0 + unit * 8) = x;
    }
    __syncwarp();  // the staging rows are rewritten by the next call
}

// The same segment for a whole warp when C is FP32 and reached through a tensor map (p.c_tma): the warp's 32 rows
// x 32 columns go into a 4 KB staging box (128-byte rows, 16-byte chunk k of row r at chunk k ^ (r & 7): the
// 128-byte swizzle of the map) and one lane issues a TMA store, or a TMA add-reduction for C += A * B, which adds
// at the destination and reads nothing back.  Edges are clipped by the tensor map.  `stg` alternates between
// two boxes; at most one newer store may still be reading the other box when this one is refilled.
__device__ __forceinline__ void gemm_store_chunk_tma(const GemmParams& p, const CUtensorMap* tmap_c, uint8_t* stg,
                                                     const uint32_t (&v)[32], int lane, int row0, int col0) {
    if (lane == 0) tma_store_wait_read<1>();
    __syncwarp();
#pragma unroll
    for (int k = 0; k < 8; ++k)
        *reinterpret_cast<uint4*>(stg + lane * 128 + ((k ^ (lane & 7)) * 16)) =
            make_uint4(v[k * 4], v[k * 4 + 1], v[k * 4 + 2], v[k * 4 + 3]);
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
        if (row0 < p.M && col0 < p.N) {
            if (p.accumulate)
                tma_reduce_add_2d(tmap_c, stg, col0, row0);
            else
                tma_store_2d(tmap_c, stg, col0, row0);
        }
        tma_store_commit();  // also when nothing was stored: the group count is what the wait above relies on
    }
    // The store works in 16-byte units, so the tensor map covers only the columns below N rounded down to a
    // multiple of 4; the up to three columns beyond are written by the thread that owns the row.
    const int n4 = p.N & ~3;
    if (n4 != p.N && col0 <= n4 && n4 < col0 + 32 && row0 + lane < p.M) {
        float* crow = p.Cf + static_cast<int64_t>(row0 + lane) * p.ldcf;
#pragma unroll
        for (int j = 0; j < 32; ++j) {  // constant indices keep v in registers
            const int col = col0 + j;
            if (col >= n4 && col < p.N) crow[col] = p.accumulate ? crow[col] + __uint_as_float(v[j]) : __uint_as_float(v[j]);
        }
    }
}

// CTA-pair kernel: work item -> (tile, first column inside the tile, width)
__device__ __forceinline__ void gemm_pair_item(const GemmParams& p, int item, int& tile, int& n_off, int& bn) {
    if (item < p.full_items) {
        tile = item;
        n_off = 0;
        bn = 256;
    } else {
        const int r = item - p.full_items;
        tile = p.full_items + (r >> 1);
        n_off = (r & 1) * 128;
        bn = 128;
    }
}

// tile index -> (tile_m, tile_n): groups of `group_m` M-tiles, M fastest inside a group, so that
// the CTAs running at the same time share few A and B panels (L2 reuse).
__device__ __forceinline__ void gemm_tile_coords(const GemmParams& p, int tile, int& tm, int& tn) {
    const int per_group = p.group_m * p.tiles_n;
    const int g = tile / per_group;
    const int first_m = g * p.group_m;
    const int rows = min(p.group_m, p.tiles_m - first_m);
    const int r = tile - g * per_group;
    tm = first_m + r % rows;
    tn = r / rows;
}

// The pieces of work of one CTA of the single-CTA kernel, in the order every role walks them: (tile, K slice) items
// handed out with a stride of the grid, or (even K hand-out) the pieces of the CTA's contiguous share of all
// (tile, K block) units.
struct GemmWork {
    int tile, kb0, kb1, slot;
};
struct GemmWorkIter {
    long long u, u_end;  // even hand-out: next unit, end of the share
    int item;            // strided hand-out: next item
    __device__ __forceinline__ GemmWorkIter(const GemmParams& p, int num_kb) {
        item = static_cast<int>(blockIdx.x);
        const long long total = static_cast<long long>(p.tiles_m) * p.tiles_n * num_kb;
        u = static_cast<long long>(blockIdx.x) * p.even_units;
        u_end = min(total, u + p.even_units);
    }
    __device__ __forceinline__ bool next(const GemmParams& p, int num_kb, GemmWork& w) {
        if (p.even_units > 0) {
            if (u >= u_end) return false;
            w.tile = static_cast<int>(u / num_kb);
            w.kb0 = static_cast<int>(u - static_cast<long long>(w.tile) * num_kb);
            w.kb1 = static_cast<int>(min(static_cast<long long>(num_kb), w.kb0 + (u_end - u)));
            w.slot = static_cast<int>(blockIdx.x) - static_cast<int>(static_cast<long long>(w.tile) * num_kb / p.even_units);
            u += w.kb1 - w.kb0;
            return true;
        }
        if (item >= p.tiles_m * p.tiles_n * p.split_k) return false;
        w.tile = item / p.split_k;
        w.slot = item % p.split_k;
        w.kb0 = w.slot * p.kb_per_split;
        w.kb1 = min(num_kb, w.kb0 + p.kb_per_split);
        item += static_cast<int>(gridDim.x);
        return true;
    }
};

#ifdef MLT_TRACE
// development builds: SM clock at a few points of CTA 0 of gemm_bf16_kernel
__device__ long long g_gemm_trace[16];
#define MLT_GT(i) do { if (blockIdx.x == 0 && (threadIdx.x & 31) == 0) g_gemm_trace[i] = clock64(); } while (0)
#define MLT_GT_NS(i) do { if (blockIdx.x == 0 && threadIdx.x == 0) { unsigned long long ns_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns_)); g_gemm_trace[i] = static_cast<long long>(ns_); } } while (0)
#else
#define MLT_GT_NS(i) do { } while (0)
#define MLT_GT(i) do { } while (0)
#endif

template <int BN, int kStages, bool kCTma>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                 const __grid_constant__ CUtensorMap tmap_c, const GemmParams p) {
    using L = GemmSmem<BN, kStages>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * L::kStageBytes);
    // 1024-byte aligned (swizzle atoms of the TMA store); present only when the launch asked for it (p.c_tma)
    uint8_t* smem_staging = smem + kStages * L::kStageBytes + 1024;
    uint64_t* full = bars;                     // [kStages]  TMA -> MMA
    uint64_t* empty = bars + kStages;          // [kStages]  MMA -> TMA
    uint64_t* acc_full = bars + 2 * kStages;   // [2]        MMA -> epilogue
    uint64_t* acc_empty = acc_full + 2;        // [2]        epilogue -> MMA
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile uint32_t* abort_flag = tmem_base_slot + 1;

    if (p.split_k > 1) pdl_launch_dependents();  // the reduce kernel's CTAs take the slots this grid's CTAs leave
    const int warp = threadIdx.x >> 5;
    if (blockIdx.x == 0 && threadIdx.x == 0) clock_probe(0, 0);
    if (threadIdx.x == 0) MLT_GT(0);
    MLT_GT_NS(6);
    const int lane = threadIdx.x & 31;
    const int num_kb = (p.K + kGemmBK - 1) / kGemmBK;
    constexpr uint32_t kTmemCols = 2 * BN;  // 512 for BN = 256, 256 for BN = 128

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&acc_full[a], 1);
            mbar_init(&acc_empty[a], 4);  // one arrive per epilogue warp
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0 && lane == 0) {
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc(tmem_base_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_slot;
    if (threadIdx.x == 0) MLT_GT(1);

    if (warp == 0) {
        // ----------------------------- producer -----------------------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            GemmWorkIter work(p, num_kb);
            GemmWork w;
            while (ok && work.next(p, num_kb, w)) {
                int tm, tn;
                gemm_tile_coords(p, w.tile, tm, tn);
                const int m0 = tm * kGemmBM, n0 = tn * BN;
                for (int kb = w.kb0; kb < w.kb1; ++kb) {
                    ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag, 0x100 + stage);
                    if (!ok) break;
                    uint8_t* sa = smem + stage * L::kStageBytes;
                    uint8_t* sb = sa + L::kABytes;
                    mbar_arrive_expect_tx(&full[stage], L::kStageBytes);
                    tma_load_2d(sa, &tmap_a, &full[stage], kb * kGemmBK, m0);
#pragma unroll
                    for (int c = 0; c < BN / 64; ++c)
                        tma_load_2d(sb + c * (kGemmBK * 128), &tmap_b, &full[stage], n0 + c * 64, kb * kGemmBK);
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ----------------------------- MMA issuer -----------------------------
        // The whole warp runs the loop (uniform control flow keeps descriptors in the uniform datapath);
        // one elected lane executes the tcgen05 instructions.
        {
            const bool leader = elect_one();
            const uint32_t idesc = gemm_idesc(kGemmBM, BN, p.f16_inputs);
            const uint32_t a_lo0 = sdesc_lo(smem_u32(smem), 16);
            const uint32_t b_lo0 = sdesc_lo(smem_u32(smem + L::kABytes), kGemmBK * 128);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            GemmWorkIter work(p, num_kb);
            GemmWork w;
            while (ok && work.next(p, num_kb, w)) {
                ok = __all_sync(0xffffffffu, mbar_wait(&acc_empty[acc], acc_phase ^ 1, abort_flag, 0x300 + acc));
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                const int kb0 = w.kb0, kb1 = w.kb1;
                for (int kb = kb0; kb < kb1; ++kb) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&full[stage], phase, abort_flag, 0x200 + stage));
                    if (!ok) break;
                    if (kb == kb0) MLT_GT(2);
                    tc_fence_after();
                    const uint32_t a_lo = a_lo0 + stage * (L::kStageBytes >> 4);
                    const uint32_t b_lo = b_lo0 + stage * (L::kStageBytes >> 4);
                    if (leader) {
                        umma_ss_lo_dyn(d_tmem, a_lo, b_lo, idesc, kb != kb0);
#pragma unroll
                        for (int k = 1; k < kGemmBK / 16; ++k)
                            umma_ss_lo<true>(d_tmem, a_lo + k * (32 >> 4), b_lo + k * (2048 >> 4), idesc);
                        umma_commit(&empty[stage]);  // frees the smem stage once these UMMAs have read it
                    }
                    __syncwarp();
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
                if (ok && leader) umma_commit(&acc_full[acc]);
                MLT_GT(3);
                __syncwarp();
                if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            }
        }
    } else {
        // ----------------------------- epilogue -----------------------------
        const int quarter = warp & 3;  // TMEM lanes this warp may touch: 32*quarter .. +31
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        GemmWorkIter work(p, num_kb);
        GemmWork w;
        while (ok && work.next(p, num_kb, w)) {
            int tm, tn;
            gemm_tile_coords(p, w.tile, tm, tn);
            const int row = tm * kGemmBM + quarter * 32 + lane;
            const int n0 = tn * BN;
            ok = __all_sync(0xffffffffu, mbar_wait(&acc_full[acc], acc_phase, abort_flag, 0x400 + acc));
            if (!ok) break;
            if (warp == 2) MLT_GT(4);
            tc_fence_after();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * BN;
            if (!kCTma && BN == 128 && !p.partial && !p.Cf && n0 + BN <= p.N) {
                // BF16 C, whole tile: through the staging rows, 64 columns at a time (on a problem of one wave the
                // epilogue is on the critical path)
                uint8_t* stg = smem_staging + quarter * (32 * kGemmBf16StagePitch);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t v[2][32];
                    tmem_ld_32x32b_x32(t_row + h * 64, v[0]);
                    tmem_ld_32x32b_x32(t_row + h * 64 + 32, v[1]);
                    tmem_wait_ld();
                    gemm_store_half_coalesced(p, stg, v, lane, tm * kGemmBM + quarter * 32, n0 + h * 64);
                }
            } else {
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld_32x32b_x32(t_row + c * 32, v);
                    tmem_wait_ld();
                    if constexpr (kCTma)
                        gemm_store_chunk_tma(p, &tmap_c, smem_staging + quarter * 8192 + (c & 1) * 4096, v, lane,
                                             tm * kGemmBM + quarter * 32, n0 + c * 32);
                    else
                        gemm_store_chunk(p, v, row, n0 + c * 32, w.slot);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[acc]);
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
        if (kCTma && lane == 0) tma_store_wait_all<0>();  // shared memory must outlive the stores that read it
    }

    // common exit: every role reaches this, also after an aborted wait
    tc_fence_before();
    __syncthreads();
    if (blockIdx.x == 0 && threadIdx.x == 0) clock_probe(0, 1);
    if (threadIdx.x == 0) MLT_GT(5);
    MLT_GT_NS(7);
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---------------------------------------------------------------------------
// CTA-pair variant for large problems: a cluster of two CTAs owns a 256 x 256 tile.
// Each CTA loads its own 128 rows of A and its own 128 columns of B (no multicast);
// the leader CTA (cluster rank 0) issues cta_group::2 UMMAs that read both CTAs'
// shared memory and write both CTAs' tensor memory (rows 0-127 / 128-255 of the tile).
// Compared with two independent 128 x 256 tiles this cuts the L2 -> SM operand traffic
// per FLOP by a third and the shared-memory reads of B by half.
//   full[s]       in the leader: both CTAs' TMA loads count bytes on it
//   empty[s]      in each CTA: the leader's commit arrives on both
//   acc_full[a]   in each CTA: the leader's commit arrives on both
//   acc_empty[a]  in the leader: the epilogue warps of both CTAs arrive on it (8 arrivals)
// ---------------------------------------------------------------------------
constexpr int kPairBM = 256;
constexpr int kPairBN = 256;

template <int kStages>
struct GemmPairSmem {
    static constexpr int kABytes = 128 * kGemmBK * 2;  // this CTA's 128 rows of A
    static constexpr int kBBytes = kGemmBK * 128 * 2;  // this CTA's 128 columns of B: 2 boxes of 64 x 64
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kNoStaging = kStages * kStageBytes + 1024 + 1024;
    static constexpr int kTotal = kNoStaging + kGemmStagingBytes;
    // BF16 output of the 128-wide kernel goes through a small staging area (see gemm_store_half_coalesced)
    static constexpr int kBf16Staging = kNoStaging + 4 * 32 * kGemmBf16StagePitch;
};

template <int kStages, bool kCTma>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
gemm_bf16_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                      const __grid_constant__ CUtensorMap tmap_c, const GemmParams p) {
    using L = GemmPairSmem<kStages>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * L::kStageBytes);
    // 1024-byte aligned (swizzle atoms of the TMA store); present only when the launch asked for it (p.c_tma)
    uint8_t* smem_staging = smem + kStages * L::kStageBytes + 1024;
    uint64_t* full = bars;
    uint64_t* empty = bars + kStages;
    uint64_t* acc_full = bars + 2 * kStages;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile uint32_t* abort_flag = tmem_base_slot + 1;

    const int warp = threadIdx.x >> 5;
    if (blockIdx.x == 0 && threadIdx.x == 0) clock_probe(0, 0);
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    const int cluster_id = blockIdx.x >> 1;
    const int num_clusters = gridDim.x >> 1;
    const int num_kb = (p.K + kGemmBK - 1) / kGemmBK;
    constexpr uint32_t kTmemCols = 512;  // two 256-column accumulators

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&acc_full[a], 1);
            mbar_init(&acc_empty[a], 8);  // 4 epilogue warps in each of the two CTAs
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0 && lane == 0) {
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_base_slot, kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    cluster_sync_all();  // barrier inits and allocations of both CTAs are visible to both
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_slot;

    if (warp == 0) {
        // ----------------------------- producer (both CTAs) -----------------------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int item = cluster_id; item < p.num_items && ok; item += num_clusters) {
                int tile, n_off, bn, tm, tn;
                gemm_pair_item(p, item, tile, n_off, bn);
                gemm_tile_coords(p, tile, tm, tn);
                const int m0 = tm * kPairBM + static_cast<int>(rank) * 128;
                const int n0 = tn * kPairBN + n_off + static_cast<int>(rank) * (bn >> 1);  // this CTA's bn/2 columns of B
                const uint32_t tx = 2u * (L::kABytes + (bn >> 1) * kGemmBK * 2);
                for (int kb = 0; kb < num_kb; ++kb) {
                    ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag, 0x100 + stage);
                    if (!ok) break;
                    uint8_t* sa = smem + stage * L::kStageBytes;
                    uint8_t* sb = sa + L::kABytes;
                    if (leader) mbar_arrive_expect_tx(&full[stage], tx);
                    const uint32_t bar = map_to_cta(smem_u32(&full[stage]), 0);
                    tma_load_2d_pair(sa, &tmap_a, bar, kb * kGemmBK, m0);
                    tma_load_2d_pair(sb, &tmap_b, bar, n0, kb * kGemmBK);
                    if (bn == 256) tma_load_2d_pair(sb + kGemmBK * 128, &tmap_b, bar, n0 + 64, kb * kGemmBK);
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ----------------------------- UMMA issuer (leader CTA only) -----------------------------
        if (leader) {
            // whole warp, uniform control flow; one elected lane executes the tcgen05 instructions
            const bool issuer = elect_one();
            const uint32_t idesc_full = gemm_idesc(kPairBM, kPairBN, p.f16_inputs);
            const uint32_t idesc_half = gemm_idesc(kPairBM, kPairBN / 2, p.f16_inputs);
            const uint32_t a_lo0 = sdesc_lo(smem_u32(smem), 16);
            const uint32_t b_lo0 = sdesc_lo(smem_u32(smem + L::kABytes), kGemmBK * 128);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int item = cluster_id; item < p.num_items && ok; item += num_clusters) {
                ok = __all_sync(0xffffffffu, mbar_wait(&acc_empty[acc], acc_phase ^ 1, abort_flag, 0x300 + acc));
                if (!ok) break;
                tc_fence_after();
                const uint32_t idesc = item < p.full_items ? idesc_full : idesc_half;
                const uint32_t d_tmem = tmem_base + acc * kPairBN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&full[stage], phase, abort_flag, 0x200 + stage));
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_lo = a_lo0 + stage * (L::kStageBytes >> 4);
                    const uint32_t b_lo = b_lo0 + stage * (L::kStageBytes >> 4);
                    if (issuer) {
#pragma unroll
                        for (int k = 0; k < kGemmBK / 16; ++k)
                            umma_ss_pair_lo(d_tmem, a_lo + k * (32 >> 4), b_lo + k * (2048 >> 4), idesc, (kb | k) != 0);
                        umma_commit_pair(&empty[stage], 3);
                    }
                    __syncwarp();
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
                if (ok && issuer) umma_commit_pair(&acc_full[acc], 3);
                __syncwarp();
                if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            }
        }
    } else {
        // ----------------------------- epilogue (both CTAs, own 128 rows) -----------------------------
        const int quarter = warp & 3;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int item = cluster_id; item < p.num_items && ok; item += num_clusters) {
            int tile, n_off, bn, tm, tn;
            gemm_pair_item(p, item, tile, n_off, bn);
            gemm_tile_coords(p, tile, tm, tn);
            const int row = tm * kPairBM + static_cast<int>(rank) * 128 + quarter * 32 + lane;
            const int n0 = tn * kPairBN + n_off;
            ok = __all_sync(0xffffffffu, mbar_wait(&acc_full[acc], acc_phase, abort_flag, 0x400 + acc));
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * kPairBN;
            // The last item of a CTA has no main loop behind it to hide its epilogue, and all CTAs reach theirs at about
            // the same time: there BF16 C goes through the staging rows in whole lines (half the time of the per-row
            // stores; not in steady state, where the extra shared-memory traffic would slow the operand reads).
            if (!kCTma && !p.Cf && item + num_clusters >= p.num_items && n0 + bn <= p.N) {
                uint8_t* stg = smem_staging + quarter * (32 * kGemmBf16StagePitch);
#pragma unroll 1
                for (int h = 0; h < bn / 64; ++h) {
                    uint32_t v[2][32];
                    tmem_ld_32x32b_x32(t_row + h * 64, v[0]);
                    tmem_ld_32x32b_x32(t_row + h * 64 + 32, v[1]);
                    tmem_wait_ld();
                    gemm_store_half_coalesced(p, stg, v, lane, tm * kPairBM + static_cast<int>(rank) * 128 + quarter * 32,
                                              n0 + h * 64);
                }
            } else {
#pragma unroll 1
            for (int c = 0; c < bn / 32; ++c) {
                uint32_t v[32];
                tmem_ld_32x32b_x32(t_row + c * 32, v);
                tmem_wait_ld();
                if constexpr (kCTma)
                    gemm_store_chunk_tma(p, &tmap_c, smem_staging + quarter * 8192 + (c & 1) * 4096, v, lane,
                                         tm * kPairBM + static_cast<int>(rank) * 128 + quarter * 32, n0 + c * 32);
                else
                    gemm_store_chunk(p, v, row, n0 + c * 32, 0);
            }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&acc_empty[acc]), 0));
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
        if (kCTma && lane == 0) tma_store_wait_all<0>();  // shared memory must outlive the stores that read it
    }

    // common exit: no CTA of the pair leaves while its peer may still touch its memory
    tc_fence_before();
    cluster_sync_all();
    if (blockIdx.x == 0 && threadIdx.x == 0) clock_probe(0, 1);
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

// ---------------------------------------------------------------------------
// Split-K inside a thread-block cluster, for skinny problems without caller scratch (paper Sec. 4.1, next-token
// shapes): the S CTAs of a cluster own one 128 x 128 output tile, CTA r accumulates K slice r in its own tensor
// memory, writes the FP32 tile into its own shared memory (the pipeline stages are free by then), and after a
// cluster barrier CTA r sums columns [r * 128 / S, (r + 1) * 128 / S) over all S CTAs' shared memory (plain
// distributed-shared-memory loads, ascending slice order: deterministic) and stores BF16.  One kernel, no partial
// tiles in global memory, no second launch.  One tile per cluster.
// ---------------------------------------------------------------------------
constexpr int kClusterKPartPad = 4;  // floats added to a row of the FP32 tile in shared memory (pitch 528 or 1040 B: conflict-free 16-byte rows)

__device__ __forceinline__ float4 ld_shared_cluster_f32x4(uint32_t cluster_addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(cluster_addr));
    return v;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}

template <int BN, int kStages>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_bf16_clusterk_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                          const GemmParams p) {
    static_assert(BN == 128 || BN == 256, "tile widths of the single-CTA kernels");
    constexpr int kPartPitch = BN + kClusterKPartPad;
    using L = GemmSmem<BN, kStages>;
    static_assert(kGemmBM * kPartPitch * 4 <= kStages * L::kStageBytes, "the FP32 tile fits the pipeline stages");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * L::kStageBytes);
    uint64_t* full = bars;
    uint64_t* empty = bars + kStages;
    uint64_t* acc_full = bars + 2 * kStages;
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(acc_full + 1);
    volatile uint32_t* abort_flag = tmem_base_slot + 1;

    const int warp = threadIdx.x >> 5;
    if (blockIdx.x == 0 && threadIdx.x == 0) clock_probe(0, 0);
    const int lane = threadIdx.x & 31;
    const int S = static_cast<int>(cluster_nctarank());
    const int slice = static_cast<int>(cluster_ctarank());
    const int tile = static_cast<int>(blockIdx.x) / S;
    const int num_kb = (p.K + kGemmBK - 1) / kGemmBK;
    const int kb0 = slice * p.kb_per_split, kb1 = min(num_kb, kb0 + p.kb_per_split);  // no slice is empty (host)
    int tm, tn;
    gemm_tile_coords(p, tile, tm, tn);
    const int m0 = tm * kGemmBM, n0 = tn * BN;
    constexpr uint32_t kTmemCols = BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        mbar_init(acc_full, 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0 && lane == 0) {
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc(tmem_base_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_slot;
    float* part = reinterpret_cast<float*>(smem);  // [128][kPartPitch], written after the main loop

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int kb = kb0; kb < kb1 && ok; ++kb) {
                ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag, 0x100 + stage);
                if (!ok) break;
                uint8_t* sa = smem + stage * L::kStageBytes;
                uint8_t* sb = sa + L::kABytes;
                mbar_arrive_expect_tx(&full[stage], L::kStageBytes);
                tma_load_2d(sa, &tmap_a, &full[stage], kb * kGemmBK, m0);
#pragma unroll
                for (int c = 0; c < BN / 64; ++c)
                    tma_load_2d(sb + c * (kGemmBK * 128), &tmap_b, &full[stage], n0 + c * 64, kb * kGemmBK);
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == 1) {
        const bool leader = elect_one();
        const uint32_t idesc = gemm_idesc(kGemmBM, BN, p.f16_inputs);
        const uint32_t a_lo0 = sdesc_lo(smem_u32(smem), 16);
        const uint32_t b_lo0 = sdesc_lo(smem_u32(smem + L::kABytes), kGemmBK * 128);
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int kb = kb0; kb < kb1; ++kb) {
            ok = __all_sync(0xffffffffu, mbar_wait(&full[stage], phase, abort_flag, 0x200 + stage));
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_lo = a_lo0 + stage * (L::kStageBytes >> 4);
            const uint32_t b_lo = b_lo0 + stage * (L::kStageBytes >> 4);
            if (leader) {
                umma_ss_lo_dyn(tmem_base, a_lo, b_lo, idesc, kb != kb0);
#pragma unroll
                for (int k = 1; k < kGemmBK / 16; ++k)
                    umma_ss_lo<true>(tmem_base, a_lo + k * (32 >> 4), b_lo + k * (2048 >> 4), idesc);
                umma_commit(&empty[stage]);
            }
            __syncwarp();
            if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (ok && leader) umma_commit(acc_full);
        __syncwarp();
    } else {
        // accumulator -> this CTA's FP32 tile in shared memory; acc_full also says that every UMMA has read its
        // operands, and the producer issued no load beyond them: the stages are free
        const int quarter = warp & 3;
        const int r = quarter * 32 + lane;  // row inside the tile
        if (__all_sync(0xffffffffu, mbar_wait(acc_full, 0, abort_flag, 0x400))) {
            tc_fence_after();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
#pragma unroll 1
            for (int h = 0; h < BN / 128; ++h) {  // 128 columns at a time: four loads in flight before the one wait
                uint32_t v[4][32];
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_ld_32x32b_x32(t_row + h * 128 + c * 32, v[c]);
                tmem_wait_ld();
                if (m0 + r < p.M) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        float4* dst = reinterpret_cast<float4*>(part + r * kPartPitch + h * 128 + c * 32);
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            dst[q] = make_float4(__uint_as_float(v[c][q * 4]), __uint_as_float(v[c][q * 4 + 1]),
                                                 __uint_as_float(v[c][q * 4 + 2]), __uint_as_float(v[c][q * 4 + 3]));
                    }
                }
            }
        }
    }

    // every CTA's tile is in its shared memory (or a wait expired there: its rows are then garbage and the status
    // word says so); sum this CTA's share of the columns over the cluster
    tc_fence_before();
    cluster_sync_all();
    {
        const int cols = BN / S;  // S in {2, 4, 8}: 16 to 128 columns, in groups of 4
        const int groups = cols / 4;
        const int rows = min(kGemmBM, p.M - m0);
        const uint32_t part_addr = smem_u32(part);
        for (int idx = threadIdx.x; idx < rows * groups; idx += kGemmThreads) {
            const int r = idx / groups, c = slice * cols + (idx % groups) * 4;
            float4 acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            for (int s2 = 0; s2 < S; ++s2) {
                const float4 v = ld_shared_cluster_f32x4(map_to_cta(part_addr + (r * kPartPitch + c) * 4, s2));
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            }
            const int col = n0 + c;
            __nv_bfloat16* dst = p.C + static_cast<int64_t>(m0 + r) * p.ldc + col;
            if (col + 4 <= p.N) {
                uint2 out;
                out.x = pack_bf16x2(acc.x, acc.y);
                out.y = pack_bf16x2(acc.z, acc.w);
                *reinterpret_cast<uint2*>(dst) = out;
            } else {
                const float a[4] = {acc.x, acc.y, acc.z, acc.w};
                for (int j = 0; j < 4 && col + j < p.N; ++j) dst[j] = __float2bfloat16(a[j]);
            }
        }
    }
    // common exit: no CTA leaves while a peer may still read its shared memory
    cluster_sync_all();
    if (blockIdx.x == 0 && threadIdx.x == 0) clock_probe(0, 1);
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// Split-K second step: C[i][j] = RNE_bf16(sum over slices of partial[slice][i][j]); 8 columns per thread.  With the
// even K hand-out the number of partials differs from tile to tile and follows from the same arithmetic as in the kernel.
__global__ void gemm_splitk_reduce_kernel(const float* partial, __nv_bfloat16* C, int64_t ldc, int M, int N, int split_k,
                                          int even_units, int num_kb, int tiles_m) {
    const int64_t groups_per_row = (N + 7) / 8;
    const int64_t total = static_cast<int64_t>(M) * groups_per_row;
    // Launched with programmatic stream serialisation: the CTAs may start while the GEMM kernel is still running
    // (which hides this kernel's launch latency) and wait here until all of its partial tiles are visible.
    cudaGridDependencySynchronize();
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int row = static_cast<int>(i / groups_per_row);
        const int col = static_cast<int>(i % groups_per_row) * 8;
        float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        int parts = split_k;
        if (even_units > 0) {  // even K hand-out: the CTAs whose shares touch this element's tile, one partial each
            const long long t = static_cast<long long>(col / 128) * tiles_m + row / kGemmBM;  // one raster group: M fastest
            parts = static_cast<int>(((t + 1) * num_kb - 1) / even_units - t * num_kb / even_units) + 1;
        }
        const bool full = col + 8 <= N && (N & 3) == 0;
        const int64_t slice_pitch = static_cast<int64_t>(M) * N;
        const float* src0 = partial + static_cast<int64_t>(row) * N + col;
        int s = 0;
        if (full) {
            // four slices' loads in flight before the first addition (the additions keep the ascending slice order)
            for (; s + 4 <= parts; s += 4) {
                float4 a[4], b[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    a[u] = *reinterpret_cast<const float4*>(src0 + (s + u) * slice_pitch);
                    b[u] = *reinterpret_cast<const float4*>(src0 + (s + u) * slice_pitch + 4);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    acc[0] += a[u].x; acc[1] += a[u].y; acc[2] += a[u].z; acc[3] += a[u].w;
                    acc[4] += b[u].x; acc[5] += b[u].y; acc[6] += b[u].z; acc[7] += b[u].w;
                }
            }
        }
        for (; s < parts; ++s) {
            const float* src = src0 + s * slice_pitch;
            if (full) {
                const float4 a = *reinterpret_cast<const float4*>(src), b = *reinterpret_cast<const float4*>(src + 4);
                acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
                acc[4] += b.x; acc[5] += b.y; acc[6] += b.z; acc[7] += b.w;
            } else {
                for (int j = 0; j < 8 && col + j < N; ++j) acc[j] += src[j];
            }
        }
        __nv_bfloat16* dst = C + static_cast<int64_t>(row) * ldc + col;
        if (col + 8 <= N) {
            uint4 out;
            out.x = pack_bf16x2(acc[0], acc[1]);
            out.y = pack_bf16x2(acc[2], acc[3]);
            out.z = pack_bf16x2(acc[4], acc[5]);
            out.w = pack_bf16x2(acc[6], acc[7]);
            *reinterpret_cast<uint4*>(dst) = out;
        } else {
            for (int j = 0; col + j < N; ++j) dst[j] = __float2bfloat16(acc[j]);
        }
    }
}

__global__ void gemm_zero_fill_f32_kernel(float* C, int64_t ldc, int M, int N) {
    const int64_t total = static_cast<int64_t>(M) * N;
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x)
        C[(i / N) * ldc + (i % N)] = 0.0f;
}

// C[i][0..N) = 0 for K == 0 (BLAS convention for an empty sum).
__global__ void gemm_zero_fill_kernel(__nv_bfloat16* C, int64_t ldc, int M, int N) {
    const int64_t total = static_cast<int64_t>(M) * N;
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        C[(i / N) * ldc + (i % N)] = __float2bfloat16(0.0f);
    }
}

}  // namespace mlt
