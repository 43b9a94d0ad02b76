// Host side of the C ABI declared in include/mlt.h: argument validation, TMA
// descriptor encoding, launch configuration.  All arithmetic of the hot path runs
// in the kernels of gemm.cuh and mha.cuh.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "../../include/mlt.h"
#include "gemm.cuh"
#include "mha.cuh"
#include "paged.cuh"

namespace {

using namespace mlt;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceInfo {
    int sm_count = 0;
    int cc_major = 0;
    bool configured = false;
    bool mha_ok = false;  // the attention kernels' compiled register count covers their in-kernel register hand-over
    // CTAs that can be resident at once as clusters of 2, 4 and 8 of the K-cutting GEMM kernel (a cluster must fit
    // one GPC, so this can be less than the SM count rounded down to a multiple of the cluster size)
    int cluster_slots[3] = {0, 0, 0};
};

std::mutex g_mutex;
EncodeTiledFn g_encode = nullptr;
DeviceInfo g_devices[64];

// Looks up cuTensorMapEncodeTiled through the runtime, so libcuda is not a link-time dependency.
int get_encoder(EncodeTiledFn* out) {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) return MLT_ERR_CUDA;
        g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    *out = g_encode;
    return MLT_OK;
}

template <class Kernel>
int set_smem(Kernel k, int bytes) {
    return cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess ? MLT_OK
                                                                                                     : MLT_ERR_CUDA;
}

// Once per device: capability check and the shared-memory opt-in of every kernel.
int get_device(DeviceInfo* out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MLT_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceInfo& d = g_devices[dev];
    if (!d.configured) {
        if (cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return MLT_ERR_CUDA;
        if (d.cc_major != 10) return MLT_ERR_ARCH;
        if (set_smem(gemm_bf16_kernel<256, 4, false>, GemmSmem<256, 4>::kNoStaging) != MLT_OK ||
            set_smem(gemm_bf16_kernel<128, 6, false>, GemmSmem<128, 6>::kBf16Staging) != MLT_OK ||
            set_smem(gemm_bf16_pair_kernel<6, false>, GemmPairSmem<6>::kBf16Staging) != MLT_OK ||
            set_smem(gemm_bf16_clusterk_kernel<128, 6>, GemmSmem<128, 6>::kNoStaging) != MLT_OK ||
            set_smem(gemm_bf16_clusterk_kernel<256, 4>, GemmSmem<256, 4>::kNoStaging) != MLT_OK ||
            set_smem(gemm_bf16_kernel<256, 4, true>, GemmSmem<256, 4>::kTotal) != MLT_OK ||
            set_smem(gemm_bf16_kernel<128, 6, true>, GemmSmem<128, 6>::kTotal) != MLT_OK ||
            set_smem(gemm_bf16_pair_kernel<6, true>, GemmPairSmem<6>::kTotal) != MLT_OK)
            return MLT_ERR_CUDA;
        for (int i = 0; i < 3; ++i) {
            const int S = 2 << i;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(static_cast<unsigned>(d.sm_count / S * S));
            cfg.blockDim = dim3(kGemmThreads);
            cfg.dynamicSmemBytes = GemmSmem<128, 6>::kNoStaging;
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = static_cast<unsigned>(S);
            attr.val.clusterDim.y = attr.val.clusterDim.z = 1;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            int clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&clusters, gemm_bf16_clusterk_kernel<128, 6>, &cfg) != cudaSuccess) {
                cudaGetLastError();
                clusters = 0;  // unknown: this cluster size is not used
            }
            d.cluster_slots[i] = clusters * S;
        }
        if (paged_configure() != 0) return MLT_ERR_CUDA;
        const int mha_rc = mha_configure();
        if (mha_rc == 1) return MLT_ERR_CUDA;
        d.mha_ok = mha_rc == 0;
        d.configured = true;
    }
    *out = d;
    return MLT_OK;
}

// BF16 tensor map with 128-byte swizzle.  dims / strides innermost first; strides[0] is implicit.
int encode_bf16(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                const uint32_t* box, int dtype = 0 /* 0 BF16, 1 FP16, 2 FP32 */) {
    EncodeTiledFn enc;
    int rc = get_encoder(&enc);
    if (rc != MLT_OK) return rc;
    cuuint64_t gdim[5];
    cuuint64_t gstride[5];
    cuuint32_t gbox[5];
    cuuint32_t estr[5];
    for (int i = 0; i < rank; ++i) {
        if (dims[i] == 0 || dims[i] > (1ull << 32)) return MLT_ERR_UNSUPPORTED;
        gdim[i] = dims[i];
        gbox[i] = box[i];
        estr[i] = 1;
        if (i > 0) {
            if (strides_bytes[i - 1] >= (1ull << 40) || strides_bytes[i - 1] % 16) return MLT_ERR_UNSUPPORTED;
            gstride[i - 1] = strides_bytes[i - 1];
        }
    }
    const CUtensorMapDataType dt = dtype == 2   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                   : dtype == 1 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                                : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    CUresult r = enc(map, dt, static_cast<cuuint32_t>(rank), const_cast<void*>(base),
                     gdim, gstride, gbox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? MLT_OK : MLT_ERR_CUDA;
}

// Debug only: MLT_FORCE_VARIANT=0|1|2 pins the GEMM tile variant (pair 256x256, 128x256, 128x128).
int forced_variant() {
    static const int v = [] {
        const char* e = std::getenv("MLT_FORCE_VARIANT");
        return e ? std::atoi(e) : -1;
    }();
    return v;
}

// Debug only: tuning overrides read once from the environment (0 = not set).  MLT_GEMM_GROUP_M: M-tiles per raster
// group of the pair kernel; MLT_GEMM_NO_HALF: no half tiles in the last wave; MLT_MHA_HEAD_GROUP / MLT_MHA_GRID: item
// list grouping and CTA count of the attention kernel; MLT_PAGED_SPLITS: CTAs per (sequence, KV head);
// MLT_GEMM_WIDE_RATIO: per cent of the current plan's cost below which 128 x 256 tiles in clusters are taken (1: never);
// MLT_GEMM_NO_EVEN: uniform K slices through scratch instead of the even hand-out; MLT_GEMM_NO_SKINNY_MODEL: the
// rule-based plan for problems of one tile row instead of the time model; MLT_GEMM_NO_CLUSTER: no K cut inside clusters.
struct DebugEnv {
    int gemm_group_m, gemm_no_half, mha_head_group, mha_grid, paged_splits, gemm_wide_ratio, gemm_no_even, gemm_no_skinny_model, gemm_no_cluster;
};
const DebugEnv& debug_env() {
    static const DebugEnv env = [] {
        auto get = [](const char* name) {
            const char* e = std::getenv(name);
            const int v = e ? std::atoi(e) : 0;
            return v > 0 ? v : 0;
        };
        return DebugEnv{get("MLT_GEMM_GROUP_M"), get("MLT_GEMM_NO_HALF"), get("MLT_MHA_HEAD_GROUP"), get("MLT_MHA_GRID"),
                        get("MLT_PAGED_SPLITS"), get("MLT_GEMM_WIDE_RATIO"), get("MLT_GEMM_NO_EVEN"), get("MLT_GEMM_NO_SKINNY_MODEL"), get("MLT_GEMM_NO_CLUSTER")};
    }();
    return env;
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing will ever complete, with a short budget.
// The wait gives up, records {timeout, barrier id 0x7E57, block, parity} in the status word and the kernel returns
// like any other; nothing traps and the context stays usable.
__global__ void debug_wait_timeout_kernel(long long budget) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_word;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_word = 0;
        fence_mbar_init();
    }
    __syncthreads();
    mbar_wait(&bar, 0, &abort_word, 0x7E57u, budget);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" {

int mlt_version(void) { return 100; }

const char* mlt_status_string(int status) {
    switch (status) {
        case MLT_OK: return "ok";
        case MLT_ERR_INVALID_ARG: return "invalid argument";
        case MLT_ERR_UNSUPPORTED: return "unsupported size or head dimension";
        case MLT_ERR_ALIGNMENT: return "pointer not 16-byte aligned or pitch not a multiple of 8 elements";
        case MLT_ERR_CUDA: return "CUDA runtime or driver call failed";
        case MLT_ERR_ARCH: return "device is not compute capability 10.x (sm_100a required)";
        case MLT_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case MLT_ERR_BAD_BLOCK: return "a block-table entry outside [0, num_blocks) was met";
        case MLT_ERR_SCRATCH_LIMIT: return "the call needs more scratch than the built-in array of mlt_paged_attn_decode_static holds";
        default: return "unknown status";
    }
}

int mlt_debug_wait_timeout_selftest(uint64_t budget_cycles, void* stream) {
    if (budget_cycles == 0 || budget_cycles > 1000000000ull) return MLT_ERR_INVALID_ARG;  // at most about half a second
    DeviceInfo dev;
    const int rc = get_device(&dev);
    if (rc != MLT_OK) return rc;
    debug_wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<long long>(budget_cycles));
    return cudaGetLastError() == cudaSuccess ? MLT_OK : MLT_ERR_CUDA;
}

#if defined(MLT_TRACE) || defined(MLT_TRACE_ITEMS)
int mlt_debug_read_trace(unsigned int* host) {  // development builds only: copies the attention kernel's clock trace
    if (cudaDeviceSynchronize() != cudaSuccess) return MLT_ERR_CUDA;
    return cudaMemcpyFromSymbol(host, g_mha_trace, sizeof(g_mha_trace)) == cudaSuccess ? MLT_OK : MLT_ERR_CUDA;
}
int mlt_debug_read_gemm_trace(long long* host) {  // development builds only
    if (cudaDeviceSynchronize() != cudaSuccess) return MLT_ERR_CUDA;
    return cudaMemcpyFromSymbol(host, g_gemm_trace, sizeof(g_gemm_trace)) == cudaSuccess ? MLT_OK : MLT_ERR_CUDA;
}
#endif

int mlt_debug_last_clock_mhz(int which, double* mhz) {
    if ((which != 0 && which != 1) || !mhz) return MLT_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return MLT_ERR_CUDA;
    unsigned long long host[2][4];
    if (cudaMemcpyFromSymbol(host, g_clock_probe, sizeof host) != cudaSuccess) return MLT_ERR_CUDA;
    const unsigned long long* h = host[which];
    *mhz = (h[3] > h[1] && h[2] > h[0]) ? 1000.0 * static_cast<double>(h[2] - h[0]) / static_cast<double>(h[3] - h[1]) : 0.0;
    return MLT_OK;
}

int mlt_last_device_error(uint32_t* detail) {
    if (cudaDeviceSynchronize() != cudaSuccess) return MLT_ERR_CUDA;
    unsigned int host[4] = {0, 0, 0, 0};
    if (cudaMemcpyFromSymbol(host, g_status, sizeof host) != cudaSuccess) return MLT_ERR_CUDA;
    if (detail) std::memcpy(detail, host, sizeof host);
    if (host[0] != 0) {
        unsigned int zero[4] = {0, 0, 0, 0};
        if (cudaMemcpyToSymbol(g_status, zero, sizeof zero) != cudaSuccess) return MLT_ERR_CUDA;
        return host[0] == kStatusTimeout ? MLT_ERR_TIMEOUT : host[0] == kStatusBadBlock ? MLT_ERR_BAD_BLOCK : MLT_ERR_CUDA;
    }
    return MLT_OK;
}

// K slices a skinny problem may be cut into through scratch: enough work items for two per SM, at least 4 blocks of
// 64 per slice; none with 512 rows or more (compute-bound: the second launch costs more than the cut saves, measured
// on 512^3)
static int gemm_max_split(int64_t M, int64_t N, int64_t K) {
    const int64_t tiles = ((M + 127) / 128) * ((N + 127) / 128);
    const int64_t num_kb = (K + kGemmBK - 1) / kGemmBK;
    if (tiles >= 1024 || num_kb < 8 || M >= 512) return 1;
    return static_cast<int>(std::min<int64_t>(32, num_kb / 4));
}

// CTAs per cluster (1, 2, 4 or 8) that cut K for one 128 x 128 tile of a skinny problem: the count that minimises
// rounds x (K blocks per CTA + fill, drain and the reduction), every slice at least 4 blocks of 64.
// cluster_slots: resident CTAs for S = 2, 4, 8 as the device reports them, or null for the SM count rounded down.
static int gemm_cluster_split(int64_t tiles, int num_kb, int sm_count, const int* cluster_slots) {
    if (tiles * 2 > sm_count || debug_env().gemm_no_cluster) return 1;  // enough tiles to occupy the GPU without cutting K
    int best_s = 1;
    int64_t best = (num_kb + 4);
    for (int S = 2, i = 0; S <= 8; S *= 2, ++i) {
        if (num_kb / S < 4 || S > sm_count) break;
        const int kbps = (num_kb + S - 1) / S;
        if (static_cast<int64_t>(kbps) * (S - 1) >= num_kb) continue;  // an empty slice
        const int64_t slots = cluster_slots ? cluster_slots[i] : sm_count / S * S;
        if (slots < S) continue;
        const int64_t rounds = (tiles * S + slots - 1) / slots;
        const int64_t cost = rounds * (kbps + 10);  // cluster launch, two cluster barriers and the reduction: about 6 blocks more
        if (cost < best) { best = cost; best_s = S; }
    }
    return best_s;
}

// What gemm_run launches for a problem: the tile shape, and for skinny problems how K is cut.
struct GemmPlan {
    int variant;       // 0: CTA pairs on 256 x 256 tiles, 1: 128 x 256 tiles, 2: 128 x 128 tiles
    int split_k;       // > 1: K slices with FP32 partials in caller scratch, summed by a second kernel
    int cluster;       // > 1: CTAs per cluster that cut K for one tile (128 x 128, or 128 x 256 with variant 1) and reduce through distributed shared memory
    int kb_per_split;  // K blocks of 64 per slice (per CTA of a cluster; per CTA's share with the even hand-out)
    int even;          // 1: even K hand-out through scratch (variant 2): every CTA the same number of (tile, K block)
                       //    units, split_k = the most partials a tile can get
};

static GemmPlan gemm_plan_base(int64_t M, int64_t N, int64_t K, bool has_workspace, size_t workspace_bytes, bool f32_out,
                               int sm_count, const int* cluster_slots, int forced) {
    // Tile shape by problem size.  Problems with at least 512 rows are compute-bound: the variant with the least
    // (waves x work per tile / efficiency) wins, with the measured relative efficiencies 1 : 0.8 : 0.62 of the three
    // kernels (the smaller tiles are bound by the shared-memory operand path).  Shorter problems stream B once and
    // are bound by memory: pairs when there is at least one tile per pair of SMs, else 128 x 256 tiles, else (most
    // SMs would idle) 128 x 128 tiles, which can also be cut along K.
    const int64_t pair_tiles = ((M + kPairBM - 1) / kPairBM) * ((N + kPairBN - 1) / kPairBN);
    const int64_t tiles_m128 = (M + kGemmBM - 1) / kGemmBM;
    const int64_t tiles1 = tiles_m128 * ((N + 255) / 256);
    const int64_t tiles2 = tiles_m128 * ((N + 127) / 128);
    const int num_kb = static_cast<int>((K + kGemmBK - 1) / kGemmBK);
    GemmPlan plan = {2, 1, 1, num_kb, 0};
    if (M <= kGemmBM && !f32_out && !(forced >= 0 && forced <= 2) && !debug_env().gemm_no_skinny_model &&
        gemm_cluster_split(tiles2, num_kb, sm_count, cluster_slots) == 1) {
        // One row of tiles, too many of them to cut K inside clusters: B streams once and the question is only which
        // launch keeps HBM busiest.  Time model in microseconds, fitted to CUDA-event timings on M = 16..128,
        // N = 14k..115k, K = 2k..8k: 5 us of launch and fill, then the larger of the stream at the copy bandwidth
        // (6.5 TB/s) and the busiest SM's bytes at what one SM pulls (67 GB/s in 512-byte rows of a 128 x 256 tile,
        // 56 GB/s in the 256-byte rows of a 128 x 128 tile; the rows of A come from L2 and count 0.3); a second kernel
        // costs 5 us more and the even hand-out's short end pieces about 2.  The CTA-pair kernel never won here (half
        // of each pair has no rows).
        const double a_bytes = 0.3 * static_cast<double>(M) * 128.0;
        const double fill = (num_kb + 4.0) / num_kb;
        const double hbm_us = 2.0 * (static_cast<double>(M) * K + static_cast<double>(K) * N + static_cast<double>(M) * N) / 6.5e6;
        auto rounds_of = [&](int64_t items) { return static_cast<double>((items + sm_count - 1) / sm_count); };
        const double t1 = 5.0 + std::max(hbm_us, rounds_of(tiles1) * num_kb * (a_bytes + 32768.0) * fill / 67e3);
        const double t2 = 5.0 + std::max(hbm_us, rounds_of(tiles2) * num_kb * (a_bytes + 16384.0) * fill / 56e3);
        plan.variant = t1 < t2 ? 1 : 2;
        double best_t = std::min(t1, t2);
        int max_split = has_workspace ? gemm_max_split(M, N, K) : 1;
        while (max_split > 1 && static_cast<size_t>(max_split) * M * N * sizeof(float) > workspace_bytes) --max_split;
        const double partial_us = static_cast<double>(M) * N * 8.0 / 6.5e6;  // one FP32 partial written and read
        for (int sl = 2; sl <= max_split; ++sl) {  // uniform slices through scratch
            const int kbps = (num_kb + sl - 1) / sl;
            const int slices = (num_kb + kbps - 1) / kbps;
            if (slices != sl) continue;
            const double t = 10.0 + sl * partial_us +
                             std::max(hbm_us, rounds_of(tiles2 * slices) * (kbps + 4.0) * (a_bytes + 16384.0) / 56e3);
            if (t < best_t) {
                best_t = t;
                plan = GemmPlan{2, slices, 1, kbps, 0};
            }
        }
        if (max_split > 1 && !debug_env().gemm_no_even) {  // the even hand-out through scratch
            const int64_t units = (tiles2 * num_kb + sm_count - 1) / sm_count;
            const int parts = static_cast<int>((num_kb + units - 1) / units) + 1;
            const double t = 12.0 + 2.0 * partial_us + std::max(hbm_us, (units + 8.0) * (a_bytes + 16384.0) / 56e3);
            if (units >= 8 && units <= INT32_MAX && static_cast<size_t>(parts) * M * N * sizeof(float) <= workspace_bytes && t < best_t) {
                best_t = t;
                plan = GemmPlan{2, parts, 1, static_cast<int>(units), 1};
            }
        }
        return plan;
    }
    // (From 129 rows on the same comparison holds as long as there are too many tiles to cut K inside clusters:
    // measured on 140..400 rows, N = 9600..28672, the model's pick was the fastest launch every time, and K cuts
    // through scratch were 10-90 % slower than it.)
    const bool by_waves = M >= 512 || (M > kGemmBM && !f32_out && gemm_cluster_split(tiles2, num_kb, sm_count, cluster_slots) == 1);
    if (by_waves) {
        const int64_t pairs = sm_count / 2;
        const double c0 = static_cast<double>((pair_tiles + pairs - 1) / pairs);
        const double c1 = static_cast<double>((tiles1 + sm_count - 1) / sm_count) / 0.8;
        const double c2 = static_cast<double>((tiles2 + sm_count - 1) / sm_count) * 0.5 / 0.62;
        plan.variant = (c0 <= c1 && c0 <= c2) ? 0 : (c1 <= c2 ? 1 : 2);
    } else if (!f32_out && (gemm_cluster_split(tiles2, num_kb, sm_count, cluster_slots) > 1 ||
                            (has_workspace && gemm_max_split(M, N, K) > 1))) {
        plan.variant = 2;  // memory-bound and K can be cut: small tiles spread the stream of B evenly over the SMs
    } else if (pair_tiles >= sm_count / 2) {
        plan.variant = 0;
    } else if (tiles1 >= sm_count) {
        plan.variant = 1;
    } else {
        plan.variant = 2;
    }
    if (forced >= 0 && forced <= 2) plan.variant = forced;
    if (plan.variant != 2 || f32_out) return plan;

    // Few tiles: clusters of S CTAs per tile when at most half the SMs would have a tile (measured equal to or faster
    // than partial tiles in scratch plus a second kernel, so it is used with or without a workspace) ...
    plan.cluster = gemm_cluster_split(tiles2, num_kb, sm_count, cluster_slots);
    if (plan.cluster > 1) {
        plan.kb_per_split = (num_kb + plan.cluster - 1) / plan.cluster;
        return plan;
    }
    if (!has_workspace || M > kGemmBM) return plan;
    // ... else slices through scratch: the count that minimises rounds x (K blocks per slice + fill/drain of an item)
    // plus the time to write and re-read the FP32 partials, in units of one K block of one tile (16 KB of B per SM).
    int max_split = gemm_max_split(M, N, K);
    while (max_split > 1 && static_cast<size_t>(max_split) * M * N * sizeof(float) > workspace_bytes) --max_split;
    int split = 1;
    double best = 1e300;
    for (int sl = 1; sl <= max_split; ++sl) {
        const int kbps = (num_kb + sl - 1) / sl;
        const int slices = (num_kb + kbps - 1) / kbps;
        if (slices != sl) continue;  // the same slicing as a smaller count
        const int64_t rounds = (tiles2 * slices + sm_count - 1) / sm_count;
        const double partial = sl > 1 ? static_cast<double>(sl) * M * N * 8.0 / (16384.0 * sm_count) : 0.0;
        const double cost = static_cast<double>(rounds) * (kbps + 4) + partial;
        if (cost < best) { best = cost; split = sl; }
    }
    if (split > 1) {
        plan.kb_per_split = (num_kb + split - 1) / split;
        plan.split_k = (num_kb + plan.kb_per_split - 1) / plan.kb_per_split;  // no empty slice
    }
    // ... or the even hand-out: all tiles x K blocks units cut into one contiguous share per SM, whatever tiles a
    // share touches (uniform slices leave the last round part empty: 672 items on 148 SMs are 4.5 rounds, paid as 5).
    // One raster group only (the reduce kernel recomputes a tile's index from its coordinates).
    if (max_split > 1 && tiles_m128 <= 16 && !debug_env().gemm_no_even) {
        const int64_t total = tiles2 * num_kb;
        const int64_t units = (total + sm_count - 1) / sm_count;
        const int parts = static_cast<int>((num_kb + units - 1) / units) + 1;  // CTAs that can touch one tile
        const double partial = 2.0 * M * N * 8.0 / (16384.0 * sm_count);        // about two partials per element
        const double cost = static_cast<double>(units) + 2 * 4 + partial;        // two pieces per share: fill and drain twice
        if (units >= 8 && units <= INT32_MAX && static_cast<size_t>(parts) * M * N * sizeof(float) <= workspace_bytes &&
            cost < (split > 1 ? best : static_cast<double>((tiles2 + sm_count - 1) / sm_count) * (num_kb + 4))) {
            plan.even = 1;
            plan.split_k = parts;
            plan.kb_per_split = static_cast<int>(units);
        }
    }
    return plan;
}

// The plan above, or for problems of 129 to 640 rows 128 x 256 tiles with K cut inside clusters, when that moves
// clearly fewer bytes through the busiest SM.  These problems are bound by what one SM can pull from L2 (about 110
// GB/s): a 128 x 128 tile pulls 32 KB per K block for 2 MFLOP, a 128 x 256 tile 48 KB for 4 MFLOP, and cutting K
// inside a cluster puts the narrower problem on all SMs all the same.  Cost of a plan = rounds x (K blocks per CTA +
// fixed blocks) x KB per block.
static GemmPlan gemm_plan(int64_t M, int64_t N, int64_t K, bool has_workspace, size_t workspace_bytes, bool f32_out,
                          int sm_count, const int* cluster_slots, int forced) {
    GemmPlan plan = gemm_plan_base(M, N, K, has_workspace, workspace_bytes, f32_out, sm_count, cluster_slots, forced);
    const int ratio = debug_env().gemm_wide_ratio ? debug_env().gemm_wide_ratio : 90;  // per cent; 1: never
    if (f32_out || M <= 128 || M > 640 || (forced >= 0 && forced <= 2) || sm_count < 8) return plan;
    const int64_t pair_tiles = ((M + kPairBM - 1) / kPairBM) * ((N + kPairBN - 1) / kPairBN);
    const int64_t tiles_m128 = (M + kGemmBM - 1) / kGemmBM;
    const int64_t tiles1 = tiles_m128 * ((N + 255) / 256);
    const int64_t tiles2 = tiles_m128 * ((N + 127) / 128);
    const int num_kb = static_cast<int>((K + kGemmBK - 1) / kGemmBK);
    auto slots_of = [&](int S) {
        const int i = S == 2 ? 0 : (S == 4 ? 1 : 2);
        return static_cast<int64_t>(cluster_slots ? cluster_slots[i] : sm_count / S * S);
    };
    auto rounds_of = [](int64_t items, int64_t slots) { return (items + slots - 1) / slots; };
    double cur;
    if (plan.variant == 0)
        cur = static_cast<double>(rounds_of(pair_tiles, sm_count / 2)) * (num_kb + 4) * 32.0;
    else if (plan.variant == 1)
        cur = static_cast<double>(rounds_of(tiles1, sm_count)) * (num_kb + 4) * 48.0;
    else if (plan.cluster > 1)
        cur = static_cast<double>(rounds_of(tiles2 * plan.cluster, std::max<int64_t>(slots_of(plan.cluster), plan.cluster))) *
              (plan.kb_per_split + 10) * 32.0;
    else if (plan.even)
        cur = static_cast<double>(plan.kb_per_split + 8) * 32.0 + 2.0 * M * N * 8.0 / (1024.0 * sm_count);
    else
        cur = static_cast<double>(rounds_of(tiles2 * plan.split_k, sm_count)) * (plan.kb_per_split + 4) * 32.0 +
              (plan.split_k > 1 ? static_cast<double>(plan.split_k) * M * N * 8.0 / (1024.0 * sm_count) : 0.0);
    int best_s = 1, best_kbps = num_kb;
    double best = 1e300;
    for (int S = 2; S <= 8; S *= 2) {
        if (num_kb / S < 4) break;
        const int kbps = (num_kb + S - 1) / S;
        if (static_cast<int64_t>(kbps) * (S - 1) >= num_kb) continue;  // an empty slice
        const int64_t slots = slots_of(S);
        if (slots < S) continue;
        if (tiles1 * S > slots) continue;  // one round only: with more the model below misjudged (160x9600x4096: 45 against 31 us)
        const double cost = static_cast<double>(kbps + 10) * 48.0;
        if (cost < best) { best = cost; best_s = S; best_kbps = kbps; }
    }
    if (best_s > 1 && best * 100.0 < cur * ratio) plan = GemmPlan{1, 1, best_s, best_kbps, 0};
    return plan;
}

int mlt_debug_gemm_plan(int64_t M, int64_t N, int64_t K, size_t workspace_bytes, int sm_count, int* out4) {
    if (!out4 || M <= 0 || N <= 0 || K <= 0 || sm_count == 1 || sm_count < 0) return MLT_ERR_INVALID_ARG;
    DeviceInfo dev;
    if (sm_count == 0) {  // the current device, with the cluster occupancy it reports
        const int rc = get_device(&dev);
        if (rc != MLT_OK) return rc;
    }
    const GemmPlan plan = sm_count == 0 ? gemm_plan(M, N, K, workspace_bytes > 0, workspace_bytes, false, dev.sm_count, dev.cluster_slots, -1)
                                        : gemm_plan(M, N, K, workspace_bytes > 0, workspace_bytes, false, sm_count, nullptr, -1);
    out4[0] = plan.even ? 3 : plan.variant;
    out4[1] = plan.split_k;
    out4[2] = plan.cluster;
    out4[3] = plan.kb_per_split;
    return MLT_OK;
}

size_t mlt_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    const int split = gemm_max_split(M, N, K);
    return split > 1 ? static_cast<size_t>(split) * M * N * sizeof(float) : 0;
}

// C is BF16 (f32_out false) or FP32 (f32_out true, optionally accumulating); A and B are BF16 or FP16.
static int gemm_run(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb,
                    int64_t ldc, void* workspace, size_t workspace_bytes, void* stream, bool f16_in = false,
                    bool f32_out = false, bool accumulate = false) {
    // ---- validation (no CUDA call before this block has passed) ----
    if (M < 0 || N < 0 || K < 0) return MLT_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return MLT_OK;
    if (!C || ldc < N) return MLT_ERR_INVALID_ARG;
    if (K > 0 && (!A || !B || lda < K || ldb < N)) return MLT_ERR_INVALID_ARG;
    if (M > INT32_MAX - 256 || N > INT32_MAX - 256 || K > INT32_MAX - 256) return MLT_ERR_UNSUPPORTED;
    if (!aligned16(C) || (ldc % (f32_out ? 4 : 8)) != 0) return MLT_ERR_ALIGNMENT;
    if (K > 0 && (!aligned16(A) || !aligned16(B) || (lda % 8) != 0 || (ldb % 8) != 0)) return MLT_ERR_ALIGNMENT;
    if (workspace && !aligned16(workspace)) return MLT_ERR_ALIGNMENT;

    DeviceInfo dev;
    int rc = get_device(&dev);
    if (rc != MLT_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    if (K == 0) {
        if (f32_out && accumulate) return MLT_OK;  // C += empty sum
        const int64_t total = M * N;
        const int blocks = static_cast<int>(std::min<int64_t>((total + 255) / 256, 4 * dev.sm_count));
        if (f32_out)
            gemm_zero_fill_f32_kernel<<<blocks, 256, 0, st>>>(static_cast<float*>(C), ldc, static_cast<int>(M),
                                                              static_cast<int>(N));
        else
            gemm_zero_fill_kernel<<<blocks, 256, 0, st>>>(static_cast<__nv_bfloat16*>(C), ldc, static_cast<int>(M),
                                                          static_cast<int>(N));
        return cudaGetLastError() == cudaSuccess ? MLT_OK : MLT_ERR_CUDA;
    }

    const GemmPlan plan = gemm_plan(M, N, K, workspace != nullptr, workspace_bytes, f32_out, dev.sm_count, dev.cluster_slots, forced_variant());
    const int variant = plan.variant;
    const int bm = variant == 0 ? kPairBM : kGemmBM;
    const int bn = variant == 2 ? 128 : 256;
    const int64_t tiles_m = (M + bm - 1) / bm;
    const int64_t tiles_n = (N + bn - 1) / bn;
    if (tiles_m * tiles_n > INT32_MAX) return MLT_ERR_UNSUPPORTED;

    CUtensorMap ta, tb;
    {
        const uint64_t dims[2] = {static_cast<uint64_t>(K), static_cast<uint64_t>(M)};
        const uint64_t strides[1] = {static_cast<uint64_t>(lda) * 2};
        const uint32_t box[2] = {kGemmBK, 128};
        rc = encode_bf16(&ta, A, 2, dims, strides, box, f16_in ? 1 : 0);
        if (rc != MLT_OK) return rc;
    }
    {
        const uint64_t dims[2] = {static_cast<uint64_t>(N), static_cast<uint64_t>(K)};
        const uint64_t strides[1] = {static_cast<uint64_t>(ldb) * 2};
        const uint32_t box[2] = {64, kGemmBK};
        rc = encode_bf16(&tb, B, 2, dims, strides, box, f16_in ? 1 : 0);
        if (rc != MLT_OK) return rc;
    }

    CUtensorMap tc = tb;  // only read by the kernels when C is FP32
    const bool c_tma = f32_out && N >= 4;
    if (c_tma) {
        // the TMA store works in 16-byte units: the map ends at N rounded down to a multiple of 4 columns
        const uint64_t dims[2] = {static_cast<uint64_t>(N) & ~3ull, static_cast<uint64_t>(M)};
        const uint64_t strides[1] = {static_cast<uint64_t>(ldc) * 4};
        const uint32_t box[2] = {32, 32};  // 128-byte rows: one epilogue warp's 32 rows x 32 columns
        rc = encode_bf16(&tc, C, 2, dims, strides, box, 2);
        if (rc != MLT_OK) return rc;
    }

    GemmParams p;
    p.C = static_cast<__nv_bfloat16*>(C);
    p.ldc = ldc;
    p.M = static_cast<int>(M);
    p.N = static_cast<int>(N);
    p.K = static_cast<int>(K);
    p.tiles_m = static_cast<int>(tiles_m);
    p.tiles_n = static_cast<int>(tiles_n);
    p.split_k = 1;
    p.kb_per_split = static_cast<int>((K + kGemmBK - 1) / kGemmBK);
    p.partial = nullptr;
    p.Cf = f32_out ? static_cast<float*>(C) : nullptr;
    p.ldcf = ldc;
    p.accumulate = accumulate ? 1 : 0;
    p.f16_inputs = f16_in ? 1u : 0u;
    p.full_items = p.num_items = 0;
    const int cluster_s = plan.cluster;
    p.even_units = 0;
    if (plan.split_k > 1) {
        // Few tiles and more than half an SM count of them: K is cut into slices, FP32 partials go to the caller's scratch
        p.kb_per_split = plan.kb_per_split;
        p.split_k = plan.split_k;
        p.partial = static_cast<float*>(workspace);
        if (plan.even) p.even_units = plan.kb_per_split;
    }
    if (variant == 0) {
        // M-tiles per raster group: wide problems re-read B once per group, so fewer, taller groups pay
        p.group_m = debug_env().gemm_group_m ? debug_env().gemm_group_m : (tiles_n >= 32 ? 16 : 8);
        // A last wave that would occupy at most half of the SM pairs runs as twice as many 256 x 128 half tiles
        const int pairs = dev.sm_count / 2;
        const int num_tiles = static_cast<int>(tiles_m * tiles_n);
        const int rem = num_tiles % pairs;
        p.full_items = (rem > 0 && 2 * rem <= pairs && !debug_env().gemm_no_half) ? num_tiles - rem : num_tiles;
        p.num_items = p.full_items + 2 * (num_tiles - p.full_items);
        const int clusters = std::min(p.num_items, pairs);
        if (c_tma)
            gemm_bf16_pair_kernel<6, true><<<2 * clusters, kGemmThreads, GemmPairSmem<6>::kTotal, st>>>(ta, tb, tc, p);
        else
            gemm_bf16_pair_kernel<6, false><<<2 * clusters, kGemmThreads, GemmPairSmem<6>::kBf16Staging, st>>>(ta, tb, tc, p);
    } else if (cluster_s > 1) {
        // Skinny problem with few tiles: K is cut inside clusters of S CTAs per tile, which reduce through
        // distributed shared memory (gemm_bf16_clusterk_kernel)
        const int S = cluster_s;
        p.group_m = 16;
        p.kb_per_split = plan.kb_per_split;
        if (static_cast<int64_t>(p.kb_per_split) * (S - 1) >= (K + kGemmBK - 1) / kGemmBK) return MLT_ERR_UNSUPPORTED;  // an empty slice: the plan never makes one
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(tiles_m * tiles_n * S));
        cfg.blockDim = dim3(kGemmThreads);
        cfg.dynamicSmemBytes = variant == 1 ? GemmSmem<256, 4>::kNoStaging : GemmSmem<128, 6>::kNoStaging;
        cfg.stream = st;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = static_cast<unsigned>(S);
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        const cudaError_t e = variant == 1 ? cudaLaunchKernelEx(&cfg, gemm_bf16_clusterk_kernel<256, 4>, ta, tb, p)
                                           : cudaLaunchKernelEx(&cfg, gemm_bf16_clusterk_kernel<128, 6>, ta, tb, p);
        if (e != cudaSuccess) return MLT_ERR_CUDA;
    } else {
        p.group_m = 16;
        const int64_t work_items = p.even_units > 0
                                       ? (tiles_m * tiles_n * ((K + kGemmBK - 1) / kGemmBK) + p.even_units - 1) / p.even_units
                                       : tiles_m * tiles_n * p.split_k;
        const int grid = static_cast<int>(std::min<int64_t>(work_items, dev.sm_count));
        if (variant == 1 && c_tma)
            gemm_bf16_kernel<256, 4, true><<<grid, kGemmThreads, GemmSmem<256, 4>::kTotal, st>>>(ta, tb, tc, p);
        else if (variant == 1)
            gemm_bf16_kernel<256, 4, false><<<grid, kGemmThreads, GemmSmem<256, 4>::kNoStaging, st>>>(ta, tb, tc, p);
        else if (c_tma)
            gemm_bf16_kernel<128, 6, true><<<grid, kGemmThreads, GemmSmem<128, 6>::kTotal, st>>>(ta, tb, tc, p);
        else
            gemm_bf16_kernel<128, 6, false><<<grid, kGemmThreads, GemmSmem<128, 6>::kBf16Staging, st>>>(ta, tb, tc, p);
        if (p.split_k > 1) {
            if (cudaGetLastError() != cudaSuccess) return MLT_ERR_CUDA;
            const int64_t groups = M * ((N + 7) / 8);
            const int blocks = static_cast<int>(std::min<int64_t>((groups + 255) / 256, 8 * dev.sm_count));
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(blocks);
            cfg.blockDim = dim3(256);
            cfg.stream = st;
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr.val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            if (cudaLaunchKernelEx(&cfg, gemm_splitk_reduce_kernel, static_cast<const float*>(p.partial), p.C, ldc, p.M, p.N,
                                   p.split_k, p.even_units, static_cast<int>((K + kGemmBK - 1) / kGemmBK), p.tiles_m) != cudaSuccess)
                return MLT_ERR_CUDA;
        }
    }
    return cudaGetLastError() == cudaSuccess ? MLT_OK : MLT_ERR_CUDA;
}

int mlt_gemm(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb,
             int64_t ldc, void* stream) {
    return gemm_run(A, B, C, M, N, K, lda, ldb, ldc, nullptr, 0, stream);
}

int mlt_gemm_f16(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb,
                 int64_t ldc, int accumulate, void* stream) {
    return gemm_run(A, B, C, M, N, K, lda, ldb, ldc, nullptr, 0, stream, /*f16_in=*/true, /*f32_out=*/true,
                    accumulate != 0);
}

int mlt_gemm_ex(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb,
                int64_t ldc, void* workspace, size_t workspace_bytes, void* stream) {
    return gemm_run(A, B, C, M, N, K, lda, ldb, ldc, workspace, workspace_bytes, stream);
}

int mlt_mha_fwd(const void* Q, const void* K, const void* V, void* O, float* LSE, int B, int H, int Nq, int Nk, int D,
                int causal, float scale, void* stream) {
    if (B < 0 || H < 0 || Nq < 0 || Nk < 0) return MLT_ERR_INVALID_ARG;
    if (static_cast<int64_t>(B) * H * Nq == 0) return MLT_OK;
    if (Nk == 0) return MLT_ERR_INVALID_ARG;
    if (!Q || !K || !V || !O) return MLT_ERR_INVALID_ARG;
    if (causal && Nq > Nk) return MLT_ERR_INVALID_ARG;
    if (!(scale > 0.0f) || scale > 3.0e38f) return MLT_ERR_INVALID_ARG;  // zero, negative, NaN or infinite
    if (D != 64 && D != 128) return MLT_ERR_UNSUPPORTED;
    if (static_cast<int64_t>(B) * H > INT32_MAX / 2) return MLT_ERR_UNSUPPORTED;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return MLT_ERR_ALIGNMENT;

    DeviceInfo dev;
    int rc = get_device(&dev);
    if (rc != MLT_OK) return rc;
    if (!dev.mha_ok) return MLT_ERR_UNSUPPORTED;  // this build of the kernel must not be launched (see mha_configure)

    CUtensorMap tq, tk, tv, to;
    const uint64_t bh = static_cast<uint64_t>(B) * H;
    const uint32_t box[3] = {64, kMhaBlock, 1};
    {
        const uint64_t dims[3] = {static_cast<uint64_t>(D), static_cast<uint64_t>(Nq), bh};
        const uint64_t strides[2] = {static_cast<uint64_t>(D) * 2, static_cast<uint64_t>(Nq) * D * 2};
        rc = encode_bf16(&tq, Q, 3, dims, strides, box);
        if (rc != MLT_OK) return rc;
        const uint32_t obox[3] = {64, 32, 1};  // the output is stored per warp: 32 rows x 64 columns
        rc = encode_bf16(&to, O, 3, dims, strides, obox);
        if (rc != MLT_OK) return rc;
    }
    {
        const uint64_t dims[3] = {static_cast<uint64_t>(D), static_cast<uint64_t>(Nk), bh};
        const uint64_t strides[2] = {static_cast<uint64_t>(D) * 2, static_cast<uint64_t>(Nk) * D * 2};
        rc = encode_bf16(&tk, K, 3, dims, strides, box);
        if (rc != MLT_OK) return rc;
        rc = encode_bf16(&tv, V, 3, dims, strides, box);
        if (rc != MLT_OK) return rc;
    }
    return mha_launch(tq, tk, tv, to, LSE, B, H, Nq, Nk, D, causal != 0, scale,
                      dev.sm_count, static_cast<cudaStream_t>(stream), debug_env().mha_head_group,
                      debug_env().mha_grid);
}

size_t mlt_paged_attn_workspace_bytes(int num_seqs, int H, int D) {
    if (num_seqs <= 0 || H <= 0 || D <= 0) return 0;
    return paged_workspace_bytes(num_seqs, H, D, kPagedMaxSplits);
}

namespace {
// Shared front end of the paged-decode entry points: validation and parameter block.  Returns MLT_OK with
// *launch = false when there is nothing to do.
int paged_prepare(const void* Q, const void* K_cache, const void* V_cache, const int32_t* block_table,
                  const int32_t* seq_lens, void* O, float* LSE, int num_seqs, int H, int H_kv, int D, int block_size,
                  int max_blocks_per_seq, int num_blocks, float scale, PagedParams* p, DeviceInfo* dev, bool* launch) {
    *launch = false;
    if (num_seqs < 0 || H < 0 || H_kv < 0 || max_blocks_per_seq < 0 || num_blocks < 0) return MLT_ERR_INVALID_ARG;
    if (num_seqs == 0 || H == 0) return MLT_OK;
    if (!Q || !K_cache || !V_cache || !block_table || !seq_lens || !O) return MLT_ERR_INVALID_ARG;
    if (H_kv == 0 || H % H_kv != 0) return MLT_ERR_INVALID_ARG;
    if (!(scale > 0.0f) || scale > 3.0e38f) return MLT_ERR_INVALID_ARG;
    const int group = H / H_kv;
    if (D != 64 && D != 128) return MLT_ERR_UNSUPPORTED;
    if (group != 1 && group != 2 && group != 4 && group != 8) return MLT_ERR_UNSUPPORTED;
    if (block_size != 8 && block_size != 16 && block_size != 32) return MLT_ERR_UNSUPPORTED;
    if (num_seqs > 65535 || H_kv > 65535) return MLT_ERR_UNSUPPORTED;  // grid.y / grid.z
    if (!aligned16(Q) || !aligned16(K_cache) || !aligned16(V_cache) || !aligned16(O)) return MLT_ERR_ALIGNMENT;
    int rc = get_device(dev);
    if (rc != MLT_OK) return rc;
    p->Q = static_cast<const __nv_bfloat16*>(Q);
    p->K_cache = static_cast<const __nv_bfloat16*>(K_cache);
    p->V_cache = static_cast<const __nv_bfloat16*>(V_cache);
    p->block_table = block_table;
    p->seq_lens = seq_lens;
    p->O = static_cast<__nv_bfloat16*>(O);
    p->LSE = LSE;
    p->part_o = nullptr;
    p->part_ml = nullptr;
    p->num_seqs = num_seqs;
    p->H = H;
    p->H_kv = H_kv;
    p->block_size = block_size;
    p->max_blocks = max_blocks_per_seq;
    p->num_blocks = num_blocks;
    p->splits = paged_choose_splits(num_seqs, H_kv, H / H_kv, max_blocks_per_seq, dev->sm_count);
    if (debug_env().paged_splits) p->splits = std::min(debug_env().paged_splits, kPagedMaxSplits);
    p->scale_log2e = scale * 1.4426950408889634f;
    p->head_groups = 1;
    p->balanced = 0;
    p->balanced_ctas = 0;
    *launch = true;
    return MLT_OK;
}
}  // namespace

int mlt_paged_attn_decode(const void* Q, const void* K_cache, const void* V_cache, const int32_t* block_table,
                          const int32_t* seq_lens, void* O, float* LSE, int num_seqs, int H, int H_kv, int D,
                          int block_size, int max_blocks_per_seq, int num_blocks, float scale, void* workspace,
                          size_t workspace_bytes, void* stream) {
    PagedParams p;
    DeviceInfo dev;
    bool launch = false;
    if (workspace && !aligned16(workspace)) return MLT_ERR_ALIGNMENT;
    int rc = paged_prepare(Q, K_cache, V_cache, block_table, seq_lens, O, LSE, num_seqs, H, H_kv, D, block_size,
                           max_blocks_per_seq, num_blocks, scale, &p, &dev, &launch);
    if (rc != MLT_OK || !launch) return rc;
    // use as many splits as the caller's scratch allows
    if (!workspace) workspace_bytes = 0;
    if (paged_use_balanced(p, dev.sm_count) && paged_workspace_bytes(num_seqs, H, D, kPagedMaxSplits) <= workspace_bytes)
        paged_set_balanced(&p, dev.sm_count);
    while (p.splits > 1 && paged_workspace_bytes(num_seqs, H, D, p.splits) > workspace_bytes) --p.splits;
    p.blocks_per_split = paged_blocks_per_split(max_blocks_per_seq, p.splits, block_size, H / H_kv);
    return paged_launch(p, D, workspace, static_cast<cudaStream_t>(stream));
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------------------
// Paged-attention decode for callers that cannot provide scratch memory.
//
// Some callers have no device memory to give and no way to get any at the point of the call: a serving engine
// whose own pool already owns the whole GPU, a plug-in that is handed tensors but no allocator, or code on a
// latency-critical path where a cudaMalloc (which synchronises the device) is forbidden once the loop runs.  For
// them the partial results of the split sequences go into a fixed array that is part of this library's device
// image.  Every GPU that loads the library carries the array until the process exits, so it is kept modest.
// ---------------------------------------------------------------------------------------------------------
namespace {

static __device__ __align__(256) unsigned char g_paged_static_scratch[MLT_PAGED_STATIC_SCRATCH_BYTES];

// In host code `g_paged_static_scratch` is only a handle for the runtime, not a device address: the address each
// device gave the array is looked up once per device (with that device current) and kept here.
void* g_paged_static_scratch_addr[64] = {};

int paged_static_scratch(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MLT_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_paged_static_scratch_addr[dev]) {
        void* addr = nullptr;
        if (cudaGetSymbolAddress(&addr, g_paged_static_scratch) != cudaSuccess || !addr) return MLT_ERR_CUDA;
        g_paged_static_scratch_addr[dev] = addr;
    }
    *out = g_paged_static_scratch_addr[dev];
    return MLT_OK;
}

}  // namespace

extern "C" int mlt_paged_attn_decode_static(const void* Q, const void* K_cache, const void* V_cache,
                                            const int32_t* block_table, const int32_t* seq_lens, void* O, float* LSE,
                                            int num_seqs, int H, int H_kv, int D, int block_size,
                                            int max_blocks_per_seq, int num_blocks, float scale, void* stream) {
    PagedParams p;
    DeviceInfo dev;
    bool launch = false;
    int rc = paged_prepare(Q, K_cache, V_cache, block_table, seq_lens, O, LSE, num_seqs, H, H_kv, D, block_size,
                           max_blocks_per_seq, num_blocks, scale, &p, &dev, &launch);
    if (rc != MLT_OK || !launch) return rc;
    // the same split as mlt_paged_attn_decode makes with a full workspace; it must fit the built-in array
    if (paged_use_balanced(p, dev.sm_count) &&
        paged_workspace_bytes(num_seqs, H, D, kPagedMaxSplits) <= static_cast<size_t>(MLT_PAGED_STATIC_SCRATCH_BYTES))
        paged_set_balanced(&p, dev.sm_count);
    if (paged_workspace_bytes(num_seqs, H, D, p.splits) > static_cast<size_t>(MLT_PAGED_STATIC_SCRATCH_BYTES))
        return MLT_ERR_SCRATCH_LIMIT;
    p.blocks_per_split = paged_blocks_per_split(max_blocks_per_seq, p.splits, block_size, H / H_kv);
    void* scratch = nullptr;
    rc = paged_static_scratch(&scratch);
    if (rc != MLT_OK) return rc;
    // nothing in the array has to start at zero: every partial the combine step reads was written by this call
    return paged_launch(p, D, scratch, static_cast<cudaStream_t>(stream));
}
