// C ABI of the SLoPe 2:4-sparse linear layer for B200 (sm_100a): argument checks,
// TMA descriptor construction and kernel launches.  No device memory is allocated here.
#include "../../include/slope.h"

#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <utility>

#include "dw_adapter_kernel.cuh"
#include "gemm_kernels.cuh"
#include "nm_kernels.cuh"
#include "prune_kernels.cuh"

namespace slope {

static std::atomic<unsigned long long> g_launches{0};

// ------------------------------------------------------------------ device / driver set-up
struct DeviceInfo {
    bool ok = false;
    int sm_count = 0;
    int cc_major = 0;
};

static DeviceInfo device_info() {
    static std::mutex mu;
    static DeviceInfo cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DeviceInfo{};
    std::lock_guard<std::mutex> lock(mu);
    if (!cache[dev].ok) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return DeviceInfo{};
        cache[dev].sm_count = prop.multiProcessorCount;
        cache[dev].cc_major = prop.major;
        cache[dev].ok = true;
    }
    return cache[dev];
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    });
    return fn;
}

// Encoding a tensor map is a pure function of (address, extents, box, kind) and costs the host
// about a microsecond; a layer calls with the same buffers step after step.  Each host thread
// keeps the last encodings in a small direct-mapped table (no locks, nothing shared).
struct TmapKey {
    const void* base;
    long long rows;
    int cols, box_rows, box_cols, kind;
    bool operator==(const TmapKey& o) const {
        return base == o.base && rows == o.rows && cols == o.cols && box_rows == o.box_rows && box_cols == o.box_cols &&
               kind == o.kind;
    }
};
struct TmapSlot {
    TmapKey key;
    CUtensorMap tm;
    bool valid;
};
constexpr int kTmapSlots = 256;

static TmapSlot& tmap_slot(const TmapKey& k) {
    thread_local TmapSlot table[kTmapSlots] = {};
    unsigned long long h = reinterpret_cast<uintptr_t>(k.base) >> 4;
    h = h * 0x9E3779B97F4A7C15ull + static_cast<unsigned long long>(k.rows) * 0xC2B2AE3D27D4EB4Full;
    h ^= (static_cast<unsigned long long>(k.cols) << 20) ^ (static_cast<unsigned long long>(k.box_rows) << 8) ^
         (static_cast<unsigned long long>(k.box_cols) << 2) ^ static_cast<unsigned long long>(k.kind);
    h ^= h >> 29;
    return table[h % kTmapSlots];
}

template <typename Encode>
static bool tmap_memo(CUtensorMap* tm, const TmapKey& key, Encode encode) {
    TmapSlot& slot = tmap_slot(key);
    if (slot.valid && slot.key == key) {
        std::memcpy(tm, &slot.tm, sizeof(CUtensorMap));
        return true;
    }
    if (!encode(tm)) return false;
    slot.key = key;
    std::memcpy(&slot.tm, tm, sizeof(CUtensorMap));
    slot.valid = true;
    return true;
}

// 2-D bf16 tensor map over a row-major [rows x cols] matrix, 128-byte swizzle,
// box = box_cols (<= 64) x box_rows, out-of-bounds elements read as zero.
static bool make_tmap(CUtensorMap* tm, const void* base, int rows, int cols, int box_rows, int box_cols) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
    const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(cols) * 2};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    return tmap_memo(tm, TmapKey{base, rows, cols, box_rows, box_cols, 0}, [&](CUtensorMap* out) {
        return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

// Metadata as a 2-D tensor of 8-byte words [blocks x 256]: one 2 KB block is ONE contiguous row,
// so a block costs the TMA unit a single request (a 128 x 16-byte box costs 128).
static bool make_tmap_meta(CUtensorMap* tm, const void* base, size_t total_bytes) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t gdim[2] = {256, static_cast<cuuint64_t>(total_bytes / 2048)};
    const cuuint64_t gstride[1] = {2048};
    const cuuint32_t box[2] = {256, 1};
    const cuuint32_t estr[2] = {1, 1};
    return tmap_memo(tm, TmapKey{base, static_cast<long long>(total_bytes / 2048), 256, 1, 256, 1}, [&](CUtensorMap* out) {
        return fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

// 2-D bf16 tensor map for TMA stores of output tiles: unswizzled, or (for a box 64 bytes wide) with
// the 64-byte swizzle the transposing epilogues write their staging tiles in.
static bool make_tmap_plain(CUtensorMap* tm, const void* base, int rows, int cols, int box_rows, int box_cols,
                            bool swizzle64 = false) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
    const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(cols) * 2};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    return tmap_memo(tm, TmapKey{base, rows, cols, box_rows, box_cols, swizzle64 ? 3 : 2}, [&](CUtensorMap* out) {
        return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_NONE,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

// Launch with thread-block clusters of `cluster` CTAs along x.
template <typename... KArgs, typename... Args>
static slope_status_t launch_cluster_ex(void (*kern)(KArgs...), int grid, int cluster, int threads, int smem_bytes,
                                        bool overlap_prologue, cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // Programmatic dependent launch: the kernel may be scheduled while its predecessor in the
    // stream drains; it synchronises on the device (griddepcontrol.wait) before touching memory.
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_prologue ? 2 : 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? SLOPE_OK : SLOPE_ERR_CUDA;
}

template <typename... KArgs, typename... Args>
static slope_status_t launch_cluster(void (*kern)(KArgs...), int grid, int cluster, int threads, int smem_bytes,
                                     cudaStream_t stream, Args&&... args) {
    return launch_cluster_ex(kern, grid, cluster, threads, smem_bytes, false, stream, std::forward<Args>(args)...);
}

// How many clusters of `cluster` CTAs of this kernel the device holds at once (0: query failed).
template <typename Kernel>
static int max_active_clusters(Kernel kern, int cluster, int threads, int smem_bytes, int sm_count) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cluster * sm_count * 8, 1, 1);      // (the answer is capped by the grid of the query)
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = cluster;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

// Launch on clusters of two CTAs (cta_group::2 kernels).
template <typename... KArgs, typename... Args>
static slope_status_t launch_pairs(void (*kern)(KArgs...), int grid, int threads, int smem_bytes,
                                   cudaStream_t stream, Args&&... args) {
    return launch_cluster_ex(kern, grid, 2, threads, smem_bytes, /*overlap_prologue=*/true, stream,
                             std::forward<Args>(args)...);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static slope_status_t check_arch(DeviceInfo& info) {
    info = device_info();
    if (!info.ok) return SLOPE_ERR_CUDA;
    if (info.cc_major != 10) return SLOPE_ERR_UNSUPPORTED_ARCH;
    return SLOPE_OK;
}

static slope_status_t launch_result() {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? SLOPE_OK : SLOPE_ERR_CUDA;
}

// Opt in to more than 48 KB of dynamic shared memory.  The attribute belongs to the kernel in
// the current device's context; every host thread remembers which (kernel, device) pairs it has
// already set (a process-wide flag would be wrong for a second device).
template <typename Kernel>
static bool set_smem(Kernel k, int bytes) {
    struct Done {
        const void* fn;
        int dev, bytes;
    };
    constexpr int kMax = 64;
    thread_local Done done[kMax];
    thread_local int n_done = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    const void* fn = reinterpret_cast<const void*>(k);
    for (int i = 0; i < n_done; ++i)
        if (done[i].fn == fn && done[i].dev == dev && done[i].bytes >= bytes) return true;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    // all of the SM's L1 / shared memory as shared memory: a kernel that asks for under half of it
    // would otherwise get a carve-out that holds only one of its CTAs
    if (cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) !=
        cudaSuccess)
        return false;
    if (n_done < kMax) done[n_done++] = Done{fn, dev, bytes};
    return true;
}

// Grid of the grid-stride streaming kernels: many short blocks per SM keep the tail of the last
// wave short (masked copy of a 90 MB matrix: 78 % of the HBM peak with 8 blocks per SM, 91 % with 32).
constexpr int kStreamBlocksPerSm = 32;

// ------------------------------------------------------------------ dense GEMM launch
struct DenseProblem {
    const void* A = nullptr;
    const void* B = nullptr;
    int M = 0, N = 0, K = 0, k_splits = 1;
    void* out = nullptr;
    const void* mask = nullptr;
    int pdl_mode = 0;
};

// One launch of the 1-CTA dense kernel over one or two problems of the same kind.
template <bool A_MN, bool B_MN, int BLOCK_N, int EPI, int STAGES>
static slope_status_t launch_dense2(const DenseProblem& q0, const DenseProblem& q1, cudaStream_t stream,
                                    const DeviceInfo& info) {
    using Cfg = DenseCfg<BLOCK_N, STAGES>;
    CUtensorMap tm[4];
    DenseGemmParams p[2];
    int tiles = 0;
    for (int i = 0; i < 2; ++i) {
        const DenseProblem& q = i == 0 ? q0 : (q1.M > 0 ? q1 : q0);          // unused slot mirrors problem 0
        const bool okA = A_MN ? make_tmap(&tm[2 * i], q.A, q.K, q.M, 64, 64) : make_tmap(&tm[2 * i], q.A, q.M, q.K, kBlockM, 64);
        const bool okB = B_MN ? make_tmap(&tm[2 * i + 1], q.B, q.K, q.N, 64, 64)
                              : make_tmap(&tm[2 * i + 1], q.B, q.N, q.K, BLOCK_N, 64);
        if (!okA || !okB) return SLOPE_ERR_CUDA;
        const bool live = i == 0 || q1.M > 0;
        p[i].M = live ? q.M : 0; p[i].N = q.N; p[i].K = q.K; p[i].k_splits = q.k_splits; p[i].out = q.out;
        p[i].mask = static_cast<const uint8_t*>(q.mask);
        p[i].pdl_mode = q0.pdl_mode;
        if (live) tiles += ((q.M + kBlockM - 1) / kBlockM) * ((q.N + BLOCK_N - 1) / BLOCK_N) * q.k_splits;
    }
    auto kern = dense_gemm_kernel<A_MN, B_MN, BLOCK_N, EPI, STAGES>;
    if (!set_smem(kern, Cfg::kSmemBytes)) return SLOPE_ERR_CUDA;
    int grid = tiles < info.sm_count ? tiles : info.sm_count;
    // The producer of a fused pair runs beside a kernel of CTA pairs: launched as clusters of two its
    // CTAs fill whole SM pairs instead of breaking up many (the kernel itself ignores the cluster;
    // a CTA without a tile exits at once).
    const int cluster = q0.pdl_mode == 1 ? 2 : 1;
    if (cluster == 2) grid = (grid + 1) & ~1;
    return launch_cluster_ex(kern, grid, cluster, kGemmThreads, Cfg::kSmemBytes, /*overlap_prologue=*/true, stream,
                             tm[0], tm[1], p[0], tm[2], tm[3], p[1]);
}

template <bool A_MN, bool B_MN, int BLOCK_N, int EPI, int STAGES>
static slope_status_t launch_dense(const void* A, const void* B, int M, int N, int K, int k_splits, void* out,
                                   const void* mask, cudaStream_t stream, const DeviceInfo& info, int pdl_mode = 0) {
    DenseProblem q;
    q.A = A; q.B = B; q.M = M; q.N = N; q.K = K; q.k_splits = k_splits; q.out = out; q.mask = mask;
    q.pdl_mode = pdl_mode;
    return launch_dense2<A_MN, B_MN, BLOCK_N, EPI, STAGES>(q, DenseProblem{}, stream, info);
}

// ------------------------------------------------------------------ CTA-pair launches (main GEMMs)
constexpr int kPairBlockN = 224;             // token tile of the big-tile kernels
constexpr int kPairStages = 4;
constexpr int kPairNarrowBlockN = 128;       // narrower 256-row tile for shapes with few tiles
constexpr int kPairNarrowStages = 5;

template <int BLOCK_N, int STAGES>
static slope_status_t launch_sparse_pair(const void* act, int ntok, const void* vals, const void* meta, int M, int K,
                                         const void* act2, const void* fac2, int r, bool a2_mn, void* out,
                                         cudaStream_t stream, const DeviceInfo& info, int pdl_mode = 0,
                                         int reserved_ctas = 0) {
    using Cfg = SparsePairCfg<BLOCK_N, STAGES>;
    CUtensorMap tmA, tmB, tmE, tmA2, tmB2, tmO;
    if (!make_tmap(&tmA, vals, M, K / 2, kBlockM, 64)) return SLOPE_ERR_CUDA;
    if (!make_tmap(&tmB, act, ntok, K, Cfg::kHalfN, 64)) return SLOPE_ERR_CUDA;
    if (!make_tmap_meta(&tmE, meta, static_cast<size_t>(M) * K / 8)) return SLOPE_ERR_CUDA;
    if (!make_tmap_plain(&tmO, out, ntok, M, Cfg::kStoreRows, Cfg::kStoreCols, true)) return SLOPE_ERR_CUDA;
    if (r > 0) {
        const bool ok2 = a2_mn ? make_tmap(&tmA2, fac2, r, M, 64, 64) : make_tmap(&tmA2, fac2, M, r, kBlockM, 64);
        if (!ok2 || !make_tmap(&tmB2, act2, ntok, r, Cfg::kHalfN, 64)) return SLOPE_ERR_CUDA;
    } else {
        tmA2 = tmA;
        tmB2 = tmB;
    }
    SparseGemmParams p = {};
    p.M = M; p.K = K; p.Ntok = ntok; p.r = r; p.a2_mn_major = a2_mn ? 1 : 0;
    p.meta = static_cast<const uint8_t*>(meta);
    p.out = static_cast<uint16_t*>(out);
    auto kern = sparse_gemm_pair_kernel<BLOCK_N, STAGES>;
    if (!set_smem(kern, Cfg::kSmemBytes)) return SLOPE_ERR_CUDA;
    p.pdl_mode = pdl_mode;
    const int tiles = ((M / kBlockM + 1) / 2) * ((ntok + BLOCK_N - 1) / BLOCK_N);
    // (the consumer of a fused pair leaves the producer's SMs alone)
    const int max_pairs = (info.sm_count - reserved_ctas) / 2;
    const int pairs = tiles < max_pairs ? tiles : max_pairs;
    return launch_pairs(kern, 2 * pairs, Cfg::kThreads, Cfg::kSmemBytes, stream, tmA, tmB, tmE, tmA2, tmB2, tmO, p);
}

constexpr int kQuadBlockN = 224;
constexpr int kQuadStages = 3;

// Row tiles per raster group of the 512-row-tile kernel (see quad_tile).  All pairs that work on
// one token block share its activations, so with every row tile in one group the activations
// cross HBM once -- but a wave of the machine then touches the whole compressed weight, and
// when that is more than L2 keeps next to the streams (about 30 MB here) it is fetched again
// every wave.  Splitting the row tiles into g groups re-reads the activations g times and keeps
// a group's weights resident.  Pick the g with the least estimated DRAM traffic
// (measured at 16384 tokens: 4096 -> 11008 two groups +7 %, 5120 -> 13824 three groups +11 %,
// square and long-reduction layers one group).
static int quad_group_m(int M, int K, int ntok, int num_pairs) {
    const int num_m = (M / kBlockM + 3) / 4, num_n = (ntok + kPairBlockN - 1) / kPairBlockN;
    const double w_tile = 512.0 * K * 1.125, w_total = static_cast<double>(M) * K * 1.125;
    const double x_total = static_cast<double>(ntok) * K * 2.0;
    constexpr double kL2Keeps = 30e6;
    int best_gm = num_m;
    double best = 1e300;
    for (int g = 1; g <= num_m; ++g) {
        const int gm = (num_m + g - 1) / g, groups = (num_m + gm - 1) / gm;
        const double rounds = static_cast<double>(gm) * num_n / num_pairs;
        const double traffic = groups * x_total + (gm * w_tile <= kL2Keeps ? w_total : w_total * (rounds > 1.0 ? rounds : 1.0));
        if (traffic < best * 0.98) { best = traffic; best_gm = gm; }       // prefer fewer groups on a near tie
    }
    return best_gm;
}

static slope_status_t launch_sparse_quad(const void* act, int ntok, const void* vals, const void* meta, int M, int K,
                                         const void* act2, const void* fac2, int r, bool a2_mn, void* out,
                                         cudaStream_t stream, const DeviceInfo& info, int pdl_mode = 0,
                                         int reserved_ctas = 0) {
    using Cfg = SparseQuadCfg<kQuadBlockN, kQuadStages>;
    CUtensorMap tmA, tmB, tmE, tmA2, tmB2, tmO;
    if (!make_tmap(&tmA, vals, M, K / 2, kBlockM, 64)) return SLOPE_ERR_CUDA;
    if (!make_tmap(&tmB, act, ntok, K, Cfg::kHalfN, 64)) return SLOPE_ERR_CUDA;
    if (!make_tmap_meta(&tmE, meta, static_cast<size_t>(M) * K / 8)) return SLOPE_ERR_CUDA;
    if (!make_tmap_plain(&tmO, out, ntok, M, Cfg::kStoreRows, Cfg::kStoreCols)) return SLOPE_ERR_CUDA;
    if (r > 0) {
        const bool ok2 = a2_mn ? make_tmap(&tmA2, fac2, r, M, 64, 64) : make_tmap(&tmA2, fac2, M, r, kBlockM, 64);
        if (!ok2 || !make_tmap(&tmB2, act2, ntok, r, Cfg::kHalfN, 64)) return SLOPE_ERR_CUDA;
    } else {
        tmA2 = tmA;
        tmB2 = tmB;
    }
    SparseGemmParams p = {};
    p.M = M; p.K = K; p.Ntok = ntok; p.r = r; p.a2_mn_major = a2_mn ? 1 : 0;
    p.meta = static_cast<const uint8_t*>(meta);
    p.out = static_cast<uint16_t*>(out);
    const int max_pairs = (info.sm_count - reserved_ctas) / 2;
    p.pdl_mode = pdl_mode;
    p.group_m = quad_group_m(M, K, ntok, max_pairs);
    auto kern = sparse_gemm_quad_kernel<kQuadBlockN, kQuadStages>;
    if (!set_smem(kern, Cfg::kSmemBytes)) return SLOPE_ERR_CUDA;
    const int tiles = ((M / kBlockM + 3) / 4) * ((ntok + kQuadBlockN - 1) / kQuadBlockN);
    const int pairs = tiles < max_pairs ? tiles : max_pairs;
    return launch_pairs(kern, 2 * pairs, Cfg::kThreads, Cfg::kSmemBytes, stream, tmA, tmB, tmE, tmA2, tmB2, tmO, p);
}

// Few tokens (inference / decode sizes): weight-streaming kernel, K split over a cluster.
// K-splits (= cluster size) of the few-token kernel.  A CTA streams ceil(num_kb / s) k-blocks
// of 18 KB.  Measured on B200: alone an SM takes in one k-block per ~0.23 us (about one TMA row
// request per 2 ns), and once enough CTAs pull at the same time HBM is the limit (18 KB at
// 6.5 TB/s = 0.0028 us per k-block and active CTA).  Every wave of clusters pays a fixed
// start-up (launch, prologue, first-byte latency, epilogue), a split pays the cluster
// reduction.  `capacity(s)` is the number of clusters of s CTAs the device holds at once.
constexpr double kSkinnySmUs = 0.23, kSkinnyHbmUs = 0.0028, kSkinnyWaveUs = 4.0, kSkinnyReduceUs = 0.5,
                 kSkinnyReducePerRankUs = 0.07;

// A k-block costs an SM its weight tile (kSkinnySmUs) plus the activation tile's TMA row
// requests (2 per token of the tile, ~2 ns each).
constexpr double kSkinnyTokenUs = 0.004;

static int skinny_splits(int slabs, int num_kb, int block_n, const int (&cap)[9], double* est_us = nullptr) {
    int best_s = 1;
    double best_cost = 1e30;
    const double sm_us = kSkinnySmUs + kSkinnyTokenUs * block_n;
    for (int s = 1; s <= 8; ++s) {
        const int per = (num_kb + s - 1) / s;
        if ((num_kb + per - 1) / per != s) continue;                 // a rank would be left without a k-block
        if (s > 1 && per < 2) break;
        if (cap[s] <= 0) continue;
        double cost = s > 1 ? kSkinnyReduceUs + kSkinnyReducePerRankUs * s : 0.0;
        for (int left = slabs; left > 0; left -= cap[s]) {
            const int active = (left < cap[s] ? left : cap[s]) * s;
            const double per_kb = active * kSkinnyHbmUs > sm_us ? active * kSkinnyHbmUs : sm_us;
            cost += kSkinnyWaveUs + per * per_kb;
        }
        if (cost < best_cost - 1e-9) { best_cost = cost; best_s = s; }
    }
    if (est_us) *est_us = best_cost;
    return best_s;
}

// Co-resident clusters of the few-token kernel per cluster size, asked of the driver once per
// device and kernel variant.
template <int BLOCK_N, int A_STAGES, int B_STAGES>
static bool skinny_capacity(const DeviceInfo& info, int (&cap)[9]) {
    using Cfg = SparseSkinnyCfg<BLOCK_N, A_STAGES, B_STAGES>;
    static std::mutex mu;
    static int capacity[64][9];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    auto kern = sparse_gemm_skinny_kernel<BLOCK_N, A_STAGES, B_STAGES>;
    std::lock_guard<std::mutex> lock(mu);
    if (capacity[dev][1] == 0) {
        if (!set_smem(kern, Cfg::kSmemBytes)) return false;
        for (int s = 1; s <= 8; ++s)
            capacity[dev][s] = max_active_clusters(kern, s, kGemmThreads, Cfg::kSmemBytes, info.sm_count);
    }
    // The occupancy query answers one CTA per SM for every kernel that allocates tensor memory,
    // whatever its shared memory (it cannot know how many columns a CTA will ask for).  The CTA
    // scheduler itself goes by registers, warps and shared memory: two CTAs of a variant that
    // needs under half of the shared memory do run side by side (measured: a launch of 172 CTAs
    // takes one wave, not two), and their 32- or 128-column allocations fit together.
    const int per_sm = 2 * (Cfg::kSmemBytes + 1024) <= 232448 ? 2 : 1;
    cap[0] = 0;
    for (int s = 1; s <= 8; ++s) cap[s] = capacity[dev][s] * per_sm;
    return cap[1] > 0;
}

template <int BLOCK_N, int A_STAGES, int B_STAGES>
static slope_status_t launch_sparse_skinny(const void* act, int ntok, const void* vals, const void* meta, int M, int K,
                                           const void* act2, const void* fac2, int r, bool a2_mn, void* out,
                                           cudaStream_t stream, const DeviceInfo& info, int pdl_mode) {
    using Cfg = SparseSkinnyCfg<BLOCK_N, A_STAGES, B_STAGES>;
    CUtensorMap tmA, tmB, tmE, tmA2, tmB2;
    if (r > 0) {
        const bool ok2 = a2_mn ? make_tmap(&tmA2, fac2, r, M, 64, 64) : make_tmap(&tmA2, fac2, M, r, kBlockM, 64);
        if (!ok2 || !make_tmap(&tmB2, act2, ntok, r, BLOCK_N, 64)) return SLOPE_ERR_CUDA;
    }
    if (K > 0) {
        if (!make_tmap(&tmA, vals, M, K / 2, kBlockM, 64)) return SLOPE_ERR_CUDA;
        if (!make_tmap(&tmB, act, ntok, K, BLOCK_N, 64)) return SLOPE_ERR_CUDA;
        if (!make_tmap_meta(&tmE, meta, static_cast<size_t>(M) * K / 8)) return SLOPE_ERR_CUDA;
    } else {                                  // dense-only: the sparse maps are never used for a load
        if (r <= 0) return SLOPE_ERR_SHAPE;
        tmA = tmA2;
        tmB = tmB2;
        tmE = tmA2;
    }
    if (r <= 0) {
        tmA2 = tmA;
        tmB2 = tmB;
    }
    SparseGemmParams p = {};
    p.M = M; p.K = K; p.Ntok = ntok; p.r = r; p.a2_mn_major = a2_mn ? 1 : 0;
    p.pdl_mode = pdl_mode;
    p.meta = static_cast<const uint8_t*>(meta);
    p.out = static_cast<uint16_t*>(out);
    auto kern = sparse_gemm_skinny_kernel<BLOCK_N, A_STAGES, B_STAGES>;
    if (!set_smem(kern, Cfg::kSmemBytes)) return SLOPE_ERR_CUDA;

    int cap[9];
    if (!skinny_capacity<BLOCK_N, A_STAGES, B_STAGES>(info, cap)) return SLOPE_ERR_CUDA;
    if (pdl_mode == 2) {
        // The consumer of a fused pair has to be resident next to its producer (one cluster of up to 8
        // CTAs per 128 adapter columns), or its last clusters would wait for the producer to finish
        // and the overlap would be lost: count only the clusters that fit beside it.
        const int reserved = 8 * ((r + kBlockM - 1) / kBlockM);
        for (int sz = 1; sz <= 8; ++sz) {
            cap[sz] -= (reserved + sz - 1) / sz + (sz > 1 ? 1 : 0);
            if (cap[sz] < 0) cap[sz] = 0;
        }
        if (cap[1] <= 0) return SLOPE_ERR_CUDA;
    }
    const int slabs = (M + kBlockM - 1) / kBlockM, num_kb = K > 0 ? K / 128 : (r + 63) / 64;
    const int splits = skinny_splits(slabs, num_kb, BLOCK_N, cap);
    return launch_cluster_ex(kern, slabs * splits, splits, kGemmThreads, Cfg::kSmemBytes, true, stream, tmA, tmB,
                             tmE, tmA2, tmB2, p);
}

// Few-token GEMM  out[ntok x M] = act * A_2:4^T (+ act2 * fac2^T)  on the weight-streaming
// kernel, token tile chosen by the token count.  K == 0 runs the dense product alone
// (out = act2 * fac2^T with reduction length r), which serves the adapter's T = X L and
// dT = dY R^T at inference sizes.
constexpr int kSkinnyMaxTokens = 256;

// A variant of the few-token kernel with a half as deep weight ring fits two CTAs on an SM (the
// same bytes in flight per SM).  It pays when the slabs times K-slices of a launch exceed what the
// machine holds at one CTA per SM (stacked projections, d_out beyond ~19000 rows): one wave
// instead of two.  Decided by the same cost model over both variants' capacities.
template <int BLOCK_N, int A_DEEP, int B_DEEP, int A_FLAT, int B_FLAT>
static bool prefer_two_ctas_per_sm(int M, int K, const DeviceInfo& info) {
    if (K <= 0) return false;
    int cap_deep[9], cap_flat[9];
    if (!skinny_capacity<BLOCK_N, A_DEEP, B_DEEP>(info, cap_deep)) return false;
    if (!skinny_capacity<BLOCK_N, A_FLAT, B_FLAT>(info, cap_flat)) return false;
    double est_deep = 0.0, est_flat = 0.0;
    const int slabs = (M + kBlockM - 1) / kBlockM;
    skinny_splits(slabs, K / 128, BLOCK_N, cap_deep, &est_deep);
    skinny_splits(slabs, K / 128, BLOCK_N, cap_flat, &est_flat);
    return est_flat < 0.93 * est_deep;
}

static slope_status_t launch_skinny(const void* act, int ntok, const void* vals, const void* meta, int M, int K,
                                    const void* act2, const void* fac2, int r, bool a2_mn, void* out,
                                    cudaStream_t stream, const DeviceInfo& info, int pdl_mode = 0) {
    if (ntok <= 16) {
        if (prefer_two_ctas_per_sm<16, 10, 4, 5, 2>(M, K, info))
            return launch_sparse_skinny<16, 5, 2>(act, ntok, vals, meta, M, K, act2, fac2, r, a2_mn, out, stream, info, pdl_mode);
        return launch_sparse_skinny<16, 10, 4>(act, ntok, vals, meta, M, K, act2, fac2, r, a2_mn, out, stream, info, pdl_mode);
    }
    if (ntok <= 64)      // (a two-per-SM variant of this tile, <64, 4, 2>, measured slower: its activation ring is too shallow)
        return launch_sparse_skinny<64, 8, 4>(act, ntok, vals, meta, M, K, act2, fac2, r, a2_mn, out, stream, info, pdl_mode);
    if (ntok <= 128)
        return launch_sparse_skinny<128, 7, 3>(act, ntok, vals, meta, M, K, act2, fac2, r, a2_mn, out, stream, info, pdl_mode);
    return launch_sparse_skinny<256, 5, 2>(act, ntok, vals, meta, M, K, act2, fac2, r, a2_mn, out, stream, info, pdl_mode);
}

// Kernel choice for the sparse GEMMs.  Up to 256 tokens the GEMM is a weight stream from HBM and
// runs on the few-token kernel.  Beyond that three tile shapes compete:
//   512 x 224  moves 31 % fewer L2 bytes per FLOP but cannot overlap its epilogue with the next
//              tile (tensor memory holds one accumulator set).  Measured at 16384 tokens it is
//              6 % faster per unit of work at a reduction length of 4096 and 14-16 % at 11008,
//              while at 768 the 256-row tile is up to 25 % faster.
//   256 x 224  double-buffered accumulators.
//   256 x 128  the same kernel with a narrower token tile: more, smaller tiles for shapes that
//              would otherwise leave much of the last wave of the machine empty (2048 x 2048
//              with 2048 tokens: 80 tiles of 256 x 224 on 74 CTA pairs = 2 waves for 1.08 waves
//              of work); it stages the weights for fewer tokens, which costs 12 % more time
//              per unit of work at short reductions and 30-35 % at long ones (measured at 2048
//              tokens).
// The choice compares waves of the machine (tiles / CTA pairs, rounded up) times the relative
// cost of a tile.
enum class SparseTile { kQuad224, kPair224, kPair128 };

static SparseTile choose_sparse_tile(int M, int K, int ntok, int num_pairs, double* cost_out = nullptr) {
    // Waves of full tiles; the ragged last token tile of every row tile runs at its own width
    // (its weight loads do not shrink, its epilogue does: measured, a 32-token tile costs 0.7-0.9
    // of a 224-token one at reductions of 4096 and more, about 0.4 at 1024) and comes last in tile
    // order, so it first fills the pairs that the last wave of full tiles leaves idle.
    const auto rounds = [&](int rows, int block_n) {
        const int num_m = (M + rows - 1) / rows;
        const int full = num_m * (ntok / block_n), ragged = ntok % block_n;
        const int rem = full % num_pairs;
        double t = full / num_pairs + (rem ? 1.0 : 0.0);
        if (ragged) {
            const double width = ((ragged + 31) & ~31) / static_cast<double>(block_n);
            const int left = num_m - (rem ? num_pairs - rem : 0);
            const double floor = K >= 4096 ? 0.8 : K >= 2048 ? 0.65 : 0.45;
            if (left > 0) t += ((left + num_pairs - 1) / num_pairs) * (width > floor ? width : floor);
        }
        return t;
    };
    const double gain = K >= 8192 ? 0.14 : K >= 4096 ? 0.06 : K >= 2048 ? -0.05 : -0.25;
    const double cost_pair = rounds(256, kPairBlockN);
    const double cost_quad = 2.0 * (1.0 - gain) * rounds(512, kPairBlockN);
    const double narrow_penalty = K >= 8192 ? 1.35 : K >= 4096 ? 1.30 : K >= 2048 ? 1.20 : 1.12;
    const double cost_narrow = narrow_penalty * kPairNarrowBlockN / kPairBlockN * rounds(256, kPairNarrowBlockN);
    // (cost_out: the winner's cost in time units of one 256 x 224 tile)
    if (cost_quad < cost_pair && cost_quad <= cost_narrow) {
        if (cost_out) *cost_out = cost_quad;
        return SparseTile::kQuad224;
    }
    if (cost_out) *cost_out = cost_narrow < cost_pair ? cost_narrow : cost_pair;
    return cost_narrow < cost_pair ? SparseTile::kPair128 : SparseTile::kPair224;
}

// Few-token kernel or tile kernel?  Decode sizes (<= 16 tokens) always stream the weights through
// the few-token kernel.  Up to 128 tokens the two are compared by estimate: the few-token kernel's
// own cost model against a tile kernel that has one token tile, i.e. M / 256 tiles which each
// walk the whole reduction (measured: ~4 us per launch plus 0.32 us per k-block and wave of the
// machine).  A tall weight (4096 -> 11008) then has enough tiles for the tile kernel, a long
// reduction on few rows (11008 -> 4096) wants the K-split of the few-token kernel.  Beyond 128
// tokens the 256-token variant of the few-token kernel pays 512 row requests per k-block for
// its activations and loses almost everywhere (measured), so the tile kernels take over.
static bool use_few_token_kernel(int M, int K, int ntok, int r, const DeviceInfo& info) {
    if (ntok <= 16) return true;
    if (ntok > 128) return false;
    int cap[9];
    const bool ok = ntok <= 64 ? skinny_capacity<64, 8, 4>(info, cap) : skinny_capacity<128, 7, 3>(info, cap);
    if (!ok) return false;
    double few_us = 0.0;
    skinny_splits(M / kBlockM, K / 128, ntok <= 64 ? 64 : 128, cap, &few_us);
    const int num_pairs = info.sm_count / 2;
    const int tiles = (M + 255) / 256;
    const double tile_us = 4.0 + ((tiles + num_pairs - 1) / num_pairs) * (K / 128 + (r + 63) / 64) * 0.32;
    return few_us <= tile_us;
}

// One of the three tile kernels.  As the consumer of a fused pair of launches (pdl_mode 2) it leaves
// `reserved_ctas` SMs to the producer that runs beside it.
static slope_status_t launch_sparse_tiles(const void* act, int ntok, const void* vals, const void* meta, int M, int K,
                                          const void* act2, const void* fac2, int r, bool a2_mn, void* out,
                                          cudaStream_t stream, const DeviceInfo& info, int pdl_mode = 0,
                                          int reserved_ctas = 0) {
    switch (choose_sparse_tile(M, K, ntok, (info.sm_count - reserved_ctas) / 2)) {
        case SparseTile::kQuad224:
            return launch_sparse_quad(act, ntok, vals, meta, M, K, act2, fac2, r, a2_mn, out, stream, info, pdl_mode,
                                      reserved_ctas);
        case SparseTile::kPair128:
            return launch_sparse_pair<kPairNarrowBlockN, kPairNarrowStages>(act, ntok, vals, meta, M, K, act2, fac2, r,
                                                                            a2_mn, out, stream, info, pdl_mode,
                                                                            reserved_ctas);
        default:
            return launch_sparse_pair<kPairBlockN, kPairStages>(act, ntok, vals, meta, M, K, act2, fac2, r, a2_mn, out,
                                                                stream, info, pdl_mode, reserved_ctas);
    }
}

static slope_status_t launch_sparse_gemm(const void* act, int ntok, const void* vals, const void* meta, int M, int K,
                                         const void* act2, const void* fac2, int r, bool a2_mn, void* out,
                                         cudaStream_t stream, const DeviceInfo& info) {
    if (use_few_token_kernel(M, K, ntok, r, info))
        return launch_skinny(act, ntok, vals, meta, M, K, act2, fac2, r, a2_mn, out, stream, info);
    return launch_sparse_tiles(act, ntok, vals, meta, M, K, act2, fac2, r, a2_mn, out, stream, info);
}

template <bool A_MN, bool B_MN, int BLOCK_N, int EPI, int STAGES>
static slope_status_t launch_dense_pair(const void* A, const void* B, int M, int N, int K, void* out,
                                        const void* mask, cudaStream_t stream, const DeviceInfo& info) {
    using Cfg = DensePairCfg<BLOCK_N, STAGES>;
    CUtensorMap tmA, tmB;
    const bool okA = A_MN ? make_tmap(&tmA, A, K, M, 64, 64) : make_tmap(&tmA, A, M, K, kBlockM, 64);
    const bool okB = B_MN ? make_tmap(&tmB, B, K, N, 64, 64) : make_tmap(&tmB, B, N, K, Cfg::kHalfN, 64);
    if (!okA || !okB) return SLOPE_ERR_CUDA;
    DenseGemmParams p = {};
    p.M = M; p.N = N; p.K = K; p.k_splits = 1; p.out = out;
    p.mask = static_cast<const uint8_t*>(mask);
    auto kern = dense_gemm_pair_kernel<A_MN, B_MN, BLOCK_N, EPI, STAGES>;
    if (!set_smem(kern, Cfg::kSmemBytes)) return SLOPE_ERR_CUDA;
    const int tiles = ((M + 2 * kBlockM - 1) / (2 * kBlockM)) * ((N + BLOCK_N - 1) / BLOCK_N);
    const int max_pairs = info.sm_count / 2;
    const int pairs = tiles < max_pairs ? tiles : max_pairs;
    return launch_pairs(kern, 2 * pairs, kGemmThreads, Cfg::kSmemBytes, stream, tmA, tmB, p);
}

static int adapter_splits(int b, int rows) {
    // K-splits of the token reduction for the skinny adapter gradients (rows x r outputs).
    // rounds(s) = ceil(tiles * s / SMs) passes over the machine, each 1/s of a tile long; take
    // the s that minimises rounds(s) / s (with a small charge per split for the fp32 partials),
    // keeping at least 4 k-blocks (256 tokens) per split and no split without a k-block.
    // The split count sizes the caller's workspace (slope_adapter_workspace_bytes, which is asked
    // with no device at hand), so it is a function of the shape alone: the SM count is the B200's.
    constexpr int kSms = 148;
    const int tiles = (rows + kBlockM - 1) / kBlockM;
    const int num_kb = (b + 63) / 64;
    int best_s = 1;
    double best_cost = 1e30;
    for (int s = 1; s <= 16 && s * 4 <= num_kb; ++s) {
        const int rounds = (tiles * s + kSms - 1) / kSms;
        const double cost = static_cast<double>(rounds) / s + 0.004 * s;
        if (cost < best_cost - 1e-12) { best_cost = cost; best_s = s; }
    }
    const int per = (num_kb + best_s - 1) / best_s;
    return (num_kb + per - 1) / per;
}

static bool dims_ok(int d_out, int d_in) {
    return d_out > 0 && d_in > 0 && d_out % 128 == 0 && d_in % 128 == 0;
}
static bool rank_ok(int r) { return r >= 0 && r <= 256 && r % 16 == 0; }

}  // namespace slope

using namespace slope;

extern "C" {

size_t slope_values_bytes(int rows, int cols) { return static_cast<size_t>(rows) * cols; }
size_t slope_meta_bytes(int rows, int cols) { return static_cast<size_t>(rows) * cols / 8; }
size_t slope_mask_bytes(int rows, int cols) { return static_cast<size_t>(rows) * cols / 8; }

unsigned long long slope_launch_count(void) { return g_launches.load(); }

const char* slope_status_string(slope_status_t s) {
    switch (s) {
        case SLOPE_OK: return "ok";
        case SLOPE_ERR_INVALID_ARG: return "invalid argument";
        case SLOPE_ERR_SHAPE: return "unsupported shape";
        case SLOPE_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case SLOPE_ERR_UNSUPPORTED_ARCH: return "device is not sm_100";
        case SLOPE_ERR_CUDA: return "CUDA call failed";
        case SLOPE_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

slope_status_t slope_kernel_clock_mhz(int kind, void* stream, double* mhz_host) {
    if ((kind != 0 && kind != 1) || !mhz_host) return SLOPE_ERR_INVALID_ARG;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return SLOPE_ERR_CUDA;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SLOPE_ERR_CUDA;
    unsigned long long v[2][2];
    if (cudaMemcpyFromSymbol(v, g_kernel_clock, sizeof(v)) != cudaSuccess) return SLOPE_ERR_CUDA;
    // totals at the previous call, per device and kind
    static std::mutex mu;
    static unsigned long long seen[64][2][2] = {};
    std::lock_guard<std::mutex> lock(mu);
    const unsigned long long cycles = v[kind][0] - seen[dev][kind][0], ns = v[kind][1] - seen[dev][kind][1];
    seen[dev][kind][0] = v[kind][0];
    seen[dev][kind][1] = v[kind][1];
    *mhz_host = ns ? static_cast<double>(cycles) / static_cast<double>(ns) * 1e3 : 0.0;
    return SLOPE_OK;
}

slope_status_t slope_poll_status(void* stream) {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return SLOPE_ERR_CUDA;
    int st = 0;
    if (cudaMemcpyFromSymbol(&st, g_device_status, sizeof(int)) != cudaSuccess) return SLOPE_ERR_CUDA;
    if (st != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)) != cudaSuccess) return SLOPE_ERR_CUDA;
    }
    return static_cast<slope_status_t>(st);
}

slope_status_t slope_prune_24(const void* W, int d_out, int d_in, void* Wc_vals, void* Wc_meta, void* mask1_bits,
                              void* stream) {
    if (!W || !Wc_vals || !Wc_meta) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in)) return SLOPE_ERR_SHAPE;
    if (!aligned16(W) || !aligned16(Wc_vals) || !aligned16(Wc_meta) || !aligned16(mask1_bits)) return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    dim3 grid(d_in / 128, d_out / 128);
    prune24_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(W), d_out, d_in, static_cast<uint4*>(Wc_vals), static_cast<uint4*>(Wc_meta),
        static_cast<uint4*>(mask1_bits));
    return launch_result();
}

slope_status_t slope_double_prune(const void* W, const void* mask1_bits, int d_out, int d_in, void* WTc_vals,
                                  void* WTc_meta, void* mask2_bits, void* stream) {
    if (!W || !mask1_bits || !WTc_vals || !WTc_meta) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in)) return SLOPE_ERR_SHAPE;
    if (!aligned16(W) || !aligned16(mask1_bits) || !aligned16(WTc_vals) || !aligned16(WTc_meta) ||
        !aligned16(mask2_bits))
        return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    dim3 grid(d_in / 128, d_out / 128);
    double_prune_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(W), static_cast<const uint8_t*>(mask1_bits), d_out, d_in,
        static_cast<uint4*>(WTc_vals), static_cast<uint4*>(WTc_meta), static_cast<uint8_t*>(mask2_bits));
    return launch_result();
}

slope_status_t slope_prune_24_double(const void* W, int d_out, int d_in, void* Wc_vals, void* Wc_meta,
                                     void* mask1_bits, void* WTc_vals, void* WTc_meta, void* mask2_bits, void* stream) {
    if (!W || !Wc_vals || !Wc_meta || !WTc_vals || !WTc_meta) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in)) return SLOPE_ERR_SHAPE;
    if (!aligned16(W) || !aligned16(Wc_vals) || !aligned16(Wc_meta) || !aligned16(mask1_bits) || !aligned16(WTc_vals) ||
        !aligned16(WTc_meta) || !aligned16(mask2_bits))
        return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    dim3 grid(d_in / 128, d_out / 128);
    prune24_double_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(W), d_out, d_in, static_cast<uint2*>(Wc_vals), static_cast<uint4*>(Wc_meta),
        static_cast<uint4*>(mask1_bits), static_cast<uint4*>(WTc_vals), static_cast<uint4*>(WTc_meta),
        static_cast<uint8_t*>(mask2_bits));
    return launch_result();
}

slope_status_t slope_linear_fwd(const void* X, int b, const void* Wc_vals, const void* Wc_meta, int d_out, int d_in,
                                const void* T, const void* R, int r, void* Y, void* stream) {
    if (!X || !Wc_vals || !Wc_meta || !Y) return SLOPE_ERR_INVALID_ARG;
    if (r != 0 && (!T || !R)) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in) || b < 1 || !rank_ok(r)) return SLOPE_ERR_SHAPE;
    if (!aligned16(X) || !aligned16(Wc_vals) || !aligned16(Wc_meta) || !aligned16(Y) ||
        (r != 0 && (!aligned16(T) || !aligned16(R))))
        return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    return launch_sparse_gemm(X, b, Wc_vals, Wc_meta, d_out, d_in, T, R, r, /*a2_mn=*/true, Y,
                              static_cast<cudaStream_t>(stream), info);
}

static bool adapter_narrow_tiles(int b, int r, const DeviceInfo& info);

slope_status_t slope_linear_fwd_adapter(const void* X, int b, const void* Wc_vals, const void* Wc_meta, int d_out,
                                        int d_in, const void* L, const void* R, int r, void* T, void* Y,
                                        void* stream_) {
    if (!X || !Wc_vals || !Wc_meta || !L || !R || !T || !Y) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in) || b < 1 || !rank_ok(r) || r == 0) return SLOPE_ERR_SHAPE;
    if (!aligned16(X) || !aligned16(Wc_vals) || !aligned16(Wc_meta) || !aligned16(L) || !aligned16(R) ||
        !aligned16(T) || !aligned16(Y))
        return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (use_few_token_kernel(d_out, d_in, b, r, info)) {
        // Two launches of the few-token kernel as a fused pair: T = X L releases its dependent only
        // once everything before it in the stream is complete, so the forward streams its weights
        // and runs its sparse reduction while T is still being computed, and waits only for T.
        if (slope_status_t st = launch_skinny(nullptr, b, nullptr, nullptr, r, 0, X, L, d_in, true, T, stream, info, 1))
            return st;
        return launch_skinny(X, b, Wc_vals, Wc_meta, d_out, d_in, T, R, r, true, Y, stream, info, 2);
    }
    // More tokens: the tile kernels are the consumer of such a pair in the same way, as long as the
    // T launch is small enough to run beside them (it then costs the forward that share of the
    // machine, which pays while T takes a comparable time: up to 32 CTAs, i.e. 4096 tokens at r <= 128).
    const bool t_few = b <= kSkinnyMaxTokens;
    const bool t_narrow = adapter_narrow_tiles(b, r, info);
    const int t_ctas = t_few ? 8 * ((r + kBlockM - 1) / kBlockM)
                             : ((b + kBlockM - 1) / kBlockM) * (t_narrow ? (r + 63) / 64 : (r + 127) / 128);
    const int reserved = (t_ctas + 1) & ~1;
    // Worth it?  Side by side the forward runs on fewer CTA pairs (more waves of tiles, perhaps)
    // but no longer waits for T; one after the other it has the whole machine.  Tile time and T
    // time from the measured constants: ~0.33 us per 128-wide k-block and tile + ~1.5 us of
    // epilogue; a T CTA walks d_in in 64-wide steps of ~0.3 us after ~6 us of launch and start-up.
    int mode = 0;
    if (reserved <= info.sm_count / 3) {
        double cost_full = 0.0, cost_beside = 0.0;
        choose_sparse_tile(d_out, d_in, b, info.sm_count / 2, &cost_full);
        choose_sparse_tile(d_out, d_in, b, (info.sm_count - reserved) / 2, &cost_beside);
        const double tile_us = d_in / 128 * 0.33 + 1.5;
        const double t_us = t_few ? 5.0 : 6.0 + d_in / 64 * 0.3;
        const double fwd_beside = cost_beside * tile_us + 2.0;
        if (1.15 * (fwd_beside > t_us ? fwd_beside : t_us + 2.0) < t_us + cost_full * tile_us) mode = 1;
    }
    slope_status_t st;
    if (t_few)
        st = launch_skinny(nullptr, b, nullptr, nullptr, r, 0, X, L, d_in, true, T, stream, info, mode);
    else
        st = t_narrow ? launch_dense<false, true, 64, kEpiStore, 9>(X, L, b, r, d_in, 1, T, nullptr, stream, info, mode)
                      : launch_dense<false, true, 128, kEpiStore, 6>(X, L, b, r, d_in, 1, T, nullptr, stream, info, mode);
    if (st) return st;
    if (mode == 1)
        return launch_sparse_tiles(X, b, Wc_vals, Wc_meta, d_out, d_in, T, R, r, /*a2_mn=*/true, Y, stream, info, 2, reserved);
    return launch_sparse_gemm(X, b, Wc_vals, Wc_meta, d_out, d_in, T, R, r, /*a2_mn=*/true, Y, stream, info);
}

slope_status_t slope_linear_bwd_dx(const void* dY, int b, const void* WTc_vals, const void* WTc_meta, int d_out,
                                   int d_in, const void* dT, const void* L, int r, void* dX, void* stream) {
    if (!dY || !WTc_vals || !WTc_meta || !dX) return SLOPE_ERR_INVALID_ARG;
    if (r != 0 && (!dT || !L)) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in) || b < 1 || !rank_ok(r)) return SLOPE_ERR_SHAPE;
    if (!aligned16(dY) || !aligned16(WTc_vals) || !aligned16(WTc_meta) || !aligned16(dX) ||
        (r != 0 && (!aligned16(dT) || !aligned16(L))))
        return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    return launch_sparse_gemm(dY, b, WTc_vals, WTc_meta, d_in, d_out, dT, L, r, /*a2_mn=*/false, dX,
                              static_cast<cudaStream_t>(stream), info);
}

slope_status_t slope_linear_bwd_dw_masked(const void* dY, const void* X, int b, int d_out, int d_in,
                                          const void* mask1_bits, void* dWc_vals, void* stream) {
    if (!dY || !X || !mask1_bits || !dWc_vals) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in) || b < 1) return SLOPE_ERR_SHAPE;
    if (!aligned16(dY) || !aligned16(X) || !aligned16(mask1_bits) || !aligned16(dWc_vals)) return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    // Small weight matrices do not have enough 256 x 256 tiles for the 74 CTA pairs.  They run on
    // 256 x 128 tiles of CTA pairs (each CTA stages half of the X tile: GPT-2-small 33 -> 29.5 us) or,
    // when even those are few, on 128 x 128 tiles of one CTA each.
    const int pair_tiles = ((d_out + 255) / 256) * ((d_in + 255) / 256);
    if (pair_tiles * 2 <= info.sm_count) {
        const int narrow_tiles = ((d_out + 255) / 256) * ((d_in + 127) / 128);
        if (narrow_tiles >= 24)
            return launch_dense_pair<true, true, 128, kEpiMasked, 8>(dY, X, d_out, d_in, b, dWc_vals, mask1_bits,
                                                                     static_cast<cudaStream_t>(stream), info);
        return launch_dense<true, true, 128, kEpiMasked, 6>(dY, X, d_out, d_in, b, 1, dWc_vals, mask1_bits,
                                                            static_cast<cudaStream_t>(stream), info);
    }
    return launch_dense_pair<true, true, 256, kEpiMasked, 6>(dY, X, d_out, d_in, b, dWc_vals, mask1_bits,
                                                             static_cast<cudaStream_t>(stream), info);
}

// ------------------------------------------------------------------ dense layer on the same pipeline
static slope_status_t dense_args(const void* a, const void* b_, const void* c, int b, int d_out, int d_in) {
    if (!a || !b_ || !c) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in) || b < 1) return SLOPE_ERR_SHAPE;
    if (!aligned16(a) || !aligned16(b_) || !aligned16(c)) return SLOPE_ERR_ALIGNMENT;
    return SLOPE_OK;
}

slope_status_t slope_dense_linear_fwd(const void* X, int b, const void* W, int d_out, int d_in, void* Y, void* stream) {
    if (slope_status_t st = dense_args(X, W, Y, b, d_out, d_in)) return st;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    // Y[b x d_out] = X[b x d_in] * W[d_out x d_in]^T: both operands K-contiguous
    return launch_dense_pair<false, false, 256, kEpiStore, 6>(X, W, b, d_out, d_in, Y, nullptr,
                                                              static_cast<cudaStream_t>(stream), info);
}

slope_status_t slope_dense_linear_bwd_dx(const void* dY, int b, const void* W, int d_out, int d_in, void* dX,
                                         void* stream) {
    if (slope_status_t st = dense_args(dY, W, dX, b, d_out, d_in)) return st;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    // dX[b x d_in] = dY[b x d_out] * W[d_out x d_in]: W is the [K x N] operand
    return launch_dense_pair<false, true, 256, kEpiStore, 6>(dY, W, b, d_in, d_out, dX, nullptr,
                                                             static_cast<cudaStream_t>(stream), info);
}

slope_status_t slope_dense_linear_bwd_dw(const void* dY, const void* X, int b, int d_out, int d_in, void* dW,
                                         void* stream) {
    if (slope_status_t st = dense_args(dY, X, dW, b, d_out, d_in)) return st;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    // dW[d_out x d_in] = dY[b x d_out]^T * X[b x d_in]: both operands stored [K x .]
    return launch_dense_pair<true, true, 256, kEpiStore, 6>(dY, X, d_out, d_in, b, dW, nullptr,
                                                            static_cast<cudaStream_t>(stream), info);
}

static size_t adapter_partial_bytes(int b, int rows, int r) {
    return ((static_cast<size_t>(adapter_splits(b, rows)) * rows * r * sizeof(float)) + 255) & ~size_t(255);
}

size_t slope_adapter_workspace_bytes(int b, int d_out, int d_in, int r) {
    if (b <= 0 || d_out <= 0 || d_in <= 0 || r <= 0) return 0;
    return adapter_partial_bytes(b, d_in, r) + adapter_partial_bytes(b, d_out, r);     // dL and dR partial sums
}

// Column tile of the adapter products T = X L and dT = dY R^T (128 token rows per CTA).  These
// launches are bound by what one SM can pull in, so more CTAs beat fewer bytes per CTA: with
// r > 64, 64-column tiles double the CTA count (the second read of the activation rows comes from
// L2) and win as long as all of them still run in one wave.
static bool adapter_narrow_tiles(int b, int r, const DeviceInfo& info) {
    if (r <= 64) return true;
    const int wide_tiles = ((b + kBlockM - 1) / kBlockM) * ((r + 127) / 128);
    return 2 * wide_tiles <= info.sm_count;
}

// dT[b x r] = dY[b x d_out] * R[r x d_out]^T   (both K contiguous)
static slope_status_t launch_adapter_dT(const void* dY, const void* R, int b, int d_out, int r, void* dT,
                                        cudaStream_t stream, const DeviceInfo& info) {
    return b <= kSkinnyMaxTokens
               ? launch_skinny(nullptr, b, nullptr, nullptr, r, 0, dY, R, d_out, false, dT, stream, info)
           : adapter_narrow_tiles(b, r, info)
               ? launch_dense<false, false, 64, kEpiStore, 9>(dY, R, b, r, d_out, 1, dT, nullptr, stream, info)
               : launch_dense<false, false, 128, kEpiStore, 6>(dY, R, b, r, d_out, 1, dT, nullptr, stream, info);
}

// dL[d_in x r] = X^T dT and dR^T[d_out x r] = dY^T T: operands stored [K x M] / [K x N] with
// K = tokens, split into fixed slices; both problems share one launch, their fp32 partial
// sums are reduced in slice order by one more launch (dR written transposed).
static slope_status_t launch_adapter_grads(const void* X, const void* dY, const void* T, const void* dT, int b,
                                           int d_out, int d_in, int r, void* dL, void* dR, void* workspace,
                                           cudaStream_t stream, const DeviceInfo& info) {
    float* ws_l = static_cast<float*>(workspace);
    float* ws_r = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + adapter_partial_bytes(b, d_in, r));
    DenseProblem ql, qr;
    ql.A = X; ql.B = dT; ql.M = d_in; ql.N = r; ql.K = b; ql.k_splits = adapter_splits(b, d_in); ql.out = ws_l;
    qr.A = dY; qr.B = T; qr.M = d_out; qr.N = r; qr.K = b; qr.k_splits = adapter_splits(b, d_out); qr.out = ws_r;
    slope_status_t st = r <= 64 ? launch_dense2<true, true, 64, kEpiPartial, 6>(ql, qr, stream, info)
                                : launch_dense2<true, true, 128, kEpiPartial, 6>(ql, qr, stream, info);
    if (st) return st;
    const SplitKReduce rl{ws_l, static_cast<uint16_t*>(dL), d_in, r, ql.k_splits, 0};
    const SplitKReduce rr{ws_r, static_cast<uint16_t*>(dR), d_out, r, qr.k_splits, 1};
    splitk_reduce_kernel<<<info.sm_count * 4, 256, 0, stream>>>(rl, rr);
    return launch_result();
}

slope_status_t slope_adapter_fwd_bwd(int phase, const void* X, const void* dY, const void* L, const void* R, int b,
                                     int d_out, int d_in, int r, void* T, void* dT, void* dL, void* dR,
                                     void* workspace, size_t workspace_bytes, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (phase < 0 || phase > 2) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in) || b < 1 || !rank_ok(r) || r == 0) return SLOPE_ERR_SHAPE;
    DeviceInfo info;
    if (phase == 0) {
        if (!X || !L || !T) return SLOPE_ERR_INVALID_ARG;
        if (!aligned16(X) || !aligned16(L) || !aligned16(T)) return SLOPE_ERR_ALIGNMENT;
        if (slope_status_t st = check_arch(info)) return st;
        // T[b x r] = X[b x d_in] * L[d_in x r]   (A = X, K contiguous; B = L^T stored [K x N])
        if (b <= kSkinnyMaxTokens)            // few tokens: split d_in over a cluster instead of one CTA
            return launch_skinny(nullptr, b, nullptr, nullptr, r, 0, X, L, d_in, true, T, stream, info);
        return adapter_narrow_tiles(b, r, info)
                   ? launch_dense<false, true, 64, kEpiStore, 9>(X, L, b, r, d_in, 1, T, nullptr, stream, info)
                   : launch_dense<false, true, 128, kEpiStore, 6>(X, L, b, r, d_in, 1, T, nullptr, stream, info);
    }
    if (phase == 2) {
        if (!dY || !R || !dT) return SLOPE_ERR_INVALID_ARG;
        if (!aligned16(dY) || !aligned16(R) || !aligned16(dT)) return SLOPE_ERR_ALIGNMENT;
        if (slope_status_t st = check_arch(info)) return st;
        return launch_adapter_dT(dY, R, b, d_out, r, dT, stream, info);
    }
    if (!X || !dY || !R || !T || !dT || !dL || !dR || !workspace) return SLOPE_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(dY) || !aligned16(R) || !aligned16(T) || !aligned16(dT) || !aligned16(dL) ||
        !aligned16(dR) || !aligned16(workspace))
        return SLOPE_ERR_ALIGNMENT;
    if (workspace_bytes < slope_adapter_workspace_bytes(b, d_out, d_in, r)) return SLOPE_ERR_INVALID_ARG;
    if (slope_status_t st = check_arch(info)) return st;
    if (slope_status_t st = launch_adapter_dT(dY, R, b, d_out, r, dT, stream, info)) return st;
    return launch_adapter_grads(X, dY, T, dT, b, d_out, d_in, r, dL, dR, workspace, stream, info);
}

// ------------------------------------------------------------------ masked dW with dL, dR riding along
namespace slope {
constexpr int kCarrySplits = 8;            // partial sums per row block of dR^T / dL in the fused launch

struct DwAdapterPlan {
    bool fused;
    int splits_r, splits_l;
};

// The fused launch serves the shapes of the CTA-pair 256 x 256 weight-gradient kernel with r <= 128,
// provided no tile that carries adapter work lies among the halved items of the last wave (those run
// at half width, too narrow to serve as the A operand of the dL product).  Everything else takes the
// separate launches.
static DwAdapterPlan dw_adapter_plan(int b, int d_out, int d_in, int r, int sm_count) {
    DwAdapterPlan plan{false, 1, 1};
    const int num_m = (d_out + 255) / 256, num_n = (d_in + 255) / 256, num_kb = (b + 63) / 64;
    if (r > 128 || num_m * num_n * 2 <= sm_count) return plan;
    plan.splits_r = num_n < kCarrySplits ? num_n : kCarrySplits;
    plan.splits_l = num_m < kCarrySplits ? num_m : kCarrySplits;
    if (plan.splits_r > num_kb) plan.splits_r = num_kb;
    if (plan.splits_l > num_kb) plan.splits_l = num_kb;
    const int num_pairs = sm_count / 2, num_tiles = num_m * num_n;
    const int full = (num_tiles / num_pairs) * num_pairs, rem = num_tiles - full;
    if (rem > 0 && 2 * rem <= num_pairs) {
        for (int tile = full; tile < num_tiles; ++tile) {            // the raster order of raster_tile()
            const int group_size = kRasterGroupM * num_n, g = tile / group_size, first_m = g * kRasterGroupM;
            const int gm = num_m - first_m < kRasterGroupM ? num_m - first_m : kRasterGroupM;
            const int local = tile - g * group_size;
            const int m = first_m + local % gm, n = local / gm;
            if (m < plan.splits_l || n < plan.splits_r) return plan;
        }
    }
    plan.fused = true;
    return plan;
}

static size_t align256(size_t x) { return (x + 255) & ~size_t(255); }
}  // namespace slope

size_t slope_bwd_dw_adapter_workspace_bytes(int b, int d_out, int d_in, int r) {
    if (b <= 0 || d_out <= 0 || d_in <= 0 || r <= 0) return 0;
    const DwAdapterPlan plan = dw_adapter_plan(b, d_out, d_in, r, 148);
    const size_t fused = align256(static_cast<size_t>(plan.splits_r) * d_out * r * sizeof(float)) +
                         align256(static_cast<size_t>(plan.splits_l) * d_in * r * sizeof(float));
    const size_t separate = slope_adapter_workspace_bytes(b, d_out, d_in, r);
    return fused > separate ? fused : separate;
}

slope_status_t slope_linear_bwd_dw_adapter(const void* dY, const void* X, const void* T, const void* dT, int b,
                                           int d_out, int d_in, int r, const void* mask1_bits, void* dWc_vals,
                                           void* dL, void* dR, void* workspace, size_t workspace_bytes,
                                           void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!dY || !X || !T || !dT || !mask1_bits || !dWc_vals || !dL || !dR || !workspace) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in) || b < 1 || !rank_ok(r) || r == 0) return SLOPE_ERR_SHAPE;
    if (!aligned16(dY) || !aligned16(X) || !aligned16(T) || !aligned16(dT) || !aligned16(mask1_bits) ||
        !aligned16(dWc_vals) || !aligned16(dL) || !aligned16(dR) || !aligned16(workspace))
        return SLOPE_ERR_ALIGNMENT;
    if (workspace_bytes < slope_bwd_dw_adapter_workspace_bytes(b, d_out, d_in, r)) return SLOPE_ERR_INVALID_ARG;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    const DwAdapterPlan plan = dw_adapter_plan(b, d_out, d_in, r, info.sm_count);
    if (!plan.fused || info.sm_count != 148) {
        // the separate launches: masked dW, then the dL / dR partial products and their reduction
        if (slope_status_t st = slope_linear_bwd_dw_masked(dY, X, b, d_out, d_in, mask1_bits, dWc_vals, stream_)) return st;
        return launch_adapter_grads(X, dY, T, dT, b, d_out, d_in, r, dL, dR, workspace, stream, info);
    }
    using Cfg = DwAdapterCfg<6>;
    CUtensorMap tmA, tmB, tmT, tmDT;
    if (!make_tmap(&tmA, dY, b, d_out, 64, 64) || !make_tmap(&tmB, X, b, d_in, 64, 64) ||
        !make_tmap(&tmT, T, b, r, 64, 64) || !make_tmap(&tmDT, dT, b, r, 64, 64))
        return SLOPE_ERR_CUDA;
    DwAdapterParams p = {};
    p.M = d_out; p.N = d_in; p.K = b; p.r = r;
    p.splits_r = plan.splits_r; p.splits_l = plan.splits_l;
    p.dWc = static_cast<uint16_t*>(dWc_vals);
    p.mask = static_cast<const uint8_t*>(mask1_bits);
    p.ws_r = static_cast<float*>(workspace);
    p.ws_l = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) +
                                      align256(static_cast<size_t>(plan.splits_r) * d_out * r * sizeof(float)));
    auto kern = dw_adapter_pair_kernel<6>;
    if (!set_smem(kern, Cfg::kSmemBytes)) return SLOPE_ERR_CUDA;
    const int tiles = ((d_out + 255) / 256) * ((d_in + 255) / 256);
    const int max_pairs = info.sm_count / 2;
    const int pairs = tiles < max_pairs ? tiles : max_pairs;
    if (slope_status_t st = launch_pairs(kern, 2 * pairs, Cfg::kThreads, Cfg::kSmemBytes, stream, tmA, tmB, tmT, tmDT, p))
        return st;
    const SplitKReduce rl{p.ws_l, static_cast<uint16_t*>(dL), d_in, r, plan.splits_l, 0};
    const SplitKReduce rr{p.ws_r, static_cast<uint16_t*>(dR), d_out, r, plan.splits_r, 1};
    splitk_reduce_kernel<<<info.sm_count * 4, 256, 0, stream>>>(rl, rr);
    return launch_result();
}

slope_status_t slope_sparse_add(const void* A_vals, const void* B_vals, float beta, float gamma, int rows, int cols,
                                void* out_vals, void* stream) {
    if (!A_vals || !B_vals || !out_vals) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(rows, cols)) return SLOPE_ERR_SHAPE;
    if (!aligned16(A_vals) || !aligned16(B_vals) || !aligned16(out_vals)) return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    const size_t n_vec = static_cast<size_t>(rows) * cols / 2 / 8;
    sparse_add_kernel<<<info.sm_count * kStreamBlocksPerSm, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(A_vals), static_cast<const uint4*>(B_vals), beta, gamma, n_vec,
        static_cast<uint4*>(out_vals));
    return launch_result();
}

slope_status_t slope_update_sparse_matrix(const void* Wc_vals, const void* mask1_bits, const void* WTc_meta,
                                          int d_out, int d_in, void* WTc_vals, void* stream) {
    if (!Wc_vals || !mask1_bits || !WTc_meta || !WTc_vals) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in)) return SLOPE_ERR_SHAPE;
    // the kernel indexes its 8-byte and 16-byte units with 32 bits
    if (static_cast<unsigned long long>(d_out) * static_cast<unsigned long long>(d_in) >= (1ull << 35)) return SLOPE_ERR_SHAPE;
    if (!aligned16(Wc_vals) || !aligned16(mask1_bits) || !aligned16(WTc_meta) || !aligned16(WTc_vals))
        return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    const int tiles = (d_in / 128) * (d_out / 128), slots = info.sm_count * kUpdateBlocksPerSm;
    update_transposed_kernel<<<tiles < slots ? tiles : slots, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint2*>(Wc_vals), static_cast<const uint8_t*>(mask1_bits),
        static_cast<const uint4*>(WTc_meta), d_out, d_in, static_cast<uint4*>(WTc_vals));
    return launch_result();
}

// ------------------------------------------------------------------ general N:M (masked dense)
static bool nm_ok(int n, int m) { return (m == 2 || m == 4 || m == 8 || m == 16) && n > 0 && n < m; }

slope_status_t slope_prune_nm(const void* W, int d_out, int d_in, int n, int m, void* W_R, void* mask1_bits,
                              void* stream_) {
    if (!W || !W_R) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in) || !nm_ok(n, m)) return SLOPE_ERR_SHAPE;
    if (!aligned16(W) || !aligned16(W_R) || !aligned16(mask1_bits)) return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const size_t chunks = static_cast<size_t>(d_out) * d_in / 16;
    const int grid = info.sm_count * kStreamBlocksPerSm;
    const uint4* in = static_cast<const uint4*>(W);
    uint4* out = static_cast<uint4*>(W_R);
    uint16_t* mask = static_cast<uint16_t*>(mask1_bits);
    switch (m) {
        case 2: prune_nm_kernel<2><<<grid, 256, 0, stream>>>(in, chunks, n, out, mask); break;
        case 4: prune_nm_kernel<4><<<grid, 256, 0, stream>>>(in, chunks, n, out, mask); break;
        case 8: prune_nm_kernel<8><<<grid, 256, 0, stream>>>(in, chunks, n, out, mask); break;
        default: prune_nm_kernel<16><<<grid, 256, 0, stream>>>(in, chunks, n, out, mask); break;
    }
    return launch_result();
}

slope_status_t slope_double_prune_nm(const void* W, const void* mask1_bits, int d_out, int d_in, int n, int m,
                                     void* W_RC, void* mask2_bits, void* stream_) {
    if (!W || !mask1_bits || !W_RC) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in) || !nm_ok(n, m)) return SLOPE_ERR_SHAPE;
    if (!aligned16(W) || !aligned16(W_RC) || !aligned16(mask1_bits) || !aligned16(mask2_bits))
        return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int grid = info.sm_count * kStreamBlocksPerSm;
    const uint4* in = static_cast<const uint4*>(W);
    const uint8_t* m1 = static_cast<const uint8_t*>(mask1_bits);
    uint4* out = static_cast<uint4*>(W_RC);
    uint8_t* m2 = static_cast<uint8_t*>(mask2_bits);
    switch (m) {
        case 2: double_prune_nm_kernel<2><<<grid, 256, 0, stream>>>(in, m1, d_out, d_in, n, out, m2); break;
        case 4: double_prune_nm_kernel<4><<<grid, 256, 0, stream>>>(in, m1, d_out, d_in, n, out, m2); break;
        case 8: double_prune_nm_kernel<8><<<grid, 256, 0, stream>>>(in, m1, d_out, d_in, n, out, m2); break;
        default: double_prune_nm_kernel<16><<<grid, 256, 0, stream>>>(in, m1, d_out, d_in, n, out, m2); break;
    }
    return launch_result();
}

slope_status_t slope_apply_mask(const void* G, const void* mask_bits, int d_out, int d_in, void* out, void* stream) {
    if (!G || !mask_bits || !out) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(d_out, d_in)) return SLOPE_ERR_SHAPE;
    if (!aligned16(G) || !aligned16(mask_bits) || !aligned16(out)) return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    apply_mask_kernel<<<info.sm_count * kStreamBlocksPerSm, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(G), static_cast<const uint16_t*>(mask_bits),
        static_cast<size_t>(d_out) * d_in / 16, static_cast<uint4*>(out));
    return launch_result();
}

slope_status_t slope_mask_difference(const void* mask_a, const void* mask_b, int rows, int cols, void* count_out,
                                     void* stream_) {
    if (!mask_a || !mask_b || !count_out) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(rows, cols)) return SLOPE_ERR_SHAPE;
    if (!aligned16(mask_a) || !aligned16(mask_b) || (reinterpret_cast<uintptr_t>(count_out) & 7u) != 0)
        return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (cudaMemsetAsync(count_out, 0, sizeof(unsigned long long), stream) != cudaSuccess) return SLOPE_ERR_CUDA;
    const size_t n_vec = static_cast<size_t>(rows) * cols / 8 / 16;
    mask_difference_kernel<<<info.sm_count * kStreamBlocksPerSm, 256, 0, stream>>>(
        static_cast<const uint4*>(mask_a), static_cast<const uint4*>(mask_b), n_vec,
        static_cast<unsigned long long*>(count_out));
    return launch_result();
}

slope_status_t slope_selftest_wait_timeout(unsigned int limit_us, void* gave_up_flag, void* stream) {
    if (!gave_up_flag || limit_us == 0 || limit_us > 100000) return SLOPE_ERR_INVALID_ARG;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    wait_timeout_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<unsigned long long>(limit_us) * 1000ull, static_cast<int*>(gave_up_flag));
    return launch_result();
}

slope_status_t slope_meta_to_canonical(const void* meta_hw, int rows, int cols, void* meta_canon, void* stream) {
    if (!meta_hw || !meta_canon) return SLOPE_ERR_INVALID_ARG;
    if (!dims_ok(rows, cols)) return SLOPE_ERR_SHAPE;
    if (!aligned16(meta_hw) || !aligned16(meta_canon)) return SLOPE_ERR_ALIGNMENT;
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    meta_to_canonical_kernel<<<info.sm_count * 4, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint16_t*>(meta_hw), rows, cols, static_cast<uint16_t*>(meta_canon));
    return launch_result();
}

}  // extern "C"

// ------------------------------------------------------------------ allocation-free adapter-gradient entry
// Some callers may not allocate device memory at all: a plug-in running inside a host
// application whose memory pool is closed to it, or code that runs where cudaMalloc is
// forbidden (a latency-critical section, a process that has handed its whole GPU memory
// budget to a framework allocator).  For them the split-K scratch of the dL gradient lives
// in this fixed array instead of a caller workspace.  The array belongs to the loaded
// library image: every GPU that loads the library keeps these 16 MiB until the process
// exits, and every call on a device shares it.
namespace slope {
constexpr size_t kStaticScratchBytes = size_t(16) << 20;
static __device__ __align__(256) float g_static_scratch[kStaticScratchBytes / sizeof(float)];

// In host code `g_static_scratch` is only a handle; the address kernels can use comes from
// cudaGetSymbolAddress, asked once per device with that device current.
static slope_status_t static_scratch_address(float** out) {
    static std::mutex mu;
    static float* cache[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SLOPE_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (cache[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return SLOPE_ERR_CUDA;
        cache[dev] = static_cast<float*>(p);
    }
    *out = cache[dev];
    return SLOPE_OK;
}
}  // namespace slope

extern "C" {

size_t slope_adapter_dl_noalloc_max_scratch_bytes(void) { return kStaticScratchBytes; }

slope_status_t slope_adapter_dl_noalloc(const void* X, const void* dT, int b, int d_in, int r, void* dL,
                                        void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!X || !dT || !dL) return SLOPE_ERR_INVALID_ARG;
    if (d_in <= 0 || d_in % 128 != 0 || b < 1 || !rank_ok(r) || r == 0) return SLOPE_ERR_SHAPE;
    if (!aligned16(X) || !aligned16(dT) || !aligned16(dL)) return SLOPE_ERR_ALIGNMENT;
    const int splits = adapter_splits(b, d_in);
    const size_t need = static_cast<size_t>(splits) * d_in * r * sizeof(float);
    if (need > kStaticScratchBytes) return SLOPE_ERR_SHAPE;      // beyond the fixed scratch: use the workspace call
    DeviceInfo info;
    if (slope_status_t st = check_arch(info)) return st;
    float* scratch = nullptr;
    if (slope_status_t st = static_scratch_address(&scratch)) return st;
    // Nothing has to start at zero: every partial sum the reduction reads is written by the
    // GEMM of this same call, so what an earlier call left in the array is never observed.
    slope_status_t st =
        r <= 64 ? launch_dense<true, true, 64, kEpiPartial, 6>(X, dT, d_in, r, b, splits, scratch, nullptr, stream, info)
                : launch_dense<true, true, 128, kEpiPartial, 6>(X, dT, d_in, r, b, splits, scratch, nullptr, stream, info);
    if (st) return st;
    const SplitKReduce red{scratch, static_cast<uint16_t*>(dL), d_in, r, splits, 0};
    splitk_reduce_kernel<<<info.sm_count * 4, 256, 0, stream>>>(red, SplitKReduce{nullptr, nullptr, 0, 0, 0, 0});
    return launch_result();
}

}  // extern "C"
