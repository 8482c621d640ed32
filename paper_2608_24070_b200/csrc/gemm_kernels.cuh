// tcgen05 GEMM kernels for sm_100a.
//
// All kernels are persistent and warp-specialised: warp 0 feeds shared memory with TMA,
// warp 1 owns tensor memory and issues the MMAs (one elected thread), the remaining warps
// drain the fp32 accumulators from tensor memory, convert to bf16 and store.  Every mbarrier
// wait is bounded (ptx.cuh); a role that gives up sets a CTA-wide flag, all roles leave their
// loops, tensor memory is released and the kernel returns.
//
//   dense_gemm_kernel          1 CTA per 128 x N tile; the skinny adapter GEMMs and small dW
//   dense_gemm_pair_kernel     CTA pair per 256 x 256 tile (cta_group::2), the last wave's tiles
//                              halved; dW (masked epilogue) and the dense layer (store epilogue)
//   sparse_gemm_pair_kernel    CTA pair per 256 x 224 (or 256 x 128) tile, tcgen05.mma.sp;
//                              forward / dX with short reductions or few tiles
//   sparse_gemm_quad_kernel    CTA pair per 512 x 224 tile (two MMA sub-tiles per activation
//                              tile); forward / dX with long reductions
//   sparse_gemm_skinny_kernel  one CTA per 128-row weight slab and K-slice, cluster reduction
//                              through distributed shared memory; forward / dX with few
//                              tokens (inference, decode) and the adapter products at such
//                              sizes, not persistent
#pragma once
#include "ptx.cuh"

namespace slope {

constexpr int kGemmThreads = 192;
constexpr int kBlockM = 128;

struct PipeState {
    int stage = 0;
    uint32_t phase = 0;
    __device__ __forceinline__ void advance(int nstages) {
        if (++stage == nstages) { stage = 0; phase ^= 1u; }
    }
};

// Give in-flight bulk copies time to land before the CTA's shared memory goes away.
__device__ __forceinline__ void drain_after_abort() {
    const unsigned long long t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
}

// =====================================================================================
// Sparse GEMM:  O[Ntok x M] (bf16) = ( A_2:4[M x K] * B[Ntok x K]^T  (+ A2[M x r] * B2[Ntok x r]^T) )^T
//   A   compressed values [M x K/2] + tensor-core-order metadata   (sparse operand)
//   B   activations, K contiguous
//   A2  dense adapter factor on the weight side: either [M x r] (K contiguous) or [r x M]
//   B2  dense adapter activations [Ntok x r]
// Used for Eq. (sparse_forward) (M = d_out, K = d_in) and Eq. (sparse_backward_input)
// (M = d_in, K = d_out, A = double-pruned transposed copy); the adapter product of
// Eq. (concat) is accumulated into the same tensor-memory tile by extra dense MMAs.
// Only the A operand of tcgen05.mma.sp can be sparse, hence the accumulator holds the
// transposed output tile (lane = feature, column = token) and the epilogue transposes.
// =====================================================================================
struct SparseGemmParams {
    int M, K, Ntok, r;
    int a2_mn_major;              // 1: A2 is stored [r x M] (M contiguous)
    int group_m;                  // 512-row-tile kernel: row tiles per raster group (0: all in one group)
    int pdl_mode;                 // few-token kernel: 0 plain, 1 producer / 2 consumer of a fused pair of launches
    const uint8_t* meta;          // metadata blocks of A
    uint16_t* out;                // [Ntok x M]
};

// =====================================================================================
// Dense GEMM:  D[M x N] = A[M x K] * B[N x K]^T, bf16 in, fp32 accumulate.
//   A_MN / B_MN: the operand is stored with its M (resp. N) index contiguous, i.e. as
//   [K x M] (resp. [K x N]) row-major; otherwise K is contiguous.
// Epilogues:
//   kEpiStore    bf16 D, row-major, leading dimension N
//   kEpiMasked   Eq. (sparse_backward_weight) + Algorithm 1 "pruneAndCompress": keep, per
//                group of 4 columns, the two columns the first-pass mask selects; bf16
//                [M x N/2]
//   kEpiPartial  fp32 partial sums of one K-split into workspace[split][M][N]
// =====================================================================================
constexpr int kEpiStore = 0, kEpiMasked = 1, kEpiPartial = 2;

struct DenseGemmParams {
    int M, N, K;
    int k_splits;
    void* out;
    const uint8_t* mask;          // kEpiMasked: [M x N/8]
    int pdl_mode;                 // 1: producer of a fused pair of launches (wait first, release dependents afterwards)
};

template <int BLOCK_N, int STAGES>
struct DenseCfg {
    static constexpr int kABytes = kBlockM * 128;                // 128 x 64 bf16
    static constexpr int kBBytes = BLOCK_N * 128;                // BLOCK_N x 64 bf16
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kSmemBytes = STAGES * kStageBytes + 256 + 1024;
    static constexpr int kTmemCols = 2 * BLOCK_N <= 32 ? 32 : (2 * BLOCK_N <= 64 ? 64 : (2 * BLOCK_N <= 128 ? 128 : (2 * BLOCK_N <= 256 ? 256 : 512)));
    static_assert(BLOCK_N % 64 == 0 && BLOCK_N <= 256, "BLOCK_N must be 64, 128, 192 or 256");
};

template <bool A_MN, bool B_MN, int BLOCK_N, int EPI, int STAGES>
__global__ void __launch_bounds__(kGemmThreads, 1)
dense_gemm_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
                  const DenseGemmParams p0, const __grid_constant__ CUtensorMap tmA1,
                  const __grid_constant__ CUtensorMap tmB1, const DenseGemmParams p1) {
    // Up to two independent problems of the same kind share one launch (p1.M == 0: only one):
    // tiles [0, tiles0) belong to problem 0, the rest to problem 1.
    using Cfg = DenseCfg<BLOCK_N, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + STAGES * Cfg::kStageBytes);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* tfull_bar = empty_bar + STAGES;
    uint64_t* tempty_bar = tfull_bar + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    auto tiles_of = [](const DenseGemmParams& q) {
        return q.M == 0 ? 0 : ((q.M + kBlockM - 1) / kBlockM) * ((q.N + BLOCK_N - 1) / BLOCK_N) * q.k_splits;
    };
    const int tiles0 = tiles_of(p0);
    const int num_tiles = tiles0 + tiles_of(p1);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&tfull_bar[a], 1); mbar_init(&tempty_bar[a], 128); }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, Cfg::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Programmatic dependent launch: the set-up above may overlap the tail of the previous kernel in
    // the stream; no thread touches global memory before that kernel has completed.
    if (p0.pdl_mode == 1) {              // see the few-token kernel: the dependent may rely on all earlier work
        griddep_wait();
        griddep_launch_dependents();
    } else {
        griddep_launch_dependents();
        griddep_wait();
    }

    // tile -> (problem, m block, n block, split): m fastest so that concurrently running CTAs share B
    auto decode = [&](int tile, int& m_blk, int& n_blk, int& kb0, int& kb1) {
        const bool second = tile >= tiles0;
        const DenseGemmParams& q = second ? p1 : p0;
        if (second) tile -= tiles0;
        const int num_m = (q.M + kBlockM - 1) / kBlockM;
        const int num_n = (q.N + BLOCK_N - 1) / BLOCK_N;
        const int num_kb_total = (q.K + 63) / 64;
        const int kb_per_split = (num_kb_total + q.k_splits - 1) / q.k_splits;
        m_blk = tile % num_m;
        const int rest = tile / num_m;
        n_blk = rest % num_n;
        const int split = rest / num_n;
        kb0 = split * kb_per_split;
        kb1 = min(num_kb_total, kb0 + kb_per_split);
        return split | (second ? 0x10000 : 0);
    };

    if (warp == 0) {
        if (elect_one()) {
            tma_prefetch_desc(&tmA0);
            tma_prefetch_desc(&tmB0);
            PipeState ps;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                int m_blk, n_blk, kb0, kb1;
                const bool second = (decode(tile, m_blk, n_blk, kb0, kb1) & 0x10000) != 0;
                const CUtensorMap* tmA = second ? &tmA1 : &tmA0;
                const CUtensorMap* tmB = second ? &tmB1 : &tmB0;
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!mbar_wait(&empty_bar[ps.stage], ps.phase ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t* sA = smem + ps.stage * Cfg::kStageBytes;
                    uint8_t* sB = sA + Cfg::kABytes;
                    uint64_t* bar = &full_bar[ps.stage];
                    mbar_expect_tx(bar, Cfg::kStageBytes);
                    if (A_MN) {
                        tma_load_2d(sA, tmA, bar, m_blk * kBlockM, kb * 64);
                        tma_load_2d(sA + 8192, tmA, bar, m_blk * kBlockM + 64, kb * 64);
                    } else {
                        tma_load_2d(sA, tmA, bar, kb * 64, m_blk * kBlockM);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int h = 0; h < BLOCK_N / 64; ++h)
                            tma_load_2d(sB + h * 8192, tmB, bar, n_blk * BLOCK_N + h * 64, kb * 64);
                    } else {
                        tma_load_2d(sB, tmB, bar, kb * 64, n_blk * BLOCK_N);
                    }
                    ps.advance(STAGES);
                }
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            constexpr uint32_t idesc = make_idesc_bf16(kBlockM, BLOCK_N, A_MN, B_MN, false);
            PipeState ps;
            bool ok = true;
            int it = 0;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++it) {
                int m_blk, n_blk, kb0, kb1;
                decode(tile, m_blk, n_blk, kb0, kb1);
                const int acc = it & 1;
                const uint32_t acc_phase = static_cast<uint32_t>(it >> 1) & 1u;
                if (!mbar_wait(&tempty_bar[acc], acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * BLOCK_N;
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!mbar_wait(&full_bar[ps.stage], ps.phase, abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t sA = smem_u32(smem + ps.stage * Cfg::kStageBytes);
                    const uint32_t sB = sA + Cfg::kABytes;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint64_t ad = A_MN ? make_smem_desc(sA + j * 2048, 8192, 1024, kSwizzle128B)
                                                 : make_smem_desc(sA + j * 32, 16, 1024, kSwizzle128B);
                        const uint64_t bd = B_MN ? make_smem_desc(sB + j * 2048, 8192, 1024, kSwizzle128B)
                                                 : make_smem_desc(sB + j * 32, 16, 1024, kSwizzle128B);
                        umma_bf16(d_tmem, ad, bd, idesc, (kb > kb0 || j > 0) ? 1u : 0u);
                    }
                    umma_commit(&empty_bar[ps.stage]);
                    ps.advance(STAGES);
                }
                if (ok) umma_commit(&tfull_bar[acc]);
            }
        }
    } else {
        const int q = warp & 3;
        bool ok = true;
        int it = 0;
        for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++it) {
            int m_blk, n_blk, kb0, kb1;
            const int code = decode(tile, m_blk, n_blk, kb0, kb1);
            const int split = code & 0xFFFF;
            const DenseGemmParams& p = (code & 0x10000) ? p1 : p0;
            const int acc = it & 1;
            const uint32_t acc_phase = static_cast<uint32_t>(it >> 1) & 1u;
            if (!mbar_wait(&tfull_bar[acc], acc_phase, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + acc * BLOCK_N + (static_cast<uint32_t>(q * 32) << 16);
            const int m = m_blk * kBlockM + q * 32 + lane;
#pragma unroll 1
            for (int c0 = 0; c0 < BLOCK_N; c0 += 16) {
                uint32_t v[16];
                tmem_ld_16(t_row + c0, v);
                tmem_ld_wait();
                const int n0 = n_blk * BLOCK_N + c0;
                if (m >= p.M || n0 >= p.N) continue;
                if (EPI == kEpiStore) {
                    uint4* dst = reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.out) + static_cast<size_t>(m) * p.N + n0);
                    uint32_t w[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) w[c] = pack_bf16x2(__uint_as_float(v[2 * c]), __uint_as_float(v[2 * c + 1]));
                    dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                    dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
                } else if (EPI == kEpiMasked) {
                    const uint32_t mbits =
                        *reinterpret_cast<const uint16_t*>(p.mask + static_cast<size_t>(m) * (p.N >> 3) + (n0 >> 3));
                    uint32_t w[4];
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const uint32_t mb = (mbits >> (4 * g)) & 0xFu;
                        // kept positions in ascending order: lowest set bit, highest set bit
                        const int p0 = __ffs(mb) - 1, p1 = 31 - __clz(mb);
                        const float e0 = __uint_as_float(v[4 * g]), e1 = __uint_as_float(v[4 * g + 1]),
                                    e2 = __uint_as_float(v[4 * g + 2]), e3 = __uint_as_float(v[4 * g + 3]);
                        const float lo = p0 == 0 ? e0 : (p0 == 1 ? e1 : e2);
                        const float hi = p1 == 1 ? e1 : (p1 == 2 ? e2 : e3);
                        w[g] = pack_bf16x2(lo, hi);
                    }
                    *reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.out) + static_cast<size_t>(m) * (p.N >> 1) + (n0 >> 1)) =
                        make_uint4(w[0], w[1], w[2], w[3]);
                } else {
                    float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.out) +
                                                            (static_cast<size_t>(split) * p.M + m) * p.N + n0);
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        dst[c] = make_float4(__uint_as_float(v[4 * c]), __uint_as_float(v[4 * c + 1]),
                                             __uint_as_float(v[4 * c + 2]), __uint_as_float(v[4 * c + 3]));
                }
            }
            tc_fence_before_sync();
            mbar_arrive(&tempty_bar[acc]);
        }
    }

    __syncwarp();
    if (*abort_flag) drain_after_abort();
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
}

// Fixed-order reduction of K-split partial sums: out = bf16( sum_s ws[s][m][n] ), written
// row-major [M x N] or transposed [N x M].  Up to two reductions per launch (second.M == 0: one).
struct SplitKReduce {
    const float* ws;
    uint16_t* out;
    int M, N, splits, transpose;
};

// A block takes 32 consecutive rows at a time: 16-byte loads of the partial sums, summed in split
// order; the transposed output goes through a padded shared-memory tile so that both the reads
// and the 2-byte writes are contiguous.  N (the adapter rank) is a multiple of 16, at most 256.
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const SplitKReduce r0, const SplitKReduce r1) {
    __shared__ float tile[32][257];
    const int units0 = (r0.M + 31) / 32, units1 = (r1.M + 31) / 32;
    for (int u = blockIdx.x; u < units0 + units1; u += gridDim.x) {
        const bool second = u >= units0;
        const SplitKReduce& r = second ? r1 : r0;
        const int m0 = 32 * (second ? u - units0 : u);
        const int rows = min(32, r.M - m0);
        const size_t total = static_cast<size_t>(r.M) * r.N;
        const float4* ws4 = reinterpret_cast<const float4*>(r.ws + static_cast<size_t>(m0) * r.N);
        const size_t split_stride4 = total / 4;
        const int chunks = rows * r.N / 4;
        for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
            float4 acc = ws4[c];
            for (int s = 1; s < r.splits; ++s) {
                const float4 t = ws4[static_cast<size_t>(s) * split_stride4 + c];
                acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
            }
            if (r.transpose) {
                const int mm = (4 * c) / r.N, n = (4 * c) % r.N;
                tile[mm][n] = acc.x; tile[mm][n + 1] = acc.y; tile[mm][n + 2] = acc.z; tile[mm][n + 3] = acc.w;
            } else {
                uint2 o;
                o.x = pack_bf16x2(acc.x, acc.y);
                o.y = pack_bf16x2(acc.z, acc.w);
                *reinterpret_cast<uint2*>(r.out + static_cast<size_t>(m0) * r.N + 4 * static_cast<size_t>(c)) = o;
            }
        }
        if (r.transpose) {
            __syncthreads();
            for (int e = threadIdx.x; e < 32 * r.N; e += blockDim.x) {
                const int n = e >> 5, mm = e & 31;
                if (mm < rows) r.out[static_cast<size_t>(n) * r.M + m0 + mm] = to_bf16(tile[mm][n]);
            }
            __syncthreads();
        }
    }
}

// =====================================================================================
// CTA-pair versions (cluster of 2, tcgen05 cta_group::2).  One MMA spans both SMs: the pair
// owns a 256-row tile of the A operand (128 rows per CTA) and each CTA stages only HALF of
// the B tile, which halves the activation bytes every SM pulls from L2 per MMA and leaves
// room for twice as many pipeline stages.  The leader CTA (rank 0) issues all MMAs; both
// CTAs run their own TMA producer (completion bytes are counted on the leader's barrier)
// and their own epilogue (each drains its 128 accumulator rows).  tcgen05.commit arrives on
// the barriers of both CTAs; the epilogues release an accumulator stage by arriving on the
// leader's barrier through the cluster shared-memory window.
// =====================================================================================
// Token tiles are BLOCK_N wide except the last one of a ragged token count, which is only as wide
// as the tokens that are left (rounded up to the 32-token block of the epilogue): the MMAs run
// with that N, the second CTA's half of the activations starts at its middle, and the epilogue
// stops there.  A 2048-token forward on 224-token tiles ends in a 32-token tile that costs a
// fraction of a full one instead of a whole wave of the machine.
__device__ __forceinline__ int token_tile_width(int ntok, int n0, int block_n) {
    const int left = ntok - n0;
    return left >= block_n ? block_n : ((left + 31) & ~31);
}

template <int BLOCK_N, int STAGES>
struct SparsePairCfg {
    static constexpr int kHalfN = BLOCK_N / 2;
    static constexpr int kABytes = kBlockM * 128;
    static constexpr int kBBytes = kHalfN * 256;
    static constexpr int kEBytes = 2048;
    static constexpr int kStageBytes = kABytes + kBBytes + kEBytes;
    static constexpr int kStoreRows = 32;                         // tokens per TMA store
    static constexpr int kStoreCols = 32;                         // features per TMA store (one warp's lanes)
    static constexpr int kStoreBytes = kStoreRows * kStoreCols * 2;
    static constexpr int kEpiWarps = 8;                           // two warps per tensor-memory lane quadrant
    static constexpr int kThreads = 64 + 32 * kEpiWarps;
    static constexpr int kOffStore = STAGES * kStageBytes;
    static constexpr int kOffBar = kOffStore + kEpiWarps * 2 * kStoreBytes;
    static constexpr int kSmemBytes = kOffBar + 256 + 1024;
    static constexpr int kECol = 2 * BLOCK_N;
    static_assert(BLOCK_N % 32 == 0 && kHalfN % 8 == 0 && 2 * BLOCK_N + 8 <= 512, "tile does not fit tensor memory");
    static_assert(kStageBytes % 1024 == 0, "stage must keep 1024-byte alignment");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

template <int BLOCK_N, int STAGES>
__global__ void __launch_bounds__(SparsePairCfg<BLOCK_N, STAGES>::kThreads, 1)
sparse_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                        const __grid_constant__ CUtensorMap tmE, const __grid_constant__ CUtensorMap tmA2,
                        const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmO,
                        const SparseGemmParams p) {
    using Cfg = SparsePairCfg<BLOCK_N, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBar);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* tfull_bar = empty_bar + STAGES;
    uint64_t* tempty_bar = tfull_bar + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta = cluster_ctarank();                  // 0 = leader
    const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_mb = p.M / kBlockM;                        // 128-row blocks of A
    const int num_m = (num_mb + 1) / 2;                      // 256-row pair tiles
    const int num_n = (p.Ntok + BLOCK_N - 1) / BLOCK_N;
    const int num_tiles = num_m * num_n;
    const int num_kb = p.K / 128;
    const int num_ab = (p.r + 63) / 64;
    const int total_kb = num_kb + num_ab;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&tfull_bar[a], 1); mbar_init(&tempty_bar[a], 2 * Cfg::kEpiWarps); }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, 512);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                                      // peer barriers are initialised
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Programmatic dependent launch: the set-up above may overlap the tail of the previous kernel in
    // the stream; no thread touches global memory before that kernel has completed.
    // (As the consumer of a fused pair of launches -- pdl_mode 2, see the few-token kernel -- only the
    // producer thread waits, right before its first load of the adapter operand T.)
    griddep_launch_dependents();
    if (p.pdl_mode != 2) griddep_wait();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs)
        if (elect_one()) {
            tma_prefetch_desc(&tmA);
            tma_prefetch_desc(&tmB);
            tma_prefetch_desc(&tmE);
            const uint64_t keep = l2_policy_evict_last();
            PipeState ps;
            bool ok = true;
            bool waited = false;
            for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs) {
                const int m_pair = tile % num_m, n_blk = tile / num_m;
                const int mb = m_pair * 2 + static_cast<int>(cta);           // this CTA's 128-row block
                const int mb_e = mb < num_mb ? mb : num_mb - 1;              // rows past M: any valid metadata block
                const int width = token_tile_width(p.Ntok, n_blk * BLOCK_N, BLOCK_N);
                const int n_row0 = n_blk * BLOCK_N + static_cast<int>(cta) * (width / 2);
                for (int kb = 0; kb < total_kb; ++kb) {
                    if (!mbar_wait(&empty_bar[ps.stage], ps.phase ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t* sA = smem + ps.stage * Cfg::kStageBytes;
                    uint8_t* sB = sA + Cfg::kABytes;
                    uint8_t* sE = sB + Cfg::kBBytes;
                    const uint32_t bar = mapa_shared(smem_u32(&full_bar[ps.stage]), 0);
                    if (kb < num_kb) {
                        if (cta == 0) mbar_expect_tx(&full_bar[ps.stage], 2 * Cfg::kStageBytes);
                        tma_load_2d_pair_hint(sA, &tmA, bar, kb * 64, mb * kBlockM, keep);
                        tma_load_2d_pair(sB, &tmB, bar, kb * 128, n_row0);
                        tma_load_2d_pair(sB + Cfg::kHalfN * 128, &tmB, bar, kb * 128 + 64, n_row0);
                        tma_load_2d_pair_hint(sE, &tmE, bar, 0, mb_e * num_kb + kb, keep);
                    } else {
                        const int ab = kb - num_kb;
                        if (p.pdl_mode == 2 && !waited) {
                            griddep_wait();
                            waited = true;
                        }
                        if (cta == 0) mbar_expect_tx(&full_bar[ps.stage], 2 * (Cfg::kABytes + Cfg::kHalfN * 128));
                        if (p.a2_mn_major) {
                            tma_load_2d_pair(sA, &tmA2, bar, mb * kBlockM, ab * 64);
                            tma_load_2d_pair(sA + 8192, &tmA2, bar, mb * kBlockM + 64, ab * 64);
                        } else {
                            tma_load_2d_pair(sA, &tmA2, bar, ab * 64, mb * kBlockM);
                        }
                        tma_load_2d_pair(sB, &tmB2, bar, ab * 64, n_row0);
                    }
                    ps.advance(STAGES);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (cta == 0 && elect_one()) {
            PipeState ps;
            bool ok = true;
            int it = 0;
            ClockProbe probe;
            if (pair_id == 0) probe.begin();
            for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs, ++it) {
                const int width = token_tile_width(p.Ntok, (tile / num_m) * BLOCK_N, BLOCK_N);
                const uint32_t idesc_sp = make_idesc_bf16(2 * kBlockM, width, false, false, true);
                const uint32_t idesc_ad = make_idesc_bf16(2 * kBlockM, width, p.a2_mn_major != 0, false, false);
                const int acc = it & 1;
                const uint32_t acc_phase = static_cast<uint32_t>(it >> 1) & 1u;
                if (!mbar_wait(&tempty_bar[acc], acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * BLOCK_N;
                for (int kb = 0; kb < total_kb; ++kb) {
                    if (!mbar_wait(&full_bar[ps.stage], ps.phase, abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t sA = smem_u32(smem + ps.stage * Cfg::kStageBytes);
                    const uint32_t sB = sA + Cfg::kABytes;
                    const uint32_t sE = sB + Cfg::kBBytes;
                    if (kb < num_kb) {
                        const uint32_t e_tmem = tmem_base + Cfg::kECol + (kb & 1) * 4;
                        tmem_cp_128x128b_pair(e_tmem, make_smem_desc(sE, 128, 128, kSwizzleNone));
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint64_t ad = make_smem_desc(sA + j * 32, 16, 1024, kSwizzle128B);
                            const uint64_t bd = make_smem_desc(sB + (j >> 1) * (Cfg::kHalfN * 128) + (j & 1) * 64, 16,
                                                               1024, kSwizzle128B);
                            umma_bf16_sp_pair(d_tmem, ad, bd, e_tmem + (j & 2), idesc_sp | (j & 1),
                                              (kb | j) != 0 ? 1u : 0u);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint64_t ad = p.a2_mn_major
                                                    ? make_smem_desc(sA + j * 2048, 8192, 1024, kSwizzle128B)
                                                    : make_smem_desc(sA + j * 32, 16, 1024, kSwizzle128B);
                            const uint64_t bd = make_smem_desc(sB + j * 32, 16, 1024, kSwizzle128B);
                            umma_bf16_pair(d_tmem, ad, bd, idesc_ad, 1u);
                        }
                    }
                    umma_commit_pair(&empty_bar[ps.stage], 3);
                    ps.advance(STAGES);
                }
                if (ok) umma_commit_pair(&tfull_bar[acc], 3);
            }
            if (pair_id == 0) probe.end(kClockSparse);
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
        // Warp w drains lane quadrant w%4; the two warps of a quadrant take alternate 32-token
        // blocks.  A block (32 features x 32 tokens) is read from tensor memory as accumulator
        // fragments, packed to bf16 pairs of adjacent tokens, and written transposed into the
        // warp's private staging buffer by four stmatrix instructions ([token][32 features],
        // 16-byte pieces XOR-swizzled as the store's tensor map expects); it leaves as a TMA store
        // of 32 tokens x 32 features, so no warp waits for another.
        const int q = warp & 3;
        const int ew = warp - 2;
        const int half = ew >> 2;
        uint8_t* my_buf = smem + Cfg::kOffStore + ew * 2 * Cfg::kStoreBytes;
        const uint64_t stream_out = l2_policy_evict_first();
        bool ok = true;
        int it = 0;
        uint32_t buf = 0;
        for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs, ++it) {
            const int m_pair = tile % num_m, n_blk = tile / num_m;
            const int acc = it & 1;
            const uint32_t acc_phase = static_cast<uint32_t>(it >> 1) & 1u;
            if (!mbar_wait(&tfull_bar[acc], acc_phase, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + acc * BLOCK_N + (static_cast<uint32_t>(q * 32) << 16);
            const int m0 = (m_pair * 2 + static_cast<int>(cta)) * kBlockM + q * 32;
            const int width = token_tile_width(p.Ntok, n_blk * BLOCK_N, BLOCK_N);
#pragma unroll 1
            for (int c0 = half * Cfg::kStoreRows; c0 < width; c0 += 2 * Cfg::kStoreRows) {
                uint32_t v0[16], v1[16];                         // features 0..15 and 16..31 of the quadrant
                tmem_ld_16x256b_x4(t_row + c0, v0);
                tmem_ld_16x256b_x4(t_row + (16u << 16) + c0, v1);
                // the staging buffer about to be overwritten must have been read by its TMA store
                if (lane == 0) tma_store_wait_read<1>();
                __syncwarp();
                tmem_ld_wait();
                // lane -> (matrix = feature group of 8, row = token within a group of 8): 64-byte token
                // rows, 16-byte piece index XOR bits 7..8 of the address (the 64-byte swizzle)
                const uint32_t row_addr = smem_u32(my_buf + buf * Cfg::kStoreBytes) + (lane & 7) * 64 +
                                          (((lane >> 3) ^ ((lane >> 1) & 3)) << 4);
#pragma unroll
                for (int j = 0; j < 4; ++j) {                    // tokens 8j .. 8j + 7
                    stmatrix_x4_trans(row_addr + j * 512,
                                      pack_bf16x2(__uint_as_float(v0[4 * j]), __uint_as_float(v0[4 * j + 1])),
                                      pack_bf16x2(__uint_as_float(v0[4 * j + 2]), __uint_as_float(v0[4 * j + 3])),
                                      pack_bf16x2(__uint_as_float(v1[4 * j]), __uint_as_float(v1[4 * j + 1])),
                                      pack_bf16x2(__uint_as_float(v1[4 * j + 2]), __uint_as_float(v1[4 * j + 3])));
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0 && m0 < p.M) {
                    tma_store_2d_hint(&tmO, my_buf + buf * Cfg::kStoreBytes, m0, n_blk * BLOCK_N + c0, stream_out);
                    tma_store_commit();
                }
                buf ^= 1u;
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&tempty_bar[acc]), 0));
        }
        if (lane == 0) tma_store_wait_all<0>();
    }

    __syncwarp();
    if (*abort_flag) drain_after_abort();
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                                      // nobody signals or reads the peer after this
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, 512);
    }
}

// Tile order for GEMMs whose two operands are both streamed once per tile (dW: dY^T X with the
// tokens as reduction).  The ~74 tiles in flight should form a near-square patch of the output:
// a patch of gm x gn tiles reads (gm + gn) operand panels, a gm x 1 strip reads gm + 1 for 1/gn
// of the work.  Tiles are numbered in groups of kRasterGroupM tile rows, column by column.
constexpr int kRasterGroupM = 8;
__device__ __forceinline__ void raster_tile(int tile, int num_m, int num_n, int& m, int& n) {
    const int group_size = kRasterGroupM * num_n;
    const int g = tile / group_size;
    const int first_m = g * kRasterGroupM;
    const int gm = min(num_m - first_m, kRasterGroupM);
    const int local = tile - g * group_size;
    m = first_m + local % gm;
    n = local / gm;
}

// Work items of the persistent CTA-pair GEMM.  Items are tiles in raster order; when the tiles
// left over after the last full wave of the machine (num_tiles mod num_pairs) fill at most
// half of the pairs, each of them is cut into two half-width items, so that the last wave
// takes half the time instead of a full tile time on a half-empty machine (4096 x 4096 weight
// gradient: 256 tiles on 74 pairs = 3 waves + 34 tiles -> 68 half items: 3.5 instead of 4 waves).
struct PairWork {
    int m_pair, n0, width;
};
template <int BLOCK_N, bool SPLIT_TAIL>
__device__ __forceinline__ bool pair_work(int item, int num_pairs, int num_m, int num_n, PairWork& w) {
    const int num_tiles = num_m * num_n;
    const int full = (num_tiles / num_pairs) * num_pairs, rem = num_tiles - full;
    const bool split = SPLIT_TAIL && rem > 0 && 2 * rem <= num_pairs;
    if (item >= (split ? full + 2 * rem : num_tiles)) return false;
    const bool halved = split && item >= full;
    const int tile = halved ? full + ((item - full) >> 1) : item;
    int n_blk;
    raster_tile(tile, num_m, num_n, w.m_pair, n_blk);
    w.width = halved ? BLOCK_N / 2 : BLOCK_N;
    w.n0 = n_blk * BLOCK_N + (halved && ((item - full) & 1) ? BLOCK_N / 2 : 0);
    return true;
}

// Dense CTA-pair GEMM: D[M x N] = A[M x K] * B[N x K]^T with a 256 x BLOCK_N tile per pair
// (each CTA: 128 rows of A, BLOCK_N/2 rows of B, 128 x BLOCK_N accumulator rows).
template <int BLOCK_N, int STAGES>
struct DensePairCfg {
    static constexpr int kHalfN = BLOCK_N / 2;
    static constexpr int kABytes = kBlockM * 128;
    static constexpr int kBBytes = kHalfN * 128;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kSmemBytes = STAGES * kStageBytes + 256 + 1024;
    static_assert(BLOCK_N % 128 == 0 && BLOCK_N <= 256, "BLOCK_N must be 128 or 256");
};

template <bool A_MN, bool B_MN, int BLOCK_N, int EPI, int STAGES>
__global__ void __launch_bounds__(kGemmThreads, 1)
dense_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                       const DenseGemmParams p) {
    using Cfg = DensePairCfg<BLOCK_N, STAGES>;
    constexpr int kTmemCols = 2 * BLOCK_N;                       // 256 or 512
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + STAGES * Cfg::kStageBytes);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* tfull_bar = empty_bar + STAGES;
    uint64_t* tempty_bar = tfull_bar + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta = cluster_ctarank();
    const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_m = (p.M + 2 * kBlockM - 1) / (2 * kBlockM);
    const int num_n = (p.N + BLOCK_N - 1) / BLOCK_N;
    const int num_kb = (p.K + 63) / 64;
    // halving needs B loads of any width: the [K x N] operand is loaded in 64-column chunks
    constexpr bool kSplitTail = B_MN && BLOCK_N == 256;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&tfull_bar[a], 1); mbar_init(&tempty_bar[a], 8); }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Programmatic dependent launch: the set-up above may overlap the tail of the previous kernel in
    // the stream; no thread touches global memory before that kernel has completed.
    griddep_launch_dependents();
    griddep_wait();

    if (warp == 0) {
        if (elect_one()) {
            tma_prefetch_desc(&tmA);
            tma_prefetch_desc(&tmB);
            PipeState ps;
            bool ok = true;
            PairWork w;
            for (int item = pair_id; ok && pair_work<BLOCK_N, kSplitTail>(item, num_pairs, num_m, num_n, w);
                 item += num_pairs) {
                const int half_w = w.width / 2;                       // B rows (columns of D) this CTA stages
                const int m0 = (w.m_pair * 2 + static_cast<int>(cta)) * kBlockM;
                const int n0 = w.n0 + static_cast<int>(cta) * half_w;
                const uint32_t stage_tx = kSplitTail ? 2 * (Cfg::kABytes + half_w * 128) : 2 * Cfg::kStageBytes;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&empty_bar[ps.stage], ps.phase ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t* sA = smem + ps.stage * Cfg::kStageBytes;
                    uint8_t* sB = sA + Cfg::kABytes;
                    const uint32_t bar = mapa_shared(smem_u32(&full_bar[ps.stage]), 0);
                    if (cta == 0) mbar_expect_tx(&full_bar[ps.stage], stage_tx);
                    if (A_MN) {
                        tma_load_2d_pair(sA, &tmA, bar, m0, kb * 64);
                        tma_load_2d_pair(sA + 8192, &tmA, bar, m0 + 64, kb * 64);
                    } else {
                        tma_load_2d_pair(sA, &tmA, bar, kb * 64, m0);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int h = 0; h < Cfg::kHalfN / 64; ++h)
                            if (h * 64 < half_w) tma_load_2d_pair(sB + h * 8192, &tmB, bar, n0 + h * 64, kb * 64);
                    } else {
                        tma_load_2d_pair(sB, &tmB, bar, kb * 64, n0);
                    }
                    ps.advance(STAGES);
                }
            }
        }
    } else if (warp == 1) {
        if (cta == 0 && elect_one()) {
            constexpr uint32_t idesc_full = make_idesc_bf16(2 * kBlockM, BLOCK_N, A_MN, B_MN, false);
            constexpr uint32_t idesc_half = make_idesc_bf16(2 * kBlockM, BLOCK_N / 2, A_MN, B_MN, false);
            PipeState ps;
            bool ok = true;
            int it = 0;
            PairWork w;
            ClockProbe probe;
            if (pair_id == 0) probe.begin();
            for (int item = pair_id; ok && pair_work<BLOCK_N, kSplitTail>(item, num_pairs, num_m, num_n, w);
                 item += num_pairs, ++it) {
                const uint32_t idesc = w.width == BLOCK_N ? idesc_full : idesc_half;
                const int acc = it & 1;
                const uint32_t acc_phase = static_cast<uint32_t>(it >> 1) & 1u;
                if (!mbar_wait(&tempty_bar[acc], acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * BLOCK_N;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&full_bar[ps.stage], ps.phase, abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t sA = smem_u32(smem + ps.stage * Cfg::kStageBytes);
                    const uint32_t sB = sA + Cfg::kABytes;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint64_t ad = A_MN ? make_smem_desc(sA + j * 2048, 8192, 1024, kSwizzle128B)
                                                 : make_smem_desc(sA + j * 32, 16, 1024, kSwizzle128B);
                        const uint64_t bd = B_MN ? make_smem_desc(sB + j * 2048, 8192, 1024, kSwizzle128B)
                                                 : make_smem_desc(sB + j * 32, 16, 1024, kSwizzle128B);
                        umma_bf16_pair(d_tmem, ad, bd, idesc, (kb | j) != 0 ? 1u : 0u);
                    }
                    umma_commit_pair(&empty_bar[ps.stage], 3);
                    ps.advance(STAGES);
                }
                if (ok) umma_commit_pair(&tfull_bar[acc], 3);
            }
            if (pair_id == 0) probe.end(kClockDense);
        }
    } else {
        const int q = warp & 3;
        bool ok = true;
        int it = 0;
        PairWork w;
        for (int item = pair_id; ok && pair_work<BLOCK_N, kSplitTail>(item, num_pairs, num_m, num_n, w);
             item += num_pairs, ++it) {
            const int m_pair = w.m_pair;
            const int acc = it & 1;
            const uint32_t acc_phase = static_cast<uint32_t>(it >> 1) & 1u;
            if (!mbar_wait(&tfull_bar[acc], acc_phase, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + acc * BLOCK_N + (static_cast<uint32_t>(q * 32) << 16);
            const int m = (m_pair * 2 + static_cast<int>(cta)) * kBlockM + q * 32 + lane;
#pragma unroll 1
            for (int c0 = 0; c0 < w.width; c0 += 16) {
                uint32_t v[16];
                tmem_ld_16(t_row + c0, v);
                tmem_ld_wait();
                const int n0 = w.n0 + c0;
                if (m >= p.M || n0 >= p.N) continue;
                if (EPI == kEpiStore) {
                    uint4* dst = reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.out) + static_cast<size_t>(m) * p.N + n0);
                    uint32_t w[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) w[c] = pack_bf16x2(__uint_as_float(v[2 * c]), __uint_as_float(v[2 * c + 1]));
                    dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                    dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
                } else {
                    const uint32_t mbits =
                        *reinterpret_cast<const uint16_t*>(p.mask + static_cast<size_t>(m) * (p.N >> 3) + (n0 >> 3));
                    uint32_t w[4];
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const uint32_t mb = (mbits >> (4 * g)) & 0xFu;
                        const int p0 = __ffs(mb) - 1, p1 = 31 - __clz(mb);
                        const float e0 = __uint_as_float(v[4 * g]), e1 = __uint_as_float(v[4 * g + 1]),
                                    e2 = __uint_as_float(v[4 * g + 2]), e3 = __uint_as_float(v[4 * g + 3]);
                        const float lo = p0 == 0 ? e0 : (p0 == 1 ? e1 : e2);
                        const float hi = p1 == 1 ? e1 : (p1 == 2 ? e2 : e3);
                        w[g] = pack_bf16x2(lo, hi);
                    }
                    *reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.out) + static_cast<size_t>(m) * (p.N >> 1) + (n0 >> 1)) =
                        make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&tempty_bar[acc]), 0));
        }
    }

    __syncwarp();
    if (*abort_flag) drain_after_abort();
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

// =====================================================================================
// Sparse CTA-pair GEMM with a 512-row tile: the pair runs TWO 256-row MMA sub-tiles against
// ONE staged activation tile, so every activation byte pulled from L2 feeds twice as many
// MMAs (L2 -> SM bytes per FLOP drop by 31 % against the 256-row tile; that fabric, not DRAM
// or the tensor pipe, is what bounds these GEMMs).  Tensor memory then holds one accumulator
// per sub-tile (2 x BLOCK_N columns) plus the metadata columns, so accumulators are single
// buffered; the epilogue is made short instead: accumulator rows are transposed through
// shared memory and leave as TMA stores of 32 tokens x 128 features.
//   128-row block of A handled by CTA c for sub-tile s of tile mt:  4*mt + 2*s + c.
// =====================================================================================
constexpr int kPrefetchAhead = 8;          // k-blocks of L2 prefetch distance for activation boxes

template <int BLOCK_N, int STAGES>
struct SparseQuadCfg {
    static constexpr int kHalfN = BLOCK_N / 2;
    static constexpr int kABytes = kBlockM * 128;                 // per sub-tile
    static constexpr int kBBytes = kHalfN * 256;
    static constexpr int kEBytes = 2048;                          // per sub-tile
    static constexpr int kOffB = 2 * kABytes;
    static constexpr int kOffE = kOffB + kBBytes;
    static constexpr int kStageBytes = kOffE + 2 * kEBytes;
    static constexpr int kStoreRows = 32;                         // tokens per TMA store
    static constexpr int kStoreCols = 32;                         // features per TMA store (one warp's lanes)
    static constexpr int kStoreBytes = kStoreRows * kStoreCols * 2;   // 2 KB staging buffer
    static constexpr int kEpiWarps = 8;                           // two warps per tensor-memory lane quadrant
    static constexpr int kThreads = 64 + 32 * kEpiWarps;
    static constexpr int kOffStore = STAGES * kStageBytes;
    static constexpr int kOffBar = kOffStore + kEpiWarps * 2 * kStoreBytes;
    static constexpr int kSmemBytes = kOffBar + 256 + 1024;
    static constexpr int kECol = 2 * BLOCK_N;
    static_assert(BLOCK_N % 32 == 0 && kHalfN % 8 == 0 && 2 * BLOCK_N + 16 <= 512, "tile does not fit tensor memory");
    static_assert(kBBytes % 2048 == 0 && kStageBytes % 1024 == 0, "stage must keep 1024-byte alignment");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

// Tile order of the 512-row-tile kernel: row tiles fastest inside a group of `group_m` row tiles,
// then token blocks, then the next group.  The pairs that work on one token block side by side
// share its activation tile; a group's share of the compressed weight is what has to stay in L2
// while the token blocks sweep by.  `first` marks the tile that prefetches the block's
// activations into L2 for its group.
__device__ __forceinline__ void quad_tile(int tile, int num_m, int num_n, int group_m, int& mt, int& n_blk,
                                          bool& first) {
    const int group_size = group_m * num_n;
    const int g = tile / group_size;
    const int first_m = g * group_m;
    const int gm = min(num_m - first_m, group_m);
    const int local = tile - g * group_size;
    mt = first_m + local % gm;
    n_blk = local / gm;
    first = local % gm == 0;
}

template <int BLOCK_N, int STAGES>
__global__ void __launch_bounds__(SparseQuadCfg<BLOCK_N, STAGES>::kThreads, 1)
sparse_gemm_quad_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                        const __grid_constant__ CUtensorMap tmE, const __grid_constant__ CUtensorMap tmA2,
                        const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmO,
                        const SparseGemmParams p) {
    using Cfg = SparseQuadCfg<BLOCK_N, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBar);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* tfull_bar = empty_bar + STAGES;                // [2], one per sub-tile accumulator
    uint64_t* tempty_bar = tfull_bar + 2;                    // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta = cluster_ctarank();
    const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_mb = p.M / kBlockM;
    const int num_m = (num_mb + 3) / 4;                      // 512-row tiles
    const int num_n = (p.Ntok + BLOCK_N - 1) / BLOCK_N;
    const int num_tiles = num_m * num_n;
    const int num_kb = p.K / 128;
    const int num_ab = (p.r + 63) / 64;
    const int total_kb = num_kb + num_ab;
    const int group_m = p.group_m > 0 && p.group_m < num_m ? p.group_m : num_m;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(&tfull_bar[0], 1);
        mbar_init(&tfull_bar[1], 1);
        mbar_init(&tempty_bar[0], 2 * Cfg::kEpiWarps);
        mbar_init(&tempty_bar[1], 2 * Cfg::kEpiWarps);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, 512);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Programmatic dependent launch: the set-up above may overlap the tail of the previous kernel in
    // the stream; no thread touches global memory before that kernel has completed.
    // (consumer of a fused pair of launches, pdl_mode 2: only the producer thread waits, before its
    // first load of the adapter operand T)
    griddep_launch_dependents();
    if (p.pdl_mode != 2) griddep_wait();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs)
        if (elect_one()) {
            tma_prefetch_desc(&tmA);
            tma_prefetch_desc(&tmB);
            tma_prefetch_desc(&tmE);
            const uint64_t keep = l2_policy_evict_last();
            PipeState ps;
            bool ok = true;
            bool waited = false;
            for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs) {
                int mt, n_blk, next_mt, next_n_blk;
                bool first, next_first = false;
                quad_tile(tile, num_m, num_n, group_m, mt, n_blk, first);
                const int nsub = (4 * mt + 2 < num_mb) ? 2 : 1;              // second sub-tile may lie past M
                const int width = token_tile_width(p.Ntok, n_blk * BLOCK_N, BLOCK_N);
                const int n_row0 = n_blk * BLOCK_N + static_cast<int>(cta) * (width / 2);
                // The pairs working on the same token block (same n_blk, different mt) run side by
                // side and would all wait on the same first-touch DRAM fetch of an activation box.
                // One of them (mt == 0) pulls the boxes into L2 kPrefetchAhead k-blocks early.
                const int next_tile = tile + num_pairs;
                if (next_tile < num_tiles) quad_tile(next_tile, num_m, num_n, group_m, next_mt, next_n_blk, next_first);
                const int next_row0 =
                    next_first ? next_n_blk * BLOCK_N +
                                     static_cast<int>(cta) * (token_tile_width(p.Ntok, next_n_blk * BLOCK_N, BLOCK_N) / 2)
                               : 0;
                for (int kb = 0; kb < total_kb; ++kb) {
                    if (kb < num_kb) {
                        const int pk = kb + kPrefetchAhead;
                        if (pk < num_kb) {
                            if (first) {
                                tma_prefetch_l2_2d(&tmB, pk * 128, n_row0);
                                tma_prefetch_l2_2d(&tmB, pk * 128 + 64, n_row0);
                            }
                        } else if (next_first && pk - num_kb < num_kb) {
                            tma_prefetch_l2_2d(&tmB, (pk - num_kb) * 128, next_row0);
                            tma_prefetch_l2_2d(&tmB, (pk - num_kb) * 128 + 64, next_row0);
                        }
                    }
                    if (!mbar_wait(&empty_bar[ps.stage], ps.phase ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t* st = smem + ps.stage * Cfg::kStageBytes;
                    uint8_t* sB = st + Cfg::kOffB;
                    const uint32_t bar = mapa_shared(smem_u32(&full_bar[ps.stage]), 0);
                    if (kb < num_kb) {
                        if (cta == 0)
                            mbar_expect_tx(&full_bar[ps.stage],
                                           2 * (Cfg::kBBytes + nsub * (Cfg::kABytes + Cfg::kEBytes)));
                        tma_load_2d_pair(sB, &tmB, bar, kb * 128, n_row0);
                        tma_load_2d_pair(sB + Cfg::kHalfN * 128, &tmB, bar, kb * 128 + 64, n_row0);
                        for (int s = 0; s < nsub; ++s) {
                            const int mb = 4 * mt + 2 * s + static_cast<int>(cta);
                            const int mb_e = mb < num_mb ? mb : num_mb - 1;
                            tma_load_2d_pair_hint(st + s * Cfg::kABytes, &tmA, bar, kb * 64, mb * kBlockM, keep);
                            tma_load_2d_pair_hint(st + Cfg::kOffE + s * Cfg::kEBytes, &tmE, bar, 0, mb_e * num_kb + kb,
                                                  keep);
                        }
                    } else {
                        const int ab = kb - num_kb;
                        if (p.pdl_mode == 2 && !waited) {
                            griddep_wait();
                            waited = true;
                        }
                        if (cta == 0)
                            mbar_expect_tx(&full_bar[ps.stage], 2 * (Cfg::kHalfN * 128 + nsub * Cfg::kABytes));
                        tma_load_2d_pair(sB, &tmB2, bar, ab * 64, n_row0);
                        for (int s = 0; s < nsub; ++s) {
                            const int m0 = (4 * mt + 2 * s + static_cast<int>(cta)) * kBlockM;
                            uint8_t* sA = st + s * Cfg::kABytes;
                            if (p.a2_mn_major) {
                                tma_load_2d_pair(sA, &tmA2, bar, m0, ab * 64);
                                tma_load_2d_pair(sA + 8192, &tmA2, bar, m0 + 64, ab * 64);
                            } else {
                                tma_load_2d_pair(sA, &tmA2, bar, ab * 64, m0);
                            }
                        }
                    }
                    ps.advance(STAGES);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (cta == 0 && elect_one()) {
            uint32_t idesc_sp = 0, idesc_ad = 0;              // set per tile: N is the tile's width
            // the MMAs of sub-tile s for k-block kb out of pipeline stage `stage`
            auto issue = [&](int s, int kb, int stage) {
                const uint32_t st = smem_u32(smem + stage * Cfg::kStageBytes);
                const uint32_t sB = st + Cfg::kOffB;
                const uint32_t d_tmem = tmem_base + s * BLOCK_N;
                const uint32_t sA = st + s * Cfg::kABytes;
                if (kb < num_kb) {
                    const uint32_t e_tmem = tmem_base + Cfg::kECol + (kb & 1) * 8 + s * 4;
                    tmem_cp_128x128b_pair(e_tmem, make_smem_desc(st + Cfg::kOffE + s * Cfg::kEBytes, 128, 128,
                                                                 kSwizzleNone));
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint64_t ad = make_smem_desc(sA + j * 32, 16, 1024, kSwizzle128B);
                        const uint64_t bd = make_smem_desc(sB + (j >> 1) * (Cfg::kHalfN * 128) + (j & 1) * 64, 16, 1024,
                                                           kSwizzle128B);
                        umma_bf16_sp_pair(d_tmem, ad, bd, e_tmem + (j & 2), idesc_sp | (j & 1), (kb | j) != 0 ? 1u : 0u);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint64_t ad = p.a2_mn_major ? make_smem_desc(sA + j * 2048, 8192, 1024, kSwizzle128B)
                                                          : make_smem_desc(sA + j * 32, 16, 1024, kSwizzle128B);
                        const uint64_t bd = make_smem_desc(sB + j * 32, 16, 1024, kSwizzle128B);
                        umma_bf16_pair(d_tmem, ad, bd, idesc_ad, 1u);
                    }
                }
                // sub-tile s is complete with its last k-block: its drain may start while the other
                // sub-tile's last MMAs still run
                if (kb == total_kb - 1) umma_commit_pair(&tfull_bar[s], 3);
            };
            PipeState ps;                                     // stage that sub-tile 0 consumes next
            bool ok = true;
            int it = 0;
            ClockProbe probe;
            if (pair_id == 0) probe.begin();
            for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs, ++it) {
                int mt, n_blk;
                bool first_unused;
                quad_tile(tile, num_m, num_n, group_m, mt, n_blk, first_unused);
                const int nsub = (4 * mt + 2 < num_mb) ? 2 : 1;
                const int width = token_tile_width(p.Ntok, n_blk * BLOCK_N, BLOCK_N);
                idesc_sp = make_idesc_bf16(2 * kBlockM, width, false, false, true);
                idesc_ad = make_idesc_bf16(2 * kBlockM, width, p.a2_mn_major != 0, false, false);
                const uint32_t acc_parity = (static_cast<uint32_t>(it) & 1u) ^ 1u;
                if (!mbar_wait(&tempty_bar[0], acc_parity, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                // The epilogue hands the second accumulator back a little after the first.  Until
                // then sub-tile 0 runs ahead through the stages that are already full (they cannot
                // be released before sub-tile 1 has used them too); then sub-tile 1 catches up.
                PipeState pc = ps;                            // stage that sub-tile 1 consumes (and releases) next
                int kb0 = 0;
                bool ready1 = nsub == 1;
                while (ok && !ready1) {
                    ready1 = mbar_test(&tempty_bar[1], acc_parity);
                    if (ready1) break;
                    if (kb0 < total_kb && kb0 < STAGES) {
                        if (!mbar_wait(&full_bar[ps.stage], ps.phase, abort_flag)) { ok = false; break; }
                        tc_fence_after_sync();
                        issue(0, kb0, ps.stage);
                        ps.advance(STAGES);
                        ++kb0;
                    } else {
                        ok = mbar_wait(&tempty_bar[1], acc_parity, abort_flag);
                        ready1 = true;
                    }
                }
                if (!ok) break;
                tc_fence_after_sync();
                if (nsub == 2) {
                    for (int kb1 = 0; kb1 < kb0; ++kb1) {       // catch up
                        issue(1, kb1, pc.stage);
                        umma_commit_pair(&empty_bar[pc.stage], 3);
                        pc.advance(STAGES);
                    }
                }
                for (int kb = kb0; kb < total_kb; ++kb) {        // in step
                    if (!mbar_wait(&full_bar[ps.stage], ps.phase, abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    issue(0, kb, ps.stage);
                    if (nsub == 2) issue(1, kb, ps.stage);
                    umma_commit_pair(&empty_bar[ps.stage], 3);
                    ps.advance(STAGES);
                }
                if (ok && nsub == 1) umma_commit_pair(&tfull_bar[1], 3);        // keep both barriers in phase
            }
            if (pair_id == 0) probe.end(kClockSparse);
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
        // Warp w drains lane quadrant w%4; the two warps of a quadrant take alternate 32-token
        // blocks.  Phase 1 empties both accumulators into registers (packed bf16) and hands them
        // back to the MMA issuer at once -- the accumulators are single buffered, so this is
        // what the next tile waits for.  Phase 2 runs under the next tile's main loop: each warp
        // transposes its 32 x 32 blocks through a private staging buffer and sends them with its
        // own TMA stores; the warps never wait for one another.
        constexpr int kBlocks = BLOCK_N / Cfg::kStoreRows;        // 32-token blocks per accumulator
        constexpr int kMyBlocks = (kBlocks + 1) / 2;              // at most this many per warp
        const int q = warp & 3;
        const int ew = warp - 2;
        const int half = ew >> 2;
        uint8_t* my_buf = smem + Cfg::kOffStore + ew * 2 * Cfg::kStoreBytes;
        const uint64_t stream_out = l2_policy_evict_first();
        bool ok = true;
        int it = 0;
        uint32_t buf = 0;
        for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs, ++it) {
            int mt, n_blk;
            bool first_unused;
            quad_tile(tile, num_m, num_n, group_m, mt, n_blk, first_unused);
            const int nsub = (4 * mt + 2 < num_mb) ? 2 : 1;
            const int width = token_tile_width(p.Ntok, n_blk * BLOCK_N, BLOCK_N);
            uint32_t pk[2][kMyBlocks][16];
            // ---- first accumulator (its drain is what the next tile's first MMA waits for).  Two
            //      16-column loads in flight per wait: the warps of a 320-thread CTA are allocated
            //      registers as twelve, which caps a thread at 168, and 128 of them hold the two
            //      packed accumulators.
            if (!mbar_wait(&tfull_bar[0], static_cast<uint32_t>(it) & 1u, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            {
                const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
#pragma unroll
                for (int j = 0; j < kMyBlocks; ++j) {
                    const int c0 = (2 * j + half) * Cfg::kStoreRows;
                    if (c0 < width) {
                        uint32_t v0[16], v1[16];
                        tmem_ld_16(t_row + c0, v0);
                        tmem_ld_16(t_row + c0 + 16, v1);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            pk[0][j][i] = pack_bf16x2(__uint_as_float(v0[2 * i]), __uint_as_float(v0[2 * i + 1]));
                            pk[0][j][8 + i] = pack_bf16x2(__uint_as_float(v1[2 * i]), __uint_as_float(v1[2 * i + 1]));
                        }
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&tempty_bar[0]), 0));
            // ---- second accumulator
            if (!mbar_wait(&tfull_bar[1], static_cast<uint32_t>(it) & 1u, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            if (nsub == 2) {
                const uint32_t t_row = tmem_base + BLOCK_N + (static_cast<uint32_t>(q * 32) << 16);
#pragma unroll
                for (int j = 0; j < kMyBlocks; ++j) {
                    const int c0 = (2 * j + half) * Cfg::kStoreRows;
                    if (c0 < width) {
                        uint32_t v0[16], v1[16];
                        tmem_ld_16(t_row + c0, v0);
                        tmem_ld_16(t_row + c0 + 16, v1);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            pk[1][j][i] = pack_bf16x2(__uint_as_float(v0[2 * i]), __uint_as_float(v0[2 * i + 1]));
                            pk[1][j][8 + i] = pack_bf16x2(__uint_as_float(v1[2 * i]), __uint_as_float(v1[2 * i + 1]));
                        }
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&tempty_bar[1]), 0));
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                if (s < nsub) {
                    const int m0 = (4 * mt + 2 * s + static_cast<int>(cta)) * kBlockM + q * 32;
#pragma unroll
                    for (int j = 0; j < kMyBlocks; ++j) {
                        const int c0 = (2 * j + half) * Cfg::kStoreRows;
                        if (c0 < width) {
                            // the staging buffer about to be overwritten must have been read by its TMA store
                            if (lane == 0) tma_store_wait_read<1>();
                            __syncwarp();
                            uint16_t* sbuf = reinterpret_cast<uint16_t*>(my_buf + buf * Cfg::kStoreBytes) + lane;
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                sbuf[(2 * i) * Cfg::kStoreCols] = static_cast<uint16_t>(pk[s][j][i] & 0xFFFFu);
                                sbuf[(2 * i + 1) * Cfg::kStoreCols] = static_cast<uint16_t>(pk[s][j][i] >> 16);
                            }
                            fence_proxy_async_smem();
                            __syncwarp();
                            if (lane == 0 && m0 < p.M) {
                                tma_store_2d_hint(&tmO, my_buf + buf * Cfg::kStoreBytes, m0, n_blk * BLOCK_N + c0,
                                                  stream_out);
                                tma_store_commit();
                            }
                            buf ^= 1u;
                        }
                    }
                }
            }
        }
        if (lane == 0) tma_store_wait_all<0>();
    }

    __syncwarp();
    if (*abort_flag) drain_after_abort();
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, 512);
    }
}

// =====================================================================================
// Sparse GEMM for few tokens (inference / decode sizes, Ntok <= BLOCK_N <= 256).
// With so few tokens the GEMM is a stream of compressed weights from HBM, and the big-tile
// kernels above would occupy only a handful of SMs.  Here one CTA owns a 128-row slab of the
// weights (1-CTA tcgen05.mma.sp, M = 128) and a slice of the reduction: a cluster of S CTAs
// splits K, each accumulates its partial tile in tensor memory, parks it in its own shared
// memory, and after a cluster barrier every CTA sums one share of the token rows over all S
// partials through distributed shared memory -- in rank order, so the result is
// deterministic and needs no global workspace.  The adapter K-steps ride on the last rank.
//
// What bounds the kernel is the number of weight bytes in flight, so the weights (values +
// metadata, from HBM, read once) and the activations (from L2, re-read by every slab) travel
// in two separate rings with their own producer threads: a deep one for the weights, a
// shallow one for the activations.
// =====================================================================================
constexpr int kSkinnyPrefetchBlocks = 6;   // k-blocks whose first-byte latency is otherwise exposed (6 x 0.23 us)

template <int BLOCK_N, int A_STAGES, int B_STAGES>
struct SparseSkinnyCfg {
    static constexpr int kABytes = kBlockM * 128;                    // compressed values of one k-block
    static constexpr int kEBytes = 2048;                             // their metadata
    static constexpr int kAStage = kABytes + kEBytes;
    static constexpr int kBStage = BLOCK_N * 256;
    static constexpr int kOffB = A_STAGES * kAStage;
    static constexpr int kOffBar = kOffB + B_STAGES * kBStage;
    static constexpr int kPartialBytes = BLOCK_N * kBlockM * 4;      // fp32 [token][feature], reuses the rings
    static constexpr int kSmemBytes = kOffBar + 512 + 1024;
    static constexpr int kTmemCols = BLOCK_N + 8 <= 32 ? 32 : (BLOCK_N + 8 <= 128 ? 128 : (BLOCK_N + 8 <= 256 ? 256 : 512));
    static_assert(BLOCK_N % 16 == 0 && BLOCK_N >= 16 && BLOCK_N <= 256, "token tile");
    static_assert(kPartialBytes <= kOffBar, "partial tile must fit in the pipeline buffers");
    static_assert(kAStage % 1024 == 0 && kBStage % 1024 == 0 && kSmemBytes <= 232448, "shared memory layout");
    static_assert(2 * (A_STAGES + B_STAGES) * 8 + 16 <= 512, "barrier block");
};

template <int BLOCK_N, int A_STAGES, int B_STAGES>
__global__ void __launch_bounds__(kGemmThreads, 1)
sparse_gemm_skinny_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                          const __grid_constant__ CUtensorMap tmE, const __grid_constant__ CUtensorMap tmA2,
                          const __grid_constant__ CUtensorMap tmB2, const SparseGemmParams p) {
    using Cfg = SparseSkinnyCfg<BLOCK_N, A_STAGES, B_STAGES>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* fullA = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBar);
    uint64_t* emptyA = fullA + A_STAGES;
    uint64_t* fullB = emptyA + A_STAGES;
    uint64_t* emptyB = fullB + B_STAGES;
    uint64_t* tfull_bar = emptyB + B_STAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tfull_bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int splits = static_cast<int>(cluster_nctarank());
    const int rank = static_cast<int>(cluster_ctarank());
    const int m_blk = blockIdx.x / splits;
    const int num_kb = p.K / 128;
    const int kb_per = (num_kb + splits - 1) / splits;
    const int kb0 = min(num_kb, rank * kb_per), kb1 = min(num_kb, kb0 + kb_per);
    const int num_sb = kb1 - kb0;                                            // sparse k-blocks of this rank
    // Dense K-steps (64 wide): the adapter product rides on the last rank; with no sparse part
    // at all (K == 0: a plain few-token dense GEMM) they are split over the ranks instead.
    const int all_ab = (p.r + 63) / 64;
    const int ab_per = num_kb == 0 ? (all_ab + splits - 1) / splits : all_ab;
    const int ab0 = num_kb == 0 ? min(all_ab, rank * ab_per) : 0;
    const int num_ab = num_kb == 0 ? min(all_ab, ab0 + ab_per) - ab0 : (rank == splits - 1 ? all_ab : 0);
    const int total_kb = num_sb + num_ab;

    if (threadIdx.x == 0) {
        for (int s = 0; s < A_STAGES; ++s) { mbar_init(&fullA[s], 1); mbar_init(&emptyA[s], 1); }
        for (int s = 0; s < B_STAGES; ++s) { mbar_init(&fullB[s], 1); mbar_init(&emptyB[s], 1); }
        mbar_init(&tfull_bar[0], 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, Cfg::kTmemCols);
        tmem_relinquish();
    }
    if (warp == 0 && elect_one()) {
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmE);
    }
    if (warp == 2 && elect_one()) tma_prefetch_desc(&tmB);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Everything above overlaps the tail of the previous kernel in the stream when the launch
    // allows it; nothing below may touch global memory before that kernel has finished.  One
    // thing is safe earlier: asking L2 to fetch this CTA's first weight tiles.  A prefetch moves no
    // data into the SM, and L2 is the point of coherence, so a line the previous kernel is still
    // writing stays correct; the first loads after the wait then come at L2 instead of HBM latency.
    //
    // Two launches issued together by one call (T = X L, then the forward that adds T R) use the
    // dependency more finely.  The producer (pdl_mode 1) waits first and releases its dependents
    // afterwards: when the consumer starts, everything that preceded the pair in the stream is
    // complete.  The consumer (pdl_mode 2) therefore streams its weights and activations and runs
    // its whole sparse reduction without waiting; only the thread that loads the producer's
    // output T waits, right before the first such load.  Everything that follows in the consumer
    // (the adapter MMAs, the cluster reduction, the stores) is ordered behind that load.
    if (p.pdl_mode == 1) {
        griddep_wait();
        griddep_launch_dependents();
    } else {
        griddep_launch_dependents();
        if (warp == 0 && elect_one()) {
            // (a short K-slice gains nothing: its few tiles are requested at once after the wait, and the
            // prefetch requests would only sit in front of them in the TMA queue)
            const int n_pf = num_sb >= 8 && p.pdl_mode == 0 ? kSkinnyPrefetchBlocks : 0;
            for (int i = 0; i < n_pf; ++i) {
                tma_prefetch_l2_2d(&tmA, (kb0 + i) * 64, m_blk * kBlockM);
                tma_prefetch_l2_2d(&tmE, 0, m_blk * num_kb + kb0 + i);
            }
        }
        __syncwarp();
        if (p.pdl_mode != 2) griddep_wait();
    }

    if (warp == 0) {
        // ---------------------------------------------------------- weight ring (values + metadata)
        if (elect_one()) {
            const uint64_t stream_once = l2_policy_evict_first();        // weights are read exactly once
            PipeState ps;
            for (int i = 0; i < total_kb; ++i) {
                if (!mbar_wait(&emptyA[ps.stage], ps.phase ^ 1u, abort_flag)) break;
                uint8_t* sA = smem + ps.stage * Cfg::kAStage;
                uint64_t* bar = &fullA[ps.stage];
                if (i < num_sb) {
                    const int kb = kb0 + i;
                    mbar_expect_tx(bar, Cfg::kAStage);
                    tma_load_2d_hint(sA, &tmA, bar, kb * 64, m_blk * kBlockM, stream_once);
                    tma_load_2d_hint(sA + Cfg::kABytes, &tmE, bar, 0, m_blk * num_kb + kb, stream_once);
                } else {
                    const int ab = ab0 + i - num_sb;
                    mbar_expect_tx(bar, Cfg::kABytes);
                    if (p.a2_mn_major) {
                        tma_load_2d(sA, &tmA2, bar, m_blk * kBlockM, ab * 64);
                        tma_load_2d(sA + 8192, &tmA2, bar, m_blk * kBlockM + 64, ab * 64);
                    } else {
                        tma_load_2d(sA, &tmA2, bar, ab * 64, m_blk * kBlockM);
                    }
                }
                ps.advance(A_STAGES);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------- MMA issue
        if (elect_one()) {
            constexpr uint32_t idesc_sp = make_idesc_bf16(kBlockM, BLOCK_N, false, false, true);
            const uint32_t idesc_ad = make_idesc_bf16(kBlockM, BLOCK_N, p.a2_mn_major != 0, false, false);
            PipeState pa, pb;
            bool ok = true;
            for (int i = 0; i < total_kb; ++i) {
                if (!mbar_wait(&fullB[pb.stage], pb.phase, abort_flag)) { ok = false; break; }
                if (!mbar_wait(&fullA[pa.stage], pa.phase, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t sA = smem_u32(smem + pa.stage * Cfg::kAStage);
                const uint32_t sE = sA + Cfg::kABytes;
                const uint32_t sB = smem_u32(smem + Cfg::kOffB + pb.stage * Cfg::kBStage);
                if (i < num_sb) {
                    const uint32_t e_tmem = tmem_base + BLOCK_N + (i & 1) * 4;
                    tmem_cp_128x128b(e_tmem, make_smem_desc(sE, 128, 128, kSwizzleNone));
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint64_t ad = make_smem_desc(sA + j * 32, 16, 1024, kSwizzle128B);
                        const uint64_t bd =
                            make_smem_desc(sB + (j >> 1) * (BLOCK_N * 128) + (j & 1) * 64, 16, 1024, kSwizzle128B);
                        umma_bf16_sp(tmem_base, ad, bd, e_tmem + (j & 2), idesc_sp | (j & 1), (i | j) != 0 ? 1u : 0u);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint64_t ad = p.a2_mn_major ? make_smem_desc(sA + j * 2048, 8192, 1024, kSwizzle128B)
                                                          : make_smem_desc(sA + j * 32, 16, 1024, kSwizzle128B);
                        const uint64_t bd = make_smem_desc(sB + j * 32, 16, 1024, kSwizzle128B);
                        umma_bf16(tmem_base, ad, bd, idesc_ad, (i | j) != 0 ? 1u : 0u);
                    }
                }
                umma_commit(&emptyA[pa.stage]);
                umma_commit(&emptyB[pb.stage]);
                pa.advance(A_STAGES);
                pb.advance(B_STAGES);
            }
            if (ok) umma_commit(&tfull_bar[0]);
        }
    } else if (warp == 2) {
        // ---------------------------------------------------------- activation ring
        if (elect_one()) {
            PipeState ps;
            for (int i = 0; i < total_kb; ++i) {
                if (!mbar_wait(&emptyB[ps.stage], ps.phase ^ 1u, abort_flag)) break;
                uint8_t* sB = smem + Cfg::kOffB + ps.stage * Cfg::kBStage;
                uint64_t* bar = &fullB[ps.stage];
                if (i < num_sb) {
                    const int kb = kb0 + i;
                    mbar_expect_tx(bar, Cfg::kBStage);
                    tma_load_2d(sB, &tmB, bar, kb * 128, 0);
                    tma_load_2d(sB + BLOCK_N * 128, &tmB, bar, kb * 128 + 64, 0);
                } else {
                    if (p.pdl_mode == 2 && i == num_sb) griddep_wait();      // T comes from the launch before this one
                    mbar_expect_tx(bar, BLOCK_N * 128);
                    tma_load_2d(sB, &tmB2, bar, (ab0 + i - num_sb) * 64, 0);
                }
                ps.advance(B_STAGES);
            }
        }
        __syncwarp();
    }

    // ---------------------------------------------------------------- epilogue (warps 2..5)
    // Park the fp32 partial tile in shared memory as [token][feature]; the pipeline buffers are
    // free once the last MMA has completed (tfull).  A rank with no k-block contributes zeros.
    float* partial = reinterpret_cast<float*>(smem);
    bool ok = true;
    if (warp >= 2) {
        const int q = warp & 3;
        if (total_kb > 0) ok = mbar_wait(&tfull_bar[0], 0u, abort_flag);
        tc_fence_after_sync();
        const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
        const int ncols = min(BLOCK_N, (p.Ntok + 15) & ~15);         // columns past the last token are never read
#pragma unroll 1
        for (int c0 = 0; c0 < ncols; c0 += 16) {
            uint32_t v[16];
            if (total_kb > 0 && ok) {
                tmem_ld_16(t_row + c0, v);
                tmem_ld_wait();
            } else {
#pragma unroll
                for (int c = 0; c < 16; ++c) v[c] = 0u;
            }
#pragma unroll
            for (int c = 0; c < 16; ++c) partial[(c0 + c) * kBlockM + q * 32 + lane] = __uint_as_float(v[c]);
        }
        tc_fence_before_sync();
    }
    __syncthreads();
    cluster_sync_all();                                       // every rank's partial tile is in place

    // Token rows are dealt round-robin to the ranks.  One warp sums one token row at a time: a
    // lane owns four consecutive features, fetches its 16 bytes from every rank's partial tile
    // (all S loads in flight together) and adds them in rank order.
    if (!*abort_flag) {
        const int ntok = min(p.Ntok, BLOCK_N);
        const int mine = ntok > rank ? (ntok - rank + splits - 1) / splits : 0;
        const uint32_t my_partial = smem_u32(partial);
        for (int i = warp; i < mine; i += kGemmThreads / 32) {
            const int n = rank + i * splits;
            const uint32_t off = my_partial + static_cast<uint32_t>(n * kBlockM + lane * 4) * 4u;
            float4 v[8];
#pragma unroll
            for (int s = 0; s < 8; ++s)
                if (s < splits) v[s] = ld_shared_cluster_v4(mapa_shared(off, s));
            float4 acc = v[0];
#pragma unroll
            for (int s = 1; s < 8; ++s)
                if (s < splits) { acc.x += v[s].x; acc.y += v[s].y; acc.z += v[s].z; acc.w += v[s].w; }
            uint2 o;
            o.x = pack_bf16x2(acc.x, acc.y);
            o.y = pack_bf16x2(acc.z, acc.w);
            const int m = m_blk * kBlockM + lane * 4;
            if (m < p.M) *reinterpret_cast<uint2*>(p.out + static_cast<size_t>(n) * p.M + m) = o;
        }
    }
    if (*abort_flag) drain_after_abort();
    cluster_sync_all();                                       // peers may still be reading this CTA's tile
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
}

}  // namespace slope
