// Masked weight gradient with the lazy adapter's factor gradients riding along.
//
//   dWc = compress_mask1(dY^T X)          Eq. (sparse_backward_weight) + Algorithm 1 "pruneAndCompress"
//   dR^T[d_out x r] = dY^T T              chain rule on Eq. (concat): dR = T^T dY
//   dL  [d_in  x r] = X^T dT              dL = X^T dT
//
// All three contract over the tokens, and the two small products use the very operand tiles the
// weight-gradient GEMM has just staged: dY^T T needs the dY tile (its A operand), X^T dT the X tile
// (its B operand, read a second time as an A operand -- both are stored tokens x features).  A
// separate pass for dL and dR streams X and dY from HBM once more (2.5 GB per step at LLaMA-7B
// sizes, all of it at the HBM roof); here they cost a few extra MMAs on data that is already in
// shared memory plus two small tiles of T and dT per carried k-block.
//
// Work split.  Tile (m, n) of dW (256 x 256, one CTA pair) carries, besides its own product,
//   - for n < splits_r: the partial sum of dR^T rows [256 m, 256 m + 256) over the k-blocks kb with
//     kb mod splits_r == n,
//   - for m < splits_l: the partial sum of dL rows [256 n, 256 n + 256) over kb mod splits_l == m,
// so that every carrier does the same small share of extra work (an MMA of N = r instead of 256 on
// one k-block in splits) and no tile is much longer than the others.  The fp32 partial sums go to a
// workspace [split][rows][r] and are added in split order by splitk_reduce_kernel: deterministic.
//
// Tensor memory: the 256-column accumulator of the tile is single buffered here (columns 0..255);
// columns 256.. and 384.. hold the two adapter accumulators (r <= 128 each).  A tile is 256
// k-blocks long at 16384 tokens, so draining the accumulator into registers before the next tile
// may start costs about one percent; the stores run under the next tile's main loop.
#pragma once
#include "gemm_kernels.cuh"

namespace slope {

struct DwAdapterParams {
    int M, N, K;                  // d_out, d_in, tokens
    int r;                        // adapter rank, multiple of 16, <= 128
    int splits_r, splits_l;       // partial sums per dR^T row block / per dL row block
    uint16_t* dWc;                // [M x N/2]
    const uint8_t* mask;          // [M x N/8]
    float* ws_r;                  // [splits_r][M][r]
    float* ws_l;                  // [splits_l][N][r]
};

template <int STAGES>
struct DwAdapterCfg {
    static constexpr int kBlockN = 256;
    static constexpr int kABytes = kBlockM * 128;               // 64 tokens x 128 rows of dY
    static constexpr int kBBytes = (kBlockN / 2) * 128;         // 64 tokens x 128 columns of X
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kSmallStages = 2;
    static constexpr int kSmallSlot = 8192;                     // one 64 x 64 box of T or dT
    static constexpr int kSmallBytes = 2 * kSmallSlot;          // T tile, dT tile
    static constexpr int kOffSmall = STAGES * kStageBytes;
    static constexpr int kOffBar = kOffSmall + kSmallStages * kSmallBytes;
    static constexpr int kSmemBytes = kOffBar + 256 + 1024;
    static constexpr int kEpiWarps = 8;
    static constexpr int kThreads = 64 + 32 * kEpiWarps;
    static constexpr int kColR = 256, kColL = 384;
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

template <int STAGES>
__global__ void __launch_bounds__(DwAdapterCfg<STAGES>::kThreads, 1)
dw_adapter_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                       const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmDT,
                       const DwAdapterParams p) {
    using Cfg = DwAdapterCfg<STAGES>;
    constexpr int BLOCK_N = Cfg::kBlockN;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBar);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* full2_bar = empty_bar + STAGES;
    uint64_t* empty2_bar = full2_bar + Cfg::kSmallStages;
    uint64_t* tfull_bar = empty2_bar + Cfg::kSmallStages;
    uint64_t* tempty_bar = tfull_bar + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta = cluster_ctarank();
    const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_m = (p.M + 2 * kBlockM - 1) / (2 * kBlockM);
    const int num_n = (p.N + BLOCK_N - 1) / BLOCK_N;
    const int num_kb = (p.K + 63) / 64;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int s = 0; s < Cfg::kSmallStages; ++s) { mbar_init(&full2_bar[s], 1); mbar_init(&empty2_bar[s], 1); }
        mbar_init(tfull_bar, 1);
        mbar_init(tempty_bar, 2 * Cfg::kEpiWarps);
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
    griddep_launch_dependents();
    griddep_wait();

    // which adapter partial sums an item carries (halved tail items never do: the host checks that
    // no carrier lies among them)
    auto carries = [&](const PairWork& w, bool& carry_r, bool& carry_l, int& n_blk) {
        n_blk = w.n0 / BLOCK_N;
        const bool full = w.width == BLOCK_N;
        carry_r = full && n_blk < p.splits_r;
        carry_l = full && w.m_pair < p.splits_l;
    };

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs)
        if (elect_one()) {
            tma_prefetch_desc(&tmA);
            tma_prefetch_desc(&tmB);
            tma_prefetch_desc(&tmT);
            tma_prefetch_desc(&tmDT);
            PipeState ps, ps2;
            bool ok = true;
            PairWork w;
            for (int item = pair_id; ok && pair_work<BLOCK_N, true>(item, num_pairs, num_m, num_n, w); item += num_pairs) {
                bool carry_r, carry_l;
                int n_blk;
                carries(w, carry_r, carry_l, n_blk);
                const int half_w = w.width / 2;
                const int m0 = (w.m_pair * 2 + static_cast<int>(cta)) * kBlockM;
                const int n0 = w.n0 + static_cast<int>(cta) * half_w;
                const int x_small = static_cast<int>(cta) * (p.r / 2);          // this CTA's half of the r columns
                const uint32_t stage_tx = 2 * (Cfg::kABytes + half_w * 128);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&empty_bar[ps.stage], ps.phase ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t* sA = smem + ps.stage * Cfg::kStageBytes;
                    uint8_t* sB = sA + Cfg::kABytes;
                    const uint32_t bar = mapa_shared(smem_u32(&full_bar[ps.stage]), 0);
                    if (cta == 0) mbar_expect_tx(&full_bar[ps.stage], stage_tx);
                    tma_load_2d_pair(sA, &tmA, bar, m0, kb * 64);
                    tma_load_2d_pair(sA + 8192, &tmA, bar, m0 + 64, kb * 64);
                    tma_load_2d_pair(sB, &tmB, bar, n0, kb * 64);
                    if (half_w > 64) tma_load_2d_pair(sB + 8192, &tmB, bar, n0 + 64, kb * 64);
                    ps.advance(STAGES);
                    const bool kr = carry_r && kb % p.splits_r == n_blk;
                    const bool kl = carry_l && kb % p.splits_l == w.m_pair;
                    if (kr || kl) {
                        if (!mbar_wait(&empty2_bar[ps2.stage], ps2.phase ^ 1u, abort_flag)) { ok = false; break; }
                        uint8_t* sS = smem + Cfg::kOffSmall + ps2.stage * Cfg::kSmallBytes;
                        const uint32_t bar2 = mapa_shared(smem_u32(&full2_bar[ps2.stage]), 0);
                        if (cta == 0) mbar_expect_tx(&full2_bar[ps2.stage], 2 * Cfg::kSmallSlot * ((kr ? 1 : 0) + (kl ? 1 : 0)));
                        // a 64-column box that starts at this CTA's half: its first r/2 columns are the
                        // half of the B operand this CTA contributes, the rest is never read
                        if (kr) tma_load_2d_pair(sS, &tmT, bar2, x_small, kb * 64);
                        if (kl) tma_load_2d_pair(sS + Cfg::kSmallSlot, &tmDT, bar2, x_small, kb * 64);
                        ps2.advance(Cfg::kSmallStages);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (cta == 0 && elect_one()) {
            constexpr uint32_t idesc_full = make_idesc_bf16(2 * kBlockM, BLOCK_N, true, true, false);
            constexpr uint32_t idesc_half = make_idesc_bf16(2 * kBlockM, BLOCK_N / 2, true, true, false);
            const uint32_t idesc_ad = make_idesc_bf16(2 * kBlockM, p.r, true, true, false);
            PipeState ps, ps2;
            bool ok = true;
            int it = 0;
            PairWork w;
            for (int item = pair_id; ok && pair_work<BLOCK_N, true>(item, num_pairs, num_m, num_n, w);
                 item += num_pairs, ++it) {
                bool carry_r, carry_l;
                int n_blk;
                carries(w, carry_r, carry_l, n_blk);
                const uint32_t idesc = w.width == BLOCK_N ? idesc_full : idesc_half;
                if (!mbar_wait(tempty_bar, (static_cast<uint32_t>(it) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                uint32_t acc_r = 0, acc_l = 0;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&full_bar[ps.stage], ps.phase, abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t sA = smem_u32(smem + ps.stage * Cfg::kStageBytes);
                    const uint32_t sB = sA + Cfg::kABytes;
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        umma_bf16_pair(tmem_base, make_smem_desc(sA + j * 2048, 8192, 1024, kSwizzle128B),
                                       make_smem_desc(sB + j * 2048, 8192, 1024, kSwizzle128B), idesc, (kb | j) != 0 ? 1u : 0u);
                    const bool kr = carry_r && kb % p.splits_r == n_blk;
                    const bool kl = carry_l && kb % p.splits_l == w.m_pair;
                    if (kr || kl) {
                        if (!mbar_wait(&full2_bar[ps2.stage], ps2.phase, abort_flag)) { ok = false; break; }
                        tc_fence_after_sync();
                        const uint32_t sS = smem_u32(smem + Cfg::kOffSmall + ps2.stage * Cfg::kSmallBytes);
                        if (kr) {          // dR^T rows of this tile row: A = the dY tile, B = T
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                umma_bf16_pair(tmem_base + Cfg::kColR, make_smem_desc(sA + j * 2048, 8192, 1024, kSwizzle128B),
                                               make_smem_desc(sS + j * 2048, 8192, 1024, kSwizzle128B), idesc_ad, acc_r | j);
                            acc_r = 1;
                        }
                        if (kl) {          // dL rows of this tile column: A = the X tile (read as [K x M]), B = dT
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                umma_bf16_pair(tmem_base + Cfg::kColL, make_smem_desc(sB + j * 2048, 8192, 1024, kSwizzle128B),
                                               make_smem_desc(sS + Cfg::kSmallSlot + j * 2048, 8192, 1024, kSwizzle128B),
                                               idesc_ad, acc_l | j);
                            acc_l = 1;
                        }
                        umma_commit_pair(&empty2_bar[ps2.stage], 3);
                        ps2.advance(Cfg::kSmallStages);
                    }
                    umma_commit_pair(&empty_bar[ps.stage], 3);
                    ps.advance(STAGES);
                }
                if (ok) umma_commit_pair(tfull_bar, 3);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
        // Two warps per tensor-memory lane quadrant; each takes half of the tile's columns, picks the two
        // kept columns of every group of four (first-pass mask), packs them to bf16 in registers and hands
        // the accumulator back; the global stores follow under the next tile's main loop.  The adapter
        // partial sums leave as fp32 before the hand-back (first warp of a quadrant: dR^T, second: dL).
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        bool ok = true;
        int it = 0;
        PairWork w;
        for (int item = pair_id; ok && pair_work<BLOCK_N, true>(item, num_pairs, num_m, num_n, w); item += num_pairs, ++it) {
            bool carry_r, carry_l;
            int n_blk;
            carries(w, carry_r, carry_l, n_blk);
            const int row_in_cta = q * 32 + lane;
            const int m = (w.m_pair * 2 + static_cast<int>(cta)) * kBlockM + row_in_cta;
            // (a CTA's accumulator rows hold the full tile width; the two warps of a quadrant split it)
            const int c_begin = half * (w.width / 2);
            const int n_first = w.n0 + c_begin;                        // first global column this warp packs
            const bool live = m < p.M && n_first < p.N;
            // first-pass mask bits of this thread's columns, fetched before the accumulator is ready
            uint32_t mbits[4] = {0u, 0u, 0u, 0u};
            if (live) {
                const uint8_t* mp = p.mask + static_cast<size_t>(m) * (p.N >> 3) + (n_first >> 3);
                if (w.width == BLOCK_N) {
                    const uint4 v = __ldg(reinterpret_cast<const uint4*>(mp));
                    mbits[0] = v.x; mbits[1] = v.y; mbits[2] = v.z; mbits[3] = v.w;
                } else {
                    const uint2 v = __ldg(reinterpret_cast<const uint2*>(mp));
                    mbits[0] = v.x; mbits[1] = v.y;
                }
            }
            if (!mbar_wait(tfull_bar, static_cast<uint32_t>(it) & 1u, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
            uint32_t pk[32];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (16 * i < w.width / 2) {
                    uint32_t v[16];
                    tmem_ld_16(t_row + c_begin + 16 * i, v);
                    tmem_ld_wait();
                    const uint32_t mb16 = (mbits[i >> 1] >> (16 * (i & 1))) & 0xFFFFu;
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const uint32_t mb = (mb16 >> (4 * g)) & 0xFu;
                        const int p0 = __ffs(mb) - 1, p1 = 31 - __clz(mb);
                        const float e0 = __uint_as_float(v[4 * g]), e1 = __uint_as_float(v[4 * g + 1]),
                                    e2 = __uint_as_float(v[4 * g + 2]), e3 = __uint_as_float(v[4 * g + 3]);
                        const float lo = p0 == 0 ? e0 : (p0 == 1 ? e1 : e2);
                        const float hi = p1 == 1 ? e1 : (p1 == 2 ? e2 : e3);
                        pk[4 * i + g] = pack_bf16x2(lo, hi);
                    }
                }
            }
            // adapter partial sums: fp32 rows of r columns into workspace[split][row][r]
            if (half == 0 ? carry_r : carry_l) {
                const int row = half == 0 ? m : n_blk * BLOCK_N + static_cast<int>(cta) * kBlockM + row_in_cta;
                const int rows_total = half == 0 ? p.M : p.N;
                const int split = half == 0 ? n_blk : w.m_pair;
                float* dst = (half == 0 ? p.ws_r : p.ws_l) + (static_cast<size_t>(split) * rows_total + row) * p.r;
                const uint32_t t_ad = t_row + (half == 0 ? Cfg::kColR : Cfg::kColL);
#pragma unroll 1
                for (int c0 = 0; c0 < p.r; c0 += 16) {
                    uint32_t v[16];
                    tmem_ld_16(t_ad + c0, v);
                    tmem_ld_wait();
                    if (row < rows_total) {
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            reinterpret_cast<float4*>(dst + c0)[c] =
                                make_float4(__uint_as_float(v[4 * c]), __uint_as_float(v[4 * c + 1]),
                                            __uint_as_float(v[4 * c + 2]), __uint_as_float(v[4 * c + 3]));
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(tempty_bar), 0));
            if (live) {
                uint4* dst = reinterpret_cast<uint4*>(p.dWc + static_cast<size_t>(m) * (p.N >> 1) + (n_first >> 1));
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (16 * i < w.width / 2) dst[i] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
            }
        }
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

}  // namespace slope
