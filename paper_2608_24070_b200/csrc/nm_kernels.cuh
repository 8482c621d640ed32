// General N:M magnitude pruning to masked-dense matrices (emulation of N:M sparsity for
// accuracy studies, and the matrices A^R and A^{R,C} of Lemma 1 / Eq. (sparsity_ratio)).
// HBM-bound streaming kernels: every element is read once and written once.
//
// Selection rule, as for 2:4: in a group of M entries keep the N of largest 15-bit bf16
// magnitude, the lower position winning ties: u beats t when key[u] > key[t], or
// key[u] == key[t] and u < t, and entry t is kept iff fewer than N entries beat it.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace slope {

// Bit t of the result: entry t of the group (keys in key[0..M)) is kept.
// COUNT: for every entry count the entries that beat it (M (M - 1) compares).
// SORT:  extend the keys by the position (key * 16 + 15 - t: distinct, and among equal
//        magnitudes the lower position is larger), sort them with a bitonic network of
//        min / max pairs, keep an entry iff its extended key reaches the N-th largest.
// Which one is faster depends on M and on the registers the calling kernel has left; the
// choices below are the measured ones (11008 x 4096, fraction of the HBM peak):
//   first pass   M = 8: count 0.58, sort 0.62;  M = 16: count 0.36, sort 0.52
//   second pass  M = 8: count 0.48, sort 0.39;  M = 16: count 0.23, sort 0.34
template <int M, bool SORT>
__device__ __forceinline__ uint32_t keep_n_of_m(const uint32_t (&key)[M], int n) {
    uint32_t keep = 0;
    if constexpr (!SORT) {
#pragma unroll
        for (int t = 0; t < M; ++t) {
            int beaten_by = 0;
#pragma unroll
            for (int u = 0; u < M; ++u) {
                if (u < t) beaten_by += key[u] >= key[t] ? 1 : 0;
                if (u > t) beaten_by += key[u] > key[t] ? 1 : 0;
            }
            keep |= (beaten_by < n ? 1u : 0u) << t;
        }
    } else {
        uint32_t ext[M], s[M];
#pragma unroll
        for (int t = 0; t < M; ++t) ext[t] = s[t] = (key[t] << 4) | static_cast<uint32_t>(15 - t);
#pragma unroll
        for (int k = 2; k <= M; k <<= 1) {
#pragma unroll
            for (int j = k >> 1; j > 0; j >>= 1) {
#pragma unroll
                for (int i = 0; i < M; ++i) {
                    const int l = i ^ j;
                    if (l > i) {
                        const uint32_t hi = max(s[i], s[l]), lo = min(s[i], s[l]);
                        const bool descending = (i & k) == 0;
                        s[i] = descending ? hi : lo;
                        s[l] = descending ? lo : hi;
                    }
                }
            }
        }
        uint32_t nth = s[0];                               // s is in descending order
#pragma unroll
        for (int t = 1; t < M; ++t) nth = t < n ? s[t] : nth;
#pragma unroll
        for (int t = 0; t < M; ++t) keep |= (ext[t] >= nth ? 1u : 0u) << t;
    }
    return keep;
}

// First pass: groups of M consecutive entries along a row.  A thread owns 16 consecutive
// entries (two 16-byte loads = 16 / M whole groups), writes them back with the pruned entries
// zeroed (+0) and, when asked, its 16 mask bits (bit j % 8 of byte j / 8: one aligned 16-bit
// store).  `out` may be `W` itself.
template <int M>
__global__ void __launch_bounds__(256)
prune_nm_kernel(const uint4* W, size_t n_chunks, int n, uint4* out, uint16_t* __restrict__ mask) {
    static_assert(M == 2 || M == 4 || M == 8 || M == 16, "group size");
    const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
    for (size_t c = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; c < n_chunks; c += stride) {
        const uint4 a = __ldcs(W + 2 * c), b = __ldcs(W + 2 * c + 1);       // streamed: read once
        uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        uint32_t keep = 0;
#pragma unroll
        for (int g = 0; g < 16 / M; ++g) {
            uint32_t key[M];
#pragma unroll
            for (int t = 0; t < M; ++t) {
                const int e = g * M + t;
                key[t] = (w[e >> 1] >> (16 * (e & 1))) & 0x7FFFu;
            }
            keep |= keep_n_of_m<M, (M >= 8)>(key, n) << (g * M);
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const uint32_t lo = (keep >> (2 * q)) & 1u ? 0x0000FFFFu : 0u;
            const uint32_t hi = (keep >> (2 * q + 1)) & 1u ? 0xFFFF0000u : 0u;
            w[q] &= lo | hi;
        }
        __stcs(out + 2 * c, make_uint4(w[0], w[1], w[2], w[3]));
        __stcs(out + 2 * c + 1, make_uint4(w[4], w[5], w[6], w[7]));
        if (mask != nullptr) mask[c] = static_cast<uint16_t>(keep);
    }
}

// Second pass: groups of M consecutive entries down a column of the already pruned matrix
// (entries outside the first-pass mask count as zeros).  A thread owns M rows x 8 columns in
// W's own orientation: M 16-byte loads at row pitch (a warp reads 512 contiguous bytes per
// row) and one mask byte per row; output in the same orientation.  mask2 = kept by both passes.
// `out` may be `W` itself.
template <int M>
__global__ void __launch_bounds__(256)
double_prune_nm_kernel(const uint4* W, const uint8_t* __restrict__ mask1, int d_out, int d_in, int n,
                       uint4* out, uint8_t* __restrict__ mask2) {
    static_assert(M == 2 || M == 4 || M == 8 || M == 16, "group size");
    const int row_u4 = d_in / 8;
    const size_t total = static_cast<size_t>(d_out / M) * row_u4;
    const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
    for (size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < total; idx += stride) {
        const size_t h = idx / row_u4, c = idx % row_u4;
        const size_t base = h * M * row_u4 + c;
        uint32_t w[M][4];
        // first-pass mask bytes and second-pass keep bits of the M rows, four rows per register (the
        // 16-row pattern otherwise needs more than 255 registers and spills)
        constexpr int kPacked = (M + 3) / 4;
        uint32_t m1p[kPacked], keep_p[kPacked];
#pragma unroll
        for (int i = 0; i < kPacked; ++i) { m1p[i] = 0; keep_p[i] = 0; }
#pragma unroll
        for (int t = 0; t < M; ++t) {
            const uint4 v = __ldcs(W + base + static_cast<size_t>(t) * row_u4);
            w[t][0] = v.x; w[t][1] = v.y; w[t][2] = v.z; w[t][3] = v.w;
            m1p[t >> 2] |= static_cast<uint32_t>(mask1[base + static_cast<size_t>(t) * row_u4]) << (8 * (t & 3));
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            uint32_t key[M];
#pragma unroll
            for (int t = 0; t < M; ++t)
                key[t] = (m1p[t >> 2] >> (8 * (t & 3) + k)) & 1u ? (w[t][k >> 1] >> (16 * (k & 1))) & 0x7FFFu : 0u;
            const uint32_t keep = keep_n_of_m<M, (M >= 16)>(key, n);
#pragma unroll
            for (int t = 0; t < M; ++t) keep_p[t >> 2] |= ((keep >> t) & 1u) << (8 * (t & 3) + k);
        }
#pragma unroll
        for (int t = 0; t < M; ++t) {
            const uint32_t both = ((keep_p[t >> 2] & m1p[t >> 2]) >> (8 * (t & 3))) & 0xFFu;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t lo = (both >> (2 * q)) & 1u ? 0x0000FFFFu : 0u;
                const uint32_t hi = (both >> (2 * q + 1)) & 1u ? 0xFFFF0000u : 0u;
                w[t][q] &= lo | hi;
            }
            __stcs(out + base + static_cast<size_t>(t) * row_u4, make_uint4(w[t][0], w[t][1], w[t][2], w[t][3]));
            if (mask2 != nullptr) mask2[base + static_cast<size_t>(t) * row_u4] = static_cast<uint8_t>(both);
        }
    }
}

// out = G where the mask bit is set, +0 elsewhere (a dense gradient restricted to a static
// N:M pattern).  A thread owns 16 consecutive entries; `out` may be `G` itself.
__global__ void __launch_bounds__(256)
apply_mask_kernel(const uint4* G, const uint16_t* __restrict__ mask, size_t n_chunks, uint4* out) {
    const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
    for (size_t c = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; c < n_chunks; c += stride) {
        const uint4 a = __ldcs(G + 2 * c), b = __ldcs(G + 2 * c + 1);
        uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        const uint32_t keep = mask[c];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const uint32_t lo = (keep >> (2 * q)) & 1u ? 0x0000FFFFu : 0u;
            const uint32_t hi = (keep >> (2 * q + 1)) & 1u ? 0xFFFF0000u : 0u;
            w[q] &= lo | hi;
        }
        __stcs(out + 2 * c, make_uint4(w[0], w[1], w[2], w[3]));
        __stcs(out + 2 * c + 1, make_uint4(w[4], w[5], w[6], w[7]));
    }
}

// Number of element positions in which two bit masks differ (the per-iteration mask change
// that the comparison with dynamically re-selected masks plots).  16-byte loads, popcount of the
// XOR, one integer atomic per warp: the count is exact whatever the order.
__global__ void __launch_bounds__(256)
mask_difference_kernel(const uint4* __restrict__ a, const uint4* __restrict__ b, size_t n_vec,
                       unsigned long long* __restrict__ count) {
    unsigned int local = 0;
    const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
    for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_vec; i += stride) {
        const uint4 x = __ldcs(a + i), y = __ldcs(b + i);
        local += __popc(x.x ^ y.x) + __popc(x.y ^ y.y) + __popc(x.z ^ y.z) + __popc(x.w ^ y.w);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(0xFFFFFFFFu, local, o);
    if ((threadIdx.x & 31) == 0 && local != 0) atomicAdd(count, static_cast<unsigned long long>(local));
}

}  // namespace slope
