// HBM-bound kernels: first-pass 2:4 magnitude selection + compression, second-pass
// (double pruning) selection on the transposed matrix, metadata diagnostics.
//
// Both pruning kernels work on 128 x 128 element tiles (one CTA of 256 threads per
// tile) so that the 2 KB metadata block of a tile -- already in the order the sparse
// tensor-core instruction reads it -- and the tile's mask rows leave the CTA as full
// 16-byte stores.  Every global access is a 16-byte vector, rows are read 256 B at a
// time per half-warp.
#pragma once
#include "ptx.cuh"

namespace slope {

// Two largest of four magnitudes, lower position wins ties.  Each candidate is folded
// into one integer (magnitude << 2 | 3 - position) so that plain max/min decide.
// Returns the kept positions p0 < p1.
__device__ __forceinline__ void top2_of_4(uint32_t k0, uint32_t k1, uint32_t k2, uint32_t k3, int& p0, int& p1) {
    const uint32_t c0 = (k0 << 2) | 3u, c1 = (k1 << 2) | 2u, c2 = (k2 << 2) | 1u, c3 = (k3 << 2);
    const uint32_t hi01 = max(c0, c1), lo01 = min(c0, c1);
    const uint32_t hi23 = max(c2, c3), lo23 = min(c2, c3);
    const uint32_t first = max(hi01, hi23);
    const uint32_t second = max(min(hi01, hi23), hi01 > hi23 ? lo01 : lo23);
    const int i1 = 3 - static_cast<int>(first & 3u), i2 = 3 - static_cast<int>(second & 3u);
    p0 = min(i1, i2);
    p1 = max(i1, i2);
}

__device__ __forceinline__ uint32_t pick16(uint32_t e0, uint32_t e1, uint32_t e2, uint32_t e3, int p) {
    return p == 0 ? e0 : (p == 1 ? e1 : (p == 2 ? e2 : e3));
}

// One group of four bf16 (two 32-bit words, element 0 in the low half of `lo`):
// returns kept pair packed as bf16x2 (ascending position), 4-bit code and 4-bit mask.
__device__ __forceinline__ uint32_t prune_group(uint32_t lo, uint32_t hi, uint32_t& code, uint32_t& mbits) {
    const uint32_t e0 = lo & 0xFFFFu, e1 = lo >> 16, e2 = hi & 0xFFFFu, e3 = hi >> 16;
    int p0, p1;
    top2_of_4(e0 & 0x7FFFu, e1 & 0x7FFFu, e2 & 0x7FFFu, e3 & 0x7FFFu, p0, p1);
    code = static_cast<uint32_t>(p0 | (p1 << 2));
    mbits = (1u << p0) | (1u << p1);
    return pick16(e0, e1, e2, e3, p0) | (pick16(e0, e1, e2, e3, p1) << 16);
}

// Byte offset, inside a 2 KB metadata block, of the byte holding the codes of local
// row rr (0..127) and local 8-column slot c8 (0..15).
__device__ __forceinline__ int meta_byte_offset(int rr, int c8) {
    const int cs = c8 >> 1;                                   // 16-column slot
    const int word = (16 * (rr >> 4) + 8 * (cs & 1) + (rr & 7)) * 4 + (cs >> 1);
    return word * 4 + ((rr >> 3) & 1) * 2 + (c8 & 1);
}

__global__ void __launch_bounds__(256) prune24_kernel(const uint4* __restrict__ W, int d_out, int d_in,
                                                      uint2* __restrict__ vals, uint4* __restrict__ meta,
                                                      uint4* __restrict__ mask /* may be null */) {
    __shared__ __align__(16) uint8_t s_meta[2048];
    __shared__ __align__(16) uint8_t s_mask[2048];
    const int cb = blockIdx.x, rb = blockIdx.y;
    const int tid = threadIdx.x;
    const int c8 = tid & 15, r0 = tid >> 4;
    const size_t row_u4 = static_cast<size_t>(d_in) >> 3;

    uint4 w[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const size_t row = static_cast<size_t>(rb) * 128 + i * 16 + r0;
        w[i] = __ldg(W + row * row_u4 + cb * 16 + c8);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int rr = i * 16 + r0;
        const size_t row = static_cast<size_t>(rb) * 128 + rr;
        uint32_t code0, code1, m0, m1;
        uint2 out;
        out.x = prune_group(w[i].x, w[i].y, code0, m0);
        out.y = prune_group(w[i].z, w[i].w, code1, m1);
        vals[row * row_u4 + cb * 16 + c8] = out;                  // d_in/8 uint2 per compressed row
        s_meta[meta_byte_offset(rr, c8)] = static_cast<uint8_t>(code0 | (code1 << 4));
        s_mask[rr * 16 + c8] = static_cast<uint8_t>(m0 | (m1 << 4));
    }
    __syncthreads();
    if (tid < 128) {
        const size_t blk = static_cast<size_t>(rb) * (d_in >> 7) + cb;
        meta[blk * 128 + tid] = reinterpret_cast<const uint4*>(s_meta)[tid];
    } else if (mask != nullptr) {
        const int rr = tid - 128;
        const size_t row = static_cast<size_t>(rb) * 128 + rr;
        mask[row * (d_in >> 7) + cb] = reinterpret_cast<const uint4*>(s_mask)[rr];
    }
}

// Second pass.  Tile (rb, cb) of W (rows = d_out, cols = d_in) produces tile (cb, rb) of
// the compressed transposed matrix.  Shared memory: the bf16 tile with a 260-byte row
// pitch (column reads are then conflict free), the first-pass mask rows, and staging for
// the three outputs.
constexpr int kDpTilePitchW = 65;            // 32-bit words per tile row (130 bf16)
constexpr int kDpOutPitch = 136;             // bytes per staged output row (128 + 8)
constexpr int kDpSmemBytes = 128 * kDpTilePitchW * 4 + 2048 + 128 * kDpOutPitch + 2048 + 2048;

__global__ void __launch_bounds__(256) double_prune_kernel(const uint4* __restrict__ W,
                                                           const uint8_t* __restrict__ mask1, int d_out, int d_in,
                                                           uint4* __restrict__ valsT, uint4* __restrict__ metaT,
                                                           uint4* __restrict__ mask2 /* may be null */) {
    extern __shared__ __align__(16) uint8_t dp_smem[];
    uint32_t* s_w = reinterpret_cast<uint32_t*>(dp_smem);
    uint8_t* s_m1 = dp_smem + 128 * kDpTilePitchW * 4;
    uint8_t* s_out = s_m1 + 2048;
    uint8_t* s_meta = s_out + 128 * kDpOutPitch;
    uint8_t* s_m2 = s_meta + 2048;

    const int cb = blockIdx.x, rb = blockIdx.y;
    const int tid = threadIdx.x;
    const int c8 = tid & 15, r0 = tid >> 4;
    const size_t row_u4 = static_cast<size_t>(d_in) >> 3;

    uint4 w[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const size_t row = static_cast<size_t>(rb) * 128 + i * 16 + r0;
        w[i] = __ldg(W + row * row_u4 + cb * 16 + c8);
    }
    if (tid < 128) {
        const size_t row = static_cast<size_t>(rb) * 128 + tid;
        reinterpret_cast<uint4*>(s_m1)[tid] =
            __ldg(reinterpret_cast<const uint4*>(mask1 + row * (d_in >> 3)) + cb);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        uint32_t* dst = s_w + (i * 16 + r0) * kDpTilePitchW + c8 * 4;
        dst[0] = w[i].x; dst[1] = w[i].y; dst[2] = w[i].z; dst[3] = w[i].w;
    }
    __syncthreads();

    const int j = tid & 127;                         // local column of W = local row of W^T
    const int lane = tid & 31;
    const uint16_t* s_w16 = reinterpret_cast<const uint16_t*>(s_w);
#pragma unroll 1
    for (int it = 0; it < 8; ++it) {
        const int ig = it * 2 + (tid >> 7);          // 8-row slot of the tile (0..15)
        uint32_t e[8], kept = 0;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const int i = ig * 8 + t;
            const uint32_t k1 = (s_m1[i * 16 + (j >> 3)] >> (j & 7)) & 1u;
            kept |= k1 << t;
            e[t] = k1 ? s_w16[i * (kDpTilePitchW * 2) + j] : 0u;
        }
        int p0, p1, q0, q1;
        top2_of_4(e[0] & 0x7FFFu, e[1] & 0x7FFFu, e[2] & 0x7FFFu, e[3] & 0x7FFFu, p0, p1);
        top2_of_4(e[4] & 0x7FFFu, e[5] & 0x7FFFu, e[6] & 0x7FFFu, e[7] & 0x7FFFu, q0, q1);
        uint2 out;
        out.x = pick16(e[0], e[1], e[2], e[3], p0) | (pick16(e[0], e[1], e[2], e[3], p1) << 16);
        out.y = pick16(e[4], e[5], e[6], e[7], q0) | (pick16(e[4], e[5], e[6], e[7], q1) << 16);
        *reinterpret_cast<uint2*>(s_out + j * kDpOutPitch + ig * 8) = out;
        s_meta[meta_byte_offset(j, ig)] = static_cast<uint8_t>(p0 | (p1 << 2) | (q0 << 4) | (q1 << 6));
        const uint32_t sel = ((1u << p0) | (1u << p1) | (16u << q0) | (16u << q1)) & kept;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const uint32_t word = __ballot_sync(0xFFFFFFFFu, (sel >> t) & 1u);
            if (lane == 0) reinterpret_cast<uint32_t*>(s_m2)[(ig * 8 + t) * 4 + (j >> 5)] = word;
        }
    }
    __syncthreads();

    // (W^T) tile (cb, rb): values rows of 128 B, metadata block, second mask rows.
    const size_t vrow_u4 = static_cast<size_t>(d_out) >> 4;        // uint4 per row of valsT (d_out/2 bf16)
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
        const int jr = pass * 32 + (tid >> 3), seg = tid & 7;
        const uint2 a = *reinterpret_cast<const uint2*>(s_out + jr * kDpOutPitch + seg * 16);
        const uint2 b = *reinterpret_cast<const uint2*>(s_out + jr * kDpOutPitch + seg * 16 + 8);
        valsT[(static_cast<size_t>(cb) * 128 + jr) * vrow_u4 + rb * 8 + seg] = make_uint4(a.x, a.y, b.x, b.y);
    }
    if (tid < 128) {
        const size_t blk = static_cast<size_t>(cb) * (d_out >> 7) + rb;
        metaT[blk * 128 + tid] = reinterpret_cast<const uint4*>(s_meta)[tid];
    } else if (mask2 != nullptr) {
        const int rr = tid - 128;
        const size_t row = static_cast<size_t>(rb) * 128 + rr;
        mask2[row * (d_in >> 7) + cb] = reinterpret_cast<const uint4*>(s_m2)[rr];
    }
}

// Tensor-core-order metadata -> canonical uint16 [rows x cols/16].
__global__ void __launch_bounds__(256) meta_to_canonical_kernel(const uint16_t* __restrict__ hw, int rows, int cols,
                                                                uint16_t* __restrict__ canon) {
    const size_t units_per_row = static_cast<size_t>(cols) >> 4;
    const size_t total = static_cast<size_t>(rows) * units_per_row;
    for (size_t idx = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; idx < total;
         idx += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const size_t i = idx / units_per_row, u = idx % units_per_row;
        const int rr = static_cast<int>(i & 127), cs = static_cast<int>(u & 7);
        const size_t blk = (i >> 7) * (cols >> 7) + (u >> 3);
        const int off = meta_byte_offset(rr, cs * 2);
        canon[idx] = hw[blk * 1024 + (off >> 1)];
    }
}

// ---------------------------------------------------------------------------------------
// Optimizer tail of Algorithm 1.
// ---------------------------------------------------------------------------------------

// "sparseAdd": out = beta * A + gamma * B on two compressed value arrays with one pattern
// (fp32 arithmetic, one rounding to bf16).  Pure streaming: 16-byte vectors, grid-stride.
__global__ void __launch_bounds__(256) sparse_add_kernel(const uint4* __restrict__ A, const uint4* __restrict__ B,
                                                         float beta, float gamma, size_t n_vec,
                                                         uint4* __restrict__ out) {
    for (size_t idx = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; idx < n_vec;
         idx += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const uint4 a = __ldg(A + idx), b = __ldg(B + idx);
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
        uint32_t r[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const float a0 = __uint_as_float(aw[t] << 16), a1 = __uint_as_float(aw[t] & 0xFFFF0000u);
            const float b0 = __uint_as_float(bw[t] << 16), b1 = __uint_as_float(bw[t] & 0xFFFF0000u);
            r[t] = pack_bf16x2(__fmaf_rn(beta, a0, gamma * b0), __fmaf_rn(beta, a1, gamma * b1));
        }
        out[idx] = make_uint4(r[0], r[1], r[2], r[3]);
    }
}

// "updateSparseMatrix" for the transposed copy: rebuild the values of the compressed
// (W^{R,C})^T from new forward values Wc_new under the static masks.  Tile (rb, cb) of W
// (128 x 128 elements = 128 x 64 compressed values) feeds tile (cb, rb) of the transposed copy:
// its metadata block says which two rows of every 4-row group were kept by the second pass,
// the first-pass mask says whether such an element exists at all and at which rank it sits
// in its row's compressed group.
constexpr int kUpdWcPitchW = 33;                 // 32-bit words per staged row of 64 bf16 (+1 pad)
constexpr int kUpdSmemBytes = 128 * kUpdWcPitchW * 4 + 2048 + 2048 + 128 * kDpOutPitch;

__global__ void __launch_bounds__(256) update_transposed_kernel(const uint4* __restrict__ Wc_new,
                                                                const uint8_t* __restrict__ mask1,
                                                                const uint4* __restrict__ metaT, int d_out, int d_in,
                                                                uint4* __restrict__ valsT) {
    extern __shared__ __align__(16) uint8_t up_smem[];
    uint32_t* s_wc = reinterpret_cast<uint32_t*>(up_smem);
    uint8_t* s_m1 = up_smem + 128 * kUpdWcPitchW * 4;
    uint8_t* s_mt = s_m1 + 2048;
    uint8_t* s_out = s_mt + 2048;

    const int cb = blockIdx.x, rb = blockIdx.y;
    const int tid = threadIdx.x;
    const size_t wc_row_u4 = static_cast<size_t>(d_in) >> 4;        // uint4 per compressed row (d_in/2 bf16)
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
        const int rr = pass * 32 + (tid >> 3), seg = tid & 7;
        const uint4 v = __ldg(Wc_new + (static_cast<size_t>(rb) * 128 + rr) * wc_row_u4 + cb * 8 + seg);
        uint32_t* dst = s_wc + rr * kUpdWcPitchW + seg * 4;
        dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
    }
    if (tid < 128) {
        const size_t row = static_cast<size_t>(rb) * 128 + tid;
        reinterpret_cast<uint4*>(s_m1)[tid] = __ldg(reinterpret_cast<const uint4*>(mask1 + row * (d_in >> 3)) + cb);
    } else {
        const size_t blk = static_cast<size_t>(cb) * (d_out >> 7) + rb;
        reinterpret_cast<uint4*>(s_mt)[tid - 128] = __ldg(metaT + blk * 128 + (tid - 128));
    }
    __syncthreads();

    const int j = tid & 127;
    const uint16_t* s_wc16 = reinterpret_cast<const uint16_t*>(s_wc);
    auto fetch = [&](int i) -> uint32_t {
        const uint32_t mbyte = s_m1[i * 16 + (j >> 3)];
        const uint32_t kept = (mbyte >> (j & 7)) & 1u;
        const uint32_t group = (mbyte >> (j & 4)) & 0xFu;
        const int rank = __popc(group & ((1u << (j & 3)) - 1u));
        return kept ? s_wc16[i * (kUpdWcPitchW * 2) + 2 * (j >> 2) + rank] : 0u;
    };
#pragma unroll 1
    for (int it = 0; it < 8; ++it) {
        const int ig = it * 2 + (tid >> 7);
        const uint32_t code = s_mt[meta_byte_offset(j, ig)];
        const int base = ig * 8;
        uint2 out;
        out.x = fetch(base + (code & 3)) | (fetch(base + ((code >> 2) & 3)) << 16);
        out.y = fetch(base + 4 + ((code >> 4) & 3)) | (fetch(base + 4 + ((code >> 6) & 3)) << 16);
        *reinterpret_cast<uint2*>(s_out + j * kDpOutPitch + ig * 8) = out;
    }
    __syncthreads();
    const size_t vrow_u4 = static_cast<size_t>(d_out) >> 4;
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
        const int jr = pass * 32 + (tid >> 3), seg = tid & 7;
        const uint2 a = *reinterpret_cast<const uint2*>(s_out + jr * kDpOutPitch + seg * 16);
        const uint2 b = *reinterpret_cast<const uint2*>(s_out + jr * kDpOutPitch + seg * 16 + 8);
        valsT[(static_cast<size_t>(cb) * 128 + jr) * vrow_u4 + rb * 8 + seg] = make_uint4(a.x, a.y, b.x, b.y);
    }
}

}  // namespace slope
