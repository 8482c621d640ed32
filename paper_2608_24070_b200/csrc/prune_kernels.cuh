// HBM-bound kernels: first-pass 2:4 magnitude selection + compression, second-pass
// (double pruning) selection on the transposed matrix, metadata diagnostics.
//
// Both pruning kernels work on 128 x 128 element tiles (one CTA of 256 threads per
// tile) so that the 2 KB metadata block of a tile -- already in the order the sparse
// tensor-core instruction reads it -- and the tile's mask rows leave the CTA as full
// 16-byte stores.  Every global access is a 16-byte vector.  The selection itself is
// done on packed half-words (two groups per 32-bit lane) because a scalar formulation
// makes these kernels issue-bound long before they reach the HBM roof.
#pragma once
#include "ptx.cuh"

namespace slope {

// ---------------------------------------------------------------------------------------
// Packed selection.  Two groups of four bf16 are processed at once: word E[i] holds element
// i of group 0 in its low half and element i of group 1 in its high half.  All arithmetic
// stays in 32-bit integer / logic instructions on both halves simultaneously:
//   - magnitudes are 15 bits, so (M[i] + 0x80008000) - M[j] never borrows across halves and
//     leaves "M[i] >= M[j]" in bits 15 and 31 (for i < j that is exactly "i beats j", the
//     lower position winning ties);
//   - an element is kept when it beats at least two of the other three (majority of three
//     comparison bits, one LOP3 each);
//   - prmt's sign-replication mode turns the keep bits into half-word masks.
// ---------------------------------------------------------------------------------------
struct PackedPick {
    uint32_t out0, out1;      // kept pair of group 0 / group 1: first kept in the low half
    uint32_t mask_byte;       // 4 keep bits of group 0 | 4 keep bits of group 1 << 4
    uint32_t meta_byte;       // code p0 | p1<<2 of group 0 | code of group 1 << 4
    uint32_t keep[4];         // element i kept: 0xFFFF in the low half (group 0) / high half (group 1)
};

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ uint32_t maj3(uint32_t a, uint32_t b, uint32_t c) { return (a & b) | (a & c) | (b & c); }
__device__ __forceinline__ uint32_t bitsel(uint32_t m, uint32_t a, uint32_t b) { return (m & a) | (~m & b); }

__device__ __forceinline__ PackedPick pick2of4_packed(uint32_t E0, uint32_t E1, uint32_t E2, uint32_t E3) {
    constexpr uint32_t G = 0x80008000u;
    const uint32_t M0 = E0 & 0x7FFF7FFFu, M1 = E1 & 0x7FFF7FFFu, M2 = E2 & 0x7FFF7FFFu, M3 = E3 & 0x7FFF7FFFu;
    const uint32_t c01 = M0 + G - M1, c02 = M0 + G - M2, c03 = M0 + G - M3;
    const uint32_t c12 = M1 + G - M2, c13 = M1 + G - M3, c23 = M2 + G - M3;
    // keep flags in bits 15 / 31
    const uint32_t k0 = maj3(c01, c02, c03);
    const uint32_t k1 = maj3(~c01, c12, c13);
    const uint32_t k2 = maj3(~c02, ~c12, c23);
    const uint32_t k3 = maj3(~c03, ~c13, ~c23);
    // half-word masks (0xFFFF where kept): bytes 0,1 <- sign of byte 1; bytes 2,3 <- sign of byte 3
    const uint32_t m0 = prmt(k0, 0u, 0xBB99u), m1 = prmt(k1, 0u, 0xBB99u);
    const uint32_t m2 = prmt(k2, 0u, 0xBB99u), m3 = prmt(k3, 0u, 0xBB99u);
    const uint32_t first = bitsel(m0, E0, bitsel(m1, E1, E2));      // lowest kept position
    const uint32_t second = bitsel(m3, E3, bitsel(m2, E2, E1));     // highest kept position
    PackedPick r;
    r.out0 = prmt(first, second, 0x5410u);
    r.out1 = prmt(first, second, 0x7632u);
    const uint32_t t = (m0 & 0x00010001u) | (m1 & 0x00020002u) | (m2 & 0x00040004u) | (m3 & 0x00080008u);
    r.mask_byte = (t | (t >> 12)) & 0xFFu;
    const uint32_t p0 = ~m0 & bitsel(m1, 0x00010001u, 0x00020002u);
    const uint32_t p1 = bitsel(m3, 0x00030003u, bitsel(m2, 0x00020002u, 0x00010001u));
    const uint32_t c = p0 | (p1 << 2);
    r.meta_byte = (c | (c >> 12)) & 0xFFu;
    r.keep[0] = m0; r.keep[1] = m1; r.keep[2] = m2; r.keep[3] = m3;
    return r;
}

// Byte offset, inside a 2 KB metadata block, of the byte holding the codes of local
// row rr (0..127) and local 8-column slot c8 (0..15).
__device__ __forceinline__ int meta_byte_offset(int rr, int c8) {
    const int cs = c8 >> 1;                                   // 16-column slot
    const int word = (16 * (rr >> 4) + 8 * (cs & 1) + (rr & 7)) * 4 + (cs >> 1);
    return word * 4 + ((rr >> 3) & 1) * 2 + (c8 & 1);
}

// First pass.  A thread owns 16 consecutive elements of a row (two 16-byte loads): four groups
// = one 16-bit metadata unit, 16 mask bits and eight kept values (one 16-byte store).
__global__ void __launch_bounds__(256) prune24_kernel(const uint4* __restrict__ W, int d_out, int d_in,
                                                      uint4* __restrict__ vals, uint4* __restrict__ meta,
                                                      uint4* __restrict__ mask /* may be null */) {
    __shared__ __align__(16) uint16_t s_meta[1024];
    __shared__ __align__(16) uint16_t s_mask[1024];
    const int cb = blockIdx.x, rb = blockIdx.y;
    const int tid = threadIdx.x;
    const int u = tid & 7, r0 = tid >> 3;                 // 16-column slot, row within a pass of 32 rows
    const size_t row_u4 = static_cast<size_t>(d_in) >> 3;

    uint4 w[4][2];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const size_t row = static_cast<size_t>(rb) * 128 + i * 32 + r0;
        const uint4* src = W + row * row_u4 + cb * 16 + 2 * u;
        w[i][0] = __ldg(src);
        w[i][1] = __ldg(src + 1);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int rr = i * 32 + r0;
        const size_t row = static_cast<size_t>(rb) * 128 + rr;
        // groups 0,1 from the first vector, groups 2,3 from the second
        const PackedPick a = pick2of4_packed(prmt(w[i][0].x, w[i][0].z, 0x5410u), prmt(w[i][0].x, w[i][0].z, 0x7632u),
                                             prmt(w[i][0].y, w[i][0].w, 0x5410u), prmt(w[i][0].y, w[i][0].w, 0x7632u));
        const PackedPick b = pick2of4_packed(prmt(w[i][1].x, w[i][1].z, 0x5410u), prmt(w[i][1].x, w[i][1].z, 0x7632u),
                                             prmt(w[i][1].y, w[i][1].w, 0x5410u), prmt(w[i][1].y, w[i][1].w, 0x7632u));
        vals[row * (row_u4 >> 1) + cb * 8 + u] = make_uint4(a.out0, a.out1, b.out0, b.out1);
        s_meta[meta_byte_offset(rr, 2 * u) >> 1] = static_cast<uint16_t>(a.meta_byte | (b.meta_byte << 8));
        s_mask[rr * 8 + u] = static_cast<uint16_t>(a.mask_byte | (b.mask_byte << 8));
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

// Second pass.  Tile (rb, cb) of W (rows = d_out, cols = d_in) produces tile (cb, rb) of the
// compressed transposed matrix.  A thread owns 8 rows x 8 columns of the tile, read straight
// from global memory (eight 16-byte loads, rows 256 B apart per half-warp).  Groups run down
// the columns here, so a 32-bit word of a row (two adjacent columns) IS the packed pair the
// selection works on: word w of rows 4g..4g+3 gives the groups of columns 2w and 2w+1 without
// any transposition of the input.  Only the outputs (half the bytes) are transposed, through
// an XOR-swizzled 16 KB staging tile whose 64-bit stores are conflict free.
__device__ __forceinline__ uint32_t halfword_mask_from_bits(uint32_t mask_byte, int w) {
    // bit 2w of the byte -> low half-word, bit 2w+1 -> high half-word (all ones where kept)
    const uint32_t z = (mask_byte << (15 - 2 * w)) | (mask_byte << (30 - 2 * w));
    return prmt(z, 0u, 0xBB99u);
}

__global__ void __launch_bounds__(256, 4) double_prune_kernel(const uint4* __restrict__ W,
                                                           const uint8_t* __restrict__ mask1, int d_out, int d_in,
                                                           uint4* __restrict__ valsT, uint4* __restrict__ metaT,
                                                           uint8_t* __restrict__ mask2 /* may be null */) {
    __shared__ __align__(16) uint8_t s_out[128 * 128];       // [column j][16 slots of 8 B], slot index XOR (j >> 3)
    __shared__ __align__(16) uint8_t s_meta[2048];

    const int cb = blockIdx.x, rb = blockIdx.y;
    const int tid = threadIdx.x;
    const int c8 = tid & 15;                                 // 8-column slot of the tile
    const int ig = tid >> 4;                                 // 8-row slot of the tile
    const size_t row_u4 = static_cast<size_t>(d_in) >> 3;
    const size_t mrow = static_cast<size_t>(d_in) >> 3;      // mask bytes per row

    uint4 w[8];
    uint32_t mb[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const size_t row = static_cast<size_t>(rb) * 128 + ig * 8 + t;
        w[t] = __ldg(W + row * row_u4 + cb * 16 + c8);
        mb[t] = __ldg(mask1 + row * mrow + cb * 16 + c8);
    }

    uint32_t sel_bits[8] = {0, 0, 0, 0, 0, 0, 0, 0};         // per row: which of the 8 columns the second pass keeps
    const int meta_base = meta_byte_offset(c8 * 8, ig);      // + 16 per column inside the 8-column slot
#pragma unroll
    for (int wi = 0; wi < 4; ++wi) {
        uint32_t e[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const uint32_t word = wi == 0 ? w[t].x : (wi == 1 ? w[t].y : (wi == 2 ? w[t].z : w[t].w));
            e[t] = word & halfword_mask_from_bits(mb[t], wi);                 // pruned in pass 1 -> +0
        }
        const PackedPick a = pick2of4_packed(e[0], e[1], e[2], e[3]);        // rows 0..3 of columns 2wi, 2wi+1
        const PackedPick b = pick2of4_packed(e[4], e[5], e[6], e[7]);        // rows 4..7
        const int j0 = c8 * 8 + 2 * wi;
        const int slot = (ig ^ c8) * 8;                                        // (j >> 3) & 15 == c8 for both columns
        *reinterpret_cast<uint2*>(s_out + j0 * 128 + slot) = make_uint2(a.out0, b.out0);
        *reinterpret_cast<uint2*>(s_out + (j0 + 1) * 128 + slot) = make_uint2(a.out1, b.out1);
        s_meta[meta_base + 16 * (2 * wi)] = static_cast<uint8_t>((a.meta_byte & 0xFu) | ((b.meta_byte & 0xFu) << 4));
        s_meta[meta_base + 16 * (2 * wi + 1)] = static_cast<uint8_t>((a.meta_byte >> 4) | (b.meta_byte & 0xF0u));
        if (mask2 != nullptr) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                sel_bits[i] |= (((a.mask_byte >> i) & 1u) << (2 * wi)) | (((a.mask_byte >> (4 + i)) & 1u) << (2 * wi + 1));
                sel_bits[4 + i] |= (((b.mask_byte >> i) & 1u) << (2 * wi)) | (((b.mask_byte >> (4 + i)) & 1u) << (2 * wi + 1));
            }
        }
    }
    if (mask2 != nullptr) {
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const size_t row = static_cast<size_t>(rb) * 128 + ig * 8 + t;
            mask2[row * mrow + cb * 16 + c8] = static_cast<uint8_t>(sel_bits[t] & mb[t]);
        }
    }
    __syncthreads();

    // (W^T) tile (cb, rb): value rows of 128 B (undo the slot swizzle), then the metadata block.
    const size_t vrow_u4 = static_cast<size_t>(d_out) >> 4;        // uint4 per row of valsT (d_out/2 bf16)
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
        const int jr = pass * 32 + (tid >> 3), seg = tid & 7;      // logical slots 2*seg, 2*seg+1
        const int x = (jr >> 3) & 15;
        const uint4 v = *reinterpret_cast<const uint4*>(s_out + jr * 128 + (((2 * seg) ^ x) >> 1) * 16);
        const uint4 o = (x & 1) ? make_uint4(v.z, v.w, v.x, v.y) : v;
        valsT[(static_cast<size_t>(cb) * 128 + jr) * vrow_u4 + rb * 8 + seg] = o;
    }
    if (tid < 128) {
        const size_t blk = static_cast<size_t>(cb) * (d_out >> 7) + rb;
        metaT[blk * 128 + tid] = reinterpret_cast<const uint4*>(s_meta)[tid];
    }
}

// Both passes in one launch.  The second pass of a 128 x 128 tile needs nothing but what the first
// pass makes of that same tile (groups of four rows never straddle a tile), so a CTA reads its tile
// of W once, runs the first pass on it in registers, writes the forward copy, and feeds the masked
// tile straight into the second pass: W is read once instead of twice and the first mask is never
// read back (4.375 bytes per weight element for both compressed copies and both masks instead of
// 6.5).  Thread layout of the second-pass kernel: 8 rows x 8 columns per thread, so a thread's row
// holds exactly two first-pass groups, the pair the packed selection works on.
// Outputs are bit for bit those of prune24_kernel followed by double_prune_kernel.
__global__ void __launch_bounds__(256, 4) prune24_double_kernel(const uint4* __restrict__ W, int d_out, int d_in,
                                                              uint2* __restrict__ vals, uint4* __restrict__ meta,
                                                              uint4* __restrict__ mask1 /* may be null */,
                                                              uint4* __restrict__ valsT, uint4* __restrict__ metaT,
                                                              uint8_t* __restrict__ mask2 /* may be null */) {
    __shared__ __align__(16) uint8_t s_out[128 * 128];       // [column j][16 slots of 8 B], slot index XOR (j >> 3)
    __shared__ __align__(16) uint8_t s_metaT[2048];
    __shared__ __align__(16) uint8_t s_meta[2048];
    __shared__ __align__(16) uint8_t s_mask[2048];           // [row][16 bytes]

    const int cb = blockIdx.x, rb = blockIdx.y;
    const int tid = threadIdx.x;
    const int c8 = tid & 15;                                 // 8-column slot of the tile
    const int ig = tid >> 4;                                 // 8-row slot of the tile
    const size_t row_u4 = static_cast<size_t>(d_in) >> 3;
    const size_t mrow = static_cast<size_t>(d_in) >> 3;      // mask bytes (= uint2 of values) per row
    const size_t at0 = (static_cast<size_t>(rb) * 128 + ig * 8) * row_u4 + cb * 16 + c8;

    uint4 w[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) w[t] = __ldg(W + at0 + t * row_u4);

    // ---- first pass: the two groups of this thread's 8 columns, row by row; W becomes W^R in place
    uint32_t mb[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const PackedPick a = pick2of4_packed(prmt(w[t].x, w[t].z, 0x5410u), prmt(w[t].x, w[t].z, 0x7632u),
                                             prmt(w[t].y, w[t].w, 0x5410u), prmt(w[t].y, w[t].w, 0x7632u));
        const int rr = ig * 8 + t;
        vals[at0 + t * mrow] = make_uint2(a.out0, a.out1);
        s_meta[meta_byte_offset(rr, c8)] = static_cast<uint8_t>(a.meta_byte);
        s_mask[rr * 16 + c8] = static_cast<uint8_t>(a.mask_byte);
        mb[t] = a.mask_byte;
        w[t].x &= prmt(a.keep[0], a.keep[1], 0x5410u);
        w[t].y &= prmt(a.keep[2], a.keep[3], 0x5410u);
        w[t].z &= prmt(a.keep[0], a.keep[1], 0x7632u);
        w[t].w &= prmt(a.keep[2], a.keep[3], 0x7632u);
    }

    // ---- second pass on the masked tile (see double_prune_kernel)
    uint32_t sel_bits[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const int meta_base = meta_byte_offset(c8 * 8, ig);
#pragma unroll
    for (int wi = 0; wi < 4; ++wi) {
        uint32_t e[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) e[t] = wi == 0 ? w[t].x : (wi == 1 ? w[t].y : (wi == 2 ? w[t].z : w[t].w));
        const PackedPick a = pick2of4_packed(e[0], e[1], e[2], e[3]);
        const PackedPick b = pick2of4_packed(e[4], e[5], e[6], e[7]);
        const int j0 = c8 * 8 + 2 * wi;
        const int slot = (ig ^ c8) * 8;
        *reinterpret_cast<uint2*>(s_out + j0 * 128 + slot) = make_uint2(a.out0, b.out0);
        *reinterpret_cast<uint2*>(s_out + (j0 + 1) * 128 + slot) = make_uint2(a.out1, b.out1);
        s_metaT[meta_base + 16 * (2 * wi)] = static_cast<uint8_t>((a.meta_byte & 0xFu) | ((b.meta_byte & 0xFu) << 4));
        s_metaT[meta_base + 16 * (2 * wi + 1)] = static_cast<uint8_t>((a.meta_byte >> 4) | (b.meta_byte & 0xF0u));
        if (mask2 != nullptr) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                sel_bits[i] |= (((a.mask_byte >> i) & 1u) << (2 * wi)) | (((a.mask_byte >> (4 + i)) & 1u) << (2 * wi + 1));
                sel_bits[4 + i] |= (((b.mask_byte >> i) & 1u) << (2 * wi)) | (((b.mask_byte >> (4 + i)) & 1u) << (2 * wi + 1));
            }
        }
    }
    if (mask2 != nullptr) {
#pragma unroll
        for (int t = 0; t < 8; ++t)
            mask2[(static_cast<size_t>(rb) * 128 + ig * 8 + t) * mrow + cb * 16 + c8] =
                static_cast<uint8_t>(sel_bits[t] & mb[t]);
    }
    __syncthreads();

    const size_t vrow_u4 = static_cast<size_t>(d_out) >> 4;        // uint4 per row of valsT (d_out/2 bf16)
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
        const int jr = pass * 32 + (tid >> 3), seg = tid & 7;
        const int x = (jr >> 3) & 15;
        const uint4 v = *reinterpret_cast<const uint4*>(s_out + jr * 128 + (((2 * seg) ^ x) >> 1) * 16);
        const uint4 o = (x & 1) ? make_uint4(v.z, v.w, v.x, v.y) : v;
        valsT[(static_cast<size_t>(cb) * 128 + jr) * vrow_u4 + rb * 8 + seg] = o;
    }
    if (tid < 128) {
        metaT[(static_cast<size_t>(cb) * (d_out >> 7) + rb) * 128 + tid] = reinterpret_cast<const uint4*>(s_metaT)[tid];
        meta[(static_cast<size_t>(rb) * (d_in >> 7) + cb) * 128 + tid] = reinterpret_cast<const uint4*>(s_meta)[tid];
    } else if (mask1 != nullptr) {
        const int rr = tid - 128;
        mask1[(static_cast<size_t>(rb) * 128 + rr) * (d_in >> 7) + cb] = reinterpret_cast<const uint4*>(s_mask)[rr];
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
// `out` may be A or B (every thread reads its vectors before it writes them), hence no __restrict__.
__global__ void __launch_bounds__(256) sparse_add_kernel(const uint4* A, const uint4* B, float beta, float gamma,
                                                         size_t n_vec, uint4* out) {
    for (size_t idx = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; idx < n_vec;
         idx += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const uint4 a = A[idx], b = B[idx];
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
// (128 x 128 elements = 128 x 64 compressed values) feeds tile (cb, rb) of the transposed copy.
// Same orientation trick as the second pruning pass: a thread owns 8 rows x 8 columns of W,
// rebuilt from 8 bytes of compressed values and one first-pass mask byte per row (a pruned entry
// is +0), so a 32-bit word is a pair of adjacent columns; the stored 2-bit codes of the
// transposed copy's metadata say which two rows of every 4-row group go into its slots.  Only the
// output is transposed, through the same XOR-swizzled staging tile.
// Byte-permute selectors that scatter the two kept values of a 4-column group (bytes 0-1 and
// 2-3 of the compressed word; bytes 4-7 of the permute read zero) to their columns: low 16 bits
// for columns 0-1, high 16 bits for columns 2-3.  One entry per 4-bit pattern of the first mask.
__device__ __forceinline__ uint32_t expand_selector(uint32_t nib) {
    uint32_t sel = 0, rank = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const bool kept = (nib >> k) & 1u;
        const uint32_t byte = kept ? 2u * min(rank, 1u) : 4u;
        sel |= (byte | ((byte + 1u) << 4)) << (8 * k);
        rank += kept ? 1u : 0u;
    }
    return sel;
}

// Blocks are persistent (three per SM) and walk over the tiles; the global loads of a block's
// next tile are issued as soon as the registers of the current one have been expanded, so that
// their latency is hidden behind the selection arithmetic instead of by other blocks.
constexpr int kUpdateBlocksPerSm = 3;
__global__ void __launch_bounds__(256, kUpdateBlocksPerSm)
update_transposed_kernel(const uint2* __restrict__ Wc_new, const uint8_t* __restrict__ mask1,
                         const uint4* __restrict__ metaT, int d_out, int d_in, uint4* __restrict__ valsT) {
    __shared__ __align__(16) uint8_t s_out[128 * 128];       // [column j][16 slots of 8 B], slot index XOR (j >> 3)
    __shared__ __align__(16) uint8_t s_meta[2048];
    __shared__ __align__(8) uint2 s_expand[16];              // per 4-bit mask pattern: selectors of columns 0-1 and 2-3

    const int tid = threadIdx.x;
    const int c8 = tid & 15;                                 // 8-column slot of the tile
    const int ig = tid >> 4;                                 // 8-row slot of the tile
    // 32-bit element offsets (the host refuses matrices of 2^35 elements or more): one integer add
    // per load instead of a 64-bit address computation
    const uint32_t row_u2 = static_cast<uint32_t>(d_in) >> 3;   // 8-byte units per compressed row = mask bytes per row
    const uint32_t vrow_u4 = static_cast<uint32_t>(d_out) >> 4; // uint4 per row of valsT (d_out/2 bf16)
    const int ncb = d_in >> 7, nrb = d_out >> 7;
    const int num_tiles = ncb * nrb;

    if (tid < 16) s_expand[tid] = make_uint2(expand_selector(tid), expand_selector(tid) >> 16);

    uint2 cw[8];
    uint32_t mb[8];
    uint4 m = make_uint4(0u, 0u, 0u, 0u);
    auto fetch = [&](int cb, int rb) {
        const uint32_t at = (static_cast<uint32_t>(rb) * 128u + ig * 8u) * row_u2 + cb * 16u + c8;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            cw[t] = __ldg(Wc_new + (at + t * row_u2));
            mb[t] = __ldg(mask1 + (at + t * row_u2));
        }
        if (tid < 128) m = __ldg(metaT + ((static_cast<uint32_t>(cb) * nrb + rb) * 128u + tid));
    };

    // tile = blockIdx.x, blockIdx.x + gridDim.x, ...: (cb, rb) advance without a division per tile
    const int step_rb = static_cast<int>(gridDim.x) / ncb, step_cb = static_cast<int>(gridDim.x) % ncb;
    int tile = blockIdx.x;
    int cb = tile % ncb, rb = tile / ncb;
    if (tile < num_tiles) fetch(cb, rb);
    __syncthreads();                                         // s_expand
    for (; tile < num_tiles; tile += gridDim.x) {
        int cb_next = cb + step_cb, rb_next = rb + step_rb;
        if (cb_next >= ncb) { cb_next -= ncb; ++rb_next; }
        if (tid < 128) {
            // The metadata block goes to shared memory regrouped by reader: the eight code bytes a
            // thread (ig, c8) needs (columns 8 c8 .. 8 c8 + 7 of row slot ig) lie 16 bytes apart in the
            // block, all in one bank for a whole warp; stored as one 8-byte word per thread they are
            // read back in a single conflict-free load.  16-byte unit `tid` of the block holds the
            // codes of column k = tid % 8 of the slots c8 = 2 (tid / 16) + bit 1 of the byte index,
            // ig = 4 (byte index / 4) + 2 ((tid / 8) % 2) + bit 0 of the byte index.
            const uint32_t mw[4] = {m.x, m.y, m.z, m.w};
            const int k = tid & 7, c8_0 = 2 * (tid >> 4), ig_0 = 2 * ((tid >> 3) & 1);
#pragma unroll
            for (int b = 0; b < 16; ++b) {
                const int ig_b = ig_0 + 4 * (b >> 2) + (b & 1), c8_b = c8_0 + ((b >> 1) & 1);
                s_meta[(ig_b * 16 + c8_b) * 8 + k] = static_cast<uint8_t>(mw[b >> 2] >> (8 * (b & 3)));
            }
        }
        uint32_t d[8][4];                                    // 8 rows x 4 column pairs of W^R
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const uint2 s0 = s_expand[mb[t] & 15u], s1 = s_expand[mb[t] >> 4];
            d[t][0] = __byte_perm(cw[t].x, 0u, s0.x);
            d[t][1] = __byte_perm(cw[t].x, 0u, s0.y);
            d[t][2] = __byte_perm(cw[t].y, 0u, s1.x);
            d[t][3] = __byte_perm(cw[t].y, 0u, s1.y);
        }
        if (tile + static_cast<int>(gridDim.x) < num_tiles) fetch(cb_next, rb_next);
        __syncthreads();                                     // s_meta written; s_out no longer read

        const uint2 codes = *reinterpret_cast<const uint2*>(s_meta + (ig * 16 + c8) * 8);   // byte k: column k of the slot
        const int slot = (ig ^ c8) * 8;
#pragma unroll
        for (int wi = 0; wi < 4; ++wi) {
            // A code byte holds four 2-bit row indices: q0, q1 (rows 0..3 -> slots 0, 1) and q2, q3
            // (rows 4..7).  Index q selects bytes 2q, 2q + 1 of the eight bytes of a row quad, i.e.
            // permute selector byte 0x10 + 0x22 q; the selector bytes of four columns are made at once.
            const uint32_t c4 = wi < 2 ? codes.x : codes.y;
            const uint32_t sq0 = (c4 & 0x03030303u) * 0x22u + 0x10101010u;
            const uint32_t sq1 = ((c4 >> 2) & 0x03030303u) * 0x22u + 0x10101010u;
            const uint32_t sq2 = ((c4 >> 4) & 0x03030303u) * 0x22u + 0x10101010u;
            const uint32_t sq3 = ((c4 >> 6) & 0x03030303u) * 0x22u + 0x10101010u;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int k = 2 * wi + half;
                // column k of rows (0,1), (2,3), (4,5), (6,7) as four words, then one byte permute per
                // row group picks rows q0 (low half) and q1 (high half)
                const uint32_t col = half ? 0x7632u : 0x5410u;
                const uint32_t r01 = __byte_perm(d[0][wi], d[1][wi], col), r23 = __byte_perm(d[2][wi], d[3][wi], col);
                const uint32_t r45 = __byte_perm(d[4][wi], d[5][wi], col), r67 = __byte_perm(d[6][wi], d[7][wi], col);
                const uint32_t pick = static_cast<uint32_t>(k & 3) * 0x11u + 0x40u;      // byte k of the first, byte k of the second
                const uint32_t sel_a = __byte_perm(sq0, sq1, pick), sel_b = __byte_perm(sq2, sq3, pick);
                const uint32_t a = __byte_perm(r01, r23, sel_a), b = __byte_perm(r45, r67, sel_b);
                *reinterpret_cast<uint2*>(s_out + (c8 * 8 + k) * 128 + slot) = make_uint2(a, b);
            }
        }
        __syncthreads();

#pragma unroll
        for (int pass = 0; pass < 4; ++pass) {
            const int jr = pass * 32 + (tid >> 3), seg = tid & 7;      // logical slots 2*seg, 2*seg+1
            const int x = (jr >> 3) & 15;
            const uint4 v = *reinterpret_cast<const uint4*>(s_out + jr * 128 + (((2 * seg) ^ x) >> 1) * 16);
            const uint4 o = (x & 1) ? make_uint4(v.z, v.w, v.x, v.y) : v;
            valsT[(static_cast<uint32_t>(cb) * 128u + jr) * vrow_u4 + rb * 8u + seg] = o;
        }
        cb = cb_next;
        rb = rb_next;
    }
}

// Self-test of the bounded wait every pipeline role uses: one warp waits on an mbarrier phase
// that nothing will ever complete.  The wait must give up after `limit_ns`, raise the device
// status to "timeout" and let the kernel return normally.
__global__ void __launch_bounds__(32) wait_timeout_probe_kernel(unsigned long long limit_ns, int* gave_up) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const bool done = mbar_wait(&bar, 0u, &abort_flag, limit_ns);
        *gave_up = done ? 0 : 1;
    }
}

}  // namespace slope
