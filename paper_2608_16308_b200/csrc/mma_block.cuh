// A 16x16 bf16 block times up to eight activation vectors as one small dense contraction on the
// tensor cores (warp-level mma.sync m16n8k16, bf16 in, fp32 accumulate), for the decode kernels
// that hold the block in shared memory: y_v[r] += sum_c A[r][c] * x_v[c].
//   M = vectors (rows of the A operand; 16, of which rows >= the vector count are zero),
//   K = the block's 16 columns, N = the block's 16 rows in two halves of 8 (two MMAs).
// The block is the B operand: a dense column-major tile (tile[c * 16 + r]) is exactly the
// k-major layout that ldmatrix with .trans turns into B fragments.  A Dense-class block's values
// lie like that in the payload already; a mask-compressed block is first expanded into a 512-byte
// tile per warp.  The products of bf16 values are exact in fp32; an x entry that is not listed is
// a zero in the operand, so this path needs finite x (0 * inf is not "no product"): the caller
// falls back to the per-column evaluation when a vector holds a non-finite entry.
#pragma once

#include "internal.cuh"

namespace dbs {

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void *row) {
    const uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(row));
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}

__device__ __forceinline__ void mma_bf16_m16n8k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                  uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Mask-compressed block (16 u16 masks, 16 u8 starts, packed bf16 values; column-major, or
// row-major for the row-major classes) -> dense column-major tile, by a whole warp: two lanes per
// column (row), eight rows (columns) each.
__device__ __forceinline__ void expand_block_bf16(const uint8_t *blk, bool row_major, uint16_t *tile, int lane) {
    const int major = lane >> 1, h = lane & 1;
    const uint32_t m = reinterpret_cast<const uint16_t *>(blk)[major];
    const uint16_t *vals = reinterpret_cast<const uint16_t *>(blk + HDR_BYTES);
    int i = blk[32 + major] + __popc(m & ((1u << (8 * h)) - 1u));
    const uint32_t sub = (m >> (8 * h)) & 0xFFu;
    if (!row_major) {
        uint32_t out[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint32_t lo = 0u, hi = 0u;
            if ((sub >> (2 * q)) & 1u) lo = vals[i++];
            if ((sub >> (2 * q + 1)) & 1u) hi = vals[i++];
            out[q] = lo | (hi << 16);
        }
        *reinterpret_cast<uint4 *>(tile + major * 16 + h * 8) = make_uint4(out[0], out[1], out[2], out[3]);
    } else {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            uint16_t v = 0;
            if ((sub >> q) & 1u) v = vals[i++];
            tile[(8 * h + q) * 16 + major] = v;
        }
    }
}

// One block: tile = dense column-major 16x16 bf16 in shared memory (16-byte aligned); xh = the
// bf16 copy of the vectors' entries of this column block (vector v at xh + v * ldh, 16 entries,
// zeros where not listed).  acc_lo / acc_hi: rows 0..7 / 8..15 of the block; a thread holds, for
// vector lane >> 2, rows 2 * (lane & 3) and + 1 of each half in [0] and [1].
__device__ __forceinline__ void mma_block(const void *tile, const uint16_t *xh, int ldh, int nvec, int lane,
                                          float (&acc_lo)[4], float (&acc_hi)[4]) {
    uint32_t b[4];
    // lane l supplies row (l & 7) of matrix l >> 3; matrices: (k half, n half) = (0,0), (1,0), (0,1), (1,1)
    const int mat = lane >> 3, kh = mat & 1, nh = mat >> 1;
    ldmatrix_x4_trans(b, static_cast<const uint16_t *>(tile) + (kh * 8 + (lane & 7)) * 16 + nh * 8);
    uint32_t a0 = 0u, a2 = 0u;
    const int v = lane >> 2;
    if (v < nvec) {
        const uint32_t *xp = reinterpret_cast<const uint32_t *>(xh + (size_t)v * ldh);
        a0 = xp[lane & 3];
        a2 = xp[4 + (lane & 3)];
    }
    mma_bf16_m16n8k16(acc_lo, a0, 0u, a2, 0u, b[0], b[1]);
    mma_bf16_m16n8k16(acc_hi, a0, 0u, a2, 0u, b[2], b[3]);
}

// The accumulators of a row block -> y (vector v at y + v * ldy), then cleared.
__device__ __forceinline__ void mma_flush(float *y, int64_t ldy, int rb, int nvec, int lane, float (&acc_lo)[4], float (&acc_hi)[4]) {
    const int v = lane >> 2, r = 2 * (lane & 3);
    if (v < nvec) {
        float *row0 = y + (size_t)v * ldy + (size_t)rb * 16;
        if (acc_lo[0] != 0.f) atomicAdd(row0 + r, acc_lo[0]);
        if (acc_lo[1] != 0.f) atomicAdd(row0 + r + 1, acc_lo[1]);
        if (acc_hi[0] != 0.f) atomicAdd(row0 + 8 + r, acc_hi[0]);
        if (acc_hi[1] != 0.f) atomicAdd(row0 + 8 + r + 1, acc_hi[1]);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) { acc_lo[k] = 0.f; acc_hi[k] = 0.f; }
}

}  // namespace dbs
