// Per-block microkernels (Sections 3.3.1 and 3.3.3).  A visited block picks one of these from
// its class and from popc of the local vector-block mask:
//   INLINE / small COO   one lane owns the whole block (hypersparse blocks dominate power-law
//                        matrices, so 32 blocks are processed per warp step)
//   larger COO           one lane per stored entry, shared-memory accumulation
//   ForceCSR             row-driven, two lanes per row (Algorithm 2)
//   CSR (dense mask)     row-driven on the column-major block (row masks rebuilt from the column masks)
//   CSR (sparse mask), ForceCSC   column-driven, half-warps split the columns (Algorithm 3)
//   Dense                column-major values, half-warp per active column (role of Algorithm 4)
// All warp-cooperative kernels leave the partial sum of row (lane & 15) in lanes 0..15 and
// return the 16-bit mask of rows that received a structural product.
#pragma once

#include "internal.cuh"

namespace dbs {

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr int COO_SERIAL_MAX = 32;  // COO blocks up to this many entries are handled by one lane

__device__ __forceinline__ uint32_t below(int k) { return (1u << k) - 1u; }

// Row-driven kernel for row-mask encodings (Algorithm 2): lane = (row, sub-lane); the two
// sub-lanes of a row take alternate active entries; value position = row start + number of
// stored entries left of the column.
template <int DT>
__device__ __forceinline__ float mk_row_pull(const uint8_t *blk, uint32_t xm, const float *s_x,
                                             int lane, uint32_t &hits) {
    const uint16_t *masks = reinterpret_cast<const uint16_t *>(blk);
    const int row = lane >> 1, sub = lane & 1;
    const uint32_t rm = masks[row];
    const int rp = blk[32 + row];
    const uint8_t *vals = blk + HDR_BYTES;
    uint32_t active = rm & xm;
    float sum = 0.f;
    int nz = 0;
    while (active) {
        const int c = __ffs(active) - 1;
        if ((nz & 1) == sub) sum += Val<DT>::load(vals, rp + __popc(rm & below(c))) * s_x[c];
        active &= active - 1;
        ++nz;
    }
    sum += __shfl_xor_sync(FULL, sum, 1);
    hits = __ballot_sync(FULL, lane < 16 && (masks[lane & 15] & xm) != 0);
    return __shfl_sync(FULL, sum, (lane & 15) * 2);
}

// Row-driven kernel for column-mask encodings: the pull-style access of the balanced (CSR)
// class (Section 3.3.3: a relatively dense vector block is reduced by rows).  The block is
// stored column-major so that sparse masks touch few bytes; here every lane first rebuilds the
// mask of its own row from the 16 column masks (staged in shared memory), then walks it like
// Algorithm 2, two lanes per row.  Value position = column start + stored entries above the row.
template <int DT>
__device__ __forceinline__ float mk_col_pull(const uint8_t *blk, uint32_t xm, const float *s_x,
                                             uint32_t *s_hdr, int lane, uint32_t &hits) {
    const uint16_t *masks = reinterpret_cast<const uint16_t *>(blk);
    __syncwarp();
    if (lane < 16) { s_hdr[lane] = masks[lane]; s_hdr[16 + lane] = blk[32 + lane]; }
    __syncwarp();
    const int row = lane >> 1, sub = lane & 1;
    const uint8_t *vals = blk + HDR_BYTES;
    uint32_t rm = 0;
#pragma unroll
    for (int c = 0; c < 16; ++c) rm |= ((s_hdr[c] >> row) & 1u) << c;
    uint32_t active = rm & xm;
    float sum = 0.f;
    int nz = 0;
    while (active) {
        const int c = __ffs(active) - 1;
        if ((nz & 1) == sub) sum += Val<DT>::load(vals, s_hdr[16 + c] + __popc(s_hdr[c] & below(row))) * s_x[c];
        active &= active - 1;
        ++nz;
    }
    sum += __shfl_xor_sync(FULL, sum, 1);
    uint32_t hm = (lane < 16 && ((xm >> lane) & 1u)) ? s_hdr[lane] : 0u;
    hits = __reduce_or_sync(FULL, hm);
    return __shfl_sync(FULL, sum, (lane & 15) * 2);
}

// Column-driven kernel for column-mask encodings (Algorithm 3): lane = row, the two
// half-warps take columns 0..7 and 8..15.
template <int DT>
__device__ __forceinline__ float mk_col_push(const uint8_t *blk, uint32_t xm, const float *s_x,
                                             int lane, uint32_t &hits) {
    const uint16_t *masks = reinterpret_cast<const uint16_t *>(blk);
    const int row = lane & 15, part = lane >> 4;
    const uint8_t *vals = blk + HDR_BYTES;
    uint32_t active = xm & (part ? 0xFF00u : 0x00FFu);
    uint32_t hm = 0;
    float sum = 0.f;
    while (active) {
        const int c = __ffs(active) - 1;
        const uint32_t cm = masks[c];
        hm |= cm;
        if ((cm >> row) & 1u) sum += Val<DT>::load(vals, blk[32 + c] + __popc(cm & below(row))) * s_x[c];
        active &= active - 1;
    }
    sum += __shfl_xor_sync(FULL, sum, 16);
    hits = hm | __shfl_xor_sync(FULL, hm, 16);
    return sum;
}

// Dense class: 16 column masks then 256 values column-major.  Same lane map as Algorithm 3;
// a padding zero never contributes (its mask bit is clear), so hits stay structural.
template <int DT>
__device__ __forceinline__ float mk_dense(const uint8_t *blk, uint32_t xm, const float *s_x,
                                          int lane, uint32_t &hits) {
    const uint16_t *masks = reinterpret_cast<const uint16_t *>(blk);
    const int row = lane & 15, part = lane >> 4;
    const uint8_t *vals = blk + 32;
    uint32_t active = xm & (part ? 0xFF00u : 0x00FFu);
    uint32_t hm = 0;
    float sum = 0.f;
    while (active) {
        const int c = __ffs(active) - 1;
        const uint32_t cm = masks[c];
        hm |= cm;
        if ((cm >> row) & 1u) sum += Val<DT>::load(vals, c * 16 + row) * s_x[c];
        active &= active - 1;
    }
    sum += __shfl_xor_sync(FULL, sum, 16);
    hits = hm | __shfl_xor_sync(FULL, hm, 16);
    return sum;
}

// Larger COO blocks: one lane per stored entry, accumulation in a 16-float shared scratch.
template <int DT>
__device__ __forceinline__ float mk_coo_warp(const uint8_t *blk, int nnz, uint32_t xm,
                                             const float *s_x, float *s_tmp, int lane,
                                             uint32_t &hits) {
    if (lane < 16) s_tmp[lane] = 0.f;
    __syncwarp();
    const uint8_t *vals = blk + ((nnz + 3) & ~3);
    uint32_t hm = 0;
    for (int k = lane; k < nnz; k += 32) {
        const uint32_t rc = blk[k];
        const int c = rc & 15, r = rc >> 4;
        if ((xm >> c) & 1u) {
            atomicAdd(&s_tmp[r], Val<DT>::load(vals, k) * s_x[c]);
            hm |= 1u << r;
        }
    }
    hits = __reduce_or_sync(FULL, hm);
    __syncwarp();
    return s_tmp[lane & 15];
}

// Dispatch of the warp-cooperative kernels: block class x popc(vector-block mask).
template <int DT>
__device__ __forceinline__ float warp_block(int type, const uint8_t *blk, int nnz, uint32_t xm,
                                            const float *s_x, float *s_tmp, int lane,
                                            int popc_threshold, uint32_t &hits) {
    switch (type) {
        case DBSPMSPV_BLK_COO: return mk_coo_warp<DT>(blk, nnz, xm, s_x, s_tmp, lane, hits);
        case DBSPMSPV_BLK_FCSR:
        case BLK_CSR_ROWMAJOR: return mk_row_pull<DT>(blk, xm, s_x, lane, hits);
        case DBSPMSPV_BLK_CSR:   // balanced blocks: the local mask decides (Section 3.3.3)
            return __popc(xm) >= popc_threshold
                       ? mk_col_pull<DT>(blk, xm, s_x, reinterpret_cast<uint32_t *>(s_tmp), lane, hits)
                       : mk_col_push<DT>(blk, xm, s_x, lane, hits);
        case DBSPMSPV_BLK_FCSC: return mk_col_push<DT>(blk, xm, s_x, lane, hits);
        default: return mk_dense<DT>(blk, xm, s_x, lane, hits);
    }
}

// ---- Lane-owned form of the mask-based classes.  When many heavier blocks sit side by side
// (layers of a pruned model, banded matrices) a warp that took them one at a time would wait
// out two dependent memory round trips per block; instead every lane walks its own block and
// the warp keeps 32 blocks in flight.  Products are added into the lane's private column of a
// shared 16 x 33 scratch (`acc` points at it, stride 33 floats: conflict free), so no atomics
// are needed; the caller then folds the column into the row block's result.
constexpr int LANE_ACC_STRIDE = 33;
template <int DT>
__device__ __forceinline__ uint32_t lane_heavy(int type, const uint8_t *blk, uint32_t xm,
                                               const float *xb, float *acc) {
    const uint16_t *masks = reinterpret_cast<const uint16_t *>(blk);
    uint32_t hit = 0;
    if (is_row_major(type)) {                   // row masks, row-major values
        const uint8_t *vals = blk + HDR_BYTES;
        for (int r = 0; r < 16; ++r) {
            const uint32_t full = masks[r];
            uint32_t act = full & xm;
            if (!act) continue;
            const int base = blk[32 + r];
            float s = 0.f;
            for (; act; act &= act - 1) {
                const int c = __ffs(act) - 1;
                s += Val<DT>::load(vals, base + __popc(full & below(c))) * xb[c];
            }
            acc[r * LANE_ACC_STRIDE] += s;
            hit |= 1u << r;
        }
        return hit;
    }
    const bool dense = type == DBSPMSPV_BLK_DENSE;
    const uint8_t *vals = blk + (dense ? 32 : HDR_BYTES);
    for (uint32_t act = xm; act; act &= act - 1) {   // column masks, column-major values
        const int c = __ffs(act) - 1;
        uint32_t cm = masks[c];
        if (!cm) continue;
        hit |= cm;
        const float xc = xb[c];
        int k = dense ? c * 16 : blk[32 + c];
        if (dense) {
            for (; cm; cm &= cm - 1) { const int r = __ffs(cm) - 1; acc[r * LANE_ACC_STRIDE] += Val<DT>::load(vals, k + r) * xc; }
        } else {
            for (; cm; cm &= cm - 1, ++k) { const int r = __ffs(cm) - 1; acc[r * LANE_ACC_STRIDE] += Val<DT>::load(vals, k) * xc; }
        }
    }
    return hit;
}

// ---- Boolean forms (Section 4.2, Algorithm 5): only reachability; values are never read.
// Returns the mask of rows with a stored entry in an active column.
template <int DT>
__device__ __forceinline__ uint32_t warp_block_bool(int type, const uint8_t *blk, int nnz,
                                                    uint32_t xm, int lane) {
    constexpr bool HAS_STARTS = Val<DT>::SIZE != 0;
    (void)HAS_STARTS;
    const uint16_t *masks = reinterpret_cast<const uint16_t *>(blk);
    if (type == DBSPMSPV_BLK_COO) {
        uint32_t hm = 0;
        for (int k = lane; k < nnz; k += 32) {
            const uint32_t rc = blk[k];
            if ((xm >> (rc & 15)) & 1u) hm |= 1u << (rc >> 4);
        }
        return __reduce_or_sync(FULL, hm);
    }
    if (is_row_major(type))
        return __ballot_sync(FULL, lane < 16 && (masks[lane & 15] & xm) != 0);
    // column masks: OR of the active columns' masks
    uint32_t hm = (lane < 16 && ((xm >> lane) & 1u)) ? masks[lane] : 0u;
    return __reduce_or_sync(FULL, hm);
}

// Half-warp streaming form for runs of mask-based blocks: lane = row, and the two half-warps take
// two different blocks, so no cross-lane reduction is needed and a row's sum stays in a register
// while consecutive blocks belong to the same row block.  Lane `row` of a half holds mask, start
// and x entry number `row` of its block in registers.
//   column-major blocks (ForceCSC, CSR, Dense; the lane map of Algorithm 3): the half walks the
//     active columns together; mask and start of a column are broadcast by shuffle and every
//     lane picks its row's element of that column, if any;
//   row-major blocks (ForceCSR, short-row CSR; Algorithm 2 with one lane per row): every lane
//     walks the active entries of its own row; only the x entry comes by shuffle.
// Up to four value loads are issued before their products are added, so several loads per lane
// are in flight (two per round was measured 25 % slower: the walk is latency bound), and the
// header of the next block pair is fetched before the current one is worked on.
// One call takes blocks of one layout (ROWS: row-major), so the loop is specialised at compile
// time and both halves stay converged.
// `emit(rb, row, sum)` is called by a lane when its row block changes and at the end.
template <int DT, bool ROWS, typename Emit>
__device__ __forceinline__ void half_stream(const uint8_t *payload, const float *x_dense, uint32_t idx_l,
                                            uint32_t w_l, uint32_t xm_l, int rb_l, uint32_t todo, int lane,
                                            Emit emit) {
    const int half = lane >> 4, row = lane & 15, hb = half << 4;
    const uint32_t below_row = below(row);
    float sum = 0.f;
    bool touched = false;
    int srb = -1;
    // header of one block for this lane: mask | start << 16, and x entry, number `row`
    auto fetch = [&](uint32_t rem, uint32_t &bxm, int &brb, int &kind, const uint8_t *&vals,
                     uint32_t &hdr, float &xr) -> uint32_t {
        const int l0 = __ffs(rem) - 1;
        rem &= rem - 1;
        int src = l0;
        if (rem) { if (half) src = __ffs(rem) - 1; rem &= rem - 1; }
        else if (half) src = -1;
        const int sl = src >= 0 ? src : l0;
        const uint32_t bidx = __shfl_sync(FULL, idx_l, sl);
        const uint32_t bw = __shfl_sync(FULL, w_l, sl);
        bxm = __shfl_sync(FULL, xm_l, sl);
        brb = __shfl_sync(FULL, rb_l, sl);
        if (src < 0) { bxm = 0u; brb = -1; }
        const uint8_t *blk = payload + (size_t)bw * 4;
        const int type = bidx >> TYPE_SHIFT;
        kind = type == DBSPMSPV_BLK_DENSE ? 2 : (is_row_major(type) ? 1 : 0);   // 0 column-major, 1 row-major, 2 dense
        vals = blk + (kind == 2 ? 32 : HDR_BYTES);
        const uint32_t st = kind == 2 ? row * 16 : (Val<DT>::SIZE ? blk[32 + row] : 0);
        hdr = reinterpret_cast<const uint16_t *>(blk)[row] | (st << 16);
        xr = x_dense[(size_t)(bidx & IDX_MASK) * 16 + row];
        return rem;
    };
    int kind;
    uint32_t bxm, hdr;
    int brb;
    const uint8_t *vals;
    float xr;
    uint32_t rem = fetch(todo, bxm, brb, kind, vals, hdr, xr);
    for (;;) {
        // prefetch the next pair while this one is processed
        int n_kind = 0;
        uint32_t n_bxm = 0, n_hdr = 0, n_rem = 0;
        int n_brb = -1;
        const uint8_t *n_vals = vals;
        float n_xr = 0.f;
        const bool more = rem != 0;
        if (more) n_rem = fetch(rem, n_bxm, n_brb, n_kind, n_vals, n_hdr, n_xr);
        if (bxm && brb != srb) {
            if (touched) emit(srb, row, sum);
            sum = 0.f; touched = false; srb = brb;
        }
        if (ROWS) {
            uint32_t a = hdr & 0xFFFFu & bxm;          // my row's entries under active columns
            while (__any_sync(FULL, a != 0)) {
                float v[4], xc[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool on = a != 0;
                    const int c = on ? __ffs(a) - 1 : 0;
                    a &= a - 1;                           // stays 0 once it is 0
                    const float xs = __shfl_sync(FULL, xr, hb | c);
                    xc[j] = 0.f;
                    v[j] = 0.f;
                    if (on) {
                        xc[j] = xs;
                        v[j] = Val<DT>::load(vals, (hdr >> 16) + __popc(hdr & 0xFFFFu & below(c)));
                        touched = true;
                    }
                }
                sum += (v[0] * xc[0] + v[1] * xc[1]) + (v[2] * xc[2] + v[3] * xc[3]);
            }
        } else {
            const bool dense = kind == 2;
            uint32_t a = bxm;                          // the active columns
            while (__any_sync(FULL, a != 0)) {
                float v[4], xc[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool on = a != 0;
                    const int c = on ? __ffs(a) - 1 : 0;
                    a &= a - 1;
                    const uint32_t hc = __shfl_sync(FULL, hdr, hb | c);
                    const float xs = __shfl_sync(FULL, xr, hb | c);
                    xc[j] = 0.f;                          // (an inactive column's x is the NaN marker)
                    v[j] = 0.f;
                    if (on && ((hc >> row) & 1u)) {
                        xc[j] = xs;
                        v[j] = Val<DT>::load(vals, (hc >> 16) + (dense ? row : __popc(hc & below_row)));
                        touched = true;
                    }
                }
                sum += (v[0] * xc[0] + v[1] * xc[1]) + (v[2] * xc[2] + v[3] * xc[3]);
            }
        }
        if (!more) break;
        rem = n_rem; bxm = n_bxm; brb = n_brb; kind = n_kind; vals = n_vals; hdr = n_hdr; xr = n_xr;
    }
    if (touched) emit(srb, row, sum);
}

// Lane-owned Boolean form: rows of one mask-based block reached from the active columns.  The 16
// masks (the first 32 bytes of every mask-based block, 16-byte aligned) come in with two
// 16-byte loads and are tested in registers without a data-dependent branch.
__device__ __forceinline__ uint32_t lane_heavy_bool(int type, const uint8_t *blk, uint32_t xm) {
    const uint4 *m4 = reinterpret_cast<const uint4 *>(blk);
    const uint4 a = m4[0], b = m4[1];
    const uint32_t wd[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};   // two masks per word
    uint32_t hit = 0;
    if (is_row_major(type)) {
        const uint32_t xx = xm | (xm << 16);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t t = wd[i] & xx;
            hit |= ((t & 0xFFFFu) ? 1u : 0u) << (2 * i);
            hit |= ((t >> 16) ? 1u : 0u) << (2 * i + 1);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t lo = 0u - ((xm >> (2 * i)) & 1u), hi = 0u - ((xm >> (2 * i + 1)) & 1u);
            hit |= (wd[i] & 0xFFFFu & lo) | ((wd[i] >> 16) & hi);
        }
    }
    return hit;
}

constexpr int HEAVY_LANE_MIN = 4;   // this many mask-based blocks in one warp step -> lane-owned form

}  // namespace dbs
