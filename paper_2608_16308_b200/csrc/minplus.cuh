// The (min, +) semiring for dbspmspv_run: y_i = min_j (A[i][j] + x_j) over the stored A[i][j]
// whose x_j is listed -- the product that GraphBLAS-style systems (Sections 1 and 6) iterate for
// single-source shortest paths; db_sssp below is that iteration.
//
// It runs over the same format, vector blocking, push worklist and compaction as the (+, *)
// product; only the traversal and the writeback differ.  The accumulator keeps, per row, a
// 32-bit KEY of the smallest sum so far instead of a running sum:
//     ordered(v) = bits(v) ^ (v < 0 ? 0xFFFFFFFF : 0x80000000)     (monotone in v)
//     key(v)     = ~ordered(v)                                      (smaller v -> larger key)
// so "take the minimum" is one atomicMax on an unsigned word, its identity is the all-zero
// word -- exactly the cleared state the compaction leaves the accumulator in -- and the first
// sum to reach a row is the one whose atomicMax returns 0 (it sets the row's flag).  The only
// value whose key would be 0 is the NaN 0x7FFFFFFF; NaN has no place in a (min, +) product and
// its key is stored as 1.  The compaction turns the keys back into values.
//
// Traversal.  Push (this file): a warp takes one task of the push worklist, 32 entries of the
// block-CSC view, lane = entry; a lane walks all stored elements of its block that sit in
// listed columns, whatever the block's class.  Pull: on hypersparse valued handles the streaming
// pull kernel runs with the semiring swapped (lean_pull.cuh); the selector is the same
// vector-block ratio as for (+, *).  Pattern handles and handles whose elements sit mostly in
// mask-based blocks always push.
#pragma once

#include "internal.cuh"
#include "worklist.cuh"

namespace dbs {

__device__ __forceinline__ uint32_t minplus_key(float v) {
    const uint32_t b = __float_as_uint(v);
    const uint32_t k = ~(b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u));
    return k ? k : 1u;
}
__device__ __forceinline__ float minplus_value(uint32_t key) {
    const uint32_t o = ~key;
    return __uint_as_float((o >> 31) ? o ^ 0x80000000u : ~o);
}

// Every stored element (r, c, a) of one block whose column c is set in xm, by one lane.
template <int DT, typename F>
__device__ __forceinline__ void block_elements(int type, uint32_t w, uint32_t aux, uint32_t xm, const uint8_t *payload, F f) {
    if (type == DBSPMSPV_BLK_INLINE) {
        if ((xm >> (aux & 15)) & 1u) f((int)(aux >> 4), (int)(aux & 15), Val<DT>::inline_value(w));
        return;
    }
    const uint8_t *blk = payload + (size_t)w * 4;
    if (type == DBSPMSPV_BLK_COO) {
        const int nnz = (int)aux + 1;
        const uint8_t *vals = blk + ((nnz + 3) & ~3);
        for (int k = 0; k < nnz; ++k) {
            const uint32_t rc = blk[k];
            if ((xm >> (rc & 15)) & 1u) f((int)(rc >> 4), (int)(rc & 15), Val<DT>::load(vals, k));
        }
        return;
    }
    constexpr bool HAS_STARTS = Val<DT>::SIZE != 0;       // pattern blocks are the 16 masks alone
    const uint16_t *masks = reinterpret_cast<const uint16_t *>(blk);
    if (is_row_major(type)) {                              // row masks, row-major values
        const uint8_t *vals = blk + HDR_BYTES;
        for (int r = 0; r < 16; ++r) {
            const uint32_t full = masks[r];
            uint32_t act = full & xm;
            if (!act) continue;
            const int base = HAS_STARTS ? blk[32 + r] : 0;
            for (; act; act &= act - 1) {
                const int c = __ffs(act) - 1;
                f(r, c, Val<DT>::load(vals, base + __popc(full & ((1u << c) - 1u))));
            }
        }
        return;
    }
    const bool dense = type == DBSPMSPV_BLK_DENSE;         // column masks, column-major values
    const uint8_t *vals = blk + (dense ? 32 : HDR_BYTES);
    for (uint32_t act = xm; act; act &= act - 1) {
        const int c = __ffs(act) - 1;
        uint32_t cm = masks[c];
        int k = dense ? c * 16 : (HAS_STARTS ? blk[32 + c] : 0);
        for (; cm; cm &= cm - 1) {
            const int r = __ffs(cm) - 1;
            f(r, c, Val<DT>::load(vals, dense ? k + r : k));
            if (!dense) ++k;
        }
    }
}

// One block with a payload taken by a whole warp, (min, +): row r's smallest a + x over the listed
// columns, reduced across the lanes, then `f(r, key)` once per row that has one (lane r calls
// it) -- one atomic per row instead of one per element (the payload blocks of a power-law
// matrix are its hub corner: their rows are the ones whose atomics queue up).  `xb`: the 16 x
// entries of the block's vector block.  A lane owns half a row (row-major classes) or half a
// column (column-major classes, Dense); COO entries are dealt out in turn.
template <int DT, typename F>
__device__ __forceinline__ void block_rows_min_warp(int type, uint32_t w, uint32_t aux, uint32_t xm, const float *xb,
                                                    const uint8_t *payload, int lane, F f) {
    const uint8_t *blk = payload + (size_t)w * 4;
    constexpr uint32_t FULLW = 0xFFFFFFFFu;
    if (type == DBSPMSPV_BLK_COO) {
        // (entries of a row are adjacent but few: one reduction per row present in the block)
        const int nnz = (int)aux + 1;
        const uint8_t *vals = blk + ((nnz + 3) & ~3);
        uint32_t key[2] = {0u, 0u};
        int row[2] = {-1, -1};
#pragma unroll
        for (int u = 0; u < 2; ++u) {               // nnz <= 64 in this class
            const int k = lane + 32 * u;
            if (k < nnz) {
                const uint32_t rc = blk[k];
                if ((xm >> (rc & 15)) & 1u) { row[u] = (int)(rc >> 4); key[u] = minplus_key(Val<DT>::load(vals, k) + xb[rc & 15]); }
            }
        }
        for (int r = 0; r < 16; ++r) {
            const uint32_t mine = max(row[0] == r ? key[0] : 0u, row[1] == r ? key[1] : 0u);
            const uint32_t m = __reduce_max_sync(FULLW, mine);
            if (lane == r && m) f(r, m);
        }
        for (int k = lane + 64; k < nnz; k += 32) {  // (forced-format blocks may be longer: element-wise)
            const uint32_t rc = blk[k];
            if ((xm >> (rc & 15)) & 1u) f((int)(rc >> 4), minplus_key(Val<DT>::load(vals, k) + xb[rc & 15]));
        }
        return;
    }
    constexpr bool HAS_STARTS = Val<DT>::SIZE != 0;
    const uint16_t *masks = reinterpret_cast<const uint16_t *>(blk);
    const int major = lane >> 1, hf = lane & 1;
    const uint32_t full = masks[major];
    if (is_row_major(type)) {
        const uint8_t *vals = blk + HDR_BYTES;
        const int base = HAS_STARTS ? blk[32 + major] : 0;
        uint32_t key = 0u;
        for (uint32_t act = full & xm & (0xFFu << (8 * hf)); act; act &= act - 1) {
            const int c = __ffs(act) - 1;
            key = max(key, minplus_key(Val<DT>::load(vals, base + __popc(full & ((1u << c) - 1u))) + xb[c]));
        }
        key = max(key, __shfl_xor_sync(FULLW, key, 1));
        if (hf == 0 && key) f(major, key);           // lane 2r holds row r
        return;
    }
    const bool dense = type == DBSPMSPV_BLK_DENSE;
    const uint8_t *vals = blk + (dense ? 32 : HDR_BYTES);
    const int base = dense ? major * 16 : (HAS_STARTS ? blk[32 + major] : 0);
    const bool listed = (xm >> major) & 1u;
    const float xc = listed ? xb[major] : 0.f;
#pragma unroll
    for (int r = 0; r < 16; ++r) {
        uint32_t key = 0u;
        if (listed && (r >> 3) == hf && ((full >> r) & 1u))
            key = minplus_key(Val<DT>::load(vals, dense ? base + r : base + __popc(full & ((1u << r) - 1u))) + xc);
        const uint32_t m = __reduce_max_sync(FULLW, key);
        if (lane == r && m) f(r, m);
    }
}

constexpr int MINPLUS_CTA = 256;

__device__ __forceinline__ int select_path(const Device &d, float th3, int force_path);

template <int DT>
__global__ void __launch_bounds__(MINPLUS_CTA, 4) k_minplus_push(Device d, float th3, int force_path) {
    pdl_wait();
    pdl_launch_dependents();
    if (select_path(d, th3, force_path) != DBSPMSPV_PATH_PUSH) return;
    const int lane = threadIdx.x & 31;
    const int gwarp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    Counters *ctr = d.ws.ctr;
    if (blockIdx.x == 0 && threadIdx.x == 0) ctr->path = DBSPMSPV_PATH_PUSH;
    const int n_recs = ctr->n_tasks, n_hubs = min(ctr->n_hubs, HUB_CAP);
    const HubTable hubs = load_hub_table(d.ws.hubs, n_hubs, lane);
    const int n_tasks = n_recs + hubs.total;
    uint32_t *keys = reinterpret_cast<uint32_t *>(d.ws.y_acc);
    for (int t = gwarp; t < n_tasks; t += nwarps) {
        const uint2 task = worklist_item(d.ws.tasks, n_recs, hubs, t);
        const int jb = (int)(task.x & IDX_MASK), cnt = (int)(task.x >> 27) + 1, start = (int)task.y;
        if (lane >= cnt || !DBS_CHK_RANGE(d, start, cnt) || !DBS_CHK_INDEX(d, jb, d.nb)) continue;
        const int p = start + lane;
        uint32_t idx = d.csc.idx[p], w = d.csc.w[p], aux = d.csc.aux[p];
        DBS_CHK_ENTRY(d, false, idx, w, aux);
        const uint32_t xm = mask_of(d.ws.x_mask32, jb);
        const float *xb = d.ws.x_dense + (size_t)jb * 16;
        const size_t row0 = (size_t)(idx & IDX_MASK) * 16;
        block_elements<DT>((int)(idx >> TYPE_SHIFT), w, aux, xm, d.payload, [&](int r, int c, float a) {
            const uint32_t old = atomicMax(keys + row0 + r, minplus_key(a + xb[c]));
            if (old == 0u) d.ws.y_hit8[row0 + r] = 1;
        });
    }
}

}  // namespace dbs
