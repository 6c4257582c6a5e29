// Blocked preprocessing (Section 3.2.1): partition A into 16 x 16 blocks, classify each block,
// encode one payload, and build the block-CSR and block-CSC views plus the pull segments
// (Section 3.3.2).  Offline step (Section 5.5): runs on the GPU, may allocate and synchronise.
// Radix sort and prefix sums are CUB library primitives; everything else is written here.
#include <cub/cub.cuh>

#include <algorithm>
#include <new>
#include <vector>

#include "internal.cuh"

namespace dbs {
namespace {

// Device scratch of the build.  A released block is kept and handed out again to a later request
// it fits without much waste (the build's buffers come in a few sizes: one per stored entry, per
// block, per view entry), because cudaMalloc/cudaFree cost more than most of the build's kernels;
// everything goes back to the driver when the build returns, or earlier if an allocation fails.
struct TempPool {
    struct Block { void *p; size_t bytes; bool free; };
    std::vector<Block> blocks;
    ~TempPool() { for (auto &b : blocks) cudaFree(b.p); }
    void trim() {
        size_t k = 0;
        for (auto &b : blocks) { if (b.free) cudaFree(b.p); else blocks[k++] = b; }
        blocks.resize(k);
    }
    template <typename T> bool get(T **out, size_t count) {
        const size_t need = (count ? count : 1) * sizeof(T);
        Block *best = nullptr;
        for (auto &b : blocks)
            if (b.free && b.bytes >= need && b.bytes <= need + need / 2 + 4096 && (!best || b.bytes < best->bytes)) best = &b;
        if (best) { best->free = false; *out = static_cast<T *>(best->p); return true; }
        void *p = nullptr;
        if (cudaMalloc(&p, need) != cudaSuccess) {
            cudaGetLastError();
            trim();
            if (cudaMalloc(&p, need) != cudaSuccess) { *out = nullptr; return false; }
        }
        blocks.push_back({p, need, false});
        *out = static_cast<T *>(p);
        return true;
    }
    // the caller has synchronised the stream that used the block
    void release(void *p) {
        for (auto &b : blocks) if (b.p == p) b.free = true;
    }
};

constexpr int TPB = 256;
inline int grid_for(int64_t n, int tpb = TPB) {
    int64_t g = (n + tpb - 1) / tpb;
    return (int)(g < 1 ? 1 : g);
}

// ---- step 1: one 64-bit key per stored entry: (row block, col block, local row, local col)
__global__ void k_keys_from_csr(int64_t m, int64_t n, int64_t nnz, const int64_t *row_ptr,
                                const int32_t *col_idx, uint64_t *keys, uint32_t *src,
                                int *bad) {
    int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (e == 0 && (row_ptr[0] != 0 || row_ptr[m] != nnz)) *bad = 1;
    if (e >= nnz) return;
    int64_t lo = 0, hi = m;  // largest i with row_ptr[i] <= e
    while (hi - lo > 1) {
        int64_t mid = (lo + hi) >> 1;
        if (row_ptr[mid] <= e) lo = mid; else hi = mid;
    }
    int64_t i = lo;
    if (!(row_ptr[i] <= e && e < row_ptr[i + 1])) { *bad = 1; keys[e] = 0; src[e] = (uint32_t)e; return; }
    int64_t j = col_idx[e];
    if (j < 0 || j >= n) { *bad = 1; j = 0; }
    keys[e] = ((uint64_t)(i >> 4) << 35) | ((uint64_t)(j >> 4) << 8) | ((uint64_t)(i & 15) << 4) | (uint64_t)(j & 15);
    src[e] = (uint32_t)e;
}

__global__ void k_keys_from_coo(int64_t m, int64_t n, int64_t nnz, const int32_t *row,
                                const int32_t *col, uint64_t *keys, uint32_t *src, int *bad) {
    int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (e >= nnz) return;
    int64_t i = row[e], j = col[e];
    if (i < 0 || i >= m || j < 0 || j >= n) { *bad = 1; i = 0; j = 0; }
    keys[e] = ((uint64_t)(i >> 4) << 35) | ((uint64_t)(j >> 4) << 8) | ((uint64_t)(i & 15) << 4) | (uint64_t)(j & 15);
    src[e] = (uint32_t)e;
}

// rows that hold at least one stored element, as 16-bit masks per row block (two per word).
// The keys are sorted by row block, so the lanes of a warp share a few words at most: the bits
// of one word are combined in the warp and set with one atomic.
__global__ void k_row_presence(int64_t nnzu, const uint64_t *ukey, uint32_t *row_present32) {
    int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const bool have = e < nnzu;
    const uint64_t k = have ? ukey[e] : 0;
    const int64_t rb = (int64_t)(k >> 35);
    const uint32_t bit = 1u << (((uint32_t)(k >> 4) & 15u) + (uint32_t)(rb & 1) * 16u);
    const int word = have ? (int)(rb >> 1) : -1;
    const uint32_t peers = __match_any_sync(0xFFFFFFFFu, word);
    const uint32_t bits = __reduce_or_sync(peers, bit);
    if (have && (threadIdx.x & 31) == __ffs(peers) - 1) atomicOr(row_present32 + word, bits);
}

// ---- step 2: merge duplicates, find block boundaries
__global__ void k_flag_new_key(int64_t n, const uint64_t *keys, int shift, int32_t *flag) {
    int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (e >= n) return;
    flag[e] = (e == 0 || (keys[e] >> shift) != (keys[e - 1] >> shift)) ? 1 : 0;
}

template <int DT>
__global__ void k_merge_duplicates(int64_t nnz, const uint64_t *keys, const uint32_t *src,
                                   const int32_t *flag, const int32_t *rank, const void *val,
                                   uint64_t *ukey, void *uval) {
    int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (e >= nnz || !flag[e]) return;
    int64_t u = rank[e] - 1;
    uint64_t k = keys[e];
    ukey[u] = k;
    if (DT == DBSPMSPV_F32) {
        const float *v = static_cast<const float *>(val);
        float s = v[src[e]];
        for (int64_t q = e + 1; q < nnz && keys[q] == k; ++q) s += v[src[q]];
        static_cast<float *>(uval)[u] = s;
    } else if (DT == DBSPMSPV_BF16) {
        const __nv_bfloat16 *v = static_cast<const __nv_bfloat16 *>(val);
        if (e + 1 < nnz && keys[e + 1] == k) {
            float s = __bfloat162float(v[src[e]]);
            for (int64_t q = e + 1; q < nnz && keys[q] == k; ++q) s += __bfloat162float(v[src[q]]);
            static_cast<__nv_bfloat16 *>(uval)[u] = __float2bfloat16_rn(s);
        } else {
            static_cast<__nv_bfloat16 *>(uval)[u] = v[src[e]];
        }
    }
}

__global__ void k_block_starts(int64_t nnzu, const int32_t *flag, const int32_t *rank,
                               int32_t *blk_start, int32_t n_blocks) {
    int64_t u = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (u == 0) blk_start[n_blocks] = (int32_t)nnzu;
    if (u >= nnzu || !flag[u]) return;
    blk_start[rank[u] - 1] = (int32_t)u;
}

// ---- step 3: classify (Section 3.2.1) and size every block.  A warp takes 32 consecutive
// blocks, one per lane: below th0 stored elements (most blocks of a hypersparse matrix) the
// class follows from the count alone; the blocks that need their row and column occupancy are
// then walked one after the other by the whole warp.
struct ClassifyParams {
    int th0, th1;
    float th2;
    int force_format;
    int dtype;
    int inline_max;   // blocks with at most this many entries are stored inline
};

__global__ void k_classify(int32_t n_blocks, const int32_t *blk_start, const uint64_t *ukey,
                           ClassifyParams cp, uint8_t *type_out, uint32_t *size_out,
                           int32_t *ecount, int32_t *brow, int32_t *bcol, unsigned long long *class_blocks,
                           unsigned long long *class_nnz) {
    __shared__ uint32_t s_row[TPB / 32][16], s_col[TPB / 32][16];
    __shared__ unsigned int s_cb[DBSPMSPV_BLK_NCLASS], s_cn[DBSPMSPV_BLK_NCLASS];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x < DBSPMSPV_BLK_NCLASS) { s_cb[threadIdx.x] = 0; s_cn[threadIdx.x] = 0; }
    __syncthreads();
    const int64_t b = (blockIdx.x * (int64_t)(TPB / 32) + warp) * 32 + lane;
    const bool have = b < n_blocks;
    const int s = have ? blk_start[b] : 0, nnz = have ? blk_start[b + 1] - s : 0;
    const bool by_shape = have && cp.force_format == DBSPMSPV_FORMAT_AUTO && nnz >= cp.th0 && nnz <= cp.th1;
    int rmax = 0, cmax = 0;   // largest row / column count of this lane's block
    for (uint32_t todo = __ballot_sync(0xFFFFFFFFu, by_shape); todo; todo &= todo - 1) {
        const int src = __ffs(todo) - 1;
        const int ss = __shfl_sync(0xFFFFFFFFu, s, src), nn = __shfl_sync(0xFFFFFFFFu, nnz, src);
        if (lane < 16) { s_row[warp][lane] = 0; s_col[warp][lane] = 0; }
        __syncwarp();
        for (int k = lane; k < nn; k += 32) {
            uint32_t rc = (uint32_t)(ukey[ss + k] & 0xFF);
            atomicOr(&s_row[warp][rc >> 4], 1u << (rc & 15));
            atomicOr(&s_col[warp][rc & 15], 1u << (rc >> 4));
        }
        __syncwarp();
        int rcount = lane < 16 ? __popc(s_row[warp][lane]) : 0;
        int ccount = lane < 16 ? __popc(s_col[warp][lane]) : 0;
        __syncwarp();
        rcount = __reduce_max_sync(0xFFFFFFFFu, rcount);
        ccount = __reduce_max_sync(0xFFFFFFFFu, ccount);
        if (lane == src) { rmax = rcount; cmax = ccount; }
    }
    int type = -1;
    if (have) {
        if (cp.force_format == DBSPMSPV_FORMAT_COO) type = DBSPMSPV_BLK_COO;
        else if (cp.force_format == DBSPMSPV_FORMAT_CSR) type = DBSPMSPV_BLK_CSR;
        else if (nnz < cp.th0) {
            // one view entry per stored element, up to inline_max of them
            type = nnz <= cp.inline_max ? DBSPMSPV_BLK_INLINE : DBSPMSPV_BLK_COO;
        } else if (nnz > cp.th1) type = DBSPMSPV_BLK_DENSE;
        // skew_c / skew_r = (max column count) / (max row count): the denominators of
        // the two axis skews are identical for square blocks
        else if ((float)cmax > cp.th2 * (float)rmax) type = DBSPMSPV_BLK_FCSC;
        else if ((float)rmax > cp.th2 * (float)cmax) type = DBSPMSPV_BLK_FCSR;
        else type = rmax <= CSR_SHORT_ROW ? BLK_CSR_ROWMAJOR : DBSPMSPV_BLK_CSR;
        const int vsize = cp.dtype == DBSPMSPV_F32 ? 4 : cp.dtype == DBSPMSPV_BF16 ? 2 : 0;
        type_out[b] = (uint8_t)type;
        size_out[b] = (uint32_t)payload_words(type, nnz, vsize);
        ecount[b] = type == DBSPMSPV_BLK_INLINE ? nnz : 1;
        const uint64_t k0 = ukey[s];
        brow[b] = (int32_t)(k0 >> 35);
        bcol[b] = (int32_t)((k0 >> 8) & IDX_MASK);
    }
    const int cls = have ? public_class(type) : -1;
    for (int c = 0; c < DBSPMSPV_BLK_NCLASS; ++c) {
        const uint32_t mine = __ballot_sync(0xFFFFFFFFu, cls == c);
        if (!mine) continue;
        const unsigned total = __reduce_add_sync(0xFFFFFFFFu, cls == c ? (unsigned)nnz : 0u);
        if (lane == 0) { atomicAdd(&s_cb[c], (unsigned)__popc(mine)); atomicAdd(&s_cn[c], total); }
    }
    __syncthreads();
    if (threadIdx.x < DBSPMSPV_BLK_NCLASS && s_cb[threadIdx.x]) {
        atomicAdd(&class_blocks[threadIdx.x], (unsigned long long)s_cb[threadIdx.x]);
        atomicAdd(&class_nnz[threadIdx.x], (unsigned long long)s_cn[threadIdx.x]);
    }
}

template <int DT>
__device__ __forceinline__ void store_value(uint8_t *vals, int pos, const void *uval, int64_t u) {
    if (DT == DBSPMSPV_F32) reinterpret_cast<float *>(vals)[pos] = static_cast<const float *>(uval)[u];
    else if (DT == DBSPMSPV_BF16) reinterpret_cast<uint16_t *>(vals)[pos] = static_cast<const uint16_t *>(uval)[u];
}

// INLINE blocks: one view entry per stored element (value in w, unused for pattern matrices;
// packed coordinate in aux).  One thread per stored element; block_of[u] is 1 + its block.
template <int DT>
__global__ void k_encode_inline(int64_t nnzu, const int32_t *block_of, const int32_t *blk_start,
                                const uint64_t *ukey, const void *uval, const uint8_t *type_in,
                                const int32_t *eoff, const int32_t *brow, const int32_t *bcol,
                                uint32_t *v_idx, uint32_t *v_w, uint8_t *v_aux, int32_t *entry_row) {
    const int64_t u = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (u >= nnzu) return;
    const int32_t b = block_of[u] - 1;
    if (type_in[b] != DBSPMSPV_BLK_INLINE) return;
    const int32_t e = eoff[b] + (int32_t)(u - blk_start[b]);
    v_idx[e] = (uint32_t)bcol[b] | ((uint32_t)DBSPMSPV_BLK_INLINE << TYPE_SHIFT);
    v_w[e] = DT == DBSPMSPV_F32    ? __float_as_uint(static_cast<const float *>(uval)[u])
             : DT == DBSPMSPV_BF16 ? (uint32_t) static_cast<const uint16_t *>(uval)[u]
                                   : 0u;
    v_aux[e] = (uint8_t)(ukey[u] & 0xFF);
    entry_row[e] = brow[b];
}

// One block with a payload, by a whole warp.
template <int DT>
__device__ __forceinline__ void encode_block(int32_t b, int s, int nnz, int type, const uint64_t *ukey,
                                             const void *uval, const uint64_t *poff, const int32_t *eoff,
                                             const int32_t *brow, const int32_t *bcol, uint8_t *payload,
                                             uint32_t *v_idx, uint32_t *v_w, uint8_t *v_aux, int32_t *entry_row,
                                             uint32_t *s_row, uint32_t *s_col, uint8_t *s_start, int lane) {
    constexpr int V = Val<DT>::SIZE;
    const uint64_t off_words = poff[b];
    uint8_t *base = payload + off_words * 4;
    const int e0 = eoff[b];
    const uint32_t tagged = (uint32_t)bcol[b] | ((uint32_t)type << TYPE_SHIFT);
    if (lane == 0) {
        v_idx[e0] = tagged;
        entry_row[e0] = brow[b];
        v_w[e0] = (uint32_t)off_words;
        v_aux[e0] = (uint8_t)(nnz - 1);
    }
    if (type == DBSPMSPV_BLK_COO) {
        uint8_t *vals = base + ((nnz + 3) & ~3);
        for (int k = lane; k < ((nnz + 3) & ~3); k += 32)
            base[k] = k < nnz ? (uint8_t)(ukey[s + k] & 0xFF) : 0;
        for (int k = lane; k < nnz; k += 32) store_value<DT>(vals, k, uval, s + k);
        if (DT == DBSPMSPV_BF16 && (nnz & 1) && lane == 0) reinterpret_cast<uint16_t *>(vals)[nnz] = 0;
        return;
    }
    // mask-based classes
    if (lane < 16) { s_row[lane] = 0; s_col[lane] = 0; }
    __syncwarp();
    for (int k = lane; k < nnz; k += 32) {
        uint32_t rc = (uint32_t)(ukey[s + k] & 0xFF);
        atomicOr(&s_row[rc >> 4], 1u << (rc & 15));
        atomicOr(&s_col[rc & 15], 1u << (rc >> 4));
    }
    __syncwarp();
    const bool row_major = is_row_major(type);
    uint32_t mine = lane < 16 ? (row_major ? s_row[lane] : s_col[lane]) : 0;
    int start = __popc(mine);  // exclusive prefix over lanes 0..15
    for (int o = 1; o < 16; o <<= 1) {
        int t = __shfl_up_sync(0xFFFFFFFFu, start, o);
        if (lane >= o) start += t;
    }
    start -= __popc(mine);
    uint16_t *masks = reinterpret_cast<uint16_t *>(base);
    if (lane < 16) masks[lane] = (uint16_t)mine;
    if (type == DBSPMSPV_BLK_DENSE) {
        if (V) {
            uint8_t *vals = base + 32;
            uint32_t *z = reinterpret_cast<uint32_t *>(vals);
            for (int k = lane; k < 256 * V / 4; k += 32) z[k] = 0;
            __syncwarp();
            for (int k = lane; k < nnz; k += 32) {
                uint32_t rc = (uint32_t)(ukey[s + k] & 0xFF);
                store_value<DT>(vals, (rc & 15) * 16 + (rc >> 4), uval, s + k);
            }
        }
        return;
    }
    if (!V) return;  // pattern: masks only
    if (lane < 16) base[32 + lane] = (uint8_t)start;
    uint8_t *vals = base + HDR_BYTES;
    if (row_major) {
        for (int k = lane; k < nnz; k += 32) store_value<DT>(vals, k, uval, s + k);
    } else {
        // column-major position of (r, c): start of column c + entries of c above row r
        if (lane < 16) s_start[lane] = (uint8_t)start;
        __syncwarp();
        for (int k = lane; k < nnz; k += 32) {
            uint32_t rc = (uint32_t)(ukey[s + k] & 0xFF);
            int r = rc >> 4, c = rc & 15;
            int pos = s_start[c] + __popc(s_col[c] & ((1u << r) - 1));
            store_value<DT>(vals, pos, uval, s + k);
        }
    }
    if (DT == DBSPMSPV_BF16 && (nnz & 1) && lane == 0) reinterpret_cast<uint16_t *>(vals)[nnz] = 0;
}

// ---- step 4: encode payload + primary (block-CSR) view entries.  A warp takes 32 consecutive
// blocks and encodes those with a payload one after the other (the INLINE ones are written
// by k_encode_inline).
template <int DT>
__global__ void k_encode(int32_t n_blocks, const int32_t *blk_start, const uint64_t *ukey,
                         const void *uval, const uint8_t *type_in, const uint64_t *poff,
                         const int32_t *eoff, const int32_t *brow, const int32_t *bcol,
                         uint8_t *payload, uint32_t *v_idx, uint32_t *v_w, uint8_t *v_aux,
                         int32_t *entry_row) {
    __shared__ uint32_t s_row[TPB / 32][16], s_col[TPB / 32][16];
    __shared__ uint8_t s_start[TPB / 32][16];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t b = (blockIdx.x * (int64_t)(TPB / 32) + warp) * 32 + lane;
    const bool have = b < n_blocks;
    const int s = have ? blk_start[b] : 0, nnz = have ? blk_start[b + 1] - s : 0;
    const int type = have ? type_in[b] : DBSPMSPV_BLK_INLINE;
    for (uint32_t todo = __ballot_sync(0xFFFFFFFFu, type != DBSPMSPV_BLK_INLINE); todo; todo &= todo - 1) {
        const int src = __ffs(todo) - 1;
        __syncwarp();   // the previous block's use of the shared masks is over
        encode_block<DT>((int32_t)(b - lane + src), __shfl_sync(0xFFFFFFFFu, s, src), __shfl_sync(0xFFFFFFFFu, nnz, src),
                         __shfl_sync(0xFFFFFFFFu, type, src), ukey, uval, poff, eoff, brow, bcol, payload,
                         v_idx, v_w, v_aux, entry_row, s_row[warp], s_col[warp], s_start[warp], lane);
    }
}

// Sort key of the block-CSR view: row block (27 bits) | group (5 bits: 0 = entry with a payload,
// 16 + r = INLINE element of local row r) | column block (27 bits) | local column (4 bits).
// Inside a row block the entries with a payload come first (by column block), then the INLINE
// elements row by row (by column): the mirror image of the block-CSC order.  The elements of a
// row are then adjacent, which turns the pull over a hypersparse matrix into a segmented sum.
constexpr int CSR_KEY_GROUP_SHIFT = 31, CSR_KEY_ROW_SHIFT = 36;
__global__ void k_csr_keys(int32_t n_entries, const int32_t *entry_row, const uint32_t *idx,
                           const uint8_t *aux, uint64_t *keys, int32_t *ids) {
    int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (b >= n_entries) return;
    const uint32_t v = idx[b];
    const bool inl = (v >> TYPE_SHIFT) == DBSPMSPV_BLK_INLINE;
    const uint32_t rc = aux[b];
    const uint64_t group = inl ? 16u + (rc >> 4) : 0u, c = inl ? rc & 15u : 0u;
    keys[b] = ((uint64_t)entry_row[b] << CSR_KEY_ROW_SHIFT) | (group << CSR_KEY_GROUP_SHIFT) |
              ((uint64_t)(v & IDX_MASK) << 4) | c;
    ids[b] = (int32_t)b;
}

// Moves the entries into their final order; the first INLINE element of every row gets ROW_FLAG.
__global__ void k_csr_gather(int32_t n_entries, const uint64_t *keys_sorted, const int32_t *ids,
                             const uint32_t *t_idx, const uint32_t *t_w, const uint8_t *t_aux,
                             uint32_t *idx, uint32_t *w, uint8_t *aux, int32_t *entry_row) {
    int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (p >= n_entries) return;
    const int32_t b = ids[p];
    const uint64_t k = keys_sorted[p];
    const bool inl = ((k >> CSR_KEY_GROUP_SHIFT) & 31u) >= 16u;
    const bool head = inl && (p == 0 || (keys_sorted[p - 1] >> CSR_KEY_GROUP_SHIFT) != (k >> CSR_KEY_GROUP_SHIFT));
    idx[p] = t_idx[b] | (head ? ROW_FLAG : 0u);
    w[p] = t_w[b];
    aux[p] = t_aux[b];
    entry_row[p] = (int32_t)(k >> CSR_KEY_ROW_SHIFT);
}

// inl[rb], rb = 0..mb: first position whose (row block, group) is >= (rb, 16): the end of row
// block rb's payload run and the start of its INLINE elements (inl[mb] = n_entries)
__global__ void k_csr_inl(int32_t mb, const uint64_t *keys_sorted, int32_t n, int32_t *inl) {
    int64_t rb = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (rb > mb) return;
    const uint64_t target = ((uint64_t)rb << 5) + 16u;
    int32_t lo = 0, hi = n;
    while (lo < hi) {
        int32_t mid = lo + ((hi - lo) >> 1);
        if ((keys_sorted[mid] >> CSR_KEY_GROUP_SHIFT) < target) lo = mid + 1; else hi = mid;
    }
    inl[rb] = lo;
}

// Payload chunks of the staged decode: one thread per row block walks its entries with a payload
// ([ptr[rb], inl[rb]), contiguous in the payload) and cuts them greedily into chunks of at most
// cap_entries entries and cap_bytes bytes.  out == nullptr: count only.
__global__ void k_stage_chunks(int32_t mb, const int32_t *ptr, const int32_t *inl, const uint32_t *idx, const uint32_t *w,
                               const uint8_t *aux, int vsize, int cap_entries, int cap_bytes, int32_t *count,
                               const int32_t *first, int4 *out) {
    const int rb = blockIdx.x * blockDim.x + threadIdx.x;
    if (rb >= mb) return;
    int n = 0, e0 = ptr[rb], words = 0;
    const int end = inl[rb];
    int4 *o = out ? out + first[rb] : nullptr;
    for (int p = e0; p < end; ++p) {
        const int sz = payload_words((int)(idx[p] >> TYPE_SHIFT), (int)aux[p] + 1, vsize);
        if (p > e0 && (p - e0 >= cap_entries || (words + sz) * 4 > cap_bytes)) {
            if (o) o[n] = make_int4(e0, rb, (int)w[e0], words | ((p - e0) << 24));
            ++n; e0 = p; words = 0;
        }
        words += sz;
    }
    if (end > e0) { if (o) o[n] = make_int4(e0, rb, (int)w[e0], words | ((end - e0) << 24)); ++n; }
    if (!out) count[rb] = n;
}

// Row list of the streaming pull: flag[p] = 1 at the first INLINE element of a row;
// rows[rank[p]] = that row; chunk_ord[c] = row heads before entry c * LEAN_CHUNK.
__global__ void k_lean_flags(int32_t n_entries, const uint32_t *idx, int32_t *flag) {
    int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (p <= n_entries) flag[p] = (p < n_entries && (idx[p] & ROW_FLAG)) ? 1 : 0;
}
__global__ void k_lean_rows(int32_t n_entries, const uint32_t *idx, const uint8_t *aux, const int32_t *entry_row,
                            const int32_t *rank, int32_t *rows, int32_t n_chunks, int32_t *chunk_ord) {
    int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (p < n_entries && (idx[p] & ROW_FLAG)) rows[rank[p]] = entry_row[p] * 16 + (int32_t)(aux[p] >> 4);
    if (p <= n_chunks) {
        const int64_t e = p * (int64_t)LEAN_CHUNK;
        chunk_ord[p] = rank[e < n_entries ? e : n_entries];
    }
}

__global__ void k_fill_words(uint32_t *p, int64_t n, uint32_t v) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) p[i] = v;
}

// first position p in a sorted int array with a[p] >= v, for v = 0..count (pointer arrays)
__global__ void k_lower_bounds(int32_t count, const int32_t *sorted, int32_t n, int32_t *ptr) {
    int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (v > count) return;
    int32_t lo = 0, hi = n;
    while (lo < hi) {
        int32_t mid = lo + ((hi - lo) >> 1);
        if (sorted[mid] < v) lo = mid + 1; else hi = mid;
    }
    ptr[v] = lo;
}

// Sort key of the block-CSC view: column block (27 bits) | group (5 bits: 0 = entry with a
// payload, 16 + c = INLINE element of local column c) | row block (27 bits) | local row (4 bits).
constexpr int CSC_KEY_GROUP_SHIFT = 31, CSC_KEY_COL_SHIFT = 36;
__global__ void k_csc_keys(int32_t n_entries, const int32_t *entry_row, const uint32_t *csr_idx,
                           const uint8_t *csr_aux, uint64_t *keys, int32_t *ids) {
    int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (b >= n_entries) return;
    const uint32_t idx = csr_idx[b];
    const bool inl = (idx >> TYPE_SHIFT) == DBSPMSPV_BLK_INLINE;
    const uint32_t rc = csr_aux[b];
    const uint64_t group = inl ? 16u + (rc & 15u) : 0u, r = inl ? rc >> 4 : 0u;
    keys[b] = ((uint64_t)(idx & IDX_MASK) << CSC_KEY_COL_SHIFT) | (group << CSC_KEY_GROUP_SHIFT) |
              ((uint64_t)entry_row[b] << 4) | r;
    ids[b] = (int32_t)b;
}

// colptr[17 * jb + k], k = 0..16: first position whose (column block, group) is >= (jb, 16 + k)
__global__ void k_csc_colptr(int32_t nb, const uint64_t *keys_sorted, int32_t n, int32_t *colptr) {
    int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (t >= (int64_t)nb * 17) return;
    const uint64_t target = ((uint64_t)(t / 17) << 5) + (uint64_t)(16 + t % 17);   // k = 16: the next column block
    int32_t lo = 0, hi = n;
    while (lo < hi) {
        int32_t mid = lo + ((hi - lo) >> 1);
        if ((keys_sorted[mid] >> CSC_KEY_GROUP_SHIFT) < target) lo = mid + 1; else hi = mid;
    }
    colptr[t] = lo;
}

__global__ void k_csc_gather(int32_t n_blocks, const uint64_t *keys_sorted,
                             const int32_t *csc2csr, const uint32_t *csr_idx,
                             const uint32_t *csr_w, const uint8_t *csr_aux, uint32_t *csc_idx,
                             uint32_t *csc_w, uint8_t *csc_aux, int32_t *bcol_sorted, const uint16_t *hub_slot) {
    int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (p >= n_blocks) return;
    int32_t b = csc2csr[p];
    uint64_t k = keys_sorted[p];
    const uint32_t rb = (uint32_t)((k >> 4) & IDX_MASK), cls = csr_idx[b] & (7u << TYPE_SHIFT);   // class, without the CSR view's flags
    const bool hub = hub_slot && (cls >> TYPE_SHIFT) == DBSPMSPV_BLK_INLINE && hub_slot[rb] != HUB_NONE;
    csc_idx[p] = rb | cls | (hub ? HUB_FLAG : 0u);
    csc_w[p] = csr_w[b];
    csc_aux[p] = csr_aux[b];
    bcol_sorted[p] = (int32_t)(k >> CSC_KEY_COL_SHIFT);
}

// ---- row-run index of the INLINE elements (DB-BFS pull levels)
__global__ void k_rowrun_keys(int32_t n_entries, int64_t m, const int32_t *entry_row, const uint32_t *csr_idx,
                              const uint8_t *csr_aux, uint64_t *keys, uint32_t *vals) {
    int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (p >= n_entries) return;
    const uint32_t idx = csr_idx[p], rc = csr_aux[p];
    const bool inl = (idx >> TYPE_SHIFT) == DBSPMSPV_BLK_INLINE;
    const uint64_t row = inl ? (uint64_t)entry_row[p] * 16 + (rc >> 4) : (uint64_t)m;   // others sort behind every row
    const uint64_t col = inl ? (uint64_t)(idx & IDX_MASK) * 16 + (rc & 15u) : 0u;
    keys[p] = (row << 31) | col;
    vals[p] = (idx & IDX_MASK) | ((rc & 15u) << 27);
}

// ptr[i] = first position whose row is >= i, i = 0..m
__global__ void k_rowrun_ptr(int64_t m, const uint64_t *keys_sorted, int32_t n, int32_t *ptr) {
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i > m) return;
    int32_t lo = 0, hi = n;
    while (lo < hi) {
        int32_t mid = lo + ((hi - lo) >> 1);
        if ((keys_sorted[mid] >> 31) < (uint64_t)i) lo = mid + 1; else hi = mid;
    }
    ptr[i] = lo;
}

__global__ void k_payload_flags(int32_t n_entries, const uint32_t *idx, int32_t *flag) {
    int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (p <= n_entries) flag[p] = (p < n_entries && (idx[p] >> TYPE_SHIFT) != DBSPMSPV_BLK_INLINE) ? 1 : 0;
}
__global__ void k_payload_list(int32_t n_entries, const int32_t *is_payload, const int32_t *rank, int32_t *payload_pos) {
    int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (p < n_entries && is_payload[p]) payload_pos[rank[p]] = (int32_t)p;
}

// ---- pull segments (Section 3.3.2): greedy walk along each row block; a segment closes
// when its accumulated weight reaches the cut.  One warp per stretch of a row block (hub row
// blocks hold 10^5 entries: a single thread walking them took tens of milliseconds, a single
// warp milliseconds), two passes.  The warp takes 32 entries per step: a scan of their weights, then the cuts inside the step one after
// the other (each restarts the running weight at zero).
struct SegParams { int cut, w_dense, w_mid, w_coo, w_inline; };

__device__ __forceinline__ int seg_weight(uint32_t idx, const SegParams &sp) {
    int t = idx >> TYPE_SHIFT;
    return t == DBSPMSPV_BLK_DENSE ? sp.w_dense : t == DBSPMSPV_BLK_INLINE ? sp.w_inline : t == DBSPMSPV_BLK_COO ? sp.w_coo : sp.w_mid;
}

// Calls close(first, end_exclusive, weight) -- by every lane, with warp-uniform arguments --
// for each segment of row block rb, in order.
template <typename Close>
__device__ __forceinline__ void seg_walk(int begin, int end, const uint32_t *idx, const SegParams &sp, int lane, Close close) {
    int acc = 0, first = begin;
    for (int base = begin; base < end; base += 32) {
        const int p = base + lane;
        const int w = p < end ? seg_weight(idx[p], sp) : 0;
        int incl = w;
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        int removed = 0;      // weight of this step already closed into segments
        for (;;) {
            const uint32_t m = __ballot_sync(0xFFFFFFFFu, p < end && incl > removed && acc + incl - removed >= sp.cut);
            if (!m) break;
            const int l = __ffs(m) - 1;
            const int upto = __shfl_sync(0xFFFFFFFFu, incl, l);
            close(first, base + l + 1, acc + upto - removed);
            first = base + l + 1;
            removed = upto;
            acc = 0;
        }
        acc += __shfl_sync(0xFFFFFFFFu, incl, 31) - removed;
    }
    if (first < end) close(first, end, acc);
}

// A warp walks one stretch of at most SEG_STRETCH entries of a row block, so that the hub row
// blocks of a power-law matrix are cut by many warps at once; the walk starts afresh at a
// stretch boundary (no segment spans one).
constexpr int SEG_STRETCH = 8192;

__global__ void k_seg_units(int32_t mb, const int32_t *row_ptr, int32_t *units) {
    const int64_t rb = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (rb > mb) return;
    units[rb] = rb < mb ? (row_ptr[rb + 1] - row_ptr[rb] + SEG_STRETCH - 1) / SEG_STRETCH : 0;
}

struct Stretch { int32_t rb, begin, end; };
__device__ __forceinline__ Stretch stretch_of(int32_t u, int32_t mb, const int32_t *unit_off, const int32_t *row_ptr) {
    int32_t lo = 0, hi = mb;   // last row block whose first unit is <= u
    while (hi - lo > 1) {
        const int32_t mid = lo + ((hi - lo) >> 1);
        if (unit_off[mid] <= u) lo = mid; else hi = mid;
    }
    Stretch s;
    s.rb = lo;
    s.begin = row_ptr[lo] + (u - unit_off[lo]) * SEG_STRETCH;
    s.end = min(row_ptr[lo + 1], s.begin + SEG_STRETCH);
    return s;
}

__global__ void k_seg_count(int32_t n_units, int32_t mb, const int32_t *unit_off, const int32_t *row_ptr,
                            const uint32_t *idx, SegParams sp, int32_t *count) {
    const int64_t u = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (u >= n_units) return;
    const Stretch s = stretch_of((int32_t)u, mb, unit_off, row_ptr);
    int c = 0;
    seg_walk(s.begin, s.end, idx, sp, lane, [&](int, int, int) { ++c; });
    if (lane == 0) count[u] = c;
}

__global__ void k_seg_write(int32_t n_units, int32_t mb, const int32_t *unit_off, const int32_t *row_ptr,
                            uint32_t *idx, SegParams sp, const int32_t *seg_off, Segment *segs, int32_t *seg_rb) {
    const int64_t u = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (u >= n_units) return;
    const Stretch st = stretch_of((int32_t)u, mb, unit_off, row_ptr);
    const int begin = row_ptr[st.rb], end = row_ptr[st.rb + 1];
    int o = seg_off[u];
    seg_walk(st.begin, st.end, idx, sp, lane, [&](int first, int stop, int weight) {
        if (lane == 0) {
            Segment s;
            s.row_block = st.rb;
            s.start = first;
            s.count = (stop - first) | ((first == begin && stop == end) ? (int32_t)0x80000000 : 0);
            s.weight = weight;
            seg_rb[o] = st.rb;
            segs[o] = s;
            idx[first] |= 1u << 28;   // first entry of a segment (bits 27, 28 of idx are spare)
        }
        ++o;
    });
}

// pull chunks: consecutive segments grouped by accumulated weight; chunk k starts at the first
// segment whose exclusive weight prefix is >= k * PULL_CH
__global__ void k_seg_weights(int32_t n_segments, const Segment *segs, int32_t *w) {
    int64_t k = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (k < n_segments) w[k] = segs[k].weight;
    if (k == n_segments) w[k] = 0;
}

__global__ void k_chunks(int32_t n_chunks, const Segment *segs, const int32_t *wprefix, int32_t n_segments,
                         int32_t n_entries, int2 *chunks) {
    int64_t k = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (k > n_chunks) return;
    if (k == n_chunks) { chunks[k] = make_int2(n_segments, n_entries); return; }
    const int64_t target = k * (int64_t)PULL_CH;
    int32_t lo = 0, hi = n_segments;
    while (lo < hi) {
        int32_t mid = lo + ((hi - lo) >> 1);
        if (wprefix[mid] < target) lo = mid + 1; else hi = mid;
    }
    chunks[k] = make_int2(lo, lo < n_segments ? segs[lo].start : n_entries);
}

template <typename T>
int exclusive_sum(TempPool &tp, const T *in, T *out, int64_t n, cudaStream_t st) {
    size_t bytes = 0;
    DBS_CUDA(cub::DeviceScan::ExclusiveSum(nullptr, bytes, in, out, n, st));
    void *tmp;
    if (!tp.get((uint8_t **)&tmp, bytes)) return DBSPMSPV_ERR_ALLOC;
    DBS_CUDA(cub::DeviceScan::ExclusiveSum(tmp, bytes, in, out, n, st));
    DBS_CUDA(cudaStreamSynchronize(st));
    tp.release(tmp);
    return DBSPMSPV_OK;
}

int inclusive_sum_i32(TempPool &tp, const int32_t *in, int32_t *out, int64_t n, cudaStream_t st) {
    size_t bytes = 0;
    DBS_CUDA(cub::DeviceScan::InclusiveSum(nullptr, bytes, in, out, n, st));
    void *tmp;
    if (!tp.get((uint8_t **)&tmp, bytes)) return DBSPMSPV_ERR_ALLOC;
    DBS_CUDA(cub::DeviceScan::InclusiveSum(tmp, bytes, in, out, n, st));
    DBS_CUDA(cudaStreamSynchronize(st));
    tp.release(tmp);
    return DBSPMSPV_OK;
}

template <typename K, typename V>
int sort_pairs(TempPool &tp, K *&keys, K *&keys_alt, V *&vals, V *&vals_alt, int64_t n,
               int end_bit, cudaStream_t st) {
    cub::DoubleBuffer<K> dk(keys, keys_alt);
    cub::DoubleBuffer<V> dv(vals, vals_alt);
    size_t bytes = 0;
    DBS_CUDA(cub::DeviceRadixSort::SortPairs(nullptr, bytes, dk, dv, n, 0, end_bit, st));
    void *tmp;
    if (!tp.get((uint8_t **)&tmp, bytes)) return DBSPMSPV_ERR_ALLOC;
    DBS_CUDA(cub::DeviceRadixSort::SortPairs(tmp, bytes, dk, dv, n, 0, end_bit, st));
    DBS_CUDA(cudaStreamSynchronize(st));
    tp.release(tmp);
    if (dk.Current() != keys) { K *t = keys; keys = keys_alt; keys_alt = t; }
    if (dv.Current() != vals) { V *t = vals; vals = vals_alt; vals_alt = t; }
    return DBSPMSPV_OK;
}

struct Widen {  // uint32 block sizes as uint64, with one extra zero so the scan yields the total
    const uint32_t *in;
    int32_t n;
    __host__ __device__ uint64_t operator()(int64_t i) const { return i < n ? in[i] : 0; }
};

int bits_for(uint64_t v) { int b = 0; while (v) { ++b; v >>= 1; } return b ? b : 1; }

#define DBS_TRY(expr) do { int s__ = (expr); if (s__ != DBSPMSPV_OK) return s__; } while (0)
#define DBS_GET(ptr, count) do { if (!tp.get(&(ptr), (size_t)(count))) return DBSPMSPV_ERR_ALLOC; } while (0)
#define DBS_KEEP(ptr, count) do { void *p__ = nullptr; \
        const size_t b__ = ((count) ? (size_t)(count) : 1) * sizeof(*(ptr)); \
        if (cudaMalloc(&p__, b__) != cudaSuccess) { cudaGetLastError(); tp.trim(); \
            if (cudaMalloc(&p__, b__) != cudaSuccess) return DBSPMSPV_ERR_ALLOC; } \
        (ptr) = static_cast<decltype(ptr)>(p__); } while (0)

int build(dbspmspv_handle_s *h, int64_t m, int64_t n, int64_t nnz, const int64_t *row_ptr,
          const int32_t *rows, const int32_t *cols, const void *val, cudaStream_t st) {
    TempPool tp;
    Device &d = h->d;
    const int dt = d.dtype;
    const int vsize = dt == DBSPMSPV_F32 ? 4 : dt == DBSPMSPV_BF16 ? 2 : 0;
    d.m = m; d.n = n;
    d.mb = (int32_t)((m + B - 1) / B);
    d.nb = (int32_t)((n + B - 1) / B);
    {
        uint32_t *rp; DBS_KEEP(rp, (d.mb + 1) / 2);
        d.row_present32 = rp;
        DBS_CUDA(cudaMemsetAsync(rp, 0, (size_t)((d.mb + 1) / 2) * 4, st));
    }

    // inputs on the host: copy once
    if (h->copts.input_on_host) {
        if (row_ptr) { int64_t *t; DBS_GET(t, m + 1); DBS_CUDA(cudaMemcpyAsync(t, row_ptr, (m + 1) * 8, cudaMemcpyHostToDevice, st)); row_ptr = t; }
        if (rows) { int32_t *t; DBS_GET(t, nnz); DBS_CUDA(cudaMemcpyAsync(t, rows, nnz * 4, cudaMemcpyHostToDevice, st)); rows = t; }
        { int32_t *t; DBS_GET(t, nnz); DBS_CUDA(cudaMemcpyAsync(t, cols, nnz * 4, cudaMemcpyHostToDevice, st)); cols = t; }
        if (vsize) { uint8_t *t; DBS_GET(t, nnz * vsize); DBS_CUDA(cudaMemcpyAsync(t, val, nnz * vsize, cudaMemcpyHostToDevice, st)); val = t; }
    }

    int *bad;
    DBS_GET(bad, 1);
    DBS_CUDA(cudaMemsetAsync(bad, 0, sizeof(int), st));

    uint64_t *keys, *keys_alt;
    uint32_t *src, *src_alt;
    DBS_GET(keys, nnz); DBS_GET(keys_alt, nnz); DBS_GET(src, nnz); DBS_GET(src_alt, nnz);
    if (nnz > 0) {
        if (row_ptr) k_keys_from_csr<<<grid_for(nnz), TPB, 0, st>>>(m, n, nnz, row_ptr, cols, keys, src, bad);
        else k_keys_from_coo<<<grid_for(nnz), TPB, 0, st>>>(m, n, nnz, rows, cols, keys, src, bad);
    }
    int bad_h = 0;
    DBS_CUDA(cudaMemcpyAsync(&bad_h, bad, sizeof(int), cudaMemcpyDeviceToHost, st));
    DBS_CUDA(cudaStreamSynchronize(st));
    if (bad_h) return DBSPMSPV_ERR_INVALID_ARG;

    int64_t nnzu = 0;
    uint64_t *ukey = nullptr;
    void *uval = nullptr;
    int32_t n_blocks = 0;
    int32_t *blk_start = nullptr, *block_of = nullptr;   // block_of[u] = 1 + the block of stored element u
    if (nnz > 0) {
        DBS_TRY(sort_pairs(tp, keys, keys_alt, src, src_alt, nnz, 35 + bits_for((uint64_t)d.mb), st));
        tp.release(keys_alt); tp.release(src_alt);
        int32_t *flag, *rank;
        DBS_GET(flag, nnz); DBS_GET(rank, nnz);
        k_flag_new_key<<<grid_for(nnz), TPB, 0, st>>>(nnz, keys, 0, flag);
        DBS_TRY(inclusive_sum_i32(tp, flag, rank, nnz, st));
        int32_t last;
        DBS_CUDA(cudaMemcpy(&last, rank + nnz - 1, 4, cudaMemcpyDeviceToHost));
        nnzu = last;
        DBS_GET(ukey, nnzu);
        { uint8_t *t; DBS_GET(t, nnzu * (vsize ? vsize : 1)); uval = t; }
        if (dt == DBSPMSPV_F32) k_merge_duplicates<DBSPMSPV_F32><<<grid_for(nnz), TPB, 0, st>>>(nnz, keys, src, flag, rank, val, ukey, uval);
        else if (dt == DBSPMSPV_BF16) k_merge_duplicates<DBSPMSPV_BF16><<<grid_for(nnz), TPB, 0, st>>>(nnz, keys, src, flag, rank, val, ukey, uval);
        else k_merge_duplicates<DBSPMSPV_PATTERN><<<grid_for(nnz), TPB, 0, st>>>(nnz, keys, src, flag, rank, val, ukey, uval);
        k_row_presence<<<grid_for(nnzu), TPB, 0, st>>>(nnzu, ukey, const_cast<uint32_t *>(d.row_present32));
        DBS_CUDA(cudaStreamSynchronize(st));
        tp.release(keys); tp.release(src);
        k_flag_new_key<<<grid_for(nnzu), TPB, 0, st>>>(nnzu, ukey, 8, flag);
        DBS_TRY(inclusive_sum_i32(tp, flag, rank, nnzu, st));
        DBS_CUDA(cudaMemcpy(&last, rank + nnzu - 1, 4, cudaMemcpyDeviceToHost));
        n_blocks = last;
        DBS_GET(blk_start, (int64_t)n_blocks + 1);
        k_block_starts<<<grid_for(nnzu), TPB, 0, st>>>(nnzu, flag, rank, blk_start, n_blocks);
        DBS_CUDA(cudaStreamSynchronize(st));
        tp.release(flag);
        block_of = rank;
    }
    h->nnz = nnzu;

    // classify + size
    uint8_t *type;
    uint32_t *psize;
    uint64_t *poff;
    int32_t *brow, *bcol, *ecount, *eoff;
    unsigned long long *cls;
    DBS_GET(type, n_blocks); DBS_GET(psize, n_blocks); DBS_GET(brow, n_blocks); DBS_GET(bcol, n_blocks);
    DBS_GET(ecount, (int64_t)n_blocks + 1); DBS_GET(eoff, (int64_t)n_blocks + 1);
    DBS_GET(cls, 2 * DBSPMSPV_BLK_NCLASS);
    DBS_CUDA(cudaMemsetAsync(cls, 0, 2 * DBSPMSPV_BLK_NCLASS * sizeof(unsigned long long), st));
    DBS_CUDA(cudaMemsetAsync(ecount, 0, ((size_t)n_blocks + 1) * 4, st));
    ClassifyParams cp{h->copts.th0, h->copts.th1, h->copts.th2, h->copts.force_format, dt, h->copts.inline_max};
    if (n_blocks) k_classify<<<grid_for(n_blocks, TPB), TPB, 0, st>>>(n_blocks, blk_start, ukey, cp, type, psize, ecount, brow, bcol, cls, cls + DBSPMSPV_BLK_NCLASS);
    // view entries: a small valued block contributes one entry per stored element
    DBS_TRY(exclusive_sum(tp, ecount, eoff, (int64_t)n_blocks + 1, st));
    int32_t n_entries = 0;
    DBS_CUDA(cudaMemcpy(&n_entries, eoff + n_blocks, 4, cudaMemcpyDeviceToHost));
    d.n_entries = n_entries;
    // 64-bit offsets for the scan (the total may exceed 2^32 words only beyond 16 GB)
    DBS_GET(poff, (int64_t)n_blocks + 1);
    {
        auto it = cub::TransformInputIterator<uint64_t, Widen, cub::CountingInputIterator<int64_t>>(cub::CountingInputIterator<int64_t>(0), Widen{psize, n_blocks});
        size_t bytes = 0;
        DBS_CUDA(cub::DeviceScan::ExclusiveSum(nullptr, bytes, it, poff, (int64_t)n_blocks + 1, st));
        uint8_t *tmp; DBS_GET(tmp, bytes);
        DBS_CUDA(cub::DeviceScan::ExclusiveSum(tmp, bytes, it, poff, (int64_t)n_blocks + 1, st));
        DBS_CUDA(cudaStreamSynchronize(st));
        tp.release(tmp);
    }
    uint64_t total_words = 0;
    DBS_CUDA(cudaMemcpy(&total_words, poff + n_blocks, 8, cudaMemcpyDeviceToHost));
    if (total_words >= (1ull << 32)) return DBSPMSPV_ERR_UNSUPPORTED;
    h->payload_bytes = (int64_t)total_words * 4;
    {
        uint8_t *p; DBS_KEEP(p, h->payload_bytes + 256);  // slack: staged copies may over-read
        DBS_CUDA(cudaMemsetAsync(p, 0, h->payload_bytes + 256, st));
        h->payload_alloc = p; d.payload = p; d.payload_words = (uint32_t)total_words;
    }
    // class census -> which kernel variant the handle uses, hence what a mask-based block costs
    unsigned long long cls_h[2 * DBSPMSPV_BLK_NCLASS];
    DBS_CUDA(cudaMemcpy(cls_h, cls, sizeof(cls_h), cudaMemcpyDeviceToHost));
    {
        unsigned long long heavy_nnz = 0;
        for (int c = DBSPMSPV_BLK_FCSR; c <= DBSPMSPV_BLK_DENSE; ++c) heavy_nnz += cls_h[DBSPMSPV_BLK_NCLASS + c];
        h->heavy_stage = heavy_nnz * 2 > (unsigned long long)nnzu;
    }
    DBS_KEEP(d.csr.ptr, d.mb + 1); DBS_KEEP(d.csr.idx, n_entries + VIEW_PAD); DBS_KEEP(d.csr.w, n_entries + VIEW_PAD); DBS_KEEP(d.csr.aux, n_entries + VIEW_PAD);
    // the slack behind the last entry is read by whole-group staging copies: a class code that no
    // kernel acts on
    k_fill_words<<<1, VIEW_PAD, 0, st>>>(d.csr.idx + n_entries, VIEW_PAD, PAD_IDX);
    DBS_CUDA(cudaMemsetAsync(d.csr.w + n_entries, 0, VIEW_PAD * 4, st)); DBS_CUDA(cudaMemsetAsync(d.csr.aux + n_entries, 0, VIEW_PAD, st));
    DBS_KEEP(d.csc.colptr, (int64_t)d.nb * 17); d.csr.colptr = nullptr;
    DBS_KEEP(d.csc.ptr, d.nb + 1); DBS_KEEP(d.csc.idx, n_entries + VIEW_PAD); DBS_KEEP(d.csc.w, n_entries + VIEW_PAD); DBS_KEEP(d.csc.aux, n_entries + VIEW_PAD);
    DBS_CUDA(cudaMemsetAsync(d.csc.idx + n_entries, 0, VIEW_PAD * 4, st)); DBS_CUDA(cudaMemsetAsync(d.csc.w + n_entries, 0, VIEW_PAD * 4, st)); DBS_CUDA(cudaMemsetAsync(d.csc.aux + n_entries, 0, VIEW_PAD, st));
    DBS_KEEP(h->csc2csr, n_entries);
    DBS_KEEP(h->block_row, n_entries);
    { int32_t *t; DBS_KEEP(t, (int64_t)d.mb + 1); d.csr_inl = t; }
    d.entry_row = h->block_row;
    {
        // The entries are encoded block by block -- (row block, column block) order -- into
        // temporaries and then moved into the block-CSR order (see k_csr_keys).
        uint32_t *t_idx, *t_w;
        uint8_t *t_aux;
        int32_t *t_row, *ids, *ids_alt;
        uint64_t *k1, *k1_alt;
        DBS_GET(t_idx, n_entries); DBS_GET(t_w, n_entries); DBS_GET(t_aux, n_entries); DBS_GET(t_row, n_entries);
        if (n_blocks) {
            uint8_t *pl = static_cast<uint8_t *>(h->payload_alloc);
            const int g = grid_for(n_blocks, TPB), gi = grid_for(nnzu);
#define DBS_ENCODE(DT) do { \
            k_encode_inline<DT><<<gi, TPB, 0, st>>>(nnzu, block_of, blk_start, ukey, uval, type, eoff, brow, bcol, t_idx, t_w, t_aux, t_row); \
            k_encode<DT><<<g, TPB, 0, st>>>(n_blocks, blk_start, ukey, uval, type, poff, eoff, brow, bcol, pl, t_idx, t_w, t_aux, t_row); } while (0)
            if (dt == DBSPMSPV_F32) DBS_ENCODE(DBSPMSPV_F32);
            else if (dt == DBSPMSPV_BF16) DBS_ENCODE(DBSPMSPV_BF16);
            else DBS_ENCODE(DBSPMSPV_PATTERN);
#undef DBS_ENCODE
        }
        DBS_CUDA(cudaStreamSynchronize(st));
        tp.release(ukey); tp.release(uval); tp.release(blk_start); tp.release(block_of); tp.release(poff); tp.release(psize);
        tp.release(brow); tp.release(bcol); tp.release(ecount); tp.release(eoff); tp.release(type);
        DBS_GET(k1, n_entries); DBS_GET(k1_alt, n_entries); DBS_GET(ids, n_entries); DBS_GET(ids_alt, n_entries);
        if (n_entries) {
            k_csr_keys<<<grid_for(n_entries), TPB, 0, st>>>(n_entries, t_row, t_idx, t_aux, k1, ids);
            DBS_TRY(sort_pairs(tp, k1, k1_alt, ids, ids_alt, (int64_t)n_entries, CSR_KEY_ROW_SHIFT + bits_for((uint64_t)d.mb), st));
            k_csr_gather<<<grid_for(n_entries), TPB, 0, st>>>(n_entries, k1, ids, t_idx, t_w, t_aux, d.csr.idx, d.csr.w, d.csr.aux, h->block_row);
        }
        k_csr_inl<<<grid_for((int64_t)d.mb + 1), TPB, 0, st>>>(d.mb, k1, n_entries, const_cast<int32_t *>(d.csr_inl));
        k_lower_bounds<<<grid_for(d.mb + 1), TPB, 0, st>>>(d.mb, h->block_row, n_entries, d.csr.ptr);
        DBS_CUDA(cudaStreamSynchronize(st));
        tp.release(t_idx); tp.release(t_w); tp.release(t_aux); tp.release(t_row);
        tp.release(k1); tp.release(k1_alt); tp.release(ids); tp.release(ids_alt);
    }

    // Hub row blocks: the (at most HUB_BLOCKS_MAX) row blocks with the most view entries, if
    // they hold HUB_BLOCK_MIN_ENTRIES or more.  Chosen on the host from the row block pointers.
    d.hub_slot = nullptr; d.hub_rb = nullptr; d.hub_acc = nullptr; d.n_hub_blocks = 0; d.hub_on = 0;
    if (d.mb > 0 && n_entries >= HUB_BLOCK_MIN_ENTRIES) {
        std::vector<int32_t> ptr((size_t)d.mb + 1);
        DBS_CUDA(cudaMemcpyAsync(ptr.data(), d.csr.ptr, ((size_t)d.mb + 1) * 4, cudaMemcpyDeviceToHost, st));
        DBS_CUDA(cudaStreamSynchronize(st));
        std::vector<int32_t> big;
        for (int32_t rb = 0; rb < d.mb; ++rb)
            if (ptr[rb + 1] - ptr[rb] >= HUB_BLOCK_MIN_ENTRIES) big.push_back(rb);
        auto deg = [&](int32_t rb) { return ptr[rb + 1] - ptr[rb]; };
        auto heavier = [&](int32_t a, int32_t b) { return deg(a) != deg(b) ? deg(a) > deg(b) : a < b; };
        if ((int)big.size() > HUB_BLOCKS_MAX) {
            std::nth_element(big.begin(), big.begin() + HUB_BLOCKS_MAX, big.end(), heavier);
            big.resize(HUB_BLOCKS_MAX);
        }
        std::sort(big.begin(), big.end(), heavier);
        if (!big.empty()) {
            std::vector<uint16_t> slot((size_t)d.mb + 2, HUB_NONE);     // padded: read two at a time
            for (size_t k = 0; k < big.size(); ++k) slot[big[k]] = (uint16_t)k;
            uint16_t *hs; float *ha; int32_t *hr;
            DBS_KEEP(hr, big.size());
            DBS_CUDA(cudaMemcpyAsync(hr, big.data(), big.size() * 4, cudaMemcpyHostToDevice, st));
            const int64_t n_acc = (int64_t)HUB_COPIES * (int64_t)big.size() * 16;
            DBS_KEEP(hs, (int64_t)d.mb + 2); DBS_KEEP(ha, n_acc);
            DBS_CUDA(cudaMemcpyAsync(hs, slot.data(), ((size_t)d.mb + 2) * 2, cudaMemcpyHostToDevice, st));
            k_fill_words<<<grid_for(n_acc), TPB, 0, st>>>(reinterpret_cast<uint32_t *>(ha), n_acc, HUB_CLEAR);
            DBS_CUDA(cudaStreamSynchronize(st));
            d.hub_slot = hs; d.hub_rb = hr; d.hub_acc = ha; d.n_hub_blocks = (int32_t)big.size();
            h->hub_bytes = ((int64_t)d.mb + 2) * 2 + (int64_t)big.size() * 4 + n_acc * 4;
        }
    }

    // block-CSC view: sort the primary entries by column block, and inside it payload entries
    // first (by row block), then the INLINE elements column by column
    {
        uint64_t *k2, *k2_alt;
        int32_t *ids, *ids_alt, *bcol_sorted;
        DBS_GET(k2, n_entries); DBS_GET(k2_alt, n_entries); DBS_GET(ids, n_entries); DBS_GET(ids_alt, n_entries);
        DBS_GET(bcol_sorted, n_entries);
        if (n_entries) {
            k_csc_keys<<<grid_for(n_entries), TPB, 0, st>>>(n_entries, h->block_row, d.csr.idx, d.csr.aux, k2, ids);
            DBS_TRY(sort_pairs(tp, k2, k2_alt, ids, ids_alt, (int64_t)n_entries, CSC_KEY_COL_SHIFT + bits_for((uint64_t)d.nb), st));
            DBS_CUDA(cudaMemcpyAsync(h->csc2csr, ids, (size_t)n_entries * 4, cudaMemcpyDeviceToDevice, st));
            k_csc_gather<<<grid_for(n_entries), TPB, 0, st>>>(n_entries, k2, h->csc2csr, d.csr.idx, d.csr.w, d.csr.aux, d.csc.idx, d.csc.w, d.csc.aux, bcol_sorted, d.hub_slot);
        }
        k_lower_bounds<<<grid_for(d.nb + 1), TPB, 0, st>>>(d.nb, bcol_sorted, n_entries, d.csc.ptr);
        k_csc_colptr<<<grid_for((int64_t)d.nb * 17), TPB, 0, st>>>(d.nb, k2, n_entries, d.csc.colptr);
        DBS_CUDA(cudaStreamSynchronize(st));
        tp.release(k2); tp.release(k2_alt); tp.release(ids); tp.release(ids_alt); tp.release(bcol_sorted);
    }

    // row-run index for the pull levels of DB-BFS
    d.rowrun_ptr = nullptr; d.rowrun_idx = nullptr;
    if (m == n && !h->copts.no_bfs_index) {
        uint64_t *rk, *rk_alt;
        uint32_t *rv, *rv_alt;
        DBS_GET(rk, n_entries); DBS_GET(rk_alt, n_entries); DBS_GET(rv, n_entries); DBS_GET(rv_alt, n_entries);
        if (n_entries) {
            k_rowrun_keys<<<grid_for(n_entries), TPB, 0, st>>>(n_entries, m, h->block_row, d.csr.idx, d.csr.aux, rk, rv);
            DBS_TRY(sort_pairs(tp, rk, rk_alt, rv, rv_alt, (int64_t)n_entries, 31 + bits_for((uint64_t)m), st));
        }
        int32_t *rp;
        DBS_KEEP(rp, m + 1);
        d.rowrun_ptr = rp;
        k_rowrun_ptr<<<grid_for(m + 1), TPB, 0, st>>>(m, rk, n_entries, rp);
        int32_t n_inline = 0;      // the entries with a payload sort behind every row
        DBS_CUDA(cudaMemcpyAsync(&n_inline, rp + m, 4, cudaMemcpyDeviceToHost, st));
        DBS_CUDA(cudaStreamSynchronize(st));
        uint32_t *ri;
        DBS_KEEP(ri, (int64_t)n_inline + 4);      // (slack: the pull reads whole aligned groups of four)
        d.rowrun_idx = ri;
        if (n_inline) DBS_CUDA(cudaMemcpyAsync(ri, rv, (size_t)n_inline * 4, cudaMemcpyDeviceToDevice, st));
        DBS_CUDA(cudaStreamSynchronize(st));
        tp.release(rk); tp.release(rk_alt); tp.release(rv); tp.release(rv_alt);
        h->bfs_index_bytes = ((int64_t)m + 1) * 4 + (int64_t)n_inline * 4;
    }

    // Streaming decode of payload-dominated handles: the chunk table
    d.stage_chunks = nullptr; d.n_stage_chunks = 0;
    d.has_inline = cls_h[DBSPMSPV_BLK_INLINE] > 0;
    d.x_nnz_seen = nullptr; h->x_nnz_seen_host = nullptr; d.x_sparse_believed = 0;
    if (h->heavy_stage) {
        // one word of mapped host memory through which the decode kernels report the x they saw
        void *hp = nullptr, *dp = nullptr;
        if (cudaHostAlloc(&hp, 64, cudaHostAllocMapped) == cudaSuccess && cudaHostGetDevicePointer(&dp, hp, 0) == cudaSuccess) {
            h->x_nnz_seen_host = static_cast<int32_t *>(hp);
            *h->x_nnz_seen_host = -1;
            d.x_nnz_seen = static_cast<int32_t *>(dp);
        } else {
            if (hp) cudaFreeHost(hp);
            cudaGetLastError();
        }
    }
    d.stage_bytes = h->heavy_stage ? decode_stage_bytes(d) : 0;
    if (d.stage_bytes > 0 && d.mb > 0) {
        int32_t *cnt, *first;
        DBS_GET(cnt, (int64_t)d.mb + 1); DBS_GET(first, (int64_t)d.mb + 1);
        DBS_CUDA(cudaMemsetAsync(cnt, 0, ((size_t)d.mb + 1) * 4, st));
        k_stage_chunks<<<grid_for(d.mb), TPB, 0, st>>>(d.mb, d.csr.ptr, d.csr_inl, d.csr.idx, d.csr.w, d.csr.aux, vsize, 32, d.stage_bytes, cnt, nullptr, nullptr);
        DBS_TRY(exclusive_sum(tp, cnt, first, (int64_t)d.mb + 1, st));
        DBS_CUDA(cudaMemcpy(&d.n_stage_chunks, first + d.mb, 4, cudaMemcpyDeviceToHost));
        int4 *chunks;
        DBS_KEEP(chunks, d.n_stage_chunks);
        k_stage_chunks<<<grid_for(d.mb), TPB, 0, st>>>(d.mb, d.csr.ptr, d.csr_inl, d.csr.idx, d.csr.w, d.csr.aux, vsize, 32, d.stage_bytes, cnt, first, chunks);
        DBS_CUDA(cudaStreamSynchronize(st));
        tp.release(cnt); tp.release(first);
        d.stage_chunks = chunks;
        h->stage_index_bytes = (int64_t)d.n_stage_chunks * 16;
    }

    // Streaming pull of hypersparse handles: the list of rows that hold INLINE elements (the
    // stream itself carries one flag bit per row start), the number of row starts before every
    // chunk of the stream, and the positions of the few entries with a payload.
    d.lean_rows = nullptr; d.lean_chunk_ord = nullptr; d.payload_pos = nullptr;
    d.n_lean_chunks = 0; d.n_payload = 0; d.n_lean_rows = 0;
    if (!h->heavy_stage) {
        int32_t *flag, *rank;
        DBS_GET(flag, (int64_t)n_entries + 1); DBS_GET(rank, (int64_t)n_entries + 1);
        k_lean_flags<<<grid_for((int64_t)n_entries + 1), TPB, 0, st>>>(n_entries, d.csr.idx, flag);
        DBS_TRY(exclusive_sum(tp, flag, rank, (int64_t)n_entries + 1, st));
        int32_t n_rows = 0;
        DBS_CUDA(cudaMemcpy(&n_rows, rank + n_entries, 4, cudaMemcpyDeviceToHost));
        d.n_lean_rows = n_rows;
        d.n_lean_chunks = (int32_t)(((int64_t)n_entries + LEAN_CHUNK - 1) / LEAN_CHUNK);
        int32_t *rows, *ord;
        DBS_KEEP(rows, n_rows); DBS_KEEP(ord, (int64_t)d.n_lean_chunks + 1);
        d.lean_rows = rows; d.lean_chunk_ord = ord;
        const int64_t span = (int64_t)n_entries > d.n_lean_chunks + 1 ? n_entries : d.n_lean_chunks + 1;
        k_lean_rows<<<grid_for(span), TPB, 0, st>>>(n_entries, d.csr.idx, d.csr.aux, h->block_row, rank, rows, d.n_lean_chunks, ord);
        // entries with a payload, in view order
        k_payload_flags<<<grid_for((int64_t)n_entries + 1), TPB, 0, st>>>(n_entries, d.csr.idx, flag);
        DBS_TRY(exclusive_sum(tp, flag, rank, (int64_t)n_entries + 1, st));
        DBS_CUDA(cudaMemcpy(&d.n_payload, rank + n_entries, 4, cudaMemcpyDeviceToHost));
        int32_t *ppos;
        DBS_KEEP(ppos, d.n_payload);
        d.payload_pos = ppos;
        if (n_entries) k_payload_list<<<grid_for(n_entries), TPB, 0, st>>>(n_entries, flag, rank, ppos);
        DBS_CUDA(cudaStreamSynchronize(st));
        tp.release(flag); tp.release(rank);
        h->lean_index_bytes = (int64_t)n_rows * 4 + ((int64_t)d.n_lean_chunks + 1) * 4 + (int64_t)d.n_payload * 4;
    }

    // pull segments.  Where mask-based blocks are the bulk of the matrix the lanes of a warp each
    // own one (cheap per block); where they are a minority a whole warp takes them one at a
    // time, which costs about as much as a few hundred INLINE entries: the weights differ.
    {
        SegParams sp{h->copts.seg_cut, h->heavy_stage ? h->copts.w_dense : h->copts.w_dense_sparse,
                     h->heavy_stage ? h->copts.w_mid : h->copts.w_mid_sparse, h->copts.w_coo, h->copts.w_inline};
        int32_t *units, *unit_off;
        DBS_GET(units, (int64_t)d.mb + 1); DBS_GET(unit_off, (int64_t)d.mb + 1);
        k_seg_units<<<grid_for((int64_t)d.mb + 1), TPB, 0, st>>>(d.mb, d.csr.ptr, units);
        DBS_TRY(exclusive_sum(tp, units, unit_off, (int64_t)d.mb + 1, st));
        int32_t n_units = 0;
        DBS_CUDA(cudaMemcpy(&n_units, unit_off + d.mb, 4, cudaMemcpyDeviceToHost));
        int32_t *cnt, *off;
        DBS_GET(cnt, (int64_t)n_units + 1); DBS_GET(off, (int64_t)n_units + 1);
        DBS_CUDA(cudaMemsetAsync(cnt, 0, ((size_t)n_units + 1) * 4, st));
        if (n_units) k_seg_count<<<grid_for((int64_t)n_units * 32), TPB, 0, st>>>(n_units, d.mb, unit_off, d.csr.ptr, d.csr.idx, sp, cnt);
        DBS_TRY(exclusive_sum(tp, cnt, off, (int64_t)n_units + 1, st));
        int32_t nseg = 0;
        DBS_CUDA(cudaMemcpy(&nseg, off + n_units, 4, cudaMemcpyDeviceToHost));
        d.n_segments = nseg;
        Segment *segs; DBS_KEEP(segs, nseg);
        int32_t *seg_rb; DBS_KEEP(seg_rb, (int64_t)nseg + 1);
        if (n_units) k_seg_write<<<grid_for((int64_t)n_units * 32), TPB, 0, st>>>(n_units, d.mb, unit_off, d.csr.ptr, d.csr.idx, sp, off, segs, seg_rb);
        d.seg_rb = seg_rb;
        d.segments = segs;
        int32_t *segw, *segpre;
        DBS_GET(segw, (int64_t)nseg + 1); DBS_GET(segpre, (int64_t)nseg + 1);
        k_seg_weights<<<grid_for((int64_t)nseg + 1), TPB, 0, st>>>(nseg, segs, segw);
        DBS_TRY(exclusive_sum(tp, segw, segpre, (int64_t)nseg + 1, st));
        int32_t total_w = 0;
        DBS_CUDA(cudaMemcpy(&total_w, segpre + nseg, 4, cudaMemcpyDeviceToHost));
        if (total_w < 0) return DBSPMSPV_ERR_UNSUPPORTED;
        d.n_chunks = (int32_t)(((int64_t)total_w + PULL_CH - 1) / PULL_CH);
        int2 *chunks; DBS_KEEP(chunks, (int64_t)d.n_chunks + 1);
        k_chunks<<<grid_for((int64_t)d.n_chunks + 1), TPB, 0, st>>>(d.n_chunks, segs, segpre, nseg, d.n_entries, chunks);
        d.chunks = chunks;
        DBS_CUDA(cudaStreamSynchronize(st));
    }

    // statistics
    dbspmspv_stats &s = h->stats;
    s.m = m; s.n = n; s.nnz = nnzu; s.n_blocks = n_blocks;
    for (int c = 0; c < DBSPMSPV_BLK_NCLASS; ++c) { s.class_blocks[c] = (int64_t)cls_h[c]; s.class_nnz[c] = (int64_t)cls_h[DBSPMSPV_BLK_NCLASS + c]; }
    s.n_row_blocks = d.mb; s.n_col_blocks = d.nb; s.n_segments = d.n_segments;
    s.payload_bytes = h->payload_bytes;
    s.n_view_entries = d.n_entries;
    s.csr_view_bytes = ((int64_t)d.mb + 1) * 8 + (int64_t)d.n_entries * 9;
    s.csc_view_bytes = ((int64_t)d.nb + 1) * 4 + (int64_t)d.nb * 17 * 4 + (int64_t)d.n_entries * 9 + h->hub_bytes;
    s.segment_bytes = (int64_t)d.n_segments * (int64_t)sizeof(Segment) + ((int64_t)d.n_chunks + 1) * 8 + (int64_t)d.n_segments * 4 + h->stage_index_bytes;
    s.bfs_index_bytes = h->bfs_index_bytes;
    s.lean_index_bytes = h->lean_index_bytes;
    s.n_hub_row_blocks = d.n_hub_blocks;
    DBS_CUDA(cudaGetLastError());
    return DBSPMSPV_OK;
}

}  // namespace

int allocate_workspace(dbspmspv_handle_s *h);  // run.cu

int create_common(dbspmspv_handle_t *out, int64_t m, int64_t n, int64_t nnz, const int64_t *row_ptr,
                  const int32_t *rows, const int32_t *cols, const void *val, int dtype, int block_size,
                  const dbspmspv_create_opts *opts, dbspmspv_stream_t stream) {
    if (!out) return DBSPMSPV_ERR_INVALID_ARG;
    *out = nullptr;
    if (m < 1 || n < 1 || nnz < 0 || m >= (1ll << 31) || n >= (1ll << 31) || nnz >= (1ll << 31)) return DBSPMSPV_ERR_INVALID_ARG;
    if ((!row_ptr && !rows) || (nnz > 0 && !cols)) return DBSPMSPV_ERR_INVALID_ARG;
    if (dtype != DBSPMSPV_F32 && dtype != DBSPMSPV_BF16 && dtype != DBSPMSPV_PATTERN) return DBSPMSPV_ERR_INVALID_ARG;
    if (dtype != DBSPMSPV_PATTERN && nnz > 0 && !val) return DBSPMSPV_ERR_INVALID_ARG;
    if (block_size != B) return DBSPMSPV_ERR_UNSUPPORTED;
    dbspmspv_handle_s *h = new (std::nothrow) dbspmspv_handle_s();
    if (!h) return DBSPMSPV_ERR_ALLOC;
    if (opts) h->copts = *opts; else dbspmspv_default_create_opts(&h->copts);
    if (h->copts.th0 < 1 || h->copts.th1 > 256 || h->copts.seg_cut < 1 || h->copts.seg_cut > MAX_SEG_ENTRIES || h->copts.w_coo < 1 || h->copts.w_inline < 1 || h->copts.w_mid_sparse < 1 || h->copts.w_dense_sparse < 1 || h->copts.w_mid < 1 || h->copts.w_dense < 1 || h->copts.inline_max < 0 || h->copts.inline_max > 31) { delete h; return DBSPMSPV_ERR_INVALID_ARG; }
    dbspmspv_default_run_opts(&h->ropts);
    h->d.dtype = dtype;
    if (cudaGetDevice(&h->device) != cudaSuccess) { delete h; return DBSPMSPV_ERR_CUDA; }
    cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device);
    int st = build(h, m, n, nnz, row_ptr, rows, cols, val, static_cast<cudaStream_t>(stream));
    if (st == DBSPMSPV_OK) st = allocate_workspace(h);
    if (st != DBSPMSPV_OK) { cudaGetLastError(); dbspmspv_destroy(h); return st; }
    *out = h;
    return DBSPMSPV_OK;
}

}  // namespace dbs

extern "C" {

void dbspmspv_default_create_opts(dbspmspv_create_opts *o) {
    if (!o) return;
    *o = dbspmspv_create_opts();
    o->th0 = 32; o->th1 = 128; o->th2 = 2.0f;
    o->seg_cut = 128; o->w_dense = 16; o->w_mid = 8; o->w_coo = 4; o->w_inline = 1;
    o->w_dense_sparse = 128; o->w_mid_sparse = 64;
    o->force_format = DBSPMSPV_FORMAT_AUTO;
    o->input_on_host = 0;
    o->inline_max = 31;
}

int dbspmspv_create_csr(dbspmspv_handle_t *out, int64_t m, int64_t n, int64_t nnz,
                        const int64_t *row_ptr, const int32_t *col_idx, const void *val,
                        int dtype, int block_size, const dbspmspv_create_opts *opts,
                        dbspmspv_stream_t stream) {
    if (!row_ptr) return DBSPMSPV_ERR_INVALID_ARG;
    return dbs::create_common(out, m, n, nnz, row_ptr, nullptr, col_idx, val, dtype, block_size, opts, stream);
}

int dbspmspv_create_coo(dbspmspv_handle_t *out, int64_t m, int64_t n, int64_t nnz,
                        const int32_t *row, const int32_t *col, const void *val, int dtype,
                        int block_size, const dbspmspv_create_opts *opts,
                        dbspmspv_stream_t stream) {
    if (!row && nnz > 0) return DBSPMSPV_ERR_INVALID_ARG;
    static const int32_t dummy = 0;
    return dbs::create_common(out, m, n, nnz, nullptr, row ? row : &dummy, col, val, dtype, block_size, opts, stream);
}

}  // extern "C"
