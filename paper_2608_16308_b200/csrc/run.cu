// One SpMSpV call (Sections 3.3 and 4.1): vector blocking + push worklist, device-side path
// selection, push / pull traversal with per-block microkernels, hierarchical writeback, and
// compaction of the dense accumulator into a sorted sparse y.  Also the dense-in / dense-out
// decode entry (Section 4.3).  Nothing here allocates or synchronises, except db_sssp (a host
// loop over (min, +) products, at the end of the file).
#include "internal.cuh"
#include "microkernels.cuh"
#include "staging.cuh"
#include "worklist.cuh"
#include "mma_block.cuh"

namespace dbs {
__device__ __forceinline__ int select_path(const Device &d, float th3, int force_path);
}
#include "lean_pull.cuh"

namespace dbs {

constexpr int CTA = 128;            // four warps per thread block (Section 3.3.2)
constexpr int WARPS = CTA / 32;
constexpr int XB_TPB = 512;         // vector blocking of a sparse x: threads per block
constexpr int CMP_TPB = 256;        // compaction: threads per tile
constexpr int TILE_WORDS = CMP_TPB / 4;  // a tile: 64 mask words = 2048 rows; placement uses 8 rows per thread

// ------------------------------------------------------------------------------------------
// Vector blocking (Section 3.2.2) fused with the push worklist (Section 3.3.2).
// Sparse input: one thread per listed nonzero scatters the value into the dense copy and sets
// its mask bit; the thread that turns a vector block from empty to nonempty emits the block's
// push tasks (runs of <= 32 entries of its block-CSC column).  Space in the worklist is
// claimed with a warp scan, a sum over the thread block's warps and one atomic per thread
// block; the count of nonempty vector blocks is aggregated the same way (Section 4.1).
// ------------------------------------------------------------------------------------------
// EMIT = false: only the dense copy, the masks and the count -- the worklist is then built by
// k_emit_from_masks, and only if the selector chooses the push (used when x is so dense that a
// pull is likely: the tasks of half a million columns would be written for nothing).
template <int DT, bool EMIT>
__global__ void k_xblock_sparse(Device d, const int32_t *__restrict__ x_idx, const void *__restrict__ x_val,
                                int32_t nnz_x, int validate) {
    pdl_launch_dependents();
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31;
    bool newly = false, fresh = false;
    int jb = 0, jcol = 0;
    int first = 0, deg = 0, pfirst = 0, pdeg = 0;
    if (t < nnz_x) {
        const int j = x_idx[t];
        // an index outside [0, n) is never written through: the entry is skipped and the call
        // reports ERR_BOUNDS (the compare is free next to the dependent scatter)
        if (j < 0 || j >= d.n) {
            d.ws.ctr->status = DBSPMSPV_ERR_BOUNDS;
        } else {
            float v = 1.0f;
            if (x_val) {
                if (DT == DBSPMSPV_BF16) v = __bfloat162float(static_cast<const __nv_bfloat16 *>(x_val)[t]);
                else v = static_cast<const float *>(x_val)[t];
            }
            // a listed NaN that happens to carry the marker's bit pattern is stored as the
            // canonical quiet NaN, so the marker itself never appears as data
            d.ws.x_dense[j] = __float_as_uint(v) == X_ABSENT ? __uint_as_float(0x7FC00000u) : v;
            // the runs this thread may have to turn into tasks are fetched before the atomic
            // whose result decides it (the loads are independent of it; the chain is shorter)
            if (EMIT) { column_run(d, j, first, deg); payload_run(d, j >> 4, pfirst, pdeg); }
            const int sh = ((j >> 4) & 1) * 16;
            const uint32_t old = atomicOr(&d.ws.x_mask32[j >> 5], 1u << ((j & 15) + sh));
            newly = ((old >> sh) & 0xFFFFu) == 0;
            fresh = ((old >> ((j & 15) + sh)) & 1u) == 0;     // (an index listed twice emits once)
            if (validate && !fresh) d.ws.ctr->status = DBSPMSPV_ERR_INVALID_ARG;   // optional check: duplicate index
            jb = j >> 4;
            jcol = j;
        }
    }
    if (!EMIT) {                                              // count the nonempty vector blocks, nothing else
        emit_tasks<true>(d, newly, jb, 0, 0, lane, &d.ws.ctr->n_tasks, &d.ws.ctr->n_nzblk);
        return;
    }
    // push tasks: the INLINE elements of this column; and, by the thread that turned the vector
    // block nonempty, the column block's entries with a payload
    if (d.payload_chunk == PUSH_CHUNK) {
        // Matrices whose elements sit mostly in blocks with a payload (banded matrices, pruned
        // layers): the thread that turned the vector block nonempty emits the whole column block
        // in one run -- payload entries and INLINE elements, the latter filtered by the mask in
        // the traversal.  Per-column runs would split a column block over several half-empty
        // tasks here (measured on the stencil: 30 % slower).
        first = pfirst;
        deg = newly ? d.csc.ptr[jb + 1] - pfirst : 0;
        emit_tasks<true>(d, newly, jb, first, deg, lane, &d.ws.ctr->n_tasks, &d.ws.ctr->n_nzblk, PUSH_CHUNK, &d.ws.ctr->n_hubs, d.ws.hubs);
        return;
    }
    if (!fresh) deg = 0;
    merge_column_runs(fresh, jcol, first, deg, lane);
    emit_tasks<true>(d, newly, jb, first, deg, lane, &d.ws.ctr->n_tasks, &d.ws.ctr->n_nzblk, PUSH_CHUNK, &d.ws.ctr->n_hubs, d.ws.hubs);
    if (!newly) pdeg = 0;
    if (__syncthreads_or(pdeg > 0))
        emit_tasks<true>(d, false, jb, pfirst, pdeg, lane, &d.ws.ctr->n_tasks, &d.ws.ctr->n_nzblk, d.payload_chunk);
}

__device__ __forceinline__ int select_path(const Device &d, float th3, int force_path);

// The push worklist from the finished vector-block masks (hypersparse matrices): runs only if
// the selector chooses the push.  A warp takes one mask word (two vector blocks) at a time,
// lane = column: listed columns emit their INLINE runs (adjacent ones merged), lanes 0 and 16
// the payload runs of the two blocks.
__global__ void k_emit_from_masks(Device d, float th3, int force_path) {
    pdl_wait();
    pdl_launch_dependents();
    if (select_path(d, th3, force_path) != DBSPMSPV_PATH_PUSH) return;
    const int lane = threadIdx.x & 31;
    const int gwarp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    const int n_words = (d.nb + 1) / 2;
    Counters *ctr = d.ws.ctr;
    for (int wd = gwarp; wd < n_words; wd += nwarps) {
        const uint32_t word = d.ws.x_mask32[wd];
        if (!word) continue;                                   // warp-uniform
        const int jb = 2 * wd + (lane >> 4), j = jb * 16 + (lane & 15);
        const bool listed = (word >> lane) & 1u;
        int first = 0, deg = 0;
        if (listed) column_run(d, j, first, deg);
        merge_column_runs(listed, j, first, deg, lane);
        emit_tasks(d, false, jb, first, deg, lane, &ctr->n_tasks, &ctr->pad, PUSH_CHUNK, &ctr->n_hubs, d.ws.hubs);
        first = 0; deg = 0;
        if ((lane & 15) == 0 && ((word >> lane) & 0xFFFFu)) payload_run(d, jb, first, deg);
        if (__any_sync(FULL, deg > 0)) emit_tasks(d, false, jb, first, deg, lane, &ctr->n_tasks, &ctr->pad, d.payload_chunk);
    }
}

// Dense input (Sections 4.1, 4.3): every warp reads 32 elements, one ballot gives the two
// 16-bit masks of its two vector blocks.  Also clears the dense output.
// Which entries of a dense activation vector take part in a decode call: |x_j| > tau, or, with
// the ReLU fused in, x_j > tau (tau = 0: x_j not zero / positive).  A NaN always takes part.
__device__ __forceinline__ bool decode_takes_part(const Device &d, float v) {
    return d.decode_relu ? !(v <= d.decode_tau) : !(fabsf(v) <= d.decode_tau);
}

template <int DT>
__global__ void k_xblock_dense(Device d, const void *__restrict__ x, float *__restrict__ y) {
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int64_t padded = (int64_t)((d.nb + 1) / 2) * 32;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j < padded; j += stride) {
        float v = 0.f;
        if (j < d.n) {
            if (DT == DBSPMSPV_BF16 && !d.decode_x_f32) v = __bfloat162float(static_cast<const __nv_bfloat16 *>(x)[j]);
            else v = static_cast<const float *>(x)[j];
            if (DT == DBSPMSPV_BF16 && d.decode_x_f32) v = __bfloat162float(__float2bfloat16_rn(v));
        }
        const bool in = j < d.n && decode_takes_part(d, v);
        if (j < (int64_t)d.nb * 16)
            d.ws.x_dense[j] = in ? (__float_as_uint(v) == X_ABSENT ? __uint_as_float(0x7FC00000u) : v)
                                 : __uint_as_float(X_ABSENT);
        const uint32_t bits = __ballot_sync(FULL, in);
        if (lane == 0) d.ws.x_mask32[j >> 5] = bits;
        const bool newly = (lane == 0 && (bits & 0xFFFFu)) || (lane == 16 && (bits >> 16));
        int first = 0, deg = 0;
        const bool listed = in && j < d.n;
        if (d.payload_chunk == PUSH_CHUNK) {                 // whole column blocks, as in the sparse-x kernel
            if (newly) { first = d.csc.ptr[j >> 4]; deg = d.csc.ptr[(j >> 4) + 1] - first; }
            emit_tasks(d, newly, (int)(j >> 4), first, deg, lane, &d.ws.ctr->n_tasks, &d.ws.ctr->n_nzblk, PUSH_CHUNK, &d.ws.ctr->n_hubs, d.ws.hubs);
            continue;
        }
        if (listed) column_run(d, (int)j, first, deg);
        merge_column_runs(listed, (int)j, first, deg, lane);
        emit_tasks(d, newly, (int)(j >> 4), first, deg, lane, &d.ws.ctr->n_tasks, &d.ws.ctr->n_nzblk, PUSH_CHUNK, &d.ws.ctr->n_hubs, d.ws.hubs);
        first = 0; deg = 0;
        if (newly) payload_run(d, (int)(j >> 4), first, deg);
        if (__any_sync(FULL, deg > 0))
            emit_tasks(d, false, (int)(j >> 4), first, deg, lane, &d.ws.ctr->n_tasks, &d.ws.ctr->n_nzblk, d.payload_chunk);
    }
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < d.m; i += stride) y[i] = 0.f;
}

// ------------------------------------------------------------------------------------------
// Traversal.  Output goes through `Out`: the sparse path accumulates into the handle's dense
// accumulator and structural-hit masks; the decode path adds straight into the caller's y.
// ------------------------------------------------------------------------------------------
struct OutSparse {
    float *acc;
    uint8_t *hit8;     // one byte per row: 1 = structurally hit (plain idempotent stores, no atomics)
    static constexpr bool MASKS = true;
    static constexpr bool MINPLUS = false;
};
struct OutDense {
    float *acc;
    uint8_t *hit8;
    static constexpr bool MASKS = false;
    static constexpr bool MINPLUS = false;
};
// (min, +) semiring: the accumulator holds keys of the smallest sum so far (minplus.cuh)
struct OutSparseMin {
    float *acc;
    uint8_t *hit8;
    static constexpr bool MASKS = true;
    static constexpr bool MINPLUS = true;
};

// One lane owns one hypersparse block (INLINE or COO).  `emit(r, v)` receives the products,
// already summed per row where the entries of a row are adjacent (COO is stored row-major);
// `xin` is the x entry of an INLINE block's single column (fetched by the caller in parallel
// with the mask); `xb` points at the 16 x entries of the block's vector block.  Returns the
// structural-hit row mask.
template <int DT, typename Emit>
__device__ __forceinline__ uint32_t lane_block(int type, uint32_t w, uint32_t aux, uint32_t xm,
                                               float xin, const float *xb, const uint8_t *payload,
                                               Emit emit) {
    uint32_t hit = 0;
    if (type == DBSPMSPV_BLK_INLINE) {
        if ((xm >> (aux & 15)) & 1u) {
            if (DT != DBSPMSPV_PATTERN) emit((int)(aux >> 4), Val<DT>::inline_value(w) * xin);
            hit = 1u << (aux >> 4);
        }
    } else {
        const int nnz = (int)aux + 1;
        const uint8_t *blk = payload + (size_t)w * 4;
        const uint32_t *cw = reinterpret_cast<const uint32_t *>(blk);
        const uint8_t *vals = blk + ((nnz + 3) & ~3);
        int cur = -1;
        float s = 0.f;
        for (int k0 = 0; k0 < nnz; k0 += 4) {
            uint32_t word = cw[k0 >> 2];
            const int lim = min(4, nnz - k0);
            for (int j = 0; j < lim; ++j, word >>= 8) {
                const int c = word & 15, r = (word >> 4) & 15;
                if ((xm >> c) & 1u) {
                    if (DT != DBSPMSPV_PATTERN) {
                        if (r != cur) { if (cur >= 0) emit(cur, s); cur = r; s = 0.f; }
                        s += Val<DT>::load(vals, k0 + j) * xb[c];
                    }
                    hit |= 1u << r;
                }
            }
        }
        if (DT != DBSPMSPV_PATTERN && cur >= 0) emit(cur, s);
    }
    return hit;
}

__device__ __forceinline__ bool lane_owned(int type, uint32_t aux) {
    return type == DBSPMSPV_BLK_INLINE || (type == DBSPMSPV_BLK_COO && aux < COO_SERIAL_MAX);
}

// The COO blocks held by the 32 lanes of a warp, processed as ONE flat list of stored entries:
// a warp scan of the per-lane entry counts lays the entries out, then every lane takes one
// entry per step and finds its owner block by a shuffle binary search over the scan.  This
// keeps all lanes busy whatever the mix of block sizes (a lane looping over its own block
// would make the whole warp wait for the largest block).  `cnt` is the lane's entry count
// (0 = no COO block here); `tag0`, `tag1` are per-block values handed back to
// `emit(tag0, tag1, r, c, value, owner_lane)` for every entry whose column is active.
template <int DT, typename Emit>
__device__ __forceinline__ void warp_flat_coo(int cnt, uint32_t w, uint32_t xm, uint32_t tag0, uint32_t tag1,
                                              const uint8_t *payload, int lane, Emit emit) {
    int incl = cnt;
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(FULL, incl, o);
        if (lane >= o) incl += t;
    }
    const int total = __shfl_sync(FULL, incl, 31);
    for (int e0 = 0; e0 < total; e0 += 32) {
        const int e = e0 + lane;
        int o = 0;
#pragma unroll
        for (int s = 16; s; s >>= 1) {
            const int v = __shfl_sync(FULL, incl, o + s - 1);
            if (v <= e) o += s;
        }
        const int bn = __shfl_sync(FULL, cnt, o);
        const int k = e - (__shfl_sync(FULL, incl, o) - bn);
        const uint32_t bw = __shfl_sync(FULL, w, o);
        const uint32_t bxm = __shfl_sync(FULL, xm, o);
        const uint32_t bt0 = __shfl_sync(FULL, tag0, o);
        const uint32_t bt1 = __shfl_sync(FULL, tag1, o);
        if (e < total) {
            const uint8_t *blk = payload + (size_t)bw * 4;
            const uint32_t rc = blk[k];
            const int c = rc & 15, r = rc >> 4;
            if ((bxm >> c) & 1u) emit(bt0, bt1, r, c, Val<DT>::load(blk + ((bn + 3) & ~3), k), o);
        }
    }
}

// Structural-hit marking: one byte per output row, set with a plain store.  Stores of the same
// value to the same byte need no atomic and no read, so hub rows that are hit by thousands of
// products per call cost nothing extra; the compaction pass packs the bytes into masks.
__device__ __forceinline__ void mark_rows(uint8_t *hit8, int rb, uint32_t rows16) {
    uint8_t *base = hit8 + (size_t)rb * 16;
    while (rows16) {
        base[__ffs(rows16) - 1] = 1;
        rows16 &= rows16 - 1;
    }
}

// Writeback of one block handled outside the shared-memory accumulator: lanes 0..15 own the 16
// rows; one global atomic and one flag store per touched row.
template <typename Out>
__device__ __forceinline__ void flush_rows(Out out, int rb, uint32_t hits, float v, int lane) {
    if (lane < 16 && ((hits >> lane) & 1u)) {
        atomicAdd(out.acc + (size_t)rb * 16 + lane, v);
        if (Out::MASKS) out.hit8[(size_t)rb * 16 + lane] = 1;
    }
}

// One product of an INLINE element whose row block is a hub (HUB_FLAG): added to one of the
// HUB_COPIES private accumulators of that row block, picked by the CTA, with an atomic whose
// reply nobody reads.  The L2 serves atomics on one line one after the other: on an R-MAT
// matrix one line of the accumulator receives 1-2 % of ALL products, and that queue, not the
// traversal, set the duration of the push (58 -> 35 us at 10 % x density when the same atomics
// go to distinct lines).  A private accumulator that nothing touched holds -0.0f: any sum of
// finite products that are neither zero nor subnormal differs from it in its bits (x + -x is
// +0 in round-to-nearest), so the fold of the compaction needs no flags.  Products that are
// zero or subnormal (an atomic may flush them to a signed zero) return false and take the
// ordinary path.
template <typename Out>
__device__ __forceinline__ bool push_private(const Device &d, uint32_t idx, uint32_t aux, float prod) {
    if (!Out::MASKS || !d.hub_on || !(idx & HUB_FLAG) || !(fabsf(prod) >= 1.17549435e-38f)) return false;
    const int slot = d.hub_slot[idx & IDX_MASK];
    if (!DBS_CHK_INDEX(d, slot, d.n_hub_blocks)) return false;
    atomicAdd(d.hub_acc + (((size_t)(blockIdx.x & (HUB_COPIES - 1)) * d.n_hub_blocks + slot) * 16 + (aux >> 4)), prod);
    return true;
}

// Per-warp staging area in shared memory: two stages of view entries for the pull; the push
// uses the same bytes as one stage for the payload of a task's blocks.
struct PullStage {
    uint32_t idx[STAGE_CAP];
    uint32_t w[STAGE_CAP];
    uint8_t aux[STAGE_CAP];
};
struct PullWarp {
    PullStage stage[2];
    uint64_t bar[2];
};

// Push (Section 3.3.2): every warp takes one task = up to PUSH_CHUNK consecutive block-CSC
// entries of one active column block (32 per step, all fetched up front); the vector block is staged once per task (Section 3.3.3).  Lanes
// own hypersparse blocks; heavier blocks are then processed by the whole warp one at a time.
// Writeback: warp-level reduction, then one global atomic per touched row and one atomicOr on
// the row block's hit mask.  The task record carries its length, so the view entries, the mask
// and the x block are all fetched in one round of independent loads.
template <int DT, typename Out, bool HV>
__device__ void push_body(const Device &d, Out out, int popc_threshold, float *s_x, float *s_tmp, float *s_lacc, PullWarp *pw) {
    constexpr int U = PUSH_CHUNK / 32;
    const int lane = threadIdx.x & 31;
    const int gwarp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    static_assert(U == 1, "one warp step per task");
    const int n_recs = d.ws.ctr->n_tasks, n_hubs = min(d.ws.ctr->n_hubs, HUB_CAP);
    const HubTable hubs = load_hub_table(d.ws.hubs, n_hubs, lane);
    const int n_tasks = n_recs + hubs.total;                       // task records, then the steps of the hub runs
    auto item = [&](int i) { return worklist_item(d.ws.tasks, n_recs, hubs, i); };
    // A task is a chain of dependent loads (record -> entries, column end, mask, x block); the
    // loop is software-pipelined: while task k is evaluated, the loads of k+1 and the record of
    // k+2 (in this warp's stride) are in flight.
    struct Loads { uint32_t idx, w, aux, xm; float xv; int start, end, jb; };
    auto loads_of = [&](int t, const uint2 &task) {
        Loads l{0u, 0u, 0u, 0u, 0.f, 0, 0, 0};
        if (t < n_tasks) {
            const int jb = (int)(task.x & IDX_MASK);
            l.jb = jb;
            const int cnt = (int)(task.x >> 27) + 1;              // entries of the task
            l.start = (int)task.y;
            if (lane < cnt && DBS_CHK_RANGE(d, l.start, cnt) && DBS_CHK_INDEX(d, jb, d.nb)) {
                const int p = l.start + lane; l.idx = d.csc.idx[p]; l.w = d.csc.w[p]; l.aux = d.csc.aux[p];
                DBS_CHK_ENTRY(d, false, l.idx, l.w, l.aux);
            }
            l.end = l.start + cnt;
            l.xm = mask_of(d.ws.x_mask32, jb);
            if (lane < 16) l.xv = d.ws.x_dense[jb * 16 + lane];
        }
        return l;
    };
    const uint2 none = make_uint2(0u, 0u);
    uint2 rec1 = gwarp + nwarps < n_tasks ? item(gwarp + nwarps) : none;
    Loads cur = loads_of(gwarp, gwarp < n_tasks ? item(gwarp) : none);
    // Payload staging (Section 3.3.3) on handles whose elements sit mostly in blocks with a payload:
    // when the payload of all blocks of a task fits the warp's staging area, every lane moves its
    // block there with one bulk copy and the microkernels read shared memory.  The point is the
    // bytes in flight: 32 blocks per warp at once instead of the two a half-warp pair walks
    // (header -> values, two dependent trips each) -- at 14 warps per SM the latter keeps about
    // 6 KB per SM in flight where the memory system wants 35.  (A second area per warp, so that
    // the next task's copies fly while this one is computed, was measured slower: the shared
    // memory it takes costs a resident thread block per SM.)
    constexpr int STAGE_AREA = (int)sizeof(PullStage) * 2;
    uint32_t stage_parity = 0u;
    // issues the copies of one task; returns the lane's byte offset in the area, or -1 (not staged)
    auto stage_issue = [&](const Loads &l) {
        const bool have = l.start + lane < l.end;
        const int type = l.idx >> TYPE_SHIFT;
        const int bytes = have && type != DBSPMSPV_BLK_INLINE ? payload_words(type, (int)l.aux + 1, Val<DT>::SIZE) * 4 : 0;
        int incl = bytes;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(FULL, incl, o);
            if (lane >= o) incl += v;
        }
        const int total = __shfl_sync(FULL, incl, 31);
        if (total <= 0 || total > STAGE_AREA) return -1;          // warp-uniform
        uint8_t *area = reinterpret_cast<uint8_t *>(pw->stage);
        if (lane == 0) mbar_arrive_expect_tx(&pw->bar[0], (uint32_t)total);
        __syncwarp();
        if (bytes) bulk_copy_g2s(area + incl - bytes, d.payload + (size_t)l.w * 4, (uint32_t)bytes, &pw->bar[0]);
        return incl - bytes;
    };
    if (HV) {
        if (lane == 0) { mbar_init(&pw->bar[0], 1); fence_barrier_init(); }
        __syncwarp();
    }
    for (int t = gwarp; t < n_tasks; t += nwarps) {
        const uint2 rec2 = t + 2 * nwarps < n_tasks ? item(t + 2 * nwarps) : none;
        const Loads nxt = loads_of(t + nwarps, rec1);
        rec1 = rec2;
        const int off_cur = HV ? stage_issue(cur) : -1;         // (the area is free: the last task's reads ended at the warp barrier)
        uint32_t idx[U] = {cur.idx}, w[U] = {cur.w}, aux[U] = {cur.aux};
        const int start = cur.start, end = cur.end, jb = cur.jb;
        const uint32_t xm = cur.xm;
        if (lane < 16) s_x[lane] = cur.xv;
        cur = nxt;
        __syncwarp();
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (start + u * 32 >= end) break;                 // warp-uniform
            const bool have = start + u * 32 + lane < end;
            bool heavy = false;
            int coo_cnt = 0;
            const int type = idx[u] >> TYPE_SHIFT;
            const int brow = idx[u] & IDX_MASK;
            const uint8_t *pl = d.payload;        // where this task's payload is read from (w[u] counts 4-byte words from it)
            if (HV && off_cur >= 0) {            // warp-uniform: this task's payload was staged
                if (!mbar_wait_bounded(&pw->bar[0], stage_parity)) {
                    // (never seen; the copies in flight get a second, equally bounded chance to land before the warp leaves)
                    d.ws.ctr->status = DBSPMSPV_ERR_TIMEOUT;
                    mbar_wait_bounded(&pw->bar[0], stage_parity);
                    return;
                }
                stage_parity ^= 1u;
                pl = reinterpret_cast<const uint8_t *>(pw->stage);
                if (have && type != DBSPMSPV_BLK_INLINE) w[u] = (uint32_t)off_cur >> 2;
            }
            if (have) {
                if (type == DBSPMSPV_BLK_INLINE) {
                    float *row0 = out.acc + (size_t)brow * 16;
                    // The structural-hit flag is stored only when the atomic returns zero: the first
                    // product that reaches a row always sees the cleared accumulator, so the flag is
                    // set once per row instead of once per product (a later zero -- an explicitly
                    // stored zero, a cancellation -- only repeats the store).  The repeated byte
                    // stores to the hub rows of a power-law matrix, not the atomics, were what the
                    // push waited for: 77 -> 57 us at 10 % x density, 326 -> 170 us at 50 %.  (The
                    // per-block writebacks of mask-based blocks keep the plain atomic and the
                    // unconditional store: on the stencil the returning atomic cost 7-15 %.)
                    bool first = false;
                    const uint32_t hit = lane_block<DT>(type, w[u], aux[u], xm, s_x[aux[u] & 15], s_x, pl,
                                                        [&](int r, float v) { if (!push_private<Out>(d, idx[u], aux[u], v)) first |= atomicAdd(row0 + r, v) == 0.0f; });
                    // (pattern matrices have no product: they count the hits in the accumulator,
                    // which the compaction clears like any other, to get the same first-touch test)
                    if (DT == DBSPMSPV_PATTERN && hit && !push_private<Out>(d, idx[u], aux[u], 1.0f)) first = atomicAdd(row0 + (aux[u] >> 4), 1.0f) == 0.0f;
                    if (Out::MASKS && hit && first) mark_rows(out.hit8, brow, hit);
                } else if (type == DBSPMSPV_BLK_COO && aux[u] < COO_SERIAL_MAX) {
                    coo_cnt = (int)aux[u] + 1;
                } else {
                    heavy = true;
                }
            }
            if (__any_sync(FULL, coo_cnt)) {
                uint32_t *s_hit = reinterpret_cast<uint32_t *>(s_tmp);   // per-owner-lane hit masks
                s_hit[lane] = 0u;
                __syncwarp();
                warp_flat_coo<DT>(coo_cnt, w[u], xm, (uint32_t)brow, 0u, pl, lane,
                                  [&](uint32_t tag, uint32_t, int r, int c, float a, int owner) {
                                      if (DT != DBSPMSPV_PATTERN) atomicAdd(out.acc + (size_t)tag * 16 + r, a * s_x[c]);
                                      if (Out::MASKS) atomicOr(&s_hit[owner], 1u << r);
                                  });
                __syncwarp();
                if (Out::MASKS && coo_cnt && s_hit[lane]) mark_rows(out.hit8, brow, s_hit[lane]);
                __syncwarp();
            }
            // dense vector block and several mask-based blocks in the step: half-warp streaming
            // form (two blocks per warp at a time, next pair prefetched; a warp that takes one
            // block at a time waits out two dependent loads per block)
            if (HV && DT != DBSPMSPV_PATTERN && __popc(xm) >= popc_threshold) {
                const bool mk = heavy && type != DBSPMSPV_BLK_COO;
                const uint32_t cs = __ballot_sync(FULL, mk);
                if (__popc(cs) >= HEAVY_LANE_MIN) {
                    auto emit = [&](int erb, int erow, float esum) {
                        atomicAdd(out.acc + (size_t)erb * 16 + erow, esum);
                        if (Out::MASKS) out.hit8[(size_t)erb * 16 + erow] = 1;
                    };
                    const uint32_t rows = __ballot_sync(FULL, mk && is_row_major(type));
                    const uint32_t tagged = (idx[u] & ~IDX_MASK) | (uint32_t)jb;     // class bits + the task's column block
                    if (cs & ~rows) half_stream<DT, false>(pl, d.ws.x_dense, tagged, w[u], xm, brow, cs & ~rows, lane, emit);
                    if (rows) half_stream<DT, true>(pl, d.ws.x_dense, tagged, w[u], xm, brow, rows, lane, emit);
                    if (mk) heavy = false;
                    __syncwarp();
                }
            }
            uint32_t hv = __ballot_sync(FULL, heavy);
            // sparse local mask -> lane-owned form; dense local mask -> warp form (Section 3.3.3:
            // the number of active entries of the vector block picks the microkernel)
            const bool lane_form = heavy && type != DBSPMSPV_BLK_COO && __popc(xm) < popc_threshold;
            const uint32_t hv_mask = HV ? __ballot_sync(FULL, lane_form) : 0u;
            if (HV && __popc(hv_mask) >= HEAVY_LANE_MIN) {
                // many mask-based blocks side by side: every lane walks its own block
                if (lane_form) {
                    const uint8_t *blk = pl + (size_t)w[u] * 4;
                    float *acc = s_lacc + lane;
                    uint32_t hits;
                    if (DT == DBSPMSPV_PATTERN) {
                        hits = lane_heavy_bool(type, blk, xm);
                    } else {
#pragma unroll
                        for (int r = 0; r < 16; ++r) acc[r * LANE_ACC_STRIDE] = 0.f;
                        hits = lane_heavy<DT>(type, blk, xm, s_x, acc);
                    }
                    for (uint32_t hh = hits; hh; hh &= hh - 1) {
                        const int r = __ffs(hh) - 1;
                        if (DT != DBSPMSPV_PATTERN) atomicAdd(out.acc + (size_t)brow * 16 + r, acc[r * LANE_ACC_STRIDE]);
                        if (Out::MASKS) out.hit8[(size_t)brow * 16 + r] = 1;
                    }
                }
                __syncwarp();
                hv &= ~hv_mask;   // oversized COO blocks (forced format) stay with the warp form
            }
            while (hv) {
                const int src = __ffs(hv) - 1;
                hv &= hv - 1;
                const uint32_t bidx = __shfl_sync(FULL, idx[u], src);
                const uint32_t bw = __shfl_sync(FULL, w[u], src);
                const int nnz = (int)__shfl_sync(FULL, aux[u], src) + 1;
                const int btype = bidx >> TYPE_SHIFT;
                const int bbrow = bidx & IDX_MASK;
                const uint8_t *blk = pl + (size_t)bw * 4;
                uint32_t hits;
                float sum = 0.f;
                if (DT == DBSPMSPV_PATTERN) hits = warp_block_bool<DT>(btype, blk, nnz, xm, lane);
                else sum = warp_block<DT>(btype, blk, nnz, xm, s_x, s_tmp, lane, popc_threshold, hits);
                flush_rows(out, bbrow, hits, sum, lane);
            }
        }
        __syncwarp();
    }
}

// Pull (Section 3.3.2).  The block-CSR view is streamed through shared memory: every warp owns
// a double-buffered stage (Section 3.3.3) that one lane fills with three bulk copies (index,
// word and aux arrays of one chunk of consecutive segments) while the warp works on the other
// stage.  Inside a chunk the lanes run over the entries 32 at a time, whatever segment they
// belong to: the first entry of every segment carries a flag bit, so a ballot and a popcount
// give each lane its segment, hence its row block.  Writeback is hierarchical where it pays:
// the segment the warp is currently "in" accumulates its 16 partial sums in shared memory
// (long hub row blocks stay there over many steps); products of the other, short segments met
// in the same step go straight to global atomics.  INLINE entries need one gather only: the
// dense copy of x carries a "not listed" marker, so presence and value come from one load.
#ifndef DBS_PULL_UNROLL
#define DBS_PULL_UNROLL 2
#endif
constexpr int PULL_UNROLL = DBS_PULL_UNROLL;
#ifndef DBS_SY_COPIES
#define DBS_SY_COPIES 4
#endif
constexpr int SY_COPIES = DBS_SY_COPIES;  // copies of the pull accumulator per warp (power of two, <= 32)
constexpr uint32_t SEG_FLAG = 1u << 28;   // view entry starts a pull segment (block-CSR view only)

// lane 0 issues the copies of the chunk [e0, e1) into stage st
__device__ __forceinline__ void pull_issue(const Device &d, int e0, int e1, PullStage *st, uint64_t *bar, int lane) {
    const int a0 = e0 & ~15, a1 = (e1 + 15) & ~15;
    if (lane == 0 && e1 > e0 && DBS_CHK_RANGE(d, e0, e1 - e0)) {      // same condition as the consumer's wait
        const uint32_t n = (uint32_t)(a1 - a0);
        fence_proxy_async_smem();
        mbar_arrive_expect_tx(bar, n * 9u);
        bulk_copy_g2s(st->idx, d.csr.idx + a0, n * 4u, bar);
        bulk_copy_g2s(st->w, d.csr.w + a0, n * 4u, bar);
        bulk_copy_g2s(st->aux, d.csr.aux + a0, n, bar);
    }
}

template <int DT, typename Out, bool HV>
__device__ void pull_body(const Device &d, Out out, int popc_threshold, float *s_x, float *s_tmp,
                          float *s_y, float *s_lacc, PullWarp *pw) {
    const int lane = threadIdx.x & 31;
    const uint32_t le_mask = 0xFFFFFFFFu >> (31 - lane);
    const int gwarp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    if (lane == 0) { mbar_init(&pw->bar[0], 1); mbar_init(&pw->bar[1], 1); fence_barrier_init(); }
    // the shared accumulator is kept in SY_COPIES copies, each fed by its own group of lanes:
    // fewer lanes per address means fewer retries of the shared-memory fp32 atomic
    for (int k = lane; k < 16 * SY_COPIES; k += 32) s_y[k] = 0.f;
    float *const my_y = s_y + (lane / (32 / SY_COPIES)) * 16;
    __syncwarp();
    uint32_t parity = 0u;             // bit s: phase parity of stage s
    int cur = 0;
    bool next_in_flight = false;
    int2 c0 = make_int2(0, 0), c1 = c0, n0 = c0, n1 = c0;
    if (gwarp < d.n_chunks) {
        c0 = d.chunks[gwarp]; c1 = d.chunks[gwarp + 1];
        pull_issue(d, c0.y, c1.y, &pw->stage[0], &pw->bar[0], lane);
    }
    if (gwarp + nwarps < d.n_chunks) { n0 = d.chunks[gwarp + nwarps]; n1 = d.chunks[gwarp + nwarps + 1]; }
    for (int c = gwarp; c < d.n_chunks; c += nwarps) {
        const int e0 = c0.y, e1 = c1.y, a0 = e0 & ~15;
        int ord_base = c0.x - 1;          // segment of the entry just before the current step
        // prefetch: next chunk's copies, and the descriptor of the one after
        const int cn = c + nwarps;
        next_in_flight = cn < d.n_chunks;
        if (next_in_flight) pull_issue(d, n0.y, n1.y, &pw->stage[cur ^ 1], &pw->bar[cur ^ 1], lane);
        c0 = n0; c1 = n1;
        if (cn + nwarps < d.n_chunks) { n0 = d.chunks[cn + nwarps]; n1 = d.chunks[cn + nwarps + 1]; }
        if (e1 > e0) {
            if (!mbar_wait_bounded(&pw->bar[cur], (parity >> cur) & 1u)) {
                d.ws.ctr->status = DBSPMSPV_ERR_TIMEOUT;
                break;
            }
            parity ^= 1u << cur;
        }
        const PullStage *st = &pw->stage[cur];
        int cur_rb = -1;                  // row block held in the shared accumulator
        int last_rb = -1;                 // row block of segment ord_base
        uint32_t hit = 0;
        for (int base = e0; base < e1; base += 32 * PULL_UNROLL) {
            uint32_t idx[PULL_UNROLL], w[PULL_UNROLL], aux[PULL_UNROLL];
            float xin[PULL_UNROLL];
#pragma unroll
            for (int u = 0; u < PULL_UNROLL; ++u) {
                const int p = base + u * 32 + lane;
                idx[u] = 0; w[u] = 0; aux[u] = 0;
                if (p < e1) { const int o = p - a0; idx[u] = st->idx[o]; w[u] = st->w[o]; aux[u] = st->aux[o]; DBS_CHK_ENTRY(d, true, idx[u], w[u], aux[u]); }
            }
#pragma unroll
            for (int u = 0; u < PULL_UNROLL; ++u) {
                const bool have = base + u * 32 + lane < e1;
                // (L2-only load: the 4-byte gathers hit L1 one time in ten and only evict each other there)
                xin[u] = have ? __ldcg(&d.ws.x_dense[(size_t)(idx[u] & IDX_MASK) * 16 + (aux[u] & 15)])
                             : __uint_as_float(X_ABSENT);
            }
#pragma unroll
            for (int u = 0; u < PULL_UNROLL; ++u) {
                if (base + u * 32 >= e1) break;   // warp-uniform
                const bool have = base + u * 32 + lane < e1;
                const uint32_t fb = __ballot_sync(FULL, (idx[u] & SEG_FLAG) != 0u);   // idx is 0 past the end
                // Most steps lie inside one segment (long row blocks are cut into segments of whole
                // steps): then the row block is warp-uniform and known without a per-lane lookup.
                const bool one_seg = (fb & ~1u) == 0u;
                int rb, rb0;
                if (one_seg) {
                    if (fb) last_rb = d.seg_rb[++ord_base];
                    rb = rb0 = last_rb;
                } else {
                    const int ord = ord_base + __popc(fb & le_mask);
                    ord_base += __popc(fb);
                    rb = have ? d.seg_rb[ord] : 0;
                    rb0 = __shfl_sync(FULL, rb, 0);
                    last_rb = __shfl_sync(FULL, rb, 31);   // (past the end only in the chunk's last step)
                }
                // the shared accumulator follows the row block of the step's first entry (a long
                // row block keeps it over all its segments of the chunk)
                if (rb0 != cur_rb) {
                    hit = __reduce_or_sync(FULL, hit);
                    __syncwarp();
                    if (lane < 16) {
                        if ((hit >> lane) & 1u) {
                            if (DT != DBSPMSPV_PATTERN) {
                                float t = 0.f;
#pragma unroll
                                for (int k = 0; k < SY_COPIES; ++k) { t += s_y[k * 16 + lane]; s_y[k * 16 + lane] = 0.f; }
                                atomicAdd(out.acc + (size_t)cur_rb * 16 + lane, t);
                            }
                            if (Out::MASKS) out.hit8[(size_t)cur_rb * 16 + lane] = 1;
                        }
                    }
                    hit = 0;
                    cur_rb = rb0;
                    __syncwarp();
                }
                const int type = idx[u] >> TYPE_SHIFT;
                const bool inl = type == DBSPMSPV_BLK_INLINE;
                if (inl && __float_as_uint(xin[u]) != X_ABSENT) {    // absent also covers "past the end"
                    const float v = Val<DT>::inline_value(w[u]) * xin[u];
                    const int r = aux[u] >> 4;
                    if (one_seg || rb == cur_rb) {
                        if (DT != DBSPMSPV_PATTERN) atomicAdd(&my_y[r], v);
                        hit |= 1u << r;
                    } else {
                        if (DT != DBSPMSPV_PATTERN) atomicAdd(out.acc + (size_t)rb * 16 + r, v);
                        if (Out::MASKS) out.hit8[(size_t)rb * 16 + r] = 1;
                    }
                }
                const bool other = have && !inl;
                if (!__any_sync(FULL, other)) continue;
                // classes that go through the vector-block mask; they write straight to global
                const int bcol_l = idx[u] & IDX_MASK;
                const uint32_t xm = other ? mask_of(d.ws.x_mask32, bcol_l) : 0u;
                bool heavy = false;
                int coo_cnt = 0;
                if (xm) {
                    if (type == DBSPMSPV_BLK_COO && aux[u] < COO_SERIAL_MAX) {
                        coo_cnt = (int)aux[u] + 1;
                    } else {
                        heavy = true;
                    }
                }
                if (__any_sync(FULL, coo_cnt)) {
                    uint32_t *s_hit = reinterpret_cast<uint32_t *>(s_tmp);   // per-owner-lane hit masks
                    s_hit[lane] = 0u;
                    __syncwarp();
                    warp_flat_coo<DT>(coo_cnt, w[u], xm, (uint32_t)rb, (uint32_t)bcol_l, d.payload, lane,
                                      [&](uint32_t trb, uint32_t tcol, int r, int c, float a, int owner) {
                                          if (DT != DBSPMSPV_PATTERN)
                                              atomicAdd(out.acc + (size_t)trb * 16 + r, a * d.ws.x_dense[(size_t)tcol * 16 + c]);
                                          if (Out::MASKS) atomicOr(&s_hit[owner], 1u << r);
                                      });
                    __syncwarp();
                    if (Out::MASKS && coo_cnt && s_hit[lane]) mark_rows(out.hit8, rb, s_hit[lane]);
                    __syncwarp();
                }
                // runs of mask-based blocks (pruned layers, banded matrices): half-warp streaming form
                if (HV && DT != DBSPMSPV_PATTERN) {
                    const bool mk = heavy && type != DBSPMSPV_BLK_COO;
                    const uint32_t cs = __ballot_sync(FULL, mk);
                    if (__popc(cs) >= HEAVY_LANE_MIN) {
                        auto emit = [&](int erb, int erow, float esum) {
                            if (erb == cur_rb) {
                                atomicAdd(&my_y[erow], esum);
                                hit |= 1u << erow;
                            } else {
                                atomicAdd(out.acc + (size_t)erb * 16 + erow, esum);
                                if (Out::MASKS) out.hit8[(size_t)erb * 16 + erow] = 1;
                            }
                        };
                        const uint32_t rows = __ballot_sync(FULL, mk && is_row_major(type));
                        if (cs & ~rows) half_stream<DT, false>(d.payload, d.ws.x_dense, idx[u], w[u], xm, rb, cs & ~rows, lane, emit);
                        if (rows) half_stream<DT, true>(d.payload, d.ws.x_dense, idx[u], w[u], xm, rb, rows, lane, emit);
                        if (mk) heavy = false;
                        __syncwarp();
                    }
                }
                uint32_t hv = __ballot_sync(FULL, heavy);
                // sparse local mask -> lane-owned form; dense local mask -> warp form
                const bool lane_form = heavy && type != DBSPMSPV_BLK_COO && __popc(xm) < popc_threshold;
                const uint32_t hv_mask = HV ? __ballot_sync(FULL, lane_form) : 0u;
                if (HV && __popc(hv_mask) >= HEAVY_LANE_MIN) {
                    // Mask-based blocks side by side under sparse local masks (banded matrices at
                    // run ends): every lane walks its own block and leaves 16 partial sums in its
                    // private scratch column, so the warp keeps up to 32 blocks going.  Blocks of
                    // the row block held in the shared accumulator are then summed across lanes
                    // by 16 lanes (no atomics); blocks of other row blocks go straight to global.
                    float *acc = s_lacc + lane;
                    uint32_t hits = 0;
                    if (lane_form) {
                        const uint8_t *blk = d.payload + (size_t)w[u] * 4;
                        if (DT == DBSPMSPV_PATTERN) {
                            hits = lane_heavy_bool(type, blk, xm);
                        } else {
#pragma unroll
                            for (int r = 0; r < 16; ++r) acc[r * LANE_ACC_STRIDE] = 0.f;
                            hits = lane_heavy<DT>(type, blk, xm, d.ws.x_dense + (size_t)bcol_l * 16, acc);
                        }
                    }
                    const bool in_cur = lane_form && rb == cur_rb;
                    const uint32_t members = __ballot_sync(FULL, in_cur);
                    __syncwarp();
                    if (in_cur) hit |= hits;
                    if (DT != DBSPMSPV_PATTERN && members && lane < 16) {
                        float t = 0.f;
                        for (uint32_t mm = members; mm; mm &= mm - 1) t += s_lacc[lane * LANE_ACC_STRIDE + __ffs(mm) - 1];
                        s_y[lane] += t;
                    }
                    if (lane_form && !in_cur) {
                        for (uint32_t hh = hits; hh; hh &= hh - 1) {
                            const int r = __ffs(hh) - 1;
                            if (DT != DBSPMSPV_PATTERN) atomicAdd(out.acc + (size_t)rb * 16 + r, acc[r * LANE_ACC_STRIDE]);
                            if (Out::MASKS) out.hit8[(size_t)rb * 16 + r] = 1;
                        }
                    }
                    __syncwarp();
                    hv &= ~hv_mask;
                }
                while (hv) {
                    const int src = __ffs(hv) - 1;
                    hv &= hv - 1;
                    const uint32_t bidx = __shfl_sync(FULL, idx[u], src);
                    const uint32_t bw = __shfl_sync(FULL, w[u], src);
                    const int nnz = (int)__shfl_sync(FULL, aux[u], src) + 1;
                    const uint32_t bxm = __shfl_sync(FULL, xm, src);
                    const int brb = __shfl_sync(FULL, rb, src);
                    const int btype = bidx >> TYPE_SHIFT;
                    const int bcol = bidx & IDX_MASK;
                    const uint8_t *blk = d.payload + (size_t)bw * 4;
                    uint32_t hits;
                    float sum = 0.f;
                    if (DT == DBSPMSPV_PATTERN) {
                        hits = warp_block_bool<DT>(btype, blk, nnz, bxm, lane);
                    } else {
                        __syncwarp();
                        if (lane < 16) s_x[lane] = d.ws.x_dense[(size_t)bcol * 16 + lane];
                        __syncwarp();
                        sum = warp_block<DT>(btype, blk, nnz, bxm, s_x, s_tmp, lane, popc_threshold, hits);
                    }
                    flush_rows(out, brb, hits, sum, lane);
                }
            }
        }
        // end of the chunk: flush what the shared accumulator still holds
        hit = __reduce_or_sync(FULL, hit);
        __syncwarp();
        if (lane < 16) {
            if ((hit >> lane) & 1u) {
                if (DT != DBSPMSPV_PATTERN) {
                    float t = 0.f;
#pragma unroll
                    for (int k = 0; k < SY_COPIES; ++k) { t += s_y[k * 16 + lane]; s_y[k * 16 + lane] = 0.f; }
                    atomicAdd(out.acc + (size_t)cur_rb * 16 + lane, t);
                }
                if (Out::MASKS) out.hit8[(size_t)cur_rb * 16 + lane] = 1;
            }
        }
        __syncwarp();
        cur ^= 1;
        next_in_flight = false;
    }
    // left early on a timeout: let the copy still in flight land before the stage memory is
    // given back (bounded, like every wait here)
    if (next_in_flight) mbar_wait_bounded(&pw->bar[cur ^ 1], (parity >> (cur ^ 1)) & 1u);
}

// Global selector (Section 3.3.1): s_b = N_nzblk / N_blk; push iff s_b < th3.  Evaluated on
// the device by every thread block from the counter the blocking kernel produced.
__device__ __forceinline__ int select_path(const Device &d, float th3, int force_path) {
    if (force_path == DBSPMSPV_PATH_PUSH || force_path == DBSPMSPV_PATH_PULL) return force_path;
    const float sb = (float)d.ws.ctr->n_nzblk / (float)d.nb;
    return sb < th3 ? DBSPMSPV_PATH_PUSH : DBSPMSPV_PATH_PULL;
}

#ifndef DBS_MIN_CTAS
#define DBS_MIN_CTAS 1
#endif
// (MODE 1: five resident thread blocks per SM -- a cap of 102 registers -- measured 7 - 10 % faster
// than the compiler's own 107 registers and four thread blocks once the push stages its payload)
#ifndef DBS_MIN_CTAS_HEAVY
#define DBS_MIN_CTAS_HEAVY 5
#endif
// Variants of the traversal kernel, chosen per handle from the class census at create:
//   MODE 0  hypersparse matrices (power-law graphs): the push only -- their pull is the
//           streaming kernel k_pull_lean, launched next in the stream
//   MODE 1  matrices whose elements sit mostly in mask-based blocks (pruned layers, banded
//           matrices): half-warp streaming and lane-owned microkernels
// Dynamic shared memory: per-warp pull stages (the push stages payload there) | lane scratch of the lane-owned form (MODE 1).
template <int MODE> constexpr size_t compute_dyn_smem() {
    return MODE >= 1 ? WARPS * sizeof(PullWarp) + WARPS * 16 * LANE_ACC_STRIDE * sizeof(float) : 0;
}

template <int DT, typename Out, int MODE>
__global__ void __launch_bounds__(CTA, MODE >= 1 ? DBS_MIN_CTAS_HEAVY : DBS_MIN_CTAS) k_compute(Device d, Out out, float th3, int force_path, int popc_threshold, int pull_done) {
    constexpr bool HV = MODE >= 1;
    __shared__ float s_x[WARPS][16], s_tmp[WARPS][32], s_y[HV ? WARPS : 1][16 * SY_COPIES];
    extern __shared__ __align__(128) uint8_t s_dyn[];
    PullWarp *s_pull = reinterpret_cast<PullWarp *>(s_dyn);
    float *s_lacc = reinterpret_cast<float *>(s_dyn + WARPS * sizeof(PullWarp));
    const int warp = threadIdx.x >> 5;
    pdl_wait();
    pdl_launch_dependents();
    const int path = select_path(d, th3, force_path);
    if (blockIdx.x == 0 && threadIdx.x == 0) d.ws.ctr->path = path;
    float *lacc = HV ? s_lacc + warp * 16 * LANE_ACC_STRIDE : nullptr;
    if (pull_done && path == DBSPMSPV_PATH_PULL) return;     // (the decode entry's own pull kernel has run)
    if (path == DBSPMSPV_PATH_PUSH) push_body<DT, Out, HV>(d, out, popc_threshold, s_x[warp], s_tmp[warp], lacc, HV ? &s_pull[warp] : nullptr);
    else if (HV) pull_body<DT, Out, HV>(d, out, popc_threshold, s_x[warp], s_tmp[warp], s_y[warp], lacc, &s_pull[warp]);
    // (MODE 0: the pull is k_pull_lean's)
}

// Pull of the decode entry for matrices whose elements sit mostly in mask-based blocks (pruned
// layers).  A warp takes 32 consecutive entries of the block-CSR view, one block per lane.  A
// lane walks the active columns of its own column-major or Dense block and keeps the 16 row sums
// in registers (a Dense column is two 16-byte loads for bf16); with activations 10 % dense a block
// has one or two active columns, and a step serves 32 blocks with the instructions the half-warp
// form spends on two.  When the 32 entries share a row block -- always, for the layer shapes of
// Section 4.3 -- the 32 x 16 sums are folded by 16 shuffles into one atomic per row; otherwise every
// lane adds its own.  Row-major blocks take the half-warp streaming form, the odd COO/INLINE
// entry its own lane.  Does nothing unless the selector says pull; the general
// kernel, launched next, then only runs the push.
#ifndef DBS_LBC
#define DBS_LBC 3
#endif
constexpr int LBC = DBS_LBC;              // columns of a lane's block per pass of lane_block_columns
constexpr int LBC_SLOT_BYTES = 48;  // staging slot of a lane: 32 bytes used; the stride keeps 16-byte stores conflict-free

// Active columns of one column-major (or Dense) block, by the lane that owns it: acc[r] += A[r][c] x[c].
// The loads of up to LBC columns are issued together, level by level (x and header, then the
// values), so a pass costs two memory latencies whatever the number of columns.  bf16 values
// come in as two 16-byte loads per column -- with 32 lanes on 32 different cache lines a load
// instruction costs the same whatever its width, so element-wise loads were 8 times the L1 work.
// A compressed column (its values packed in row order from a 2-byte aligned start) is then
// expanded to its rows through the lane's own 48 bytes of shared memory: the 32 aligned bytes
// that hold it are stored there and each row with a set mask bit reads the next 2 bytes.  No
// other lane touches the slot, so no barrier is involved.
template <int DT>
__device__ __forceinline__ void lane_block_columns(const uint8_t *blk, bool dense, uint32_t xm, const float *xb,
                                                   float (&acc)[16], uint4 *slot) {
    const uint16_t *masks = reinterpret_cast<const uint16_t *>(blk);
    for (uint32_t a = xm; a;) {
        int c[LBC];
        bool on[LBC];
        float xs[LBC];
        uint32_t mc[LBC];
        int pos[LBC];
#pragma unroll
        for (int j = 0; j < LBC; ++j) { on[j] = a != 0; c[j] = on[j] ? __ffs(a) - 1 : 0; a &= a - 1; }
#pragma unroll
        for (int j = 0; j < LBC; ++j) {
            xs[j] = 0.f; mc[j] = 0u; pos[j] = 0;
            if (on[j]) {
                xs[j] = xb[c[j]];
                if (!dense) { mc[j] = masks[c[j]]; pos[j] = blk[32 + c[j]]; }
            }
        }
        if (DT == DBSPMSPV_BF16) {
            uint4 lo[LBC], hi[LBC];
            int off[LBC];          // halfword offset of the column's first value inside lo|hi
#pragma unroll
            for (int j = 0; j < LBC; ++j) {
                lo[j] = make_uint4(0u, 0u, 0u, 0u); hi[j] = lo[j]; off[j] = 0;
                if (on[j]) {
                    const int byte0 = dense ? 32 + c[j] * 32 : HDR_BYTES + ((pos[j] * 2) & ~15);
                    off[j] = dense ? 0 : pos[j] & 7;
                    const uint4 *src = reinterpret_cast<const uint4 *>(blk + byte0);
                    lo[j] = src[0]; hi[j] = src[1];       // (the payload has slack behind its last block)
                }
            }
#pragma unroll
            for (int j = 0; j < LBC; ++j) {
                if (!on[j]) continue;
                if (dense) {
                    // absent elements are stored as zeros: only a non-finite x needs the mask
                    uint32_t gate = 0xFFFFu;
                    if ((__float_as_uint(xs[j]) & 0x7F800000u) == 0x7F800000u) gate = masks[c[j]];
                    const uint32_t u[8] = {lo[j].x, lo[j].y, lo[j].z, lo[j].w, hi[j].x, hi[j].y, hi[j].z, hi[j].w};
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const float v0 = __uint_as_float(u[q] << 16), v1 = __uint_as_float(u[q] & 0xFFFF0000u);
                        if ((gate >> (2 * q)) & 1u) acc[2 * q] += v0 * xs[j];
                        if ((gate >> (2 * q + 1)) & 1u) acc[2 * q + 1] += v1 * xs[j];
                    }
                } else if (off[j] + __popc(mc[j]) <= 16) {
                    slot[0] = lo[j]; slot[1] = hi[j];
                    asm volatile("" ::: "memory");
                    const uint16_t *sv = reinterpret_cast<const uint16_t *>(slot) + off[j];
                    int i = 0;
#pragma unroll
                    for (int r = 0; r < 16; ++r)
                        if ((mc[j] >> r) & 1u) { acc[r] += __uint_as_float((uint32_t)sv[i] << 16) * xs[j]; ++i; }
                    asm volatile("" ::: "memory");
                } else {
                    // the column straddles the 32 staged bytes: element-wise
                    const uint8_t *vals = blk + HDR_BYTES;
                    int i = pos[j];
#pragma unroll
                    for (int r = 0; r < 16; ++r)
                        if ((mc[j] >> r) & 1u) { acc[r] += Val<DT>::load(vals, i) * xs[j]; ++i; }
                }
            }
        } else {
            const uint8_t *vals = blk + (dense ? 32 : HDR_BYTES);
#pragma unroll
            for (int j = 0; j < LBC; ++j) {
                if (!on[j]) continue;
                if (dense) {
                    uint32_t gate = 0xFFFFu;
                    if ((__float_as_uint(xs[j]) & 0x7F800000u) == 0x7F800000u) gate = masks[c[j]];
#pragma unroll
                    for (int r = 0; r < 16; ++r)
                        if ((gate >> r) & 1u) acc[r] += Val<DT>::load(vals, c[j] * 16 + r) * xs[j];
                } else {
                    int i = pos[j];
#pragma unroll
                    for (int r = 0; r < 16; ++r)
                        if ((mc[j] >> r) & 1u) { acc[r] += Val<DT>::load(vals, i) * xs[j]; ++i; }
                }
            }
        }
    }
}

// Sum of acc[r] over the 32 lanes, for all 16 rows: afterwards the lane pair (2k, 2k + 1) holds
// the total of row folded_row(lane).
__device__ __forceinline__ float fold_rows(const float (&acc)[16], int lane) {
    float a8[8], a4[4], a2[2];
    const bool u16 = lane & 16, u8 = lane & 8, u4 = lane & 4, u2 = lane & 2;
#pragma unroll
    for (int i = 0; i < 8; ++i) a8[i] = (u16 ? acc[i + 8] : acc[i]) + __shfl_xor_sync(FULL, u16 ? acc[i] : acc[i + 8], 16);
#pragma unroll
    for (int i = 0; i < 4; ++i) a4[i] = (u8 ? a8[i + 4] : a8[i]) + __shfl_xor_sync(FULL, u8 ? a8[i] : a8[i + 4], 8);
#pragma unroll
    for (int i = 0; i < 2; ++i) a2[i] = (u4 ? a4[i + 2] : a4[i]) + __shfl_xor_sync(FULL, u4 ? a4[i] : a4[i + 2], 4);
    const float a1 = (u2 ? a2[1] : a2[0]) + __shfl_xor_sync(FULL, u2 ? a2[0] : a2[1], 2);
    return a1 + __shfl_xor_sync(FULL, a1, 1);
}
__device__ __forceinline__ int folded_row(int lane) { return ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1); }

template <int DT>
__global__ void __launch_bounds__(CTA) k_decode_pull(Device d, const int32_t *__restrict__ entry_row,
                                                     float *__restrict__ y, float th3, int force_path) {
    __shared__ __align__(16) uint8_t s_slots[CTA * LBC_SLOT_BYTES];
    pdl_wait();
    pdl_launch_dependents();
    if (select_path(d, th3, force_path) != DBSPMSPV_PATH_PULL) return;
    if (blockIdx.x == 0 && threadIdx.x == 0) d.ws.ctr->path = DBSPMSPV_PATH_PULL;
    const int lane = threadIdx.x & 31;
    uint4 *slot = reinterpret_cast<uint4 *>(s_slots + threadIdx.x * LBC_SLOT_BYTES);
    const int gwarp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    const int n_tasks = (d.n_entries + 31) >> 5;
    auto emit = [&](int erb, int erow, float esum) { atomicAdd(y + (size_t)erb * 16 + erow, esum); };
    for (int task = gwarp; task < n_tasks; task += nwarps) {
        const int p = task * 32 + lane;
        const bool have = p < d.n_entries;
        uint32_t idx = 0, w = 0, aux = 0, xm = 0;
        int rb = -1;
        if (have) {
            idx = d.csr.idx[p]; w = d.csr.w[p]; aux = d.csr.aux[p]; rb = entry_row[p];
            DBS_CHK_ENTRY(d, true, idx, w, aux);
            if (!DBS_CHK_INDEX(d, rb, d.mb)) rb = 0;
            xm = mask_of(d.ws.x_mask32, idx & IDX_MASK);
        }
        const int type = idx >> TYPE_SHIFT;
        const bool mk = have && xm && type > DBSPMSPV_BLK_COO;
        const bool rowm = mk && is_row_major(type);
        const float *xb = d.ws.x_dense + (size_t)(idx & IDX_MASK) * 16;
        float acc[16];
#pragma unroll
        for (int r = 0; r < 16; ++r) acc[r] = 0.f;
        if (mk && !rowm) lane_block_columns<DT>(d.payload + (size_t)w * 4, type == DBSPMSPV_BLK_DENSE, xm, xb, acc, slot);
        __syncwarp();
        const int rb0 = __shfl_sync(FULL, rb, 0);
        if (__all_sync(FULL, rb == rb0)) {
            const float total = fold_rows(acc, lane);
            if (!(lane & 1) && total != 0.f) atomicAdd(y + (size_t)rb0 * 16 + folded_row(lane), total);
        } else if (mk && !rowm) {
#pragma unroll
            for (int r = 0; r < 16; ++r)
                if (acc[r] != 0.f) atomicAdd(y + (size_t)rb * 16 + r, acc[r]);
        }
        const uint32_t rows = __ballot_sync(FULL, rowm);
        if (rows) half_stream<DT, true>(d.payload, d.ws.x_dense, idx, w, xm, rb, rows, lane, emit);
        if (have && xm && type <= DBSPMSPV_BLK_COO) {       // the odd hypersparse block: its own lane
            float *row0 = y + (size_t)rb * 16;
            if (type == DBSPMSPV_BLK_INLINE) {
                if ((xm >> (aux & 15)) & 1u) atomicAdd(row0 + (aux >> 4), Val<DT>::inline_value(w) * xb[aux & 15]);
            } else {
                const int nnz = (int)aux + 1;
                const uint8_t *blk = d.payload + (size_t)w * 4, *vals = blk + ((nnz + 3) & ~3);
                for (int k = 0; k < nnz; ++k) {
                    const int c = blk[k] & 15, r = blk[k] >> 4;
                    if ((xm >> c) & 1u) atomicAdd(row0 + r, Val<DT>::load(vals, k) * xb[c]);
                }
            }
        }
    }
}

// Active columns of the column-major and Dense blocks of one warp step, when all 32 blocks lie in
// ONE row block: then any lane may take any (block, column) pair -- its 16 sums go into the
// same rows -- and the pairs are dealt out evenly, 32 per round, instead of every lane walking
// the columns of its own block (with activations 10 % dense a block has 1.6 active columns on
// average but the busiest of 32 has five).  `cols` is the lane's own block's active-column mask
// (0: not a block of these classes).  Column values are fetched and expanded as in
// lane_block_columns, Dense columns through the same staged form.
// WC_ILP = (block, column) pairs a lane works on at a time: 2 where a warp has several steps per
// row block (wide layers: measured 45 -> 41 us on 4096 x 11008), 1 where it has one or two
// (12288 x 4096: 2 measured 10 % slower).
__host__ __device__ constexpr int wc_ilp(int warps_per_block) { return warps_per_block >= 8 ? 2 : 1; }
// staging bytes per lane; the stride keeps 16-byte stores conflict-free
__host__ __device__ constexpr int wc_slot_bytes(int ilp) { return 48 * ilp + (ilp > 1 ? 16 : 0); }

// DIRECT: the payload lies in shared memory, so the values are indexed where they are (no staging slot).
template <int DT, int WC_ILP, bool DIRECT = false>
__device__ __forceinline__ void warp_columns(const uint8_t *payload, const float *x_blocks, uint32_t idx, uint32_t w,
                                             uint32_t cols, int lane, float (&acc)[16], uint4 *slot) {
    int incl = __popc(cols);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(FULL, incl, o);
        if (lane >= o) incl += t;
    }
    const int excl = incl - __popc(cols);
    const int total = __shfl_sync(FULL, incl, 31);
    for (int k0 = 0; k0 < total; k0 += 32 * WC_ILP) {
        // WC_ILP pairs per lane and round, worked on side by side: their dependent loads (header ->
        // values -> staged expansion) overlap
        bool on[WC_ILP], dense[WC_ILP];
        uint32_t m[WC_ILP], bidx[WC_ILP], bw[WC_ILP], gate[WC_ILP];
        int j[WC_ILP], pos[WC_ILP];
        float xv[WC_ILP];
        const uint8_t *blk[WC_ILP];
#pragma unroll
        for (int u = 0; u < WC_ILP; ++u) {
            const int k = k0 + 32 * u + lane;
            int b = 0;                   // owner of pair k: the last lane whose exclusive prefix is <= k
#pragma unroll
            for (int s = 16; s; s >>= 1) {
                const int t = __shfl_sync(FULL, excl, b + s);
                if (t <= k) b += s;
            }
            m[u] = __shfl_sync(FULL, cols, b);
            j[u] = k - __shfl_sync(FULL, excl, b);
            bidx[u] = __shfl_sync(FULL, idx, b);
            bw[u] = __shfl_sync(FULL, w, b);
            on[u] = k < total;
        }
#pragma unroll
        for (int u = 0; u < WC_ILP; ++u) {
            gate[u] = 0u; pos[u] = 0; xv[u] = 0.f; dense[u] = false; blk[u] = payload;
            if (on[u]) {
                uint32_t mm = m[u];
                for (int t = 0; t < j[u]; ++t) mm &= mm - 1;
                const int c = __ffs(mm) - 1;   // the j-th active column of that block
                dense[u] = (bidx[u] >> TYPE_SHIFT) == DBSPMSPV_BLK_DENSE;
                blk[u] = payload + (size_t)bw[u] * 4;
                xv[u] = x_blocks[(size_t)(bidx[u] & IDX_MASK) * 16 + c];
                // absent elements of a Dense block are stored as zeros: only a non-finite x needs its mask
                const bool finite = (__float_as_uint(xv[u]) & 0x7F800000u) != 0x7F800000u;
                gate[u] = dense[u] && finite ? 0xFFFFu : reinterpret_cast<const uint16_t *>(blk[u])[c];
                pos[u] = dense[u] ? c * 16 : blk[u][32 + c];
            }
        }
        if (DT == DBSPMSPV_BF16 && !DIRECT) {
            int off[WC_ILP];
#pragma unroll
            for (int u = 0; u < WC_ILP; ++u) {
                off[u] = pos[u] & 7;
                if (on[u]) {
                    const int nvals = dense[u] ? 16 : __popc(gate[u]);
                    const uint4 *src = reinterpret_cast<const uint4 *>(blk[u] + (dense[u] ? 32 : HDR_BYTES) + ((pos[u] * 2) & ~15));
                    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                    const uint4 q0 = src[0], q1 = off[u] + nvals > 8 ? src[1] : zero, q2 = off[u] + nvals > 16 ? src[2] : zero;
                    slot[3 * u] = q0; slot[3 * u + 1] = q1; slot[3 * u + 2] = q2;
                }
            }
            asm volatile("" ::: "memory");
            int i[WC_ILP];
#pragma unroll
            for (int u = 0; u < WC_ILP; ++u) i[u] = 0;
#pragma unroll
            for (int r = 0; r < 16; ++r) {
#pragma unroll
                for (int u = 0; u < WC_ILP; ++u) {
                    const uint16_t *sv = reinterpret_cast<const uint16_t *>(slot + 3 * u) + off[u];
                    const uint32_t bit = (gate[u] >> r) & 1u;
                    if (bit) acc[r] += __uint_as_float((uint32_t)sv[i[u]] << 16) * xv[u];
                    i[u] += (int)bit | (dense[u] ? 1 : 0);
                }
            }
            asm volatile("" ::: "memory");
        } else {
#pragma unroll
            for (int u = 0; u < WC_ILP; ++u) {
                const uint8_t *vals = blk[u] + (dense[u] ? 32 : HDR_BYTES);
                int i = pos[u];
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                    const uint32_t bit = (gate[u] >> r) & 1u;
                    if (bit) acc[r] += Val<DT>::load(vals, i) * xv[u];
                    i += (int)bit | (dense[u] ? 1 : 0);
                }
            }
        }
    }
}

// x -> 16-bit masks and fp32 blocks in shared memory (absent entries carry the marker), by all
// `threads` threads of the block; s_cnt[0] and s_cnt[1] (zeroed by the caller, barrier in
// between) receive the numbers of nonzero vector blocks and of nonzero elements.  The caller synchronises afterwards.
template <int DT>
__device__ __forceinline__ void stage_x_blocks(const Device &d, const void *__restrict__ x, float *s_x, uint16_t *s_xm,
                                               int *s_cnt, int tid, int T) {
    const int lane = tid & 31;
    const bool aligned = (reinterpret_cast<uintptr_t>(x) & 15u) == 0;
    // (a bf16 handle may be given its x in fp32 -- the fp32 output of the layer before --, which
    // is rounded to bf16 here, to nearest even, so that the products stay exact)
    const bool x16 = DT == DBSPMSPV_BF16 && !d.decode_x_f32;
    int mine = 0;
    for (int cb = tid; cb < d.nb; cb += T) {
        const int64_t j0 = (int64_t)cb * 16;
        float v[16];
        if (aligned && j0 + 16 <= d.n) {
            if (x16) {
                const uint4 *src = reinterpret_cast<const uint4 *>(static_cast<const uint16_t *>(x) + j0);
                const uint4 a = src[0], b = src[1];
                const uint32_t u[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
                for (int q = 0; q < 8; ++q) { v[2 * q] = __uint_as_float(u[q] << 16); v[2 * q + 1] = __uint_as_float(u[q] & 0xFFFF0000u); }
            } else {
                const float4 *src = reinterpret_cast<const float4 *>(static_cast<const float *>(x) + j0);
#pragma unroll
                for (int q = 0; q < 4; ++q) { const float4 f = src[q]; v[4 * q] = f.x; v[4 * q + 1] = f.y; v[4 * q + 2] = f.z; v[4 * q + 3] = f.w; }
            }
        } else {
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                v[k] = 0.f;
                if (j0 + k < d.n) v[k] = x16 ? __uint_as_float((uint32_t) static_cast<const uint16_t *>(x)[j0 + k] << 16)
                                             : static_cast<const float *>(x)[j0 + k];
            }
        }
        uint32_t bits = 0;
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            if (DT == DBSPMSPV_BF16 && !x16) v[k] = __bfloat162float(__float2bfloat16_rn(v[k]));
            const bool nz = decode_takes_part(d, v[k]);
            bits |= (nz ? 1u : 0u) << k;
            // (a widened bf16 has zero low bits: it cannot collide with the marker)
            if (DT != DBSPMSPV_BF16 && __float_as_uint(v[k]) == X_ABSENT) v[k] = __uint_as_float(0x7FC00000u);
            v[k] = nz ? v[k] : __uint_as_float(X_ABSENT);
        }
        float4 *dst = reinterpret_cast<float4 *>(s_x + j0);
#pragma unroll
        for (int q = 0; q < 4; ++q) dst[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        s_xm[cb] = (uint16_t)bits;
        mine += (bits != 0) | (__popc(bits) << 16);           // nonzero blocks, nonzero elements
    }
    mine = __reduce_add_sync(FULL, mine);
    if (lane == 0 && mine) { atomicAdd(&s_cnt[0], mine & 0xFFFF); atomicAdd(&s_cnt[1], mine >> 16); }
}

// Streaming reads the whole payload whatever x holds; the single-kernel form above fetches only
// the columns x reaches, which is less than half of the bytes once x has fewer nonzero elements
// than this share (measured on the three layer shapes: 22.6 against 27.6 us at 10 %, 37.9
// against 33.8 us at 30 %).  The choice follows the x of the handle's previous decode call --
// both kernels report the number of nonzero elements they saw through a word of mapped host
// memory, read without waiting: activations of one layer keep their sparsity from token to token.
constexpr float STREAM_MIN_X_DENSITY = 0.15f;

// The whole decode call in one kernel, for payload-dominated handles whose x fits in shared
// memory (Section 4.3: one layer, one token).  One thread block per row block.  Every block
// first reads the dense activation vector itself -- a few KB -- into shared memory as the
// vector-block masks and the fp32 x blocks the microkernels expect, counts the nonzero vector
// blocks and evaluates the selector; nothing of that touches the handle's workspace, so there
// is no blocking kernel before and no cleanup after.
//   pull: the warps take the row block's view entries 32 at a time, one block per lane (see
//         k_decode_pull);
//   push: the lanes take the nonzero vector blocks instead and look their column block up in
//         the row block's entries (sorted by column block) by bisection, so only blocks under a
//         nonzero vector block are fetched.
// The 16 row sums are folded over the warp, added up over the warps in shared memory and
// stored: a thread block owns its rows, so y needs neither zeroing nor atomics.
struct FusedLayout {
    int x_bytes, slot_off, part_off, y_off, cnt_off, active_off, xm_off, total;
    __host__ __device__ FusedLayout(int nb, int threads) {
        x_bytes = nb * 64;
        slot_off = x_bytes;
        part_off = slot_off + threads * wc_slot_bytes(wc_ilp(threads / 32));
        y_off = part_off + (threads / 32) * 64;
        cnt_off = y_off + 64;
        active_off = cnt_off + 16;
        xm_off = active_off + nb * 4;
        total = (xm_off + nb * 2 + 15) & ~15;
    }
};
constexpr int FUSED_MAX_SMEM = 200 * 1024;   // of the 227 KB a thread block may have

template <int DT, int NW>
__global__ void __launch_bounds__(NW * 32, 768 / (NW * 32))
k_decode_fused(Device d, const void *__restrict__ x, float *__restrict__ y, float th3, int force_path) {
    extern __shared__ __align__(16) uint8_t s_dyn[];
    constexpr int T = NW * 32;
    const FusedLayout lay(d.nb, T);
    float *s_x = reinterpret_cast<float *>(s_dyn);
    float *s_part = reinterpret_cast<float *>(s_dyn + lay.part_off);
    float *s_y = reinterpret_cast<float *>(s_dyn + lay.y_off);
    int *s_cnt = reinterpret_cast<int *>(s_dyn + lay.cnt_off);       // [0] nonzero vector blocks
    int *s_active = reinterpret_cast<int *>(s_dyn + lay.active_off);  // their indices, ascending (push)
    uint16_t *s_xm = reinterpret_cast<uint16_t *>(s_dyn + lay.xm_off);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint4 *slot = reinterpret_cast<uint4 *>(s_dyn + lay.slot_off + tid * wc_slot_bytes(wc_ilp(NW)));
    if (tid == 0) { s_cnt[0] = 0; s_cnt[1] = 0; }
    if (tid < 16) s_y[tid] = 0.f;
    __syncthreads();

    stage_x_blocks<DT>(d, x, s_x, s_xm, s_cnt, tid, T);
    __syncthreads();
    const int n_nzblk = s_cnt[0];
    int path = force_path;
    if (path != DBSPMSPV_PATH_PUSH && path != DBSPMSPV_PATH_PULL)
        path = (float)n_nzblk / (float)d.nb < th3 ? DBSPMSPV_PATH_PUSH : DBSPMSPV_PATH_PULL;
    if (blockIdx.x == 0 && tid == 0) {
        Counters *c = d.ws.ctr;
        c->last_n_nzblk = n_nzblk; c->last_n_tasks = 0; c->last_path = path; c->last_y_nnz = (int32_t)d.m;
        // (a store to host memory: only when it changes what the host goes by)
        if (d.x_nnz_seen && ((float)s_cnt[1] < STREAM_MIN_X_DENSITY * (float)d.n) != (d.x_sparse_believed != 0)) *d.x_nnz_seen = s_cnt[1];
    }
    if (path == DBSPMSPV_PATH_PUSH) {
        if (warp == 0) {
            int count = 0;
            for (int base = 0; base < d.nb; base += 32) {
                const bool on = base + lane < d.nb && s_xm[base + lane] != 0;
                const uint32_t m = __ballot_sync(FULL, on);
                if (on) s_active[count + __popc(m & below(lane))] = base + lane;
                count += __popc(m);
            }
        }
        __syncthreads();
    }

    const int rb = blockIdx.x;
    const int begin = d.csr.ptr[rb], end = d.csr.ptr[rb + 1];
    float acc[16];
#pragma unroll
    for (int r = 0; r < 16; ++r) acc[r] = 0.f;
    auto emit = [&](int, int erow, float esum) { atomicAdd(&s_y[erow], esum); };
    // one step: the lane's entry (idx, w, aux), if `have`
    auto step = [&](uint32_t idx, uint32_t w, uint32_t aux, bool have) {
        const uint32_t xm = have ? s_xm[idx & IDX_MASK] : 0u;
        const int type = idx >> TYPE_SHIFT;
        const bool mk = have && xm && type > DBSPMSPV_BLK_COO;
        const bool rowm = mk && is_row_major(type);
        const float *xb = s_x + (size_t)(idx & IDX_MASK) * 16;
        warp_columns<DT, wc_ilp(NW)>(d.payload, s_x, idx, w, mk && !rowm ? xm : 0u, lane, acc, slot);
        __syncwarp();
        const uint32_t rows = __ballot_sync(FULL, rowm);
        if (rows) half_stream<DT, true>(d.payload, s_x, idx, w, xm, rb, rows, lane, emit);
        if (have && xm && type <= DBSPMSPV_BLK_COO) {       // the odd hypersparse block: its own lane
            if (type == DBSPMSPV_BLK_INLINE) {
                if ((xm >> (aux & 15)) & 1u) atomicAdd(&s_y[aux >> 4], Val<DT>::inline_value(w) * xb[aux & 15]);
            } else {
                const int nnz = (int)aux + 1;
                const uint8_t *blk = d.payload + (size_t)w * 4, *vals = blk + ((nnz + 3) & ~3);
                for (int k = 0; k < nnz; ++k) {
                    const int c = blk[k] & 15, r = blk[k] >> 4;
                    if ((xm >> c) & 1u) atomicAdd(&s_y[r], Val<DT>::load(vals, k) * xb[c]);
                }
            }
        }
    };
    auto fetch = [&](int p, bool have, uint32_t &idx, uint32_t &w, uint32_t &aux) {
        idx = 0; w = 0; aux = 0;
        if (have && DBS_CHK_INDEX(d, p, d.n_entries)) { idx = d.csr.idx[p]; w = d.csr.w[p]; aux = d.csr.aux[p]; DBS_CHK_ENTRY(d, true, idx, w, aux); }
    };
    if (path == DBSPMSPV_PATH_PULL) {
        // the next step's entries are fetched before this step's blocks are worked on
        uint32_t idx, w, aux, n_idx, n_w, n_aux;
        int base = begin + warp * 32;
        fetch(base + lane, base + lane < end, idx, w, aux);
        for (; base < end; base += T) {
            const int nb_ = base + T;
            fetch(nb_ + lane, nb_ + lane < end, n_idx, n_w, n_aux);
            step(idx, w, aux, base + lane < end);
            idx = n_idx; w = n_w; aux = n_aux;
        }
    } else {
        // the row block's entries with a payload are sorted by column block: [begin, pend)
        const int pend = d.csr_inl[rb];
        for (int i0 = warp * 32; i0 < n_nzblk; i0 += T) {
            int lo = 0, hi = 0;
            if (i0 + lane < n_nzblk) {
                const uint32_t cb = (uint32_t)s_active[i0 + lane];
                int a = begin, b = pend;          // first entry with column block >= cb
                while (a < b) { const int mid = a + ((b - a) >> 1); if ((d.csr.idx[mid] & IDX_MASK) < cb) a = mid + 1; else b = mid; }
                lo = a; b = pend;                 // first entry with column block > cb
                while (a < b) { const int mid = a + ((b - a) >> 1); if ((d.csr.idx[mid] & IDX_MASK) <= cb) a = mid + 1; else b = mid; }
                hi = a;
            }
            for (int t = 0; __any_sync(FULL, lo + t < hi); ++t) {
                uint32_t idx, w, aux;
                fetch(lo + t, lo + t < hi, idx, w, aux);
                step(idx, w, aux, lo + t < hi);
            }
        }
        // its INLINE elements (row by row, rare in these handles): each tested against its mask
        for (int base = pend + warp * 32; base < end; base += T) {
            uint32_t idx, w, aux;
            fetch(base + lane, base + lane < end, idx, w, aux);
            step(idx, w, aux, base + lane < end);
        }
    }
    {
        const float total = fold_rows(acc, lane);
        if (!(lane & 1)) s_part[warp * 16 + folded_row(lane)] = total;
    }
    __syncthreads();
    if (tid < 16) {
        float sum = s_y[tid];
#pragma unroll
        for (int k = 0; k < NW; ++k) sum += s_part[k * 16 + tid];
        const int64_t row = (int64_t)rb * 16 + tid;
        if (row < d.m) y[row] = sum;
    }
}

// ------------------------------------------------------------------------------------------
// Streaming decode (Section 4.3: one layer, one token) for payload-dominated handles: the whole
// call in one persistent kernel that reads the payload as a stream.
//   * The payload of a row block is one contiguous byte range; at create it is cut into chunks
//     of whole blocks (a few KB, at most 32 blocks).  The chunk list is split evenly over all
//     warps of the grid, every warp taking a contiguous piece.
//   * Every warp runs its own ring of STREAM_DEPTH stages in shared memory: one lane moves a
//     chunk's payload bytes with one bulk copy while the warp works on an earlier chunk (the
//     chunk's view entries, 9 bytes per block, are loaded into registers a round ahead).  The microkernels' chains of
//     dependent loads (entry -> header -> column start -> values) then cost shared-memory
//     latency, no load goes through the L1 tag stage one sector at a time, and HBM sees
//     sequential reads whatever the activation sparsity.
//   * x is read once per thread block (a few KB) into masks and fp32 blocks, as in the
//     single-kernel form above; the 16 row sums of a warp stay in registers while its chunks
//     belong to one row block and go to y with one atomic per row when the row block changes
//     (y is zeroed by a memset in front of the kernel).
// A call whose x fills few vector blocks (push) walks the row blocks' entries by bisection
// straight from global memory, as the single-kernel form does.
#ifndef DBS_STREAM_WARPS
#define DBS_STREAM_WARPS 16
#endif
#ifndef DBS_STREAM_BUDGET
#define DBS_STREAM_BUDGET (220 * 1024)
#endif
constexpr int STREAM_WARPS = DBS_STREAM_WARPS;
constexpr int STREAM_CTA = STREAM_WARPS * 32;
#ifndef DBS_STREAM_DEPTH
#define DBS_STREAM_DEPTH 2
#endif
constexpr int STREAM_DEPTH = DBS_STREAM_DEPTH;
constexpr int STREAM_MAX_SMEM = 227 * 1024;   // all a thread block may have
__host__ __device__ constexpr int stream_stride(int stage_bytes) { return (stage_bytes + 127) & ~127; }
struct StreamLayout {
    int xm_off, cnt_off, active_off, bar_off, ring_off, total;
    __host__ __device__ StreamLayout(int nb, int stage_bytes) {
        xm_off = nb * 64;
        cnt_off = (xm_off + nb * 2 + 15) & ~15;
        active_off = cnt_off + 16;
        bar_off = (active_off + nb * 4 + 15) & ~15;
        ring_off = (bar_off + STREAM_WARPS * STREAM_DEPTH * 8 + 127) & ~127;
        total = ring_off + STREAM_WARPS * STREAM_DEPTH * stream_stride(stage_bytes);
    }
};

template <int DT>
__global__ void __launch_bounds__(STREAM_CTA, STREAM_WARPS <= 8 ? 2 : 1)
k_decode_stream(Device d, const void *__restrict__ x, float *__restrict__ y, float th3, int force_path) {
    extern __shared__ __align__(128) uint8_t s_dyn[];
    constexpr int T = STREAM_CTA, NW = STREAM_WARPS;
    const StreamLayout lay(d.nb, d.stage_bytes);
    float *s_x = reinterpret_cast<float *>(s_dyn);
    uint16_t *s_xm = reinterpret_cast<uint16_t *>(s_dyn + lay.xm_off);
    int *s_cnt = reinterpret_cast<int *>(s_dyn + lay.cnt_off);
    int *s_active = reinterpret_cast<int *>(s_dyn + lay.active_off);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int stride = stream_stride(d.stage_bytes);
    uint64_t *s_bar = reinterpret_cast<uint64_t *>(s_dyn + lay.bar_off) + warp * STREAM_DEPTH;
    uint8_t *s_ring = s_dyn + lay.ring_off + (size_t)warp * STREAM_DEPTH * stride;
    if (tid == 0) { s_cnt[0] = 0; s_cnt[1] = 0; }

    // this warp's piece of the chunk list; lane i keeps the descriptor of its i-th chunk (32 at a time)
    const int gw = blockIdx.x * NW + warp, W = gridDim.x * NW;
    const int lo = (int)((int64_t)d.n_stage_chunks * gw / W), hi = (int)((int64_t)d.n_stage_chunks * (gw + 1) / W);
    const int n_mine = hi - lo;
    int4 my_desc = make_int4(0, 0, 0, 0);
    if (lane < n_mine) my_desc = d.stage_chunks[lo + lane];
    auto desc_of = [&](int k) {                               // (whole warp)
        return make_int4(__shfl_sync(FULL, my_desc.x, k & 31), __shfl_sync(FULL, my_desc.y, k & 31),
                         __shfl_sync(FULL, my_desc.z, k & 31), __shfl_sync(FULL, my_desc.w, k & 31));
    };
    // descriptor: x = first view entry, y = row block, z = payload offset in words, w = words | entries << 24
    auto issue = [&](const int4 &ch, int st) {               // lane 0 only
        uint8_t *base = s_ring + (size_t)st * stride;
        uint32_t pb = ((uint32_t)ch.w & 0xFFFFFFu) * 4u;
        if (!DBS_CHK_INDEX(d, pb, d.stage_bytes + 1) || !DBS_CHK_INDEX(d, (uint64_t)(uint32_t)ch.z + (pb >> 2), (uint64_t)d.payload_words + 1)) pb = 0u;
        fence_proxy_async_smem();
        mbar_arrive_expect_tx(&s_bar[st], pb);
        if (pb) bulk_copy_g2s(base, d.payload + (size_t)(uint32_t)ch.z * 4, pb, &s_bar[st]);
    };
    // the chunk's view entries, one per lane, by plain loads a round ahead of their use (they
    // are 9 bytes per block; bulk copies of 48-256 bytes cost the copy engine as much as the payload's)
    auto entries_of = [&](const int4 &ch, uint32_t &idx, uint32_t &w, uint32_t &aux) {
        idx = 0; w = 0; aux = 0;
        if (lane < (int)((uint32_t)ch.w >> 24) && DBS_CHK_RANGE(d, ch.x, (uint32_t)ch.w >> 24)) {
            const int p_ = ch.x + lane; idx = d.csr.idx[p_]; w = d.csr.w[p_]; aux = d.csr.aux[p_];
            DBS_CHK_ENTRY(d, true, idx, w, aux);
            // (the staged copy holds exactly the chunk's words: the block must start inside them)
            if ((idx >> TYPE_SHIFT) != DBSPMSPV_BLK_INLINE && !DBS_CHK_INDEX(d, (int64_t)w - (uint32_t)ch.z, (uint32_t)ch.w & 0xFFFFFFu)) { idx = 0u; w = 0u; aux = 0u; }
        }
    };
    int issued = 0;                                           // chunks of mine whose copies were started
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < STREAM_DEPTH; ++k) mbar_init(&s_bar[k], 1);
        fence_barrier_init();
    }
    __syncwarp();
    // the first copies start before x is even looked at
    for (; issued < STREAM_DEPTH - 1 && issued < n_mine; ++issued) {
        const int4 ch = desc_of(issued);
        if (lane == 0) issue(ch, issued);
    }
    __syncthreads();
    stage_x_blocks<DT>(d, x, s_x, s_xm, s_cnt, tid, T);
    __syncthreads();
    const int n_nzblk = s_cnt[0];
    int path = force_path;
    if (path != DBSPMSPV_PATH_PUSH && path != DBSPMSPV_PATH_PULL)
        path = (float)n_nzblk / (float)d.nb < th3 ? DBSPMSPV_PATH_PUSH : DBSPMSPV_PATH_PULL;
    if (blockIdx.x == 0 && tid == 0) {
        Counters *c = d.ws.ctr;
        c->last_n_nzblk = n_nzblk; c->last_n_tasks = 0; c->last_path = path; c->last_y_nnz = (int32_t)d.m;
        // (a store to host memory: only when it changes what the host goes by)
        if (d.x_nnz_seen && ((float)s_cnt[1] < STREAM_MIN_X_DENSITY * (float)d.n) != (d.x_sparse_believed != 0)) *d.x_nnz_seen = s_cnt[1];
    }

    // y is zeroed by the kernel in front, which this one may overlap up to here
    pdl_wait();

    float acc[16];
#pragma unroll
    for (int r = 0; r < 16; ++r) acc[r] = 0.f;
    int cur_rb = -1;
    // the warp's 16 row sums -> y (rows past m hold nothing: their sums are exact zeros)
    auto flush = [&]() {
        if (cur_rb >= 0) {
            const float total = fold_rows(acc, lane);
            if (!(lane & 1) && total != 0.f) atomicAdd(y + (size_t)cur_rb * 16 + folded_row(lane), total);
#pragma unroll
            for (int r = 0; r < 16; ++r) acc[r] = 0.f;
        }
    };
    auto emit = [&](int erb, int erow, float esum) { atomicAdd(y + (size_t)erb * 16 + erow, esum); };
    // one step: the lane's entry (idx, w, aux) of row block cur_rb, if `have`; the payload pointer
    // is the staged copy (shifted so that the entry's offset applies) or, on the rare paths that
    // read global memory, the payload itself -- the values are indexed where they are either way
    auto step = [&](const uint8_t *payload, uint32_t idx, uint32_t w, uint32_t aux, bool have) {
        const uint32_t xm = have ? s_xm[idx & IDX_MASK] : 0u;
        const int type = idx >> TYPE_SHIFT;
        const bool mk = have && xm && type > DBSPMSPV_BLK_COO;
        const bool rowm = mk && is_row_major(type);
        const float *xb = s_x + (size_t)(idx & IDX_MASK) * 16;
        warp_columns<DT, 2, true>(payload, s_x, idx, w, mk && !rowm ? xm : 0u, lane, acc, static_cast<uint4 *>(nullptr));
        __syncwarp();
        const uint32_t rows = __ballot_sync(FULL, rowm);
        if (rows) half_stream<DT, true>(payload, s_x, idx, w, xm, cur_rb, rows, lane, emit);
        if (have && xm && type <= DBSPMSPV_BLK_COO) {       // the odd hypersparse block: its own lane
            float *row0 = y + (size_t)cur_rb * 16;
            if (type == DBSPMSPV_BLK_INLINE) {
                if ((xm >> (aux & 15)) & 1u) atomicAdd(row0 + (aux >> 4), Val<DT>::inline_value(w) * xb[aux & 15]);
            } else {
                const int nnz = (int)aux + 1;
                const uint8_t *blk = payload + (size_t)w * 4, *vals = blk + ((nnz + 3) & ~3);
                for (int k = 0; k < nnz; ++k) {
                    const int c = blk[k] & 15, r = blk[k] >> 4;
                    if ((xm >> c) & 1u) atomicAdd(row0 + r, Val<DT>::load(vals, k) * xb[c]);
                }
            }
        }
    };
    auto fetch = [&](int p, bool have, uint32_t &idx, uint32_t &w, uint32_t &aux) {
        idx = 0; w = 0; aux = 0;
        if (have && DBS_CHK_INDEX(d, p, d.n_entries)) { idx = d.csr.idx[p]; w = d.csr.w[p]; aux = d.csr.aux[p]; DBS_CHK_ENTRY(d, true, idx, w, aux); }
    };

    if (path == DBSPMSPV_PATH_PULL) {
        bool timed_out = false;
        uint32_t idx = 0, w = 0, aux = 0, n_idx, n_w, n_aux;
        if (n_mine > 0) entries_of(desc_of(0), idx, w, aux);
        for (int k = 0; k < n_mine; ++k) {
            // keep STREAM_DEPTH - 1 chunks in flight beside this one: chunk i goes into the stage
            // that chunk i - STREAM_DEPTH was read from, in a round before this one
            for (const int lim = min(n_mine, min(k + STREAM_DEPTH, (k & ~31) + 32)); issued < lim; ++issued) {
                const int4 nch = desc_of(issued);
                if (lane == 0) issue(nch, issued % STREAM_DEPTH);
            }
            const int st = k % STREAM_DEPTH;
            const int4 ch = desc_of(k);
            n_idx = 0; n_w = 0; n_aux = 0;
            if (k + 1 < n_mine && ((k + 1) & 31)) entries_of(desc_of(k + 1), n_idx, n_w, n_aux);
            if (!mbar_wait_bounded(&s_bar[st], (uint32_t)(k / STREAM_DEPTH) & 1u)) { timed_out = true; break; }
            if (ch.y != cur_rb) { flush(); cur_rb = DBS_CHK_INDEX(d, ch.y, d.mb) ? ch.y : 0; }
            const uint8_t *base = s_ring + (size_t)st * stride;
            step(base - (size_t)(uint32_t)ch.z * 4, idx, w, aux, lane < (int)((uint32_t)ch.w >> 24));
            __syncwarp();
            idx = n_idx; w = n_w; aux = n_aux;
            if (k + 1 < n_mine && !((k + 1) & 31)) {           // first chunk of the next descriptor batch: fetched late
                my_desc = make_int4(0, 0, 0, 0);
                if (k + 1 + lane < n_mine) my_desc = d.stage_chunks[lo + k + 1 + lane];
                entries_of(desc_of(k + 1), idx, w, aux);
            }
        }
        flush();
        if (timed_out) { d.ws.ctr->status = DBSPMSPV_ERR_TIMEOUT; return; }
        // the INLINE elements of the row blocks (row by row, rare in these handles)
        for (int rb = gw; rb < d.mb && d.has_inline; rb += W) {
            const int b0 = d.csr_inl[rb], b1 = d.csr.ptr[rb + 1];
            cur_rb = rb;
            for (int base = b0; base < b1; base += 32) {
                uint32_t idx, w, aux;
                fetch(base + lane, base + lane < b1, idx, w, aux);
                step(d.payload, idx, w, aux, base + lane < b1);
            }
            if (b1 > b0) flush();
        }
    } else {
        // copies of the first chunks are in flight: they must have landed before the block ends
        for (int k = 0; k < issued; ++k) mbar_wait_bounded(&s_bar[k], 0u);
        if (warp == 0) {
            int count = 0;
            for (int base = 0; base < d.nb; base += 32) {
                const bool on = base + lane < d.nb && s_xm[base + lane] != 0;
                const uint32_t m = __ballot_sync(FULL, on);
                if (on) s_active[count + __popc(m & below(lane))] = base + lane;
                count += __popc(m);
            }
        }
        __syncthreads();
        for (int rb = blockIdx.x; rb < d.mb; rb += gridDim.x) {
            const int begin = d.csr.ptr[rb], pend = d.csr_inl[rb], end = d.csr.ptr[rb + 1];
            cur_rb = rb;
            // the row block's entries with a payload are sorted by column block: [begin, pend)
            for (int i0 = warp * 32; i0 < n_nzblk; i0 += T) {
                int lo_ = 0, hi_ = 0;
                if (i0 + lane < n_nzblk) {
                    const uint32_t cb = (uint32_t)s_active[i0 + lane];
                    int a = begin, b = pend;          // first entry with column block >= cb
                    while (a < b) { const int mid = a + ((b - a) >> 1); if ((d.csr.idx[mid] & IDX_MASK) < cb) a = mid + 1; else b = mid; }
                    lo_ = a; b = pend;                // first entry with column block > cb
                    while (a < b) { const int mid = a + ((b - a) >> 1); if ((d.csr.idx[mid] & IDX_MASK) <= cb) a = mid + 1; else b = mid; }
                    hi_ = a;
                }
                for (int t = 0; __any_sync(FULL, lo_ + t < hi_); ++t) {
                    uint32_t idx, w, aux;
                    fetch(lo_ + t, lo_ + t < hi_, idx, w, aux);
                    step(d.payload, idx, w, aux, lo_ + t < hi_);
                }
            }
            for (int base = pend + warp * 32; base < end; base += T) {
                uint32_t idx, w, aux;
                fetch(base + lane, base + lane < end, idx, w, aux);
                step(d.payload, idx, w, aux, base + lane < end);
            }
            flush();
        }
    }
}

}  // namespace dbs
#include "decode_batch.cuh"
#include "small_call.cuh"
namespace dbs {

// ------------------------------------------------------------------------------------------
// Output compaction: the hit masks of the row blocks are scanned in order, so y comes out
// sorted.  Pass 1 counts per tile, pass 2 places the entries, clears the accumulator and the
// masks it read, clears the vector-block state of this call's x, and rolls the counters over.
// ------------------------------------------------------------------------------------------
// Fold of the private accumulators of one hub row block (see push_private), by a whole warp:
// every lane takes four rows of two copies, a shuffle tree adds the copies up in a fixed
// order, the totals go into the accumulator proper (no atomics: every push has ended) and the
// rows that any copy touched get their structural-hit flag; touched copies are put back to
// HUB_CLEAR.  A kernel of its own, one warp per hub row block, between the traversal and the
// compaction: hub row blocks are neighbours (the low vertex numbers of an R-MAT graph), so a
// fold inside the compaction, by the warp that owns the rows, took 40 folds one after the other.
static_assert(HUB_COPIES % 8 == 0, "a warp folds eight copies per step");
__device__ __forceinline__ void fold_hub_block(const Device &d, int rb, int slot, int lane) {
    const int q = lane & 3;
    float4 tot = make_float4(0.f, 0.f, 0.f, 0.f);
    uint32_t touched = 0u;
#pragma unroll
    for (int k = 0; k < HUB_COPIES / 8; ++k) {
        const int c = (lane >> 2) + 8 * k;
        float4 *p = reinterpret_cast<float4 *>(d.hub_acc + ((size_t)c * d.n_hub_blocks + slot) * 16) + q;
        const float4 v = __ldcg(p);
        const uint32_t t = (__float_as_uint(v.x) != HUB_CLEAR ? 1u : 0u) | (__float_as_uint(v.y) != HUB_CLEAR ? 2u : 0u) |
                           (__float_as_uint(v.z) != HUB_CLEAR ? 4u : 0u) | (__float_as_uint(v.w) != HUB_CLEAR ? 8u : 0u);
        // (an untouched -0.0f adds nothing)
        tot.x += v.x; tot.y += v.y; tot.z += v.z; tot.w += v.w;
        if (t) { const float z = __uint_as_float(HUB_CLEAR); *p = make_float4(z, z, z, z); }
        touched |= t;
    }
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
        tot.x += __shfl_xor_sync(FULL, tot.x, o); tot.y += __shfl_xor_sync(FULL, tot.y, o);
        tot.z += __shfl_xor_sync(FULL, tot.z, o); tot.w += __shfl_xor_sync(FULL, tot.w, o);
        touched |= __shfl_xor_sync(FULL, touched, o);
    }
    if (lane < 4 && touched) {
        float *a = d.ws.y_acc + (size_t)rb * 16 + 4 * q;
        uint8_t *f = d.ws.y_hit8 + (size_t)rb * 16 + 4 * q;
        if (touched & 1u) { a[0] += tot.x; f[0] = 1; }
        if (touched & 2u) { a[1] += tot.y; f[1] = 1; }
        if (touched & 4u) { a[2] += tot.z; f[2] = 1; }
        if (touched & 8u) { a[3] += tot.w; f[3] = 1; }
    }
}

__global__ void __launch_bounds__(128) k_fold_hubs(Device d) {
    pdl_wait();
    pdl_launch_dependents();
    const int slot = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (slot < d.n_hub_blocks && DBS_CHK_INDEX(d, d.hub_rb[slot], d.mb)) fold_hub_block(d, d.hub_rb[slot], slot, threadIdx.x & 31);
}

__global__ void __launch_bounds__(TILE_WORDS) k_compact_count(Device d, int parity, const uint32_t *__restrict__ row_mask, int complement) {
    __shared__ int s_red[TILE_WORDS / 32];
    pdl_wait();
    pdl_launch_dependents();
    const int n_words = (d.mb + 1) / 2;
    const int wi = blockIdx.x * TILE_WORDS + threadIdx.x;
    int c = 0;
    if (wi < n_words) {
        // 32 row flags (bytes, 0 or 1) -> one mask word; the flags are cleared for the next call
        uint4 *f4 = reinterpret_cast<uint4 *>(d.ws.y_hit8 + (size_t)wi * 32);
        const uint4 a = f4[0], b = f4[1];
        const uint32_t v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        uint32_t word = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) word |= (((v[q] & 0x01010101u) * 0x01020408u) >> 24 & 0xFu) << (4 * q);
        if (word) {
            f4[0] = make_uint4(0u, 0u, 0u, 0u);
            f4[1] = make_uint4(0u, 0u, 0u, 0u);
        }
        d.ws.y_mask32[wi] = word;
        // (an output mask drops rows from y; their accumulator entries are still cleared by pass 2)
        c = __popc(row_mask ? word & (complement ? ~row_mask[wi] : row_mask[wi]) : word);
    }
    c = __reduce_add_sync(FULL, c);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int k = 0; k < TILE_WORDS / 32; ++k) t += s_red[k];
        d.ws.tile_count[blockIdx.x] = t;
        // totals of groups of 32 tiles, so that pass 2 adds up a few dozen numbers per tile
        // instead of one per earlier tile (all thread blocks reading the same few lines of
        // counts was most of pass 2 on a large m: 2,100 tiles -> 2.2 M loads on 64 lines)
        if (t) atomicAdd(d.ws.tile_group + parity * d.ws.n_tile_groups + (blockIdx.x >> 5), t);
    }
}

__global__ void __launch_bounds__(CMP_TPB) k_compact_write(Device d, int32_t *__restrict__ y_idx, float *__restrict__ y_val,
                                                           int64_t y_capacity, int32_t *__restrict__ y_nnz, int boolean,
                                                           const int32_t *__restrict__ x_idx, int32_t nnz_x, int clear_all, int parity,
                                                           const uint32_t *__restrict__ row_mask, int complement) {
    __shared__ int s_before[CMP_TPB / 32], s_cnt[CMP_TPB / 32];
    __shared__ int32_t s_oidx[TILE_WORDS * 32];
    __shared__ float s_oval[TILE_WORDS * 32];
    const int n_tiles = d.ws.n_tiles;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    pdl_wait();
    // The kernel is a chain of dependent loads, not bandwidth: everything that can be fetched
    // up front is fetched before the first barrier.
    const int stride = gridDim.x * CMP_TPB;
    const int k0 = blockIdx.x * CMP_TPB + threadIdx.x;
    const int j0 = (!clear_all && k0 < nnz_x) ? x_idx[k0] : -1;
    if ((int)blockIdx.x < n_tiles) {
        const int n_words = (d.mb + 1) / 2;
        // every thread owns 8 consecutive rows (a quarter of a mask word)
        const int wi = blockIdx.x * TILE_WORDS + (threadIdx.x >> 2);
        const int sub = threadIdx.x & 3;
        const uint32_t word = wi < n_words ? d.ws.y_mask32[wi] : 0u;
        int before = 0;               // entries in all earlier tiles: whole groups of 32, then the tiles of this group
        {
            const int g = (int)blockIdx.x >> 5, r = (int)blockIdx.x & 31;
            const int32_t *grp = d.ws.tile_group + parity * d.ws.n_tile_groups;
            for (int k = threadIdx.x; k < g + r; k += CMP_TPB) before += k < g ? grp[k] : d.ws.tile_count[g * 32 + (k - g)];
            // the group totals of the other parity served the call before: cleared for the next one
            if (blockIdx.x == 0)
                for (int k = threadIdx.x; k < d.ws.n_tile_groups; k += CMP_TPB) d.ws.tile_group[(parity ^ 1) * d.ws.n_tile_groups + k] = 0;
        }
        const uint32_t keep = row_mask && wi < n_words ? (complement ? ~row_mask[wi] : row_mask[wi]) : 0xFFFFFFFFu;
        const uint32_t hits = (word >> (8 * sub)) & 0xFFu;    // rows to clear
        const uint32_t bits = hits & (keep >> (8 * sub));     // rows that go to y
        const int c = __popc(bits);
        const int row0 = wi * 32 + sub * 8;
        float4 v4[2];
        if (hits) {                   // two independent 16-byte loads fetch the 8 accumulator entries
            float4 *acc4 = reinterpret_cast<float4 *>(d.ws.y_acc + row0);
            v4[0] = acc4[0]; v4[1] = acc4[1];
            acc4[0] = make_float4(0.f, 0.f, 0.f, 0.f);
            acc4[1] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        int incl = c;
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(FULL, incl, o);
            if (lane >= o) incl += t;
        }
        before = __reduce_add_sync(FULL, before);
        if (lane == 31) s_cnt[warp] = incl;
        if (lane == 0) s_before[warp] = before;
        __syncthreads();
        int base = 0, local = 0, tile_total = 0;
#pragma unroll
        for (int k = 0; k < CMP_TPB / 32; ++k) {
            base += s_before[k];
            if (k < warp) local += s_cnt[k];
            tile_total += s_cnt[k];
        }
        // the tile's entries are gathered in shared memory, then written out in whole lines
        if (bits) {
            const float *v = reinterpret_cast<const float *>(v4);
            int pos = local + incl - c;
#pragma unroll
            for (int bit = 0; bit < 8; ++bit) {
                if ((bits >> bit) & 1u) {
                    s_oidx[pos] = row0 + bit;
                    // boolean 1: a Boolean result; 2: the accumulator holds (min, +) keys
                    s_oval[pos] = boolean == 1 ? 1.0f : boolean == 2 ? minplus_value(__float_as_uint(v[bit])) : v[bit];
                    ++pos;
                }
            }
        }
        __syncthreads();
        for (int k = threadIdx.x; k < tile_total; k += CMP_TPB) {
            const int64_t pos = (int64_t)base + k;
            if (pos < y_capacity) {
                y_idx[pos] = s_oidx[k];
                if (y_val) y_val[pos] = s_oval[k];
            }
        }
        if ((int)blockIdx.x == n_tiles - 1 && threadIdx.x == 0) {
            Counters *c2 = d.ws.ctr;
            const int total = base + tile_total;
            *y_nnz = total;
            if (total > y_capacity) c2->status = DBSPMSPV_ERR_CAPACITY;
            c2->last_y_nnz = total;
            c2->last_n_nzblk = c2->n_nzblk;
            c2->last_n_tasks = c2->n_tasks;
            c2->last_path = c2->path;
            c2->n_nzblk = 0;
            c2->n_tasks = 0;
            c2->n_hubs = 0;
        }
    }
    // vector-block state of this call's x: clear the masks and put the "not listed" marker back
    // -- entry by entry, or, for an x that lists a good part of all columns, by streaming over
    // the whole dense copy (full-line stores instead of scattered 4-byte ones)
    if (clear_all) {
        const int n_words = (d.nb + 1) / 2;
        const uint32_t mk = X_ABSENT;
        uint4 *xd4 = reinterpret_cast<uint4 *>(d.ws.x_dense);
        for (int k = k0; k < n_words * 8; k += stride) xd4[k] = make_uint4(mk, mk, mk, mk);
        for (int k = k0; k < n_words; k += stride) d.ws.x_mask32[k] = 0u;
        return;
    }
    if (j0 >= 0 && j0 < d.n) { d.ws.x_mask32[j0 >> 5] = 0u; d.ws.x_dense[j0] = __uint_as_float(X_ABSENT); }
    for (int k = k0 + stride; k < nnz_x; k += stride) {
        const int j = x_idx[k];
        if (j >= 0 && j < d.n) { d.ws.x_mask32[j >> 5] = 0u; d.ws.x_dense[j] = __uint_as_float(X_ABSENT); }
    }
}

__global__ void k_decode_cleanup(Device d) {
    pdl_wait();
    const int n_words = (d.nb + 1) / 2;
    const int stride = gridDim.x * blockDim.x;
    for (int k = blockIdx.x * blockDim.x + threadIdx.x; k < n_words; k += stride) d.ws.x_mask32[k] = 0u;
    for (int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j < (int64_t)d.nb * 16; j += stride)
        d.ws.x_dense[j] = __uint_as_float(X_ABSENT);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        Counters *c = d.ws.ctr;
        c->last_n_nzblk = c->n_nzblk;
        c->last_n_tasks = c->n_tasks;
        c->last_path = c->path;
        c->last_y_nnz = (int32_t)d.m;
        c->n_nzblk = 0;
        c->n_tasks = 0;
        c->n_hubs = 0;
    }
}

// Test hook: the bounded wait of the staging code on a barrier that nothing will ever arrive on
// (no copy is in flight, so there is nothing to drain): the wait gives up after `max_tries`
// tries and the kernel records DBSPMSPV_ERR_TIMEOUT, exactly as the pull traversal would.
__global__ void k_wait_probe(Device d, int max_tries) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_barrier_init();
        if (!mbar_wait_bounded(&bar, 0u, max_tries)) d.ws.ctr->status = DBSPMSPV_ERR_TIMEOUT;
    }
}

__global__ void k_fill_u32(uint32_t *p, int64_t n, uint32_t v) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) p[i] = v;
}

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
template <typename T> static int dev_alloc_zero(T **p, size_t count, int64_t *total) {
    void *q = nullptr;
    size_t bytes = (count ? count : 1) * sizeof(T);
    if (cudaMalloc(&q, bytes) != cudaSuccess) return DBSPMSPV_ERR_ALLOC;
    if (cudaMemset(q, 0, bytes) != cudaSuccess) return DBSPMSPV_ERR_CUDA;
    *p = static_cast<T *>(q);
    *total += (int64_t)bytes;
    return DBSPMSPV_OK;
}

// Launch with the programmatic-stream-serialisation attribute (see pdl_wait): the kernel may be
// scheduled while its predecessor in the stream is still draining.
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Persistent grid of the traversal kernel: as many thread blocks as fit (0 on error).
template <int DT, typename Out, int MODE> static int compute_grid(int sm_count) {
    const size_t smem = compute_dyn_smem<MODE>();
    if (cudaFuncSetAttribute(k_compute<DT, Out, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return 0;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_compute<DT, Out, MODE>, CTA, smem) != cudaSuccess || per_sm < 1) return 0;
    return sm_count * per_sm;
}

template <int DT, typename Out, int MODE>
static int launch_compute(dbspmspv_handle_s *h, Out out, float th3, bool pdl, cudaStream_t st, int pull_done = 0) {
    // (one handle launches one instantiation per output kind; the decode entry of a handle and its
    // run entry differ in Out, hence the two slots)
    int &grid = Out::MASKS ? h->grid_compute : h->grid_compute_dense;
    if (!grid) grid = compute_grid<DT, Out, MODE>(h->sm_count);
    if (!grid) return DBSPMSPV_ERR_CUDA;
    const size_t smem = compute_dyn_smem<MODE>();
    if (pdl) {
        DBS_CUDA(launch_pdl(k_compute<DT, Out, MODE>, grid, CTA, smem, st, h->d, out, th3, h->ropts.force_path, h->ropts.popc_threshold, pull_done));
    } else {
        k_compute<DT, Out, MODE><<<grid, CTA, smem, st>>>(h->d, out, th3, h->ropts.force_path, h->ropts.popc_threshold, pull_done);
    }
    ++h->kernel_launches;
    return DBSPMSPV_OK;
}

// The streaming pull of hypersparse handles (lean_pull.cuh), launched behind k_compute.
template <int DT, typename Out>
static int launch_lean(dbspmspv_handle_s *h, Out out, float th3, cudaStream_t st) {
    bool &configured = Out::MINPLUS ? h->lean_configured_min : Out::MASKS ? h->lean_configured : h->lean_configured_dense;
    // filter size: the power of two that holds one bit per column, capped
    const int n_words = (h->d.nb + 1) / 2;
    int filter_words = 32;
    while (filter_words < n_words && filter_words < LEAN_FILTER_MAX_WORDS) filter_words <<= 1;
    const size_t smem = (size_t)filter_words * 4 + LEAN_WARPS * sizeof(LeanScratch);
    if (!configured) {
        auto kernel = k_pull_lean<DT, Out>;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DBSPMSPV_ERR_CUDA;
        configured = true;
    }
    DBS_CUDA(launch_pdl(k_pull_lean<DT, Out>, h->sm_count, LEAN_CTA, smem, st, h->d, out, th3, h->ropts.force_path,
                        h->ropts.popc_threshold, filter_words));
    ++h->kernel_launches;
    return DBSPMSPV_OK;
}

// Upper bound of the selector's ratio known on the host: with at most `nnz_x` listed columns no
// more than min(nnz_x, nb) vector blocks are nonempty.  When even that stays below th3 the push
// is certain and the pull kernel need not be launched.
static bool pull_possible(const dbspmspv_handle_s *h, int64_t nnz_x, float th3) {
    if (h->ropts.force_path == DBSPMSPV_PATH_PUSH) return false;
    if (h->ropts.force_path == DBSPMSPV_PATH_PULL) return true;
    const int64_t most = nnz_x < h->d.nb ? nnz_x : h->d.nb;
    return !((float)most / (float)h->d.nb < th3);
}

int allocate_workspace(dbspmspv_handle_s *h) {
    Device &d = h->d;
    Workspace &ws = d.ws;
    int64_t total = 0;
    const size_t xwords = (size_t)(d.nb + 1) / 2 + 4, ywords = (size_t)(d.mb + 1) / 2 + 4;
    // Entries with a payload per push task: a full warp step where such blocks are the bulk of
    // the matrix (the lanes then share them out); a few where they are the exception and a warp
    // takes them one at a time (32 of them in one task would keep one warp busy for tens of
    // microseconds while the others have long finished).
    d.payload_chunk = h->heavy_stage ? PUSH_CHUNK : 4;
    // one partial task at most per column (INLINE run) and per column block (payload run)
    ws.task_capacity = (int64_t)d.n_entries / d.payload_chunk + 17 * (int64_t)d.nb + 32;
    ws.n_tiles = (int32_t)ceil_div<int64_t>((d.mb + 1) / 2, TILE_WORDS);
    if (ws.n_tiles < 1) ws.n_tiles = 1;
    // One allocation for the whole workspace, carved at 512-byte boundaries (a dozen cudaMalloc
    // calls fewer per handle).  Where the driver places its pages still matters: the same push
    // kernel measured 68 .. 83 us on the same data from one allocation history to the next.
    size_t off = 0;
    // (arrays of a megabyte or more start on a 2 MB boundary, the others on a 512-byte one)
    auto carve = [&](size_t bytes) {
        const size_t a = bytes >= ((size_t)1 << 20) ? ((size_t)2 << 20) : 512;
        off = (off + a - 1) / a * a;
        const size_t o = off;
        off += (bytes + 511) & ~(size_t)511;
        return o;
    };
    const size_t zwords = xwords > ywords ? xwords : ywords;
    const size_t o_xd = carve(xwords * 32 * sizeof(float)), o_yacc = carve(ywords * 32 * sizeof(float)),
                 o_hit = carve(ywords * 32), o_tasks = carve((size_t)ws.task_capacity * sizeof(*ws.tasks)),
                 o_xm = carve(xwords * 4), o_ym = carve(ywords * 4), o_zm = carve(zwords * 4),
                 o_words = carve(4 * zwords * sizeof(*ws.bfs_words)), o_vis = carve((d.m == d.n ? ywords : 1) * 4),
                 o_hubs = carve((size_t)3 * HUB_CAP * sizeof(*ws.hubs)), o_tile = carve((size_t)ws.n_tiles * sizeof(*ws.tile_count)),
                 o_group = carve((size_t)2 * ((ws.n_tiles + 31) / 32) * sizeof(*ws.tile_group)),
                 o_ctr = carve(sizeof(*ws.ctr));
    void *arena = nullptr;
    if (cudaMalloc(&arena, off) != cudaSuccess) return DBSPMSPV_ERR_ALLOC;
    h->ws_arena = arena;
    if (cudaMemset(arena, 0, off) != cudaSuccess) return DBSPMSPV_ERR_CUDA;
    uint8_t *base = static_cast<uint8_t *>(arena);
    ws.x_dense = reinterpret_cast<decltype(ws.x_dense)>(base + o_xd);
    ws.y_acc = reinterpret_cast<decltype(ws.y_acc)>(base + o_yacc);
    ws.y_hit8 = reinterpret_cast<decltype(ws.y_hit8)>(base + o_hit);
    ws.tasks = reinterpret_cast<decltype(ws.tasks)>(base + o_tasks);
    ws.x_mask32 = reinterpret_cast<decltype(ws.x_mask32)>(base + o_xm);
    ws.y_mask32 = reinterpret_cast<decltype(ws.y_mask32)>(base + o_ym);
    ws.z_mask32 = reinterpret_cast<decltype(ws.z_mask32)>(base + o_zm);
    ws.bfs_words = reinterpret_cast<decltype(ws.bfs_words)>(base + o_words);
    ws.bfs_words_stride = (int32_t)zwords;
    ws.visited32 = reinterpret_cast<decltype(ws.visited32)>(base + o_vis);
    ws.hubs = reinterpret_cast<decltype(ws.hubs)>(base + o_hubs);
    ws.tile_count = reinterpret_cast<decltype(ws.tile_count)>(base + o_tile);
    ws.tile_group = reinterpret_cast<decltype(ws.tile_group)>(base + o_group);
    ws.n_tile_groups = (ws.n_tiles + 31) / 32;
    ws.ctr = reinterpret_cast<decltype(ws.ctr)>(base + o_ctr);
    total = (int64_t)off;
    h->stats.workspace_bytes = total;
    if (cudaMemset(ws.x_dense, 0xFF, xwords * 32 * sizeof(float)) != cudaSuccess) return DBSPMSPV_ERR_CUDA;
    {   // 0xFFFFFFFF -> the marker pattern 0x7FFFFFFF needs a kernel; a tiny fill does it
        uint32_t *p = reinterpret_cast<uint32_t *>(ws.x_dense);
        k_fill_u32<<<256, 256>>>(p, (int64_t)xwords * 32, X_ABSENT);
        if (cudaDeviceSynchronize() != cudaSuccess) return DBSPMSPV_ERR_CUDA;
    }
    // events for the optional kernel timing are made here so that run-time calls create nothing
    if (cudaEventCreate(&h->ev[0]) != cudaSuccess || cudaEventCreate(&h->ev[1]) != cudaSuccess) return DBSPMSPV_ERR_CUDA;
    return DBSPMSPV_OK;
}

template <int DT>
static int run_typed(dbspmspv_handle_s *h, const int32_t *x_idx, const void *x_val, int32_t nnz_x,
                     int semiring, int32_t *y_idx, float *y_val, int64_t y_capacity, int32_t *y_nnz,
                     cudaStream_t st, const uint32_t *row_mask = nullptr, int complement = 0) {
    const Device &d = h->d;
    // a short x on a hypersparse handle: the whole call as one kernel of one thread-block cluster (small_call.cuh)
    {
        const size_t ywords = (size_t)(d.mb + 1) / 2, cbwords = (size_t)(d.nb + 31) / 32;
        const size_t smem = ((ywords + SMALL_CLUSTER - 1) / SMALL_CLUSTER + (cbwords + SMALL_CLUSTER - 1) / SMALL_CLUSTER) * sizeof(uint32_t);
        if (nnz_x > 0 && nnz_x <= SMALL_MAX_NNZ_X && d.n_entries > 0 && !h->heavy_stage && !h->ropts.validate && !h->ropts.timing &&
            !h->ropts.no_small_call && h->ropts.force_path != DBSPMSPV_PATH_PULL && !pull_possible(h, nnz_x, h->ropts.th3) &&
            smem <= SMALL_MAX_SMEM && (int64_t)ywords * 32 * (int64_t)sizeof(int32_t) <= d.ws.task_capacity * (int64_t)sizeof(*d.ws.tasks)) {
            const int mode = semiring == DBSPMSPV_OR_AND ? 1 : semiring == DBSPMSPV_MIN_PLUS ? 2 : 0;
            k_run_small<DT><<<SMALL_CLUSTER, SMALL_CTA, smem, st>>>(d, x_idx, x_val, nnz_x, mode, y_idx, y_val, y_capacity, y_nnz, row_mask, complement);
            ++h->kernel_launches;
            DBS_CUDA(cudaGetLastError());
            return DBSPMSPV_OK;
        }
    }
    // x lists a quarter of the columns or more: a pull is likely (on hypersparse matrices), so
    // the worklist is built afterwards from the masks, and only if the selector does choose the push
    const bool minplus = semiring == DBSPMSPV_MIN_PLUS;
    // (min, +) pulls only with the streaming kernel of hypersparse valued handles
    const bool minplus_pull = minplus && !h->heavy_stage && DT != DBSPMSPV_PATTERN;
    const bool late_emit = (!minplus || minplus_pull) && !h->heavy_stage && h->ropts.force_path != DBSPMSPV_PATH_PUSH && (int64_t)nnz_x * 4 >= d.n;
    const void *xv = semiring == DBSPMSPV_OR_AND ? nullptr : x_val;
    if (nnz_x > 0) {
        const int g = (nnz_x + XB_TPB - 1) / XB_TPB;
        if (late_emit) {
            k_xblock_sparse<DT, false><<<g, XB_TPB, 0, st>>>(d, x_idx, xv, nnz_x, h->ropts.validate);
            int ge = ((d.nb + 1) / 2 + 7) / 8;
            if (ge > 8 * h->sm_count) ge = 8 * h->sm_count;
            DBS_CUDA(launch_pdl(k_emit_from_masks, ge, 256, 0, st, d, h->ropts.th3, h->ropts.force_path));
            ++h->kernel_launches;
        } else {
            k_xblock_sparse<DT, true><<<g, XB_TPB, 0, st>>>(d, x_idx, xv, nnz_x, h->ropts.validate);
        }
        ++h->kernel_launches;
    }
    OutSparse out{d.ws.y_acc, d.ws.y_hit8};
    if (h->ropts.timing) DBS_CUDA(cudaEventRecord(h->ev[0], st));
    // private accumulators for the hub row blocks: when x is long enough for their atomics to
    // queue up, and not so long that the call will most likely pull
    const int hub_min = h->ropts.hub_min_nnz_x ? h->ropts.hub_min_nnz_x : HUB_MIN_NNZ_X;
    h->d.hub_on = !minplus && d.n_hub_blocks > 0 && hub_min > 0 && nnz_x >= hub_min && h->ropts.force_path != DBSPMSPV_PATH_PULL &&
                  (!late_emit || h->heavy_stage);
    if (minplus && nnz_x > 0 && d.n_entries > 0) {
        const int fp = minplus_pull ? h->ropts.force_path : DBSPMSPV_PATH_PUSH;
        if (fp != DBSPMSPV_PATH_PULL) {
            DBS_CUDA(launch_pdl(k_minplus_push<DT>, 4 * h->sm_count, MINPLUS_CTA, 0, st, d, h->ropts.th3, fp));
            ++h->kernel_launches;
        }
        if (minplus_pull && pull_possible(h, nnz_x, h->ropts.th3)) {
            const int s = launch_lean<DT, OutSparseMin>(h, OutSparseMin{d.ws.y_acc, d.ws.y_hit8}, h->ropts.th3, st);
            if (s != DBSPMSPV_OK) return s;
        }
    } else if (nnz_x > 0 && d.n_entries > 0) {
        int s = DBSPMSPV_OK;
        if (h->heavy_stage) {
            s = launch_compute<DT, OutSparse, 1>(h, out, h->ropts.th3, true, st);
        } else {
            // push by k_compute, pull by the streaming kernel: each returns at once when the
            // selector (evaluated on the device) chose the other; a kernel whose path cannot be
            // chosen is not launched at all
            if (h->ropts.force_path != DBSPMSPV_PATH_PULL) s = launch_compute<DT, OutSparse, 0>(h, out, h->ropts.th3, true, st);
            if (s == DBSPMSPV_OK && pull_possible(h, nnz_x, h->ropts.th3)) s = launch_lean<DT, OutSparse>(h, out, h->ropts.th3, st);
        }
        if (s != DBSPMSPV_OK) return s;
        if (d.hub_on) {
            DBS_CUDA(launch_pdl(k_fold_hubs, (d.n_hub_blocks + 3) / 4, 128, 0, st, d));
            ++h->kernel_launches;
        }
    }
    if (h->ropts.timing) { DBS_CUDA(cudaEventRecord(h->ev[1], st)); h->timed = true; }
    h->kernel_launches += 2;
    const int nt = d.ws.n_tiles;
    const int parity = (int)(++h->compact_calls & 1u);
    DBS_CUDA(launch_pdl(k_compact_count, nt, TILE_WORDS, 0, st, d, parity, row_mask, complement));
    int extra = (nnz_x + CMP_TPB * 8 - 1) / (CMP_TPB * 8);
    if (extra > 4 * h->sm_count) extra = 4 * h->sm_count;
    const int clear_all = (int64_t)nnz_x * 8 > d.n;     // scattered clears cost more than a full sweep
    DBS_CUDA(launch_pdl(k_compact_write, nt + extra, CMP_TPB, 0, st, d, y_idx, y_val, y_capacity, y_nnz,
                        minplus ? 2 : (int)(semiring == DBSPMSPV_OR_AND || DT == DBSPMSPV_PATTERN), x_idx, nnz_x, clear_all, parity, row_mask, complement));
    DBS_CUDA(cudaGetLastError());
    return DBSPMSPV_OK;
}

// payload bytes of one stage of a warp's ring in the streaming decode: what shared memory leaves
// when two thread blocks share an SM (else one), at most STAGE_BYTES; 0 = no room (a block must fit)
int decode_stage_bytes(const Device &d) {
    const StreamLayout lay(d.nb, 0);
    for (int budget : {DBS_STREAM_BUDGET, STREAM_MAX_SMEM}) {
        const int room = budget - lay.ring_off;
        if (room <= 0) continue;
        int sb = (room / (STREAM_WARPS * STREAM_DEPTH)) & ~511;
        if (sb > STAGE_BYTES) sb = STAGE_BYTES;
        if (sb >= 2048) return sb;
    }
    return 0;
}

template <int DT>
static int decode_typed(dbspmspv_handle_s *h, const void *x, float *y, cudaStream_t st) {
    const Device &d = h->d;
    h->d.decode_tau = h->ropts.decode_threshold;
    h->d.decode_relu = h->ropts.decode_relu != 0;
    h->d.decode_x_f32 = h->ropts.decode_x_f32 != 0;
    // (-1: no decode call has reported yet)
    const int seen = h->x_nnz_seen_host ? *const_cast<volatile int32_t *>(h->x_nnz_seen_host) : -1;
    const bool sparse_x = seen >= 0 && (float)seen < STREAM_MIN_X_DENSITY * (float)d.n;
    h->d.x_sparse_believed = sparse_x;
    if (h->heavy_stage && d.stage_chunks != nullptr && (h->ropts.no_fused_decode == 3 || (h->ropts.no_fused_decode == 0 && !sparse_x))) {
        // the streaming form: one persistent kernel behind a memset of y
        const StreamLayout lay(d.nb, d.stage_bytes);
        if (!h->stream_grid) {
            // (the attribute belongs to the kernel, not to the handle: always the largest size)
            DBS_CUDA(cudaFuncSetAttribute(k_decode_stream<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, STREAM_MAX_SMEM));
            int per_sm = 0;
            DBS_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_decode_stream<DT>, STREAM_CTA, lay.total));
            if (per_sm < 1) return DBSPMSPV_ERR_CUDA;
            h->stream_grid = per_sm * h->sm_count;
        }
        if (h->ropts.timing) DBS_CUDA(cudaEventRecord(h->ev[0], st));
        k_fill_u32<<<(int)((d.m + 1023) / 1024), 256, 0, st>>>(reinterpret_cast<uint32_t *>(y), d.m, 0u);
        DBS_CUDA(launch_pdl(k_decode_stream<DT>, h->stream_grid, STREAM_CTA, (size_t)lay.total, st, d, x, y, h->ropts.th3_decode, h->ropts.force_path));
        ++h->kernel_launches;
        if (h->ropts.timing) { DBS_CUDA(cudaEventRecord(h->ev[1], st)); h->timed = true; }
        ++h->kernel_launches;
        DBS_CUDA(cudaGetLastError());
        return DBSPMSPV_OK;
    }
    if (h->heavy_stage && h->ropts.no_fused_decode != 1) {
        // one kernel for the whole call, when x fits in shared memory
        const int per_rb = d.mb ? d.n_entries / d.mb : 0;
        // warps per thread block from the entries per row block (measured on the three layer
        // shapes: more, smaller warps-per-block steps were 5-30 % slower)
        const int nw = per_rb <= 384 ? 4 : per_rb <= 1024 ? 8 : 16;
        const FusedLayout lay(d.nb, nw * 32);
        if (lay.total <= FUSED_MAX_SMEM) {
            auto kernel = nw == 4 ? k_decode_fused<DT, 4> : nw == 8 ? k_decode_fused<DT, 8> : k_decode_fused<DT, 16>;
            bool &done = h->fused_configured[nw == 4 ? 0 : nw == 8 ? 1 : 2];
            if (!done) {
                DBS_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FUSED_MAX_SMEM));
                done = true;
            }
            if (h->ropts.timing) DBS_CUDA(cudaEventRecord(h->ev[0], st));
            kernel<<<d.mb, nw * 32, lay.total, st>>>(d, x, y, h->ropts.th3_decode, h->ropts.force_path);
            if (h->ropts.timing) { DBS_CUDA(cudaEventRecord(h->ev[1], st)); h->timed = true; }
            ++h->kernel_launches;
            DBS_CUDA(cudaGetLastError());
            return DBSPMSPV_OK;
        }
    }
    const int64_t padded = (int64_t)((d.nb + 1) / 2) * 32;
    int64_t work = padded > d.m ? padded : d.m;
    int g = (int)((work + 255) / 256);
    if (g > 8 * h->sm_count) g = 8 * h->sm_count;
    k_xblock_dense<DT><<<g, 256, 0, st>>>(d, x, y);
    OutDense out{y, nullptr};
    if (h->ropts.timing) DBS_CUDA(cudaEventRecord(h->ev[0], st));
    if (d.n_entries > 0) {
        int s;
        if (h->heavy_stage) {
            // pull by the lean kernel of its own; the general kernel then only runs a push
            int &grid = h->grid_decode_pull;
            if (!grid) {
                int per_sm = 0;
                if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_decode_pull<DT>, CTA, 0) != cudaSuccess || per_sm < 1) return DBSPMSPV_ERR_CUDA;
                grid = per_sm * h->sm_count;
            }
            DBS_CUDA(launch_pdl(k_decode_pull<DT>, grid, CTA, 0, st, d, (const int32_t *)h->block_row, y, h->ropts.th3_decode, h->ropts.force_path));
            ++h->kernel_launches;
            s = launch_compute<DT, OutDense, 1>(h, out, h->ropts.th3_decode, true, st, 1);
        } else {
            s = DBSPMSPV_OK;
            if (h->ropts.force_path != DBSPMSPV_PATH_PULL) s = launch_compute<DT, OutDense, 0>(h, out, h->ropts.th3_decode, true, st);
            if (s == DBSPMSPV_OK && pull_possible(h, d.n, h->ropts.th3_decode)) s = launch_lean<DT, OutDense>(h, out, h->ropts.th3_decode, st);
        }
        if (s != DBSPMSPV_OK) return s;
    }
    if (h->ropts.timing) { DBS_CUDA(cudaEventRecord(h->ev[1], st)); h->timed = true; }
    h->kernel_launches += 2;
    int gc = ((d.nb + 1) / 2 + 255) / 256;
    if (gc > h->sm_count) gc = h->sm_count;
    DBS_CUDA(launch_pdl(k_decode_cleanup, gc, 256, 0, st, d));
    DBS_CUDA(cudaGetLastError());
    return DBSPMSPV_OK;
}

// dbspmspv_decode_batch: where the handle has the streaming form, groups of vectors share one
// pass over the payload -- bf16 handles: up to eight per group on the tensor cores
// (k_decode_batch_mma), with the per-column kernel launched behind it as the fallback for
// non-finite activations; fp32 handles: up to four per group in the per-column kernel.  What is
// left over (and every vector of a handle without the streaming form) goes through decode_typed.
template <int DT>
static int decode_batch_typed(dbspmspv_handle_s *h, const void *x, int64_t ldx, float *y, int64_t ldy, int32_t batch,
                              cudaStream_t st) {
    const Device &d = h->d;
    const size_t esize = (DT == DBSPMSPV_BF16 && !h->ropts.decode_x_f32) ? 2 : 4;
    const bool stream_ok = h->heavy_stage && d.stage_chunks != nullptr && (h->ropts.no_fused_decode == 0 || h->ropts.no_fused_decode == 3);
    int max_nb = 1, max_mma = 1;
    if (stream_ok) {
        for (int nb : {2, 4})
            if (BatchLayout(d.nb, nb, d.stage_bytes).total <= STREAM_MAX_SMEM) max_nb = nb;
        if (DT == DBSPMSPV_BF16)
            for (int nb : {2, 4, 8})
                if (max_nb >= (nb < 4 ? nb : 4) && BatchMmaLayout(d.nb, nb, d.stage_bytes).total <= STREAM_MAX_SMEM) max_mma = nb;
    }
    h->d.decode_tau = h->ropts.decode_threshold;
    h->d.decode_relu = h->ropts.decode_relu != 0;
    h->d.decode_x_f32 = h->ropts.decode_x_f32 != 0;
    // the per-column kernel on vectors [b0, b0 + g), g <= 4
    auto scalar_group = [&](const void *xg, float *yg, int g, int only_as_fallback) -> int {
        const int nb = g <= 2 ? 2 : 4;
        const BatchLayout lay(d.nb, nb, d.stage_bytes);
        auto kernel = nb == 2 ? k_decode_stream_batch<DT, 2> : k_decode_stream_batch<DT, 4>;
        bool &done = h->batch_configured[nb == 2 ? 0 : 1];
        if (!done) {
            DBS_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, STREAM_MAX_SMEM));
            done = true;
        }
        DBS_CUDA(launch_pdl(kernel, h->sm_count, BATCH_CTA, (size_t)lay.total, st, d, xg, ldx, yg, ldy, g, only_as_fallback));
        ++h->kernel_launches;
        return DBSPMSPV_OK;
    };
    for (int32_t b0 = 0; b0 < batch;) {
        const int left = batch - b0;
        const void *xg = static_cast<const uint8_t *>(x) + (size_t)b0 * (size_t)ldx * esize;
        float *yg = y + (size_t)b0 * (size_t)ldy;
        const int cap = DT == DBSPMSPV_BF16 && max_mma > 1 ? max_mma : max_nb;
        const int g = left < cap ? left : cap;
        if (g == 1) {
            const int s = decode_typed<DT>(h, xg, yg, st);
            if (s != DBSPMSPV_OK) return s;
            b0 += 1;
            continue;
        }
        if (h->ropts.timing) DBS_CUDA(cudaEventRecord(h->ev[0], st));
        k_zero_rows<<<(int)((d.m + 1023) / 1024), 256, 0, st>>>(yg, ldy, d.m, g);
        ++h->kernel_launches;
        if (DT == DBSPMSPV_BF16 && max_mma > 1) {
            const int nb = g <= 2 ? 2 : g <= 4 ? 4 : 8;
            const BatchMmaLayout lay(d.nb, nb, d.stage_bytes);
            auto kernel = nb == 2 ? k_decode_batch_mma<2> : nb == 4 ? k_decode_batch_mma<4> : k_decode_batch_mma<8>;
            bool &done = h->batch_mma_configured[nb == 2 ? 0 : nb == 4 ? 1 : 2];
            if (!done) {
                DBS_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, STREAM_MAX_SMEM));
                done = true;
            }
            DBS_CUDA(launch_pdl(kernel, h->sm_count, BATCH_MMA_CTA, (size_t)lay.total, st, d, xg, ldx, yg, ldy, g));
            ++h->kernel_launches;
            // the fallback for non-finite activations: returns at once unless the kernel above asked for it
            for (int q = 0; q < g; q += 4) {
                const int gq = g - q < 4 ? g - q : 4;
                const int s = scalar_group(static_cast<const uint8_t *>(xg) + (size_t)q * (size_t)ldx * esize, yg + (size_t)q * (size_t)ldy, gq, 1);
                if (s != DBSPMSPV_OK) return s;
            }
        } else {
            const int s = scalar_group(xg, yg, g, 0);
            if (s != DBSPMSPV_OK) return s;
        }
        if (h->ropts.timing) { DBS_CUDA(cudaEventRecord(h->ev[1], st)); h->timed = true; }
        DBS_CUDA(cudaGetLastError());
        b0 += g;
    }
    return DBSPMSPV_OK;
}

// ------------------------------------------------------------------------------------------
// db_sssp: single-source shortest paths as the iteration of (min, +) products (Sections 1, 6:
// SpMSpV as the primitive of GraphBLAS-style graph algorithms).  x = the vertices whose
// distance improved in the last step, with their distances; y = A (min,+) x; every y_i below
// dist_i replaces it and puts i on the next x.  The rows of y are distinct, so the relaxation
// needs no atomics on dist.
// ------------------------------------------------------------------------------------------
__global__ void k_sssp_init(float *dist, int64_t n, int32_t src, int32_t *x_idx, float *x_val, int32_t *count) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; v < n; v += stride) dist[v] = v == src ? 0.0f : __int_as_float(0x7F800000);
    if (blockIdx.x == 0 && threadIdx.x == 0) { x_idx[0] = src; x_val[0] = 0.0f; count[0] = 0; count[2] = 0; count[3] = 0; }
}

// A step whose x reaches more than this share of the stored elements is pulled (where the handle
// has a (min, +) pull): such an x is a handful of hubs or half the graph, its push is a queue of
// atomics on the hub rows, and the streaming pull reads the matrix once whatever x holds.
#ifndef DBS_SSSP_PULL_EDGE_FRAC
#define DBS_SSSP_PULL_EDGE_FRAC 0.1f
#endif

// count[0]: entries of the next x; count[2..3]: the out-edges they hold (64 bits; INLINE runs of the block-CSC view)
__global__ void k_sssp_relax(Device d, const int32_t *__restrict__ y_idx, const float *__restrict__ y_val, const int32_t *__restrict__ y_nnz,
                             float *__restrict__ dist, int32_t *__restrict__ x_idx, float *__restrict__ x_val, int32_t *count) {
    const int n = *y_nnz;
    const int lane = threadIdx.x & 31;
    const int stride = gridDim.x * blockDim.x;
    for (int k0 = (blockIdx.x * blockDim.x + threadIdx.x) - lane; k0 < n; k0 += stride) {     // warp-uniform trip count
        const int k = k0 + lane;
        bool better = false;
        int i = 0;
        float v = 0.f;
        if (k < n) { i = y_idx[k]; v = y_val[k]; better = v < dist[i]; }
        const uint32_t m = __ballot_sync(0xFFFFFFFFu, better);
        if (!m) continue;
        int base = 0;
        if (lane == 0) base = atomicAdd(count, __popc(m));
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        int deg = 0;
        if (better) {
            const int pos = base + __popc(m & ((1u << lane) - 1u));
            dist[i] = v;
            x_idx[pos] = i;
            x_val[pos] = v;
            int first;
            column_run(d, i, first, deg);
        }
        deg = __reduce_add_sync(0xFFFFFFFFu, deg);
        if (lane == 0 && deg) atomicAdd(reinterpret_cast<unsigned long long *>(count + 2), (unsigned long long)deg);
    }
}

template <int DT>
static int sssp_typed(dbspmspv_handle_s *h, int32_t src, float *dist, int32_t *n_steps, cudaStream_t st) {
    const Device &d = h->d;
    const int64_t n = d.n;
    if (!h->sssp_arena) {
        // two x lists (the relaxation writes the one the running product does not read), y, two counters
        const size_t bytes = (size_t)n * (4 * sizeof(int32_t) + 2 * sizeof(float)) + 64;
        if (cudaMalloc(&h->sssp_arena, bytes) != cudaSuccess) { h->sssp_arena = nullptr; return DBSPMSPV_ERR_ALLOC; }
        if (cudaHostAlloc(reinterpret_cast<void **>(&h->sssp_host), 4 * sizeof(int32_t), cudaHostAllocDefault) != cudaSuccess) return DBSPMSPV_ERR_ALLOC;
    }
    int32_t *xi[2], *y_idx, *ctr;
    float *xv[2], *y_val;
    {
        uint8_t *p = static_cast<uint8_t *>(h->sssp_arena);
        xi[0] = reinterpret_cast<int32_t *>(p); p += n * sizeof(int32_t);
        xi[1] = reinterpret_cast<int32_t *>(p); p += n * sizeof(int32_t);
        y_idx = reinterpret_cast<int32_t *>(p); p += n * sizeof(int32_t);
        xv[0] = reinterpret_cast<float *>(p); p += n * sizeof(float);
        xv[1] = reinterpret_cast<float *>(p); p += n * sizeof(float);
        y_val = reinterpret_cast<float *>(p); p += n * sizeof(float);
        ctr = reinterpret_cast<int32_t *>(p);                 // [0] next x count, [1] y_nnz, [2..3] out-edges of the next x
    }
    k_sssp_init<<<4 * h->sm_count, 256, 0, st>>>(dist, n, src, xi[0], xv[0], ctr);
    ++h->kernel_launches;
    int32_t nnz_x = 1;
    int64_t edges = 0;
    int steps = 0, cur = 0, status = DBSPMSPV_OK;
    const int user_path = h->ropts.force_path;
    while (nnz_x > 0) {
        if (++steps > n + 1) { status = DBSPMSPV_ERR_UNSUPPORTED; break; }          // a cycle of negative weight
        // direction of this step: the caller's, else by the share of the stored elements x reaches
        if (user_path == DBSPMSPV_PATH_AUTO)
            h->ropts.force_path = (double)edges > (double)DBS_SSSP_PULL_EDGE_FRAC * (double)d.n_entries ? DBSPMSPV_PATH_PULL : DBSPMSPV_PATH_PUSH;
        status = run_typed<DT>(h, xi[cur], xv[cur], nnz_x, DBSPMSPV_MIN_PLUS, y_idx, y_val, n, ctr + 1, st);
        if (status != DBSPMSPV_OK) break;
        k_sssp_relax<<<2 * h->sm_count, 256, 0, st>>>(d, y_idx, y_val, ctr + 1, dist, xi[cur ^ 1], xv[cur ^ 1], ctr);
        ++h->kernel_launches;
        if (cudaMemcpyAsync(h->sssp_host, ctr, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaMemsetAsync(ctr, 0, 4 * sizeof(int32_t), st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) {
            status = DBSPMSPV_ERR_CUDA;
            break;
        }
        nnz_x = h->sssp_host[0];
        edges = (int64_t)(uint32_t)h->sssp_host[2] | ((int64_t)h->sssp_host[3] << 32);
        cur ^= 1;
    }
    h->ropts.force_path = user_path;
    if (status != DBSPMSPV_OK) return status;
    if (n_steps) *n_steps = steps;
    return DBSPMSPV_OK;
}

}  // namespace dbs

extern "C" {

void dbspmspv_default_run_opts(dbspmspv_run_opts *o) {
    if (!o) return;
    *o = dbspmspv_run_opts();
    o->th3 = 0.95f;
    o->th3_bfs = 0.05f;
    o->th3_decode = 0.01f;
    o->bfs_push_max_edge_frac = 0.08f;
    o->force_path = DBSPMSPV_PATH_AUTO;
    o->popc_threshold = 8;
    o->validate = 0;
}

int dbspmspv_set_run_opts(dbspmspv_handle_t h, const dbspmspv_run_opts *opts) {
    if (!h || !opts) return DBSPMSPV_ERR_INVALID_ARG;
    if (opts->force_path < DBSPMSPV_PATH_AUTO || opts->force_path > DBSPMSPV_PATH_PULL) return DBSPMSPV_ERR_INVALID_ARG;
    if (!(opts->th3 >= 0.f) || !(opts->th3_bfs >= 0.f) || !(opts->th3_decode >= 0.f) || !(opts->bfs_push_max_edge_frac >= 0.f) ||
        !(opts->decode_threshold >= 0.f)) return DBSPMSPV_ERR_INVALID_ARG;
    h->ropts = *opts;
    return DBSPMSPV_OK;
}

static int run_checked(dbspmspv_handle_t h, const int32_t *x_idx, const void *x_val, int32_t nnz_x,
                       int semiring, int32_t *y_idx, float *y_val, int64_t y_capacity, int32_t *y_nnz,
                       dbspmspv_stream_t stream, const uint32_t *row_mask, int complement) {
    if (!h || nnz_x < 0 || y_capacity < 0 || !y_nnz) return DBSPMSPV_ERR_INVALID_ARG;
    if (nnz_x > 0 && !x_idx) return DBSPMSPV_ERR_INVALID_ARG;
    if (y_capacity > 0 && !y_idx) return DBSPMSPV_ERR_INVALID_ARG;
    if (semiring != DBSPMSPV_PLUS_TIMES && semiring != DBSPMSPV_OR_AND && semiring != DBSPMSPV_MIN_PLUS) return DBSPMSPV_ERR_INVALID_ARG;
    if (semiring == DBSPMSPV_PLUS_TIMES && h->d.dtype == DBSPMSPV_PATTERN) return DBSPMSPV_ERR_UNSUPPORTED;
    if (semiring != DBSPMSPV_OR_AND && ((nnz_x > 0 && !x_val) || (y_capacity > 0 && !y_val))) return DBSPMSPV_ERR_INVALID_ARG;
    if ((int64_t)nnz_x > h->d.n) return DBSPMSPV_ERR_INVALID_ARG;
    if (!dbs::on_handle_device(h)) return DBSPMSPV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    switch (h->d.dtype) {
        case DBSPMSPV_F32: return dbs::run_typed<DBSPMSPV_F32>(h, x_idx, x_val, nnz_x, semiring, y_idx, y_val, y_capacity, y_nnz, st, row_mask, complement);
        case DBSPMSPV_BF16: return dbs::run_typed<DBSPMSPV_BF16>(h, x_idx, x_val, nnz_x, semiring, y_idx, y_val, y_capacity, y_nnz, st, row_mask, complement);
        default: return dbs::run_typed<DBSPMSPV_PATTERN>(h, x_idx, x_val, nnz_x, semiring, y_idx, y_val, y_capacity, y_nnz, st, row_mask, complement);
    }
}

int dbspmspv_run(dbspmspv_handle_t h, const int32_t *x_idx, const void *x_val, int32_t nnz_x,
                 int semiring, int32_t *y_idx, float *y_val, int64_t y_capacity, int32_t *y_nnz,
                 dbspmspv_stream_t stream) {
    return run_checked(h, x_idx, x_val, nnz_x, semiring, y_idx, y_val, y_capacity, y_nnz, stream, nullptr, 0);
}

int dbspmspv_run_masked(dbspmspv_handle_t h, const int32_t *x_idx, const void *x_val, int32_t nnz_x,
                        int semiring, const uint32_t *row_mask, int complement, int32_t *y_idx, float *y_val,
                        int64_t y_capacity, int32_t *y_nnz, dbspmspv_stream_t stream) {
    if (!row_mask || (complement != 0 && complement != 1)) return DBSPMSPV_ERR_INVALID_ARG;
    return run_checked(h, x_idx, x_val, nnz_x, semiring, y_idx, y_val, y_capacity, y_nnz, stream, row_mask, complement);
}

int db_sssp(dbspmspv_handle_t h, int32_t src, float *dist, int32_t *n_steps, dbspmspv_stream_t stream) {
    if (!h || !dist) return DBSPMSPV_ERR_INVALID_ARG;
    if (h->d.m != h->d.n) return DBSPMSPV_ERR_UNSUPPORTED;
    if (h->d.dtype == DBSPMSPV_BF16) return DBSPMSPV_ERR_UNSUPPORTED;    // distances are fp32; x would have to be bf16
    if (src < 0 || src >= h->d.n) return DBSPMSPV_ERR_INVALID_ARG;
    if (!dbs::on_handle_device(h)) return DBSPMSPV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    return h->d.dtype == DBSPMSPV_F32 ? dbs::sssp_typed<DBSPMSPV_F32>(h, src, dist, n_steps, st)
                                      : dbs::sssp_typed<DBSPMSPV_PATTERN>(h, src, dist, n_steps, st);
}

int dbspmspv_test_bounded_wait(dbspmspv_handle_t h, int32_t max_tries, dbspmspv_stream_t stream) {
    if (!h || max_tries < 1 || max_tries > 4096) return DBSPMSPV_ERR_INVALID_ARG;
    if (!dbs::on_handle_device(h)) return DBSPMSPV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    dbs::k_wait_probe<<<1, 32, 0, st>>>(h->d, max_tries);
    ++h->kernel_launches;
    DBS_CUDA(cudaGetLastError());
    return DBSPMSPV_OK;
}

int dbspmspv_decode_batch(dbspmspv_handle_t h, const void *x, int64_t ldx, float *y, int64_t ldy, int32_t batch,
                          dbspmspv_stream_t stream) {
    if (!h || !x || !y || batch < 1 || ldx < h->d.n || ldy < h->d.m) return DBSPMSPV_ERR_INVALID_ARG;
    if (!dbs::on_handle_device(h)) return DBSPMSPV_ERR_INVALID_ARG;
    if (h->d.dtype == DBSPMSPV_PATTERN) return DBSPMSPV_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    return h->d.dtype == DBSPMSPV_F32 ? dbs::decode_batch_typed<DBSPMSPV_F32>(h, x, ldx, y, ldy, batch, st)
                                      : dbs::decode_batch_typed<DBSPMSPV_BF16>(h, x, ldx, y, ldy, batch, st);
}

int dbspmspv_test_corrupt_entry(dbspmspv_handle_t h, int32_t position, uint32_t block_index) {
#ifdef DBS_BOUNDS_CHECK
    if (!h || position < 0 || position >= h->d.n_entries || block_index > dbs::IDX_MASK) return DBSPMSPV_ERR_INVALID_ARG;
    if (!dbs::on_handle_device(h)) return DBSPMSPV_ERR_INVALID_ARG;
    uint32_t v = 0;
    DBS_CUDA(cudaMemcpy(&v, h->d.csr.idx + position, 4, cudaMemcpyDeviceToHost));
    v = (v & ~dbs::IDX_MASK) | block_index;
    DBS_CUDA(cudaMemcpy(h->d.csr.idx + position, &v, 4, cudaMemcpyHostToDevice));
    return DBSPMSPV_OK;
#else
    (void)h; (void)position; (void)block_index;
    return DBSPMSPV_ERR_UNSUPPORTED;
#endif
}

int dbspmspv_decode(dbspmspv_handle_t h, const void *x, float *y, dbspmspv_stream_t stream) {
    if (!h || !x || !y) return DBSPMSPV_ERR_INVALID_ARG;
    if (!dbs::on_handle_device(h)) return DBSPMSPV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    switch (h->d.dtype) {
        case DBSPMSPV_F32: return dbs::decode_typed<DBSPMSPV_F32>(h, x, y, st);
        case DBSPMSPV_BF16: return dbs::decode_typed<DBSPMSPV_BF16>(h, x, y, st);
        default: return DBSPMSPV_ERR_UNSUPPORTED;
    }
}

}  // extern "C"
