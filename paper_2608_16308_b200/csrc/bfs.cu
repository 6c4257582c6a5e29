// DB-BFS (Section 4.2, Algorithm 5): level-synchronous BFS where every level is one Boolean
// SpMSpV.  The frontier lives directly in the vector-block masks, visited vertices are stripped
// with a second set of masks, and push or pull is chosen per level from the ratio of nonempty
// frontier blocks (Section 3.3.1) without rebuilding anything.  The whole traversal is ONE
// cooperative launch: levels are separated by grid-wide barriers (co-residency is guaranteed
// by the cooperative launch), so there is no host round trip per level.
#include <cooperative_groups.h>

#include "internal.cuh"
#include "microkernels.cuh"
#include "worklist.cuh"

namespace cg = cooperative_groups;

namespace dbs {

#ifndef DBS_BFS_CTA
#define DBS_BFS_CTA 1024   // one thread block per SM: a grid barrier over 148 blocks costs far less than over a thousand
#endif
constexpr int BFS_CTA = DBS_BFS_CTA;

// Rows of one hypersparse block reached from the active columns (one lane per block).
template <int DT>
__device__ __forceinline__ uint32_t lane_block_bool(int type, uint32_t w, uint32_t aux, uint32_t xm,
                                                    const uint8_t *payload) {
    uint32_t hit = 0;
    if (type == DBSPMSPV_BLK_INLINE) {
        hit = ((xm >> (aux & 15)) & 1u) << (aux >> 4);
    } else {
        const uint8_t *blk = payload + (size_t)w * 4;
        for (uint32_t k = 0; k <= aux; ++k) {
            const uint32_t rc = blk[k];
            if ((xm >> (rc & 15)) & 1u) hit |= 1u << (rc >> 4);
        }
    }
    return hit;
}

__device__ __forceinline__ void write_levels(int32_t *levels, int rb, uint32_t fresh, int depth) {
    while (fresh) {
        const int r = __ffs(fresh) - 1;
        fresh &= fresh - 1;
        levels[rb * 16 + r] = depth;
    }
}

// The threads that share a level's work (the whole cooperative grid).
struct Scope {
    int tid, nthreads;      // thread index / count in the scope
    int gwarp, nwarps;      // warp index / count in the scope
};

// Appends word indices (one per lane with `word` >= 0) to a list: one atomic per warp.
__device__ __forceinline__ void append_words(int word, int32_t *list, int32_t *count, int lane) {
    const uint32_t m = __ballot_sync(FULL, word >= 0);
    if (!m) return;
    int base = 0;
    if (lane == __ffs(m) - 1) base = atomicAdd(count, __popc(m));
    base = __shfl_sync(FULL, base, __ffs(m) - 1);
    if (word >= 0) list[base + __popc(m & ((1u << lane) - 1u))] = word;
}

// Boolean push: tasks of the active frontier blocks (a task is at most PUSH_CHUNK = 32 view
// entries: one warp step); newly reached rows are claimed with one atomicOr per entry on the
// next-frontier masks (the winner writes the level).  Like the pull, the loop is software-
// pipelined: while task k is evaluated, the visited masks of k+1, the view entries of k+2 and
// the task record of k+3 (in this warp's stride) are in flight.  The thread whose atomic turns a
// word of the next-frontier masks nonzero lists that word, so that the bookkeeping after the
// level visits the nonzero words only.
template <int DT>
__device__ void bfs_push(const Device &d, const Scope &sc, const uint32_t *F, uint32_t *N, int n_recs, const int4 *hubs, int n_hubs,
                         int32_t *levels, int depth, int32_t *words_out, int32_t *nwords_out) {
    static_assert(PUSH_CHUNK == 32, "one warp step per task");
    const int lane = threadIdx.x & 31;
    const int gwarp = sc.gwarp, nwarps = sc.nwarps;
    const HubTable table = load_hub_table(hubs, n_hubs, lane);
    const int n_tasks = n_recs + table.total;                    // task records, then the steps of the hub runs
    auto item = [&](int i) { return worklist_item(d.ws.tasks, n_recs, table, i); };
    const uint2 none = make_uint2(0u, 0u);
    struct Entries { uint32_t idx, aux, xm; int n, start; };   // n: entries of the task (0 = no task)
    auto entries_of = [&](int t, const uint2 &task) {
        Entries e{0u, 0u, 0u, 0, 0};
        if (t < n_tasks) {
            const int jb = (int)(task.x & IDX_MASK), start = (int)task.y;
            e.n = (int)(task.x >> 27) + 1;
            e.start = start;
            if (lane < e.n && DBS_CHK_RANGE(d, start, e.n) && DBS_CHK_INDEX(d, jb, d.nb)) {
                e.idx = d.csc.idx[start + lane]; e.aux = d.csc.aux[start + lane];
#ifdef DBS_BOUNDS_CHECK
                uint32_t w_ = d.csc.w[start + lane];
                DBS_CHK_ENTRY(d, false, e.idx, w_, e.aux);
#endif
            }
            e.xm = mask_of(F, jb);
        }
        return e;
    };
    auto need_of = [&](const Entries &e) { return lane < e.n ? ~mask_of(d.ws.visited32, e.idx & IDX_MASK) & 0xFFFFu : 0u; };
    uint2 t1 = gwarp + nwarps < n_tasks ? item(gwarp + nwarps) : none;
    uint2 t2 = gwarp + 2 * nwarps < n_tasks ? item(gwarp + 2 * nwarps) : none;
    uint2 t0 = gwarp < n_tasks ? item(gwarp) : none;
    Entries e0 = entries_of(gwarp, t0);
    Entries e1 = entries_of(gwarp + nwarps, t1);
    uint32_t need0 = need_of(e0);
    for (int t = gwarp; t < n_tasks; t += nwarps) {
        const uint2 t3 = t + 3 * nwarps < n_tasks ? item(t + 3 * nwarps) : none;          // stage 1
        const Entries e2 = entries_of(t + 2 * nwarps, t2);                                // stage 2
        const uint32_t need1 = need_of(e1);                                               // stage 3
        // stage 4: evaluate task t
        {
            const uint32_t idx = e0.idx, aux = e0.aux, xm = e0.xm;
            const int type = idx >> TYPE_SHIFT, brow = idx & IDX_MASK;
            bool heavy = false;
            uint32_t w = 0;
            int fresh_word = -1;           // a mask word this lane turned nonzero
            if (need0) {
                uint32_t hit = 0;
                if (type == DBSPMSPV_BLK_INLINE) {
                    hit = ((xm >> (aux & 15)) & 1u) << (aux >> 4);
                } else {
                    w = d.csc.w[e0.start + lane];
                    if (type == DBSPMSPV_BLK_COO) {
                        if (aux < COO_SERIAL_MAX) hit = lane_block_bool<DT>(type, w, aux, xm, d.payload);
                        else heavy = true;
                    } else {
                        hit = lane_heavy_bool(type, d.payload + (size_t)w * 4, xm);
                    }
                }
                hit &= need0;
                if (hit) {
                    const int sh = (brow & 1) * 16;
                    const uint32_t old = atomicOr(&N[brow >> 1], hit << sh);
                    write_levels(levels, brow, hit & ~(old >> sh), depth);
                    if (!old) fresh_word = brow >> 1;
                }
            }
            append_words(fresh_word, words_out, nwords_out, lane);
            uint32_t hv = __ballot_sync(FULL, heavy);
            while (hv) {
                const int src = __ffs(hv) - 1;
                hv &= hv - 1;
                const uint32_t bidx = __shfl_sync(FULL, idx, src);
                const uint32_t bw = __shfl_sync(FULL, w, src);
                const int nnz = (int)__shfl_sync(FULL, aux, src) + 1;
                const int btype = bidx >> TYPE_SHIFT, bbrow = bidx & IDX_MASK;
                uint32_t hits = warp_block_bool<DT>(btype, d.payload + (size_t)bw * 4, nnz, xm, lane);
                hits &= ~mask_of(d.ws.visited32, bbrow);
                if (lane == 0 && hits) {
                    const int sh = (bbrow & 1) * 16;
                    const uint32_t old = atomicOr(&N[bbrow >> 1], hits << sh);
                    write_levels(levels, bbrow, hits & ~(old >> sh), depth);
                    if (!old) words_out[atomicAdd(nwords_out, 1)] = bbrow >> 1;
                }
            }
        }
        // rotate the pipeline
        e0 = e1; e1 = e2; need0 = need1; t2 = t3;
    }
}

// Boolean pull: one warp per row-block segment (a segment has at most MAX_SEG_ENTRIES = 4 x 32
// view entries, so one round of four warp steps covers it); row blocks with nothing left to
// discover are skipped.  A segment costs a chain of dependent loads (descriptor -> visited mask
// -> view entries -> frontier masks); the loop is software-pipelined four deep so that only the
// last link is waited for: while segment k is evaluated, the entries of k+1, the visited mask
// of k+2 and the descriptor of k+3 (k counted in this warp's stride) are already in flight.
template <int DT>
__device__ void bfs_pull(const Device &d, const Scope &sc, const uint32_t *F, uint32_t *N, int32_t *levels, int depth) {
    constexpr int U = MAX_SEG_ENTRIES / 32;
    const int lane = threadIdx.x & 31;
    const int gwarp = sc.gwarp, nwarps = sc.nwarps;
    const int nseg = d.n_segments;
    const Segment none = Segment{0, 0, 0, 0};
    auto need_of = [&](const Segment &sg) { return (sg.count & 0x7FFFFFFF) ? ~mask_of(d.ws.visited32, sg.row_block) & 0xFFFFu : 0u; };
    // prologue: fill the pipeline
    Segment s0 = gwarp < nseg ? d.segments[gwarp] : none;
    Segment s1 = gwarp + nwarps < nseg ? d.segments[gwarp + nwarps] : none;
    Segment s2 = gwarp + 2 * nwarps < nseg ? d.segments[gwarp + 2 * nwarps] : none;
    uint32_t need0 = need_of(s0), need1 = need_of(s1);
    // the entries of a segment: lane l takes positions l, l + 32, ... (constant offsets from one
    // pointer per array, one comparison per step)
    auto fetch = [&](const Segment &sg, uint32_t need, uint32_t (&idx)[U], uint32_t (&aux)[U]) {
        const uint32_t *ip = d.csr.idx + sg.start + lane;
        const uint8_t *ap = d.csr.aux + sg.start + lane;
        const int rem = need && DBS_CHK_RANGE(d, sg.start, sg.count & 0x7FFFFFFF) ? (sg.count & 0x7FFFFFFF) - lane : 0;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            idx[u] = 0; aux[u] = 0;
            if (rem > u * 32) { idx[u] = ip[u * 32]; aux[u] = ap[u * 32]; }
        }
    };
    uint32_t idx0[U], aux0[U];
    fetch(s0, need0, idx0, aux0);
    for (int sg = gwarp; sg < nseg; sg += nwarps) {
        // stage 1: descriptor three strides ahead
        const Segment s3 = sg + 3 * nwarps < nseg ? d.segments[sg + 3 * nwarps] : none;
        // stage 2: visited mask two strides ahead
        const uint32_t need2 = need_of(s2);
        // stage 3: view entries one stride ahead
        uint32_t idx1[U], aux1[U];
        fetch(s1, need1, idx1, aux1);
        // stage 4: evaluate this segment
        if (need0) {
            const int cnt0 = s0.count & 0x7FFFFFFF;
            const int rb = s0.row_block;
            // frontier masks: only for entries that can still contribute -- past-the-end entries
            // are all-zero (INLINE, row 0); an INLINE entry whose row is not wanted is skipped
            // (late pull levels want one or two rows of a row block: most gathers fall away)
            const int rem0 = cnt0 - lane;
            uint32_t xm[U];
            bool heavy_any = false;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const bool inl = (idx0[u] >> TYPE_SHIFT) == DBSPMSPV_BLK_INLINE;
                const bool want = rem0 > u * 32 && (!inl || ((need0 >> (aux0[u] >> 4)) & 1u));
                xm[u] = want ? mask_of(F, idx0[u] & IDX_MASK) : 0u;
                heavy_any |= want && !inl;
            }
            uint32_t hit = 0;
#pragma unroll
            for (int u = 0; u < U; ++u)        // INLINE entries: branch-free (xm is 0 where not wanted)
                hit |= ((idx0[u] >> TYPE_SHIFT) == DBSPMSPV_BLK_INLINE ? (xm[u] >> (aux0[u] & 15)) & 1u : 0u) << (aux0[u] >> 4);
            if (__any_sync(FULL, heavy_any)) {   // rare: packed-COO and mask-based blocks
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (u * 32 >= cnt0) break;      // warp-uniform
                    const int type = idx0[u] >> TYPE_SHIFT;
                    bool heavy = false;
                    uint32_t w = 0;
                    if (xm[u] && type != DBSPMSPV_BLK_INLINE) {
                        w = d.csr.w[s0.start + u * 32 + lane];
                        if (type == DBSPMSPV_BLK_COO) {
                            if (aux0[u] < COO_SERIAL_MAX) hit |= lane_block_bool<DT>(type, w, aux0[u], xm[u], d.payload);
                            else heavy = true;
                        } else {
                            hit |= lane_heavy_bool(type, d.payload + (size_t)w * 4, xm[u]);
                        }
                    }
                    uint32_t hv = __ballot_sync(FULL, heavy);
                    while (hv) {
                        const int src = __ffs(hv) - 1;
                        hv &= hv - 1;
                        const uint32_t bidx = __shfl_sync(FULL, idx0[u], src);
                        const uint32_t bw = __shfl_sync(FULL, w, src);
                        const int nnz = (int)__shfl_sync(FULL, aux0[u], src) + 1;
                        const uint32_t bxm = __shfl_sync(FULL, xm[u], src);
                        hit |= warp_block_bool<DT>(bidx >> TYPE_SHIFT, d.payload + (size_t)bw * 4, nnz, bxm, lane);
                    }
                }
            }
            hit = __reduce_or_sync(FULL, hit) & need0;
            if (hit) {
                if (s0.count < 0) {          // the segment is its whole row block: plain stores
                    if (lane == 0) reinterpret_cast<uint16_t *>(N)[rb] = (uint16_t)hit;
                    if (lane < 16 && ((hit >> lane) & 1u)) levels[rb * 16 + lane] = depth;
                } else if (lane == 0) {
                    const int sh = (rb & 1) * 16;
                    const uint32_t old = atomicOr(&N[rb >> 1], hit << sh);
                    write_levels(levels, rb, hit & ~(old >> sh), depth);
                }
            }
        }
        // rotate the pipeline
        s0 = s1; s1 = s2; s2 = s3;
        need0 = need1; need1 = need2;
#pragma unroll
        for (int u = 0; u < U; ++u) { idx0[u] = idx1[u]; aux0[u] = aux1[u]; }
    }
}

// Boolean pull over the row-run index (square matrices, unless the index was switched off).
// Entries with a payload are evaluated first, from the per-row-block position list, and a row
// block is left as soon as each of its wanted rows has a parent; then every row that is still
// wanted walks its own INLINE run and stops at its first frontier neighbour -- the early exit of
// Algorithm 5 per row instead of per row block: in the big levels a row finds a parent within a
// few entries, so a fraction of the edges is read at all.
// A warp takes a block of W = 32 consecutive mask words (1024 rows; fewer on small graphs) and lane l walks one row of
// every word (row (l + k) mod 32 of the block's word k), one row after the other, each lane at its own pace.  (With lane = row inside ONE word a
// word costs as many dependent rounds as its slowest row -- and at the levels with a small
// frontier almost every word holds a row without a frontier neighbour, which is walked to its
// end -- so a warp's time would be the sum over its words of the maximum; here it is the maximum
// over the lanes of the sum, about a third of the rounds.)  Four entries are fetched per round
// and lane (eight when the frontier is small), then their frontier masks; the run of the lane's
// next row is fetched meanwhile.  A row that has not finished after eight rounds is long (a hub
// with no frontier neighbour so far) and is finished by the whole warp, 32 * 8 entries per step.
// Found rows are collected as one bit per (lane, word) and transposed back with ballots, so the
// warp owns its mask words: plain stores, no atomics.
// a pull level over a frontier that fills fewer than this share of the vector blocks reads two groups of four entries per round
#ifndef DBS_BFS_WIDE_PULL
#define DBS_BFS_WIDE_PULL 0.3f
#endif
constexpr float BFS_WIDE_PULL = DBS_BFS_WIDE_PULL;

template <int DT>
__device__ void bfs_pull_rows(const Device &d, const uint32_t *F, uint32_t *N, uint32_t *Z, int32_t *nz_out, int32_t *words_out,
                                int32_t *nwords_out, int32_t *levels, int depth, bool wide, uint32_t *s_need) {
    const int lane = threadIdx.x & 31;
    const int gwarp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    const int n_words = (d.mb + 1) / 2;
    constexpr uint32_t NONE = 0xFFFFFFFFu;          // no entry: local column 31 never matches a 16-bit mask
    constexpr int LONG_UNROLL = 8, MAX_ROUNDS = 8;
    const int per_round = wide ? 8 : 4;
    int n_found = 0, n_nz = 0;
    // words per warp: 32, or -- on a graph with fewer mask words than that keeps every warp busy --
    // the smallest power of two with which one pass of all warps covers the words (a lane then
    // walks W rows; with 32-word blocks a graph of 2^18 vertices gave work to 256 of 4736 warps)
    int W = 32;
    while (W > 1 && (int64_t)nwarps * (W / 2) >= n_words) W >>= 1;
    for (int w0 = gwarp * W; w0 < n_words; w0 += nwarps * W) {
        const int wd = w0 + lane;                    // this lane's word (bookkeeping); rows: lane = row of every word
        const bool in = lane < W && wd < n_words;
        const uint32_t need = in ? ~d.ws.visited32[wd] : 0u;   // (rows without stored elements and rows past m count as visited)
        if (in) Z[wd] = 0u;
        if (!__any_sync(FULL, need != 0u)) { if (in) N[wd] = 0u; continue; }
        uint32_t found = 0u;
        // entries with a payload: the words that have any (their two row blocks' ranges), one word at a time
        {
            int pb0 = 0, pe0 = 0, pb1 = 0, pe1 = 0;
            if (need) {
                const int rb = 2 * wd;
                if (rb < d.mb) { pb0 = d.csr.ptr[rb]; pe0 = d.csr_inl[rb]; }
                if (rb + 1 < d.mb) { pb1 = d.csr.ptr[rb + 1]; pe1 = d.csr_inl[rb + 1]; }
            }
            uint32_t todo = __ballot_sync(FULL, need && (pe0 > pb0 || pe1 > pb1));
            while (todo) {
                const int k = __ffs(todo) - 1;
                todo &= todo - 1;
                const uint32_t need_k = __shfl_sync(FULL, need, k);
                uint32_t fk = 0u;
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const uint32_t need16 = (need_k >> (16 * hf)) & 0xFFFFu;
                    const int pbeg = __shfl_sync(FULL, hf ? pb1 : pb0, k), pend = __shfl_sync(FULL, hf ? pe1 : pe0, k);
                    if (!need16 || pend <= pbeg) continue;        // warp-uniform
                    uint32_t hit = 0;
                    for (int base = pbeg; base < pend; base += 32) {
                        const int pos = base + lane;
                        if (pos < pend) {
                            uint32_t idx = d.csr.idx[pos], aux = d.csr.aux[pos];
#ifdef DBS_BOUNDS_CHECK
                            { uint32_t w_ = d.csr.w[pos]; DBS_CHK_ENTRY(d, true, idx, w_, aux); }
#endif
                            const uint32_t xm = mask_of(F, idx & IDX_MASK);
                            if (xm) {
                                const int type = idx >> TYPE_SHIFT;
                                const uint32_t w = d.csr.w[pos];
                                hit |= type == DBSPMSPV_BLK_COO ? lane_block_bool<DT>(type, w, aux, xm, d.payload)
                                                                : lane_heavy_bool(type, d.payload + (size_t)w * 4, xm);
                            }
                        }
                        hit = __reduce_or_sync(FULL, hit);
                        if ((hit & need16) == need16) break;      // every wanted row of the block has a parent
                    }
                    fk |= (hit & need16) << (16 * hf);
                }
                if ((fk >> lane) & 1u) levels[(size_t)(w0 + k) * 32 + lane] = depth;
                if (lane == k) found |= fk;
            }
        }
        // rows: bit k of `mine` = row (lane + k) mod 32 of word w0 + k is still wanted.  (The rotation matters where
        // the degree goes with the low bits of the row number, as in an R-MAT graph that was not relabelled: with
        // row = lane, lane 0 would own the heaviest row of every word.)
        __syncwarp();
        s_need[lane] = need & ~found;
        __syncwarp();
        uint32_t mine = 0u;
#pragma unroll 8
        for (int k = 0; k < 32; ++k) mine |= ((s_need[k] >> ((lane + k) & 31)) & 1u) << k;
        uint32_t res = 0u, longm = 0u;
        int k = 0, p = 0, e = 0, rounds = 0;
        bool active = false;
        // (the run of the lane's next row is fetched while the current one is walked)
        int kn = 0, pn = 0, en = 0;
        bool have_next = false;
        auto fetch_next = [&]() {
            have_next = mine != 0u;
            if (have_next) {
                kn = __ffs(mine) - 1;
                mine &= mine - 1;
                const size_t row = (size_t)(w0 + kn) * 32 + ((lane + kn) & 31);
                pn = d.rowrun_ptr[row];
                en = d.rowrun_ptr[row + 1];
            }
        };
        fetch_next();
        while (__any_sync(FULL, active || have_next)) {
            if (!active && have_next) {               // next row of this lane
                k = kn; p = pn; e = en;
                active = p < e;
                rounds = 0;
                fetch_next();
            }
            if (active) {
                // a round = the aligned group(s) of four entries from position p on: 16-byte loads
                const int q0 = p & ~3;
                uint4 v4 = __ldcs(reinterpret_cast<const uint4 *>(d.rowrun_idx + q0)), w4 = make_uint4(NONE, NONE, NONE, NONE);   // (the array has slack behind its end)
                if (wide && q0 + 4 < e) w4 = __ldcs(reinterpret_cast<const uint4 *>(d.rowrun_idx + q0 + 4));
                uint32_t v[8] = {v4.x, v4.y, v4.z, v4.w, w4.x, w4.y, w4.z, w4.w}, xm[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) if (q0 + j < p || q0 + j >= e || (v[j] != NONE && !DBS_CHK_INDEX(d, v[j] & IDX_MASK, d.nb))) v[j] = NONE;
#pragma unroll
                for (int j = 0; j < 8; ++j) xm[j] = v[j] != NONE ? mask_of(F, v[j] & IDX_MASK) : 0u;
                bool got = false;
#pragma unroll
                for (int j = 0; j < 8; ++j) got |= ((xm[j] >> (v[j] >> 27)) & 1u) != 0;
                p = q0 + per_round;
                if (got) { res |= 1u << k; levels[(size_t)(w0 + k) * 32 + ((lane + k) & 31)] = depth; active = false; }
                else if (p >= e) active = false;
                else if (++rounds == MAX_ROUNDS) { longm |= 1u << k; active = false; }     // a long row: finished by the whole warp below
            }
        }
        // long rows (hubs with no frontier neighbour among their first entries): the whole warp, 32 * LONG_UNROLL entries per round
        uint32_t lanes_long = __ballot_sync(FULL, longm != 0u);
        while (lanes_long) {
            const int src = __ffs(lanes_long) - 1;
            lanes_long &= lanes_long - 1;
            uint32_t lm = __shfl_sync(FULL, longm, src);
            while (lm) {
                const int kk = __ffs(lm) - 1;
                lm &= lm - 1;
                const size_t row = (size_t)(w0 + kk) * 32 + ((src + kk) & 31);
                const int lp = (d.rowrun_ptr[row] & ~3) + MAX_ROUNDS * per_round, le = d.rowrun_ptr[row + 1];
                bool hit = false;
                for (int q = lp; q < le && !hit; q += 32 * LONG_UNROLL) {
                    uint32_t v[LONG_UNROLL], xm[LONG_UNROLL];
#pragma unroll
                    for (int u = 0; u < LONG_UNROLL; ++u) {
                        const int p_ = q + 32 * u + lane;
                        v[u] = p_ < le ? d.rowrun_idx[p_] : NONE;
                        if (v[u] != NONE && !DBS_CHK_INDEX(d, v[u] & IDX_MASK, d.nb)) v[u] = NONE;
                    }
#pragma unroll
                    for (int u = 0; u < LONG_UNROLL; ++u) xm[u] = v[u] != NONE ? mask_of(F, v[u] & IDX_MASK) : 0u;
                    bool m1 = false;
#pragma unroll
                    for (int u = 0; u < LONG_UNROLL; ++u) m1 |= ((xm[u] >> (v[u] >> 27)) & 1u) != 0;
                    hit = __any_sync(FULL, m1);
                }
                if (hit && lane == src) { res |= 1u << kk; levels[row] = depth; }
            }
        }
        // back to one word per lane: bit (l + k) mod 32 of word w0 + k <- bit k of lane l's result
        for (int kk = 0; kk < W; ++kk) {
            const uint32_t fk = __ballot_sync(FULL, (res >> kk) & 1u);
            if (lane == kk) found |= __funnelshift_l(fk, fk, kk);
        }
        found &= need;
        if (in) N[wd] = found;
        if (found) d.ws.visited32[wd] |= found;
        n_found += __popc(found);
        n_nz += ((found & 0xFFFFu) != 0) + ((found >> 16) != 0);
        const uint32_t listed = __ballot_sync(FULL, found != 0u);
        if (listed) {
            int base = 0;
            if (lane == 0) base = atomicAdd(nwords_out, __popc(listed));
            base = __shfl_sync(FULL, base, 0);
            if (found) words_out[base + __popc(listed & ((1u << lane) - 1u))] = wd;
        }
    }
    n_found = __reduce_add_sync(FULL, n_found);
    n_nz = __reduce_add_sync(FULL, n_nz);
    if (lane == 0 && n_found) { atomicAdd(&d.ws.ctr->bfs_reached, n_found); atomicAdd(nz_out, n_nz); }
}

// Per-level selector (Section 3.3.1): push iff N_nzblk / N_blk < th3.  Monotone in n_nzblk.
__device__ __forceinline__ int bfs_path(int n_nzblk, int nb, float th3, int force_path) {
    if (force_path == DBSPMSPV_PATH_PUSH || force_path == DBSPMSPV_PATH_PULL) return force_path;
    return ((float)n_nzblk / (float)nb < th3) ? DBSPMSPV_PATH_PUSH : DBSPMSPV_PATH_PULL;
}

// Worklist of the frontier F from the listed nonzero words of its masks: a warp takes one word
// (two vector blocks) at a time, lane = column; frontier columns emit their INLINE runs (adjacent
// ones merged), lanes 0 and 16 the payload runs of the two blocks.  (With the words in index
// order, the few warps that held the hub blocks of an early frontier wrote almost the whole
// worklist.)  With UPDATE the same pass also does the level's bookkeeping for the word: visited
// is updated and the vertices found and the nonempty blocks are counted.
template <bool UPDATE>
__device__ void bfs_worklist(const Device &d, const Scope &sc, const uint32_t *F, const int32_t *words, int n_listed,
                             int32_t *n_tasks, int32_t *n_hubs, int4 *hubs, int32_t *nz_out) {
    const int lane = threadIdx.x & 31;
    Counters *ctr = d.ws.ctr;
    int found = 0, nz = 0;
    for (int i = sc.gwarp; i < n_listed; i += sc.nwarps) {
        const int wd = words[i];
        const uint32_t word = F[wd];
        if (UPDATE) {
            if (lane == 0) d.ws.visited32[wd] |= word;
            found += __popc(word);
            nz += ((word & 0xFFFFu) != 0) + ((word >> 16) != 0);
        }
        const int jb = 2 * wd + (lane >> 4), j = jb * 16 + (lane & 15);
        const bool listed = (word >> lane) & 1u;
        int first = 0, deg = 0;
        if (listed) column_run(d, j, first, deg);
        merge_column_runs(listed, j, first, deg, lane);
        emit_tasks(d, false, jb, first, deg, lane, n_tasks, &ctr->pad, PUSH_CHUNK, n_hubs, hubs);
        first = 0; deg = 0;
        if ((lane & 15) == 0 && ((word >> lane) & 0xFFFFu)) payload_run(d, jb, first, deg);
        if (__any_sync(FULL, deg > 0)) emit_tasks(d, false, jb, first, deg, lane, n_tasks, &ctr->pad, d.payload_chunk);
    }
    if (UPDATE && lane == 0 && found) { atomicAdd(&ctr->bfs_reached, found); atomicAdd(nz_out, nz); }
}

// Path of the level whose counters are set `cur` (Section 3.3.1): push iff the ratio of nonempty
// frontier blocks is below th3 -- and, the worklist of a push level being built by then, iff that
// worklist is short: a frontier of a few hub vertices fills few vector blocks but owns a good
// part of all stored elements, and a pull, which stops every row at its first frontier
// neighbour, reads less than the push of all those elements would (edge_frac = the share of
// the view's entries above which the push is given up; 0 = block ratio only).
__device__ __forceinline__ int bfs_level_path(const Device &d, int cur, float th3, float edge_frac, int force_path) {
    const Counters *ctr = d.ws.ctr;
    int path = bfs_path(ctr->bfs_cnt[cur][0], d.nb, th3, force_path);
    if (path == DBSPMSPV_PATH_PUSH && force_path == DBSPMSPV_PATH_AUTO && edge_frac > 0.f && d.rowrun_ptr != nullptr) {
        // warp steps of the worklist: the task records plus the steps of the listed hub runs
        const int n_hubs = min(ctr->bfs_hubs[cur], HUB_CAP);
        int64_t steps = ctr->bfs_cnt[cur][1];
        for (int k = 0; k < n_hubs; ++k) steps += (d.ws.hubs[cur * HUB_CAP + k].z + PUSH_CHUNK - 1) / PUSH_CHUNK;
        if ((float)steps * (float)PUSH_CHUNK > edge_frac * (float)d.n_entries) path = DBSPMSPV_PATH_PULL;
    }
    return path;
}

// One level of the search: the expansion of the frontier of level lv.  Three mask buffers rotate:
// F holds the frontier, N receives the next one, Z (the frontier before) is cleared meanwhile and
// becomes N of the next level.  Four lists of nonzero mask words rotate with them -- the list of
// the frontier produced by level L is list L % 4 -- and three sets of per-level counters, so
// that nothing is moved or reset behind an extra barrier.
template <int DT>
__device__ void bfs_level(const Device &d, cg::grid_group &grid, const Scope &sc, int lv, int32_t *levels, float th3,
                          float edge_frac, int force_path, uint32_t *s_need) {
    Counters *ctr = d.ws.ctr;
    const int lane = threadIdx.x & 31;
    const int n_words = (d.mb + 1) / 2;
    uint32_t *const buf[3] = {d.ws.x_mask32, d.ws.y_mask32, d.ws.z_mask32};
    const int cur = lv % 3, nxt = (lv + 1) % 3, spare = (lv + 2) % 3;
    const uint32_t *F = buf[cur];
    uint32_t *N = buf[nxt], *Z = buf[spare];
    const int q_out = lv & 3, q_z = (lv + 2) & 3, q_next = (lv + 1) & 3;    // lists: produced now / of Z / produced next
    int32_t *words_out = d.ws.bfs_words + (size_t)q_out * d.ws.bfs_words_stride;
    const int32_t *words_z = d.ws.bfs_words + (size_t)q_z * d.ws.bfs_words_stride;
    const int depth = lv + 1;
    const int n_nzblk = ctr->bfs_cnt[cur][0];
    const int n_tasks = ctr->bfs_cnt[cur][1];
    const int path = bfs_level_path(d, cur, th3, edge_frac, force_path);
    // counters that come into use at the next level are reset now: nobody reads or writes them
    // during this one (the previous level was their last reader, behind a barrier)
    if (sc.tid == 0) {
        ctr->bfs_cnt[spare][0] = 0;
        ctr->bfs_cnt[spare][1] = 0;
        ctr->bfs_hubs[spare] = 0;
        ctr->bfs_nwords[q_next] = 0;
        if (depth <= DBSPMSPV_MAX_BFS_LEVELS_RECORDED) {
            ctr->bfs_level_path[depth - 1] = path;
            ctr->bfs_level_nzblk[depth - 1] = n_nzblk;
            ctr->bfs_stamp[depth] = global_timer_ns();
        }
    }
    int4 *hubs_next = d.ws.hubs + nxt * HUB_CAP;
    if (path != DBSPMSPV_PATH_PUSH && d.rowrun_ptr != nullptr) {
        // a pull over the row-run index does its own bookkeeping (it owns the mask words it writes)
        bfs_pull_rows<DT>(d, F, N, Z, &ctr->bfs_cnt[nxt][0], words_out, &ctr->bfs_nwords[q_out], levels, depth,
                          (float)n_nzblk < BFS_WIDE_PULL * (float)d.nb, s_need + (threadIdx.x >> 5) * 32);
        grid.sync();
    } else if (path == DBSPMSPV_PATH_PUSH) {
        bfs_push<DT>(d, sc, F, N, n_tasks, d.ws.hubs + cur * HUB_CAP, min(ctr->bfs_hubs[cur], HUB_CAP), levels, depth,
                     words_out, &ctr->bfs_nwords[q_out]);
        grid.sync();
        // Z (the frontier before this one) is cleared through its list
        const int nz_words = ctr->bfs_nwords[q_z];
        for (int i = sc.tid; i < nz_words; i += sc.nthreads) Z[words_z[i]] = 0u;
        const int n_listed = ctr->bfs_nwords[q_out];
        // With so few nonzero words that the next level is a push whatever their content, the
        // bookkeeping and the next worklist are one pass (one barrier less); otherwise the
        // bookkeeping first, then -- the selector's input being known -- the worklist if needed.
        const bool surely_push = bfs_path(min(2 * n_listed, d.nb), d.nb, th3, force_path) == DBSPMSPV_PATH_PUSH;
        if (surely_push) {
            bfs_worklist<true>(d, sc, N, words_out, n_listed, &ctr->bfs_cnt[nxt][1], &ctr->bfs_hubs[nxt], hubs_next, &ctr->bfs_cnt[nxt][0]);
            grid.sync();
            return;
        }
        int found = 0, nz = 0;
        for (int i = sc.tid; i < n_listed; i += sc.nthreads) {
            const int k = words_out[i];
            const uint32_t nm = N[k];
            d.ws.visited32[k] |= nm;
            found += __popc(nm);
            nz += ((nm & 0xFFFFu) != 0) + ((nm >> 16) != 0);
        }
        found = __reduce_add_sync(FULL, found);
        nz = __reduce_add_sync(FULL, nz);
        if (lane == 0 && found) { atomicAdd(&ctr->bfs_reached, found); atomicAdd(&ctr->bfs_cnt[nxt][0], nz); }
        grid.sync();
    } else {
        // pull over the row-block segments (no row-run index): the masks produced are scanned as a
        // whole: visited is updated, the nonempty blocks counted, the nonzero words listed
        bfs_pull<DT>(d, sc, F, N, levels, depth);
        grid.sync();
        int found = 0, nz = 0;
        for (int k0 = sc.tid & ~31; k0 < n_words; k0 += sc.nthreads) {
            const int k = k0 + lane;
            uint32_t nm = 0;
            if (k < n_words) {
                nm = N[k];
                if (nm) {
                    d.ws.visited32[k] |= nm;
                    found += __popc(nm);
                    nz += ((nm & 0xFFFFu) != 0) + ((nm >> 16) != 0);
                }
                if (Z[k]) Z[k] = 0u;
            }
            append_words(nm ? k : -1, words_out, &ctr->bfs_nwords[q_out], lane);
        }
        found = __reduce_add_sync(FULL, found);
        nz = __reduce_add_sync(FULL, nz);
        if (lane == 0 && found) { atomicAdd(&ctr->bfs_reached, found); atomicAdd(&ctr->bfs_cnt[nxt][0], nz); }
        grid.sync();
    }
    // the push worklist is rebuilt if the block ratio of the next level asks for a push (the
    // selector's input is known now; the level may still turn to a pull when the list is long)
    const int next_n = ctr->bfs_cnt[nxt][0];
    if (next_n && bfs_path(next_n, d.nb, th3, force_path) == DBSPMSPV_PATH_PUSH) {
        bfs_worklist<false>(d, sc, N, words_out, ctr->bfs_nwords[q_out], &ctr->bfs_cnt[nxt][1], &ctr->bfs_hubs[nxt], hubs_next, nullptr);
        grid.sync();
    }
}

template <int DT>
__global__ void __launch_bounds__(BFS_CTA) k_bfs(Device d, int32_t src, int32_t *levels, float th3, float edge_frac,
                                                 int force_path, int max_levels) {
    __shared__ uint32_t s_need[BFS_CTA];                      // per warp: the wanted rows of its 32 words (transposed pull)
    cg::grid_group grid = cg::this_grid();
    const int tid = blockIdx.x * blockDim.x + threadIdx.x;
    const int nthreads = gridDim.x * blockDim.x;
    const int lane = threadIdx.x & 31;
    const int n_words = (d.mb + 1) / 2;
    Counters *ctr = d.ws.ctr;
    const Scope sc{tid, nthreads, tid >> 5, nthreads >> 5};
    if (tid == 0) ctr->bfs_stamp[0] = global_timer_ns();

    // levels = -1 (16-byte stores over the aligned middle, the ragged ends one by one)
    {
        const uintptr_t addr = reinterpret_cast<uintptr_t>(levels);
        int64_t head = (int64_t)((16 - (addr & 15)) & 15) / 4;
        if (head > d.n) head = d.n;
        const int64_t n4 = (d.n - head) / 4;
        int4 *mid = reinterpret_cast<int4 *>(levels + head);
        for (int64_t v = tid; v < n4; v += nthreads) mid[v] = make_int4(-1, -1, -1, -1);
        for (int64_t v = tid; v < head; v += nthreads) levels[v] = -1;
        for (int64_t v = head + n4 * 4 + tid; v < d.n; v += nthreads) levels[v] = -1;
    }
    // rows without a stored element can never be reached through a pull: they start out as
    // "visited", so that a row block is skipped (and a segment left early) once every row that
    // can be found has been found
    for (int k = tid; k < n_words; k += nthreads) { d.ws.visited32[k] = ~d.row_present32[k]; d.ws.x_mask32[k] = 0u; d.ws.y_mask32[k] = 0u; d.ws.z_mask32[k] = 0u; }
    if (tid == 0) {
        for (int k = 0; k < 3; ++k) { ctr->bfs_cnt[k][0] = 0; ctr->bfs_cnt[k][1] = 0; ctr->bfs_hubs[k] = 0; }
        for (int k = 0; k < 4; ++k) ctr->bfs_nwords[k] = 0;
        ctr->bfs_reached = 1;
    }
    grid.sync();
    // level 0: the source is the first frontier (its mask word is list 3 = "produced by level -1")
    if (blockIdx.x == 0 && threadIdx.x < 32) {
        const int jb = src >> 4;
        if (lane == 0) {
            levels[src] = 0;
            const uint32_t bit = 1u << ((src & 15) + (jb & 1) * 16);
            d.ws.x_mask32[jb >> 1] = bit;
            d.ws.visited32[jb >> 1] |= bit;
            d.ws.bfs_words[(size_t)3 * d.ws.bfs_words_stride] = jb >> 1;
            ctr->bfs_nwords[3] = 1;
        }
        int first = 0, deg = 0;
        if (lane == 0) column_run(d, src, first, deg);
        else if (lane == 1) payload_run(d, jb, first, deg);
        emit_tasks(d, lane == 0, jb, first, deg, lane, &ctr->bfs_cnt[0][1], &ctr->bfs_cnt[0][0], PUSH_CHUNK, &ctr->bfs_hubs[0], d.ws.hubs);
    }
    grid.sync();
    int lv = 0;
    while (lv < max_levels && ctr->bfs_cnt[lv % 3][0] != 0) {
        bfs_level<DT>(d, grid, sc, lv, levels, th3, edge_frac, force_path, s_need);    // ends with a grid barrier
        ++lv;
    }
    // leave the shared workspace as dbspmspv_run expects it: all masks clear.  The frontier before
    // the last one (buffer (lv + 2) % 3) is cleared through its list; the last frontier is empty
    // unless the level cap ended the search; the third buffer is clear.
    {
        uint32_t *const buf[3] = {d.ws.x_mask32, d.ws.y_mask32, d.ws.z_mask32};
        uint32_t *Z = buf[(lv + 2) % 3], *F = buf[lv % 3];
        const int32_t *wz = d.ws.bfs_words + (size_t)((lv + 2) & 3) * d.ws.bfs_words_stride;
        const int nz_words = ctr->bfs_nwords[(lv + 2) & 3];
        for (int i = tid; i < nz_words; i += nthreads) Z[wz[i]] = 0u;
        if (ctr->bfs_cnt[lv % 3][0] != 0)
            for (int k = tid; k < n_words; k += nthreads) F[k] = 0u;
    }
    if (tid == 0) {
        ctr->bfs_levels = lv;
        if (lv < DBSPMSPV_MAX_BFS_LEVELS_RECORDED + 1) ctr->bfs_stamp[lv + 1] = global_timer_ns();
    }
}

template <int DT>
static int bfs_typed(dbspmspv_handle_s *h, int32_t src, int32_t *levels, cudaStream_t st) {
    Device d = h->d;
    if (!h->bfs_grid) {
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_bfs<DT>, BFS_CTA, 0) != cudaSuccess || per_sm < 1) return DBSPMSPV_ERR_CUDA;
        h->bfs_grid = per_sm * h->sm_count;
    }
    float th3 = h->ropts.th3_bfs;
    float edge_frac = h->ropts.bfs_push_max_edge_frac;
    int force = h->ropts.force_path;
    int max_levels = d.n > 0x7FFFFFFF ? 0x7FFFFFFF : (int)d.n;
    void *args[] = {&d, &src, &levels, &th3, &edge_frac, &force, &max_levels};
    DBS_CUDA(cudaLaunchCooperativeKernel((void *)k_bfs<DT>, dim3(h->bfs_grid), dim3(BFS_CTA), args, 0, st));
    ++h->kernel_launches;
    return DBSPMSPV_OK;
}

}  // namespace dbs

extern "C" int db_bfs(dbspmspv_handle_t h, int32_t src, int32_t *levels, dbspmspv_stream_t stream) {
    if (!h || !levels) return DBSPMSPV_ERR_INVALID_ARG;
    if (h->d.m != h->d.n) return DBSPMSPV_ERR_UNSUPPORTED;
    if (src < 0 || src >= h->d.n) return DBSPMSPV_ERR_INVALID_ARG;
    if (!dbs::on_handle_device(h)) return DBSPMSPV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    h->last_stream = st;
    switch (h->d.dtype) {
        case DBSPMSPV_F32: return dbs::bfs_typed<DBSPMSPV_F32>(h, src, levels, st);
        case DBSPMSPV_BF16: return dbs::bfs_typed<DBSPMSPV_BF16>(h, src, levels, st);
        default: return dbs::bfs_typed<DBSPMSPV_PATTERN>(h, src, levels, st);
    }
}
