// dbspmspv_run for a short x on a hypersparse handle, as ONE kernel of ONE thread-block cluster
// (Section 4.1: vector-metadata construction fused with the SpMSpV kernel, no extra launch, no
// host round trip).  The chain of the general path -- blocking, traversal, two compaction
// passes -- costs four dependent launches, each with its own cold first loads, whatever x
// holds; for up to a few hundred listed columns that chain IS the call (18 - 26 us for 10 .. 100
// nonzeros on a matrix with a million rows; 14 - 22 us here).  Here nothing of x is staged at all:
//   * a warp takes one listed column j (consecutive columns in different thread blocks): its
//     value stays in a register, its run of INLINE
//     elements comes from the column pointers of the block-CSC view, the column block's few
//     entries with a payload are walked with the one-column mask 1 << (j mod 16); four entries
//     are fetched per lane before the first is used; hub columns are listed and walked by the
//     whole cluster;
//   * a product goes to the handle's dense accumulator with a reply-free atomic, and sets the
//     row's bit in a bitmap of ALL rows that the cluster's thread blocks hold together in their
//     shared memories (4 bytes per 32 rows, an eighth of the rows per thread block; remote bits
//     are set through distributed shared memory) -- the structural-hit record, exact whatever
//     the sums are;
//   * after one cluster barrier the bitmap is the compaction's input: every thread block counts
//     its slice, the eight totals are exchanged through distributed shared memory, the set bits
//     become the result's row list (parked in the unused task array), and all threads of the
//     cluster take result positions in turn: gather the sum, clear it, write y.
// The dense copy of x, the vector-block masks, the row flags and the worklist are never
// written, so there is nothing to clean up.  Used when x is short, the selector is certain to
// say push, the bitmap fits, and no option asks for the general path; results are identical
// to the general path's up to the order of the fp32 additions.  The cluster barriers are the
// hardware's (all thread blocks of a cluster are co-resident by construction): no spin-waits.
#pragma once

#include <cooperative_groups.h>
#ifdef DBS_SMALL_STAMPS
#include <cstdio>
#endif

#include "internal.cuh"
#include "minplus.cuh"
#include "worklist.cuh"

namespace dbs {

constexpr int SMALL_CTA = 1024;
constexpr int SMALL_CLUSTER = 8;               // thread blocks of the cluster (the portable maximum)
constexpr int SMALL_MAX_NNZ_X = 256;           // one warp per listed column
constexpr int SMALL_HUB_RUN = 512;             // a run from this length on is walked by the whole cluster
constexpr int SMALL_HUB_CAP = 128;
constexpr int SMALL_ILP = 4;                   // view entries a thread fetches before it works on them
constexpr size_t SMALL_MAX_SMEM = 40 * 1024;   // bitmap slices of one thread block (dynamic shared memory)

struct SmallShared {
    int wsum[SMALL_CTA / 32];
    int total[SMALL_CLUSTER];      // result entries of every thread block's slice (each block holds a full copy)
    int nzblk;                     // (thread block 0) nonempty vector blocks
    int n_hubs;                    // (thread block 0) listed hub runs
    int4 hubs[SMALL_HUB_CAP];      // (thread block 0) first position, entries, x value bits, local column | payload flag << 8
};

// mode: 0 = (+, *), 1 = Boolean, 2 = (min, +)
template <int DT>
__global__ void __cluster_dims__(SMALL_CLUSTER, 1, 1) __launch_bounds__(SMALL_CTA, 1)
k_run_small(Device d, const int32_t *__restrict__ x_idx, const void *__restrict__ x_val, int32_t nnz_x, int mode,
            int32_t *__restrict__ y_idx, float *__restrict__ y_val, int64_t y_capacity, int32_t *__restrict__ y_nnz,
            const uint32_t *__restrict__ row_mask, int complement) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ __align__(16) uint32_t s_small[];
    __shared__ SmallShared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rank = (int)cluster.block_rank();
#ifdef DBS_SMALL_STAMPS
    unsigned long long ts[8]; int nts = 0;
#define STAMP() do { ts[nts++] = global_timer_ns(); } while (0)
#else
#define STAMP() do { } while (0)
#endif
    STAMP();
    const int ywords = (d.mb + 1) / 2, cbwords = (d.nb + 31) / 32;
    const int yper = (ywords + SMALL_CLUSTER - 1) / SMALL_CLUSTER, cper = (cbwords + SMALL_CLUSTER - 1) / SMALL_CLUSTER;
    // this block's slices: row words [rank * yper, ...), vector-block words [rank * cper, ...)
    for (int k = tid; k < yper + cper; k += SMALL_CTA) s_small[k] = 0u;
    if (tid == 0) { sh.nzblk = 0; sh.n_hubs = 0; }
    cluster.sync();
    STAMP();
    SmallShared *sh0 = cluster.map_shared_rank(&sh, 0);
    uint32_t *keys = reinterpret_cast<uint32_t *>(d.ws.y_acc);
    auto add = [&](int row, float a, float xv) {
        if (mode == 2) atomicMax(keys + row, minplus_key(a + xv));
        else if (mode == 0 && DT != DBSPMSPV_PATTERN) atomicAdd(d.ws.y_acc + row, a * xv);
        const int wi = row >> 5, owner = wi / yper;
        atomicOr(cluster.map_shared_rank(s_small, owner) + (wi - owner * yper), 1u << (row & 31));
    };
    // INLINE entries p, p + step, ... below `end`: SMALL_ILP of them are fetched before the first is used
    // (a run is a chain of cold loads otherwise: the address of an entry's atomic depends on the entry)
    auto inline_run = [&](int p, int end, int step, float xv) {
        for (; p < end; p += SMALL_ILP * step) {
            uint32_t ix[SMALL_ILP], wv[SMALL_ILP], ax[SMALL_ILP];
#pragma unroll
            for (int u = 0; u < SMALL_ILP; ++u) {
                const int q = p + u * step;
                ix[u] = 0xFFFFFFFFu; wv[u] = 0u; ax[u] = 0u;
                if (q < end) { ix[u] = d.csc.idx[q]; wv[u] = d.csc.w[q]; ax[u] = d.csc.aux[q]; }
            }
#pragma unroll
            for (int u = 0; u < SMALL_ILP; ++u) {
                if (ix[u] == 0xFFFFFFFFu || !DBS_CHK_INDEX(d, ix[u] & IDX_MASK, d.mb)) continue;
                add((int)(ix[u] & IDX_MASK) * 16 + (int)(ax[u] >> 4), Val<DT>::inline_value(wv[u]), xv);
            }
        }
    };
    auto payload_entry = [&](int p, int c, float xv) {
        uint32_t idx = d.csc.idx[p], w = d.csc.w[p], aux = d.csc.aux[p];
        DBS_CHK_ENTRY(d, false, idx, w, aux);
        const int row0 = (int)(idx & IDX_MASK) * 16;
        block_elements<DT>((int)(idx >> TYPE_SHIFT), w, aux, 1u << c, d.payload, [&](int r, int, float a) { add(row0 + r, a, xv); });
    };
    // a run that the whole cluster should share: listed in thread block 0 (true), or left to the warp
    auto list_hub = [&](int first, int deg, float xv, int tag) {
        const int slot = atomicAdd(&sh0->n_hubs, 1);
        if (slot >= SMALL_HUB_CAP) return false;
        sh0->hubs[slot] = make_int4(first, deg, __float_as_int(xv), tag);
        return true;
    };
    // ---- traversal: a warp per listed column (256 warps in the cluster); consecutive columns go
    // to different thread blocks.  (Several columns per warp were measured too: from about a
    // thousand columns on, the tails of the longer runs make the slowest warp take longer than
    // the general path's whole chain of kernels, whose worklist spreads them over the GPU.)
    constexpr int G = 32;
    static_assert(SMALL_MAX_NNZ_X * G <= SMALL_CLUSTER * SMALL_CTA, "every listed column has its own group of lanes");
    {
        const int gl = tid & (G - 1);
        const int k = (tid / G) * SMALL_CLUSTER + rank;
        bool have = k < nnz_x;
        int j = have ? x_idx[k] : 0;
        if (have && (j < 0 || j >= d.n)) { if (gl == 0) d.ws.ctr->status = DBSPMSPV_ERR_BOUNDS; have = false; }
        if (have) {
            float xv = 1.0f;
            if (mode != 1 && x_val) {
                if (DT == DBSPMSPV_BF16) xv = __bfloat162float(static_cast<const __nv_bfloat16 *>(x_val)[k]);
                else xv = static_cast<const float *>(x_val)[k];
            }
            int first, deg, pfirst, pdeg;
            column_run(d, j, first, deg);
            payload_run(d, j >> 4, pfirst, pdeg);
            if (gl == 0) {
                const int cw = j >> 9, owner = cw / cper;
                const uint32_t bit = 1u << ((j >> 4) & 31);
                if (!(atomicOr(cluster.map_shared_rank(s_small, owner) + yper + (cw - owner * cper), bit) & bit)) atomicAdd(&sh0->nzblk, 1);
            }
            // a hub run is listed for the whole cluster (by the group's first lane; the others skip it)
            if (deg >= SMALL_HUB_RUN) { if (gl == 0 && !list_hub(first, deg, xv, 0)) inline_run(first, first + deg, 1, xv); deg = 0; }
            if (pdeg >= SMALL_HUB_RUN) {
                if (gl == 0 && !list_hub(pfirst, pdeg, xv, (j & 15) | 256)) for (int p = pfirst; p < pfirst + pdeg; ++p) payload_entry(p, j & 15, xv);
                pdeg = 0;
            }
            inline_run(first + gl, first + deg, G, xv);
            for (int p = pfirst + gl; p < pfirst + pdeg; p += G) payload_entry(p, j & 15, xv);
        }
    }
    STAMP();
    cluster.sync();
    STAMP();
    // hub runs: every thread of the cluster strides over them
    {
        const int n_hubs = min(sh0->n_hubs, SMALL_HUB_CAP);
        const int gt = rank * SMALL_CTA + tid;
        for (int q = 0; q < n_hubs; ++q) {
            const int4 hb = sh0->hubs[q];
            const float xs = __int_as_float(hb.z);
            if (hb.w & 256) for (int p = hb.x + gt; p < hb.x + hb.y; p += SMALL_CLUSTER * SMALL_CTA) payload_entry(p, hb.w & 15, xs);
            else inline_run(hb.x + gt, hb.x + hb.y, SMALL_CLUSTER * SMALL_CTA, xs);
        }
        if (n_hubs) cluster.sync();          // (cluster-uniform: every block read the same count)
    }
    STAMP();
    // ---- compaction from the bitmap.  This block's slice; thread t owns the words [t * per, (t + 1) * per).
    const int my_words = max(0, min(yper, ywords - rank * yper));
    const int per = (yper + SMALL_CTA - 1) / SMALL_CTA;
    const int w0 = min(tid * per, my_words), w1 = min(w0 + per, my_words);
    const int wbase = rank * yper;
    auto keep_of = [&](int wi) { return row_mask ? (complement ? ~row_mask[wi] : row_mask[wi]) : 0xFFFFFFFFu; };
    int cnt = 0;
    for (int wi = w0; wi < w1; ++wi) {
        const uint32_t word = s_small[wi];
        if (word) cnt += __popc(word & keep_of(wbase + wi));
    }
    int incl = cnt;
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) sh.wsum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int v = sh.wsum[lane], s = v;
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, s, o);
            if (lane >= o) s += t;
        }
        sh.wsum[lane] = s - v;
        // this block's total goes into every block's table
        if (lane == 31)
            for (int r = 0; r < SMALL_CLUSTER; ++r) cluster.map_shared_rank(&sh, r)->total[rank] = s;
    }
    cluster.sync();
    int before = 0, total = 0;
#pragma unroll
    for (int r = 0; r < SMALL_CLUSTER; ++r) { if (r < rank) before += sh.total[r]; total += sh.total[r]; }
    int pos = before + sh.wsum[warp] + incl - cnt;
    const int64_t room = y_capacity < (int64_t)total ? y_capacity : (int64_t)total;
    // the result's rows, in order, parked in the (unused) task array; rows that do not go to y
    // (masked out, or beyond the capacity) are cleared here
    int32_t *rows = reinterpret_cast<int32_t *>(d.ws.tasks);
    for (int wi = w0; wi < w1; ++wi) {
        const uint32_t word = s_small[wi];
        if (!word) continue;
        const uint32_t keep = keep_of(wbase + wi);
        for (uint32_t bb = word; bb; bb &= bb - 1) {
            const int bit = __ffs(bb) - 1, row = (wbase + wi) * 32 + bit;
            if (((keep >> bit) & 1u) && pos < room) rows[pos++] = row;
            else { if ((keep >> bit) & 1u) ++pos; d.ws.y_acc[row] = 0.f; }
        }
    }
    cluster.sync();          // (release / acquire at cluster scope: the row list is visible to every block)
    STAMP();
    // every thread of the cluster takes result positions in turn: the gathers of a round are independent
    for (int64_t p0 = rank * SMALL_CTA + tid; p0 < room; p0 += (int64_t)SMALL_ILP * SMALL_CLUSTER * SMALL_CTA) {
        int r[SMALL_ILP];
        float v[SMALL_ILP];
#pragma unroll
        for (int u = 0; u < SMALL_ILP; ++u) {
            const int64_t q = p0 + (int64_t)u * SMALL_CLUSTER * SMALL_CTA;
            r[u] = q < room ? __ldcg(rows + q) : -1;
        }
#pragma unroll
        for (int u = 0; u < SMALL_ILP; ++u) v[u] = r[u] >= 0 ? __ldcg(d.ws.y_acc + r[u]) : 0.f;      // (the sums were made by atomics in L2)
#pragma unroll
        for (int u = 0; u < SMALL_ILP; ++u) {
            if (r[u] < 0) continue;
            const int64_t q = p0 + (int64_t)u * SMALL_CLUSTER * SMALL_CTA;
            d.ws.y_acc[r[u]] = 0.f;
            y_idx[q] = r[u];
            if (y_val) y_val[q] = mode == 1 || (mode == 0 && DT == DBSPMSPV_PATTERN) ? 1.0f : mode == 2 ? minplus_value(__float_as_uint(v[u])) : v[u];
        }
    }
    if (rank == 0 && tid == 0) {
        Counters *c = d.ws.ctr;
        *y_nnz = total;
        if ((int64_t)total > y_capacity) c->status = DBSPMSPV_ERR_CAPACITY;
        c->last_y_nnz = total;
        c->last_n_nzblk = sh.nzblk;
        c->last_n_tasks = 0;
        c->last_path = DBSPMSPV_PATH_PUSH;
        c->path = DBSPMSPV_PATH_PUSH;
    }
    STAMP();
    cluster.sync();          // (no block may leave while another still reads its shared memory)
    STAMP();
#ifdef DBS_SMALL_STAMPS
    if (tid == 0 && (rank == 0 || rank == 7)) printf("rank %d: init %llu trav %llu sync %llu hubs %llu count+list %llu emit %llu endsync %llu (hubs %d)\n", rank, ts[1]-ts[0], ts[2]-ts[1], ts[3]-ts[2], ts[4]-ts[3], ts[5]-ts[4], ts[6]-ts[5], ts[7]-ts[6], sh0->n_hubs);
#endif
#undef STAMP
}

}  // namespace dbs
