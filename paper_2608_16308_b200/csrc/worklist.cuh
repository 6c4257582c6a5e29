// Push worklist (Section 3.3.2): the work of the active column blocks is flattened into
// block-level tasks, each a run of at most PUSH_CHUNK consecutive entries of one block-CSC
// column, so that a long column block is spread over many warps.
#pragma once

#include "internal.cuh"

namespace dbs {

// Called by a full warp -- or, with CTA_WIDE, by every thread of the thread block.  Every lane
// hands in one run [first, first + deg) of block-CSC positions of column block `jb` (deg = 0:
// nothing) and appends its tasks, `chunk` entries each (at most PUSH_CHUNK); lanes with `newly`
// set own a vector block that has just become nonempty (counted).  Space is claimed hierarchically (Section 4.1): a warp scan, then either
// one atomic per warp or -- CTA_WIDE -- a sum over the block's warps in shared memory and one
// atomic per thread block (thousands of warps queueing on one counter serialise in L2
// otherwise).  The count of nonempty vector blocks is aggregated the same way.
template <bool CTA_WIDE = false>
__device__ __forceinline__ void emit_tasks(const Device &d, bool newly, int jb, int first, int deg, int lane,
                                           int32_t *n_tasks, int32_t *n_nzblk, int chunk = PUSH_CHUNK,
                                           int32_t *n_hubs = nullptr, int4 *hubs = nullptr) {
    // a hub run is listed, not cut up (writing tens of thousands of task records from one warp
    // took longer than the traversal of the level they belonged to)
    if (n_hubs && deg >= HUB_MIN_ENTRIES) {
        const int slot = atomicAdd(n_hubs, 1);
        if (slot < HUB_CAP) { hubs[slot] = make_int4(jb, first, deg, 0); deg = 0; }
    }
    const int nchunks = (deg + chunk - 1) / chunk;
    int incl = nchunks;
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
    }
    const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
    const int n_new = __popc(__ballot_sync(0xFFFFFFFFu, newly));
    int base = 0;
    if (CTA_WIDE) {
        __shared__ int s_tot[32], s_new[32], s_base;
        const int warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
        __syncthreads();                       // (the arrays may still be read by an earlier call)
        if (lane == 0) { s_tot[warp] = total; s_new[warp] = n_new; }
        __syncthreads();
        if (warp == 0) {
            const int t = lane < nw ? s_tot[lane] : 0, c = lane < nw ? s_new[lane] : 0;
            const int tsum = __reduce_add_sync(0xFFFFFFFFu, t), csum = __reduce_add_sync(0xFFFFFFFFu, c);
            if (lane == 0) {
                s_base = tsum ? atomicAdd(n_tasks, tsum) : 0;
                if (csum) atomicAdd(n_nzblk, csum);
            }
        }
        __syncthreads();
        if (lane == 0) {
            base = s_base;
            for (int k = 0; k < warp; ++k) base += s_tot[k];
        }
    } else if (lane == 0) {
        if (total) base = atomicAdd(n_tasks, total);
        if (n_new) atomicAdd(n_nzblk, n_new);
    }
    base = __shfl_sync(0xFFFFFFFFu, base, 0) + incl - nchunks;
    // task record: column block in bits 0..26, entries - 1 in bits 27..31, first position.
    // Short columns are written by their own lane; a long column block (a hub) is written by
    // the whole warp so that one lane does not serialise thousands of stores.
    constexpr int SMALL = 4;
    if (nchunks <= SMALL)
        for (int k = 0; k < nchunks; ++k) {
            const int cnt = min(chunk, deg - k * chunk);
            d.ws.tasks[base + k] = make_uint2((uint32_t)jb | ((uint32_t)(cnt - 1) << 27), (uint32_t)(first + k * chunk));
        }
    uint32_t big = __ballot_sync(0xFFFFFFFFu, nchunks > SMALL);
    while (big) {
        const int src = __ffs(big) - 1;
        big &= big - 1;
        const int bjb = __shfl_sync(0xFFFFFFFFu, jb, src);
        const int bfirst = __shfl_sync(0xFFFFFFFFu, first, src);
        const int bdeg = __shfl_sync(0xFFFFFFFFu, deg, src);
        const int bbase = __shfl_sync(0xFFFFFFFFu, base, src);
        const int bn = (bdeg + chunk - 1) / chunk;
        for (int k = lane; k < bn; k += 32) {
            const int cnt = min(chunk, bdeg - k * chunk);
            d.ws.tasks[bbase + k] = make_uint2((uint32_t)bjb | ((uint32_t)(cnt - 1) << 27), (uint32_t)(bfirst + k * chunk));
        }
    }
}

// The listed hub runs of one worklist, held by a warp in registers: lane h keeps hub h, the
// number of its 32-entry steps and the number of steps of the hubs before it.
struct HubTable {
    int4 hub;        // (column block, first position, entries, -) of hub number `lane`
    int start;       // steps of the hubs before this one
    int steps;       // steps of this one (0: no hub in this lane)
    int total;       // steps of all hubs (warp-uniform)
};
__device__ __forceinline__ HubTable load_hub_table(const int4 *hubs, int n_hubs, int lane) {
    static_assert(HUB_CAP <= 32, "one hub per lane");
    HubTable t;
    t.hub = lane < n_hubs ? hubs[lane] : make_int4(0, 0, 0, 0);
    t.steps = (t.hub.z + PUSH_CHUNK - 1) / PUSH_CHUNK;
    int incl = t.steps;
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
    }
    t.start = incl - t.steps;
    t.total = __shfl_sync(0xFFFFFFFFu, incl, 31);
    return t;
}
// Item i of a push worklist made of n_tasks task records followed by the steps of the hub runs.
// Called by a full warp with a warp-uniform i.
__device__ __forceinline__ uint2 worklist_item(const uint2 *tasks, int n_tasks, const HubTable &t, int i) {
    if (i < n_tasks) return tasks[i];
    const int k = i - n_tasks;
    const uint32_t m = __ballot_sync(0xFFFFFFFFu, k >= t.start && k < t.start + t.steps);
    if (!m) return make_uint2(0u, 0u);
    const int src = __ffs(m) - 1;
    const int jb = __shfl_sync(0xFFFFFFFFu, t.hub.x, src), first = __shfl_sync(0xFFFFFFFFu, t.hub.y, src);
    const int deg = __shfl_sync(0xFFFFFFFFu, t.hub.z, src), kk = k - __shfl_sync(0xFFFFFFFFu, t.start, src);
    const int cnt = min(PUSH_CHUNK, deg - kk * PUSH_CHUNK);
    return make_uint2((uint32_t)jb | ((uint32_t)(cnt - 1) << 27), (uint32_t)(first + kk * PUSH_CHUNK));
}

// The two kinds of run of a column block in the block-CSC view (see View::colptr).
__device__ __forceinline__ void payload_run(const Device &d, int jb, int &first, int &deg) {
    first = d.csc.ptr[jb];
    deg = d.csc.colptr[17 * jb] - first;
    if (!DBS_CHK_RANGE(d, first, deg)) deg = 0;
}
__device__ __forceinline__ void column_run(const Device &d, int j, int &first, int &deg) {
    const int32_t *cp = d.csc.colptr + 17 * (j >> 4) + (j & 15);
    first = cp[0];
    deg = cp[1] - first;
    if (!DBS_CHK_RANGE(d, first, deg)) deg = 0;
}

// Runs of consecutive columns of one column block are adjacent in the view, so lanes that hold
// consecutive columns (a sorted x with clustered nonzeros; a dense x) are merged into one run
// owned by the first lane of the chain; the others are left with deg = 0.  Called by a full
// warp; `has`: the lane holds column j with the run [first, first + deg).
__device__ __forceinline__ void merge_column_runs(bool has, int j, int &first, int &deg, int lane) {
    const int pj = __shfl_up_sync(0xFFFFFFFFu, j, 1);
    const bool phas = __shfl_up_sync(0xFFFFFFFFu, (int)has, 1) != 0;
    const bool cont = lane > 0 && has && phas && j == pj + 1 && (j >> 4) == (pj >> 4);
    const uint32_t contm = __ballot_sync(0xFFFFFFFFu, cont);
    const int end = first + deg;
    const uint32_t after = ~contm & ~((2u << lane) - 1u);    // lanes behind me that do not continue a chain
    const int stop = after ? __ffs(after) - 1 : 32;           // my chain is lanes [lane, stop)
    const int tail_end = __shfl_sync(0xFFFFFFFFu, end, stop - 1);
    if (cont) deg = 0;
    else if (has) deg = tail_end - first;
}

}  // namespace dbs
