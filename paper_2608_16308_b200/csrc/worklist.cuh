// Push worklist (Section 3.3.2): the work of the active column blocks is flattened into
// block-level tasks, each a run of at most PUSH_CHUNK consecutive entries of one block-CSC
// column, so that a long column block is spread over many warps.
#pragma once

#include "internal.cuh"

namespace dbs {

// Called by a full warp -- or, with CTA_WIDE, by every thread of the thread block.  Lanes with
// `newly` set own a vector block `jb` that has just become nonempty; each appends that block's
// tasks.  Space is claimed hierarchically (Section 4.1): a warp scan, then either one atomic per
// warp or -- CTA_WIDE -- a sum over the block's warps in shared memory and one atomic per thread
// block (thousands of warps queueing on one counter serialise in L2 otherwise).  The count of
// nonempty vector blocks is aggregated the same way.
template <bool CTA_WIDE = false>
__device__ __forceinline__ void emit_tasks(const Device &d, bool newly, int jb, int lane,
                                           int32_t *n_tasks, int32_t *n_nzblk) {
    int first = 0, deg = 0;
    if (newly) {
        first = d.csc.ptr[jb];
        deg = d.csc.ptr[jb + 1] - first;
    }
    const int nchunks = (deg + PUSH_CHUNK - 1) / PUSH_CHUNK;
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
    } else if (lane == 0 && n_new) {
        if (total) base = atomicAdd(n_tasks, total);
        atomicAdd(n_nzblk, n_new);
    }
    base = __shfl_sync(0xFFFFFFFFu, base, 0) + incl - nchunks;
    // task record: column block in bits 0..26, ceil(entries / 4) - 1 in bits 27..31 (the exact
    // end comes from the column pointer), first position.
    // Short columns are written by their own lane; a long column block (a hub) is written by
    // the whole warp so that one lane does not serialise thousands of stores.
    constexpr int SMALL = 4;
    if (nchunks <= SMALL)
        for (int k = 0; k < nchunks; ++k) {
            const int cnt = min(PUSH_CHUNK, deg - k * PUSH_CHUNK);
            d.ws.tasks[base + k] = make_uint2((uint32_t)jb | ((uint32_t)((cnt + 3) / 4 - 1) << 27), (uint32_t)(first + k * PUSH_CHUNK));
        }
    uint32_t big = __ballot_sync(0xFFFFFFFFu, nchunks > SMALL);
    while (big) {
        const int src = __ffs(big) - 1;
        big &= big - 1;
        const int bjb = __shfl_sync(0xFFFFFFFFu, jb, src);
        const int bfirst = __shfl_sync(0xFFFFFFFFu, first, src);
        const int bdeg = __shfl_sync(0xFFFFFFFFu, deg, src);
        const int bbase = __shfl_sync(0xFFFFFFFFu, base, src);
        const int bn = (bdeg + PUSH_CHUNK - 1) / PUSH_CHUNK;
        for (int k = lane; k < bn; k += 32) {
            const int cnt = min(PUSH_CHUNK, bdeg - k * PUSH_CHUNK);
            d.ws.tasks[bbase + k] = make_uint2((uint32_t)bjb | ((uint32_t)((cnt + 3) / 4 - 1) << 27), (uint32_t)(bfirst + k * PUSH_CHUNK));
        }
    }
}

}  // namespace dbs
