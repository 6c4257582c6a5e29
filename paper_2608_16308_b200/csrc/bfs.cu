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

constexpr int BFS_CTA = 128;

// Rows of one hypersparse block reached from the active columns (one lane per block).
template <int DT>
__device__ __forceinline__ uint32_t lane_block_bool(int type, uint32_t w, uint32_t aux, uint32_t xm,
                                                    const uint8_t *payload) {
    uint32_t hit = 0;
    if (type == DBSPMSPV_BLK_INLINE) {
        if (DT == DBSPMSPV_PATTERN) {
#pragma unroll
            for (uint32_t k = 0; k < 4; ++k) {      // up to four packed coordinates, no branch
                const uint32_t rc = (w >> (8 * k)) & 0xFFu;
                hit |= (k <= aux ? (xm >> (rc & 15)) & 1u : 0u) << (rc >> 4);
            }
        } else if ((xm >> (aux & 15)) & 1u) {
            hit = 1u << (aux >> 4);
        }
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

// Boolean push: tasks of the active frontier blocks; newly reached rows are claimed with one
// atomicOr per block on the next-frontier masks (the winner writes the level).
template <int DT>
__device__ void bfs_push(const Device &d, int n_tasks, int32_t *levels, int depth) {
    const int lane = threadIdx.x & 31;
    const int gwarp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    for (int t = gwarp; t < n_tasks; t += nwarps) {
        const uint2 task = d.ws.tasks[t];
        const int jb = (int)(task.x & IDX_MASK);
        const int start = (int)task.y;
        const int end = min(start + PUSH_CHUNK, d.csc.ptr[jb + 1]);
        const uint32_t xm = mask_of(d.ws.x_mask32, jb);
        for (int base = start; base < end; base += 32) {
            const int p = base + lane;
            bool heavy = false;
            uint32_t idx = 0, w = 0, aux = 0;
            if (p < end) {
                idx = d.csc.idx[p];
                const int type = idx >> TYPE_SHIFT, brow = idx & IDX_MASK;
                const uint32_t need = ~mask_of(d.ws.visited32, brow) & 0xFFFFu;
                if (need) {
                    w = d.csc.w[p]; aux = d.csc.aux[p];
                    if (type != DBSPMSPV_BLK_COO || aux < COO_SERIAL_MAX) {
                        // one lane per block: hypersparse blocks from their coordinates,
                        // mask-based blocks from their 16 masks
                        const uint32_t hit = need & (type <= DBSPMSPV_BLK_COO ? lane_block_bool<DT>(type, w, aux, xm, d.payload)
                                                                             : lane_heavy_bool(type, d.payload + (size_t)w * 4, xm));
                        if (hit) {
                            const int sh = (brow & 1) * 16;
                            const uint32_t old = atomicOr(&d.ws.y_mask32[brow >> 1], hit << sh);
                            write_levels(levels, brow, hit & ~(old >> sh), depth);
                        }
                    } else {
                        heavy = true;
                    }
                }
            }
            uint32_t hv = __ballot_sync(FULL, heavy);
            while (hv) {
                const int src = __ffs(hv) - 1;
                hv &= hv - 1;
                const uint32_t bidx = __shfl_sync(FULL, idx, src);
                const uint32_t bw = __shfl_sync(FULL, w, src);
                const int nnz = (int)__shfl_sync(FULL, aux, src) + 1;
                const int type = bidx >> TYPE_SHIFT, brow = bidx & IDX_MASK;
                uint32_t hits = warp_block_bool<DT>(type, d.payload + (size_t)bw * 4, nnz, xm, lane);
                hits &= ~mask_of(d.ws.visited32, brow);
                if (lane == 0 && hits) {
                    const int sh = (brow & 1) * 16;
                    const uint32_t old = atomicOr(&d.ws.y_mask32[brow >> 1], hits << sh);
                    write_levels(levels, brow, hits & ~(old >> sh), depth);
                }
            }
        }
    }
}

// Boolean pull: one warp per row-block segment; row blocks with nothing left to discover are
// skipped, and a segment stops as soon as all its unvisited rows are found (the early exit of
// Algorithm 5 lifted to the row block).
template <int DT>
__device__ void bfs_pull(const Device &d, int32_t *levels, int depth) {
    const int lane = threadIdx.x & 31;
    const int gwarp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    // the descriptor and the visited mask of the warp's next segment are fetched while the
    // current one is processed (two of the four dependent loads per segment leave the chain)
    Segment seg_n = Segment{0, 0, 0, 0};
    uint32_t need_n = 0;
    if (gwarp < d.n_segments) {
        seg_n = d.segments[gwarp];
        need_n = ~mask_of(d.ws.visited32, seg_n.row_block) & 0xFFFFu;
    }
    for (int sg = gwarp; sg < d.n_segments; sg += nwarps) {
        const Segment seg = seg_n;
        const uint32_t need = need_n;
        if (sg + nwarps < d.n_segments) {
            seg_n = d.segments[sg + nwarps];
            need_n = ~mask_of(d.ws.visited32, seg_n.row_block) & 0xFFFFu;
        }
        const int rb = seg.row_block;
        if (!need) continue;
        const bool whole = seg.count < 0;
        const int end = seg.start + (seg.count & 0x7FFFFFFF);
        uint32_t hit = 0;
        // up to four warp steps of view entries are fetched at once, then their frontier masks,
        // so that every lane keeps several independent loads in flight
        constexpr int U = 4;
        bool done = false;
        for (int base = seg.start; base < end && !done; base += 32 * U) {
            uint32_t idx[U], w[U], aux[U], xm[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int p = base + u * 32 + lane;
                idx[u] = 0; w[u] = 0; aux[u] = 0;
                if (p < end) { idx[u] = d.csr.idx[p]; w[u] = d.csr.w[p]; aux[u] = d.csr.aux[p]; }
            }
#pragma unroll
            for (int u = 0; u < U; ++u)
                xm[u] = base + u * 32 + lane < end ? mask_of(d.ws.x_mask32, idx[u] & IDX_MASK) : 0u;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (base + u * 32 >= end) break;
                bool heavy = false;
                if (xm[u]) {
                    const int type = idx[u] >> TYPE_SHIFT;
                    if (type <= DBSPMSPV_BLK_COO) {
                        if (type == DBSPMSPV_BLK_INLINE || aux[u] < COO_SERIAL_MAX) hit |= lane_block_bool<DT>(type, w[u], aux[u], xm[u], d.payload);
                        else heavy = true;
                    } else {
                        hit |= lane_heavy_bool(type, d.payload + (size_t)w[u] * 4, xm[u]);
                    }
                }
                uint32_t hv = __ballot_sync(FULL, heavy);
                while (hv) {
                    const int src = __ffs(hv) - 1;
                    hv &= hv - 1;
                    const uint32_t bidx = __shfl_sync(FULL, idx[u], src);
                    const uint32_t bw = __shfl_sync(FULL, w[u], src);
                    const int nnz = (int)__shfl_sync(FULL, aux[u], src) + 1;
                    const uint32_t bxm = __shfl_sync(FULL, xm[u], src);
                    hit |= warp_block_bool<DT>(bidx >> TYPE_SHIFT, d.payload + (size_t)bw * 4, nnz, bxm, lane);
                }
                hit = __reduce_or_sync(FULL, hit);
                if ((hit & need) == need) { done = true; break; }
            }
        }
        hit &= need;
        if (hit) {
            if (whole) {
                if (lane == 0) reinterpret_cast<uint16_t *>(d.ws.y_mask32)[rb] = (uint16_t)hit;
                if (lane < 16 && ((hit >> lane) & 1u)) levels[rb * 16 + lane] = depth;
            } else if (lane == 0) {
                const int sh = (rb & 1) * 16;
                const uint32_t old = atomicOr(&d.ws.y_mask32[rb >> 1], hit << sh);
                write_levels(levels, rb, hit & ~(old >> sh), depth);
            }
        }
    }
}

// Per-level selector (Section 3.3.1): push iff N_nzblk / N_blk < th3.  Monotone in n_nzblk.
__device__ __forceinline__ int bfs_path(int n_nzblk, int nb, float th3, int force_path) {
    if (force_path == DBSPMSPV_PATH_PUSH || force_path == DBSPMSPV_PATH_PULL) return force_path;
    return ((float)n_nzblk / (float)nb < th3) ? DBSPMSPV_PATH_PUSH : DBSPMSPV_PATH_PULL;
}

template <int DT>
__global__ void __launch_bounds__(BFS_CTA) k_bfs(Device d, int32_t src, int32_t *levels, float th3,
                                                 int force_path, int max_levels) {
    cg::grid_group grid = cg::this_grid();
    const int tid = blockIdx.x * blockDim.x + threadIdx.x;
    const int nthreads = gridDim.x * blockDim.x;
    const int lane = threadIdx.x & 31;
    const int n_words = (d.mb + 1) / 2;
    Counters *ctr = d.ws.ctr;

    for (int64_t v = tid; v < d.n; v += nthreads) levels[v] = -1;
    // rows without a stored element can never be reached through a pull: they start out as
    // "visited", so that a row block is skipped (and a segment left early) once every row that
    // can be found has been found
    for (int k = tid; k < n_words; k += nthreads) { d.ws.visited32[k] = ~d.row_present32[k]; d.ws.x_mask32[k] = 0u; d.ws.y_mask32[k] = 0u; }
    if (tid == 0) { ctr->bfs_cnt[0][0] = 0; ctr->bfs_cnt[0][1] = 0; ctr->bfs_cnt[1][0] = 0; ctr->bfs_cnt[1][1] = 0; ctr->bfs_reached = 1; }
    grid.sync();
    // level 0: the source is the first frontier
    if (blockIdx.x == 0 && threadIdx.x < 32) {
        const int jb = src >> 4;
        if (lane == 0) {
            levels[src] = 0;
            const uint32_t bit = 1u << ((src & 15) + (jb & 1) * 16);
            d.ws.x_mask32[jb >> 1] = bit;
            d.ws.visited32[jb >> 1] |= bit;
        }
        emit_tasks(d, lane == 0, jb, lane, &ctr->bfs_cnt[0][1], &ctr->bfs_cnt[0][0]);
    }
    grid.sync();

    int cur = 0, depth = 0;
    while (depth < max_levels) {
        const int n_nzblk = ctr->bfs_cnt[cur][0];
        const int n_tasks = ctr->bfs_cnt[cur][1];
        if (n_nzblk == 0) break;
        ++depth;
        const int path = bfs_path(n_nzblk, d.nb, th3, force_path);
        if (tid == 0) {
            ctr->bfs_cnt[cur ^ 1][0] = 0;
            ctr->bfs_cnt[cur ^ 1][1] = 0;
            if (depth <= DBSPMSPV_MAX_BFS_LEVELS_RECORDED) {
                ctr->bfs_level_path[depth - 1] = path;
                ctr->bfs_level_nzblk[depth - 1] = n_nzblk;
            }
        }
        if (path == DBSPMSPV_PATH_PUSH) bfs_push<DT>(d, n_tasks, levels, depth);
        else bfs_pull<DT>(d, levels, depth);
        grid.sync();
        // next frontier: masks produced above become the vector-block masks of the next level;
        // visited is updated; the push worklist and block statistics are rebuilt on the fly.
        // The worklist is only needed if the next level is a push: the running count of nonempty
        // blocks only grows, so once it has reached the selector's threshold the next level is
        // known to be a pull and the remaining warps just count (a push is only ever chosen
        // when no warp has skipped).
        int found = 0;
        for (int k0 = (tid & ~31); k0 < n_words; k0 += nthreads) {
            const int k = k0 + lane;
            uint32_t nm = 0;
            if (k < n_words) {
                nm = d.ws.y_mask32[k];
                if (nm) {
                    d.ws.y_mask32[k] = 0u;
                    d.ws.visited32[k] |= nm;
                    found += __popc(nm);
                }
                if (nm || d.ws.x_mask32[k]) d.ws.x_mask32[k] = nm;
            }
            const bool lo = (nm & 0xFFFFu) != 0, hi = (nm >> 16) != 0;
            int seen = 0;     // read by one lane: the branch below must be warp-uniform
            if (lane == 0) seen = *reinterpret_cast<volatile int32_t *>(&ctr->bfs_cnt[cur ^ 1][0]);
            seen = __shfl_sync(FULL, seen, 0);
            if (bfs_path(seen, d.nb, th3, force_path) == DBSPMSPV_PATH_PULL) {
                const int nz = __popc(__ballot_sync(FULL, lo)) + __popc(__ballot_sync(FULL, hi));
                if (lane == 0 && nz) atomicAdd(&ctr->bfs_cnt[cur ^ 1][0], nz);
            } else {
                emit_tasks(d, lo, 2 * k, lane, &ctr->bfs_cnt[cur ^ 1][1], &ctr->bfs_cnt[cur ^ 1][0]);
                emit_tasks(d, hi, 2 * k + 1, lane, &ctr->bfs_cnt[cur ^ 1][1], &ctr->bfs_cnt[cur ^ 1][0]);
            }
        }
        found = __reduce_add_sync(FULL, found);
        if (lane == 0 && found) atomicAdd(&ctr->bfs_reached, found);
        grid.sync();
        cur ^= 1;
    }
    // leave the shared workspace as dbspmspv_run expects it: all masks clear
    if (ctr->bfs_cnt[cur][0] != 0)
        for (int k = tid; k < n_words; k += nthreads) d.ws.x_mask32[k] = 0u;
    if (tid == 0) ctr->bfs_levels = depth;
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
    int force = h->ropts.force_path;
    int max_levels = d.n > 0x7FFFFFFF ? 0x7FFFFFFF : (int)d.n;
    void *args[] = {&d, &src, &levels, &th3, &force, &max_levels};
    DBS_CUDA(cudaLaunchCooperativeKernel((void *)k_bfs<DT>, dim3(h->bfs_grid), dim3(BFS_CTA), args, 0, st));
    ++h->kernel_launches;
    return DBSPMSPV_OK;
}

}  // namespace dbs

extern "C" int db_bfs(dbspmspv_handle_t h, int32_t src, int32_t *levels, dbspmspv_stream_t stream) {
    if (!h || !levels) return DBSPMSPV_ERR_INVALID_ARG;
    if (h->d.m != h->d.n) return DBSPMSPV_ERR_UNSUPPORTED;
    if (src < 0 || src >= h->d.n) return DBSPMSPV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    switch (h->d.dtype) {
        case DBSPMSPV_F32: return dbs::bfs_typed<DBSPMSPV_F32>(h, src, levels, st);
        case DBSPMSPV_BF16: return dbs::bfs_typed<DBSPMSPV_BF16>(h, src, levels, st);
        default: return dbs::bfs_typed<DBSPMSPV_PATTERN>(h, src, levels, st);
    }
}
