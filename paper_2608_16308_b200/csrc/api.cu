// Handle lifetime, statistics and the test hooks that decode the blocked format back to
// coordinates (used to check that create() loses nothing).
#include <cub/cub.cuh>

#include "internal.cuh"

namespace dbs {
namespace {

__device__ __forceinline__ int block_nnz(int dtype, uint32_t idx, uint32_t aux) {
    const int type = idx >> TYPE_SHIFT;
    if (type == DBSPMSPV_BLK_INLINE) return 1;
    return (int)aux + 1;
}

__global__ void k_block_nnz(Device d, int32_t *out) {
    int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (b < d.n_entries) out[b] = block_nnz(d.dtype, d.csr.idx[b], d.csr.aux[b]);
}

template <int DT>
__device__ __forceinline__ void put(int32_t *row, int32_t *col, void *val, int64_t pos, int r, int c,
                                    const uint8_t *vals, int k) {
    row[pos] = r;
    col[pos] = c;
    if (val && DT == DBSPMSPV_F32) static_cast<float *>(val)[pos] = reinterpret_cast<const float *>(vals)[k];
    if (val && DT == DBSPMSPV_BF16) static_cast<uint16_t *>(val)[pos] = reinterpret_cast<const uint16_t *>(vals)[k];
}

// One warp per block: walk the block's encoding and emit (row, col, value) triples.
template <int DT>
__global__ void k_export(Device d, const int32_t *block_row, const int32_t *elem_start, int32_t *row,
                         int32_t *col, void *val) {
    const int lane = threadIdx.x & 31;
    int64_t b = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    if (b >= d.n_entries) return;
    const uint32_t idx = d.csr.idx[b], w = d.csr.w[b], aux = d.csr.aux[b];
    const int type = idx >> TYPE_SHIFT;
    const int r0 = block_row[b] * 16, c0 = (int)(idx & IDX_MASK) * 16;
    const int64_t o = elem_start[b];
    if (type == DBSPMSPV_BLK_INLINE) {
        if (lane == 0) {
            row[o] = r0 + (aux >> 4); col[o] = c0 + (aux & 15);
            if (val && DT == DBSPMSPV_F32) static_cast<uint32_t *>(val)[o] = w;
            if (val && DT == DBSPMSPV_BF16) static_cast<uint16_t *>(val)[o] = (uint16_t)w;
        }
        return;
    }
    const int nnz = (int)aux + 1;
    const uint8_t *blk = d.payload + (size_t)w * 4;
    if (type == DBSPMSPV_BLK_COO) {
        const uint8_t *vals = blk + ((nnz + 3) & ~3);
        for (int k = lane; k < nnz; k += 32) put<DT>(row, col, val, o + k, r0 + (blk[k] >> 4), c0 + (blk[k] & 15), vals, k);
        return;
    }
    const uint16_t *masks = reinterpret_cast<const uint16_t *>(blk);
    const uint32_t mine = lane < 16 ? masks[lane] : 0u;
    int start = __popc(mine);
    for (int s = 1; s < 16; s <<= 1) {
        int t = __shfl_up_sync(0xFFFFFFFFu, start, s);
        if (lane >= s) start += t;
    }
    start -= __popc(mine);
    if (lane >= 16) return;
    const bool row_major = is_row_major(type);
    if (type == DBSPMSPV_BLK_DENSE) {
        const uint8_t *vals = blk + 32;
        int k = 0;
        for (uint32_t mm = mine; mm; mm &= mm - 1, ++k) {
            const int r = __ffs(mm) - 1;
            put<DT>(row, col, val, o + start + k, r0 + r, c0 + lane, vals, lane * 16 + r);
        }
        return;
    }
    const uint8_t *vals = blk + HDR_BYTES;
    const int stored_start = DT == DBSPMSPV_PATTERN ? start : blk[32 + lane];
    int k = 0;
    for (uint32_t mm = mine; mm; mm &= mm - 1, ++k) {
        const int other = __ffs(mm) - 1;
        const int r = row_major ? lane : other, c = row_major ? other : lane;
        put<DT>(row, col, val, o + start + k, r0 + r, c0 + c, vals, stored_start + k);
    }
}

__global__ void k_export_blocks(Device d, const int32_t *brow, int32_t *block_row, int32_t *block_col,
                                int32_t *block_class, int32_t *nnz) {
    int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (b >= d.n_entries) return;
    const uint32_t idx = d.csr.idx[b];
    if (block_row) block_row[b] = brow[b];
    if (block_col) block_col[b] = (int32_t)(idx & IDX_MASK);
    if (block_class) block_class[b] = (int32_t)public_class((int)(idx >> TYPE_SHIFT));
    if (nnz) nnz[b] = block_nnz(d.dtype, idx, d.csr.aux[b]);
}

__global__ void k_export_csc_rows(Device d, int32_t *csc_row) {
    int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (p < d.n_entries) csc_row[p] = (int32_t)(d.csc.idx[p] & IDX_MASK);
}

}  // namespace
}  // namespace dbs

extern "C" {

int dbspmspv_get_stats(dbspmspv_handle_t h, dbspmspv_stats *out) {
    if (!h || !out) return DBSPMSPV_ERR_INVALID_ARG;
    if (!dbs::on_handle_device(h)) return DBSPMSPV_ERR_INVALID_ARG;
    // wait for the handle's own work only: the stream its last call was enqueued on
    DBS_CUDA(cudaStreamSynchronize(h->last_stream));
    dbs::Counters c;
    DBS_CUDA(cudaMemcpy(&c, h->d.ws.ctr, sizeof(c), cudaMemcpyDeviceToHost));
    *out = h->stats;
    out->last_path = c.last_path;
    out->last_n_nzblk = c.last_n_nzblk;
    out->last_n_tasks = c.last_n_tasks;
    out->last_y_nnz = c.last_y_nnz;
    out->bfs_levels = c.bfs_levels;
    out->bfs_reached = c.bfs_reached;
    for (int k = 0; k < DBSPMSPV_MAX_BFS_LEVELS_RECORDED; ++k) {
        out->bfs_level_path[k] = c.bfs_level_path[k];
        out->bfs_level_nzblk[k] = c.bfs_level_nzblk[k];
    }
    {
        const int nl = c.bfs_levels < DBSPMSPV_MAX_BFS_LEVELS_RECORDED ? c.bfs_levels : DBSPMSPV_MAX_BFS_LEVELS_RECORDED;
        out->bfs_setup_us = nl >= 0 ? (float)((double)(c.bfs_stamp[1] - c.bfs_stamp[0]) * 1e-3) : 0.f;
        for (int k = 0; k < DBSPMSPV_MAX_BFS_LEVELS_RECORDED; ++k)
            out->bfs_level_us[k] = k < nl ? (float)((double)(c.bfs_stamp[k + 2] - c.bfs_stamp[k + 1]) * 1e-3) : 0.f;
    }
    out->device_status = c.status;
    out->kernel_launches = h->kernel_launches;
    out->last_compute_ms = -1.0f;
    if (h->timed) {
        float ms = -1.0f;
        if (cudaEventElapsedTime(&ms, h->ev[0], h->ev[1]) == cudaSuccess) out->last_compute_ms = ms;
    }
    if (c.status != DBSPMSPV_OK) {  // report once, then clear
        int32_t zero = 0;
        DBS_CUDA(cudaMemcpy(&h->d.ws.ctr->status, &zero, sizeof(zero), cudaMemcpyHostToDevice));
    }
    return c.status;
}

int dbspmspv_export_coo(dbspmspv_handle_t h, int32_t *row, int32_t *col, void *val) {
    if (!h || !row || !col) return DBSPMSPV_ERR_INVALID_ARG;
    const dbs::Device &d = h->d;
    if (d.n_entries == 0) return DBSPMSPV_OK;
    int32_t *cnt = nullptr, *start = nullptr;
    void *tmp = nullptr;
    size_t bytes = 0;
    int status = DBSPMSPV_OK;
    const int nb = d.n_entries;
    if (cudaMalloc(&cnt, (size_t)nb * 4) != cudaSuccess || cudaMalloc(&start, (size_t)nb * 4) != cudaSuccess) status = DBSPMSPV_ERR_ALLOC;
    if (status == DBSPMSPV_OK) {
        dbs::k_block_nnz<<<(nb + 255) / 256, 256>>>(d, cnt);
        cub::DeviceScan::ExclusiveSum(nullptr, bytes, cnt, start, nb);
        if (cudaMalloc(&tmp, bytes ? bytes : 1) != cudaSuccess) status = DBSPMSPV_ERR_ALLOC;
    }
    if (status == DBSPMSPV_OK) {
        cub::DeviceScan::ExclusiveSum(tmp, bytes, cnt, start, nb);
        const int g = (int)(((int64_t)nb * 32 + 255) / 256);
        if (d.dtype == DBSPMSPV_F32) dbs::k_export<DBSPMSPV_F32><<<g, 256>>>(d, h->block_row, start, row, col, val);
        else if (d.dtype == DBSPMSPV_BF16) dbs::k_export<DBSPMSPV_BF16><<<g, 256>>>(d, h->block_row, start, row, col, val);
        else dbs::k_export<DBSPMSPV_PATTERN><<<g, 256>>>(d, h->block_row, start, row, col, val);
        if (cudaDeviceSynchronize() != cudaSuccess) status = DBSPMSPV_ERR_CUDA;
    }
    cudaFree(cnt); cudaFree(start); cudaFree(tmp);
    return status;
}

int dbspmspv_export_blocks(dbspmspv_handle_t h, int32_t *block_row, int32_t *block_col,
                           int32_t *block_class, int32_t *block_nnz) {
    if (!h) return DBSPMSPV_ERR_INVALID_ARG;
    const dbs::Device &d = h->d;
    if (d.n_entries) dbs::k_export_blocks<<<(d.n_entries + 255) / 256, 256>>>(d, h->block_row, block_row, block_col, block_class, block_nnz);
    DBS_CUDA(cudaDeviceSynchronize());
    return DBSPMSPV_OK;
}

int dbspmspv_export_views(dbspmspv_handle_t h, int32_t *csr_row_ptr, int32_t *csc_col_ptr,
                          int32_t *csc_row, int32_t *csc2csr) {
    if (!h) return DBSPMSPV_ERR_INVALID_ARG;
    const dbs::Device &d = h->d;
    if (csr_row_ptr) DBS_CUDA(cudaMemcpy(csr_row_ptr, d.csr.ptr, ((size_t)d.mb + 1) * 4, cudaMemcpyDeviceToDevice));
    if (csc_col_ptr) DBS_CUDA(cudaMemcpy(csc_col_ptr, d.csc.ptr, ((size_t)d.nb + 1) * 4, cudaMemcpyDeviceToDevice));
    if (csc_row && d.n_entries) dbs::k_export_csc_rows<<<(d.n_entries + 255) / 256, 256>>>(d, csc_row);
    if (csc2csr && d.n_entries) DBS_CUDA(cudaMemcpy(csc2csr, h->csc2csr, (size_t)d.n_entries * 4, cudaMemcpyDeviceToDevice));
    DBS_CUDA(cudaDeviceSynchronize());
    return DBSPMSPV_OK;
}

int dbspmspv_destroy(dbspmspv_handle_t h) {
    if (!h) return DBSPMSPV_ERR_INVALID_ARG;
    dbs::Device &d = h->d;
    cudaDeviceSynchronize();
    cudaFree(d.csr.ptr); cudaFree(d.csr.idx); cudaFree(d.csr.w); cudaFree(d.csr.aux);
    cudaFree(d.csc.ptr); cudaFree(d.csc.idx); cudaFree(d.csc.w); cudaFree(d.csc.aux); cudaFree(d.csc.colptr);
    cudaFree(h->payload_alloc);
    cudaFree(const_cast<dbs::Segment *>(d.segments));
    cudaFree(const_cast<int2 *>(d.chunks));
    cudaFree(const_cast<int32_t *>(d.seg_rb));
    cudaFree(const_cast<uint32_t *>(d.row_present32));
    cudaFree(const_cast<int32_t *>(d.rowrun_ptr)); cudaFree(const_cast<uint32_t *>(d.rowrun_idx));
    cudaFree(const_cast<int32_t *>(d.csr_inl)); cudaFree(const_cast<int32_t *>(d.payload_pos));
    cudaFree(const_cast<int32_t *>(d.lean_rows)); cudaFree(const_cast<int32_t *>(d.lean_chunk_ord));
    cudaFree(const_cast<int4 *>(d.stage_chunks));
    if (h->x_nnz_seen_host) cudaFreeHost(h->x_nnz_seen_host);
    cudaFree(const_cast<uint16_t *>(d.hub_slot)); cudaFree(const_cast<int32_t *>(d.hub_rb)); cudaFree(d.hub_acc);
    cudaFree(h->csc2csr); cudaFree(h->block_row);
    cudaFree(h->ws_arena);
    cudaFree(h->sssp_arena);
    if (h->sssp_host) cudaFreeHost(h->sssp_host);
    if (h->ev[0]) cudaEventDestroy(h->ev[0]);
    if (h->ev[1]) cudaEventDestroy(h->ev[1]);
    delete h;
    return DBSPMSPV_OK;
}

const char *dbspmspv_strerror(int status) {
    switch (status) {
        case DBSPMSPV_OK: return "ok";
        case DBSPMSPV_ERR_INVALID_ARG: return "invalid argument";
        case DBSPMSPV_ERR_UNSUPPORTED: return "unsupported configuration";
        case DBSPMSPV_ERR_ALLOC: return "allocation failed";
        case DBSPMSPV_ERR_CUDA: return "CUDA runtime error";
        case DBSPMSPV_ERR_CAPACITY: return "output capacity too small";
        case DBSPMSPV_ERR_TIMEOUT: return "bounded device wait ran out";
        case DBSPMSPV_ERR_BOUNDS: return "x index out of range";
        case DBSPMSPV_ERR_TOO_LARGE: return "more rows than the fixed scratch of the no-allocation entry point covers";
        case DBSPMSPV_ERR_INTERNAL: return "a range check failed inside a kernel (range-checked build)";
        default: return "unknown status";
    }
}

}  // extern "C"
