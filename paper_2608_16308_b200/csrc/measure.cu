// Measurement aids (untimed): a counting pass that walks the format exactly as a traversal of the
// given path would and reports the bytes it reads, and two latency probes (an empty kernel and a
// chain of dependent loads).  None of this is on the timed path; the benchmark uses it to check
// its host-side byte model against the format as built and to put the latency-bound calls next
// to the floor of the machine.
#include "internal.cuh"

namespace dbs {
namespace {

struct CountAcc {            // device-side totals (unsigned long long for atomicAdd)
    unsigned long long view_entries, payload_blocks, payload_bytes, pointer_bytes, active_blocks;
};

__device__ __forceinline__ int vsize_of(int dtype) { return dtype == DBSPMSPV_F32 ? 4 : dtype == DBSPMSPV_BF16 ? 2 : 0; }

// payload entries [first, first + n) of a view: their count and payload bytes
__device__ __forceinline__ void count_payload(const Device &d, const View &v, int first, int n, unsigned long long &blocks,
                                              unsigned long long &bytes) {
    const int vs = vsize_of(d.dtype);
    for (int p = first; p < first + n; ++p) {
        const int type = v.idx[p] >> TYPE_SHIFT;
        if (type == DBSPMSPV_BLK_INLINE) continue;
        ++blocks;
        bytes += 4ull * (unsigned long long)payload_words(type, (int)v.aux[p] + 1, vs);
    }
}

// Push: one thread per listed x index marks its vector block (the masks of the workspace, as the
// blocking kernel does) and counts what a push reads for it.
__global__ void k_count_push(Device d, const int32_t *x_idx, int32_t nnz_x, CountAcc *acc) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= nnz_x) return;
    const int j = x_idx[t];
    if (j < 0 || j >= d.n) return;
    const int sh = ((j >> 4) & 1) * 16;
    const uint32_t old = atomicOr(&d.ws.x_mask32[j >> 5], 1u << ((j & 15) + sh));
    const bool newly = ((old >> sh) & 0xFFFFu) == 0, fresh = ((old >> ((j & 15) + sh)) & 1u) == 0;
    const int jb = j >> 4;
    unsigned long long entries = 0, blocks = 0, bytes = 0, ptrs = 0;
    if (d.payload_chunk == PUSH_CHUNK) {
        // handles whose elements sit mostly in blocks with a payload: the whole column block
        if (newly) {
            const int first = d.csc.ptr[jb], n = d.csc.ptr[jb + 1] - first;
            entries += n;
            ptrs += 8;
            count_payload(d, d.csc, first, n, blocks, bytes);
        }
    } else {
        if (fresh) {                                   // the INLINE run of the listed column
            const int32_t *cp = d.csc.colptr + 17 * jb + (j & 15);
            entries += cp[1] - cp[0];
            ptrs += 8;
        }
        if (newly) {                                   // the payload run of the column block
            const int first = d.csc.ptr[jb], n = d.csc.colptr[17 * jb] - first;
            entries += n;
            ptrs += 8;
            count_payload(d, d.csc, first, n, blocks, bytes);
        }
    }
    if (entries) atomicAdd(&acc->view_entries, entries);
    if (blocks) { atomicAdd(&acc->payload_blocks, blocks); atomicAdd(&acc->payload_bytes, bytes); }
    if (ptrs) atomicAdd(&acc->pointer_bytes, ptrs);
    if (newly) atomicAdd(&acc->active_blocks, 1ull);
}

__global__ void k_count_mark(Device d, const int32_t *x_idx, int32_t nnz_x, CountAcc *acc) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= nnz_x) return;
    const int j = x_idx[t];
    if (j < 0 || j >= d.n) return;
    const int sh = ((j >> 4) & 1) * 16;
    const uint32_t old = atomicOr(&d.ws.x_mask32[j >> 5], 1u << ((j & 15) + sh));
    if (((old >> sh) & 0xFFFFu) == 0) atomicAdd(&acc->active_blocks, 1ull);
}

// Pull: every entry of the block-CSR view is read; payloads only under a nonempty vector block.
__global__ void k_count_pull(Device d, CountAcc *acc) {
    const int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (p >= d.n_entries) return;
    const uint32_t idx = d.csr.idx[p];
    const int type = idx >> TYPE_SHIFT;
    if (type == DBSPMSPV_BLK_INLINE) return;
    if (!mask_of(d.ws.x_mask32, idx & IDX_MASK)) return;
    atomicAdd(&acc->payload_blocks, 1ull);
    atomicAdd(&acc->payload_bytes, 4ull * (unsigned long long)payload_words(type, (int)d.csr.aux[p] + 1, vsize_of(d.dtype)));
}

__global__ void k_count_clear(Device d, const int32_t *x_idx, int32_t nnz_x) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= nnz_x) return;
    const int j = x_idx[t];
    if (j >= 0 && j < d.n) d.ws.x_mask32[j >> 5] = 0u;
}

__global__ void k_probe_empty() {}

// `steps` dependent loads by one thread: chain[i] holds the index of the next element.
__global__ void k_probe_chase(const int32_t *chain, int32_t start, int32_t steps, int32_t *out) {
    int32_t i = start;
    for (int32_t s = 0; s < steps; ++s) i = __ldcg(chain + i);
    *out = i;
}

}  // namespace
}  // namespace dbs

extern "C" {

int dbspmspv_count_call_bytes(dbspmspv_handle_t h, const int32_t *x_idx, int32_t nnz_x, int path,
                              dbspmspv_call_bytes *out) {
    using namespace dbs;
    if (!h || !out || nnz_x < 0 || (nnz_x > 0 && !x_idx)) return DBSPMSPV_ERR_INVALID_ARG;
    if (path != DBSPMSPV_PATH_PUSH && path != DBSPMSPV_PATH_PULL) return DBSPMSPV_ERR_INVALID_ARG;
    if (!on_handle_device(h)) return DBSPMSPV_ERR_INVALID_ARG;
    const Device &d = h->d;
    DBS_CUDA(cudaStreamSynchronize(h->last_stream));
    CountAcc *acc = nullptr;
    if (cudaMalloc(&acc, sizeof(CountAcc)) != cudaSuccess) return DBSPMSPV_ERR_ALLOC;
    cudaMemset(acc, 0, sizeof(CountAcc));
    const int g = (nnz_x + 255) / 256;
    if (nnz_x > 0) {
        if (path == DBSPMSPV_PATH_PUSH) {
            k_count_push<<<g, 256>>>(d, x_idx, nnz_x, acc);
        } else {
            k_count_mark<<<g, 256>>>(d, x_idx, nnz_x, acc);
            if (d.n_entries) k_count_pull<<<(d.n_entries + 255) / 256, 256>>>(d, acc);
        }
        k_count_clear<<<g, 256>>>(d, x_idx, nnz_x);
    }
    CountAcc hst;
    const bool ok = cudaMemcpy(&hst, acc, sizeof(hst), cudaMemcpyDeviceToHost) == cudaSuccess;
    cudaFree(acc);
    if (!ok) return DBSPMSPV_ERR_CUDA;
    *out = dbspmspv_call_bytes();
    out->payload_blocks = (int64_t)hst.payload_blocks;
    out->payload_bytes = (int64_t)hst.payload_bytes;
    out->active_vector_blocks = (int64_t)hst.active_blocks;
    if (path == DBSPMSPV_PATH_PUSH) {
        out->view_entries = (int64_t)hst.view_entries;
        out->pointer_bytes = (int64_t)hst.pointer_bytes;
    } else if (nnz_x > 0) {
        if (!h->heavy_stage) {
            // streaming pull: whole chunks of the view, the chunk table, the row list, the list of payload positions
            out->view_entries = (int64_t)d.n_lean_chunks * LEAN_CHUNK;
            out->pointer_bytes = 4 * ((int64_t)d.n_lean_chunks + d.n_lean_rows + d.n_payload);
        } else {
            // pull over weighted chunks of segments: the view, the chunk table, the segments' row blocks
            out->view_entries = d.n_entries;
            out->pointer_bytes = 8 * ((int64_t)d.n_chunks + 1) + 4 * (int64_t)d.n_segments;
        }
    }
    out->view_bytes = 9 * out->view_entries;
    return DBSPMSPV_OK;
}

int dbspmspv_probe_floor(int kind, const int32_t *chain, int32_t start, int32_t steps, int32_t *out,
                         dbspmspv_stream_t stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (kind == 0) {
        dbs::k_probe_empty<<<1, 32, 0, st>>>();
    } else if (kind == 1) {
        if (!chain || !out || steps < 1 || start < 0) return DBSPMSPV_ERR_INVALID_ARG;
        dbs::k_probe_chase<<<1, 1, 0, st>>>(chain, start, steps, out);
    } else {
        return DBSPMSPV_ERR_INVALID_ARG;
    }
    DBS_CUDA(cudaGetLastError());
    return DBSPMSPV_OK;
}

}  // extern "C"
