// dbspmspv_compact_noalloc: the output-compaction step (dense accumulator + row-hit bitmap ->
// sorted sparse vector) as a stand-alone entry point that allocates nothing.  It is meant for
// callers that are not allowed to allocate device memory at the point of the call: code that
// runs between fixed-memory-budget phases of a larger application, real-time loops that must
// not enter the allocator, or plug-ins whose host owns every byte of the device heap.
//
// The compaction kernels need one counter per tile of 8192 rows.  The library's normal path
// keeps those counters in the handle's workspace (allocated by create); here they live in a
// file-scope __device__ array of fixed size, which every GPU that loads the library holds
// until the process exits (16 KB).
#include <mutex>

#include "internal.cuh"

namespace dbs {
namespace {

constexpr int NA_TPB = 256;                       // one 32-row bitmap word per thread
constexpr int NA_TILE_ROWS = NA_TPB * 32;         // 8192 rows per tile
constexpr int NA_MAX_TILES = 4096;                // -> at most 33,554,432 rows per call

static __device__ __align__(256) int32_t g_tile_scratch[NA_MAX_TILES];

// Host code must not hand `g_tile_scratch` itself to a kernel: on the host that name is only a
// stand-in for the symbol.  The real device address is looked up once per device and kept for
// the life of the process (a cudaDeviceReset would invalidate it: not supported while the
// library is in use).
constexpr int NA_MAX_DEVICES = 64;
int32_t *g_scratch_addr[NA_MAX_DEVICES] = {};
std::mutex g_setup_lock;

// Bits at or beyond row m in the last bitmap word are ignored by both passes (so the count and
// the placement agree whatever the caller left there).
__device__ __forceinline__ uint32_t na_word(const uint32_t *hit, int wi, int n_words, int64_t m) {
    if (wi >= n_words) return 0u;
    uint32_t word = hit[wi];
    if (wi == n_words - 1 && (m & 31)) word &= (1u << (m & 31)) - 1u;
    return word;
}

__global__ void __launch_bounds__(NA_TPB) k_na_count(const uint32_t *__restrict__ hit, int64_t m, int n_words, int32_t *tiles) {
    __shared__ int s_red[NA_TPB / 32];
    const int wi = blockIdx.x * NA_TPB + threadIdx.x;
    int c = __popc(na_word(hit, wi, n_words, m));
    c = __reduce_add_sync(0xFFFFFFFFu, c);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int k = 0; k < NA_TPB / 32; ++k) t += s_red[k];
        tiles[blockIdx.x] = t;     // every slot this call reads later is written here first
    }
}

__global__ void __launch_bounds__(NA_TPB) k_na_write(const float *__restrict__ acc, const uint32_t *__restrict__ hit,
                                                     int64_t m, int n_words, const int32_t *tiles,
                                                     int32_t *__restrict__ y_idx, float *__restrict__ y_val,
                                                     int64_t capacity, int32_t *__restrict__ y_nnz) {
    __shared__ int s_red[NA_TPB / 32];
    __shared__ int s_base;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int before = 0;
    for (int k = threadIdx.x; k < (int)blockIdx.x; k += NA_TPB) before += tiles[k];
    before = __reduce_add_sync(0xFFFFFFFFu, before);
    if (lane == 0) s_red[warp] = before;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int k = 0; k < NA_TPB / 32; ++k) t += s_red[k];
        s_base = t;
    }
    __syncthreads();
    const int wi = blockIdx.x * NA_TPB + threadIdx.x;
    const uint32_t word = na_word(hit, wi, n_words, m);
    const int c = __popc(word);
    int incl = c;
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();
    if (lane == 31) s_red[warp] = incl;
    __syncthreads();
    int64_t pos = s_base + incl - c;
    for (int k = 0; k < warp; ++k) pos += s_red[k];
    for (uint32_t wd = word; wd; wd &= wd - 1) {
        const int64_t row = (int64_t)wi * 32 + (__ffs(wd) - 1);
        if (pos < capacity) {
            y_idx[pos] = (int32_t)row;
            if (y_val) y_val[pos] = acc[row];
        }
        ++pos;
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == NA_TPB - 1) *y_nnz = (int32_t)pos;
}

}  // namespace
}  // namespace dbs

extern "C" int dbspmspv_compact_noalloc(const float *acc, const uint32_t *hit_bitmap, int64_t m,
                                        int32_t *y_idx, float *y_val, int64_t y_capacity,
                                        int32_t *y_nnz, dbspmspv_stream_t stream) {
    using namespace dbs;
    if (!hit_bitmap || !y_nnz || m < 1 || y_capacity < 0) return DBSPMSPV_ERR_INVALID_ARG;
    if (y_capacity > 0 && !y_idx) return DBSPMSPV_ERR_INVALID_ARG;
    if (y_val && !acc) return DBSPMSPV_ERR_INVALID_ARG;
    const int64_t n_tiles64 = (m + NA_TILE_ROWS - 1) / NA_TILE_ROWS;
    if (n_tiles64 > NA_MAX_TILES) return DBSPMSPV_ERR_TOO_LARGE;   // the fixed scratch is too small
    int dev = 0;
    DBS_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= NA_MAX_DEVICES) return DBSPMSPV_ERR_UNSUPPORTED;
    int32_t *tiles = nullptr;
    {
        // set-up, once per device, with that device current: resolve the symbol to its address
        std::lock_guard<std::mutex> guard(g_setup_lock);
        if (!g_scratch_addr[dev]) {
            int32_t *p = nullptr;
            if (cudaGetSymbolAddress((void **)&p, g_tile_scratch) != cudaSuccess || !p) {
                cudaGetLastError();          // do not leave the error behind for the caller's next check
                return DBSPMSPV_ERR_CUDA;
            }
            g_scratch_addr[dev] = p;
        }
        tiles = g_scratch_addr[dev];
    }
    const int n_words = (int)((m + 31) / 32);
    const int n_tiles = (int)n_tiles64;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    k_na_count<<<n_tiles, NA_TPB, 0, st>>>(hit_bitmap, m, n_words, tiles);
    k_na_write<<<n_tiles, NA_TPB, 0, st>>>(acc, hit_bitmap, m, n_words, tiles, y_idx, y_val, y_capacity, y_nnz);
    DBS_CUDA(cudaGetLastError());
    return DBSPMSPV_OK;
}
