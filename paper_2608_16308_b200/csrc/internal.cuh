// Internal definitions shared by the .cu files of libdbspmspv: the in-memory block format,
// the handle, and small device helpers.  Nothing here is part of the public ABI.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dbspmspv.h"

namespace dbs {

// ---------------------------------------------------------------------------------------
// Block format (the dual-view storage of Section 3.2.1, laid out for B200)
//
// A "view" is three parallel arrays with one entry per nonempty block:
//   idx[p]  bits 0..26  the block's index along the *other* dimension (column block in the
//                       block-CSR view, row block in the block-CSC view)
//           bit  27     block-CSR view: first INLINE element of its row (ROW_FLAG);
//                       block-CSC view: INLINE element of a hub row block (HUB_FLAG)
//           bit  28     block-CSR view only: first entry of a pull segment
//           bits 29..31 block class (DBSPMSPV_BLK_*)
//   w[p]    payload offset in 4-byte words -- or, for INLINE entries, the stored value itself
//           (fp32 bits, or bf16 bits in the low half; unused for pattern matrices)
//   aux[p]  nnz-1 -- or, for INLINE entries, the packed local coordinate
// A block with at most inline_max stored elements has no payload: it is one INLINE view entry
// per element (adjacent in both views).
// A packed local coordinate is one byte: (row << 4) | col.
// Both views carry the same (w, aux) for a block, so either traversal direction reaches the
// payload in one hop; the payload itself is stored once, in (row block, column block) order.
// The two views mirror each other.  Block-CSR: by row block; inside a row block first the
// entries with a payload (by column block), then the INLINE elements row by row (by column),
// with Device::csr_inl marking where they start.  Block-CSC: by column block; inside it the
// entries with a payload (by row block), then the INLINE elements column by column (by row),
// see View::colptr.  So the elements of one row are adjacent in the block-CSR view (a pull is a
// segmented sum over a stream) and those of one column in the block-CSC view (a push visits
// the listed columns only).
//
// Payload per class (V = value size: 4 fp32, 2 bf16, 0 pattern; every block starts on a
// 16-byte boundary and is padded to a multiple of 16 bytes):
//   COO    nnz coordinate bytes, padded to 4 | nnz values
//   FCSR   16 x u16 row masks | 16 x u8 row starts | values row-major          (Alg. 2)
//   FCSC   16 x u16 column masks | 16 x u8 column starts | values column-major (Alg. 3)
//   CSR    balanced blocks: same encoding as FCSC (column-major suits sparse vector blocks;
//          row access by mask arithmetic) -- except blocks whose longest row has at most
//          CSR_SHORT_ROW entries (banded/stencil blocks), which use the FCSR encoding: two
//          lanes per row then finish in one or two steps (internal code BLK_CSR_ROWMAJOR)
//   DENSE  16 x u16 column masks | 256 values column-major (absent entries 0)
// Pattern matrices keep only the masks (and coordinate bytes).
// ---------------------------------------------------------------------------------------
constexpr int B = 16;                       // block edge
// Internal class code 6: a balanced (CSR-class) block whose rows are short, stored row-major
// like ForceCSR; statistics and exports report it as DBSPMSPV_BLK_CSR.
constexpr int BLK_CSR_ROWMAJOR = 6;
constexpr int CSR_SHORT_ROW = 4;            // longest row at most this -> row-major sub-form
__host__ __device__ inline bool is_row_major(int type) { return type == DBSPMSPV_BLK_FCSR || type == BLK_CSR_ROWMAJOR; }
__host__ __device__ inline int public_class(int type) { return type == BLK_CSR_ROWMAJOR ? DBSPMSPV_BLK_CSR : type; }
constexpr uint32_t IDX_MASK = 0x07FFFFFFu;  // 27 bits
constexpr int TYPE_SHIFT = 29;
constexpr uint32_t ROW_FLAG = 1u << 27;     // block-CSR view: first INLINE element of its row
// Hub row blocks: the few row blocks that hold a large share of a power-law matrix.  Atomics on
// one line are served one after the other by the L2 slice that owns it, so the push gives
// every hub row block HUB_COPIES private accumulators (Device::hub_acc); the compaction folds them.
constexpr uint32_t HUB_FLAG = 1u << 27;     // block-CSC view: INLINE element whose row block is a hub
#ifndef DBS_HUB_COPIES
#define DBS_HUB_COPIES 16
#endif
#ifndef DBS_HUB_BLOCKS_MAX
#define DBS_HUB_BLOCKS_MAX 256
#endif
#ifndef DBS_HUB_MIN_ENTRIES
#define DBS_HUB_MIN_ENTRIES 4096
#endif
constexpr int HUB_COPIES = DBS_HUB_COPIES;              // private accumulator copies per hub row block (power of two)
constexpr int HUB_BLOCKS_MAX = DBS_HUB_BLOCKS_MAX;      // hub row blocks per handle, at most
constexpr int HUB_BLOCK_MIN_ENTRIES = DBS_HUB_MIN_ENTRIES; // view entries that make a row block a hub
constexpr uint16_t HUB_NONE = 0xFFFFu;
constexpr int HUB_MIN_NNZ_X = 32768;        // shorter x: too few products for a queue, and the fold kernel is one more step in the chain
constexpr uint32_t HUB_CLEAR = 0x80000000u; // an untouched private accumulator: -0.0f (see push_private)
constexpr uint32_t PAD_IDX = 7u << TYPE_SHIFT;   // class code of the slack behind the last view entry: no kernel acts on it
// The streaming pull of hypersparse handles takes the block-CSR view in chunks of LEAN_CHUNK
// entries, one chunk (eight entries per lane) per warp pass.
#ifndef DBS_LEAN_CHUNK
#define DBS_LEAN_CHUNK 256
#endif
constexpr int LEAN_CHUNK = DBS_LEAN_CHUNK;
#ifndef DBS_PUSH_CHUNK
#define DBS_PUSH_CHUNK 32
#endif
constexpr int PUSH_CHUNK = DBS_PUSH_CHUNK;   // CSC-view entries per push task (32 per warp step)
static_assert(PUSH_CHUNK == 32, "a push task is one warp step; its record stores the exact entry count in 5 bits");
// A run of the push worklist with at least HUB_MIN_ENTRIES entries (a hub column) is not cut
// into tasks: it is listed once and every warp of the traversal strides over its 32-entry steps.
constexpr int HUB_MIN_ENTRIES = 8192;
constexpr int HUB_CAP = 32;
// Stage of the single-kernel decode: payload bytes per chunk, at most (a chunk also has at
// most 32 view entries: one per lane)
#ifndef DBS_STAGE_BYTES
#define DBS_STAGE_BYTES (6 * 1024)
#endif
constexpr int STAGE_BYTES = DBS_STAGE_BYTES;
constexpr int HDR_BYTES = 48;               // masks + starts of a valued mid-class block

// Payload size in 4-byte words; every block is padded to 16 bytes so that it can be moved with
// one bulk copy.  vsize = bytes per value (4 fp32, 2 bf16, 0 pattern).
__host__ __device__ inline int payload_words(int type, int nnz, int vsize) {
    int bytes;
    switch (type) {
        case DBSPMSPV_BLK_INLINE: return 0;
        case DBSPMSPV_BLK_COO: bytes = ((nnz + 3) & ~3) + nnz * vsize; break;
        case DBSPMSPV_BLK_DENSE: bytes = 32 + 256 * vsize; break;
        default: bytes = vsize ? HDR_BYTES + nnz * vsize : 32; break;
    }
    return ((bytes + 15) & ~15) / 4;
}

struct View {
    int32_t *ptr;    // nb_major + 1
    uint32_t *idx;   // n_entries
    uint32_t *w;     // n_entries
    uint8_t *aux;    // n_entries
    // Block-CSC view only.  Inside a column block the entries are ordered: first the block
    // entries with a payload (by row block), then the INLINE elements column by column (by row).
    // colptr[17 * jb + c], c = 0..16, delimits them: the payload run is [ptr[jb], colptr[17 jb]),
    // the INLINE elements of local column c are [colptr[17 jb + c], colptr[17 jb + c + 1]), and
    // colptr[17 jb + 16] = ptr[jb + 1].  A push therefore visits only the elements of the columns
    // x actually lists, not every element of an active column block.
    int32_t *colptr;
};

struct Segment {     // pull work unit: a run of consecutive view entries inside one row block
    int32_t row_block;
    int32_t start;   // first position in the block-CSR view
    int32_t count;   // bit 31: the segment covers its whole row block (plain stores allowed)
    int32_t weight;  // accumulated cost weight (Section 3.3.2)
};

// Pull streams the block-CSR view through shared memory in chunks: chunk k owns the consecutive
// segments whose exclusive weight prefix lies in [k * PULL_CH, (k+1) * PULL_CH).  Every entry
// weighs at least 1 and a segment has at most MAX_SEG_ENTRIES entries, so a chunk spans fewer
// than PULL_CH + MAX_SEG_ENTRIES entries, and equal weight per chunk balances the warps.
#ifndef DBS_PULL_CH
#define DBS_PULL_CH 256
#endif
constexpr int PULL_CH = DBS_PULL_CH;
constexpr int MAX_SEG_ENTRIES = 128;
constexpr int STAGE_CAP = PULL_CH + MAX_SEG_ENTRIES + 32;   // + alignment slack (16 each side)
constexpr int VIEW_PAD = LEAN_CHUNK + 32;                    // view arrays are over-allocated by this (a whole staging chunk and alignment slack)

// Dense-x marker for "not listed": a NaN bit pattern that listed values never take (listed
// NaNs are stored as the canonical quiet NaN), so one gather yields presence and value.
constexpr uint32_t X_ABSENT = 0x7FFFFFFFu;

struct Counters {    // device-resident scalars of one call
    int32_t n_nzblk;      // nonempty vector blocks
    int32_t n_tasks;      // push worklist length
    int32_t path;         // chosen path of the call (DBSPMSPV_PATH_PUSH / _PULL)
    int32_t y_nnz;
    int32_t status;       // deferred device status
    int32_t last_n_nzblk, last_n_tasks, last_path, last_y_nnz;
    int32_t bfs_levels, bfs_reached;
    int32_t pad;
    int32_t batch_fallback;   // decode_batch: the tensor-core kernel left its vectors to the per-column kernel behind it
    int32_t n_hubs;         // hub runs of this call's push worklist (may exceed HUB_CAP: the rest became tasks)
    int32_t bfs_hubs[3];    // BFS: the same per level (the per-level counters rotate three ways: the
                            // level's own, the ones it accumulates for the next level, and a spare
                            // set that is reset meanwhile)
    int32_t bfs_nwords[4];  // BFS: lengths of the four rotating lists of nonzero mask words (Workspace::bfs_words)
    int32_t bfs_cnt[3][2];  // BFS: {nonempty frontier blocks, tasks}
    int32_t bfs_level_path[DBSPMSPV_MAX_BFS_LEVELS_RECORDED];
    int32_t bfs_level_nzblk[DBSPMSPV_MAX_BFS_LEVELS_RECORDED];
    // BFS: device time stamps (ns): [0] kernel start, [1 + L] start of level L, then the end of the last level
    unsigned long long bfs_stamp[DBSPMSPV_MAX_BFS_LEVELS_RECORDED + 2];
};

struct Workspace {
    float *x_dense;       // n (padded to a multiple of 32): dense copy of x (Section 3.2.2)
    uint32_t *x_mask32;   // vector-block masks, two 16-bit masks per word
    uint2 *tasks;         // push worklist: (column block | (entries - 1) << 27, first CSC-view position)
    int4 *hubs;           // 3 x HUB_CAP hub runs (column block, first position, entries, -): see worklist.cuh
    float *y_acc;         // m (padded): dense accumulator, all zero between calls
    uint32_t *y_mask32;   // run: hit masks packed by the compaction pass; BFS: next-frontier masks
    uint8_t *y_hit8;      // run: one structural-hit flag byte per row, all zero between calls
    int32_t *tile_count;  // compaction: result entries per tile of row blocks
    int32_t *tile_group;  // compaction: [2][n_tile_groups] totals of groups of 32 tiles, by call parity
    int32_t n_tile_groups;
    uint32_t *visited32;  // BFS: visited masks
    uint32_t *z_mask32;   // BFS: third mask buffer (frontier / next / being cleared rotate)
    int32_t *bfs_words;   // BFS: four lists of bfs_words_stride ints: the nonzero mask words of the frontiers produced by
                          // the levels L, L-1, L-2 (rotating, list L % 4 is written while level L runs)
    int32_t bfs_words_stride;
    Counters *ctr;
    int64_t task_capacity;
    int32_t n_tiles;
};

struct Device {           // everything the kernels need, passed by value
    int64_t m, n;
    int32_t mb, nb;       // row blocks, column blocks
    int32_t n_entries;    // view entries (>= nonempty blocks: a small block is one entry per stored element)
    int32_t n_segments;
    int32_t dtype;
    View csr, csc;
    const uint8_t *payload;
    uint32_t payload_words;   // its size in 4-byte words
    const Segment *segments;
    const int32_t *seg_rb;  // row block of every segment (compact copy for the pull kernel)
    const int2 *chunks;   // n_chunks + 1: {first segment, first entry} of every pull chunk
    int32_t n_chunks;
    int32_t payload_chunk;  // entries with a payload per push task (see allocate_workspace)
    // Row-run index for the pull levels of DB-BFS (square matrices, unless switched off): the
    // INLINE elements once more, row by row -- rowrun_idx[k] = column block | local column << 27
    // for k in [rowrun_ptr[i], rowrun_ptr[i + 1]) -- so that a row can stop at its first frontier
    // neighbour.  Null when not built.
    const int32_t *rowrun_ptr;
    const uint32_t *rowrun_idx;
    // Block-CSR view: csr_inl[rb] = first INLINE element of row block rb; its entries with a
    // payload are [csr.ptr[rb], csr_inl[rb]), its INLINE elements [csr_inl[rb], csr.ptr[rb + 1]).
    const int32_t *csr_inl;
    const int32_t *entry_row;   // row block of every block-CSR view entry
    // Streaming pull (hypersparse handles only, else null): lean_rows[k] = the k-th row that
    // holds INLINE elements (the k-th ROW_FLAG of the view); lean_chunk_ord[c] = ROW_FLAGs before
    // entry c * LEAN_CHUNK; payload_pos[0 .. n_payload) = view positions of the entries with a payload.
    const int32_t *lean_rows;
    const int32_t *lean_chunk_ord;
    const int32_t *payload_pos;
    int32_t n_lean_chunks;
    int32_t n_lean_rows;
    int32_t n_payload;
    // Streaming decode (handles whose elements sit mostly in blocks with a payload; null
    // otherwise): the payload of a row block is one contiguous byte range, cut into chunks of
    // whole blocks that fit a warp's shared-memory stage.  stage_chunks[c] = {first view entry,
    // row block, payload offset in words, words | entries << 24}, in payload order.
    const int4 *stage_chunks;
    int32_t n_stage_chunks;
    int32_t stage_bytes;        // payload bytes of one stage (a multiple of 512)
    int32_t has_inline;         // the handle holds INLINE elements at all
    float decode_tau;           // per call: activation magnitude cut of dbspmspv_decode (run option)
    int32_t decode_relu;        // per call: ReLU fused into the cut (x_j > tau instead of |x_j| > tau)
    int32_t decode_x_f32;       // per call: x of a bf16 handle is given in fp32 (rounded to bf16 here)
    int32_t x_sparse_believed;  // per call: what the host currently takes x for (1: sparse)
    int32_t *x_nnz_seen;        // mapped host word: nonzero elements of the x of the last single-kernel decode (null: none)
    // Hub row blocks (null / 0 when the matrix has none): hub_slot[rb] = slot of row block rb or
    // HUB_NONE; hub_acc[(copy * n_hub_blocks + slot) * 16 + row] = private accumulators, all
    // HUB_CLEAR between calls.
    // hub_rb[slot] = the row block; hub_on: this call's push uses them (set per call by the host).
    const uint16_t *hub_slot;
    const int32_t *hub_rb;
    float *hub_acc;
    int32_t n_hub_blocks;
    int32_t hub_on;
    const uint32_t *row_present32;  // per row block: rows that hold a stored element (two 16-bit masks per word)
    Workspace ws;
};

}  // namespace dbs

struct dbspmspv_handle_s {
    dbs::Device d;
    int device;                 // CUDA device ordinal the handle lives on
    int sm_count;
    int64_t nnz;
    int32_t *csc2csr;           // CSC-view position -> primary block id (Section 3.2.1)
    int32_t *block_row;         // primary order: row block of every block
    dbspmspv_create_opts copts;
    dbspmspv_run_opts ropts;
    dbspmspv_stats stats;       // host copy of the static part
    void *payload_alloc;
    int64_t payload_bytes;
    int bfs_grid;               // co-resident grid size of the BFS kernel
    // launch configurations, worked out on first use (function attributes and occupancy are per
    // device, and a handle lives on one device; calls on a handle are stream ordered, so plain fields)
    int grid_compute, grid_compute_dense, grid_decode_pull;
    bool lean_configured, lean_configured_dense, lean_configured_min;
    bool fused_configured[3];
    bool batch_configured[2];
    bool batch_mma_configured[3];
    uint32_t compact_calls;     // compaction launches so far (their parity picks the group-total buffer)
    int stream_grid;            // thread blocks of the streaming decode (0: not configured yet)
    int32_t *x_nnz_seen_host;   // host view of Device::x_nnz_seen (page-locked, mapped)
    bool heavy_stage;           // most stored elements sit in mask-based blocks: MODE 1 kernels
    cudaEvent_t ev[2];          // optional timing of the traversal kernel (run_opts.timing)
    bool timed;
    int64_t kernel_launches;    // kernels this handle has launched (run / decode / bfs)
    int64_t bfs_index_bytes;
    int64_t lean_index_bytes;
    int64_t hub_bytes;
    int64_t stage_index_bytes;
    void *ws_arena;             // the one allocation that holds the whole workspace
    void *sssp_arena;           // db_sssp: frontier lists, y and counters (allocated by the first search)
    int32_t *sssp_host;         // db_sssp: page-locked word the size of the next frontier is copied to
    cudaStream_t last_stream;   // stream of the last run / decode / bfs call (get_stats waits on it)
};

namespace dbs {

#define DBS_CUDA(call)                                      \
    do {                                                    \
        cudaError_t e__ = (call);                           \
        if (e__ != cudaSuccess) return DBSPMSPV_ERR_CUDA;   \
    } while (0)

template <typename T>
__host__ __device__ inline T ceil_div(T a, T b) { return (a + b - 1) / b; }

// Streaming decode (run.cu): the payload bytes of one stage that shared memory leaves room for
// on this handle (0: none).
int decode_stage_bytes(const Device &d);

// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may
// start while its predecessor drains; `pdl_wait` blocks until the predecessor has completed and
// its writes are visible (a no-op for a normally launched kernel), `pdl_launch_dependents`
// lets the successor's launch proceed early.  This hides the launch latency between the short
// kernels of one call.
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Range-checked build (-DDBS_BOUNDS_CHECK; it stands in for a memory checker on the small parity
// cases): every index that a kernel READS from the handle's arrays -- the other-dimension block
// index and the payload offset of a view entry, the entry range of a task, a column run, a
// segment or a chunk, a listed row -- is tested before it is used; a violation records
// DBSPMSPV_ERR_INTERNAL in the status word and the access is skipped (the entry is replaced
// by a harmless one, the range is emptied).  Nothing traps.  In the normal build these compile to nothing.
#ifdef DBS_BOUNDS_CHECK
__device__ __forceinline__ bool chk_fail(const Device &d) { d.ws.ctr->status = DBSPMSPV_ERR_INTERNAL; return false; }
__device__ __forceinline__ bool chk_index(const Device &d, int64_t i, int64_t n) { return (i >= 0 && i < n) || chk_fail(d); }
// entries [first, first + count) of a view
__device__ __forceinline__ bool chk_range(const Device &d, int64_t first, int64_t count) {
    return (first >= 0 && count >= 0 && first + count <= (int64_t)d.n_entries) || chk_fail(d);
}
// a view entry as loaded: one that points outside the handle is replaced by an INLINE element
// (0, 0) of block 0 with the value 0 -- every access it leads to is in range
template <typename A>
__device__ __forceinline__ void chk_entry(const Device &d, bool csr_view, uint32_t &idx, uint32_t &w, A &aux) {
    const int type = (int)(idx >> TYPE_SHIFT);
    if (type == 7) return;                                       // padding behind the last entry
    const int vsize = d.dtype == DBSPMSPV_F32 ? 4 : d.dtype == DBSPMSPV_BF16 ? 2 : 0;
    bool ok = (int)(idx & IDX_MASK) < (csr_view ? d.nb : d.mb) && type <= BLK_CSR_ROWMAJOR;
    if (ok && type != DBSPMSPV_BLK_INLINE) ok = (uint64_t)w + (uint64_t)payload_words(type, (int)aux + 1, vsize) <= (uint64_t)d.payload_words;
    if (!ok) { chk_fail(d); idx = (uint32_t)DBSPMSPV_BLK_INLINE << TYPE_SHIFT; w = 0u; aux = 0; }
}
#define DBS_CHK_INDEX(d, i, n) dbs::chk_index((d), (int64_t)(i), (int64_t)(n))
#define DBS_CHK_RANGE(d, first, count) dbs::chk_range((d), (int64_t)(first), (int64_t)(count))
#define DBS_CHK_ENTRY(d, csr_view, idx, w, aux) dbs::chk_entry((d), (csr_view), (idx), (w), (aux))
#else
#define DBS_CHK_INDEX(d, i, n) true
#define DBS_CHK_RANGE(d, first, count) true
#define DBS_CHK_ENTRY(d, csr_view, idx, w, aux) ((void)0)
#endif

// 16-bit mask of one block.  The mask arrays are updated as 32-bit words (two blocks per word,
// the even block in the low half: atomics need the word) but read as the halfword itself: one
// 16-bit load instead of a word load plus shift and mask (the GPU is little-endian).
__device__ __forceinline__ uint32_t mask_of(const uint32_t *mask32, int blk) {
    return reinterpret_cast<const uint16_t *>(mask32)[blk];
}

// value loads from the payload, widened to fp32
template <int DT> struct Val;
template <> struct Val<DBSPMSPV_F32> {
    static constexpr int SIZE = 4;
    __device__ static __forceinline__ float load(const uint8_t *base, int k) {
        return reinterpret_cast<const float *>(base)[k];
    }
    __device__ static __forceinline__ float inline_value(uint32_t w) { return __uint_as_float(w); }
};
template <> struct Val<DBSPMSPV_BF16> {
    static constexpr int SIZE = 2;
    __device__ static __forceinline__ float load(const uint8_t *base, int k) {
        return __uint_as_float(uint32_t(reinterpret_cast<const uint16_t *>(base)[k]) << 16);
    }
    __device__ static __forceinline__ float inline_value(uint32_t w) {
        return __uint_as_float((w & 0xFFFFu) << 16);
    }
};
template <> struct Val<DBSPMSPV_PATTERN> {
    static constexpr int SIZE = 0;
    __device__ static __forceinline__ float load(const uint8_t *, int) { return 1.0f; }
    __device__ static __forceinline__ float inline_value(uint32_t) { return 1.0f; }
};

// The entry points enqueue on the calling thread's current device: it has to be the handle's.
inline bool on_handle_device(const dbspmspv_handle_s *h) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == h->device;
}

}  // namespace dbs
