/*
 * dbspmspv.h -- C ABI of the B200 (sm_100a) DB-SpMSpV library.
 *
 * y = A * x with a sparse matrix A held in fixed 16 x 16 blocks and a sparse vector x
 * (problem statement: Section 2.1).  One block payload is stored once; a block-level CSR view
 * (entry point of the pull path) and a block-level CSC view (entry point of the push path)
 * index it (Section 3.2.1).  Per call the input vector is cut into aligned 16-element vector
 * blocks with a 16-bit nonzero mask each (Section 3.2.2), the ratio of nonempty vector blocks
 * selects push or pull (Section 3.3.1), every visited block picks a microkernel from its class
 * and the local mask (Sections 3.3.1, 3.3.3), and results are reduced in the warp and in shared
 * memory before they reach global memory (Section 3.3.3).
 *
 * Conventions
 *   - Every array argument is a DEVICE pointer owned by the caller unless stated otherwise.
 *   - `stream` is a cudaStream_t (passed as an opaque pointer; NULL = the legacy default
 *     stream).  dbspmspv_run / db_bfs / dbspmspv_decode only enqueue work on it: they allocate
 *     nothing, never synchronise, and return as soon as the kernels are queued.  Calls on the
 *     same handle must be stream ordered (the handle owns one workspace).  A handle lives on
 *     the device that was current when it was created; run / db_bfs / decode return
 *     DBSPMSPV_ERR_INVALID_ARG when the calling thread's current device is another one.
 *   - Functions return a dbspmspv_status_t.  Argument errors are reported synchronously.
 *     Conditions detected on the device (output capacity, a bounded wait that ran out) are
 *     recorded in the handle and returned by the next dbspmspv_get_stats; a kernel never traps.
 *   - Bit k of every 16-bit mask is local index k, least significant bit first (Figure 4
 *     caption: mask value 10 = 0b1010 = positions 1 and 3).
 *   - A stored entry A[i][j] is the graph edge j -> i (what y = A*x propagates from x_j).
 *   - "Structural" output: row i is reported iff some stored A[i][j] meets some listed x_j,
 *     whatever the numeric sum is.
 */
#ifndef DBSPMSPV_H
#define DBSPMSPV_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dbspmspv_handle_s *dbspmspv_handle_t;
typedef void *dbspmspv_stream_t; /* cudaStream_t */

typedef enum {
    DBSPMSPV_OK = 0,
    DBSPMSPV_ERR_INVALID_ARG = 1, /* null pointer, negative size, index out of range, ... */
    DBSPMSPV_ERR_UNSUPPORTED = 2, /* block size other than 16, semiring/dtype mismatch    */
    DBSPMSPV_ERR_ALLOC = 3,       /* device or host allocation failed (create only)       */
    DBSPMSPV_ERR_CUDA = 4,        /* a CUDA runtime call failed                           */
    DBSPMSPV_ERR_CAPACITY = 5,    /* y_capacity too small; nothing was written out of bounds */
    DBSPMSPV_ERR_TIMEOUT = 6,     /* a bounded device-side wait ran out                   */
    DBSPMSPV_ERR_BOUNDS = 7,      /* an x index was out of range (the entry was skipped)  */
    DBSPMSPV_ERR_TOO_LARGE = 8,   /* dbspmspv_compact_noalloc: more rows than its fixed scratch covers */
    DBSPMSPV_ERR_INTERNAL = 9     /* range-checked build only (-DDBS_BOUNDS_CHECK): an index read from the
                                     handle's own arrays was out of range; the access was skipped   */
} dbspmspv_status_t;

typedef enum {
    DBSPMSPV_F32 = 0,    /* fp32 values, fp32 accumulation                                 */
    DBSPMSPV_BF16 = 1,   /* bf16 values and bf16 x, fp32 accumulation (Section 4.3 layers) */
    DBSPMSPV_PATTERN = 2 /* no values: Boolean matrices (Section 4.2 graphs)               */
} dbspmspv_dtype_t;

typedef enum {
    DBSPMSPV_PLUS_TIMES = 0,
    DBSPMSPV_OR_AND = 1, /* Boolean: only reachability is computed (Section 4.2)           */
    DBSPMSPV_MIN_PLUS = 2 /* y_i = min_j (A[i][j] + x_j): the shortest-path product of
                             GraphBLAS-style systems (Sections 1, 6)                       */
} dbspmspv_semiring_t;

enum { DBSPMSPV_PATH_AUTO = 0, DBSPMSPV_PATH_PUSH = 1, DBSPMSPV_PATH_PULL = 2 };
enum { DBSPMSPV_FORMAT_AUTO = 0, DBSPMSPV_FORMAT_COO = 1, DBSPMSPV_FORMAT_CSR = 2 };

/* Block classes (Section 3.2.1).  INLINE is this library's sub-case of COO: a block whose few
 * entries fit in its view entry and therefore has no payload at all.                        */
enum {
    DBSPMSPV_BLK_INLINE = 0,
    DBSPMSPV_BLK_COO = 1,
    DBSPMSPV_BLK_FCSR = 2,
    DBSPMSPV_BLK_FCSC = 3,
    DBSPMSPV_BLK_CSR = 4,
    DBSPMSPV_BLK_DENSE = 5,
    DBSPMSPV_BLK_NCLASS = 6
};

/* Options of the format build.  Zero-initialise, then call dbspmspv_default_create_opts.    */
typedef struct {
    int32_t th0;             /* blocks with fewer than th0 entries use packed COO   (32)     */
    int32_t th1;             /* blocks with more than th1 entries use Dense         (128)    */
    float th2;               /* directional skew ratio for ForceCSR / ForceCSC      (2.0)    */
    int32_t seg_cut;         /* a pull segment closes when its weight reaches this  (128, max)*/
    int32_t w_dense;         /* pull segment weight of a Dense block                (16)     */
    int32_t w_mid;           /* ... of a ForceCSR / ForceCSC / CSR block            (8)      */
    int32_t w_coo;           /* ... of a COO block                                  (4)      */
    int32_t force_format;    /* DBSPMSPV_FORMAT_*: ablation knob (Section 5.4)               */
    int32_t input_on_host;   /* 1: the create arrays are HOST pointers (copied once)         */
    int32_t inline_max;      /* a block with at most this many entries keeps
                                them in its view entries, one entry per element      (31)    */
    int32_t w_inline;        /* ... of an INLINE view entry                         (1)      */
    int32_t w_dense_sparse;  /* Dense / CSR-like weights used instead when such blocks are a */
    int32_t w_mid_sparse;    /* minority of the matrix (hypersparse matrices)  (128 / 64)    */
    int32_t no_bfs_index;    /* 1: do not build the row-run index that square matrices get for
                                the pull levels of db_bfs (4 bytes per stored element; a pull
                                level then walks whole row-block segments)          (0)    */
    int32_t reserved[2];
} dbspmspv_create_opts;

/* Run-time options; may be changed between calls with dbspmspv_set_run_opts.               */
typedef struct {
    float th3;               /* dbspmspv_run: push iff the nonempty-vector-block ratio is
                                below th3.  0.01 in the paper; default 0.95, the crossover
                                measured on B200 (the table `bench.py --crossover` prints)    */
    int32_t force_path;      /* DBSPMSPV_PATH_*                                              */
    int32_t popc_threshold;  /* CSR-class blocks: popc(mask) >= this -> row-driven (pull-style)
                                microkernel, below -> column-driven (push-style)             */
    int32_t validate;        /* x indices outside [0, n) are always skipped and reported as
                                ERR_BOUNDS; 1: an index listed twice is reported as well
                                (deferred ERR_INVALID_ARG; it contributes once either way)   */
    int32_t timing;          /* 1: bracket the traversal kernel of run/decode with two CUDA
                                events (made at create); read back as last_compute_ms      */
    float th3_bfs;           /* db_bfs: same rule per level.  Default 0.05, measured on the
                                symmetrised R-MAT scale 22 graph (0.03 .. 0.07 are within 3 %;
                                a pull level stops every row at its first frontier neighbour,
                                a push level pays one atomic per reached entry)             */
    float th3_decode;        /* dbspmspv_decode: same rule; the output is dense and every row block
                                takes part, so pull wins much earlier (0.01, the paper's value) */
    int32_t no_fused_decode; /* dbspmspv_decode on handles whose elements sit mostly in blocks with
                                a payload and whose x fits in shared memory has two one-kernel
                                forms: a streaming one (the whole payload is moved through
                                shared memory by bulk copies) and a selective one (only the
                                block columns x reaches are fetched).
                                0: streaming, or selective when the x of the handle's previous
                                   decode call had fewer than 15 % nonzero elements (default);
                                1: neither -- the blocking / traversal / cleanup kernels of
                                   dbspmspv_run;   2: selective only;   3: streaming only      */
    float bfs_push_max_edge_frac; /* db_bfs (with the row-run index): a level whose push worklist
                                covers more than this share of the view's entries is pulled
                                even when the block ratio says push -- a frontier of a few
                                thousand vertices that include hubs fills few vector blocks but
                                owns a good part of all elements (R-MAT scale 22: 7,800
                                vertices, 19 M of 128 M entries: 189 us pushed, ~90 us
                                pulled).  0 = block ratio only, the paper's rule.  Default
                                0.08, measured (0.06 .. 0.1 are within 1 %)                */
    int32_t hub_min_nnz_x;   /* dbspmspv_run: shortest x list for which the push adds into the
                                private accumulators of hub row blocks (they cost one more
                                kernel in the chain); 0 = default (32768), < 0 = never     */
    float decode_threshold;  /* dbspmspv_decode: activation magnitude cut fused into the vector
                                blocking (Section 5.3: activation sparsity by magnitude
                                thresholding) -- x_j takes part iff |x_j| > decode_threshold;
                                0 (default): iff x_j is not zero.  A NaN always takes part.  */
    int32_t decode_relu;     /* dbspmspv_decode: 1 = ReLU fused into the cut: x_j takes part iff
                                x_j > decode_threshold (negative entries are zeros)        (0) */
    int32_t decode_x_f32;    /* dbspmspv_decode on a bf16 handle: 1 = x is given as n fp32 values
                                (e.g. the y of the layer before, fed straight back in) and
                                rounded to bf16, to nearest even, while it is blocked      (0) */
    int32_t no_small_call;   /* dbspmspv_run on a hypersparse handle with at most 256 entries in x
                                (and a selector that is certain to say push, up to ~2.5 M rows,
                                validate and timing off) runs as one kernel of one cluster of
                                eight thread blocks that keep the result's row bitmap in their
                                shared memories; 1 = use
                                the general chain of kernels instead                      (0) */
    int32_t reserved[2];
} dbspmspv_run_opts;

#define DBSPMSPV_MAX_BFS_LEVELS_RECORDED 64

typedef struct {
    /* matrix / format (fixed at create) */
    int64_t m, n, nnz;             /* nnz after merging duplicates                            */
    int64_t n_blocks;              /* nonempty 16 x 16 blocks                                 */
    int64_t n_view_entries;        /* entries per view (>= n_blocks: INLINE blocks of valued
                                      matrices hold one entry per stored element)            */
    int64_t class_blocks[DBSPMSPV_BLK_NCLASS]; /* per DBSPMSPV_BLK_* class                    */
    int64_t class_nnz[DBSPMSPV_BLK_NCLASS];
    int64_t n_row_blocks, n_col_blocks;        /* ceil(m/16), ceil(n/16)                      */
    int64_t n_segments;            /* pull segments                                           */
    int64_t payload_bytes;         /* the single block payload                                */
    int64_t csr_view_bytes;        /* block-CSR view: row pointers + per-block entries        */
    int64_t csc_view_bytes;        /* block-CSC view: column pointers + per-block entries (+ the
                                      slot table and private accumulators of hub row blocks)  */
    int64_t segment_bytes;
    int64_t workspace_bytes;       /* per-call scratch owned by the handle                    */
    /* last dbspmspv_run / dbspmspv_decode */
    int32_t last_path;             /* DBSPMSPV_PATH_PUSH or _PULL                             */
    int32_t last_n_nzblk;          /* nonempty vector blocks                                  */
    int32_t last_n_tasks;          /* push worklist length                                    */
    int32_t last_y_nnz;
    /* last db_bfs */
    int32_t bfs_levels;            /* number of expansion steps executed                      */
    int32_t bfs_reached;           /* vertices with level >= 0                                */
    int32_t bfs_level_path[DBSPMSPV_MAX_BFS_LEVELS_RECORDED];  /* per level DBSPMSPV_PATH_*   */
    int32_t bfs_level_nzblk[DBSPMSPV_MAX_BFS_LEVELS_RECORDED]; /* frontier vector blocks      */
    /* deferred device status of the last call (DBSPMSPV_OK if none) */
    int32_t device_status;
    float last_compute_ms;         /* traversal kernel time of the last run/decode (timing=1),
                                      else -1                                                 */
    int64_t kernel_launches;       /* kernels launched through this handle so far             */
    int64_t bfs_index_bytes;       /* row-run index of DB-BFS (0 when not built)              */
    int64_t lean_index_bytes;      /* row list / chunk table of the streaming pull (hypersparse
                                      handles; 0 otherwise)                                   */
    /* last db_bfs, from time stamps taken on the device: microseconds before the first level
       (initialisation of levels and masks) and per level (traversal + frontier bookkeeping)    */
    float bfs_setup_us;
    float bfs_level_us[DBSPMSPV_MAX_BFS_LEVELS_RECORDED];
    int32_t n_hub_row_blocks;      /* row blocks with private push accumulators (0: none)     */
} dbspmspv_stats;

/* Paper thresholds (th0 = 32, th1 = 128, th2 = 2.0, Section 3.2.1).  The segment weights keep
 * the paper's ordering Dense > CSR-like > COO (Section 3.3.2) but are rescaled (16 / 8 / 4 / 1
 * against a cut of 128) because one warp step here covers 32 INLINE entries but one heavier
 * block.  Run-time defaults are this library's measured ones.                                      */
void dbspmspv_default_create_opts(dbspmspv_create_opts *opts);
void dbspmspv_default_run_opts(dbspmspv_run_opts *opts);

/*
 * Build the dual-view blocked format from CSR (Section 3.2.1).  Runs on the GPU and
 * synchronises `stream` before returning (it is the offline step, Section 5.5).
 *   m, n     matrix shape (1 <= m, n < 2^31); nnz >= 0 stored entries (< 2^31)
 *   row_ptr  m+1 int64 offsets; col_idx nnz int32 columns (any order within a row)
 *   val      nnz values of type `dtype` (float or bf16 bit patterns); ignored for PATTERN
 *   Duplicate (i, j) entries are summed (PATTERN: merged); explicitly stored zeros are kept as
 *   structural entries.  block_size must be 16 (the only size the paper evaluates).
 *   opts     NULL = defaults.  The input arrays are not referenced after return.
 * Errors: INVALID_ARG (null/negative/out-of-range index), UNSUPPORTED, ALLOC, CUDA.
 */
int dbspmspv_create_csr(dbspmspv_handle_t *out, int64_t m, int64_t n, int64_t nnz,
                        const int64_t *row_ptr, const int32_t *col_idx, const void *val,
                        int dtype, int block_size, const dbspmspv_create_opts *opts,
                        dbspmspv_stream_t stream);

/* Same from coordinate triples (row[k], col[k], val[k]), any order.                          */
int dbspmspv_create_coo(dbspmspv_handle_t *out, int64_t m, int64_t n, int64_t nnz,
                        const int32_t *row, const int32_t *col, const void *val, int dtype,
                        int block_size, const dbspmspv_create_opts *opts,
                        dbspmspv_stream_t stream);

/*
 * One SpMSpV call y = A * x (Sections 3.3, 4.1): vector blocking, path selection, worklist,
 * block microkernels, writeback and compaction, all enqueued on `stream`.
 *   x_idx    nnz_x distinct indices in [0, n), any order; x_val nnz_x values of the handle's
 *            dtype (float, or bf16 bit patterns; ignored/NULL for OR_AND).  Both must stay
 *            valid and unchanged until the call has finished on the stream.
 *   semiring PLUS_TIMES (F32/BF16 handles), OR_AND (any handle; values are then 1.0f) or
 *            MIN_PLUS (any handle; a pattern handle's elements weigh 1): y_i is the smallest
 *            A[i][j] + x_j over the stored elements of row i whose x_j is listed, in fp32; a
 *            listed 0 takes part like any other value; NaN operands give unspecified values.
 *            MIN_PLUS always takes the push path (force_path is ignored).
 *   y_idx    out: row indices of the structural result, ascending; y_val out: fp32 sums
 *            (may be NULL for OR_AND); both with room for y_capacity entries
 *   y_nnz    out: one int32, the number of result entries (the full count even when it
 *            exceeds y_capacity; then only the first y_capacity are written and the deferred
 *            status is ERR_CAPACITY)
 * x_idx, x_val, y_idx, y_val and y_nnz are device pointers -- or page-locked host memory that
 * the device addresses directly (cudaHostAlloc / cudaHostRegister under unified addressing):
 * the call's kernels then read x and write y across the bus themselves, with no staging copy
 * (x_idx is read a second time by the clean-up pass unless x lists more than n / 8 columns).
 * nnz_x = 0 gives y_nnz = 0.  Errors: INVALID_ARG, UNSUPPORTED synchronously.
 */
int dbspmspv_run(dbspmspv_handle_t h, const int32_t *x_idx, const void *x_val, int32_t nnz_x,
                 int semiring, int32_t *y_idx, float *y_val, int64_t y_capacity,
                 int32_t *y_nnz, dbspmspv_stream_t stream);

/*
 * DB-BFS (Section 4.2, Algorithm 5): level-synchronous BFS in which each level is one Boolean
 * SpMSpV with the frontier masks as x, visited vertices stripped, and push or pull chosen per
 * level by the same vector-block ratio.  The whole traversal runs in one cooperative launch.
 *   src      source vertex in [0, n); the matrix must be square (any dtype; values ignored)
 *   levels   out: n int32 on the device; source 0, unreachable -1
 */
int db_bfs(dbspmspv_handle_t h, int32_t src, int32_t *levels, dbspmspv_stream_t stream);

/*
 * Single-source shortest paths as the iteration of MIN_PLUS products (SpMSpV as the primitive
 * of GraphBLAS-style graph algorithms, Sections 1 and 6): x holds the vertices whose distance
 * improved in the last step, y = A (min,+) x relaxes their out-edges, the improved rows of y
 * become the next x.  A stored A[i][j] is the edge j -> i of weight A[i][j] (1 on a pattern
 * handle), as in db_bfs.  Weights may be negative as long as no cycle is.
 *   src      source vertex in [0, n); square F32 or PATTERN handle (BF16: ERR_UNSUPPORTED)
 *   dist     out: n fp32 on the device; source 0, unreachable +infinity.  Every path sum is
 *            accumulated in fp32 in path order.
 *   n_steps  out (host, may be NULL): products made, the last one with an empty result
 * Direction per step: run_opts.force_path if set; else a step whose x holds more than a tenth
 * of the stored elements as out-edges is pulled (hypersparse F32 handles; the others always
 * push), the rest pushed.
 * Unlike the other calls this one is a host loop: it waits on `stream` once per step to read
 * the size of the next x and its out-edge count (16 bytes), and the first call on a handle allocates 24 n bytes of
 * device memory and one page-locked word (freed by dbspmspv_destroy).  More than n + 1 steps
 * (a negative cycle) end the search with ERR_UNSUPPORTED.
 */
int db_sssp(dbspmspv_handle_t h, int32_t src, float *dist, int32_t *n_steps, dbspmspv_stream_t stream);

/*
 * Single-token linear layer (Section 4.3): dense x in, dense y out.  The nonzero mask of x is
 * generated on the GPU by warp ballot (Section 4.1) and drives the same engine.
 *   x        n values of the handle's dtype (F32 or BF16 handles); zeros (+0.0 and -0.0) are
 *            structurally absent
 *   y        out: m fp32 values; rows without a structural hit are exactly 0
 */
int dbspmspv_decode(dbspmspv_handle_t h, const void *x, float *y, dbspmspv_stream_t stream);

/* Waits for the stream the handle's last run / decode / db_bfs call was enqueued on (not for the
 * whole device) and copies the statistics to the HOST struct `out`.  Returns the deferred
 * device status of the last call, which is then cleared.                                      */
int dbspmspv_get_stats(dbspmspv_handle_t h, dbspmspv_stats *out);

/* Test hook: decode the blocked format back to coordinates.  row/col/val: device arrays with
 * room for stats.nnz entries (val may be NULL; element type = the handle's dtype).  Order: the
 * elements of every block-CSR view entry together, entries in view order (see
 * dbspmspv_export_blocks); sort before comparing with a matrix.  Synchronises.               */
int dbspmspv_export_coo(dbspmspv_handle_t h, int32_t *row, int32_t *col, void *val);

/* Test hook: per view entry, in block-CSR view order: block coordinates, class code
 * (DBSPMSPV_BLK_*) and stored elements of the entry.  Device arrays of stats.n_view_entries
 * int32 (any may be NULL).  Block-CSR view order: by row block; inside a row block the entries
 * with a payload first (by column block), then the INLINE elements (one entry each) by
 * (local row, column) -- the elements of one row are adjacent.                               */
int dbspmspv_export_blocks(dbspmspv_handle_t h, int32_t *block_row, int32_t *block_col,
                           int32_t *block_class, int32_t *block_nnz);

/* Test hook: copy the dual view out: csr_row_ptr (n_row_blocks+1), csc_col_ptr
 * (n_col_blocks+1), csc_row (n_view_entries: row block of every CSC-view position), csc2csr
 * (n_view_entries: CSC-view position -> primary entry id).  Device int32 arrays; any may be
 * NULL.  CSC-view order: by column block; inside a column block the entries with a payload
 * first (by row block), then the INLINE elements by (local column, row block, local row).    */
int dbspmspv_export_views(dbspmspv_handle_t h, int32_t *csr_row_ptr, int32_t *csc_col_ptr,
                          int32_t *csc_row, int32_t *csc2csr);

/*
 * Output compaction without any allocation.  (The paper has no counterpart: it returns a dense
 * y.  This entry point exists for callers that may not allocate device memory at the point of
 * the call -- real-time loops that must stay out of the allocator, hosts that own the whole
 * device heap, phases of a larger program with a frozen memory budget -- and that already hold
 * a dense result plus a row-hit bitmap, for instance from their own kernels.)
 *
 *   acc         m fp32 values (device); only rows whose bit is set are read
 *   hit_bitmap  ceil(m/32) uint32 words (device): bit (i & 31) of word (i >> 5) set iff row i
 *               belongs to the result; bits at or beyond m in the last word are ignored
 *   y_idx/y_val out: the set rows in ascending order and their values, room for y_capacity
 *               entries (y_val may be NULL); y_nnz out: one int32 on the device, the full count
 *   Inputs are not modified.  Handles are not involved.  m must be at least 1 (m = 0 and
 *   negative sizes return DBSPMSPV_ERR_INVALID_ARG).
 *
 * Scratch: one counter per 8192 rows, kept in a fixed 16 KB __device__ array inside the
 * library (every GPU that loads the library holds it until the process exits).  Hence
 *   - m may be at most 33,554,432 rows; larger m returns DBSPMSPV_ERR_TOO_LARGE and does nothing;
 *   - the array is shared by every call and keeps the previous call's contents; each call
 *     overwrites every counter it will read before reading it, so nothing has to be cleared;
 *   - two calls whose kernels overlap on the GPU (different streams, or threads) race on it:
 *     serialise calls to this entry point on one device;
 *   - the first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress) and keeps it for the life of the process; make that first call
 *     before any stream capture begins, and do not reset the device while the library is in use.
 * It calls no cudaMalloc / cudaFree or other allocating routine, enqueues two kernels on
 * `stream` and returns without synchronising.
 */
int dbspmspv_compact_noalloc(const float *acc, const uint32_t *hit_bitmap, int64_t m,
                             int32_t *y_idx, float *y_val, int64_t y_capacity, int32_t *y_nnz,
                             dbspmspv_stream_t stream);

/* Measurement aid (untimed; allocates and synchronises): the bytes of the format that ONE call
 * with this x would read on the given path (DBSPMSPV_PATH_PUSH or _PULL), counted by walking
 * the format as built -- the check of the benchmark's host-side byte model (Section 5.1 reports
 * time only; achieved bandwidth needs a numerator).  x_idx: nnz_x device indices.
 *   push, hypersparse handle: the INLINE run of every listed column and the payload run of
 *     every nonempty vector block's column block, 8 bytes of pointers each;
 *   push, handle whose elements sit mostly in blocks with a payload: every entry of the column
 *     blocks of the nonempty vector blocks;
 *   pull: the whole block-CSR view (streaming pull: in whole chunks) and its tables;
 *   both: the payload of every visited block under a nonempty vector block.
 * x and y traffic is not included (it follows from nnz_x and y_nnz).                          */
typedef struct {
    int64_t view_entries;         /* view entries read                                         */
    int64_t view_bytes;           /* 9 bytes each (index word, value / offset word, byte)      */
    int64_t payload_blocks;       /* blocks whose payload is fetched                           */
    int64_t payload_bytes;
    int64_t pointer_bytes;        /* pointer words, chunk / segment tables, row list           */
    int64_t active_vector_blocks; /* nonempty vector blocks of x                               */
    int64_t reserved[2];
} dbspmspv_call_bytes;
int dbspmspv_count_call_bytes(dbspmspv_handle_t h, const int32_t *x_idx, int32_t nnz_x, int path,
                              dbspmspv_call_bytes *out);

/* Measurement aid: latency floors of the machine, enqueued on `stream`.  kind 0: an empty
 * kernel (launch + completion); kind 1: one thread follows `steps` dependent loads through
 * `chain` (device int32 array in which element i holds the index of the next element, e.g. one
 * long random cycle), starting at `start`, and stores where it ended in `out` (device).        */
int dbspmspv_probe_floor(int kind, const int32_t *chain, int32_t start, int32_t steps, int32_t *out,
                         dbspmspv_stream_t stream);

/* Test hook for the bounded device-side waits (Section 3.3.3's asynchronous staging completes
 * on barriers in shared memory, and every wait on them has an iteration limit): launches one
 * warp that waits on such a barrier with NO copy in flight, so the wait runs out after
 * `max_tries` tries (1 .. 4096, about 2 us each) and the kernel records DBSPMSPV_ERR_TIMEOUT,
 * which the next dbspmspv_get_stats returns.  The context stays usable.                       */
int dbspmspv_test_bounded_wait(dbspmspv_handle_t h, int32_t max_tries, dbspmspv_stream_t stream);

/* y<mask> = A x: dbspmspv_run with an output mask (the GraphBLAS form of the primitive; the
 * "strip the visited vertices" step of DB-BFS, Section 4.2, as an option of the call).
 * row_mask is a device bitmap over the rows, bit i of word i / 32 = row i, at least
 * ceil(ceil(m / 16) / 2) words (the last one padded with anything).  complement = 0: a row goes
 * to y iff its bit is set; complement = 1: iff its bit is clear (the mask then names what is
 * already known, e.g. a visited set).  y holds the structural result restricted to those rows,
 * ascending; y_nnz counts them.  The mask is applied where y is compacted: the traversal does
 * the same work as dbspmspv_run.  Everything else as dbspmspv_run.                             */
int dbspmspv_run_masked(dbspmspv_handle_t h, const int32_t *x_idx, const void *x_val, int32_t nnz_x,
                        int semiring, const uint32_t *row_mask, int complement, int32_t *y_idx, float *y_val,
                        int64_t y_capacity, int32_t *y_nnz, dbspmspv_stream_t stream);

/* Several activation vectors through one layer (multi-vector input: the extension the paper
 * leaves open in its limitations).  x holds `batch` dense vectors of n entries each, vector b
 * at x + b * ldx entries (the handle's value type; fp32 with run option decode_x_f32); y
 * receives `batch` dense fp32 vectors of m entries, vector b at y + b * ldy.  ldx >= n,
 * ldy >= m.  Every y vector equals what dbspmspv_decode gives for its x vector (up to the
 * order of the fp32 additions).  Where the handle has the streaming decode form, groups of up
 * to four vectors share one pass over the payload (the selector is not evaluated for them: the
 * payload is streamed whatever the vectors hold); otherwise the vectors are taken one by one.
 * The activation options (decode_threshold, decode_relu, decode_x_f32) apply to every vector.
 * Device pointers; allocates nothing; asynchronous on `stream`.  Pattern handles:
 * DBSPMSPV_ERR_UNSUPPORTED.                                                                   */
int dbspmspv_decode_batch(dbspmspv_handle_t h, const void *x, int64_t ldx, float *y, int64_t ldy, int32_t batch,
                          dbspmspv_stream_t stream);

/* Test hook of the range-checked build (-DDBS_BOUNDS_CHECK; any other build returns
 * DBSPMSPV_ERR_UNSUPPORTED and does nothing): overwrites the other-dimension block index of
 * block-CSR view entry `position` with `block_index` (27 bits), so that a test can show that a
 * kernel which meets the entry records DBSPMSPV_ERR_INTERNAL and skips it.  Synchronous.  The
 * handle is meant to be destroyed afterwards.                                                  */
int dbspmspv_test_corrupt_entry(dbspmspv_handle_t h, int32_t position, uint32_t block_index);

int dbspmspv_set_run_opts(dbspmspv_handle_t h, const dbspmspv_run_opts *opts);
int dbspmspv_destroy(dbspmspv_handle_t h);
const char *dbspmspv_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* DBSPMSPV_H */
