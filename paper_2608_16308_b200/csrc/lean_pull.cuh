// Streaming pull for hypersparse handles (Sections 3.3.2, 3.3.3): almost every stored element of
// such a matrix is an INLINE entry of the block-CSR view, and that view keeps the elements of a
// row adjacent, so y = A x is a segmented sum over one stream.
//
//   * The view is cut into chunks of LEAN_CHUNK consecutive entries, whatever row they belong to
//     (equal bytes per chunk: no weights, no segment table).  A lane reads its eight entries of
//     a chunk with 16-byte streaming loads, and the loads of the warp's NEXT chunk are issued
//     before the current one is worked on: the registers are the staging buffer (Section 3.3.3's
//     double buffering), which leaves the shared memory to the filter below and the rest of the
//     SM's on-chip memory to the L1 that serves the hot columns of a power-law matrix.
//   * One thread block per SM keeps the presence bitmap of x (the vector-block masks, one bit per
//     column) in shared memory and tests it before every gather: an absent x_j costs a
//     shared-memory load instead of a trip through the L1 tag stage, which is what bounds this
//     kernel (one 4-byte gather per stored element, one cache line each).
//   * A warp pass covers one chunk, eight CONSECUTIVE entries per lane.  A lane gathers the x
//     entries that pass the filter (one load each: the dense copy of x carries a "not listed"
//     marker), multiplies, and sums runs of equal row inside its eight entries in registers;
//     ROW_FLAG in the entry marks where a row starts.
//   * Across the lanes a segmented shuffle scan adds up the pieces of every row that spans
//     several lanes (Section 3.3.3: registers, then warp shuffle), and one lane per row adds the
//     sum to global memory -- a row cut by a pass or chunk boundary simply contributes one atomic
//     per piece.  The row a sum belongs to comes from the row list (lean_rows), indexed by the
//     running count of ROW_FLAGs; structural hits are tracked as bit masks beside the sums.
//   * The few entries with a payload are skipped by the stream and taken afterwards, one block
//     per warp at a time, from the list of their positions.
//   * The same kernel serves the (min, +) semiring (Out::MINPLUS): products become sums, sums
//     minima with identity +infinity, and the writeback keeps the smaller value (minplus.cuh).
#pragma once

#include "internal.cuh"
#include "microkernels.cuh"
#include "minplus.cuh"

namespace dbs {

#ifndef DBS_LEAN_WARPS
#define DBS_LEAN_WARPS 32
#endif
constexpr int LEAN_WARPS = DBS_LEAN_WARPS;     // warps per thread block; one thread block per SM
constexpr int LEAN_CTA = LEAN_WARPS * 32;
// Presence filter of x in shared memory: one bit per column (folded modulo the filter size when
// x has more columns than bits), tested before every gather.
constexpr int LEAN_FILTER_MAX_WORDS = 32768;   // 128 KB: exact up to 1,048,576 columns
#ifndef DBS_LEAN_FILTER
#define DBS_LEAN_FILTER 1
#endif
#ifndef DBS_LEAN_LDCA
#define DBS_LEAN_LDCA 1
#endif
// The x gathers go through L1: on a power-law matrix a few hundred columns draw a third of all
// gathers, and with L2-only loads those lines saturate single L2 slices.
__device__ __forceinline__ float lean_gather(const float *p) {
#if DBS_LEAN_LDCA
    return __ldg(p);
#else
    return __ldcg(p);
#endif
}

constexpr int LEAN_ROWS_CACHED = 64;
constexpr int LEAN_PER_LANE = LEAN_CHUNK / 32;
static_assert(LEAN_PER_LANE == 8, "a lane takes two 16-byte loads of view indices");

// A lane's eight consecutive entries of one chunk.
struct LeanRegs {
    uint4 i0, i1;      // view indices
    uint2 a;           // packed coordinates
    uint4 w0, w1;      // values
};
template <bool VAL>
__device__ __forceinline__ LeanRegs lean_fetch(const Device &d, int c, int lane) {
    // (always a whole chunk: the view arrays have that much slack behind the last entry, filled
    // with PAD_IDX entries; streaming loads: the bytes are never read again)
    const size_t e = (size_t)c * LEAN_CHUNK + (size_t)LEAN_PER_LANE * lane;
    LeanRegs r;
    r.i0 = __ldcs(reinterpret_cast<const uint4 *>(d.csr.idx + e));
    r.i1 = __ldcs(reinterpret_cast<const uint4 *>(d.csr.idx + e + 4));
    r.a = __ldcs(reinterpret_cast<const uint2 *>(d.csr.aux + e));
    r.w0 = r.w1 = make_uint4(0u, 0u, 0u, 0u);
    if (VAL) {
        r.w0 = __ldcs(reinterpret_cast<const uint4 *>(d.csr.w + e));
        r.w1 = __ldcs(reinterpret_cast<const uint4 *>(d.csr.w + e + 4));
    }
    return r;
}

template <int DT, typename Out>
__device__ __forceinline__ void lean_add(Out out, int row, float v) {
    if (Out::MINPLUS) {          // keep the smaller sum (an atomic whose reply nobody waits for)
        atomicMax(reinterpret_cast<uint32_t *>(out.acc) + row, minplus_key(v));
        out.hit8[row] = 1;
        return;
    }
    if (DT != DBSPMSPV_PATTERN) atomicAdd(out.acc + row, v);
    if (Out::MASKS) out.hit8[row] = 1;
}
// The semiring of the segmented reduction: (+, *) or, for Out::MINPLUS, (min, +).
template <typename Out> __device__ __forceinline__ float lean_identity() { return Out::MINPLUS ? __int_as_float(0x7F800000) : 0.f; }
template <typename Out> __device__ __forceinline__ float lean_mul(float a, float x) { return Out::MINPLUS ? a + x : a * x; }
template <typename Out> __device__ __forceinline__ float lean_sum(float s, float p) { return Out::MINPLUS ? fminf(s, p) : s + p; }

// One chunk = one warp pass, eight consecutive entries per lane, arranged so that the chunk costs
// one exposed memory latency: first what needs the entries only (the row-start bits and, from a
// ballot of them, how many rows start in the lanes below), then all dependent global loads at
// once (the x gathers and the slice of the row list the chunk adds to), then the sums.
// `ord` = ROW_FLAGs before the chunk (lean_rows[ord - 1] is the row that runs into it).
template <int DT, typename Out>
__device__ __forceinline__ void lean_chunk(const Device &d, Out out, const LeanRegs &r, const uint32_t *filter,
                                           uint32_t filter_mask, int *s_rows, int ord, int lane) {
    constexpr bool VAL = DT != DBSPMSPV_PATTERN;
    constexpr int K = LEAN_PER_LANE;
    const uint32_t lt = (1u << lane) - 1u;
    const uint32_t idx[K] = {r.i0.x, r.i0.y, r.i0.z, r.i0.w, r.i1.x, r.i1.y, r.i1.z, r.i1.w};
    const uint32_t wv[K] = {r.w0.x, r.w0.y, r.w0.z, r.w0.w, r.w1.x, r.w1.y, r.w1.z, r.w1.w};
    uint32_t hb = 0u;            // bit k: entry k starts a row
#pragma unroll
    for (int k = 0; k < K; ++k) hb |= ((idx[k] >> 27) & 1u) << k;
    const int cnt = __popc(hb);
    const uint32_t hm = __ballot_sync(FULL, hb != 0u);      // lanes in which a row starts
    const bool multi = __any_sync(FULL, cnt > 1);           // some lane holds several row starts
    int excl, total;                                         // row starts in the lanes below / in the chunk
    if (multi) {
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(FULL, incl, o);
            if (lane >= o) incl += t;
        }
        excl = incl - cnt;
        total = __shfl_sync(FULL, incl, 31);
    } else {
        excl = __popc(hm & lt);
        total = __popc(hm);
    }
    // ---- dependent global loads: the rows this chunk adds to (lean_rows[ord - 1 .. ord + total - 1]:
    // a lane fetches numbers l and 32 + l of them, they go to shared memory where any lane can
    // look its rows up; a chunk of rows of one to three entries has more than 64 and reads the
    // rest from the list directly), and the x entries
    int rowp0 = 0, rowp1 = 0;
    {
        const int o = ord - 1 + lane;
        if (lane <= total && o >= 0 && o < d.n_lean_rows) rowp0 = __ldg(d.lean_rows + o);
        if (lane + 32 <= total && o + 32 < d.n_lean_rows) rowp1 = __ldg(d.lean_rows + o + 32);
    }
    // row of the chunk's row start number k (k = 0: the row that runs into the chunk)
    auto row_of = [&](int k) { return k < LEAN_ROWS_CACHED ? s_rows[k] : d.lean_rows[ord - 1 + k]; };
    float xin[K];
#pragma unroll
    for (int k = 0; k < K; ++k) {
        // INLINE is class 0: any other entry (a block with a payload, the slack) is skipped here
        bool go = idx[k] < (1u << TYPE_SHIFT) && DBS_CHK_INDEX(d, idx[k] & IDX_MASK, d.nb);
        const uint32_t a = k < 4 ? r.a.x : r.a.y;
        const uint32_t col = (idx[k] & IDX_MASK) * 16u + ((a >> (8 * (k & 3))) & 15u);
#if DBS_LEAN_FILTER
        // (a set filter bit may belong to another column when the filter is folded: the gather
        // then returns the "not listed" marker, as it would without the filter)
        go = go && ((filter[(col >> 5) & filter_mask] >> (col & 31u)) & 1u);
#endif
        xin[k] = go ? lean_gather(d.ws.x_dense + col) : __uint_as_float(X_ABSENT);
    }
    __syncwarp();                // (the previous chunk's look-ups are over)
    s_rows[lane] = rowp0;
    s_rows[lane + 32] = rowp1;
    __syncwarp();
    // ---- sums.  Thread-serial part: `lead` = sum of the lane's entries before its first row
    // start (they belong to the row that was open when the lane began), `seg` = sum from its last
    // row start on; rows that lie wholly inside the lane are added to global memory by the lane.
    const float ID = lean_identity<Out>();
    float lead = ID, seg = ID;
    uint32_t lead_hit = 0u, seg_hit = 0u;
    if (!multi) {
        // at most one row start per lane (the usual case): entries below it, entries from it on
        const int f = hb ? __ffs(hb) - 1 : K;
        uint32_t pb = 0u;
#pragma unroll
        for (int k = 0; k < K; ++k) {
            if (__float_as_uint(xin[k]) != X_ABSENT) {
                pb |= 1u << k;
                if (VAL) {
                    const float p = lean_mul<Out>(Val<DT>::inline_value(wv[k]), xin[k]);
                    if (k < f) lead = lean_sum<Out>(lead, p); else seg = lean_sum<Out>(seg, p);
                }
            }
        }
        const uint32_t below = (1u << f) - 1u;
        lead_hit = pb & below;
        seg_hit = pb & ~below;
    } else {
        int nh = 0;
#pragma unroll
        for (int k = 0; k < K; ++k) {
            if ((hb >> k) & 1u) {
                if (nh == 0) { lead = seg; lead_hit = seg_hit; }
                else if (seg_hit) lean_add<DT>(out, row_of(excl + nh), seg);   // a whole row inside the lane
                ++nh;
                seg = ID; seg_hit = 0u;
            }
            if (__float_as_uint(xin[k]) != X_ABSENT) {
                if (VAL) seg = lean_sum<Out>(seg, lean_mul<Out>(Val<DT>::inline_value(wv[k]), xin[k]));
                seg_hit = 1u;
            }
        }
        if (nh == 0) { lead = seg; lead_hit = seg_hit; seg = ID; seg_hit = 0u; }
    }
    // Warp part.  A lane with a row start closes the row that was open before it.  S = inclusive
    // sum of `lead` over the lanes since the last lane with a row start (exclusive): at a lane with
    // a row start, or at lane 31, S is the whole tail of the row that started before.
    const uint32_t lh = __ballot_sync(FULL, lead_hit != 0u);
    float S = lead;
    if (VAL) {
        const int reach = lane - (32 - __clz(hm & lt));       // lanes to my left in my run
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(FULL, S, o);
            if (reach >= o) S = lean_sum<Out>(S, t);
        }
    }
    // (a) the row that runs into the chunk: closed by the first lane with a row start (lane 31 if none)
    const int wl = hm ? __ffs(hm) - 1 : 31;
    if (lane == wl && (lh & ((2u << wl) - 1u))) lean_add<DT>(out, row_of(0), S);
    // (b) the row that starts at a lane's last row start: its piece here, plus the leads of the
    // lanes up to and including the next lane with a row start (or lane 31)
    const uint32_t above = hm & ~lt & ~(1u << lane);
    const int nx = above ? __ffs(above) - 1 : 31;
    float tail = ID;
    if (VAL) { tail = __shfl_sync(FULL, S, nx); if (lane == 31) tail = ID; }
    if (cnt) {
        const uint32_t tail_hit = ((lh >> 1) >> lane) & ((1u << (nx - lane)) - 1u);
        if (seg_hit | tail_hit) lean_add<DT>(out, row_of(excl + cnt), lean_sum<Out>(seg, tail));
    }
}

struct LeanScratch {        // per warp
    int rows[LEAN_ROWS_CACHED];   // the slice of the row list the current chunk adds to
    float sx[16];                 // the microkernels of the entries with a payload
    float stmp[32];
};

template <int DT, typename Out>
__global__ void __launch_bounds__(LEAN_CTA, 1)
k_pull_lean(Device d, Out out, float th3, int force_path, int popc_threshold, int filter_words) {
    extern __shared__ __align__(128) uint8_t s_lean[];
    constexpr bool VAL = DT != DBSPMSPV_PATTERN;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t *filter = reinterpret_cast<uint32_t *>(s_lean);
    LeanScratch *ls = reinterpret_cast<LeanScratch *>(s_lean + (size_t)filter_words * 4) + warp;
    pdl_wait();
    pdl_launch_dependents();
    if (select_path(d, th3, force_path) != DBSPMSPV_PATH_PULL) return;
    if (blockIdx.x == 0 && threadIdx.x == 0) d.ws.ctr->path = DBSPMSPV_PATH_PULL;
    const int gwarp = blockIdx.x * LEAN_WARPS + warp;
    const int nwarps = gridDim.x * LEAN_WARPS;
    LeanRegs nxt = {};
    int ord_next = 0;
    if (gwarp < d.n_lean_chunks) { nxt = lean_fetch<VAL>(d, gwarp, lane); ord_next = d.lean_chunk_ord[gwarp]; }
    // the filter: the vector-block masks are the presence bitmap of x (bit j of the array = column
    // j); folded by OR when x has more columns than the filter has bits
    {
        const int n_words = (d.nb + 1) / 2;
        for (int f = threadIdx.x; f < filter_words; f += LEAN_CTA) {
            uint32_t v = 0u;
            for (int q = f; q < n_words; q += filter_words) v |= d.ws.x_mask32[q];
            filter[f] = v;
        }
    }
    __syncthreads();
    const uint32_t filter_mask = (uint32_t)filter_words - 1u;
    for (int c = gwarp; c < d.n_lean_chunks; c += nwarps) {
        const LeanRegs cur = nxt;
        const int ord = ord_next;
        if (c + nwarps < d.n_lean_chunks) { nxt = lean_fetch<VAL>(d, c + nwarps, lane); ord_next = d.lean_chunk_ord[c + nwarps]; }
        lean_chunk<DT, Out>(d, out, cur, filter, filter_mask, ls->rows, ord, lane);
    }
    // entries with a payload: one block per warp at a time (they are the exception in these handles)
    for (int q = gwarp; q < d.n_payload; q += nwarps) {
        const int pos = d.payload_pos[q];
        if (!DBS_CHK_INDEX(d, pos, d.n_entries)) continue;            // warp-uniform
        uint32_t idx = d.csr.idx[pos];
#ifdef DBS_BOUNDS_CHECK
        {
            uint32_t w_ = d.csr.w[pos], a_ = d.csr.aux[pos];
            DBS_CHK_ENTRY(d, true, idx, w_, a_);
            if ((idx >> TYPE_SHIFT) == DBSPMSPV_BLK_INLINE || !DBS_CHK_INDEX(d, d.entry_row[pos], d.mb)) continue;   // (only a replaced entry is INLINE here)
        }
#endif
        const int cb = idx & IDX_MASK, type = idx >> TYPE_SHIFT;
        const uint32_t xm = mask_of(d.ws.x_mask32, cb);
        if (!xm) continue;                                            // warp-uniform
        const uint8_t *blk = d.payload + (size_t)d.csr.w[pos] * 4;
        const int nnz = (int)d.csr.aux[pos] + 1;
        const int rb = d.entry_row[pos];
        if (Out::MINPLUS) {
            block_rows_min_warp<DT>(type, d.csr.w[pos], d.csr.aux[pos], xm, d.ws.x_dense + (size_t)cb * 16, d.payload, lane, [&](int r, uint32_t key) {
                atomicMax(reinterpret_cast<uint32_t *>(out.acc) + (size_t)rb * 16 + r, key);
                out.hit8[(size_t)rb * 16 + r] = 1;
            });
            continue;
        }
        uint32_t hits;
        float sum = 0.f;
        if (DT == DBSPMSPV_PATTERN) {
            hits = warp_block_bool<DT>(type, blk, nnz, xm, lane);
        } else {
            __syncwarp();
            if (lane < 16) ls->sx[lane] = d.ws.x_dense[(size_t)cb * 16 + lane];
            __syncwarp();
            sum = warp_block<DT>(type, blk, nnz, xm, ls->sx, ls->stmp, lane, popc_threshold, hits);
        }
        if (lane < 16 && ((hits >> lane) & 1u)) {
            if (DT != DBSPMSPV_PATTERN) atomicAdd(out.acc + (size_t)rb * 16 + lane, sum);
            if (Out::MASKS) out.hit8[(size_t)rb * 16 + lane] = 1;
        }
    }
}

}  // namespace dbs
