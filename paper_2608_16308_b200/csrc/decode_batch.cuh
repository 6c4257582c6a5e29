// Batched streaming decode (the paper names the single vector as its limit, Section 6: "multi-
// vector" inputs): NB activation vectors share ONE pass over the payload.  Same structure as
// k_decode_stream -- persistent grid, the chunk list split evenly over all warps, per-warp
// two-stage rings fed by bulk copies, row sums in registers until the row block changes -- with
//   * NB staged copies of x (masks + fp32 blocks) in shared memory and the OR of the masks,
//     which decides what columns of a block are walked at all;
//   * NB x 16 row sums per lane: a stored value is loaded once and multiplied by the x entry
//     of every vector that has one in that column.
// The selector is not evaluated: the payload is streamed whatever the vectors hold (a batch
// whose union fills few vector blocks is the caller's to split into dbspmspv_decode calls).
// Included by run.cu after the single-vector kernels it shares its helpers with.
#pragma once

namespace dbs {

constexpr int BATCH_WARPS = 8;
constexpr int BATCH_CTA = BATCH_WARPS * 32;

struct BatchLayout {
    int x_stride, xm_off, um_off, cnt_off, bar_off, ring_off, total;
    __host__ __device__ BatchLayout(int nb, int nvec, int stage_bytes) {
        x_stride = nb * 16;                                   // floats per staged vector
        xm_off = nvec * nb * 64;
        um_off = (xm_off + nvec * nb * 2 + 15) & ~15;
        cnt_off = (um_off + nb * 2 + 15) & ~15;
        bar_off = (cnt_off + 16 * 4 + 15) & ~15;
        ring_off = (bar_off + BATCH_WARPS * STREAM_DEPTH * 8 + 127) & ~127;
        total = ring_off + BATCH_WARPS * STREAM_DEPTH * stream_stride(stage_bytes);
    }
};

// (block, active column) pairs of one warp step dealt out evenly over the lanes, as in
// warp_columns; `cols` = the lane's block's columns that some vector reaches.
template <int DT, int NB>
__device__ __forceinline__ void warp_columns_batch(const uint8_t *payload, const float *s_x, int x_stride, uint32_t idx,
                                                   uint32_t w, uint32_t cols, int lane, float (&acc)[NB][16]) {
    int incl = __popc(cols);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(FULL, incl, o);
        if (lane >= o) incl += t;
    }
    const int excl = incl - __popc(cols);
    const int total = __shfl_sync(FULL, incl, 31);
    for (int k0 = 0; k0 < total; k0 += 32) {
        const int k = k0 + lane;
        int b = 0;                       // owner of pair k: the last lane whose exclusive prefix is <= k
#pragma unroll
        for (int s = 16; s; s >>= 1) {
            const int t = __shfl_sync(FULL, excl, b + s);
            if (t <= k) b += s;
        }
        uint32_t mm = __shfl_sync(FULL, cols, b);
        const int j = k - __shfl_sync(FULL, excl, b);
        const uint32_t bidx = __shfl_sync(FULL, idx, b), bw = __shfl_sync(FULL, w, b);
        if (k >= total) continue;
        for (int t = 0; t < j; ++t) mm &= mm - 1;
        const int c = __ffs(mm) - 1;     // the j-th active column of that block
        const bool dense = (bidx >> TYPE_SHIFT) == DBSPMSPV_BLK_DENSE;
        const uint8_t *blk = payload + (size_t)bw * 4;
        float xv[NB];
        bool on[NB];
#pragma unroll
        for (int v = 0; v < NB; ++v) {
            xv[v] = s_x[(size_t)v * x_stride + (size_t)(bidx & IDX_MASK) * 16 + c];
            on[v] = __float_as_uint(xv[v]) != X_ABSENT;
        }
        // (Dense blocks carry their column masks too: absent elements are stored as zeros and
        // must not meet a non-finite x)
        const uint32_t gate = reinterpret_cast<const uint16_t *>(blk)[c];
        const uint8_t *vals = blk + (dense ? 32 : HDR_BYTES);
        int i = dense ? c * 16 : blk[32 + c];
#pragma unroll
        for (int r = 0; r < 16; ++r) {
            const uint32_t bit = (gate >> r) & 1u;
            if (bit) {
                const float a = Val<DT>::load(vals, i);
#pragma unroll
                for (int v = 0; v < NB; ++v)
                    if (on[v]) acc[v][r] += a * xv[v];
            }
            i += (int)bit | (dense ? 1 : 0);
        }
    }
}

template <int DT, int NB>
__global__ void __launch_bounds__(BATCH_CTA, 1)
k_decode_stream_batch(Device d, const void *__restrict__ x, int64_t ldx, float *__restrict__ y, int64_t ldy, int nvec,
                      int only_as_fallback) {
    extern __shared__ __align__(128) uint8_t s_dyn[];
    // launched behind the tensor-core kernel: it runs only if that one met a non-finite x entry
    // and left the vectors to this kernel (a flag in the handle's counters)
    if (only_as_fallback) {
        pdl_wait();
        if (d.ws.ctr->batch_fallback == 0) return;
    }
    constexpr int T = BATCH_CTA, NW = BATCH_WARPS;
    const BatchLayout lay(d.nb, NB, d.stage_bytes);
    float *s_x = reinterpret_cast<float *>(s_dyn);
    uint16_t *s_xm = reinterpret_cast<uint16_t *>(s_dyn + lay.xm_off);
    uint16_t *s_um = reinterpret_cast<uint16_t *>(s_dyn + lay.um_off);
    int *s_cnt = reinterpret_cast<int *>(s_dyn + lay.cnt_off);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int stride = stream_stride(d.stage_bytes);
    uint64_t *s_bar = reinterpret_cast<uint64_t *>(s_dyn + lay.bar_off) + warp * STREAM_DEPTH;
    uint8_t *s_ring = s_dyn + lay.ring_off + (size_t)warp * STREAM_DEPTH * stride;
    if (tid < 16) s_cnt[tid] = 0;

    const int gw = blockIdx.x * NW + warp, W = gridDim.x * NW;
    const int lo = (int)((int64_t)d.n_stage_chunks * gw / W), hi = (int)((int64_t)d.n_stage_chunks * (gw + 1) / W);
    const int n_mine = hi - lo;
    int4 my_desc = make_int4(0, 0, 0, 0);
    if (lane < n_mine) my_desc = d.stage_chunks[lo + lane];
    auto desc_of = [&](int k) {
        return make_int4(__shfl_sync(FULL, my_desc.x, k & 31), __shfl_sync(FULL, my_desc.y, k & 31),
                         __shfl_sync(FULL, my_desc.z, k & 31), __shfl_sync(FULL, my_desc.w, k & 31));
    };
    auto issue = [&](const int4 &ch, int st) {               // lane 0 only
        uint8_t *base = s_ring + (size_t)st * stride;
        uint32_t pb = ((uint32_t)ch.w & 0xFFFFFFu) * 4u;
        if (!DBS_CHK_INDEX(d, pb, d.stage_bytes + 1) || !DBS_CHK_INDEX(d, (uint64_t)(uint32_t)ch.z + (pb >> 2), (uint64_t)d.payload_words + 1)) pb = 0u;
        fence_proxy_async_smem();
        mbar_arrive_expect_tx(&s_bar[st], pb);
        if (pb) bulk_copy_g2s(base, d.payload + (size_t)(uint32_t)ch.z * 4, pb, &s_bar[st]);
    };
    auto entries_of = [&](const int4 &ch, uint32_t &idx, uint32_t &w, uint32_t &aux) {
        idx = 0; w = 0; aux = 0;
        if (lane < (int)((uint32_t)ch.w >> 24) && DBS_CHK_RANGE(d, ch.x, (uint32_t)ch.w >> 24)) {
            const int p_ = ch.x + lane; idx = d.csr.idx[p_]; w = d.csr.w[p_]; aux = d.csr.aux[p_];
            DBS_CHK_ENTRY(d, true, idx, w, aux);
            if ((idx >> TYPE_SHIFT) != DBSPMSPV_BLK_INLINE && !DBS_CHK_INDEX(d, (int64_t)w - (uint32_t)ch.z, (uint32_t)ch.w & 0xFFFFFFu)) { idx = 0u; w = 0u; aux = 0u; }
        }
    };
    int issued = 0;
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < STREAM_DEPTH; ++k) mbar_init(&s_bar[k], 1);
        fence_barrier_init();
    }
    __syncwarp();
    for (; issued < STREAM_DEPTH - 1 && issued < n_mine; ++issued) {
        const int4 ch = desc_of(issued);
        if (lane == 0) issue(ch, issued);
    }
    __syncthreads();
    // the vectors -> masks and fp32 blocks; vectors past nvec are empty
    const size_t esize = (DT == DBSPMSPV_BF16 && !d.decode_x_f32) ? 2 : 4;
#pragma unroll
    for (int v = 0; v < NB; ++v) {
        if (v < nvec) {
            stage_x_blocks<DT>(d, static_cast<const uint8_t *>(x) + (size_t)v * (size_t)ldx * esize, s_x + (size_t)v * lay.x_stride,
                               s_xm + (size_t)v * d.nb, s_cnt + 2 * v, tid, T);
        } else {
            for (int cb = tid; cb < d.nb; cb += T) {
                s_xm[(size_t)v * d.nb + cb] = 0;
                for (int k = 0; k < 16; ++k) s_x[(size_t)v * lay.x_stride + cb * 16 + k] = __uint_as_float(X_ABSENT);
            }
        }
    }
    __syncthreads();
    int nz_union = 0;
    for (int cb = tid; cb < d.nb; cb += T) {
        uint32_t u = 0;
#pragma unroll
        for (int v = 0; v < NB; ++v) u |= s_xm[(size_t)v * d.nb + cb];
        s_um[cb] = (uint16_t)u;
        nz_union += u != 0;
    }
    nz_union = __reduce_add_sync(FULL, nz_union);
    if (lane == 0 && nz_union) atomicAdd(&s_cnt[15], nz_union);
    __syncthreads();
    if (blockIdx.x == 0 && tid == 0) {
        Counters *c = d.ws.ctr;
        c->last_n_nzblk = s_cnt[15]; c->last_n_tasks = 0; c->last_path = DBSPMSPV_PATH_PULL; c->last_y_nnz = (int32_t)d.m;
    }
    // y is zeroed by the kernel in front, which this one may overlap up to here
    pdl_wait();

    float acc[NB][16];
#pragma unroll
    for (int v = 0; v < NB; ++v)
#pragma unroll
        for (int r = 0; r < 16; ++r) acc[v][r] = 0.f;
    int cur_rb = -1;
    auto flush = [&]() {
        if (cur_rb >= 0) {
#pragma unroll
            for (int v = 0; v < NB; ++v) {
                const float total = fold_rows(acc[v], lane);
                if (!(lane & 1) && total != 0.f) atomicAdd(y + (size_t)v * ldy + (size_t)cur_rb * 16 + folded_row(lane), total);
#pragma unroll
                for (int r = 0; r < 16; ++r) acc[v][r] = 0.f;
            }
        }
    };
    auto step = [&](const uint8_t *payload, uint32_t idx, uint32_t w, uint32_t aux, bool have) {
        const uint32_t um = have ? s_um[idx & IDX_MASK] : 0u;
        const int type = idx >> TYPE_SHIFT;
        const bool mk = have && um && type > DBSPMSPV_BLK_COO;
        const bool rowm = mk && is_row_major(type);
        warp_columns_batch<DT, NB>(payload, s_x, lay.x_stride, idx, w, mk && !rowm ? um : 0u, lane, acc);
        __syncwarp();
        // the other classes (rare in these handles): vector by vector, as the single-vector kernel does
        if (__any_sync(FULL, rowm || (have && um && type <= DBSPMSPV_BLK_COO))) {
#pragma unroll 1
            for (int v = 0; v < NB; ++v) {
                const float *sxv = s_x + (size_t)v * lay.x_stride;
                float *yv = y + (size_t)v * ldy;
                const uint32_t xm = have ? s_xm[(size_t)v * d.nb + (idx & IDX_MASK)] : 0u;
                auto emit = [&](int erb, int erow, float esum) { atomicAdd(yv + (size_t)erb * 16 + erow, esum); };
                const uint32_t rows = __ballot_sync(FULL, rowm && xm);
                if (rows) half_stream<DT, true>(payload, sxv, idx, w, xm, cur_rb, rows, lane, emit);
                if (have && xm && type <= DBSPMSPV_BLK_COO) {
                    const float *xb = sxv + (size_t)(idx & IDX_MASK) * 16;
                    float *row0 = yv + (size_t)cur_rb * 16;
                    if (type == DBSPMSPV_BLK_INLINE) {
                        if ((xm >> (aux & 15)) & 1u) atomicAdd(row0 + (aux >> 4), Val<DT>::inline_value(w) * xb[aux & 15]);
                    } else {
                        const int nnz = (int)aux + 1;
                        const uint8_t *blk = payload + (size_t)w * 4, *vals = blk + ((nnz + 3) & ~3);
                        for (int k = 0; k < nnz; ++k) {
                            const int c = blk[k] & 15, r = blk[k] >> 4;
                            if ((xm >> c) & 1u) atomicAdd(row0 + r, Val<DT>::load(vals, k) * xb[c]);
                        }
                    }
                }
            }
        }
    };

    bool timed_out = false;
    uint32_t idx = 0, w = 0, aux = 0, n_idx, n_w, n_aux;
    if (n_mine > 0) entries_of(desc_of(0), idx, w, aux);
    for (int k = 0; k < n_mine; ++k) {
        for (const int lim = min(n_mine, min(k + STREAM_DEPTH, (k & ~31) + 32)); issued < lim; ++issued) {
            const int4 nch = desc_of(issued);
            if (lane == 0) issue(nch, issued % STREAM_DEPTH);
        }
        const int st = k % STREAM_DEPTH;
        const int4 ch = desc_of(k);
        n_idx = 0; n_w = 0; n_aux = 0;
        if (k + 1 < n_mine && ((k + 1) & 31)) entries_of(desc_of(k + 1), n_idx, n_w, n_aux);
        if (!mbar_wait_bounded(&s_bar[st], (uint32_t)(k / STREAM_DEPTH) & 1u)) { timed_out = true; break; }
        if (ch.y != cur_rb) { flush(); cur_rb = DBS_CHK_INDEX(d, ch.y, d.mb) ? ch.y : 0; }
        const uint8_t *base = s_ring + (size_t)st * stride;
        step(base - (size_t)(uint32_t)ch.z * 4, idx, w, aux, lane < (int)((uint32_t)ch.w >> 24));
        __syncwarp();
        idx = n_idx; w = n_w; aux = n_aux;
        if (k + 1 < n_mine && !((k + 1) & 31)) {
            my_desc = make_int4(0, 0, 0, 0);
            if (k + 1 + lane < n_mine) my_desc = d.stage_chunks[lo + k + 1 + lane];
            entries_of(desc_of(k + 1), idx, w, aux);
        }
    }
    flush();
    if (timed_out) { d.ws.ctr->status = DBSPMSPV_ERR_TIMEOUT; return; }
    // the INLINE elements of the row blocks (row by row, rare in these handles)
    for (int rb = gw; rb < d.mb && d.has_inline; rb += W) {
        const int b0 = d.csr_inl[rb], b1 = d.csr.ptr[rb + 1];
        cur_rb = rb;
        for (int base = b0; base < b1; base += 32) {
            uint32_t e_idx = 0, e_w = 0, e_aux = 0;
            const bool have = base + lane < b1;
            if (have && DBS_CHK_INDEX(d, base + lane, d.n_entries)) {
                e_idx = d.csr.idx[base + lane]; e_w = d.csr.w[base + lane]; e_aux = d.csr.aux[base + lane];
                DBS_CHK_ENTRY(d, true, e_idx, e_w, e_aux);
            }
            step(d.payload, e_idx, e_w, e_aux, have);
        }
        if (b1 > b0) flush();
    }
}

// ---- bf16 handles: the same pass with the block products on the tensor cores (mma_block.cuh):
// up to eight vectors are the rows of one MMA operand, so a block costs the same whatever the
// vectors hold and however many they are.  12 warps per thread block; x is staged as bf16 only
// (zeros where an entry does not take part) plus the masks.  A non-finite x entry cannot be a
// zero-padded operand (0 * inf): the kernel then sets Counters::batch_fallback and leaves the
// vectors to k_decode_stream_batch, which is launched behind it.
constexpr int BATCH_MMA_WARPS = 12;
constexpr int BATCH_MMA_CTA = BATCH_MMA_WARPS * 32;

struct BatchMmaLayout {
    int ldh, xm_off, um_off, cnt_off, tile_off, bar_off, ring_off, total;
    __host__ __device__ BatchMmaLayout(int nb, int nvec, int stage_bytes) {
        ldh = nb * 16;                                        // bf16 entries per staged vector (first in the buffer)
        xm_off = nvec * nb * 32;
        um_off = (xm_off + nvec * nb * 2 + 15) & ~15;
        cnt_off = (um_off + nb * 2 + 15) & ~15;
        tile_off = (cnt_off + 16 + 127) & ~127;               // two expanded blocks per warp
        bar_off = tile_off + BATCH_MMA_WARPS * 1024;
        ring_off = (bar_off + BATCH_MMA_WARPS * STREAM_DEPTH * 8 + 127) & ~127;
        total = ring_off + BATCH_MMA_WARPS * STREAM_DEPTH * stream_stride(stage_bytes);
    }
};

template <int NB>
__global__ void __launch_bounds__(BATCH_MMA_CTA, 1)
k_decode_batch_mma(Device d, const void *__restrict__ x, int64_t ldx, float *__restrict__ y, int64_t ldy, int nvec) {
    extern __shared__ __align__(128) uint8_t s_dyn[];
    constexpr int T = BATCH_MMA_CTA, NW = BATCH_MMA_WARPS;
    const BatchMmaLayout lay(d.nb, NB, d.stage_bytes);
    uint16_t *s_xh = reinterpret_cast<uint16_t *>(s_dyn);
    uint16_t *s_xm = reinterpret_cast<uint16_t *>(s_dyn + lay.xm_off);
    uint16_t *s_um = reinterpret_cast<uint16_t *>(s_dyn + lay.um_off);
    int *s_cnt = reinterpret_cast<int *>(s_dyn + lay.cnt_off);     // [0] nonzero vector blocks of the union, [1] non-finite entry seen
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint16_t *s_tile = reinterpret_cast<uint16_t *>(s_dyn + lay.tile_off) + warp * 512;
    const int stride = stream_stride(d.stage_bytes);
    uint64_t *s_bar = reinterpret_cast<uint64_t *>(s_dyn + lay.bar_off) + warp * STREAM_DEPTH;
    uint8_t *s_ring = s_dyn + lay.ring_off + (size_t)warp * STREAM_DEPTH * stride;
    if (tid < 4) s_cnt[tid] = 0;

    const int gw = blockIdx.x * NW + warp, W = gridDim.x * NW;
    const int lo = (int)((int64_t)d.n_stage_chunks * gw / W), hi = (int)((int64_t)d.n_stage_chunks * (gw + 1) / W);
    const int n_mine = hi - lo;
    int4 my_desc = make_int4(0, 0, 0, 0);
    if (lane < n_mine) my_desc = d.stage_chunks[lo + lane];
    auto desc_of = [&](int k) {
        return make_int4(__shfl_sync(FULL, my_desc.x, k & 31), __shfl_sync(FULL, my_desc.y, k & 31),
                         __shfl_sync(FULL, my_desc.z, k & 31), __shfl_sync(FULL, my_desc.w, k & 31));
    };
    auto issue = [&](const int4 &ch, int st) {               // lane 0 only
        uint8_t *base = s_ring + (size_t)st * stride;
        uint32_t pb = ((uint32_t)ch.w & 0xFFFFFFu) * 4u;
        if (!DBS_CHK_INDEX(d, pb, d.stage_bytes + 1) || !DBS_CHK_INDEX(d, (uint64_t)(uint32_t)ch.z + (pb >> 2), (uint64_t)d.payload_words + 1)) pb = 0u;
        fence_proxy_async_smem();
        mbar_arrive_expect_tx(&s_bar[st], pb);
        if (pb) bulk_copy_g2s(base, d.payload + (size_t)(uint32_t)ch.z * 4, pb, &s_bar[st]);
    };
    auto entries_of = [&](const int4 &ch, uint32_t &idx, uint32_t &w, uint32_t &aux) {
        idx = 0; w = 0; aux = 0;
        if (lane < (int)((uint32_t)ch.w >> 24) && DBS_CHK_RANGE(d, ch.x, (uint32_t)ch.w >> 24)) {
            const int p_ = ch.x + lane; idx = d.csr.idx[p_]; w = d.csr.w[p_]; aux = d.csr.aux[p_];
            DBS_CHK_ENTRY(d, true, idx, w, aux);
            if ((idx >> TYPE_SHIFT) != DBSPMSPV_BLK_INLINE && !DBS_CHK_INDEX(d, (int64_t)w - (uint32_t)ch.z, (uint32_t)ch.w & 0xFFFFFFu)) { idx = 0u; w = 0u; aux = 0u; }
        }
    };
    int issued = 0;
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < STREAM_DEPTH; ++k) mbar_init(&s_bar[k], 1);
        fence_barrier_init();
    }
    __syncwarp();
    for (; issued < STREAM_DEPTH - 1 && issued < n_mine; ++issued) {
        const int4 ch = desc_of(issued);
        if (lane == 0) issue(ch, issued);
    }
    __syncthreads();
    // the vectors -> bf16 copies (zeros where an entry does not take part), masks, their union
    {
        int nz_union = 0;
        bool bad = false;
        for (int cb = tid; cb < d.nb; cb += T) {
            uint32_t um = 0;
#pragma unroll 2
            for (int v = 0; v < NB; ++v) {
                uint32_t bits = 0;
                uint16_t hv[16];
#pragma unroll
                for (int k = 0; k < 16; ++k) hv[k] = 0;
                if (v < nvec) {
                    const int64_t j0 = (int64_t)cb * 16;
                    float fv[16];
                    const uint16_t *xh_g = static_cast<const uint16_t *>(x) + (size_t)v * ldx + j0;
                    if (!d.decode_x_f32 && j0 + 16 <= d.n && (reinterpret_cast<uintptr_t>(xh_g) & 15u) == 0) {
                        // sixteen bf16 entries with two 16-byte loads
                        const uint4 a = reinterpret_cast<const uint4 *>(xh_g)[0], b = reinterpret_cast<const uint4 *>(xh_g)[1];
                        const uint32_t u[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
                        for (int q = 0; q < 8; ++q) { fv[2 * q] = __uint_as_float(u[q] << 16); fv[2 * q + 1] = __uint_as_float(u[q] & 0xFFFF0000u); }
                    } else {
#pragma unroll
                        for (int k = 0; k < 16; ++k) {
                            fv[k] = 0.f;
                            if (j0 + k < d.n) {
                                if (d.decode_x_f32) fv[k] = __bfloat162float(__float2bfloat16_rn(static_cast<const float *>(x)[(size_t)v * ldx + j0 + k]));
                                else fv[k] = __uint_as_float((uint32_t)xh_g[k] << 16);
                            }
                        }
                    }
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        const float f = fv[k];
                        if (decode_takes_part(d, f)) {
                            bits |= 1u << k;
                            hv[k] = (uint16_t)(__float_as_uint(f) >> 16);
                            bad |= (__float_as_uint(f) & 0x7F800000u) == 0x7F800000u;
                        }
                    }
                }
                uint4 *dst = reinterpret_cast<uint4 *>(s_xh + (size_t)v * lay.ldh + (size_t)cb * 16);
                dst[0] = make_uint4(hv[0] | (uint32_t)hv[1] << 16, hv[2] | (uint32_t)hv[3] << 16, hv[4] | (uint32_t)hv[5] << 16, hv[6] | (uint32_t)hv[7] << 16);
                dst[1] = make_uint4(hv[8] | (uint32_t)hv[9] << 16, hv[10] | (uint32_t)hv[11] << 16, hv[12] | (uint32_t)hv[13] << 16, hv[14] | (uint32_t)hv[15] << 16);
                s_xm[(size_t)v * d.nb + cb] = (uint16_t)bits;
                um |= bits;
            }
            s_um[cb] = (uint16_t)um;
            nz_union += um != 0;
        }
        nz_union = __reduce_add_sync(FULL, nz_union);
        if (lane == 0 && nz_union) atomicAdd(&s_cnt[0], nz_union);
        if (bad) s_cnt[1] = 1;
    }
    __syncthreads();
    const bool fallback = s_cnt[1] != 0;
    if (blockIdx.x == 0 && tid == 0) {
        Counters *c = d.ws.ctr;
        c->last_n_nzblk = s_cnt[0]; c->last_n_tasks = 0; c->last_path = DBSPMSPV_PATH_PULL; c->last_y_nnz = (int32_t)d.m;
        c->batch_fallback = fallback ? 1 : 0;
    }
    if (fallback) {
        // (the copies in flight must have landed before the block ends)
        for (int k = 0; k < issued; ++k) mbar_wait_bounded(&s_bar[k], 0u);
        return;
    }
    // y is zeroed by the kernel in front, which this one may overlap up to here
    pdl_wait();

    float mma_lo[4] = {0.f, 0.f, 0.f, 0.f}, mma_hi[4] = {0.f, 0.f, 0.f, 0.f};
    int cur_rb = -1;
    auto flush = [&]() { if (cur_rb >= 0) mma_flush(y, ldy, cur_rb, nvec, lane, mma_lo, mma_hi); };
    // one step: the lane's entry of row block cur_rb; mask-based blocks two at a time on the
    // tensor cores (staged payload only: ldmatrix reads shared memory), the odd hypersparse entry
    // vector by vector in its own lane
    auto step = [&](const uint8_t *payload, uint32_t idx, uint32_t w, uint32_t aux, bool have, bool staged) {
        const uint32_t um = have ? s_um[idx & IDX_MASK] : 0u;
        const int type = idx >> TYPE_SHIFT;
        const bool mk = staged && have && um && type > DBSPMSPV_BLK_COO;
        uint32_t todo = __ballot_sync(FULL, mk);
        while (todo) {
            const int src0 = __ffs(todo) - 1;
            todo &= todo - 1;
            const int src1 = todo ? __ffs(todo) - 1 : -1;
            if (todo) todo &= todo - 1;
            const uint32_t bidx0 = __shfl_sync(FULL, idx, src0), bw0 = __shfl_sync(FULL, w, src0);
            const uint32_t bidx1 = __shfl_sync(FULL, idx, src1 < 0 ? src0 : src1), bw1 = __shfl_sync(FULL, w, src1 < 0 ? src0 : src1);
            const int t0 = bidx0 >> TYPE_SHIFT, t1 = bidx1 >> TYPE_SHIFT;
            const uint8_t *blk0 = payload + (size_t)bw0 * 4, *blk1 = payload + (size_t)bw1 * 4;
            __syncwarp();                                     // (the tiles of the round before have been read)
            if (t0 != DBSPMSPV_BLK_DENSE) expand_block_bf16(blk0, is_row_major(t0), s_tile, lane);
            if (src1 >= 0 && t1 != DBSPMSPV_BLK_DENSE) expand_block_bf16(blk1, is_row_major(t1), s_tile + 256, lane);
            __syncwarp();
            // (Dense: the values lie in the payload as the tile wants them)
            mma_block(t0 != DBSPMSPV_BLK_DENSE ? static_cast<const void *>(s_tile) : blk0 + 32, s_xh + (size_t)(bidx0 & IDX_MASK) * 16,
                      lay.ldh, nvec, lane, mma_lo, mma_hi);
            if (src1 >= 0)
                mma_block(t1 != DBSPMSPV_BLK_DENSE ? static_cast<const void *>(s_tile + 256) : blk1 + 32, s_xh + (size_t)(bidx1 & IDX_MASK) * 16,
                          lay.ldh, nvec, lane, mma_lo, mma_hi);
        }
        if (have && um && type <= DBSPMSPV_BLK_COO) {
            for (int v = 0; v < nvec; ++v) {
                const uint32_t xm = s_xm[(size_t)v * d.nb + (idx & IDX_MASK)];
                if (!xm) continue;
                const uint16_t *xb = s_xh + (size_t)v * lay.ldh + (size_t)(idx & IDX_MASK) * 16;
                float *row0 = y + (size_t)v * ldy + (size_t)cur_rb * 16;
                if (type == DBSPMSPV_BLK_INLINE) {
                    if ((xm >> (aux & 15)) & 1u)
                        atomicAdd(row0 + (aux >> 4), Val<DBSPMSPV_BF16>::inline_value(w) * __uint_as_float((uint32_t)xb[aux & 15] << 16));
                } else {
                    const int nnz = (int)aux + 1;
                    const uint8_t *blk = payload + (size_t)w * 4, *vals = blk + ((nnz + 3) & ~3);
                    for (int k = 0; k < nnz; ++k) {
                        const int c = blk[k] & 15, r = blk[k] >> 4;
                        if ((xm >> c) & 1u) atomicAdd(row0 + r, Val<DBSPMSPV_BF16>::load(vals, k) * __uint_as_float((uint32_t)xb[c] << 16));
                    }
                }
            }
        }
    };

    bool timed_out = false;
    uint32_t idx = 0, w = 0, aux = 0, n_idx, n_w, n_aux;
    if (n_mine > 0) entries_of(desc_of(0), idx, w, aux);
    for (int k = 0; k < n_mine; ++k) {
        for (const int lim = min(n_mine, min(k + STREAM_DEPTH, (k & ~31) + 32)); issued < lim; ++issued) {
            const int4 nch = desc_of(issued);
            if (lane == 0) issue(nch, issued % STREAM_DEPTH);
        }
        const int st = k % STREAM_DEPTH;
        const int4 ch = desc_of(k);
        n_idx = 0; n_w = 0; n_aux = 0;
        if (k + 1 < n_mine && ((k + 1) & 31)) entries_of(desc_of(k + 1), n_idx, n_w, n_aux);
        if (!mbar_wait_bounded(&s_bar[st], (uint32_t)(k / STREAM_DEPTH) & 1u)) { timed_out = true; break; }
        if (ch.y != cur_rb) { flush(); cur_rb = DBS_CHK_INDEX(d, ch.y, d.mb) ? ch.y : 0; }
        const uint8_t *base = s_ring + (size_t)st * stride;
        step(base - (size_t)(uint32_t)ch.z * 4, idx, w, aux, lane < (int)((uint32_t)ch.w >> 24), true);
        __syncwarp();
        idx = n_idx; w = n_w; aux = n_aux;
        if (k + 1 < n_mine && !((k + 1) & 31)) {
            my_desc = make_int4(0, 0, 0, 0);
            if (k + 1 + lane < n_mine) my_desc = d.stage_chunks[lo + k + 1 + lane];
            entries_of(desc_of(k + 1), idx, w, aux);
        }
    }
    flush();
    if (timed_out) { d.ws.ctr->status = DBSPMSPV_ERR_TIMEOUT; return; }
    // the INLINE elements of the row blocks (row by row, rare in these handles)
    for (int rb = gw; rb < d.mb && d.has_inline; rb += W) {
        const int b0 = d.csr_inl[rb], b1 = d.csr.ptr[rb + 1];
        cur_rb = rb;
        for (int base = b0; base < b1; base += 32) {
            uint32_t e_idx = 0, e_w = 0, e_aux = 0;
            const bool have = base + lane < b1;
            if (have && DBS_CHK_INDEX(d, base + lane, d.n_entries)) {
                e_idx = d.csr.idx[base + lane]; e_w = d.csr.w[base + lane]; e_aux = d.csr.aux[base + lane];
                DBS_CHK_ENTRY(d, true, e_idx, e_w, e_aux);
            }
            step(d.payload, e_idx, e_w, e_aux, have, false);
        }
    }
}

__global__ void k_zero_rows(float *y, int64_t ldy, int64_t m, int nvec) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int v = 0; v < nvec; ++v)
        for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < m; i += stride) y[(size_t)v * ldy + i] = 0.f;
}

}  // namespace dbs
