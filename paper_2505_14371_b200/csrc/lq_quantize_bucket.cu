// ENCODE in bucket scope (Section 7.1 runs the quantizer on buckets of 128 consecutive coordinates, each with
// its own norm): a bucket is one row of a message block, which a warp holds as one float4 per lane, so the norm
// is a reduction over the warp and the separate norm pass disappears.  One pass over the values: a block's 8
// rows travel into a per-warp ring in shared memory with 16-byte asynchronous copies (a lane reads back only
// the bytes it copied itself, so the ring needs no barrier), the 8 norms are formed at once, and the rows are
// then quantized from the ring like in the other scopes (lq_quantize.cuh), with the value tables holding the
// plain signed levels and every row bringing its own norm.  While a row is consumed, the same row of the
// warp's next block is already on its way into the ring.
#include "lq_quantize.cuh"

namespace lq {

constexpr int kRingRows = 8;                       // rows of 512 bytes in flight per warp

struct BucketCtx {
    const float* g;              // first coordinate of the layer in this worker's row
    int64_t size;                // d_m
    uint32_t ring;               // shared-memory address of this lane's 16 bytes in ring row 0
    const float4* ring_ptr;      // the same place as a pointer
    int lane;
    const float* prev_bn;        // bucket norms of the previous message for this (worker, layer), or nullptr
    float* bn_out;               // bucket norms of this message for this (worker, layer)
    int q;
    double energy;               // this lane's share of the sum of squared bucket norms
    uint32_t flags;              // bit 0: a bucket held NaN or Inf, bit 1: a bucket with a nonzero norm
};

// Starts the copies of all 8 rows of a block that may reach past the layer's end (zero-filled there).
__device__ __forceinline__ void issue_ragged_block(const BucketCtx& c, int64_t blk)
{
#pragma unroll
    for (int j = 0; j < kRingRows; ++j) {
        const int64_t pos = blk * kBlockCoords + 128 * j + 4 * c.lane;
        const int64_t rem = c.size - pos;
        const int bytes = rem >= 4 ? 16 : (rem > 0 ? 4 * (int)rem : 0);
        cp_async16(c.ring + 512u * j, rem > 0 ? c.g + pos : c.g, bytes);
        cp_async_commit();
    }
}

// The L^q norms of the 8 rows (buckets) of the block in this lane's ring slots, all at once.  Every lane forms its
// fp64 partial of each row; a butterfly that halves the set of rows a lane carries at each of its first three steps
// leaves the total of row (lane >> 2) in every lane, so the root, the rounding to fp32, the checks and the
// reciprocal run once per block, for all 8 rows in parallel.  Returns this lane's row's norm (0 for a bucket that is
// all zero, below the smallest normal float, or non-finite: then `bad`) and its fp32 reciprocal (or 0).
template <bool kMax>
__device__ __forceinline__ double pair_op(double x, double y) { return kMax ? fmax(x, y) : x + y; }

template <bool kMax>
__device__ __forceinline__ double rows_butterfly(double (&part)[8], int lane)
{
    const bool h16 = lane & 16, h8 = lane & 8, h4 = lane & 4;
    double s[4], t[2];
#pragma unroll
    for (int i = 0; i < 4; ++i)
        s[i] = pair_op<kMax>(h16 ? part[4 + i] : part[i], __shfl_xor_sync(0xffffffffu, h16 ? part[i] : part[4 + i], 16));
#pragma unroll
    for (int i = 0; i < 2; ++i)
        t[i] = pair_op<kMax>(h8 ? s[2 + i] : s[i], __shfl_xor_sync(0xffffffffu, h8 ? s[i] : s[2 + i], 8));
    double tot = pair_op<kMax>(h4 ? t[1] : t[0], __shfl_xor_sync(0xffffffffu, h4 ? t[0] : t[1], 4));
    tot = pair_op<kMax>(tot, __shfl_xor_sync(0xffffffffu, tot, 2));
    tot = pair_op<kMax>(tot, __shfl_xor_sync(0xffffffffu, tot, 1));
    return tot;
}

// mode 0: max |v|   1: sum |v|   2: sum v^2   3: sum |v|^q (integer q >= 3)
template <int kMode>
__device__ __forceinline__ void row_partials(const float4* ring_ptr, int q, uint32_t badbits, double (&part)[8])
{
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float4 v = ring_ptr[32 * j];
        const float a[4] = {fabsf(v.x), fabsf(v.y), fabsf(v.z), fabsf(v.w)};
        double acc = 0.0;
        if (kMode == 0) {
            acc = (double)fmaxf(fmaxf(a[0], a[1]), fmaxf(a[2], a[3]));
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const double x = (double)a[e];
                if (kMode == 1)      acc += x;
                else if (kMode == 2) acc = fma(x, x, acc);
                else { double pw = x; for (int r = 1; r < q; ++r) pw = __dmul_rn(pw, x); acc += pw; }
            }
        }
        part[j] = ((badbits >> j) & 1u) ? 0.0 : acc;     // a row with NaN or Inf is zeroed whatever it sums to
    }
}

__device__ __forceinline__ void bucket_norms8(const float4* ring_ptr, int q, int lane, float& norm, float& rnorm,
                                              bool& bad)
{
    // per row, the largest |v| of this lane as an integer pattern: >= 0x7f800000 means NaN or Inf, 0 means all zero
    uint32_t badbits = 0, nzbits = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint4 w = *reinterpret_cast<const uint4*>(ring_ptr + 32 * j);
        const uint32_t mb = max(max(w.x & 0x7fffffffu, w.y & 0x7fffffffu), max(w.z & 0x7fffffffu, w.w & 0x7fffffffu));
        badbits |= ((mb + 0x00800000u) >> 31) << j;      // mb <= 0x7fffffff: the sum reaches bit 31 iff mb >= 0x7f800000
        nzbits |= ((mb + 0x7fffffffu) >> 31) << j;       // ... iff mb >= 1
    }
    badbits = __reduce_or_sync(0xffffffffu, badbits);
    nzbits = __reduce_or_sync(0xffffffffu, nzbits);
    norm = 0.0f; rnorm = 0.0f; bad = false;
    if ((badbits | nzbits) == 0u) return;                // a block of zeros (untouched embedding rows): nothing to reduce
    double part[8];
    double tot;
    if (q == 0)      { row_partials<0>(ring_ptr, q, badbits, part); tot = rows_butterfly<true>(part, lane); }
    else if (q == 1) { row_partials<1>(ring_ptr, q, badbits, part); tot = rows_butterfly<false>(part, lane); }
    else if (q == 2) { row_partials<2>(ring_ptr, q, badbits, part); tot = rows_butterfly<false>(part, lane); }
    else             { row_partials<3>(ring_ptr, q, badbits, part); tot = rows_butterfly<false>(part, lane); }
    const int row = lane >> 2;
    const double n64 = (q == 0 || q == 1) ? tot : (q == 2 ? sqrt(tot) : pow(tot, 1.0 / (double)q));
    const float n = (float)n64;
    bad = ((badbits >> row) & 1u) || !(fabs(n64) <= 1.7976931348623157e308) || !(fabsf(n) <= 3.402823466e38f);
    const bool live = !bad && ((nzbits >> row) & 1u) && n >= 1.17549435e-38f;
    norm = live ? n : 0.0f;
    rnorm = live ? __fdiv_rn(1.0f, n) : 0.0f;
}

// One block of 1024 coordinates from the ring.  `next` is this lane's first float4 of the block whose rows
// replace the consumed ones (nullptr: nothing to fetch); `prev_rows` says which rows may be nonzero in the
// previous message and lanes 0..7 of prev_norm8 hold that message's norms of rows 0..7.  Returns this lane's
// statistic term.
template <int B, int kSearch, bool kHist>
__device__ __forceinline__ double quantize_block(const PlanDev& p, const PhiloxConsts& pc, BucketCtx& c, QuantEnv ev,
                                                 int64_t blk, uint32_t prev_rows, const float* __restrict__ next,
                                                 uint32_t* __restrict__ out, const uint32_t (&pw)[B + 1],
                                                 float prev_norm8)
{
    constexpr int C = B + 1;
    const int lane = c.lane;
    float my_norm, my_rnorm;                     // norm and reciprocal of row (lane >> 2)
    bool bad;
    cp_async_wait<0>();                          // all 8 rows of the block have landed
    bucket_norms8(c.ring_ptr, c.q, lane, my_norm, my_rnorm, bad);
    if ((lane & 3) == 0) c.energy = fma((double)my_norm, (double)my_norm, c.energy);
    c.flags |= (bad ? 1u : 0u) | (my_norm > 0.0f ? 2u : 0u);
    const uint32_t live_lanes = __ballot_sync(0xffffffffu, my_norm > 0.0f);     // bit 4 j: row j sends something
    const int64_t woff = blk * (int64_t)C * 32 + lane;
    if (prev_rows == 0u && live_lanes == 0u) {
        // every bucket of the block is zeroed and the previous message is zero here too: zero words, zero
        // norms, nothing for the statistic; the ring takes the next block's rows at once
#pragma unroll
        for (int j = 0; j < kRingRows; ++j) {
            if (next) cp_async16(c.ring + 512u * j, next + 128 * j, 16);
            cp_async_commit();
        }
#pragma unroll
        for (int w = 0; w < C; ++w) __stcs(out + woff + w * 32, 0u);
        if ((lane & 3) == 0) c.bn_out[blk * 8 + (lane >> 2)] = 0.0f;
        return 0.0;
    }
    uint32_t cw[C];
    pack_begin<C>(cw, ev.ld);
    double stat = 0.0;
    const uint32_t ctr0 = (uint32_t)(blk * 256) + (uint32_t)lane;     // index / 4 of this lane's row 0

#pragma unroll
    for (int j = 0; j < kRingRows; ++j) {
        // this row's norm now and in the previous message
        const float nrow = __shfl_sync(0xffffffffu, my_norm, 4 * j);
        ev.r = __shfl_sync(0xffffffffu, my_rnorm, 4 * j);
        const float pn = __shfl_sync(0xffffffffu, prev_norm8, j);
        if ((live_lanes >> (4 * j)) & 1u) {                  // a zeroed bucket sends zeros and draws nothing
            const float4 v = c.ring_ptr[32 * j];
            const float vv[4] = {v.x, v.y, v.z, v.w};
            uint32_t x[4];
            philox4x32_10_folded(ctr0 + 32 * j, pc, p, x);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool counted = !kHist || blk * kBlockCoords + 128 * j + 4 * lane + e < c.size;
                quantize_coord<B, kSearch, kHist, true, true>(ev, vv[e], x[e], 4 * j + e, cw, pw, stat, nrow, pn, counted);
            }
        } else {
            pack_zero_row<C>(cw, j, ev.ld);
            if ((prev_rows >> j) & 1u) {
#pragma unroll
                for (int e = 0; e < 4; ++e) stat_prev_only<C, true>(ev, pw, 4 * j + e, pn, stat);
            }
        }
        if (next) cp_async16(c.ring + 512u * j, next + 128 * j, 16);
        cp_async_commit();
    }
#pragma unroll
    for (int w = 0; w < C; ++w) __stcs(out + woff + w * 32, cw[w]);
    if ((lane & 3) == 0) c.bn_out[blk * 8 + (lane >> 2)] = my_norm;
    return stat;
}

// A warp's share of a tile: blocks warp, warp + 8, ...
template <int B, int kSearch, bool kHist>
__device__ __forceinline__ double quantize_tile(const PlanDev& p, const PhiloxConsts& pc, BucketCtx& c, const QuantEnv& ev,
                                                const Tile& tile, uint32_t* __restrict__ out,
                                                const uint32_t* __restrict__ prev)
{
    constexpr int C = B + 1;
    const int warp = threadIdx.x >> 5;
    const int64_t nfull = c.size / kBlockCoords;          // blocks below this index lie inside the layer
    double stat = 0.0;
    bool primed = false;                                  // the ring holds (or awaits) the rows of block b
    for (int b = warp; b < tile.nblocks; b += kQWarps) {
        const int64_t blk = tile.block0 + b;
        if (!primed) {
            if (blk < nfull) {
                const float* src = c.g + blk * kBlockCoords + 4 * c.lane;
#pragma unroll
                for (int j = 0; j < kRingRows; ++j) {
                    cp_async16(c.ring + 512u * j, src + 128 * j, 16);
                    cp_async_commit();
                }
            } else {
                issue_ragged_block(c, blk);
            }
        }
        // the previous message's norms tell which of its rows are all zero: those add nothing to the statistic
        float prev_norm8 = 0.0f;
        uint32_t pmask = 0u;
        if (prev) {
            if (c.lane < 8) prev_norm8 = __ldg(c.prev_bn + blk * 8 + c.lane);
            pmask = __ballot_sync(0xffffffffu, prev_norm8 != 0.0f) & 0xffu;
        }
        uint32_t pw[C];
#pragma unroll
        for (int w = 0; w < C; ++w) pw[w] = pmask ? __ldcs(prev + blk * (int64_t)C * 32 + c.lane + w * 32) : 0u;
        const int nb = b + kQWarps;
        const bool has_next = nb < tile.nblocks;
        const int64_t nblk = tile.block0 + nb;
        const float* next = (has_next && nblk < nfull) ? c.g + nblk * kBlockCoords + 4 * c.lane : nullptr;
        stat += quantize_block<B, kSearch, kHist>(p, pc, c, ev, blk, pmask, next, out, pw, prev_norm8);
        primed = has_next;
        if (has_next && nblk >= nfull) issue_ragged_block(c, nblk);   // the layer's last, partial block
    }
    cp_async_wait<0>();
    return stat;
}

template <bool kHist>
__global__ void __launch_bounds__(kQThreads, 3) quantize_pack_bucket_kernel(
    PlanDev p, const float* __restrict__ grads, uint32_t step, uint32_t* __restrict__ packed,
    float* __restrict__ bucket_norms, uint32_t* __restrict__ hist,
    const uint32_t* __restrict__ prev_packed, const float* __restrict__ prev_norms,
    const float* __restrict__ levels_cur, const float* __restrict__ levels_prev, SearchTables st)
{
    extern __shared__ unsigned char dyn_smem[];
    uint32_t base;
    unsigned char* sm = table_base(dyn_smem, base);
    const Tile tile = p.tiles[blockIdx.x];
    const int layer = tile.layer;
    const LayerDesc L = p.layers[layer];
    const int k = blockIdx.y + p.worker0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t kl = (int64_t)k * p.num_layers + layer;
    const int search = st.fast[layer];                      // 1: one lookup; 1 + R: byte table and up to R steps

    // the tables hold the plain levels (norm 1) and each row multiplies by its own norm
    fill_tables(sm, st, layer, L.nlevels, true, levels_cur, levels_prev, 1.0f, 1.0f, kHist);
    __syncthreads();

    BucketCtx c;
    c.g = grads + (int64_t)blockIdx.y * p.padded_elems + L.elem_off;
    c.size = L.size;
    c.ring_ptr = reinterpret_cast<const float4*>(sm + kSmRing) + (warp * kRingRows) * 32 + lane;
    c.ring = (uint32_t)__cvta_generic_to_shared(c.ring_ptr);
    c.lane = lane;
    const int64_t bo = (int64_t)k * p.total_blocks * 8 + L.block_off * 8;
    c.prev_bn = prev_norms ? prev_norms + bo : nullptr;
    c.bn_out = bucket_norms + bo;
    c.q = p.q;
    c.energy = 0.0;
    c.flags = 0u;
    QuantEnv ev;
    ev.lut = base + kSmLut; ev.ld = base + kSmLd; ev.tprev = base + kSmTprev;
    ev.r = 1.0f;
    ev.refine = search - 1;
    ev.hist = reinterpret_cast<uint32_t*>(sm + kSmHist);
    if (step == LQ_STEP_AUTO) step = (uint32_t)p.scalars->t;      // the plan's own iteration counter (graph replays)
    const PhiloxConsts pc = philox_fold((uint32_t)layer, (uint32_t)k, step, p.seed_lo, p.seed_hi);
    uint32_t* out = packed + (int64_t)k * p.packed_words + L.word_off;
    const uint32_t* prev = prev_packed ? prev_packed + (int64_t)k * p.packed_words + L.word_off : nullptr;

    double stat = 0.0;
    switch (L.bits * 2 + (search == 1 ? 1 : 0)) {
#define LQ_CASE(BB)                                                                              \
    case 2 * BB:     stat = quantize_tile<BB, 2, kHist>(p, pc, c, ev, tile, out, prev); break;  \
    case 2 * BB + 1: stat = quantize_tile<BB, 1, kHist>(p, pc, c, ev, tile, out, prev); break;
        LQ_CASE(1) LQ_CASE(2) LQ_CASE(3) LQ_CASE(4) LQ_CASE(5) LQ_CASE(6) LQ_CASE(7) LQ_CASE(8)
#undef LQ_CASE
        default: break;
    }
    double* scratch = reinterpret_cast<double*>(sm + kSmScratch);
    const double total = block_reduce<false>(stat, scratch);
    const double energy = block_reduce<false>(c.energy, scratch);
    const int any_bad = __syncthreads_or((int)(c.flags & 1u));
    const int any_live = __syncthreads_or((int)(c.flags & 2u));
    if (threadIdx.x == 0) {
        p.stat_partial[(int64_t)k * p.num_tiles + blockIdx.x] = total;
        p.energy_partial[(int64_t)k * p.num_tiles + blockIdx.x] = energy;
        p.flag_partial[(int64_t)k * p.num_tiles + blockIdx.x] = (any_bad ? 1u : 0u) | (any_live ? 2u : 0u);
    }

    if (kHist) {
        __syncthreads();
        uint32_t* h = hist + kl * LQ_HIST_STRIDE;
        for (int i = threadIdx.x; i < LQ_NUM_BINS; i += blockDim.x)
            if (ev.hist[i]) atomicAdd(h + i, ev.hist[i]);
    }
}

// Per (layer, worker), in tile order: the statistic, the layer's energy (its weight in the level fit,
// as the square root of the summed squared bucket norms) and its flags: LQ_STATUS_NONFINITE if a bucket was
// zeroed because it held NaN or Inf, else LQ_STATUS_ZERO_NORM if no bucket has a nonzero norm.
__global__ void __launch_bounds__(128) bucket_finalize_kernel(PlanDev p)
{
    __shared__ double scratch[4];
    const int m = blockIdx.x, k = blockIdx.y + p.worker0;
    const LayerDesc L = p.layers[m];
    const int64_t o = (int64_t)k * p.num_tiles + L.first_tile;
    double acc = 0.0, en = 0.0;
    uint32_t fl = 0;
    for (int i = threadIdx.x; i < L.ntiles; i += blockDim.x) {
        acc += p.stat_partial[o + i];
        en += p.energy_partial[o + i];
        fl |= p.flag_partial[o + i];
    }
    const double total = block_reduce<false>(acc, scratch);
    const double energy = block_reduce<false>(en, scratch);
    const int any_bad = __syncthreads_or((int)(fl & 1u));
    const int any_live = __syncthreads_or((int)(fl & 2u));
    if (threadIdx.x == 0) {
        const int64_t kl = (int64_t)k * p.num_layers + m;
        p.sq_diff[kl] = total;
        p.layer_weight[kl] = (float)sqrt(energy);
        p.status[kl] = any_bad ? LQ_STATUS_NONFINITE : (any_live ? 0u : LQ_STATUS_ZERO_NORM);
    }
}

cudaError_t launch_quantize_bucketed(const PlanDev& p, const float* grads, uint32_t step, uint32_t* packed,
                                     float* bucket_norms, uint32_t* hist, const uint32_t* prev_packed,
                                     const float* prev_norms, const float* levels_cur,
                                     const float* levels_prev, SearchTables t, cudaStream_t s)
{
    if (p.num_tiles == 0) return cudaSuccess;
    const dim3 grid((unsigned)p.num_tiles, (unsigned)p.worker_count);
    constexpr unsigned smem = kSmTables + kRingBytes + LQ_HIST_STRIDE * 4 + kSmSlack;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {            // more than 48 KB of dynamic shared memory: opt in once
        cudaError_t e = cudaFuncSetAttribute(quantize_pack_bucket_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(quantize_pack_bucket_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    if (hist)
        quantize_pack_bucket_kernel<true><<<grid, kQThreads, smem, s>>>(p, grads, step, packed, bucket_norms, hist,
                                                                        prev_packed, prev_norms, levels_cur, levels_prev, t);
    else
        quantize_pack_bucket_kernel<false><<<grid, kQThreads, smem, s>>>(p, grads, step, packed, bucket_norms, hist,
                                                                         prev_packed, prev_norms, levels_cur, levels_prev, t);
    return cudaGetLastError();
}

cudaError_t launch_bucket_finalize(const PlanDev& p, cudaStream_t s)
{
    bucket_finalize_kernel<<<dim3((unsigned)p.num_layers, (unsigned)p.worker_count), 128, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace lq
