// ENCODE for all workers in the layer and global norm scopes: normalise, round stochastically between
// neighbouring levels, pack one (b+1)-bit symbol per coordinate (Section 3.1 quantizer, Section 3.2 message;
// Algorithm 1 line 12), with the optional histogram of normalised magnitudes (Algorithm 1 line 4) and the
// sender-side term of the adaptive step size, sum ||V^_{k,t+1/2} - V^_{k,t-1/2}||^2 (Eq. general_stepsize).
//
// Work decomposition: one CTA of 8 warps per (tile, worker); a tile is up to 128 blocks of 1024
// coordinates of one layer, taken round-robin by the warps.  A lane owns the 32 coordinates
// {128 j + 4 lane + e} of a block (row j = one float4 per lane, 512 contiguous bytes per warp).  Rows
// travel from global memory into a per-warp ring of 8 rows in shared memory with 16-byte
// asynchronous copies, so a warp always has up to 4 KB in flight and the values never sit in registers
// while they wait; every lane reads back only the bytes it copied itself, so the ring needs no
// barrier.  Per row the lane draws one Philox4x32-10 block (4 uniforms); after 8 rows it holds
// exactly b+1 words of symbols, which it stores plane by plane (128 contiguous bytes per warp and
// plane).  No shuffles, ballots or atomics on the per-coordinate path.  The kernel is bound by
// instruction issue (about 42 instructions per coordinate: 10 Philox, 7 the statistic), not by DRAM.
//
// The level search and the tables are described in lq_quantize.cuh.  Layers whose levels are denser than the
// search table's bins take a byte table over finer bins and step up from its entry (build_search_kernel).
//
// The norm pass, which reads the same values just before, leaves one bit per row of 128 values
// that says whether the row holds anything but zeros.  An all-zero row (untouched embedding rows)
// is never fetched, draws no random numbers and needs no search: its symbols are 0.  If the
// previous message is all zero there as well, the row adds nothing to the statistic and is
// skipped entirely.  The masks are made warp-uniform by a reduction, so the per-row tests are uniform
// branches.  The unrolled code handles whole blocks only; a layer's last, partial block goes through a
// plain loop (once per layer and worker).
#include "lq_quantize.cuh"

namespace lq {

// Everything a warp needs to walk its blocks of one (tile, worker).
struct WarpCtx {
    const float* g;              // first coordinate of the layer in this worker's row
    int64_t size;                // d_m
    int64_t nfull;               // blocks below this index lie wholly inside the layer
    int lane;
};

// x of lane i, the same in every lane and known to be (a reduction's result is warp-uniform)
__device__ __forceinline__ uint32_t lane_value(uint32_t x, int i, int lane)
{
    return __reduce_or_sync(0xffffffffu, lane == i ? x : 0u);
}

// The layer's last, partial block (one per layer and worker): a plain loop over the lane's 32 positions with a
// binary search over the levels, the coordinates past the layer's end sending zeros.  Same arithmetic as
// quantize_coord; speed does not matter here.
__device__ __noinline__ double quantize_partial_block(const PlanDev& p, const QuantEnv& ev, const float* __restrict__ g,
                                                      int64_t size, int64_t blk, int bits, uint32_t layer, uint32_t worker,
                                                      uint32_t step, uint32_t* __restrict__ out,
                                                      const uint32_t* __restrict__ prev, bool hist, int lane)
{
    const int C = bits + 1, n = 1 << bits;
    const int64_t woff = blk * (int64_t)C * 32 + lane;
    uint64_t acc = 0, pacc = 0;
    int fill = 0, wi = 0, pfill = 0, pwi = 0;
    double stat = 0.0;
    for (int pp = 0; pp < 32; ++pp) {
        const int64_t pos = blk * kBlockCoords + 128 * (pp >> 2) + 4 * lane + (pp & 3);
        uint32_t sym = 0;
        if (pos < size) {
            const float v = __ldg(g + pos);
            uint32_t x[4];
            philox4x32_10((uint32_t)(pos >> 2), layer, worker, step, p.seed_lo, p.seed_hi, x);
            const float u = __fmul_rn(fabsf(v), ev.r);
            int tau = 0;
            for (int s = n >> 1; s > 0; s >>= 1)
                if (lds_f32(ev.ld + 8u * (uint32_t)(tau + s)) <= u) tau += s;
            tau = min(tau, n - 2);
            const float2 ld = lds_f32x2(ev.ld + 8u * (uint32_t)tau);
            const float num = __fsub_rn(u, ld.x);
            const float f = __uint_as_float((x[pos & 3] >> 9) | 0x3F800000u);
            const float t = __fmaf_rn(f, ld.y, -ld.y);
            sym = 2u * (uint32_t)(tau + (t < num ? 1 : 0)) + (v < 0.0f ? 1u : 0u);
            if (hist) atomicAdd(ev.hist + ((max(__float_as_uint(u), kHistClamp) - kHistClamp) >> 19), 1u);
        }
        if (pfill < C) {
            if (prev && pwi < C) pacc |= (uint64_t)__ldg(prev + woff + 32 * pwi) << pfill;
            pfill += 32; ++pwi;
        }
        const uint32_t psym = (uint32_t)pacc & ((1u << C) - 1u);
        pacc >>= C; pfill -= C;
        const double dd = (double)__fsub_rn(lds_f32(ev.ld + (kSmTcur - kSmLd) + 4u * sym), lds_f32(ev.tprev + 4u * psym));
        stat = fma(dd, dd, stat);
        acc |= (uint64_t)sym << fill;
        fill += C;
        if (fill >= 32) { __stcs(out + woff + 32 * wi, (uint32_t)acc); acc >>= 32; fill -= 32; ++wi; }
    }
    return stat;
}

// A warp's share of a tile: the whole blocks warp, warp + 8, ...  A block whose rows are all zero in this input
// and in the input behind the previous message is an all-zero piece of message that adds nothing to the
// statistic: its words are stored and nothing is read.  The other blocks are taken in order.
template <int B, int kSearch, bool kHist, bool kStat>
__device__ __forceinline__ double quantize_tile(const PlanDev& p, const PhiloxConsts& pc, const WarpCtx& c,
                                                const Tile& tile, uint32_t* __restrict__ out,
                                                const uint32_t* __restrict__ prev, const QuantEnv& ev,
                                                const uint8_t* rows_cur, const uint8_t* rows_prev, uint32_t ring_base)
{
    constexpr int C = B + 1;
    const int warp = threadIdx.x >> 5, lane = c.lane;
    double stat = 0.0;
    const int64_t nf = c.nfull - tile.block0;                 // whole blocks of this tile
    const int nfb = nf < tile.nblocks ? (int)nf : tile.nblocks;

    // lane i < 16 keeps the masks of the warp's i-th block (this input's rows in bits 0..7, the previous input's
    // in bits 8..15, bit 16: the block exists)
    uint32_t mymask = 0;
    {
        const int b = warp + kQWarps * lane;
        if (lane < kTileBlocks / kQWarps && b < nfb) mymask = (uint32_t)rows_cur[b] | ((uint32_t)rows_prev[b] << 8) | 0x10000u;
    }
    uint32_t zero = __ballot_sync(0xffffffffu, mymask == 0x10000u);
    uint32_t todo = __ballot_sync(0xffffffffu, (mymask & 0xffffu) != 0u);
    while (zero) {
        const int i = __ffs(zero) - 1;
        zero &= zero - 1;
        const int64_t blk = tile.block0 + warp + kQWarps * i;
        const int64_t woff = blk * (int64_t)C * 32 + lane;
#pragma unroll
        for (int w = 0; w < C; ++w) __stcs(out + woff + w * 32, 0u);
        if (kHist && lane == 0) atomicAdd(ev.hist, (uint32_t)kBlockCoords);     // its coordinates all have u = 0
    }
    if (todo == 0u) return stat;

    auto block_base = [&](int i) { return c.g + (tile.block0 + warp + kQWarps * i) * (int64_t)kBlockCoords; };
    int i = __ffs(todo) - 1;
    todo &= todo - 1;
    uint32_t m = lane_value(mymask, i, lane);
    const float* src = block_base(i) + 4 * lane;             // this lane's float4 of row 0
    // While a lane works on row j of a block, row j of the next block with content is already on its way into
    // the slot that row j has just left (one commit group per row slot, so waiting for all but the last 7
    // groups means the row is there).
    const uint32_t ring = ring_base + (uint32_t)(warp * 8 * 512 + lane * 16);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        if ((m >> j) & 1u) cp_async16(ring + 512u * j, src + 128 * j, 16);
        cp_async_commit();
    }
    for (;;) {
        const int64_t blk = tile.block0 + warp + kQWarps * i;
        const uint32_t rows = m & 0xffu, prows = (m >> 8) & 0xffu;
        // the next block with content: its rows follow this block's
        const int inext = todo ? __ffs(todo) - 1 : 0;
        const uint32_t mnext = todo ? lane_value(mymask, inext, lane) : 0u;
        const float* nsrc = block_base(inext) + 4 * lane;
        uint32_t pw[C];
#pragma unroll
        for (int w = 0; w < C; ++w)
            pw[w] = (kStat && prev && prows) ? __ldcs(prev + blk * (int64_t)C * 32 + lane + w * 32) : 0u;
        uint32_t cw[C];
        pack_begin<C>(cw, ev.ld);
        const uint32_t ctr0 = (uint32_t)(blk * 256) + (uint32_t)lane;     // index / 4 of this lane's row 0
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if ((rows >> j) & 1u) {
                float4 v;
                cp_async_wait<7>();
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                             : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(ring + 512u * j));
                if ((mnext >> j) & 1u) cp_async16(ring + 512u * j, nsrc + 128 * j, 16);
                cp_async_commit();
                uint32_t x[4];
                philox4x32_10_folded(ctr0 + 32 * j, pc, p, x);
                const float vv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    quantize_coord<B, kSearch, kHist, kStat, false>(ev, vv[e], x[e], 4 * j + e, cw, pw, stat, 0.f, 0.f, true);
            } else {
                if ((mnext >> j) & 1u) cp_async16(ring + 512u * j, nsrc + 128 * j, 16);
                cp_async_commit();
                pack_zero_row<C>(cw, j, ev.ld);
                if (kStat && ((prows >> j) & 1u)) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) stat_prev_only<C, false>(ev, pw, 4 * j + e, 0.f, stat);
                }
                if (kHist && lane == 0) atomicAdd(ev.hist, 128u);   // an all-zero row: its coordinates have u = 0
            }
        }
        const int64_t woff = blk * (int64_t)C * 32 + lane;
#pragma unroll
        for (int w = 0; w < C; ++w) __stcs(out + woff + w * 32, cw[w]);
        if (todo == 0u) break;
        i = inext;
        todo &= todo - 1;
        m = mnext;
        src = nsrc;
    }
    cp_async_wait<0>();
    return stat;
}

template <bool kHist, bool kStat>
__global__ void __launch_bounds__(kQThreads, 4) quantize_pack_kernel(
    PlanDev p, const float* __restrict__ grads, uint32_t step, uint32_t* __restrict__ packed,
    const float* __restrict__ norms, uint32_t* __restrict__ hist,
    const uint32_t* __restrict__ prev_packed, const float* __restrict__ prev_norms,
    const float* __restrict__ levels_cur, const float* __restrict__ levels_prev, SearchTables st)
{
    extern __shared__ unsigned char dyn_smem[];
    uint32_t base;
    unsigned char* sm = table_base(dyn_smem, base);
    // CTAs start in the order of their flat index: the workers of one tile next to each other, tiles in the plan's
    // launch order, so that the last CTAs to start are every worker's short tiles (the ends of the layers) and not
    // one worker's whole message
    const int flat = blockIdx.y * gridDim.x + blockIdx.x;
    const int slot = flat / (int)gridDim.y, kk = flat - slot * (int)gridDim.y;
    const TileJob J = p.jobs[slot];
    const int tile_id = J.tile, layer = J.layer;
    Tile tile;
    tile.layer = J.layer; tile.block0 = J.block0; tile.nblocks = J.nblocks; tile.pad_ = 0;
    LayerDesc L;
    L.elem_off = J.elem_off; L.word_off = J.word_off; L.size = J.size; L.bits = J.bits; L.nlevels = 1 << J.bits;
    L.block_off = J.block_off;
    const int k = kk + p.worker0;
    const int lane = threadIdx.x & 31;
    const int64_t kl = (int64_t)k * p.num_layers + layer;

    // Everything below depends on the job record only, so all of it is requested at once: the norms, this thread's
    // two pieces of the search table, the zero-row masks of its block, the levels of its table entries.
    const float ncur = norms[kl];
    const float nprev = prev_norms ? prev_norms[kl] : 0.0f;
    const float rn = p.rnorm[kl];
    const int search = st.fast[layer];                      // 1: one lookup; 1 + R: byte table and up to R steps
    const uint4* lsrc = reinterpret_cast<const uint4*>(st.lut + (int64_t)layer * kLutEntries);
    const uint4 lut0 = __ldg(lsrc + threadIdx.x), lut1 = __ldg(lsrc + kQThreads + threadIdx.x);
    uint32_t mcur = 0, mprev = 0;
    if (threadIdx.x < tile.nblocks) {
        // a previous message whose masks are unknown is taken as nonzero everywhere
        const int64_t mb = (int64_t)k * p.total_blocks + L.block_off + tile.block0 + threadIdx.x;
        mcur = p.row_mask[mb];
        mprev = (!kStat || !prev_packed) ? 0u : (p.row_mask_prev ? (uint32_t)p.row_mask_prev[mb] : 0xffu);
    }
    float lc = 0.f, lp = 0.f;
    float2 lg = make_float2(0.f, 0.f);
    if (threadIdx.x < L.nlevels) {
        lc = levels_cur[(int64_t)layer * kLevelStride + threadIdx.x];
        lp = levels_prev[(int64_t)layer * kLevelStride + threadIdx.x];
        lg = st.ld[(int64_t)layer * kMaxLevels + threadIdx.x];
    }
    {
        uint4* ldst = reinterpret_cast<uint4*>(sm + kSmLut);
        ldst[threadIdx.x] = lut0;
        ldst[kQThreads + threadIdx.x] = lut1;
        if (threadIdx.x < L.nlevels) {
            const float cv = __fmul_rn(ncur, lc), pv = __fmul_rn(nprev, lp);
            reinterpret_cast<float2*>(sm + kSmLd)[threadIdx.x] = lg;
            reinterpret_cast<float2*>(sm + kSmTcur)[threadIdx.x] = make_float2(cv, -cv);
            reinterpret_cast<float2*>(sm + kSmTprev)[threadIdx.x] = make_float2(pv, -pv);
        }
        if (kHist) {
            uint32_t* h = reinterpret_cast<uint32_t*>(sm + kSmHist);
            for (int i = threadIdx.x; i < LQ_HIST_STRIDE; i += kQThreads) h[i] = 0;
        }
    }
    uint8_t* rows_cur = sm + kSmRows;
    uint8_t* rows_prev = rows_cur + kTileBlocks;
    if (threadIdx.x < tile.nblocks) {
        rows_cur[threadIdx.x] = (uint8_t)mcur;
        rows_prev[threadIdx.x] = (uint8_t)mprev;
    }
    __syncthreads();

    WarpCtx c;
    c.g = grads + (int64_t)kk * p.padded_elems + L.elem_off;
    c.size = L.size;
    c.nfull = L.size / kBlockCoords;
    c.lane = lane;
    QuantEnv ev;
    ev.lut = base + kSmLut; ev.ld = base + kSmLd; ev.tprev = base + kSmTprev;
    ev.r = rn;
    ev.refine = search - 1;
    ev.hist = reinterpret_cast<uint32_t*>(sm + kSmHist);
    const bool zeroed = ev.r == 0.0f;
    if (step == LQ_STEP_AUTO) step = (uint32_t)p.scalars->t;      // the plan's own iteration counter (graph replays)
    const PhiloxConsts pc = philox_fold((uint32_t)layer, (uint32_t)k, step, p.seed_lo, p.seed_hi);
    uint32_t* out = packed + (int64_t)k * p.packed_words + L.word_off;
    const uint32_t* prev = prev_packed ? prev_packed + (int64_t)k * p.packed_words + L.word_off : nullptr;

    double stat = 0.0;
    switch (zeroed ? -L.bits : L.bits * 2 + (search == 1 ? 1 : 0)) {
#define LQ_CASE(BB)                                                                              \
    case -BB:        stat = kStat ? zeroed_tile<BB>(tile, lane, out, prev, ev.tprev)             \
                                  : zeroed_tile<BB>(tile, lane, out, nullptr, ev.tprev); break;  \
    case 2 * BB:     stat = quantize_tile<BB, 2, kHist, kStat>(p, pc, c, tile, out, prev, ev, rows_cur, rows_prev, base + kSmRing); break;  \
    case 2 * BB + 1: stat = quantize_tile<BB, 1, kHist, kStat>(p, pc, c, tile, out, prev, ev, rows_cur, rows_prev, base + kSmRing); break;
        LQ_CASE(1) LQ_CASE(2) LQ_CASE(3) LQ_CASE(4) LQ_CASE(5) LQ_CASE(6) LQ_CASE(7) LQ_CASE(8)
#undef LQ_CASE
        default: break;
    }
    // the layer's last, partial block, if this tile holds it: one warp, after its whole blocks
    {
        const int64_t bp = c.nfull - tile.block0;
        if (!zeroed && (L.size % kBlockCoords) != 0 && bp >= 0 && bp < tile.nblocks && (int)(bp % kQWarps) == (threadIdx.x >> 5)) {
            const double s2 = quantize_partial_block(p, ev, c.g, c.size, c.nfull, L.bits, (uint32_t)layer, (uint32_t)k, step, out,
                                                     kStat ? prev : nullptr, kHist, lane);
            if (kStat) stat += s2;
        }
    }
    const double total = block_reduce<false>(stat, reinterpret_cast<double*>(sm + kSmScratch));
    if (threadIdx.x == 0) p.stat_partial[(int64_t)k * p.num_tiles + tile_id] = total;

    if (kHist) {
        __syncthreads();
        uint32_t* h = hist + kl * LQ_HIST_STRIDE;
        for (int i = threadIdx.x; i < LQ_NUM_BINS; i += blockDim.x)
            if (ev.hist[i]) atomicAdd(h + i, ev.hist[i]);
    }
}

// Adds the per-tile statistic partials of one (layer, worker) in a fixed order.
__global__ void __launch_bounds__(128) stat_finalize_kernel(PlanDev p)
{
    __shared__ double scratch[4];
    const int m = blockIdx.x, k = blockIdx.y + p.worker0;
    const LayerDesc L = p.layers[m];
    const double* part = p.stat_partial + (int64_t)k * p.num_tiles + L.first_tile;
    double acc = 0.0;
    for (int i = threadIdx.x; i < L.ntiles; i += blockDim.x) acc += part[i];
    const double total = block_reduce<false>(acc, scratch);
    if (threadIdx.x == 0) p.sq_diff[(int64_t)k * p.num_layers + m] = total;
}

// One CTA per layer: derives the encode-side tables from the layer's levels.
//   ld[tau]  = {l_tau, l_{tau+1} - l_tau}                 tau = 0..n-2 (other entries: {l_tau, 0})
//   lut[bin] = 8 * tau0 | code << 13    bin = bits(u) >> 19, i.e. the values [lo, hi) with bits(lo) = bin << 19;
//              tau0 = last level (<= n-2) at or below lo; code = (low 19 bits of l_{tau0+1}) - 1 if that level
//              (<= n-2) lies inside the bin, else all ones, so that  (bits(u) << 13) > lut[bin]  iff  u >= l_{tau0+1}
//   fast     = 1: no bin holds two or more levels (then tau is tau0 or tau0 + 1)
// Layers with denser levels (8-bit codes) get a byte table over the top 15 bits instead, in the same 8 KB:
//   lut8[bits(u) >> 17] = tau0 of that finer bin; tau is found by stepping up while l_{tau+1} <= u, at most R times,
//   R = the most levels inside one bin;  fast = 1 + R.
__global__ void __launch_bounds__(256) build_search_kernel(PlanDev p, const float* __restrict__ levels,
                                                           SearchTables t)
{
    __shared__ float lev[kMaxLevels];
    __shared__ int slow, most;
    const int m = blockIdx.x;
    const int n = p.layers[m].nlevels;
    if (threadIdx.x == 0) { slow = 0; most = 0; }
    for (int i = threadIdx.x; i < n; i += blockDim.x) lev[i] = levels[(int64_t)m * kLevelStride + i];
    __syncthreads();
    for (int i = threadIdx.x; i < kMaxLevels; i += blockDim.x) {
        float2 e = make_float2(i < n ? lev[i] : 0.f, 0.f);
        if (i <= n - 2) e.y = __fsub_rn(lev[i + 1], lev[i]);
        t.ld[(int64_t)m * kMaxLevels + i] = e;
    }
    for (int bin = threadIdx.x; bin < kLutEntries; bin += blockDim.x) {
        const uint32_t lob = (uint32_t)bin << 19;
        // bins past 1.0 (and the patterns of Inf / NaN) behave like the bin of 1.0: the last interval
        const bool top = lob >= 0x3f800000u;
        const float lo = __uint_as_float(top ? 0x3f800000u : lob);
        int tau0 = 0;
        for (int j = 1; j <= n - 2; ++j) if (lev[j] <= lo) tau0 = j;
        uint32_t code = 0x7ffffu;
        if (!top && tau0 + 1 <= n - 2) {
            const uint32_t nb = __float_as_uint(lev[tau0 + 1]);
            if ((nb >> 19) == (uint32_t)bin) {                         // l_{tau0+1} > lo lies inside this bin
                code = (nb & 0x7ffffu) - 1u;
                if (tau0 + 2 <= n - 2 && (__float_as_uint(lev[tau0 + 2]) >> 19) == (uint32_t)bin) atomicOr(&slow, 1);
            }
        }
        const uint32_t entry = (code << 13) | (8u * (uint32_t)tau0);
        t.lut[(int64_t)m * kLutEntries + bin] = entry;
    }
    __syncthreads();
    if (slow) {
        uint8_t* lut8 = reinterpret_cast<uint8_t*>(t.lut + (int64_t)m * kLutEntries);
        for (int bin = threadIdx.x; bin < 4 * kLutEntries; bin += blockDim.x) {
            const uint32_t lob = (uint32_t)bin << 17;
            const bool top = lob >= 0x3f800000u;
            const float lo = __uint_as_float(top ? 0x3f800000u : lob);
            int tau0 = 0, inside = 0;
            for (int j = 1; j <= n - 2; ++j) {
                if (lev[j] <= lo) tau0 = j;
                else if (!top && (__float_as_uint(lev[j]) >> 17) == (uint32_t)bin) ++inside;
            }
            lut8[bin] = (uint8_t)tau0;
            atomicMax(&most, inside);
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) t.fast[m] = slow ? 1 + most : 1;
}

cudaError_t launch_build_search(const PlanDev& p, const float* levels, SearchTables t, cudaStream_t s)
{
    if (p.num_layers == 0) return cudaSuccess;
    build_search_kernel<<<(unsigned)p.num_layers, 256, 0, s>>>(p, levels, t);
    return cudaGetLastError();
}

cudaError_t launch_quantize(const PlanDev& p, const float* grads, uint32_t step, uint32_t* packed,
                            const float* norms, uint32_t* hist, const uint32_t* prev_packed,
                            const float* prev_norms, const float* levels_cur,
                            const float* levels_prev, SearchTables t, bool need_stat, cudaStream_t s)
{
    if (p.num_tiles == 0) return cudaSuccess;
    const dim3 grid((unsigned)p.num_tiles, (unsigned)p.worker_count);
    // the ring follows the tables; the histogram (histogram mode only) follows the ring
    constexpr unsigned smem = kSmTables + kRingBytes + kSmSlack, smem_hist = smem + LQ_HIST_STRIDE * 4;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {            // more than 48 KB of dynamic shared memory: opt in once
        cudaError_t e = cudaFuncSetAttribute(quantize_pack_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_hist);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(quantize_pack_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(quantize_pack_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    if (hist)
        quantize_pack_kernel<true, true><<<grid, kQThreads, smem_hist, s>>>(p, grads, step, packed, norms, hist,
                                                                       prev_packed, prev_norms, levels_cur, levels_prev, t);
    else if (need_stat)
        quantize_pack_kernel<false, true><<<grid, kQThreads, smem, s>>>(p, grads, step, packed, norms, hist,
                                                                        prev_packed, prev_norms, levels_cur, levels_prev, t);
    else
        quantize_pack_kernel<false, false><<<grid, kQThreads, smem, s>>>(p, grads, step, packed, norms, hist,
                                                                         prev_packed, prev_norms, levels_cur, levels_prev, t);
    return cudaGetLastError();
}

cudaError_t launch_stat_finalize(const PlanDev& p, cudaStream_t s)
{
    stat_finalize_kernel<<<dim3((unsigned)p.num_layers, (unsigned)p.worker_count), 128, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace lq
