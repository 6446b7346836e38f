// DECODE + aggregate of the K workers' messages, alone or fused with the optimistic dual averaging
// update (Algorithm 1 lines 15-18 and line 10 of the next iteration; Eq. ODA; Eq. general_stepsize).
//
// One CTA per sub-tile (up to 32 blocks of 1024 coordinates of one layer, taken round-robin by 8 warps).  A lane
// owns the same 32 coordinates it owned at encode time, so it reads (b+1) words per worker with
// 128-byte coalesced warp loads, looks the signed decoded values up by symbol in a per-(worker, layer) table in shared
// memory, sums them in worker order in registers, and finishes with float4 reads of Y and X_1 and
// float4 writes of Y and X_{t+3/2}.  Every packed word and every state element is touched once.
#include "lq_internal.cuh"

namespace lq {

constexpr int kWorkerChunk = 8;   // workers whose value tables sit in shared memory at once
#ifndef LQ_DEC_PARTS
#define LQ_DEC_PARTS 2
#endif
#ifndef LQ_DEC_CTAS
#define LQ_DEC_CTAS 4
#endif
constexpr int kParts = LQ_DEC_PARTS;            // a block is decoded in kParts pieces of 8 / kParts rows
constexpr int kPartSyms = 32 / kParts;          // symbols of a lane per piece
constexpr int kPartRows = 8 / kParts;
constexpr int kStageBytes = kWarps * 2 * kPartRows * 512;   // per CTA: each warp stages its piece's rows of Y and X_1


// Adds up to kWorkerChunk workers' decoded half blocks into acc, in worker order.  Half H of a lane's
// string holds its symbols 16 H .. 16 H + 15 (rows 4 H .. 4 H + 3 of the block); only the words that
// carry those symbols are read.  All workers' words are requested before the first one is used, so
// that a warp keeps a few KB in flight.  `table[kk]` holds N * l_j at 2j and -N * l_j at 2j + 1 for
// worker kk of the chunk.  Bucket scope: table[0] holds the plain signed levels for every worker, and `bn` points
// at worker k0's norms of this piece's rows (one per row of 128 coordinates; the next worker's `bn_stride` further).
template <int B, int H, bool kBucket>
__device__ __forceinline__ void decode_accumulate(float (&acc)[kPartSyms], const uint32_t* __restrict__ words,
                                                  int64_t worker_stride, int kc,
                                                  const float (*table)[2 * kMaxLevels],
                                                  const float* __restrict__ bn, int64_t bn_stride, uint32_t live)
{
    // `live`: bit kk clear = worker kk's block is known to be all zero words, which are then not read (their
    // symbols are 0 and add the table's +0)
    constexpr int C = B + 1;
    constexpr int kFirst = (kPartSyms * H * C) >> 5;                  // first and last word of this piece
    constexpr int kLast = ((kPartSyms * (H + 1) * C) - 1) >> 5;
    uint32_t w[kWorkerChunk][C];
#pragma unroll
    for (int kk = 0; kk < kWorkerChunk; ++kk)
#pragma unroll
        for (int i = 0; i < C; ++i)
            w[kk][i] = (i >= kFirst && i <= kLast && kk < kc && ((live >> kk) & 1u)) ? __ldcs(words + kk * worker_stride + i * 32) : 0u;
    float nr[kBucket ? kWorkerChunk : 1][kPartRows];
    if (kBucket) {
#pragma unroll
        for (int kk = 0; kk < kWorkerChunk; ++kk)
#pragma unroll
            for (int jj = 0; jj < kPartRows; ++jj) nr[kk][jj] = kk < kc ? __ldg(bn + kk * bn_stride + jj) : 0.0f;
    }
#pragma unroll
    for (int kk = 0; kk < kWorkerChunk; ++kk) {
        if (kk < kc) {
            const char* tb = reinterpret_cast<const char*>(table[kBucket ? 0 : kk]);
#pragma unroll
            for (int p = 0; p < kPartSyms; ++p) {
                const float val = *reinterpret_cast<const float*>(tb + symbol4_at<C>(w[kk], kPartSyms * H + p));
                acc[p] += kBucket ? __fmul_rn(val, nr[kk][p >> 2]) : val;
            }
        }
    }
}

// The rates one QODA update uses: X_{t+1} = X_1 + eta Y_{t+1}, X_{t+3/2} = X_{t+1} - gamma gbar; eta_cur made X_t.
struct Rates { float eta, gamma, eta_cur; };

struct DecodeArgs {
    const uint32_t* live;    // per block of 1024 coordinates: bit k set = worker k's words are not all zero; or nullptr
    const uint32_t* packed;
    const float* norms;
    const float* levels;
    const float* X1;
    float* Y;
    float* Xhalf;
    float* X;
    float* gbar;
};

// Fills the value tables of workers k0 .. k0 + kc - 1 of one layer (CTA-wide, between two barriers); in bucket
// scope one table of plain signed levels.
template <bool kBucket>
__device__ __forceinline__ void fill_tables(const PlanDev& p, const LayerDesc& L, int layer, const DecodeArgs& a,
                                            float (*table)[2 * kMaxLevels], int k0, int kc)
{
    __syncthreads();
    for (int i = threadIdx.x; i < (kBucket ? 1 : kc) * L.nlevels; i += blockDim.x) {
        const int kk = i / L.nlevels, j = i - kk * L.nlevels;
        const float lv = a.levels[(int64_t)layer * kLevelStride + j];
        const float mag = kBucket ? lv : __fmul_rn(a.norms[(int64_t)(k0 + kk) * p.num_layers + layer], lv);
        table[kk][2 * j] = mag;                       // symbol = 2 * idx + sign
        table[kk][2 * j + 1] = -mag;
    }
    __syncthreads();
}

// One half block: the mean of the K decoded messages for rows 4 H .. 4 H + 3, then the update.
// Any worker count: the accumulators live across chunks of kWorkerChunk workers; with a single chunk
// the tables are filled once per CTA (`resident`).
template <int B, int H, int kMode, bool kBucket>
__device__ __forceinline__ void decode_half(const PlanDev& p, const LayerDesc& L, int layer, const DecodeArgs& a,
                                            float (*table)[2 * kMaxLevels], const Rates& rt, float invK,
                                            int64_t blk, bool active, bool& resident, float4* stage,
                                            double& lam_acc, double& mu_acc, uint32_t block_live)
{
    constexpr bool kQoda = kMode >= 1, kAlt = kMode == 2;
    const float eta = rt.eta, gamma = rt.gamma;
    const int lane = threadIdx.x & 31;
    const int K = p.num_workers;
    const int64_t woff = L.word_off + blk * (int64_t)(B + 1) * 32 + lane;
    const int64_t base = L.elem_off + blk * kBlockCoords + 4 * lane;
    const int64_t limit = L.elem_off + L.size;
    // the state rows of this piece travel to shared memory while the messages are read and decoded
    // (`stage`: this lane's slots, rows of Y then rows of X_1, 32 float4 apart; only this lane reads them)
    if (kQoda && active) {
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(stage);
#pragma unroll
        for (int jj = 0; jj < kPartRows; ++jj) {
            const int64_t pos = base + 128 * (kPartRows * H + jj);
            if (pos < limit) {
                cp_async16(dst + 512u * jj, a.Y + pos, 16);
                cp_async16(dst + 512u * (kPartRows + jj), a.X1 + pos, 16);
            }
        }
        cp_async_commit();
    }
    float acc[kPartSyms];
#pragma unroll
    for (int i = 0; i < kPartSyms; ++i) acc[i] = 0.0f;
    for (int k0 = 0; k0 < K; k0 += kWorkerChunk) {
        const int kc = min(kWorkerChunk, K - k0);
        // the chunk's workers in the low bits; the masks cover at most 32 workers, and beyond that (masks unknown,
        // block_live all ones) every word is read: a shift by 32 or more is not defined
        const uint32_t live = k0 < 32 ? block_live >> k0 : 0xffffffffu;
        if (!resident) fill_tables<kBucket>(p, L, layer, a, table, k0, kc);
        if (kBucket || K <= kWorkerChunk) resident = true;
        const int64_t bn_stride = p.total_blocks * 8;
        const float* bn = kBucket ? a.norms + (int64_t)k0 * bn_stride + (L.block_off + blk) * 8 + kPartRows * H : nullptr;
        if (active) decode_accumulate<B, H, kBucket>(acc, a.packed + (int64_t)k0 * p.packed_words + woff, p.packed_words,
                                                     kc, table, bn, bn_stride, live);
    }
    if (!active) return;
    if (kQoda) cp_async_wait<0>();
#pragma unroll
    for (int jj = 0; jj < kPartRows; ++jj) {
        const int64_t pos = base + 128 * (kPartRows * H + jj);
        if (pos >= limit) continue;
        float4 g;
        g.x = __fmul_rn(acc[4 * jj + 0], invK);
        g.y = __fmul_rn(acc[4 * jj + 1], invK);
        g.z = __fmul_rn(acc[4 * jj + 2], invK);
        g.w = __fmul_rn(acc[4 * jj + 3], invK);
        if (a.gbar) *reinterpret_cast<float4*>(a.gbar + pos) = g;
        if (kQoda) {
            const float4 y0 = stage[32 * jj];
            const float4 x1 = stage[32 * (kPartRows + jj)];
            float4 y, x, h;
            y.x = __fsub_rn(y0.x, g.x); y.y = __fsub_rn(y0.y, g.y);
            y.z = __fsub_rn(y0.z, g.z); y.w = __fsub_rn(y0.w, g.w);
            x.x = fmaf(eta, y.x, x1.x); x.y = fmaf(eta, y.y, x1.y);
            x.z = fmaf(eta, y.z, x1.z); x.w = fmaf(eta, y.w, x1.w);
            h.x = fmaf(-gamma, g.x, x.x); h.y = fmaf(-gamma, g.y, x.y);
            h.z = fmaf(-gamma, g.z, x.z); h.w = fmaf(-gamma, g.w, x.w);
            if (kAlt) {
                // this iteration's terms of lambda = sum ||gbar||^2 and mu = sum ||X_t - X_{t+1}||^2, with
                // X_t recomputed from Y_t and the rate that produced it; padding coordinates do not count
                const float gv[4] = {g.x, g.y, g.z, g.w};
                const float dv[4] = {__fsub_rn(fmaf(rt.eta_cur, y0.x, x1.x), x.x), __fsub_rn(fmaf(rt.eta_cur, y0.y, x1.y), x.y),
                                     __fsub_rn(fmaf(rt.eta_cur, y0.z, x1.z), x.z), __fsub_rn(fmaf(rt.eta_cur, y0.w, x1.w), x.w)};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (pos + e < limit) {
                        const double gd = (double)gv[e], dd = (double)dv[e];
                        lam_acc = fma(gd, gd, lam_acc);
                        mu_acc = fma(dd, dd, mu_acc);
                    }
                }
            }
            if (block_live) *reinterpret_cast<float4*>(a.Y + pos) = y;   // no worker sent anything here: y = y0 - 0
            *reinterpret_cast<float4*>(a.Xhalf + pos) = h;
            if (a.X) *reinterpret_cast<float4*>(a.X + pos) = x;
        }
    }
}

template <int B, int kMode, bool kBucket>
__device__ __forceinline__ void decode_block_chunked(const PlanDev& p, const LayerDesc& L, int layer,
                                                     const Tile& tile, const DecodeArgs& a,
                                                     float (*table)[2 * kMaxLevels], const Rates& rt,
                                                     double& lam_acc, double& mu_acc)
{
    const int warp = threadIdx.x >> 5;
    const float invK = __fdiv_rn(1.0f, (float)p.num_workers);
    bool resident = false;
    extern __shared__ float4 stage_mem[];                 // [warp][Y rows, X_1 rows][lane]
    float4* stage = stage_mem + warp * (2 * kPartRows * 32) + (threadIdx.x & 31);
    // each warp takes the tile's blocks round-robin; all warps run the same number of rounds so
    // that the table refills (CTA-wide barriers) stay aligned
    for (int b0 = 0; b0 < tile.nblocks; b0 += kWarps) {
        const bool active = b0 + warp < tile.nblocks;
        const int64_t blk = tile.block0 + b0 + warp;
        // which workers sent anything in this block (all of them when that is not known)
        const uint32_t block_live = (!kBucket && a.live && active) ? __ldg(a.live + L.block_off + blk) : 0xffffffffu;
        decode_half<B, 0, kMode, kBucket>(p, L, layer, a, table, rt, invK, blk, active, resident, stage, lam_acc, mu_acc, block_live);
        decode_half<B, 1, kMode, kBucket>(p, L, layer, a, table, rt, invK, blk, active, resident, stage, lam_acc, mu_acc, block_live);
        if (kParts == 4) {
            decode_half<B, 2 % kParts, kMode, kBucket>(p, L, layer, a, table, rt, invK, blk, active, resident, stage, lam_acc, mu_acc, block_live);
            decode_half<B, 3 % kParts, kMode, kBucket>(p, L, layer, a, table, rt, invK, blk, active, resident, stage, lam_acc, mu_acc, block_live);
        }
    }
}

template <int kMode, bool kBucket>
__global__ void __launch_bounds__(kThreads, kBucket ? 2 : (kMode == 2 ? 3 : LQ_DEC_CTAS)) decode_kernel(PlanDev p, DecodeArgs a)
{
    __shared__ float table[kWorkerChunk][2 * kMaxLevels];
    constexpr bool kAlt = kMode == 2;
    const int ncta = p.num_tiles * p.sub_tiles;
    Tile tile = p.tiles[blockIdx.x >> p.sub_shift];                    // this CTA takes one sub-tile of it
    const int sub0 = (blockIdx.x & (p.sub_tiles - 1)) * kSubBlocks;
    if (sub0 >= tile.nblocks) {
        if (kAlt && threadIdx.x == 0) { p.alt_partial[blockIdx.x] = 0.0; p.alt_partial[ncta + blockIdx.x] = 0.0; }
        return;
    }
    tile.block0 += sub0;
    tile.nblocks = min(kSubBlocks, tile.nblocks - sub0);
    const int layer = tile.layer;
    const LayerDesc L = p.layers[layer];
    Rates rt{0.0f, 0.0f, 0.0f};
    if (kMode >= 1) {
        rt.eta = p.scalars->eta;
        rt.gamma = kAlt ? p.scalars->gamma : rt.eta;
        rt.eta_cur = kAlt ? p.scalars->eta_cur : 0.0f;
    }
    double lam_acc = 0.0, mu_acc = 0.0;

    switch (L.bits) {
#define LQ_CASE(BB) case BB: decode_block_chunked<BB, kMode, kBucket>(p, L, layer, tile, a, table, rt, lam_acc, mu_acc); break;
        LQ_CASE(1) LQ_CASE(2) LQ_CASE(3) LQ_CASE(4) LQ_CASE(5) LQ_CASE(6) LQ_CASE(7) LQ_CASE(8)
#undef LQ_CASE
        default: break;
    }
    if (kAlt) {                                  // one term per CTA, added in CTA order by the finalize kernel
        double* scratch = reinterpret_cast<double*>(&table[0][0]);   // the tables are no longer needed (the
                                                                     // reduction starts with a barrier)
        const double lam = block_reduce<false>(lam_acc, scratch);
        const double mu = block_reduce<false>(mu_acc, scratch);
        if (threadIdx.x == 0) { p.alt_partial[blockIdx.x] = lam; p.alt_partial[ncta + blockIdx.x] = mu; }
    }
}

// Eq. (Alt), before the update of iteration t: eta_{t+1} and gamma_{t+1} from the sums through iteration t-1.
__global__ void alt_scalars_kernel(PlanDev p, double qhat)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        QodaScalars* q = p.scalars;
        q->eta_cur = q->eta;
        q->eta = (float)(1.0 / sqrt(1.0 + q->lambda + q->mu));
        q->gamma = (float)pow(1.0 + q->lambda, qhat - 0.5);
        q->t = q->t + 1;
    }
}

// Eq. (Alt), after the update: adds the CTAs' terms of this iteration to lambda and mu in a fixed order.
__global__ void __launch_bounds__(256) alt_finalize_kernel(PlanDev p)
{
    __shared__ double scratch[8];
    const int n = p.num_tiles * p.sub_tiles;
    double lam = 0.0, mu = 0.0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) { lam += p.alt_partial[i]; mu += p.alt_partial[n + i]; }
    const double lam_t = block_reduce<false>(lam, scratch);
    const double mu_t = block_reduce<false>(mu, scratch);
    if (threadIdx.x == 0) { p.scalars->lambda += lam_t; p.scalars->mu += mu_t; }
}

// S_t = S_{t-1} + (sum over workers and layers of the squared differences) / K^2,
// eta_{t+1} = fp32((1 + S_t)^(-1/2)); one CTA, fixed summation order.
__global__ void __launch_bounds__(256) qoda_scalars_kernel(PlanDev p)
{
    __shared__ double scratch[8];
    const int n = p.num_workers * p.num_layers;
    double acc = 0.0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) acc += p.sq_diff[i];
    const double total = block_reduce<false>(acc, scratch);
    if (threadIdx.x == 0) {
        QodaScalars* q = p.scalars;
        const double K = (double)p.num_workers;
        const double delta = total / (K * K);
        q->last_delta = delta;
        q->S = q->S + delta;
        q->eta = (float)(1.0 / sqrt(1.0 + q->S));
        q->gamma = q->eta;
        q->t = q->t + 1;
    }
}

__global__ void qoda_init_kernel(PlanDev p, const float* __restrict__ X1, float* __restrict__ Y,
                                 float* __restrict__ Xhalf)
{
    const int64_t n4 = p.padded_elems / 4;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4;
         i += (int64_t)gridDim.x * blockDim.x) {
        reinterpret_cast<float4*>(Y)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        reinterpret_cast<float4*>(Xhalf)[i] = reinterpret_cast<const float4*>(X1)[i];
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        QodaScalars* q = p.scalars;
        q->S = 0.0; q->last_delta = 0.0; q->t = 1; q->eta = 1.0f;
        q->gamma = 1.0f; q->eta_cur = 1.0f; q->lambda = 0.0; q->mu = 0.0;
    }
}

// xsum += Xhalf in fp64 (the running sum behind the ergodic average of the half iterates)
__global__ void __launch_bounds__(256) average_kernel(const float* __restrict__ Xhalf, double* __restrict__ xsum, int64_t n4)
{
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
        const float4 x = __ldcs(reinterpret_cast<const float4*>(Xhalf) + i);
        double2 a = reinterpret_cast<double2*>(xsum)[2 * i], b = reinterpret_cast<double2*>(xsum)[2 * i + 1];
        a.x += (double)x.x; a.y += (double)x.y; b.x += (double)x.z; b.y += (double)x.w;
        reinterpret_cast<double2*>(xsum)[2 * i] = a;
        reinterpret_cast<double2*>(xsum)[2 * i + 1] = b;
    }
}

cudaError_t launch_average(const PlanDev& p, const float* Xhalf, double* xsum, cudaStream_t s)
{
    const int64_t n4 = p.padded_elems / 4;
    const unsigned blocks = (unsigned)((n4 + 255) / 256 < 148 * 16 ? (n4 + 255) / 256 + 1 : 148 * 16);
    average_kernel<<<blocks, 256, 0, s>>>(Xhalf, xsum, n4);
    return cudaGetLastError();
}

cudaError_t launch_decode(const PlanDev& p, const uint32_t* packed, const float* norms,
                          const float* levels, const float* X1, float* Y, float* Xhalf, float* X,
                          float* gbar, int mode, const uint32_t* live, cudaStream_t s)
{
    if (p.num_tiles == 0) return cudaSuccess;
    DecodeArgs a{live, packed, norms, levels, X1, Y, Xhalf, X, gbar};
    const unsigned grid = (unsigned)p.num_tiles * p.sub_tiles;
    if (p.bucket_norm) {
        if (mode == 2)      decode_kernel<2, true><<<grid, kThreads, kStageBytes, s>>>(p, a);
        else if (mode == 1) decode_kernel<1, true><<<grid, kThreads, kStageBytes, s>>>(p, a);
        else                decode_kernel<0, true><<<grid, kThreads, kStageBytes, s>>>(p, a);
    } else {
        if (mode == 2)      decode_kernel<2, false><<<grid, kThreads, kStageBytes, s>>>(p, a);
        else if (mode == 1) decode_kernel<1, false><<<grid, kThreads, kStageBytes, s>>>(p, a);
        else                decode_kernel<0, false><<<grid, kThreads, kStageBytes, s>>>(p, a);
    }
    return cudaGetLastError();
}

// block_live[b] = bitmask of the workers whose block b holds a nonzero value, from the K zero-row mask arrays
__global__ void __launch_bounds__(256) block_live_kernel(PlanDev p)
{
    const int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (b >= p.total_blocks) return;
    uint32_t m = 0;
    for (int k = 0; k < p.num_workers; ++k) m |= (p.row_mask[(int64_t)k * p.total_blocks + b] != 0 ? 1u : 0u) << k;
    p.block_live[b] = m;
}

cudaError_t launch_block_live(const PlanDev& p, cudaStream_t s)
{
    if (p.total_blocks == 0) return cudaSuccess;
    block_live_kernel<<<(unsigned)((p.total_blocks + 255) / 256), 256, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_alt_scalars(const PlanDev& p, double qhat, cudaStream_t s)
{
    alt_scalars_kernel<<<1, 32, 0, s>>>(p, qhat);
    return cudaGetLastError();
}

cudaError_t launch_alt_finalize(const PlanDev& p, cudaStream_t s)
{
    if (p.num_tiles == 0) return cudaSuccess;
    alt_finalize_kernel<<<1, 256, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_qoda_scalars(const PlanDev& p, cudaStream_t s)
{
    qoda_scalars_kernel<<<1, 256, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_qoda_init(const PlanDev& p, const float* X1, float* Y, float* Xhalf, cudaStream_t s)
{
    const int64_t n4 = p.padded_elems / 4;
    const unsigned blocks = (unsigned)((n4 + 255) / 256 < 148 * 8 ? (n4 + 255) / 256 + 1 : 148 * 8);
    qoda_init_kernel<<<blocks, 256, 0, s>>>(p, X1, Y, Xhalf);
    return cudaGetLastError();
}

}  // namespace lq
