// ENCODE for all workers: normalise, round stochastically between neighbouring levels, pack
// sign + index words (Section 3.1 quantizer, Section 3.2 message; Algorithm 1 line 12), with the
// optional histogram of normalised magnitudes (Algorithm 1 line 4) and the sender-side term of the
// adaptive step size, sum ||V^_{k,t+1/2} - V^_{k,t-1/2}||^2 (Eq. general_stepsize).
//
// Work decomposition: one CTA per (tile, worker); a tile is up to 8 blocks of 1024 coordinates of
// one layer; one warp per block.  A lane owns the 32 coordinates {128 j + 4 lane + e}: it reads
// them as 8 coalesced float4 loads, draws one Philox4x32-10 block per float4 (4 uniforms), and
// ends up with exactly one sign word and b index words, which it stores plane by plane so that a
// warp writes 128 contiguous bytes per plane.  No shuffles, ballots or atomics on the main path.
#include "lq_internal.cuh"

namespace lq {

template <int B>
__device__ __forceinline__ void put_code(uint32_t (&cw)[B], int p, uint32_t idx)
{
    const int off = p * B, w = off >> 5, s = off & 31;
    cw[w] |= idx << s;
    if (s + B > 32) cw[w + 1] |= idx >> (32 - s);
}

template <int B>
__device__ __forceinline__ uint32_t get_code(const uint32_t (&cw)[B], int p)
{
    const int off = p * B, w = off >> 5, s = off & 31;
    uint32_t v = cw[w] >> s;
    if (s + B > 32) v |= cw[w + 1] << (32 - s);
    return v & ((1u << B) - 1u);
}

struct QuantSmem {
    float lev[kMaxLevels];        // levels of this layer used for encoding
    double tcur[kMaxLevels];      // (double) fp32(N_cur * l_j)
    double tprev[kMaxLevels];     // (double) fp32(N_prev * lprev_j)
    uint32_t hist[LQ_HIST_STRIDE];
    double scratch[kThreads / 32];
};

template <int B, bool kHist>
__device__ __forceinline__ double quantize_block(const PlanDev& p, const LayerDesc& L, int layer, int k,
                                                 int64_t blk, const float* __restrict__ g, float r,
                                                 uint32_t step, uint32_t* __restrict__ out,
                                                 const uint32_t* __restrict__ prev, QuantSmem& sm)
{
    constexpr int n = 1 << B;
    const int lane = threadIdx.x & 31;
    const int64_t base = blk * kBlockCoords + 4 * lane;

    float4 v[8];
    if (r == 0.0f) {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    } else if (blk * kBlockCoords + kBlockCoords <= L.size) {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = __ldg(reinterpret_cast<const float4*>(g + base + 128 * j));
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int64_t pos = base + 128 * j;
            v[j].x = pos + 0 < L.size ? __ldg(g + pos + 0) : 0.f;
            v[j].y = pos + 1 < L.size ? __ldg(g + pos + 1) : 0.f;
            v[j].z = pos + 2 < L.size ? __ldg(g + pos + 2) : 0.f;
            v[j].w = pos + 3 < L.size ? __ldg(g + pos + 3) : 0.f;
        }
    }

    uint32_t psign = 0, pcw[B];
    const int64_t woff = blk * (int64_t)(B + 1) * 32 + lane;
    if (prev) {
        psign = __ldg(prev + woff);
#pragma unroll
        for (int w = 0; w < B; ++w) pcw[w] = __ldg(prev + woff + (w + 1) * 32);
    } else {
#pragma unroll
        for (int w = 0; w < B; ++w) pcw[w] = 0;
    }

    uint32_t signw = 0, cw[B];
#pragma unroll
    for (int w = 0; w < B; ++w) cw[w] = 0;
    double stat = 0.0;

#pragma unroll
    for (int j = 0; j < 8; ++j) {
        uint32_t x[4];
        philox4x32_10((uint32_t)(blk * 256 + 32 * j + lane), (uint32_t)layer, (uint32_t)k, step,
                      p.seed_lo, p.seed_hi, x);
        const float vv[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int pp = 4 * j + e;
            const uint32_t bits = __float_as_uint(vv[e]);
            const float u = fminf(__fmul_rn(fabsf(vv[e]), r), 1.0f);
            // tau = largest j <= n-2 with lev[j] <= u
            int tau = 0;
#pragma unroll
            for (int s = B - 1; s >= 0; --s) {
                const int cand = tau + (1 << s);
                if (sm.lev[cand] <= u) tau = cand;
            }
            tau = min(tau, n - 2);
            const float lo = sm.lev[tau], hi = sm.lev[tau + 1];
            const float num = __fsub_rn(u, lo);
            const float den = __fsub_rn(hi, lo);
            const float rho = __fmul_rn(__uint2float_rn(x[e] >> 8), 5.9604644775390625e-08f);
            const uint32_t idx = (uint32_t)tau + (__fmul_rn(rho, den) < num ? 1u : 0u);
            const uint32_t sg = bits >> 31;
            signw |= sg << pp;
            put_code<B>(cw, pp, idx);

            if (kHist) {
                const int64_t pos = base + 128 * j + e;
                if (r != 0.0f && pos < L.size) {
                    const uint32_t ub = __float_as_uint(u);
                    const uint32_t bin = ub < 0x33800000u ? 0u : 1u + ((ub - 0x33800000u) >> 19);
                    atomicAdd(&sm.hist[bin], 1u);
                }
            }

            // step-size statistic: exact fp64 difference of the two fp32 decoded values
            double cur = sm.tcur[idx];
            cur = sg ? -cur : cur;
            double prv = sm.tprev[get_code<B>(pcw, pp)];
            prv = ((psign >> pp) & 1u) ? -prv : prv;
            const double dd = cur - prv;
            stat = fma(dd, dd, stat);
        }
    }

    out[woff] = signw;
#pragma unroll
    for (int w = 0; w < B; ++w) out[woff + (w + 1) * 32] = cw[w];
    return stat;
}

template <bool kHist>
__global__ void __launch_bounds__(kThreads) quantize_pack_kernel(
    PlanDev p, const float* __restrict__ grads, uint32_t step, uint32_t* __restrict__ packed,
    const float* __restrict__ norms, uint32_t* __restrict__ hist,
    const uint32_t* __restrict__ prev_packed, const float* __restrict__ prev_norms,
    const float* __restrict__ levels_cur, const float* __restrict__ levels_prev)
{
    __shared__ QuantSmem sm;
    const Tile tile = p.tiles[blockIdx.x];
    const int layer = tile.layer;
    const LayerDesc L = p.layers[layer];
    const int k = blockIdx.y;
    const int warp = threadIdx.x >> 5;
    const int64_t kl = (int64_t)k * p.num_layers + layer;
    const float r = p.rnorm[kl];
    const float ncur = norms[kl];
    const float nprev = prev_norms ? prev_norms[kl] : 0.0f;

    for (int i = threadIdx.x; i < L.nlevels; i += blockDim.x) {
        const float l = levels_cur[(int64_t)layer * kLevelStride + i];
        sm.lev[i] = l;
        sm.tcur[i] = (double)__fmul_rn(ncur, l);
        sm.tprev[i] = (double)__fmul_rn(nprev, levels_prev[(int64_t)layer * kLevelStride + i]);
    }
    if (kHist)
        for (int i = threadIdx.x; i < LQ_HIST_STRIDE; i += blockDim.x) sm.hist[i] = 0;
    __syncthreads();

    const float* g = grads + (int64_t)k * p.padded_elems + L.elem_off;
    uint32_t* out = packed + (int64_t)k * p.packed_words + L.word_off;
    const uint32_t* prev = prev_packed ? prev_packed + (int64_t)k * p.packed_words + L.word_off : nullptr;

    double stat = 0.0;
    if (warp < tile.nblocks) {
        const int64_t blk = tile.block0 + warp;
        switch (L.bits) {
#define LQ_CASE(BB) case BB: stat = quantize_block<BB, kHist>(p, L, layer, k, blk, g, r, step, out, prev, sm); break;
            LQ_CASE(1) LQ_CASE(2) LQ_CASE(3) LQ_CASE(4) LQ_CASE(5) LQ_CASE(6) LQ_CASE(7) LQ_CASE(8)
#undef LQ_CASE
            default: break;
        }
    }
    const double total = block_reduce<false>(stat, sm.scratch);
    if (threadIdx.x == 0) p.stat_partial[(int64_t)k * p.num_tiles + blockIdx.x] = total;

    if (kHist) {
        __syncthreads();
        uint32_t* h = hist + kl * LQ_HIST_STRIDE;
        for (int i = threadIdx.x; i < LQ_NUM_BINS; i += blockDim.x)
            if (sm.hist[i]) atomicAdd(h + i, sm.hist[i]);
    }
}

// Adds the per-tile statistic partials of one (layer, worker) in a fixed order.
__global__ void __launch_bounds__(128) stat_finalize_kernel(PlanDev p)
{
    __shared__ double scratch[4];
    const int m = blockIdx.x, k = blockIdx.y;
    const LayerDesc L = p.layers[m];
    const double* part = p.stat_partial + (int64_t)k * p.num_tiles + L.first_tile;
    double acc = 0.0;
    for (int i = threadIdx.x; i < L.ntiles; i += blockDim.x) acc += part[i];
    const double total = block_reduce<false>(acc, scratch);
    if (threadIdx.x == 0) p.sq_diff[(int64_t)k * p.num_layers + m] = total;
}

cudaError_t launch_quantize(const PlanDev& p, const float* grads, uint32_t step, uint32_t* packed,
                            const float* norms, uint32_t* hist, const uint32_t* prev_packed,
                            const float* prev_norms, const float* levels_cur,
                            const float* levels_prev, cudaStream_t s)
{
    if (p.num_tiles > 0) {
        const dim3 grid((unsigned)p.num_tiles, (unsigned)p.num_workers);
        if (hist)
            quantize_pack_kernel<true><<<grid, kThreads, 0, s>>>(p, grads, step, packed, norms, hist,
                                                                 prev_packed, prev_norms, levels_cur, levels_prev);
        else
            quantize_pack_kernel<false><<<grid, kThreads, 0, s>>>(p, grads, step, packed, norms, hist,
                                                                  prev_packed, prev_norms, levels_cur, levels_prev);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    stat_finalize_kernel<<<dim3((unsigned)p.num_layers, (unsigned)p.num_workers), 128, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace lq
