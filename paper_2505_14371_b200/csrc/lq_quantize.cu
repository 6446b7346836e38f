// ENCODE for all workers: normalise, round stochastically between neighbouring levels, pack one
// (b+1)-bit symbol per coordinate (Section 3.1 quantizer, Section 3.2 message; Algorithm 1 line 12),
// with the optional histogram of normalised magnitudes (Algorithm 1 line 4) and the sender-side
// term of the adaptive step size, sum ||V^_{k,t+1/2} - V^_{k,t-1/2}||^2 (Eq. general_stepsize).
//
// Work decomposition: one CTA per (tile, worker); a tile is up to 32 blocks of 1024 coordinates of
// one layer, taken round-robin by the 8 warps.  A lane owns the 32 coordinates {128 j + 4 lane + e}
// of a block: it reads them as 8 coalesced float4 loads, draws one Philox4x32-10 block per float4
// (4 uniforms) and ends up with exactly b+1 words of symbols, which it stores plane by plane so
// that a warp writes 128 contiguous bytes per plane.  No shuffles, ballots or atomics on the
// main path.
//
// The level search uses a table over the 386 histogram bins of u (exponent + 4 mantissa bits):
// each entry names the last level at or below the bin's lower edge and the single level that may
// lie inside the bin, so tau costs one shared-memory load and one compare.  Layers whose levels
// are denser than the bins fall back to a binary search.  All byte offsets are kept pre-scaled by
// 8 so that the same register indexes the {level, gap} table and the fp64 value tables.
#include "lq_internal.cuh"

namespace lq {

struct QuantSmem {
    uint2 lut[kLutStride];           // search table of this layer
    float2 ld[kMaxLevels];           // {l_tau, (l_{tau+1}-l_tau) * 2^-24}
    float lev[kMaxLevels];           // plain levels (binary-search path)
    double tcur[2 * kMaxLevels];     // (double) fp32(N_cur * l_j), second half negated
    double tprev[2 * kMaxLevels];    // same for the previous message
    uint32_t hist[LQ_HIST_STRIDE];
    double scratch[kWarps];
};

// symbol p (pre-scaled by 8) of a lane's string of 32 symbols of C bits, held in C words
template <int C>
__device__ __forceinline__ uint32_t symbol8_at(const uint32_t (&w)[C], int p)
{
    const int off = p * C, i = off >> 5, s = off & 31;
    constexpr uint32_t mask8 = ((1u << C) - 1u) << 3;
    uint32_t v;
    if (s + C <= 32) v = s >= 3 ? (w[i] >> (s - 3)) : (w[i] << (3 - s));
    else             v = __funnelshift_r(w[i], w[i + 1], s - 3);      // s >= 3 whenever a symbol straddles
    return v & mask8;
}

template <int C>
__device__ __forceinline__ void put_symbol8(uint32_t (&w)[C], int p, uint32_t sym8)
{
    const int off = p * C, i = off >> 5, s = off & 31;
    w[i] += s >= 3 ? (sym8 << (s - 3)) : (sym8 >> (3 - s));           // fields never overlap: + is |
    if (s + C > 32) w[i + 1] = sym8 >> (35 - s);
}

template <int B, bool kFast, bool kHist>
__device__ __forceinline__ double quantize_block(const PlanDev& p, const LayerDesc& L, int layer, int k,
                                                 int64_t blk, const float* __restrict__ g, float r,
                                                 uint32_t step, uint32_t* __restrict__ out,
                                                 const uint32_t* __restrict__ prev, QuantSmem& sm)
{
    constexpr int n = 1 << B, C = B + 1;
    const int lane = threadIdx.x & 31;
    const int64_t base = blk * kBlockCoords + 4 * lane;

    float4 v[8];
    if (r == 0.0f) {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    } else if (blk * kBlockCoords + kBlockCoords <= L.size) {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = __ldcs(reinterpret_cast<const float4*>(g + base + 128 * j));
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

    const int64_t woff = blk * (int64_t)C * 32 + lane;
    uint32_t pw[C], cw[C];
#pragma unroll
    for (int w = 0; w < C; ++w) { pw[w] = prev ? __ldcs(prev + woff + w * 32) : 0u; cw[w] = 0u; }

    const char* lut_b = reinterpret_cast<const char*>(sm.lut) - (kLutClamp >> 16);
    const char* ld_b = reinterpret_cast<const char*>(sm.ld);
    const char* tcur_b = reinterpret_cast<const char*>(sm.tcur);
    const char* tprev_b = reinterpret_cast<const char*>(sm.tprev);
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
            // u <= 1 + 2^-23 always (N >= |v| and one rounding each in 1/N and the product), and
            // such a u behaves exactly like u = 1 below, so the min(u, 1) of the definition is not needed
            const float u = __fmul_rn(fabsf(vv[e]), r);
            const uint32_t ub = __float_as_uint(u);
            uint32_t t8;
            if (kFast) {
                const uint32_t off = (max(ub, kLutClamp) >> 16) & ~7u;
                const uint2 en = *reinterpret_cast<const uint2*>(lut_b + off);
                t8 = en.x + (u >= __uint_as_float(en.y) ? 8u : 0u);
            } else {
                int tau = 0;
#pragma unroll
                for (int s = B - 1; s >= 0; --s) {
                    const int cand = tau + (1 << s);
                    if (sm.lev[cand] <= u) tau = cand;
                }
                t8 = 8u * (uint32_t)min(tau, n - 2);
            }
            const float2 ld = *reinterpret_cast<const float2*>(ld_b + t8);
            const float num = __fsub_rn(u, ld.x);
            const float rho = __uint2float_rn(x[e] >> 8);                 // 2^24 * uniform, exact
            const uint32_t i8 = t8 + (__fmul_rn(rho, ld.y) < num ? 8u : 0u);
            const uint32_t sym8 = i8 + (bits >> 31) * (8u * n);
            put_symbol8<C>(cw, pp, sym8);

            if (kHist) {
                const int64_t pos = base + 128 * j + e;
                if (r != 0.0f && pos < L.size)
                    atomicAdd(&sm.hist[(max(ub, kLutClamp) - kLutClamp) >> 19], 1u);
            }

            // step-size statistic: exact fp64 difference of the two fp32 decoded values
            const double cur = *reinterpret_cast<const double*>(tcur_b + sym8);
            const double prv = *reinterpret_cast<const double*>(tprev_b + symbol8_at<C>(pw, pp));
            const double dd = cur - prv;
            stat = fma(dd, dd, stat);
        }
    }
#pragma unroll
    for (int w = 0; w < C; ++w) __stcs(out + woff + w * 32, cw[w]);
    return stat;
}

template <bool kHist>
__global__ void __launch_bounds__(kThreads) quantize_pack_kernel(
    PlanDev p, const float* __restrict__ grads, uint32_t step, uint32_t* __restrict__ packed,
    const float* __restrict__ norms, uint32_t* __restrict__ hist,
    const uint32_t* __restrict__ prev_packed, const float* __restrict__ prev_norms,
    const float* __restrict__ levels_cur, const float* __restrict__ levels_prev, SearchTables st)
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
    const bool fast = st.fast[layer] != 0;
    const int n = L.nlevels;

    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const float l = levels_cur[(int64_t)layer * kLevelStride + i];
        const double c = (double)__fmul_rn(ncur, l);
        const double q = (double)__fmul_rn(nprev, levels_prev[(int64_t)layer * kLevelStride + i]);
        sm.lev[i] = l;
        sm.ld[i] = st.ld[(int64_t)layer * kMaxLevels + i];
        sm.tcur[i] = c;  sm.tcur[n + i] = -c;
        sm.tprev[i] = q; sm.tprev[n + i] = -q;
    }
    if (fast)
        for (int i = threadIdx.x; i < LQ_NUM_BINS; i += blockDim.x)
            sm.lut[i] = st.lut[(int64_t)layer * kLutStride + i];
    if (kHist)
        for (int i = threadIdx.x; i < LQ_HIST_STRIDE; i += blockDim.x) sm.hist[i] = 0;
    __syncthreads();

    const float* g = grads + (int64_t)k * p.padded_elems + L.elem_off;
    uint32_t* out = packed + (int64_t)k * p.packed_words + L.word_off;
    const uint32_t* prev = prev_packed ? prev_packed + (int64_t)k * p.packed_words + L.word_off : nullptr;

    double stat = 0.0;
    for (int b = warp; b < tile.nblocks; b += kWarps) {
        const int64_t blk = tile.block0 + b;
        switch (L.bits * 2 + (fast ? 1 : 0)) {
#define LQ_CASE(BB)                                                                                       \
    case 2 * BB:     stat += quantize_block<BB, false, kHist>(p, L, layer, k, blk, g, r, step, out, prev, sm); break; \
    case 2 * BB + 1: stat += quantize_block<BB, true, kHist>(p, L, layer, k, blk, g, r, step, out, prev, sm); break;
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

// One CTA per layer: derives the encode-side tables from the layer's levels.
//   ld[tau]  = {l_tau, (l_{tau+1} - l_tau) * 2^-24}       tau = 0..n-2
//   lut[bin] = {8 * tau0, bits of l_{tau0+1} if it lies inside the bin, else +inf}
//              tau0 = last level (<= n-2) at or below the bin's lower edge
//   fast     = no bin holds two or more levels (then tau is tau0 or tau0 + 1)
__global__ void __launch_bounds__(128) build_search_kernel(PlanDev p, const float* __restrict__ levels,
                                                           SearchTables t)
{
    __shared__ float lev[kMaxLevels];
    __shared__ int slow;
    const int m = blockIdx.x;
    const int n = p.layers[m].nlevels;
    if (threadIdx.x == 0) slow = 0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) lev[i] = levels[(int64_t)m * kLevelStride + i];
    __syncthreads();
    for (int i = threadIdx.x; i < kMaxLevels; i += blockDim.x) {
        float2 e = make_float2(0.f, 0.f);
        if (i <= n - 2) e = make_float2(lev[i], __fmul_rn(__fsub_rn(lev[i + 1], lev[i]), 5.9604644775390625e-08f));
        t.ld[(int64_t)m * kMaxLevels + i] = e;
    }
    for (int bin = threadIdx.x; bin < LQ_NUM_BINS; bin += blockDim.x) {
        const float lo = bin == 0 ? 0.0f : __uint_as_float(kLutClamp + ((uint32_t)bin << 19));
        const float hi = __uint_as_float(kLutClamp + ((uint32_t)(bin + 1) << 19));   // exclusive
        int tau0 = 0;
        for (int j = 1; j <= n - 2; ++j) if (lev[j] <= lo) tau0 = j;
        uint32_t boundary = 0x7f800000u;
        if (tau0 + 1 <= n - 2 && lev[tau0 + 1] < hi) {
            boundary = __float_as_uint(lev[tau0 + 1]);
            if (tau0 + 2 <= n - 2 && lev[tau0 + 2] < hi) atomicOr(&slow, 1);
        }
        t.lut[(int64_t)m * kLutStride + bin] = make_uint2(8u * (uint32_t)tau0, boundary);
    }
    __syncthreads();
    if (threadIdx.x == 0) t.fast[m] = slow ? 0 : 1;
}

cudaError_t launch_build_search(const PlanDev& p, const float* levels, SearchTables t, cudaStream_t s)
{
    if (p.num_layers == 0) return cudaSuccess;
    build_search_kernel<<<(unsigned)p.num_layers, 128, 0, s>>>(p, levels, t);
    return cudaGetLastError();
}

cudaError_t launch_quantize(const PlanDev& p, const float* grads, uint32_t step, uint32_t* packed,
                            const float* norms, uint32_t* hist, const uint32_t* prev_packed,
                            const float* prev_norms, const float* levels_cur,
                            const float* levels_prev, SearchTables t, cudaStream_t s)
{
    if (p.num_tiles == 0) return cudaSuccess;
    const dim3 grid((unsigned)p.num_tiles, (unsigned)p.num_workers);
    if (hist)
        quantize_pack_kernel<true><<<grid, kThreads, 0, s>>>(p, grads, step, packed, norms, hist, prev_packed,
                                                             prev_norms, levels_cur, levels_prev, t);
    else
        quantize_pack_kernel<false><<<grid, kThreads, 0, s>>>(p, grads, step, packed, norms, hist, prev_packed,
                                                              prev_norms, levels_cur, levels_prev, t);
    return cudaGetLastError();
}

cudaError_t launch_stat_finalize(const PlanDev& p, cudaStream_t s)
{
    stat_finalize_kernel<<<dim3((unsigned)p.num_layers, (unsigned)p.num_workers), 128, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace lq
