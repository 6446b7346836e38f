// Code-length accounting (the paper's appendix on the coding framework): the probability that each
// level of a layer is emitted, from the same histogram-based CDF estimate the level fit uses, and a
// count of the level indices a message actually carries, to set against those probabilities.
//
//   p^_j = int hat_j(u) dF~(u):  stochastic rounding sends u in [l_tau, l_{tau+1}] to l_tau with
//   probability (l_{tau+1} - u) / (l_{tau+1} - l_tau) and to l_{tau+1} otherwise, so level j collects
//   the rising half of its hat function from [l_{j-1}, l_j] and the falling half from [l_j, l_{j+1}].
//   F~ is piecewise linear inside the histogram bins, plus the point mass at u = 1 of the last bin.
// Compiled without FMA contraction: the sequence of fp64 roundings is the plain one.
#include "lq_internal.cuh"

namespace lq {
namespace {

constexpr int kBins = 385;            // bins 0..384 carry density; bin 385 is the point mass at u = 1

__device__ __forceinline__ double edge_of(int i)
{
    if (i <= 0) return 0.0;
    const int o = (i - 1) >> 4, m = (i - 1) & 15;
    return ldexp(1.0 + (double)m * 0.0625, o - 24);
}

// One CTA per layer, one thread per level.
__global__ void __launch_bounds__(kMaxLevels) level_probabilities_kernel(PlanDev p, const uint32_t* __restrict__ hist,
                                                                         const float* __restrict__ norms, int Z,
                                                                         const float* __restrict__ levels,
                                                                         double* __restrict__ probs)
{
    __shared__ double mass[LQ_NUM_BINS];
    __shared__ double lev[kMaxLevels];
    __shared__ double wsum_s;
    const int m = blockIdx.x, tid = threadIdx.x;
    const LayerDesc L = p.layers[m];
    const int n = L.nlevels;
    double* out = probs + (int64_t)m * kMaxLevels;
    if (tid == 0) {
        double w = 0.0;
        for (int z = 0; z < Z; ++z) { const double x = (double)norms[(int64_t)z * p.num_layers + m]; w += x * x; }
        wsum_s = w;
    }
    if (tid < n) lev[tid] = (double)levels[(int64_t)m * kLevelStride + tid];
    __syncthreads();
    const double wsum = wsum_s;
    if (!(wsum > 0.0) || L.size <= 0) { out[tid] = 0.0; return; }
    for (int i = tid; i < LQ_NUM_BINS; i += blockDim.x) {
        double acc = 0.0;
        for (int z = 0; z < Z; ++z) {
            const double x = (double)norms[(int64_t)z * p.num_layers + m];
            acc += ((x * x) / wsum) * (double)hist[((int64_t)z * p.num_layers + m) * LQ_HIST_STRIDE + i];
        }
        mass[i] = acc / (double)L.size;
    }
    __syncthreads();
    if (tid >= n) { out[tid] = 0.0; return; }
    const int j = tid;
    double pj = 0.0;
    // the pieces of every bin, in ascending order of u, that lie under the two halves of hat_j
    for (int i = 0; i < kBins; ++i) {
        if (mass[i] == 0.0) continue;
        const double lo = edge_of(i), hi = edge_of(i + 1), dens = mass[i] / (hi - lo);
        if (j >= 1) {                                      // rising half on [a, c] = [l_{j-1}, l_j]
            const double a = lev[j - 1], c = lev[j];
            const double x0 = fmax(lo, a), x1 = fmin(hi, c);
            if (x1 > x0) pj += dens * (x1 - x0) * (0.5 * (x0 + x1) - a) / (c - a);
        }
        if (j <= n - 2) {                                  // falling half on [a, c] = [l_j, l_{j+1}]
            const double a = lev[j], c = lev[j + 1];
            const double x0 = fmax(lo, a), x1 = fmin(hi, c);
            if (x1 > x0) pj += dens * (x1 - x0) * (c - 0.5 * (x0 + x1)) / (c - a);
        }
    }
    if (j == n - 1) pj += mass[LQ_NUM_BINS - 1];           // the point mass at u = 1
    out[j] = pj;
}

// One CTA per (sub-tile, worker): counts the level indices of the message's real coordinates.
__global__ void __launch_bounds__(kThreads) symbol_counts_kernel(PlanDev p, const uint32_t* __restrict__ packed,
                                                                 uint32_t* __restrict__ counts)
{
    __shared__ uint32_t cnt[kMaxLevels];
    Tile tile = p.tiles[blockIdx.x >> p.sub_shift];
    const int sub0 = (blockIdx.x & (p.sub_tiles - 1)) * kSubBlocks;
    if (sub0 >= tile.nblocks) return;
    const int sub1 = min(sub0 + kSubBlocks, tile.nblocks);
    const int layer = tile.layer, k = blockIdx.y;
    const LayerDesc L = p.layers[layer];
    const int C = L.bits + 1, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < kMaxLevels; i += blockDim.x) cnt[i] = 0;
    __syncthreads();
    const uint32_t* msg = packed + (int64_t)k * p.packed_words + L.word_off;
    for (int b = sub0 + warp; b < sub1; b += kWarps) {
        const int64_t blk = tile.block0 + b;
        uint32_t w[LQ_MAX_BITS + 2];
        for (int i = 0; i < C; ++i) w[i] = msg[blk * (int64_t)C * 32 + i * 32 + lane];
        w[C] = 0u;
        for (int pp = 0; pp < 32; ++pp) {
            const int64_t coord = blk * kBlockCoords + 128 * (pp >> 2) + 4 * lane + (pp & 3);
            if (coord >= L.size) continue;
            const int off = pp * C, i = off >> 5, s = off & 31;
            const uint64_t two = ((uint64_t)w[i + 1] << 32) | w[i];
            const uint32_t sym = (uint32_t)(two >> s) & ((1u << C) - 1u);
            atomicAdd(&cnt[sym >> 1], 1u);
        }
    }
    __syncthreads();
    uint32_t* out = counts + ((int64_t)k * p.num_layers + layer) * kMaxLevels;
    for (int i = threadIdx.x; i < L.nlevels; i += blockDim.x)
        if (cnt[i]) atomicAdd(out + i, cnt[i]);
}

}  // namespace

cudaError_t launch_level_probabilities(const PlanDev& p, const uint32_t* hist, const float* norms, int num_samples,
                                       const float* levels, double* probs, cudaStream_t s)
{
    if (p.num_layers == 0) return cudaSuccess;
    level_probabilities_kernel<<<(unsigned)p.num_layers, kMaxLevels, 0, s>>>(p, hist, norms, num_samples, levels, probs);
    return cudaGetLastError();
}

cudaError_t launch_symbol_counts(const PlanDev& p, const uint32_t* packed, uint32_t* counts, cudaStream_t s)
{
    if (p.num_tiles == 0) return cudaSuccess;
    const dim3 grid((unsigned)p.num_tiles * p.sub_tiles, (unsigned)p.num_workers);
    symbol_counts_kernel<<<grid, kThreads, 0, s>>>(p, packed, counts);
    return cudaGetLastError();
}

}  // namespace lq
