// Per-layer L^q norms of K workers' gradients (Section 2.2 of the paper: v is represented by
// (||v||_q, sign, u)).  Two launches: a streaming pass that leaves one fp64 partial per
// (worker, tile), and a small pass that adds a layer's partials in a fixed order, so the
// result does not depend on scheduling.  The streaming pass also leaves one byte per block of 1024
// values whose bit j says whether row j (the 128 values 128 j .. 128 j + 127) holds anything but
// zeros, so that the encoder, which reads the same values next, can leave all-zero rows unread.
#include "lq_internal.cuh"

namespace lq {

template <int kMode>
__global__ void __launch_bounds__(kThreads) norm_partial_kernel(PlanDev p, const float* __restrict__ grads,
                                                                bool write_mask)
{
    __shared__ double scratch[kThreads / 32];
    const Tile tile = p.tiles[blockIdx.x >> p.sub_shift];
    const int sub0 = (blockIdx.x & (p.sub_tiles - 1)) * kSubBlocks;          // this CTA's blocks of the tile
    const int sub1 = min(sub0 + kSubBlocks, tile.nblocks);
    const LayerDesc L = p.layers[tile.layer];
    const int k = blockIdx.y + p.worker0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float* __restrict__ g = grads + (int64_t)blockIdx.y * p.padded_elems + L.elem_off;

    double acc = 0.0;
    uint32_t maxbits = 0;
    uint8_t* __restrict__ mask = p.row_mask + (int64_t)k * p.total_blocks + L.block_off;
    for (int b = sub0 + warp; b < sub1; b += kWarps) {
        const int64_t blk0 = (int64_t)(tile.block0 + b) * kBlockCoords;
        const int64_t base = blk0 + 4 * lane;
        uint32_t rows = 0;                       // bit j: this lane's part of row j holds a value that is not +-0 (NaN counts)
        if (blk0 + kBlockCoords <= L.size) {
            float4 v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
                v[j] = __ldg(reinterpret_cast<const float4*>(g + base + 128 * j));
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                accumulate<kMode>(acc, maxbits, v[j].x, p.q);
                accumulate<kMode>(acc, maxbits, v[j].y, p.q);
                accumulate<kMode>(acc, maxbits, v[j].z, p.q);
                accumulate<kMode>(acc, maxbits, v[j].w, p.q);
                const float mag = (fabsf(v[j].x) + fabsf(v[j].y)) + (fabsf(v[j].z) + fabsf(v[j].w));
                rows |= (mag != 0.0f ? 1u : 0u) << j;
            }
        } else {
            for (int j = 0; j < 8; ++j) {
                const int64_t pos = base + 128 * j;
                float mag = 0.0f;
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (pos + e < L.size) {
                        const float x = __ldg(g + pos + e);
                        accumulate<kMode>(acc, maxbits, x, p.q);
                        mag += fabsf(x);
                    }
                rows |= (mag != 0.0f ? 1u : 0u) << j;
            }
        }
        rows = __reduce_or_sync(0xffffffffu, rows);      // a row is live if any lane's part of it is
        if (write_mask && lane == 0) mask[tile.block0 + b] = (uint8_t)rows;
    }
    if (kMode == 0)   // a non-finite maximum is handed on as NaN so that the final pass sees it
        acc = maxbits >= 0x7f800000u ? __longlong_as_double(0x7ff8000000000000LL)
                                     : (double)__uint_as_float(maxbits);
    double r;
    if (kMode == 0) {
        // fmax drops NaNs: reduce a "bad" flag next to the maximum
        const unsigned bad = __syncthreads_or(acc != acc);
        r = block_reduce<true>(acc == acc ? acc : 0.0, scratch);
        if (bad) r = __longlong_as_double(0x7ff8000000000000LL);
    } else {
        r = block_reduce<false>(acc, scratch);
    }
    if (threadIdx.x == 0) p.norm_partial[(int64_t)k * p.num_tiles * p.sub_tiles + blockIdx.x] = r;
}

// One CTA per (layer, worker): adds the layer's tile partials (thread i takes partials
// i, i+128, ... in order; then the fixed CTA tree), takes the root, rounds to fp32 and stores
// the norm, its fp32 reciprocal and the status flags.
__global__ void __launch_bounds__(128) norm_finalize_kernel(PlanDev p, float* __restrict__ norms)
{
    __shared__ double scratch[4];
    const int m = blockIdx.x, k = blockIdx.y + p.worker0;
    const LayerDesc L = p.layers[m];
    const double* part = p.norm_partial + ((int64_t)k * p.num_tiles + L.first_tile) * p.sub_tiles;
    const LayerNorm r = layer_norm_from_partials(part, L.ntiles * p.sub_tiles, p.q, scratch);
    if (threadIdx.x == 0) {
        const int64_t o = (int64_t)k * p.num_layers + m;
        if (p.global_norm) {                     // the layers' totals are combined per worker by norm_global_kernel
            p.layer_total[o] = r.bad ? __longlong_as_double(0x7ff8000000000000LL) : r.total;
            return;
        }
        norms[o] = r.norm;
        p.rnorm[o] = r.rnorm;
        p.status[o] = r.status;
    }
}

// Global norm scope (the formal definition of Q in Section 3.1: one ||v||_q over the whole vector): one CTA per
// worker combines the layers' totals in layer order and writes the same norm into every layer's slot, so the
// message keeps its format.  A non-finite value anywhere zeroes the worker's whole message.
__global__ void __launch_bounds__(128) norm_global_kernel(PlanDev p, float* __restrict__ norms)
{
    __shared__ double scratch[4];
    __shared__ float n_s;
    __shared__ uint32_t st_s;
    const int k = blockIdx.x + p.worker0;
    const double* tot = p.layer_total + (int64_t)k * p.num_layers;
    double acc = 0.0;
    int bad = 0;
    for (int m = threadIdx.x; m < p.num_layers; m += blockDim.x) {
        const double v = tot[m];
        if (!(fabs(v) <= 1.7976931348623157e308)) bad = 1;
        if (p.q == 0) acc = fmax(acc, v); else acc += v;
    }
    bad = __syncthreads_or(bad);
    const double total = p.q == 0 ? block_reduce<true>(acc, scratch) : block_reduce<false>(acc, scratch);
    if (threadIdx.x == 0) {
        double n64;
        if (p.q == 0 || p.q == 1) n64 = total;
        else if (p.q == 2)        n64 = sqrt(total);
        else                      n64 = pow(total, 1.0 / (double)p.q);
        float n = (float)n64;
        uint32_t st = 0;
        if (bad || !(fabs(n64) <= 1.7976931348623157e308) || !(fabsf(n) <= 3.402823466e38f))
            st = LQ_STATUS_NONFINITE;
        else if (n < 1.17549435e-38f)
            st = LQ_STATUS_ZERO_NORM;
        n_s = st ? 0.0f : n;
        st_s = st;
    }
    __syncthreads();
    const float n = n_s;
    const uint32_t st = st_s;
    for (int m = threadIdx.x; m < p.num_layers; m += blockDim.x) {
        const int64_t o = (int64_t)k * p.num_layers + m;
        norms[o] = n;
        p.rnorm[o] = st ? 0.0f : __fdiv_rn(1.0f, n);
        p.status[o] = st;
    }
}

cudaError_t launch_norm_partial(const PlanDev& p, const float* grads, bool write_mask, cudaStream_t s)
{
    if (p.num_tiles == 0) return cudaSuccess;
    const dim3 grid((unsigned)p.num_tiles * p.sub_tiles, (unsigned)p.worker_count);
    if (p.q == 0)      norm_partial_kernel<0><<<grid, kThreads, 0, s>>>(p, grads, write_mask);
    else if (p.q == 1) norm_partial_kernel<1><<<grid, kThreads, 0, s>>>(p, grads, write_mask);
    else if (p.q == 2) norm_partial_kernel<2><<<grid, kThreads, 0, s>>>(p, grads, write_mask);
    else               norm_partial_kernel<3><<<grid, kThreads, 0, s>>>(p, grads, write_mask);
    return cudaGetLastError();
}

cudaError_t launch_norm_finalize(const PlanDev& p, float* norms, cudaStream_t s)
{
    norm_finalize_kernel<<<dim3((unsigned)p.num_layers, (unsigned)p.worker_count), 128, 0, s>>>(p, norms);
    if (p.global_norm) norm_global_kernel<<<(unsigned)p.worker_count, 128, 0, s>>>(p, norms);
    return cudaGetLastError();
}

}  // namespace lq
