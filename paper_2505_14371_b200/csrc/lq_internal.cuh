// Internal declarations shared by the .cu files of liblq (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "lq.h"

namespace lq {

constexpr int kBlockCoords = 1024;    // coordinates per message block (32 lanes x 32 positions)
constexpr int kTileBlocks = 128;      // most blocks per tile (the encoder's unit: its per-CTA tables are amortised over a
                                      // tile); a plan uses 32, 64 or 128, the largest that still gives several waves of CTAs
constexpr int kSubBlocks = 32;        // blocks per sub-tile (the unit of the norm and decode kernels)
constexpr int kWarps = 8;
constexpr int kThreads = 256;
constexpr int kLevelStride = 256;     // floats per layer in a level table
constexpr int kMaxLevels = 256;
constexpr int kCodeMaxLen = 12;       // longest code word of the entropy stage (LQ_CODE_MAX_LEN)
constexpr int kLutEntries = 2048;     // u32 entries per layer in the encoder's search table: one per value of the
                                      // top 13 bits of a non-negative float (16 bins per octave); 2033 are reachable

struct LayerDesc {
    int64_t elem_off;     // first element of the layer inside a worker's fp32 row
    int64_t word_off;     // first word of the layer inside a worker's message
    int64_t size;         // d_m
    int32_t bits;         // b_m
    int32_t nlevels;      // 2^b_m
    int32_t nblocks;      // ceil(d_m / 1024)
    int32_t first_tile;   // tiles of one layer are contiguous in the tile table
    int32_t ntiles;
    int32_t pad_;
    int64_t block_off;    // first block of the layer in a worker's row of the zero-row masks
};

struct Tile {
    int32_t layer;
    int32_t block0;       // first block of the tile inside its layer
    int32_t nblocks;      // 1..kTileBlocks
    int32_t pad_;
};

// What an encoder CTA needs to know about its tile, one record per CTA in launch order (read with one round trip
// instead of the chain launch order -> tile -> layer).
struct TileJob {
    int32_t tile;         // index in the tile table (the per-tile partials are kept by it)
    int32_t layer;
    int32_t block0;       // first block of the tile inside its layer
    int32_t nblocks;      // 1..kTileBlocks
    int32_t bits;         // b_m
    int32_t pad_;
    int64_t size;         // d_m
    int64_t elem_off;     // first coordinate of the layer inside a worker's row of `grads`
    int64_t word_off;     // first word of the layer inside a worker's message
    int64_t block_off;    // first block of the layer in a worker's row of the zero-row masks
    int64_t pad2_;
};
static_assert(sizeof(TileJob) == 64, "TileJob is read as four 16-byte words");

struct QodaScalars {
    double S;             // running sum of Eq. (general_stepsize)
    double last_delta;    // the term added by the last qoda_step
    long long t;          // index of the next iteration
    float eta;            // eta_t (= gamma_t under Eq. general_stepsize)
    float gamma;          // gamma_t (differs from eta_t only under Eq. Alt)
    double lambda;        // Eq. (Alt): running sum of ||gbar||^2
    double mu;            // Eq. (Alt): running sum of ||X_s - X_{s+1}||^2
    float eta_cur;        // Eq. (Alt): the eta that produced the current X_t (needed to recompute X_t from Y_t)
    float pad_;
};

// Device-side view of a plan, passed to kernels by value.
struct PlanDev {
    const LayerDesc* layers;
    const Tile* tiles;
    const TileJob* jobs;         // the encoder's tiles in the order in which its CTAs take them: all layers advance
                                 // together, so that layers of different character (dense, mostly zero rows) share the
                                 // SMs at any time
    int32_t num_layers;
    int32_t num_tiles;
    int32_t num_workers;
    int32_t q;            // 0 = infinity norm
    int32_t sub_tiles;    // sub-tiles per tile: the plan's tile size / kSubBlocks (1, 2 or 4)
    int32_t sub_shift;    // log2(sub_tiles)
    int32_t global_norm;  // 1: one norm per worker over all layers (Section 3.1), 0: one per layer
    int32_t bucket_norm;  // 1: one norm per bucket of 128 consecutive coordinates of a layer (Section 7.1)
    int32_t worker0;      // the encode-side kernels cover workers worker0 .. worker0 + worker_count - 1 (grid.y =
    int32_t worker_count; // worker_count); `grads` holds only those rows, every other buffer all K rows
    int64_t padded_elems; // D_pad
    int64_t packed_words; // W
    uint32_t seed_lo, seed_hi;
    uint32_t rk0[8], rk1[8];  // Philox keys of rounds 2..9 (seed words plus multiples of the Weyl constants): kernels
                              // read them straight from the parameter bank
    double* norm_partial; // [K][num_tiles * sub_tiles]
    double* stat_partial; // [K][num_tiles]
    double* sq_diff;      // [K][L]
    float* rnorm;         // [K][L]   1/N, or 0 for a zeroed layer
    uint32_t* status;     // [K][L]
    double* layer_total;  // [K][L]  per-layer sums (or maxima) before the root, for the global norm
    double* alt_partial;  // [2][num_tiles * sub_tiles]  per-CTA terms of lambda and mu (Eq. Alt)
    uint8_t* row_mask;    // [K][total_blocks]  bit j of a block's byte: row j (128 values) holds a nonzero value
    const uint8_t* row_mask_prev;   // the same for the input behind the previous message, or NULL when unknown
    int64_t total_blocks; // blocks of 1024 values per worker, all layers
    uint32_t* block_live; // [total_blocks]  bit k: worker k's block holds a nonzero value (built from row_mask; K <= 32)
    double* energy_partial;   // [K][num_tiles]  bucket scope: per-tile sums of squared bucket norms
    uint32_t* flag_partial;   // [K][num_tiles]  bucket scope: bit 0 a non-finite bucket, bit 1 a nonzero bucket
    float* layer_weight;      // [K][L]          bucket scope: sqrt of a layer's summed squared bucket norms
    QodaScalars* scalars;
};

// Stores a printf-style reason for lq_last_error() (calling thread) and returns `code`.
int lq_set_error(int code, const char* fmt, ...);

// ---- launchers (each enqueues on `s` and returns the launch status) ----
// `write_mask`: also record the zero-row masks of `grads` in p.row_mask
cudaError_t launch_norm_partial(const PlanDev& p, const float* grads, bool write_mask, cudaStream_t s);
cudaError_t launch_norm_finalize(const PlanDev& p, float* norms, cudaStream_t s);
// Encode-side tables derived from one level table (rebuilt whenever the levels change).
struct SearchTables {
    uint32_t* lut;     // [L][kLutEntries] per bin: 8 * tau0 | (low 19 bits of the level inside the bin, minus 1) << 13
    float2* ld;        // [L][kMaxLevels]  {l_tau, l_{tau+1} - l_tau}
    int32_t* fast;     // [L]              1 if every bin holds at most one level; else 1 + R (byte table over the top 15
                       //                  bits in lut's place, at most R levels per bin)
};
cudaError_t launch_build_search(const PlanDev& p, const float* levels, SearchTables t, cudaStream_t s);
cudaError_t launch_quantize(const PlanDev& p, const float* grads, uint32_t step, uint32_t* packed,
                            const float* norms, uint32_t* hist, const uint32_t* prev_packed,
                            const float* prev_norms, const float* levels_cur,
                            const float* levels_prev, SearchTables t, bool need_stat, cudaStream_t s);
// bucket scope: `bucket_norms` [K][8 * total_blocks] is written, `prev_norms` has the same shape
cudaError_t launch_quantize_bucketed(const PlanDev& p, const float* grads, uint32_t step, uint32_t* packed,
                                     float* bucket_norms, uint32_t* hist, const uint32_t* prev_packed,
                                     const float* prev_norms, const float* levels_cur,
                                     const float* levels_prev, SearchTables t, cudaStream_t s);
cudaError_t launch_bucket_finalize(const PlanDev& p, cudaStream_t s);
cudaError_t launch_stat_finalize(const PlanDev& p, cudaStream_t s);
// mode 0: decode + aggregate only; 1: + QODA update, Eq. (general_stepsize); 2: + QODA update, Eq. (Alt)
// live: per block the bitmask of workers whose words are not all zero, for exactly this message, or nullptr
cudaError_t launch_decode(const PlanDev& p, const uint32_t* packed, const float* norms,
                          const float* levels, const float* X1, float* Y, float* Xhalf, float* X,
                          float* gbar, int mode, const uint32_t* live, cudaStream_t s);
cudaError_t launch_level_probabilities(const PlanDev& p, const uint32_t* hist, const float* norms, int num_samples,
                                       const float* levels, double* probs, cudaStream_t s);
cudaError_t launch_symbol_counts(const PlanDev& p, const uint32_t* packed, uint32_t* counts, cudaStream_t s);
cudaError_t launch_block_live(const PlanDev& p, cudaStream_t s);
cudaError_t launch_alt_scalars(const PlanDev& p, double qhat, cudaStream_t s);
cudaError_t launch_alt_finalize(const PlanDev& p, cudaStream_t s);
cudaError_t launch_qoda_scalars(const PlanDev& p, cudaStream_t s);
cudaError_t launch_average(const PlanDev& p, const float* Xhalf, double* xsum, cudaStream_t s);
cudaError_t launch_qoda_init(const PlanDev& p, const float* X1, float* Y, float* Xhalf,
                             cudaStream_t s);
cudaError_t launch_fit(const PlanDev& p, const uint32_t* hist, const float* norms, int num_samples,
                       float* levels_stage, cudaStream_t s);
cudaError_t launch_fit_shared(const PlanDev& p, const uint32_t* hist, const float* norms, int num_samples,
                              float* levels_stage, const int32_t* member_off, const int32_t* member_layer,
                              int num_types, cudaStream_t s);

// ---- device helpers ----
#ifdef __CUDACC__

// Philox4x32-10 (Salmon et al., SC'11): 10 rounds of two 32x32->64 multiplies and xors,
// the key bumped by the Weyl constants between rounds.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t (&out)[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// symbol p (pre-scaled by 4) of a lane's string of 32 symbols of C bits, held in C words
template <int C>
__device__ __forceinline__ uint32_t symbol4_at(const uint32_t (&w)[C], int p)
{
    const int off = p * C, i = off >> 5, s = off & 31;
    constexpr uint32_t mask4 = ((1u << C) - 1u) << 2;
    uint32_t v;
    if (s + C <= 32) v = s >= 2 ? (w[i] >> (s - 2)) : (w[i] << (2 - s));
    else             v = __funnelshift_r(w[i], w[i + 1], s - 2);      // s >= 2 whenever a symbol straddles
    return v & mask4;
}

// 16-byte asynchronous copies global -> shared (completion by commit / wait groups of the issuing thread)
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int bytes)
{
    // copies `bytes` (0..16) bytes and fills the rest of the 16 with zeros
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ double warp_max(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Sum over the CTA in a fixed order (xor tree inside a warp, warps added in index order).
// The result is valid in thread 0.  `scratch` holds one double per warp.
template <bool kMax>
__device__ __forceinline__ double block_reduce(double v, double* scratch)
{
    v = kMax ? warp_max(v) : warp_sum(v);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    double r = 0.0;
    if (threadIdx.x == 0) {
        const int nw = (blockDim.x + 31) >> 5;
        r = scratch[0];
        for (int w = 1; w < nw; ++w) r = kMax ? fmax(r, scratch[w]) : r + scratch[w];
    }
    return r;
}

// One value's term of a layer's L^q norm (Section 2.2), accumulated in fp64 (the maximum as an integer pattern).
// mode 0: max |v|   1: sum |v|   2: sum v^2   3: sum |v|^q (integer q >= 3)
template <int kMode>
__device__ __forceinline__ void accumulate(double& acc, uint32_t& maxbits, float v, int q)
{
    if (kMode == 0) {
        // |v| as an unsigned integer orders like the float; NaN and Inf have the largest patterns
        const uint32_t b = __float_as_uint(v) & 0x7fffffffu;
        maxbits = max(maxbits, b);
    } else if (kMode == 1) {
        acc += (double)fabsf(v);
    } else if (kMode == 2) {
        const double a = (double)v;
        acc = fma(a, a, acc);            // the product of two floats is exact in fp64
    } else {
        const double a = fabs((double)v);
        double p = a;
        for (int r = 1; r < q; ++r) p = __dmul_rn(p, a);
        acc += p;
    }
}

// A layer's norm from the norm pass's partials, in a fixed order: thread i < 128 takes partials i, i + 128, ...,
// then the CTA tree; the root, the rounding to fp32, the flags and the fp32 reciprocal.  Every thread of the CTA
// calls it (128 threads or more); the result is valid in thread 0.  `scratch`: one double per warp.
struct LayerNorm {
    double total;        // the sum (or maximum) before the root
    float norm, rnorm;   // fp32(||v||_q) and 1 / norm, both 0 when flagged
    uint32_t status;
    bool bad;            // a partial was NaN or Inf
};
__device__ __forceinline__ LayerNorm layer_norm_from_partials(const double* part, int n, int q, double* scratch)
{
    double acc = 0.0;
    int bad = 0;
    if (threadIdx.x < 128)
        for (int i = threadIdx.x; i < n; i += 128) {
            const double v = __ldcg(part + i);                   // (from L2: another CTA of this launch may have written it)
            if (!(fabs(v) <= 1.7976931348623157e308)) bad = 1;
            if (q == 0) acc = fmax(acc, v); else acc += v;
        }
    bad = __syncthreads_or(bad);
    LayerNorm r;
    r.total = q == 0 ? block_reduce<true>(acc, scratch) : block_reduce<false>(acc, scratch);
    r.bad = bad != 0;
    double n64;
    if (q == 0 || q == 1) n64 = r.total;
    else if (q == 2)      n64 = sqrt(r.total);
    else                  n64 = pow(r.total, 1.0 / (double)q);
    float nf = (float)n64;
    r.status = 0;
    if (bad || !(fabs(n64) <= 1.7976931348623157e308) || !(fabsf(nf) <= 3.402823466e38f))
        r.status = LQ_STATUS_NONFINITE;
    else if (nf < 1.17549435e-38f)
        r.status = LQ_STATUS_ZERO_NORM;
    r.norm = r.status ? 0.0f : nf;
    r.rnorm = r.status ? 0.0f : __fdiv_rn(1.0f, nf);
    return r;
}

#endif  // __CUDACC__

}  // namespace lq
