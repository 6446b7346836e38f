// ENCODE for all workers: normalise, round stochastically between neighbouring levels, pack one
// (b+1)-bit symbol per coordinate (Section 3.1 quantizer, Section 3.2 message; Algorithm 1 line 12),
// with the optional histogram of normalised magnitudes (Algorithm 1 line 4) and the sender-side
// term of the adaptive step size, sum ||V^_{k,t+1/2} - V^_{k,t-1/2}||^2 (Eq. general_stepsize).
//
// Work decomposition: one CTA of 8 warps per (tile, worker); a tile is up to 128 blocks of 1024
// coordinates of one layer, taken round-robin by the warps.  A lane owns the 32 coordinates
// {128 j + 4 lane + e} of a block (row j = one float4 per lane, 512 contiguous bytes per warp).  Rows
// travel from global memory into a per-warp ring of 8 rows in shared memory with 16-byte
// asynchronous copies, so a warp always has 4 KB in flight and the values never sit in registers
// while they wait; every lane reads back only the bytes it copied itself, so the ring needs no
// barrier.  Per row the lane draws one Philox4x32-10 block (4 uniforms); after 8 rows it holds
// exactly b+1 words of symbols, which it stores plane by plane (128 contiguous bytes per warp and
// plane).  No shuffles, ballots or atomics on the main path.
//
// The level search uses a table over the 386 histogram bins of u (exponent + 4 mantissa bits): each
// entry names the last level at or below the bin's lower edge and the single level that may lie
// inside the bin, so tau costs one shared-memory load and one compare.  Layers whose levels are
// denser than the bins fall back to a binary search.  {level, gap} pairs and the decoded values of the current and the previous message
// sit in small tables; every table offset derives from one register (8 * tau, then 4 * symbol with
// symbol = 2 * idx + sign).
//
// The norm pass, which reads the same values just before, leaves one bit per row of 128 values
// that says whether the row holds anything but zeros.  An all-zero row (untouched embedding rows)
// is never fetched, draws no random numbers and needs no search: its symbols are 0.  If the
// previous message is all zero there as well, the row adds nothing to the statistic and is
// skipped entirely.
#include "lq_internal.cuh"

namespace lq {

constexpr int kQWarps = kWarps;                    // warps per CTA of the quantize kernel
constexpr int kQThreads = kQWarps * 32;
constexpr int kRingRows = 8;                       // rows of 512 bytes in flight per warp
constexpr int kRingBytes = kQWarps * kRingRows * 512;

struct QuantSmem {
    uint2 lut[kLutStride];           // search table of this layer: {8 * tau0, boundary bits}
    float2 ld[kMaxLevels];           // {l_tau, l_{tau+1} - l_tau}
    float lev[kMaxLevels];           // plain levels (binary-search path)
    float tcur[2 * kMaxLevels];      // fp32(N_cur * l_idx) at 2 * idx, its negative at 2 * idx + 1
    float tprev[2 * kMaxLevels];     // same for the previous message
    uint32_t hist[LQ_HIST_STRIDE];
    double scratch[kQWarps];
    uint8_t rows_cur[kTileBlocks];   // per block of the tile: which rows of the input are not all zero
    uint8_t rows_prev[kTileBlocks];  // the same for the input behind the previous message
};

// x + 8 when a >= b (resp. a < b), else x: one compare and one predicated add
__device__ __forceinline__ uint32_t add8_if_ge(uint32_t x, float a, float b)
{
    asm("{\n\t.reg .pred p;\n\tsetp.ge.f32 p, %1, %2;\n\t@p add.u32 %0, %0, 8;\n\t}" : "+r"(x) : "f"(a), "f"(b));
    return x;
}
__device__ __forceinline__ uint32_t add8_if_lt(uint32_t x, float a, float b)
{
    asm("{\n\t.reg .pred p;\n\tsetp.lt.f32 p, %1, %2;\n\t@p add.u32 %0, %0, 8;\n\t}" : "+r"(x) : "f"(a), "f"(b));
    return x;
}

// x + 4 when v < 0 (so neither zero sets the sign bit of a symbol), else x
__device__ __forceinline__ uint32_t add4_if_negative(uint32_t x, float v)
{
    asm("{\n\t.reg .pred p;\n\tsetp.lt.f32 p, %1, 0f00000000;\n\t@p add.u32 %0, %0, 4;\n\t}" : "+r"(x) : "f"(v));
    return x;
}

template <int C>
__device__ __forceinline__ void put_symbol4(uint32_t (&w)[C], int p, uint32_t sym4)
{
    const int off = p * C, i = off >> 5, s = off & 31;
    w[i] += s >= 2 ? (sym4 << (s - 2)) : (sym4 >> (2 - s));           // fields never overlap: + is |
    if (s + C > 32) w[i + 1] = sym4 >> (34 - s);
}

// Philox4x32-10 with counter (c0, layer, worker, step): within one CTA only c0 changes, so half of
// round 0 (the product with the worker word) and half of round 1 (the product with a word that
// depends only on round 0's constant half) are the same for every call and are computed once.
struct PhiloxConsts {
    uint32_t b;      // step ^ k1                       (round 0: c2' = hi(M0 c0) ^ b)
    uint32_t c1;     // lo(M1 worker) ^ (k0 + W0)       (round 1: c0'' = hi(M1 c2') ^ c1)
    uint32_t c2;     // hi(M0 a0) ^ (k1 + W1)           (round 1: c2'' = lo(M0 c0) ^ c2)
    uint32_t l0;     // lo(M0 a0)                       (round 1: c3'')
};

__device__ __forceinline__ PhiloxConsts philox_fold(uint32_t layer, uint32_t worker, uint32_t step,
                                                    uint32_t k0, uint32_t k1)
{
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * worker;
    const uint32_t a0 = (uint32_t)(p1 >> 32) ^ layer ^ k0;            // round 0's c0'
    const uint64_t q0 = (uint64_t)0xD2511F53u * a0;
    PhiloxConsts pc;
    pc.b = step ^ k1;
    pc.c1 = (uint32_t)p1 ^ (k0 + 0x9E3779B9u);
    pc.c2 = (uint32_t)(q0 >> 32) ^ (k1 + 0xBB67AE85u);
    pc.l0 = (uint32_t)q0;
    return pc;
}

// (the keys of rounds 2..9 depend on the seed only and come from the kernel's parameters)
__device__ __forceinline__ void philox4x32_10_folded(uint32_t ctr0, const PhiloxConsts& pc, const PlanDev& p,
                                                     uint32_t (&out)[4])
{
    // rounds 0 and 1 with their constant halves folded
    const uint64_t p0 = (uint64_t)0xD2511F53u * ctr0;
    const uint32_t c2a = (uint32_t)(p0 >> 32) ^ pc.b;
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2a;
    uint32_t c0 = (uint32_t)(p1 >> 32) ^ pc.c1;
    uint32_t c1 = (uint32_t)p1;
    uint32_t c2 = (uint32_t)p0 ^ pc.c2;
    uint32_t c3 = pc.l0;
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        const uint64_t q0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t q1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(q1 >> 32) ^ c1 ^ p.rk0[r];
        const uint32_t n2 = (uint32_t)(q0 >> 32) ^ c3 ^ p.rk1[r];
        c1 = (uint32_t)q1;
        c3 = (uint32_t)q0;
        c0 = n0;
        c2 = n2;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Everything a warp needs to walk its blocks of one (tile, worker).
struct WarpCtx {
    const float* g;              // first coordinate of the layer in this worker's row
    int64_t size;                // d_m
    uint32_t ring;               // shared-memory address of this lane's 16 bytes in ring row 0
    const float4* ring_ptr;      // the same place as a pointer
    float r;                     // 1/N (zeroed layers, r = 0, take another path)
    int lane;
};

// Starts the copies of all 8 rows of a block that may reach past the layer's end (zero-filled there).
__device__ __forceinline__ void issue_ragged_block(const WarpCtx& c, int64_t blk)
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

// Bucket scope (Section 7.1 runs the quantizer on buckets of 128 consecutive coordinates, each with its own
// norm): a bucket is one row of a block, which a warp holds as one float4 per lane, so the norm is a reduction
// over the warp and the separate norm pass disappears.
struct BucketCtx {
    const float* prev_bn;        // bucket norms of the previous message for this (worker, layer), or nullptr
    float* bn_out;               // bucket norms of this message for this (worker, layer)
    int q;
    double energy;               // this lane's share of the sum of squared bucket norms
    uint32_t flags;              // bit 0: a bucket held NaN or Inf, bit 1: a bucket with a nonzero norm
};

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

// One block of 1024 coordinates from the ring.  `rows` says which of its 8 rows hold anything but
// zeros (only those were fetched); `next` is this lane's first float4 of the block whose rows
// replace the consumed ones (nullptr: nothing to fetch) and `next_rows` its row mask; `prev_rows`
// says which rows may be nonzero in the previous message.  Returns this lane's statistic term.
// In bucket scope the value tables hold the plain signed levels and every row brings its own norm.
template <int B, bool kFast, bool kHist, bool kBucket>
__device__ __forceinline__ double quantize_block(const PlanDev& p, const PhiloxConsts& pc, const WarpCtx& c,
                                                 int64_t blk, uint32_t rows, uint32_t prev_rows,
                                                 const float* __restrict__ next, uint32_t next_rows,
                                                 uint32_t* __restrict__ out, const uint32_t (&pw)[B + 1],
                                                 QuantSmem& sm, BucketCtx& bk, float prev_norm8)
{
    // prev_norm8 (bucket scope): lanes 0..7 hold the previous message's norms of rows 0..7 of this block
    constexpr int n = 1 << B, C = B + 1;
    const int lane = c.lane;
    float r = c.r;
    float my_norm = 0.0f, my_rnorm = 0.0f;       // bucket scope: norm and reciprocal of row (lane >> 2)
    if (kBucket) {
        bool bad;
        cp_async_wait<0>();                      // all 8 rows of the block have landed
        bucket_norms8(c.ring_ptr, bk.q, lane, my_norm, my_rnorm, bad);
        if ((lane & 3) == 0) bk.energy = fma((double)my_norm, (double)my_norm, bk.energy);
        bk.flags |= (bad ? 1u : 0u) | (my_norm > 0.0f ? 2u : 0u);
        if (prev_rows == 0u && !__any_sync(0xffffffffu, my_norm > 0.0f)) {
            // every bucket of the block is zeroed and the previous message is zero here too: zero words, zero
            // norms, nothing for the statistic; the ring takes the next block's rows at once
#pragma unroll
            for (int j = 0; j < kRingRows; ++j) {
                if (next && ((next_rows >> j) & 1u)) cp_async16(c.ring + 512u * j, next + 128 * j, 16);
                cp_async_commit();
            }
            const int64_t woff = blk * (int64_t)C * 32 + lane;
#pragma unroll
            for (int w = 0; w < C; ++w) __stcs(out + woff + w * 32, 0u);
            if ((lane & 3) == 0) bk.bn_out[blk * 8 + (lane >> 2)] = 0.0f;
            return 0.0;
        }
    }
    uint32_t cw[C];
#pragma unroll
    for (int w = 0; w < C; ++w) cw[w] = 0u;

    const char* lut_b = reinterpret_cast<const char*>(sm.lut) - (kLutClamp >> 16);
    const char* ld_b = reinterpret_cast<const char*>(sm.ld);
    const char* tcur_b = reinterpret_cast<const char*>(sm.tcur);
    const char* tprev_b = reinterpret_cast<const char*>(sm.tprev);
    double stat = 0.0;
    const uint32_t ctr0 = (uint32_t)(blk * 256) + (uint32_t)lane;     // index / 4 of this lane's row 0

#pragma unroll
    for (int j = 0; j < kRingRows; ++j) {
        bool live = (rows >> j) & 1u;                    // the same for the whole warp
        float nrow = 0.0f, pn = 0.0f;                    // bucket scope: this row's norm now and in the previous message
        if (kBucket) {
            nrow = __shfl_sync(0xffffffffu, my_norm, 4 * j);
            r = __shfl_sync(0xffffffffu, my_rnorm, 4 * j);
            live = nrow > 0.0f;                          // a zeroed bucket sends zeros and draws nothing
            pn = __shfl_sync(0xffffffffu, prev_norm8, j);
        }
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (live) {
            cp_async_wait<kRingRows - 1>();
            v = c.ring_ptr[32 * j];
        }
        const float vv[4] = {v.x, v.y, v.z, v.w};
        if (live) {
            uint32_t x[4];
            philox4x32_10_folded(ctr0 + 32 * j, pc, p, x);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int pp = 4 * j + e;
                // u <= 1 + 2^-23 always (N >= |v| and one rounding each in 1/N and the product), and
                // such a u behaves exactly like u = 1 below, so the min(u, 1) of the definition is not needed
                const float u = __fmul_rn(fabsf(vv[e]), r);
                const uint32_t ub = __float_as_uint(u);
                uint32_t t8;
                if (kFast) {
                    const uint32_t off = (max(ub, kLutClamp) >> 16) & ~7u;
                    const uint2 en = *reinterpret_cast<const uint2*>(lut_b + off);
                    t8 = add8_if_ge(en.x, u, __uint_as_float(en.y));
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
                const float den = ld.y;
                const float num = __fsub_rn(u, ld.x);
                // rho = (x >> 9) * 2^-23; f = 1 + rho is built from the bits, and fma(f, den, -den)
                // rounds the exact product rho * den once, like the plain multiplication
                // (one funnel shift: the 64-bit value {0x7F, x} moved right by 9 is (x >> 9) | 0x3F800000)
                const float f = __uint_as_float(__funnelshift_r(x[e], 0x7Fu, 9));
                const float t = __fmaf_rn(f, den, -den);
                const uint32_t i8 = add8_if_lt(t8, t, num);
                const uint32_t sym4 = add4_if_negative(i8, vv[e]);                // 4 * (2 * idx + sign), sign = (v < 0)
                put_symbol4<C>(cw, pp, sym4);

                if (kHist) {
                    const int64_t pos = blk * kBlockCoords + 128 * j + 4 * lane + e;
                    if (pos < c.size) atomicAdd(&sm.hist[(max(ub, kLutClamp) - kLutClamp) >> 19], 1u);
                }

                // step-size statistic: fp32 difference of the two decoded values, squared in fp64
                float cur = *reinterpret_cast<const float*>(tcur_b + sym4);
                float prv = *reinterpret_cast<const float*>(tprev_b + symbol4_at<C>(pw, pp));
                if (kBucket) { cur = __fmul_rn(cur, nrow); prv = __fmul_rn(prv, pn); }
                const double dd = (double)__fsub_rn(cur, prv);
                stat = fma(dd, dd, stat);
            }
        } else if ((prev_rows >> j) & 1u) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float prv = *reinterpret_cast<const float*>(tprev_b + symbol4_at<C>(pw, 4 * j + e));
                if (kBucket) prv = __fmul_rn(prv, pn);
                const double dd = (double)prv;
                stat = fma(dd, dd, stat);
            }
        }
        if (kHist && !kBucket && !live && lane == 0) {
            // an all-zero row of a layer with a norm: its coordinates have u = 0 and count in the first bin
            const int64_t rem = c.size - (blk * kBlockCoords + 128 * j);
            if (rem > 0) atomicAdd(&sm.hist[0], (uint32_t)(rem < 128 ? rem : 128));
        }
        if (next && ((next_rows >> j) & 1u)) cp_async16(c.ring + 512u * j, next + 128 * j, 16);
        cp_async_commit();
    }
    const int64_t woff = blk * (int64_t)C * 32 + lane;
#pragma unroll
    for (int w = 0; w < C; ++w) __stcs(out + woff + w * 32, cw[w]);
    if (kBucket && (lane & 3) == 0) bk.bn_out[blk * 8 + (lane >> 2)] = my_norm;
    return stat;
}

// A layer whose message is all zero (zero norm, NaN or Inf inside): zero words, and the statistic is
// the squared previous message.
template <int B>
__device__ __forceinline__ double zeroed_tile(const Tile& tile, int lane, uint32_t* __restrict__ out,
                                              const uint32_t* __restrict__ prev, QuantSmem& sm)
{
    constexpr int C = B + 1;
    double stat = 0.0;
    for (int b = threadIdx.x >> 5; b < tile.nblocks; b += kQWarps) {
        const int64_t woff = (tile.block0 + b) * (int64_t)C * 32 + lane;
        uint32_t pw[C];
#pragma unroll
        for (int w = 0; w < C; ++w) {
            pw[w] = prev ? __ldcs(prev + woff + w * 32) : 0u;
            __stcs(out + woff + w * 32, 0u);
        }
#pragma unroll
        for (int pp = 0; pp < 32; ++pp) {
            const double dd = (double)sm.tprev[symbol4_at<C>(pw, pp) >> 2];
            stat = fma(dd, dd, stat);
        }
    }
    return stat;
}

// A warp's share of a tile: blocks warp, warp + 8, ...  A block whose rows are all zero in this input and
// in the input behind the previous message is an all-zero piece of message that adds nothing to the
// statistic: its words are stored and nothing is read.
template <int B, bool kFast, bool kHist, bool kBucket>
__device__ __forceinline__ double quantize_tile(const PlanDev& p, const PhiloxConsts& pc, const WarpCtx& c, const Tile& tile,
                                                uint32_t* __restrict__ out,
                                                const uint32_t* __restrict__ prev, QuantSmem& sm, BucketCtx& bk)
{
    constexpr int C = B + 1;
    const int warp = threadIdx.x >> 5;
    const int64_t nfull = c.size / kBlockCoords;          // blocks below this index lie inside the layer
    double stat = 0.0;
    bool primed = false;                                  // the ring holds (or awaits) the rows of block b
    for (int b = warp; b < tile.nblocks; b += kQWarps) {
        const int64_t blk = tile.block0 + b;
        const uint32_t rows = sm.rows_cur[b], prows = sm.rows_prev[b];
        if ((rows | prows) == 0u) {
            const int64_t woff = blk * (int64_t)C * 32 + c.lane;
#pragma unroll
            for (int w = 0; w < C; ++w) __stcs(out + woff + w * 32, 0u);
            if (kHist && c.lane == 0) {                   // its coordinates all have u = 0
                const int64_t rem = c.size - blk * kBlockCoords;
                atomicAdd(&sm.hist[0], (uint32_t)(rem < kBlockCoords ? rem : kBlockCoords));
            }
            continue;
        }
        if (!primed) {
            if (blk < nfull) {
                const float* src = c.g + blk * kBlockCoords + 4 * c.lane;
#pragma unroll
                for (int j = 0; j < kRingRows; ++j) {
                    if ((rows >> j) & 1u) cp_async16(c.ring + 512u * j, src + 128 * j, 16);
                    cp_async_commit();
                }
            } else {
                issue_ragged_block(c, blk);
            }
        }
        float prev_norm8 = 0.0f;
        uint32_t pmask = prows;
        if (kBucket && prev) {
            // the previous message's norms tell which of its rows are all zero: those add nothing to the statistic
            if (c.lane < 8) prev_norm8 = __ldg(bk.prev_bn + blk * 8 + c.lane);
            pmask = __ballot_sync(0xffffffffu, prev_norm8 != 0.0f) & 0xffu;
        }
        uint32_t pw[C];
#pragma unroll
        for (int w = 0; w < C; ++w) pw[w] = (prev && pmask) ? __ldcs(prev + blk * (int64_t)C * 32 + c.lane + w * 32) : 0u;
        // the next block of this warp that has anything in it: its rows replace the consumed ones
        int nb = b + kQWarps;
        while (nb < tile.nblocks && (sm.rows_cur[nb] | sm.rows_prev[nb]) == 0u) {
            const int64_t woff = (tile.block0 + nb) * (int64_t)C * 32 + c.lane;
#pragma unroll
            for (int w = 0; w < C; ++w) __stcs(out + woff + w * 32, 0u);
            if (kHist && c.lane == 0) {
                const int64_t rem = c.size - (tile.block0 + nb) * kBlockCoords;
                atomicAdd(&sm.hist[0], (uint32_t)(rem < kBlockCoords ? rem : kBlockCoords));
            }
            nb += kQWarps;
        }
        const bool has_next = nb < tile.nblocks;
        const int64_t nblk = tile.block0 + nb;
        const uint32_t next_rows = has_next ? sm.rows_cur[nb] : 0u;
        const float* next = (has_next && nblk < nfull) ? c.g + nblk * kBlockCoords + 4 * c.lane : nullptr;
        stat += quantize_block<B, kFast, kHist, kBucket>(p, pc, c, blk, rows, pmask, next, next_rows, out, pw, sm, bk, prev_norm8);
        primed = has_next;
        if (has_next && nblk >= nfull) issue_ragged_block(c, nblk);   // the layer's last, partial block
        b = nb - kQWarps;                                             // the loop's increment lands on nb
    }
    cp_async_wait<0>();
    return stat;
}

template <bool kHist, bool kBucket>
__global__ void __launch_bounds__(kQThreads, kBucket ? 3 : 4) quantize_pack_kernel(
    PlanDev p, const float* __restrict__ grads, uint32_t step, uint32_t* __restrict__ packed,
    const float* __restrict__ norms, float* __restrict__ bucket_norms, uint32_t* __restrict__ hist,
    const uint32_t* __restrict__ prev_packed, const float* __restrict__ prev_norms,
    const float* __restrict__ levels_cur, const float* __restrict__ levels_prev, SearchTables st)
{
    __shared__ QuantSmem sm;
    extern __shared__ float4 ring_mem[];              // [warp][row][lane] float4
    const Tile tile = p.tiles[blockIdx.x];
    const int layer = tile.layer;
    const LayerDesc L = p.layers[layer];
    const int k = blockIdx.y + p.worker0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t kl = (int64_t)k * p.num_layers + layer;
    // bucket scope: the tables hold the plain levels (norm 1) and each row multiplies by its own norm
    const float ncur = kBucket ? 1.0f : norms[kl];
    const float nprev = kBucket ? 1.0f : (prev_norms ? prev_norms[kl] : 0.0f);
    const bool fast = st.fast[layer] != 0;
    const int n = L.nlevels;

    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const float l = levels_cur[(int64_t)layer * kLevelStride + i];
        const float c = __fmul_rn(ncur, l);
        const float q = __fmul_rn(nprev, levels_prev[(int64_t)layer * kLevelStride + i]);
        sm.ld[i] = st.ld[(int64_t)layer * kMaxLevels + i];
        sm.lev[i] = l;
        sm.tcur[2 * i] = c;  sm.tcur[2 * i + 1] = -c;
        sm.tprev[2 * i] = q; sm.tprev[2 * i + 1] = -q;
    }
    if (fast)
        for (int i = threadIdx.x; i < LQ_NUM_BINS; i += blockDim.x)
            sm.lut[i] = st.lut[(int64_t)layer * kLutStride + i];
    if (kHist)
        for (int i = threadIdx.x; i < LQ_HIST_STRIDE; i += blockDim.x) sm.hist[i] = 0;
    if (threadIdx.x < tile.nblocks) {
        // a previous message whose masks are unknown is taken as nonzero everywhere
        const int64_t mb = (int64_t)k * p.total_blocks + L.block_off + tile.block0 + threadIdx.x;
        sm.rows_cur[threadIdx.x] = kBucket ? (uint8_t)0xff : p.row_mask[mb];
        sm.rows_prev[threadIdx.x] = !prev_packed ? (uint8_t)0
                                    : ((p.row_mask_prev && !kBucket) ? p.row_mask_prev[mb] : (uint8_t)0xff);
    }
    __syncthreads();

    WarpCtx c;
    c.g = grads + (int64_t)blockIdx.y * p.padded_elems + L.elem_off;
    c.size = L.size;
    c.ring_ptr = ring_mem + (warp * kRingRows) * 32 + lane;
    c.ring = (uint32_t)__cvta_generic_to_shared(c.ring_ptr);
    c.r = kBucket ? 1.0f : p.rnorm[kl];
    c.lane = lane;
    const bool zeroed = c.r == 0.0f;
    BucketCtx bk{nullptr, nullptr, p.q, 0.0, 0u};
    if (kBucket) {
        const int64_t bo = (int64_t)k * p.total_blocks * 8 + L.block_off * 8;
        bk.prev_bn = prev_norms ? prev_norms + bo : nullptr;
        bk.bn_out = bucket_norms + bo;
    }
    if (step == LQ_STEP_AUTO) step = (uint32_t)p.scalars->t;      // the plan's own iteration counter (graph replays)
    const PhiloxConsts pc = philox_fold((uint32_t)layer, (uint32_t)k, step, p.seed_lo, p.seed_hi);
    uint32_t* out = packed + (int64_t)k * p.packed_words + L.word_off;
    const uint32_t* prev = prev_packed ? prev_packed + (int64_t)k * p.packed_words + L.word_off : nullptr;

    double stat = 0.0;
    switch (zeroed ? -L.bits : L.bits * 2 + (fast ? 1 : 0)) {
#define LQ_CASE(BB)                                                                              \
    case -BB:        stat = zeroed_tile<BB>(tile, lane, out, prev, sm); break;                   \
    case 2 * BB:     stat = quantize_tile<BB, false, kHist, kBucket>(p, pc, c, tile, out, prev, sm, bk); break;  \
    case 2 * BB + 1: stat = quantize_tile<BB, true, kHist, kBucket>(p, pc, c, tile, out, prev, sm, bk); break;
        LQ_CASE(1) LQ_CASE(2) LQ_CASE(3) LQ_CASE(4) LQ_CASE(5) LQ_CASE(6) LQ_CASE(7) LQ_CASE(8)
#undef LQ_CASE
        default: break;
    }
    const double total = block_reduce<false>(stat, sm.scratch);
    if (threadIdx.x == 0) p.stat_partial[(int64_t)k * p.num_tiles + blockIdx.x] = total;
    if (kBucket) {
        const double energy = block_reduce<false>(bk.energy, sm.scratch);
        const int any_bad = __syncthreads_or((int)(bk.flags & 1u));
        const int any_live = __syncthreads_or((int)(bk.flags & 2u));
        if (threadIdx.x == 0) {
            p.energy_partial[(int64_t)k * p.num_tiles + blockIdx.x] = energy;
            p.flag_partial[(int64_t)k * p.num_tiles + blockIdx.x] = (any_bad ? 1u : 0u) | (any_live ? 2u : 0u);
        }
    }

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
    const int m = blockIdx.x, k = blockIdx.y + p.worker0;
    const LayerDesc L = p.layers[m];
    const double* part = p.stat_partial + (int64_t)k * p.num_tiles + L.first_tile;
    double acc = 0.0;
    for (int i = threadIdx.x; i < L.ntiles; i += blockDim.x) acc += part[i];
    const double total = block_reduce<false>(acc, scratch);
    if (threadIdx.x == 0) p.sq_diff[(int64_t)k * p.num_layers + m] = total;
}

// Bucket scope: per (layer, worker), in tile order: the statistic, the layer's energy (its weight in the level fit,
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

// One CTA per layer: derives the encode-side tables from the layer's levels.
//   ld[tau]  = {l_tau, l_{tau+1} - l_tau}                 tau = 0..n-2 (other entries: {l_tau, 0})
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
        float2 e = make_float2(i < n ? lev[i] : 0.f, 0.f);
        if (i <= n - 2) e.y = __fsub_rn(lev[i + 1], lev[i]);
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
    const dim3 grid((unsigned)p.num_tiles, (unsigned)p.worker_count);
    if (hist)
        quantize_pack_kernel<true, false><<<grid, kQThreads, kRingBytes, s>>>(p, grads, step, packed, norms, nullptr, hist,
                                                                                prev_packed, prev_norms, levels_cur, levels_prev, t);
    else
        quantize_pack_kernel<false, false><<<grid, kQThreads, kRingBytes, s>>>(p, grads, step, packed, norms, nullptr, hist,
                                                                                 prev_packed, prev_norms, levels_cur, levels_prev, t);
    return cudaGetLastError();
}

cudaError_t launch_quantize_bucketed(const PlanDev& p, const float* grads, uint32_t step, uint32_t* packed,
                                     float* bucket_norms, uint32_t* hist, const uint32_t* prev_packed,
                                     const float* prev_norms, const float* levels_cur,
                                     const float* levels_prev, SearchTables t, cudaStream_t s)
{
    if (p.num_tiles == 0) return cudaSuccess;
    const dim3 grid((unsigned)p.num_tiles, (unsigned)p.worker_count);
    if (hist)
        quantize_pack_kernel<true, true><<<grid, kQThreads, kRingBytes, s>>>(p, grads, step, packed, nullptr, bucket_norms, hist,
                                                                               prev_packed, prev_norms, levels_cur, levels_prev, t);
    else
        quantize_pack_kernel<false, true><<<grid, kQThreads, kRingBytes, s>>>(p, grads, step, packed, nullptr, bucket_norms, hist,
                                                                                prev_packed, prev_norms, levels_cur, levels_prev, t);
    return cudaGetLastError();
}

cudaError_t launch_bucket_finalize(const PlanDev& p, cudaStream_t s)
{
    bucket_finalize_kernel<<<dim3((unsigned)p.num_layers, (unsigned)p.worker_count), 128, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_stat_finalize(const PlanDev& p, cudaStream_t s)
{
    stat_finalize_kernel<<<dim3((unsigned)p.num_layers, (unsigned)p.worker_count), 128, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace lq
