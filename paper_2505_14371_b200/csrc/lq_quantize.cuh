// Pieces shared by the two encoder kernels (lq_quantize.cu: layer and global norm scope; lq_quantize_bucket.cu:
// bucket scope): the shared-memory map of a CTA's tables, the folded Philox4x32-10, the per-coordinate
// step (Section 3.1: normalise, find the interval, round stochastically; Section 3.2: form the symbol) and the
// packing of a lane's 32 symbols into b+1 words.
//
// Table lookups dominate the per-coordinate work, so every table sits at a fixed offset from one base that is
// aligned to 8 KB, and the code carries ABSOLUTE 32-bit shared-memory addresses from one lookup to the next:
//   search table  u32[2048]  at +0x0000, indexed by the top 13 bits of the pattern of u (sign, exponent, 4 mantissa
//                            bits: 16 bins per octave over the whole fp32 range).  Entry = 8 * tau0 in bits 3..10,
//                            tau0 the last level at or below the bin's lower edge, and in bits 13..31 the low 19
//                            bits of the one level that may lie inside the bin, minus one (all ones: no such level),
//                            so that "u is at or above that level" is one unsigned compare of (bits(u) << 13) with
//                            the entry.  A 4-byte entry per bin spreads neighbouring bins over all 32 banks.
//   {l, gap}      float2[256] at +0x2000: {l_tau, l_{tau+1} - l_tau}
//   cur values    float[512]  at +0x2800: fp32(N * l_idx) at 2 * idx, its negative at 2 * idx + 1 (bucket scope: N = 1)
//   prev values   float[512]  at +0x3000: the same for the previous message
// The address of the {l, gap} entry is (entry & 0x7F8) | base_ld: one logic operation.  Adding 8 for each of the two
// decisions and 4 for the sign turns it into base_ld + 4 * symbol, from which the current value is a load at a
// constant offset; the previous value's address is (shifted word & mask) | base_prev.  No address additions.
// The packed words are accumulated from these absolute values as well: every word starts at minus the sum of
// what the constant part (base_ld) contributes to it, so the part that is left is exactly the symbols.
#pragma once

#include "lq_internal.cuh"

namespace lq {

constexpr int kQWarps = kWarps;                    // warps per CTA of the encoder kernels
constexpr int kQThreads = kQWarps * 32;

constexpr uint32_t kSmLut = 0x0000;
constexpr uint32_t kSmLd = 0x2000;
constexpr uint32_t kSmTcur = 0x2800;
constexpr uint32_t kSmTprev = 0x3000;
constexpr uint32_t kSmRows = 0x3800;               // u8[kTileBlocks] rows of this input, u8[kTileBlocks] of the previous one
constexpr uint32_t kSmScratch = 0x3900;            // double[kQWarps]
constexpr uint32_t kSmTables = 0x3A00;             // end of the tables = start of the per-warp rings (a multiple of 512)
constexpr uint32_t kSmRing = kSmTables;
constexpr uint32_t kRingBytes = kQWarps * 8 * 512; // 8 rows of 512 bytes per warp
constexpr uint32_t kSmHist = kSmRing + kRingBytes; // u32[LQ_HIST_STRIDE], histogram mode only
constexpr uint32_t kSmAlign = 0x2000;              // the base is rounded up to this inside the dynamic allocation,
constexpr uint32_t kSmSlack = kSmAlign - 16;       // which is 16-byte aligned at least: the most the rounding can skip
// (tables + ring + slack = 55 792 bytes: four CTAs fit in the 227 KB of an SM)
constexpr uint32_t kHistClamp = 0x33780000u;       // bit pattern one histogram bin below 2^-24

// ---- shared-memory loads by absolute 32-bit address (volatile only pins their place after the barrier that
// ---- follows the table fill; the tables do not change afterwards)
__device__ __forceinline__ uint32_t lds_u32(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds_u8(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ float lds_f32(uint32_t a)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(a));
    return v;
}
template <int kOff>
__device__ __forceinline__ float lds_f32_at(uint32_t a)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(a), "n"(kOff));
    return v;
}
__device__ __forceinline__ float2 lds_f32x2(uint32_t a)
{
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(a));
    return v;
}

// x + 8 when the comparison holds, else x: one compare and one predicated add
__device__ __forceinline__ uint32_t add8_if_gt_u32(uint32_t x, uint32_t a, uint32_t b)
{
    asm("{\n\t.reg .pred p;\n\tsetp.gt.u32 p, %1, %2;\n\t@p add.u32 %0, %0, 8;\n\t}" : "+r"(x) : "r"(a), "r"(b));
    return x;
}
__device__ __forceinline__ uint32_t add8_if_lt(uint32_t x, float a, float b)
{
    asm("{\n\t.reg .pred p;\n\tsetp.lt.f32 p, %1, %2;\n\t@p add.u32 %0, %0, 8;\n\t}" : "+r"(x) : "f"(a), "f"(b));
    return x;
}
// x + 8 when a <= b, else x
__device__ __forceinline__ uint32_t add8_if_le(uint32_t x, float a, float b)
{
    asm("{\n\t.reg .pred p;\n\tsetp.le.f32 p, %1, %2;\n\t@p add.u32 %0, %0, 8;\n\t}" : "+r"(x) : "f"(a), "f"(b));
    return x;
}
// x + 4 when v < 0 (so neither zero sets the sign bit of a symbol), else x
__device__ __forceinline__ uint32_t add4_if_negative(uint32_t x, float v)
{
    asm("{\n\t.reg .pred p;\n\tsetp.lt.f32 p, %1, 0f00000000;\n\t@p add.u32 %0, %0, 4;\n\t}" : "+r"(x) : "f"(v));
    return x;
}

// ---- packing: symbol p of a lane (C = b + 1 bits) sits at bit offset p * C of the lane's string of C words ----
// What the constant part a2 = base_ld / 4 of the absolute values adds to word i: a2 * pack_mult(i), plus
// a2 >> pack_carry(i) from the one symbol that straddles into word i (pack_carry = 0: none).
template <int C>
__host__ __device__ constexpr uint32_t pack_mult(int i)
{
    uint32_t m = 0;
    for (int p = 0; p < 32; ++p)
        if (((p * C) >> 5) == i) m += 1u << ((p * C) & 31);
    return m;
}
template <int C>
__host__ __device__ constexpr int pack_carry(int i)
{
    for (int p = 0; p < 32; ++p) {
        const int s = (p * C) & 31;
        if (s + C > 32 && ((p * C) >> 5) + 1 == i) return 32 - s;
    }
    return 0;
}
// Words of an empty block, prepared for absolute values: minus the constant part's contribution.
// base_ld is a multiple of 2048, so a2 is a multiple of 512 >= 2^(bits a straddling symbol carries over).
template <int C>
__device__ __forceinline__ void pack_begin(uint32_t (&w)[C], uint32_t base_ld)
{
    const uint32_t a2 = base_ld >> 2;
#pragma unroll
    for (int i = 0; i < C; ++i) {
        const uint32_t m = pack_mult<C>(i);
        const int cs = pack_carry<C>(i);
        w[i] = 0u - (a2 * m + (cs ? (a2 >> cs) : 0u));
    }
}
// Adds symbol p given as base_ld + 4 * symbol.
template <int C>
__device__ __forceinline__ void pack_symbol(uint32_t (&w)[C], int p, uint32_t abs4)
{
    const int off = p * C, i = off >> 5, s = off & 31;
    w[i] += s >= 2 ? (abs4 << (s - 2)) : (abs4 >> (2 - s));
    if (s + C > 32) w[i + 1] += abs4 >> (34 - s);
}
// A row that sends zeros (symbols 0): only the constant part.
template <int C>
__device__ __forceinline__ void pack_zero_row(uint32_t (&w)[C], int j, uint32_t base_ld)
{
#pragma unroll
    for (int e = 0; e < 4; ++e) pack_symbol<C>(w, 4 * j + e, base_ld);
}

// shared-memory address of the previous value of symbol p: (its 4 * symbol) | base_prev (a multiple of 2048)
template <int C>
__device__ __forceinline__ uint32_t prev_value_addr(const uint32_t (&w)[C], int p, uint32_t base_prev)
{
    const int off = p * C, i = off >> 5, s = off & 31;
    constexpr uint32_t mask4 = ((1u << C) - 1u) << 2;
    uint32_t v;
    if (s + C <= 32) v = s >= 2 ? (w[i] >> (s - 2)) : (w[i] << (2 - s));
    else             v = __funnelshift_r(w[i], w[i + 1], s - 2);      // s >= 2 whenever a symbol straddles
    return (v & mask4) | base_prev;
}

// ---- Philox4x32-10 with counter (c0, layer, worker, step): within one CTA only c0 changes, so half of
// ---- round 0 (the product with the worker word) and half of round 1 (the product with a word that
// ---- depends only on round 0's constant half) are the same for every call and are computed once.
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

// The table bases of this CTA (absolute shared-memory addresses) and the layer's 1/N.
struct QuantEnv {
    uint32_t lut, ld, tprev;
    float r;
    int refine;          // layers whose levels are too dense for the one-lookup search: byte table over the top 15
                         // bits, then up to `refine` steps upwards
    uint32_t* hist;      // the CTA's histogram (generic pointer), histogram mode only
};

// One coordinate: v -> symbol, added to the lane's words `cw` at position pp; its term of the step-size
// statistic (Eq. general_stepsize: fp32 difference of the two decoded values, squared in fp64) added to `stat`.
// x: the coordinate's Philox word.  Bucket scope: the value tables hold the plain signed levels and the row's
// norms (nrow now, pn in the previous message) scale them.  `counted`: the coordinate lies inside the layer
// (histogram mode).
template <int B, int kSearch, bool kHist, bool kStat, bool kBucket>
__device__ __forceinline__ void quantize_coord(const QuantEnv& ev, float v, uint32_t x, int pp,
                                               uint32_t (&cw)[B + 1], const uint32_t (&pw)[B + 1], double& stat,
                                               float nrow, float pn, bool counted)
{
    constexpr int n = 1 << B, C = B + 1;
    // u <= 1 + 2^-23 always (N >= |v| and one rounding each in 1/N and the product), and such a u
    // behaves exactly like u = 1 below, so the min(u, 1) of the definition is not needed
    const float u = __fmul_rn(fabsf(v), ev.r);
    const uint32_t ub = __float_as_uint(u);
    uint32_t t8;                                             // address of {l_tau, gap}
    if (kSearch == 1) {
        const uint32_t e = lds_u32(((ub >> 17) & 0x1FFCu) | ev.lut);
        t8 = add8_if_gt_u32((e & 0x7F8u) | ev.ld, ub << 13, e);
    } else {
        // (u <= 1 + 2^-23 gives bits(u) >> 17 <= 8128; the mask keeps the pattern of a NaN inside the table too)
        t8 = ev.ld + 8u * lds_u8(((ub >> 17) & 0x1FFFu) | ev.lut);
        for (int s = 0; s < ev.refine; ++s) t8 = add8_if_le(t8, lds_f32(t8 + 8u), u);
        t8 = min(t8, ev.ld + 8u * (uint32_t)(n - 2));
    }
    const float2 ld = lds_f32x2(t8);
    const float den = ld.y;
    const float num = __fsub_rn(u, ld.x);
    // rho = (x >> 9) * 2^-23; f = 1 + rho is built from the bits, and fma(f, den, -den) rounds the exact
    // product rho * den once, like the plain multiplication
    // (one funnel shift: the 64-bit value {0x7F, x} moved right by 9 is (x >> 9) | 0x3F800000)
    const float f = __uint_as_float(__funnelshift_r(x, 0x7Fu, 9));
    const float t = __fmaf_rn(f, den, -den);
    const uint32_t i8 = add8_if_lt(t8, t, num);
    const uint32_t abs4 = add4_if_negative(i8, v);          // base_ld + 4 * (2 * idx + sign), sign = (v < 0)
    pack_symbol<C>(cw, pp, abs4);

    if (kHist && counted) atomicAdd(ev.hist + ((max(ub, kHistClamp) - kHistClamp) >> 19), 1u);

    if (kStat) {
        float cur = lds_f32_at<(int)(kSmTcur - kSmLd)>(abs4);
        float prv = lds_f32(prev_value_addr<C>(pw, pp, ev.tprev));
        if (kBucket) { cur = __fmul_rn(cur, nrow); prv = __fmul_rn(prv, pn); }
        const double dd = (double)__fsub_rn(cur, prv);
        stat = fma(dd, dd, stat);
    }
}

// A coordinate that sends zero while the previous message may not: its statistic term is the squared previous value.
template <int C, bool kBucket>
__device__ __forceinline__ void stat_prev_only(const QuantEnv& ev, const uint32_t (&pw)[C], int pp, float pn, double& stat)
{
    float prv = lds_f32(prev_value_addr<C>(pw, pp, ev.tprev));
    if (kBucket) prv = __fmul_rn(prv, pn);
    const double dd = (double)prv;
    stat = fma(dd, dd, stat);
}

// Fills the CTA's tables (all threads; the caller synchronises afterwards).  `sm` is the generic pointer to the
// aligned base.  ncur / nprev: the norms that scale the value tables (1 in bucket scope).
__device__ __forceinline__ void fill_tables(unsigned char* sm, const SearchTables& st, int layer, int n, bool fast,
                                            const float* __restrict__ levels_cur, const float* __restrict__ levels_prev,
                                            float ncur, float nprev, bool hist)
{
    float2* ld = reinterpret_cast<float2*>(sm + kSmLd);
    float* tcur = reinterpret_cast<float*>(sm + kSmTcur);
    float* tprev = reinterpret_cast<float*>(sm + kSmTprev);
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const float c = __fmul_rn(ncur, levels_cur[(int64_t)layer * kLevelStride + i]);
        const float q = __fmul_rn(nprev, levels_prev[(int64_t)layer * kLevelStride + i]);
        ld[i] = st.ld[(int64_t)layer * kMaxLevels + i];
        tcur[2 * i] = c;  tcur[2 * i + 1] = -c;
        tprev[2 * i] = q; tprev[2 * i + 1] = -q;
    }
    if (fast) {
        const uint4* src = reinterpret_cast<const uint4*>(st.lut + (int64_t)layer * kLutEntries);
        uint4* dst = reinterpret_cast<uint4*>(sm + kSmLut);
        for (int i = threadIdx.x; i < kLutEntries / 4; i += blockDim.x) dst[i] = __ldg(src + i);
    }
    if (hist) {
        uint32_t* h = reinterpret_cast<uint32_t*>(sm + kSmHist);
        for (int i = threadIdx.x; i < LQ_HIST_STRIDE; i += blockDim.x) h[i] = 0;
    }
}

// A layer whose message is all zero (zero norm, NaN or Inf inside): zero words, and the statistic is
// the squared previous message.
template <int B>
__device__ __forceinline__ double zeroed_tile(const Tile& tile, int lane, uint32_t* __restrict__ out,
                                              const uint32_t* __restrict__ prev, uint32_t base_prev)
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
            const double dd = (double)lds_f32(prev_value_addr<C>(pw, pp, base_prev));
            stat = fma(dd, dd, stat);
        }
    }
    return stat;
}

// The aligned base of the CTA's tables inside the dynamic shared-memory allocation.
__device__ __forceinline__ unsigned char* table_base(unsigned char* dyn, uint32_t& base_addr)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(dyn);
    base_addr = (a + kSmAlign - 1u) & ~(kSmAlign - 1u);
    return dyn + (base_addr - a);
}

}  // namespace lq
