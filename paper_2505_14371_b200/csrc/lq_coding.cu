// Entropy stage on top of the fixed-width message (appendix on the coding framework: with the level
// frequencies known or estimated, a Huffman code on the level symbols; one sign bit per non-zero entry).
//
// A layer's code is a set of word lengths (1..12 bits) for its 2^b level indices; the words are the
// canonical ones (symbols ordered by length, then index; first word all zeros, each next word the
// previous plus one, shifted left when the length grows), written most significant bit first.
//
// Stream format of one worker: the blocks of 1024 coordinates of the fixed-width layout, layer after
// layer, each block starting on a 32-bit word.  Inside a block the coordinates come in the order
// s = 32 * lane + p (lane = 0..31, p = 0..31), i.e. coordinate 128 * (p / 4) + 4 * lane + p % 4 of the block;
// padding coordinates past the layer's end are left out.  Each coordinate contributes its level's word and,
// when the level index is not 0, its sign bit.  Stream bit t of a block is bit t % 32 of its word t / 32.
// block_offsets[k][i] is the first word of block i in worker k's stream, block_offsets[k][blocks] its length.
#include <algorithm>
#include <vector>

#include "lq_internal.cuh"

namespace lq {

// ---- host: Huffman lengths and canonical tables ------------------------------------------------

// Lengths of a Huffman code for n symbols (two-queue construction on the sorted weights), every symbol
// with a word; weights below a floor are raised to it, and the floor doubles until no word is longer
// than max_len.
bool huffman_lengths_host(const double* w, int n, int max_len, uint8_t* len)
{
    if (n == 1) { len[0] = 1; return true; }
    double total = 0.0;
    for (int i = 0; i < n; ++i) { if (!(w[i] >= 0.0)) return false; total += w[i]; }
    if (!(total > 0.0)) total = 1.0;
    double floor_w = total * 9.094947017729282e-13;            // 2^-40 of the total
    std::vector<int> order(n), parent(2 * n), depth(2 * n);
    std::vector<double> wt(2 * n);
    for (;;) {
        for (int i = 0; i < n; ++i) { wt[i] = std::max(w[i], floor_w); order[i] = i; }
        std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return wt[a] < wt[b]; });
        // leaves are taken from `order`, merged trees from a second queue that is born sorted
        int leaf = 0, tree = n, made = n;
        auto take = [&]() {
            if (leaf < n && (tree >= made || wt[order[leaf]] <= wt[tree])) return order[leaf++];
            return tree++;
        };
        for (int m = 0; m < n - 1; ++m) {
            const int a = take(), b = take();
            wt[made] = wt[a] + wt[b];
            parent[a] = made; parent[b] = made;
            ++made;
        }
        parent[made - 1] = -1;
        depth[made - 1] = 0;
        for (int v = made - 2; v >= 0; --v) depth[v] = depth[parent[v]] + 1;
        int longest = 0;
        for (int i = 0; i < n; ++i) { len[i] = (uint8_t)depth[i]; longest = std::max(longest, depth[i]); }
        if (longest <= max_len) return true;
        floor_w *= 2.0;
    }
}

// Canonical words of the lengths; returns false unless the lengths describe a prefix code (Kraft sum <= 1).
bool canonical_codes_host(const uint8_t* len, int n, int max_len, uint32_t* code)
{
    uint64_t kraft = 0;                                        // in units of 2^-max_len
    for (int i = 0; i < n; ++i) {
        if (len[i] < 1 || len[i] > max_len) return false;
        kraft += (uint64_t)1 << (max_len - len[i]);
    }
    if (kraft > ((uint64_t)1 << max_len)) return false;
    uint32_t next = 0; int prev = 0;
    for (int l = 1; l <= max_len; ++l)
        for (int i = 0; i < n; ++i)
            if (len[i] == l) { next <<= (l - prev); code[i] = next; next += 1; prev = l; }
    return true;
}

static uint32_t reverse_bits(uint32_t v, int l)
{
    uint32_t r = 0;
    for (int j = 0; j < l; ++j) r |= ((v >> j) & 1u) << (l - 1 - j);
    return r;
}

// enc[sym] = word with its first bit in bit 0 | length << 16.  dec[next kCodeMaxLen stream bits] = symbol |
// length << 8, or 0xffff where no word matches (incomplete codes).
void build_code_tables_host(const uint8_t* len, const uint32_t* code, int n, uint32_t* enc, uint16_t* dec)
{
    for (int i = 0; i < kMaxLevels; ++i) enc[i] = 0;
    for (int i = 0; i < (1 << kCodeMaxLen); ++i) dec[i] = 0xffffu;
    for (int s = 0; s < n; ++s) {
        const int l = len[s];
        const uint32_t rev = reverse_bits(code[s], l);
        enc[s] = rev | ((uint32_t)l << 16);
        for (uint32_t hi = 0; hi < ((uint32_t)1 << (kCodeMaxLen - l)); ++hi)
            dec[rev | (hi << l)] = (uint16_t)(s | (l << 8));
    }
}

// ---- device ------------------------------------------------------------------------------------
namespace {

// symbol p of a lane's string of 32 symbols of C bits held in C words (C is a run-time value here)
__device__ __forceinline__ uint32_t symbol_at(const uint32_t* w, int C, int p)
{
    const int off = p * C, i = off >> 5, s = off & 31;
    const uint64_t two = ((uint64_t)w[i + 1] << 32) | w[i];
    return (uint32_t)(two >> s) & ((1u << C) - 1u);
}

// Number of real coordinates among the 32 of this lane in block `blk`: coordinate of position p is
// blk * 1024 + 128 * (p / 4) + 4 * lane + p % 4.
__device__ __forceinline__ bool real_coord(int64_t blk, int lane, int p, int64_t size)
{
    return blk * kBlockCoords + 128 * (p >> 2) + 4 * lane + (p & 3) < size;
}

// mode 0: words needed by every block -> sizes[k][block].   mode 1: write the blocks at their offsets.
template <int kModeWrite>
__global__ void __launch_bounds__(kThreads) entropy_encode_kernel(PlanDev p, const uint32_t* __restrict__ packed,
                                                                  const uint32_t* __restrict__ enc_tables,
                                                                  uint32_t* __restrict__ offsets,
                                                                  uint32_t* __restrict__ out, int64_t capacity,
                                                                  uint16_t* __restrict__ run_offsets)
{
    __shared__ uint32_t enc[kMaxLevels];
    __shared__ uint32_t buf[kWarps][1056];
    Tile tile = p.tiles[blockIdx.x >> p.sub_shift];
    const int sub0 = (blockIdx.x & (p.sub_tiles - 1)) * kSubBlocks;
    if (sub0 >= tile.nblocks) return;
    const int sub1 = min(sub0 + kSubBlocks, tile.nblocks);
    const int layer = tile.layer, k = blockIdx.y;
    const LayerDesc L = p.layers[layer];
    const int C = L.bits + 1, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < kMaxLevels; i += blockDim.x) enc[i] = enc_tables[(int64_t)layer * kMaxLevels + i];
    __syncthreads();
    const uint32_t* msg = packed + (int64_t)k * p.packed_words + L.word_off;
    uint32_t* off_k = offsets + (int64_t)k * (p.total_blocks + 1);
    for (int b = sub0 + warp; b < sub1; b += kWarps) {
        const int64_t blk = tile.block0 + b;
        uint32_t w[LQ_MAX_BITS + 2];
        for (int i = 0; i < C; ++i) w[i] = msg[blk * (int64_t)C * 32 + i * 32 + lane];
        w[C] = 0u;
        uint32_t bits = 0;                                   // bits of this lane's 32 coordinates
        for (int pp = 0; pp < 32; ++pp) {
            if (!real_coord(blk, lane, pp, L.size)) continue;
            const uint32_t sym = symbol_at(w, C, pp);
            bits += (enc[sym >> 1] >> 16) + ((sym >> 1) != 0u ? 1u : 0u);
        }
        uint32_t incl = bits;                                // inclusive prefix sum over the lanes
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
        const uint32_t nwords = (total + 31u) >> 5;
        if (!kModeWrite) {
            if (lane == 0) off_k[L.block_off + blk] = nwords;
            continue;
        }
        for (uint32_t i = lane; i < nwords; i += 32) buf[warp][i] = 0u;
        __syncwarp();
        uint32_t pos = incl - bits;
        // where the runs of four lanes (128 coordinates) start inside the block's stream: lets a decoder work on
        // eight runs of a block at once
        if (run_offsets && (lane & 3) == 0)
            run_offsets[((int64_t)k * p.total_blocks + L.block_off + blk) * LQ_CODE_RUNS + (lane >> 2)] = (uint16_t)pos;
        for (int pp = 0; pp < 32; ++pp) {
            if (!real_coord(blk, lane, pp, L.size)) continue;
            const uint32_t sym = symbol_at(w, C, pp), idx = sym >> 1;
            const uint32_t e = enc[idx], l = e >> 16;
            uint32_t val = e & 0xffffu, nb = l;
            if (idx != 0u) { val |= (sym & 1u) << l; nb += 1u; }
            const uint32_t wi = pos >> 5, sh = pos & 31u;
            atomicOr(&buf[warp][wi], val << sh);
            if (sh + nb > 32u) atomicOr(&buf[warp][wi + 1], val >> (32u - sh));
            pos += nb;
        }
        __syncwarp();
        const int64_t first = off_k[L.block_off + blk];
        if (first + nwords <= capacity) {                    // a stream buffer that is too small is never overrun
            uint32_t* dst = out + (int64_t)k * capacity + first;
            for (uint32_t i = lane; i < nwords; i += 32) dst[i] = buf[warp][i];
        }
        __syncwarp();
    }
}

// Exclusive prefix sum of each worker's block sizes, in place; entry [blocks] receives the total.
__global__ void __launch_bounds__(1024) entropy_scan_kernel(PlanDev p, uint32_t* __restrict__ offsets)
{
    __shared__ uint32_t part[1024];
    uint32_t* a = offsets + (int64_t)blockIdx.x * (p.total_blocks + 1);
    const int64_t n = p.total_blocks;
    const int64_t per = (n + 1023) / 1024, lo = threadIdx.x * per, hi = min(n, lo + per);
    uint32_t sum = 0;
    for (int64_t i = lo; i < hi; ++i) sum += a[i];
    part[threadIdx.x] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t run = 0;
        for (int i = 0; i < 1024; ++i) { const uint32_t t = part[i]; part[i] = run; run += t; }
        a[n] = run;
    }
    __syncthreads();
    uint32_t run = part[threadIdx.x];
    for (int64_t i = lo; i < hi; ++i) { const uint32_t t = a[i]; a[i] = run; run += t; }
}

// One thread per (block, worker): walks the block's stream and rebuilds the fixed-width words.
__global__ void __launch_bounds__(128) entropy_decode_kernel(PlanDev p, const uint32_t* __restrict__ in, int64_t capacity,
                                                             const uint32_t* __restrict__ offsets,
                                                             const uint16_t* __restrict__ dec_tables,
                                                             uint32_t* __restrict__ packed, uint32_t* __restrict__ bad)
{
    const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int k = blockIdx.y;
    if (g >= p.total_blocks) return;
    // the layer that owns global block g (layers are few: a linear search over their block ranges)
    int layer = 0;
    while (layer + 1 < p.num_layers && p.layers[layer + 1].block_off <= g) ++layer;
    while (p.layers[layer].nblocks == 0 && layer + 1 < p.num_layers) ++layer;
    const LayerDesc L = p.layers[layer];
    const int64_t blk = g - L.block_off;
    const int C = L.bits + 1;
    const uint16_t* dec = dec_tables + (int64_t)layer * (1 << kCodeMaxLen);
    const uint32_t* off_k = offsets + (int64_t)k * (p.total_blocks + 1);
    const int64_t first = off_k[g], last = min((int64_t)off_k[g + 1], capacity);
    const uint32_t* src = in + (int64_t)k * capacity;
    uint32_t* dst = packed + (int64_t)k * p.packed_words + L.word_off + blk * (int64_t)C * 32;
    int64_t wi = first;                                       // next word to load
    uint64_t window = 0; int have = 0;                        // `have` valid bits in the low end of `window`
    bool broken = false;
    for (int lane = 0; lane < 32; ++lane) {
        uint32_t cw[LQ_MAX_BITS + 2];
        for (int i = 0; i <= C; ++i) cw[i] = 0u;
        for (int pp = 0; pp < 32; ++pp) {
            if (!real_coord(blk, lane, pp, L.size)) continue;
            while (have <= 32) { const uint32_t x = wi < last ? src[wi] : 0u; ++wi; window |= (uint64_t)x << have; have += 32; }
            const uint32_t e = dec[window & ((1u << kCodeMaxLen) - 1u)];
            if (e == 0xffffu) { broken = true; continue; }
            const uint32_t idx = e & 0xffu, l = e >> 8;
            window >>= l; have -= (int)l;
            uint32_t sym = idx << 1;
            if (idx != 0u) { sym |= (uint32_t)(window & 1u); window >>= 1; have -= 1; }
            const int off = pp * C, i = off >> 5, s = off & 31;
            cw[i] |= sym << s;
            if (s + C > 32) cw[i + 1] |= sym >> (32 - s);
        }
        for (int i = 0; i < C; ++i) dst[i * 32 + lane] = cw[i];
    }
    if (broken || wi - 2 > last) atomicOr(bad, 1u);           // no valid word, or the block ran past its end
}

// One thread per run of four lanes (128 coordinates) of a block, eight threads per block, one CTA per sub-tile
// (32 blocks of one layer): every thread starts at its run's recorded bit offset and rebuilds its four lanes' words.
// The decode table of the layer sits in shared memory.  A thread that meets no valid word, that would read past
// the block's end, or that does not end where the next run starts reports a broken stream; nothing is read or
// written out of bounds.
template <int C>
__device__ __forceinline__ void decode_run(const uint32_t* __restrict__ src, int64_t first, int64_t last, uint32_t start_bit,
                                           uint32_t end_bit, bool check_end, const uint16_t* dec, int64_t blk, int run,
                                           int64_t size, uint32_t* __restrict__ dst, bool& broken)
{
    int64_t wi = first + (start_bit >> 5);                    // next word to load
    uint64_t window = 0;
    int have = 0;                                             // valid bits in the low end of `window`
    {
        const uint32_t x = wi < last ? __ldg(src + wi) : 0u; ++wi;
        window = (uint64_t)(x >> (start_bit & 31u));
        have = 32 - (int)(start_bit & 31u);
    }
    uint32_t used = start_bit;
    const bool full = (blk + 1) * kBlockCoords <= size;
    // A run of 128 one-bit words "0" for level index 0 (what untouched rows turn into when 0 is the most frequent
    // level): 128 zero bits, recognised without walking them.
    if (full && check_end && end_bit - start_bit == 128u && dec[0] == (uint16_t)(1u << 8)) {
        const int sh = (int)(start_bit & 31u);
        const int64_t w0 = first + (start_bit >> 5);
        uint32_t any = 0;
        if (w0 + 4 + (sh ? 1 : 0) <= last) {
            any = __ldg(src + w0) >> sh;
#pragma unroll
            for (int i = 1; i < 4; ++i) any |= __ldg(src + w0 + i);
            if (sh) any |= __ldg(src + w0 + 4) << (32 - sh);
            if (any == 0u) {
                for (int l4 = 0; l4 < 4; ++l4)
#pragma unroll
                    for (int i = 0; i < C; ++i) dst[i * 32 + 4 * run + l4] = 0u;
                return;
            }
        }
    }
    for (int l4 = 0; l4 < 4; ++l4) {
        const int lane = 4 * run + l4;
        uint32_t cw[C + 1];
#pragma unroll
        for (int i = 0; i <= C; ++i) cw[i] = 0u;
#pragma unroll
        for (int pp = 0; pp < 32; ++pp) {
            if (!full && !(blk * kBlockCoords + 128 * (pp >> 2) + 4 * lane + (pp & 3) < size)) continue;
            if (have <= 32) { const uint32_t x = wi < last ? __ldg(src + wi) : 0u; ++wi; window |= (uint64_t)x << have; have += 32; }
            const uint32_t e = dec[window & ((1u << kCodeMaxLen) - 1u)];
            if (e == 0xffffu) { broken = true; continue; }
            const uint32_t idx = e & 0xffu, l = e >> 8;
            window >>= l; have -= (int)l; used += l;
            uint32_t sym = idx << 1;
            if (idx != 0u) { sym |= (uint32_t)(window & 1u); window >>= 1; have -= 1; used += 1u; }
            const int off = pp * C, i = off >> 5, s = off & 31;
            cw[i] |= sym << s;
            if (s + C > 32) cw[i + 1] |= sym >> (32 - s);
        }
#pragma unroll
        for (int i = 0; i < C; ++i) dst[i * 32 + lane] = cw[i];
    }
    if (check_end ? used != end_bit : ((int64_t)((used + 31u) >> 5) > last - first)) broken = true;
}

__global__ void __launch_bounds__(kThreads) entropy_decode_runs_kernel(PlanDev p, const uint32_t* __restrict__ in, int64_t capacity,
                                                                       const uint32_t* __restrict__ offsets,
                                                                       const uint16_t* __restrict__ run_offsets,
                                                                       const uint16_t* __restrict__ dec_tables,
                                                                       uint32_t* __restrict__ packed, uint32_t* __restrict__ bad)
{
    __shared__ uint16_t dec[1 << kCodeMaxLen];
    const Tile tile = p.tiles[blockIdx.x >> p.sub_shift];
    const int sub0 = (blockIdx.x & (p.sub_tiles - 1)) * kSubBlocks;
    if (sub0 >= tile.nblocks) return;
    const int layer = tile.layer, k = blockIdx.y;
    const LayerDesc L = p.layers[layer];
    {
        const uint4* src = reinterpret_cast<const uint4*>(dec_tables + ((int64_t)layer << kCodeMaxLen));
        uint4* dst = reinterpret_cast<uint4*>(dec);
        for (int i = threadIdx.x; i < (1 << kCodeMaxLen) / 8; i += blockDim.x) dst[i] = __ldg(src + i);
    }
    __syncthreads();
    const int b = sub0 + (threadIdx.x >> 3), run = threadIdx.x & 7;
    if (b >= tile.nblocks) return;
    const int64_t blk = tile.block0 + b, g = L.block_off + blk;
    const uint32_t* off_k = offsets + (int64_t)k * (p.total_blocks + 1);
    const int64_t first = off_k[g], last = min((int64_t)off_k[g + 1], capacity);
    const uint16_t* ro = run_offsets + ((int64_t)k * p.total_blocks + g) * LQ_CODE_RUNS;
    const uint32_t start_bit = ro[run];
    const uint32_t end_bit = run + 1 < LQ_CODE_RUNS ? (uint32_t)ro[run + 1] : 0u;
    const int C = L.bits + 1;
    uint32_t* dst = packed + (int64_t)k * p.packed_words + L.word_off + blk * (int64_t)C * 32;
    const uint32_t* src = in + (int64_t)k * capacity;
    bool broken = first + (start_bit >> 5) > last;            // an offset that points past the block's end
    if (broken) {                                             // the run's words are still written (zeros), nothing is read
        for (int l4 = 0; l4 < 4; ++l4)
            for (int i = 0; i < C; ++i) dst[i * 32 + 4 * run + l4] = 0u;
    } else {
        switch (C) {
#define LQ_CASE(CC) case CC: decode_run<CC>(src, first, last, start_bit, end_bit, run + 1 < LQ_CODE_RUNS, dec, blk, run, L.size, dst, broken); break;
            LQ_CASE(2) LQ_CASE(3) LQ_CASE(4) LQ_CASE(5) LQ_CASE(6) LQ_CASE(7) LQ_CASE(8) LQ_CASE(9)
#undef LQ_CASE
            default: break;
        }
    }
    if (broken) atomicOr(bad, 1u);
}

}  // namespace

cudaError_t launch_entropy_encode(const PlanDev& p, const uint32_t* packed, const uint32_t* enc_tables,
                                  uint32_t* offsets, uint32_t* out, int64_t capacity, uint16_t* run_offsets, cudaStream_t s)
{
    if (p.num_tiles == 0) return cudaSuccess;
    const dim3 grid((unsigned)p.num_tiles * p.sub_tiles, (unsigned)p.num_workers);
    entropy_encode_kernel<0><<<grid, kThreads, 0, s>>>(p, packed, enc_tables, offsets, out, capacity, nullptr);
    entropy_scan_kernel<<<(unsigned)p.num_workers, 1024, 0, s>>>(p, offsets);
    entropy_encode_kernel<1><<<grid, kThreads, 0, s>>>(p, packed, enc_tables, offsets, out, capacity, run_offsets);
    return cudaGetLastError();
}

cudaError_t launch_entropy_decode(const PlanDev& p, const uint32_t* in, int64_t capacity, const uint32_t* offsets,
                                  const uint16_t* run_offsets, const uint16_t* dec_tables, uint32_t* packed, uint32_t* bad,
                                  cudaStream_t s)
{
    if (p.total_blocks == 0) return cudaSuccess;
    if (run_offsets) {
        const dim3 grid_r((unsigned)p.num_tiles * p.sub_tiles, (unsigned)p.num_workers);
        entropy_decode_runs_kernel<<<grid_r, kThreads, 0, s>>>(p, in, capacity, offsets, run_offsets, dec_tables, packed, bad);
        return cudaGetLastError();
    }
    const dim3 grid((unsigned)((p.total_blocks + 127) / 128), (unsigned)p.num_workers);
    entropy_decode_kernel<<<grid, 128, 0, s>>>(p, in, capacity, offsets, dec_tables, packed, bad);
    return cudaGetLastError();
}

}  // namespace lq
