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

#include "lq_coding.cuh"

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

// enc[level] = word with its first bit in bit 0 | length << 16.  dec: the table of lq_coding.cuh.
void build_code_tables_host(const uint8_t* len, const uint32_t* code, int n, uint32_t* enc, uint16_t* dec)
{
    for (int i = 0; i < kMaxLevels; ++i) enc[i] = 0;
    for (int i = 0; i < kDecEntries; ++i) dec[i] = (uint16_t)(kDecInvalid | (1u << kDecLenShift));
    for (int s = 0; s < n; ++s) {
        const int l = len[s];
        const uint32_t rev = reverse_bits(code[s], l);
        enc[s] = rev | ((uint32_t)l << 16);
        for (uint32_t hi = 0; hi < ((uint32_t)1 << (kDecBits - l)); ++hi) {
            const uint32_t sign = s != 0 ? (hi & 1u) : 0u;             // the bit right after the word
            dec[rev | (hi << l)] = (uint16_t)((2u * (uint32_t)s + sign) | ((uint32_t)(l + (s != 0 ? 1 : 0)) << kDecLenShift));
        }
    }
}

// ---- device ------------------------------------------------------------------------------------
namespace {

// Number of real coordinates among the 32 of this lane in block `blk`: coordinate of position p is
// blk * 1024 + 128 * (p / 4) + 4 * lane + p % 4.
__device__ __forceinline__ bool real_coord(int64_t blk, int lane, int p, int64_t size)
{
    return blk * kBlockCoords + 128 * (p >> 2) + 4 * lane + (p & 3) < size;
}

// symbol p of a lane's string of 32 symbols of C bits held in C words
template <int C>
__device__ __forceinline__ uint32_t symbol_at(const uint32_t (&w)[C + 1], int p)
{
    const int off = p * C, i = off >> 5, s = off & 31;
    const uint32_t v = s + C <= 32 ? w[i] >> s : __funnelshift_r(w[i], w[i + 1], s);
    return v & ((1u << C) - 1u);
}

// Bits that a lane's 32 coordinates take in the stream.  code[symbol] = stream bits of the coordinate (word, then
// the sign bit of a non-zero level; first bit in bit 0) | their number << 16.
template <int C, bool kFull>
__device__ __forceinline__ uint32_t lane_bits(const uint32_t* code, const uint32_t (&w)[C + 1], int64_t blk, int lane,
                                              int64_t size)
{
    uint32_t bits = 0;
#pragma unroll
    for (int pp = 0; pp < 32; ++pp) {
        if (!kFull && !real_coord(blk, lane, pp, size)) continue;
        bits += code[symbol_at<C>(w, pp)] >> 16;
    }
    return bits;
}

// Writes a lane's coordinates into the block's buffer from bit `pos` on.  The lane's bits gather in a 64-bit word and
// leave 32 at a time: the first and the last word it touches may be shared with its neighbours (atomic OR into the
// zeroed buffer), the words between them are its own (plain stores).  Whole blocks are taken two coordinates at a
// time: with fewer than 32 bits waiting, two coordinates (at most 26 bits) still fit.
template <int C, bool kFull>
__device__ __forceinline__ void lane_emit(const uint32_t* code, const uint32_t (&w)[C + 1], int64_t blk, int lane,
                                          int64_t size, uint32_t pos, uint32_t* buf)
{
    uint64_t acc = 0;
    uint32_t f = pos & 31u;
    uint32_t* dst = buf + (pos >> 5);
    bool first = true;
#pragma unroll
    for (int pp = 0; pp < 32; ++pp) {
        if (!kFull && !real_coord(blk, lane, pp, size)) continue;
        const uint32_t e = code[symbol_at<C>(w, pp)];
        acc |= (uint64_t)(e & 0xffffu) << f;
        f += e >> 16;
        if ((kFull ? (pp & 1) == 1 : true) && f >= 32u) {
            if (first) atomicOr(dst, (uint32_t)acc); else *dst = (uint32_t)acc;
            first = false;
            ++dst; acc >>= 32; f -= 32u;
        }
    }
    if (f) atomicOr(dst, (uint32_t)acc);
}

constexpr int kCodeBufWords = kBlockCoords * (kCodeMaxLen + 1) / 32;      // longest block: every coordinate 13 bits

// What the warps of an encoder CTA share about their sub-tile.
struct EncodeJob {
    const uint32_t* msg;         // the layer's words in this worker's message
    uint32_t* off;               // this worker's block sizes / offsets, at the layer's first block
    uint32_t* out;               // this worker's stream
    uint16_t* runs;              // this worker's run offsets at the layer's first block, or NULL
    uint16_t* lane_bits;         // this worker's bits per lane and block, at the layer's first block
    int64_t capacity, size;      // words of the stream buffer; coordinates of the layer
    int block0, block1;          // the sub-tile's blocks [block0, block1) of the layer
};

// A warp's blocks of a sub-tile for one symbol width (its own function per width, so that each is compiled with
// its own register budget).  kWrite = false: the words each block needs -> off[block].  true: the blocks are
// written at off[block].
template <int C, bool kWrite>
__device__ __noinline__ void encode_blocks(const EncodeJob& J, const uint32_t* code, uint32_t* bb)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t zero_code = code[0];
    for (int64_t blk = J.block0 + warp; blk < J.block1; blk += kWarps) {
        const bool full = (blk + 1) * kBlockCoords <= J.size;
        uint32_t w[C + 1];
        uint32_t any = 0;
#pragma unroll
        for (int i = 0; i < C; ++i) {
            w[i] = J.msg[blk * (int64_t)C * 32 + i * 32 + lane];
            any |= w[i];
        }
        w[C] = 0u;
        // a lane whose coordinates are all level 0 (untouched rows): 32 times the word of level 0
        const bool plain = full && any == 0u;
        uint32_t bits;
        if (kWrite) bits = J.lane_bits[blk * 32 + lane];     // sized by the first pass
        else {
            bits = 32u * (zero_code >> 16);
            if (!plain) bits = full ? lane_bits<C, true>(code, w, blk, lane, J.size) : lane_bits<C, false>(code, w, blk, lane, J.size);
            J.lane_bits[blk * 32 + lane] = (uint16_t)bits;
        }
        uint32_t incl = bits;                                // inclusive prefix sum over the lanes
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
        const uint32_t nwords = (total + 31u) >> 5;
        if constexpr (!kWrite) {
            if (lane == 0) J.off[blk] = nwords;
        } else {
        for (uint32_t i = lane; i < nwords; i += 32) bb[i] = 0u;
        __syncwarp();
        const uint32_t pos = incl - bits;
        // where the runs of four lanes (128 coordinates) start inside the block's stream: lets a decoder work on
        // eight runs of a block at once
        if (J.runs && (lane & 3) == 0) J.runs[blk * LQ_CODE_RUNS + (lane >> 2)] = (uint16_t)pos;
        if (!(plain && (zero_code & 0xffffu) == 0u)) {       // (32 words "0...0" of level 0 are already there)
            if (full) lane_emit<C, true>(code, w, blk, lane, J.size, pos, bb);
            else      lane_emit<C, false>(code, w, blk, lane, J.size, pos, bb);
        }
        __syncwarp();
        const int64_t first = J.off[blk];
        if (first + nwords <= J.capacity) {                  // a stream buffer that is too small is never overrun
            for (uint32_t i = lane; i < nwords; i += 32) J.out[first + i] = bb[i];
        }
        __syncwarp();
        }
    }
}

// One warp per block, one CTA per sub-tile (32 blocks of one layer).
// kModeWrite = 0: words needed by every block -> sizes[k][block].   1: write the blocks at their offsets.
template <int kModeWrite>
__global__ void __launch_bounds__(kThreads, 4) entropy_encode_kernel(PlanDev p, const uint32_t* __restrict__ packed,
                                                                     const uint32_t* __restrict__ enc_tables,
                                                                     uint32_t* __restrict__ offsets,
                                                                     uint32_t* __restrict__ out, int64_t capacity,
                                                                     uint16_t* __restrict__ run_offsets,
                                                                     uint16_t* __restrict__ lane_bits)
{
    __shared__ uint32_t code[2 * kMaxLevels];
    __shared__ uint32_t buf[kModeWrite ? kWarps : 1][kModeWrite ? kCodeBufWords : 1];
    Tile tile = p.tiles[blockIdx.x >> p.sub_shift];
    const int sub0 = (blockIdx.x & (p.sub_tiles - 1)) * kSubBlocks;
    if (sub0 >= tile.nblocks) return;
    const int layer = tile.layer, k = blockIdx.y;
    const LayerDesc L = p.layers[layer];
    // per symbol (2 * level + sign): the level's word, the sign bit behind it unless the level is 0, and their length
    for (int sym = threadIdx.x; sym < 2 * L.nlevels; sym += blockDim.x) {
        const uint32_t e = enc_tables[(int64_t)layer * kMaxLevels + (sym >> 1)], l = e >> 16;
        code[sym] = (sym >> 1) ? ((e & 0xffffu) | ((uint32_t)(sym & 1) << l) | ((l + 1u) << 16)) : e;
    }
    __syncthreads();
    EncodeJob J;
    J.msg = packed + (int64_t)k * p.packed_words + L.word_off;
    J.off = offsets + (int64_t)k * (p.total_blocks + 1) + L.block_off;
    J.out = out + (int64_t)k * capacity;
    J.runs = run_offsets ? run_offsets + ((int64_t)k * p.total_blocks + L.block_off) * LQ_CODE_RUNS : nullptr;
    J.lane_bits = lane_bits + ((int64_t)k * p.total_blocks + L.block_off) * 32;
    J.capacity = capacity; J.size = L.size;
    J.block0 = tile.block0 + sub0; J.block1 = tile.block0 + min(sub0 + kSubBlocks, tile.nblocks);
    uint32_t* bb = buf[kModeWrite ? (threadIdx.x >> 5) : 0];
    switch (L.bits + 1) {
#define LQ_CASE(CC) case CC: encode_blocks<CC, kModeWrite != 0>(J, code, bb); break;
        LQ_CASE(2) LQ_CASE(3) LQ_CASE(4) LQ_CASE(5) LQ_CASE(6) LQ_CASE(7) LQ_CASE(8) LQ_CASE(9)
#undef LQ_CASE
        default: break;
    }
}

// Exclusive prefix sum of each worker's block sizes, in place; entry [blocks] receives the total.  Two launches:
// the sum of every 1024 consecutive sizes, then each CTA adds the sums before its chunk and scans the chunk.
__global__ void __launch_bounds__(1024) entropy_scan_sums_kernel(PlanDev p, const uint32_t* __restrict__ offsets,
                                                                 uint32_t* __restrict__ part)
{
    __shared__ uint32_t red[32];
    const uint32_t* a = offsets + (int64_t)blockIdx.y * (p.total_blocks + 1);
    const int64_t i = (int64_t)blockIdx.x * 1024 + threadIdx.x;
    uint32_t v = i < p.total_blocks ? a[i] : 0u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x < 32) {
        v = red[threadIdx.x];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (threadIdx.x == 0) part[(int64_t)blockIdx.y * gridDim.x + blockIdx.x] = v;
    }
}

__global__ void __launch_bounds__(1024) entropy_scan_apply_kernel(PlanDev p, uint32_t* __restrict__ offsets,
                                                                  const uint32_t* __restrict__ part)
{
    __shared__ uint32_t red[32];
    __shared__ uint32_t base_s;
    uint32_t* a = offsets + (int64_t)blockIdx.y * (p.total_blocks + 1);
    const uint32_t* pk = part + (int64_t)blockIdx.y * gridDim.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // the sum of the chunks before this one (and, in the last CTA, of all chunks: the stream's length)
    uint32_t before = 0, all = 0;
    for (int c = threadIdx.x; c < (int)gridDim.x; c += 1024) {
        const uint32_t v = pk[c];
        all += v;
        if (c < (int)blockIdx.x) before += v;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { before += __shfl_xor_sync(0xffffffffu, before, o); all += __shfl_xor_sync(0xffffffffu, all, o); }
    if (lane == 0) red[warp] = before;
    __syncthreads();
    if (threadIdx.x == 0) { uint32_t t = 0; for (int w = 0; w < 32; ++w) t += red[w]; base_s = t; }
    __syncthreads();
    if (blockIdx.x == gridDim.x - 1) {
        if (lane == 0) red[warp] = all;
        __syncthreads();
        if (threadIdx.x == 0) { uint32_t t = 0; for (int w = 0; w < 32; ++w) t += red[w]; a[p.total_blocks] = t; }
    }
    __syncthreads();
    const int64_t i = (int64_t)blockIdx.x * 1024 + threadIdx.x;
    const uint32_t v = i < p.total_blocks ? a[i] : 0u;
    uint32_t incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) red[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = red[lane], wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += t;
        }
        red[lane] = wi - w;                                  // exclusive over the warps
    }
    __syncthreads();
    if (i < p.total_blocks) a[i] = base_s + red[warp] + incl - v;
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
    const uint16_t* dec = dec_tables + (int64_t)layer * kDecEntries;
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
            const uint32_t e = dec[window & (uint32_t)(kDecEntries - 1)];
            if (e & kDecInvalid) { broken = true; continue; }
            const uint32_t sym = e & 0x1ffu, l = e >> kDecLenShift;
            window >>= l; have -= (int)l;
            const int off = pp * C, i = off >> 5, s = off & 31;
            cw[i] |= sym << s;
            if (s + C > 32) cw[i + 1] |= sym >> (32 - s);
        }
        for (int i = 0; i < C; ++i) dst[i * 32 + lane] = cw[i];
    }
    if (broken || wi - 2 > last) atomicOr(bad, 1u);           // no valid word, or the block ran past its end
}

// Decoder on the run offsets.  A run is four lanes (128 coordinates) of a block; one CTA takes a sub-tile (32 blocks
// of one layer = 256 runs) with the layer's decode table in shared memory.  First every thread looks at one run: a
// run of 128 zero bits where "0" is the word of level 0 (what untouched rows turn into) is written as zeros at once;
// the other runs are collected in a list, so that the walk below is done by full warps and not by the few lanes of
// every warp whose run happens to hold values.  Then thread i walks the i-th run of the list from its recorded bit
// offset: the next 13 stream bits come from a funnel shift over two of three words kept in registers, one table
// lookup gives the symbol and the bits taken (the words are refilled every second coordinate).  A run that meets no
// valid word, that would read past the block's end, or that does not end where the next run starts reports a broken
// stream; nothing is read or written out of bounds.
struct RunRef {
    const uint32_t* src;     // first word of the block's stream
    int nwords;              // words of the block that may be read
    uint32_t start_bit, end_bit;
    bool check_end;          // the run is followed by another run of the block (end_bit is known)
};

__device__ __forceinline__ uint32_t stream_word(const RunRef& r, int i) { return i < r.nwords ? __ldg(r.src + i) : 0u; }

template <int C, bool kFull>
__device__ __forceinline__ bool decode_run(const RunRef& r, const uint16_t* dec, int64_t blk, int run, int64_t size,
                                           uint32_t* __restrict__ dst)
{
    int wi = (int)(r.start_bit >> 5);
    uint32_t lo = stream_word(r, wi), hi = stream_word(r, wi + 1), nx = stream_word(r, wi + 2);
    wi += 3;                                                  // next word to load; `lo` is word wi - 3
    uint32_t sh = r.start_bit & 31u, flags = 0, win = 0;
    // Coordinates are taken in pairs: with sh < 32 the 32 bits from the current position lie inside {lo, hi}, and
    // after the first coordinate (at most 13 bits) they still hold the second one whole.
#pragma unroll 1
    for (int l4 = 0; l4 < 4; ++l4) {
        const int lane = 4 * run + l4;
        uint32_t cw[C + 1];
#pragma unroll
        for (int i = 0; i <= C; ++i) cw[i] = 0u;
#pragma unroll
        for (int pp = 0; pp < 32; ++pp) {
            if (!kFull && !(blk * kBlockCoords + 128 * (pp >> 2) + 4 * lane + (pp & 3) < size)) continue;
            if (kFull ? (pp & 1) == 0 : true) {
                if (sh >= 32u) { sh -= 32u; lo = hi; hi = nx; nx = stream_word(r, wi); ++wi; }
                win = __funnelshift_r(lo, hi, sh);           // 32 stream bits from the current position
            }
            const uint32_t e = dec[win & (uint32_t)(kDecEntries - 1)];
            flags |= e;
            win >>= e >> kDecLenShift;                       // at least 19 bits are left for the pair's second coordinate
            sh += e >> kDecLenShift;
            const uint32_t sym = e & 0x1ffu;
            const int off = pp * C, i = off >> 5, s = off & 31;
            cw[i] += sym << s;                               // the fields do not overlap: a multiply-add
            if (s + C > 32) cw[i + 1] |= sym >> (32 - s);
        }
#pragma unroll
        for (int i = 0; i < C; ++i) dst[i * 32 + lane] = cw[i];
    }
    if (sh >= 32u) { sh -= 32u; ++wi; }                      // (what the next pair's refill would have done)
    const uint32_t used = 32u * (uint32_t)(wi - 3) + sh;
    return (flags & kDecInvalid) != 0u || (r.check_end ? used != r.end_bit : used > 32u * (uint32_t)r.nwords);
}

__global__ void __launch_bounds__(kThreads) entropy_decode_runs_kernel(PlanDev p, const uint32_t* __restrict__ in, int64_t capacity,
                                                                       const uint32_t* __restrict__ offsets,
                                                                       const uint16_t* __restrict__ run_offsets,
                                                                       const uint16_t* __restrict__ dec_tables,
                                                                       uint32_t* __restrict__ packed, uint32_t* __restrict__ bad)
{
    __shared__ __align__(16) uint16_t dec[kDecEntries];
    __shared__ uint8_t todo[kSubBlocks * LQ_CODE_RUNS];
    __shared__ int ntodo;
    static_assert(kSubBlocks * LQ_CODE_RUNS == kThreads, "one thread per run of a sub-tile");
    const Tile tile = p.tiles[blockIdx.x >> p.sub_shift];
    const int sub0 = (blockIdx.x & (p.sub_tiles - 1)) * kSubBlocks;
    if (sub0 >= tile.nblocks) return;
    const int layer = tile.layer, k = blockIdx.y;
    const LayerDesc L = p.layers[layer];
    {
        const uint4* src = reinterpret_cast<const uint4*>(dec_tables + (int64_t)layer * kDecEntries);
        uint4* dst = reinterpret_cast<uint4*>(dec);
        for (int i = threadIdx.x; i < kDecEntries / 8; i += blockDim.x) dst[i] = __ldg(src + i);
    }
    if (threadIdx.x == 0) ntodo = 0;
    const int C = L.bits + 1;
    const uint32_t* off_k = offsets + (int64_t)k * (p.total_blocks + 1);
    const uint32_t* stream = in + (int64_t)k * capacity;
    uint32_t* msg = packed + (int64_t)k * p.packed_words + L.word_off;
    // the run with index t of this sub-tile: block sub0 + t / 8, run t % 8
    auto run_ref = [&](int t, int64_t& blk) {
        blk = tile.block0 + sub0 + (t >> 3);
        const int64_t g = L.block_off + blk;
        const int64_t first = off_k[g], last = min((int64_t)off_k[g + 1], capacity);
        const uint16_t* ro = run_offsets + ((int64_t)k * p.total_blocks + g) * LQ_CODE_RUNS;
        const int run = t & 7;
        RunRef r;
        r.src = stream + first;
        r.nwords = (int)max((int64_t)0, last - first);
        r.start_bit = ro[run];
        r.check_end = run + 1 < LQ_CODE_RUNS;
        r.end_bit = r.check_end ? (uint32_t)ro[run + 1] : 0u;
        return r;
    };
    __syncthreads();

    bool broken = false, walk = false;
    if (sub0 + (threadIdx.x >> 3) < tile.nblocks) {
        int64_t blk;
        const RunRef r = run_ref(threadIdx.x, blk);
        uint32_t* dst = msg + blk * (int64_t)C * 32;
        const int run = threadIdx.x & 7;
        walk = true;
        if ((int64_t)(r.start_bit >> 5) > (int64_t)r.nwords) {            // an offset that points past the block's end:
            broken = true; walk = false;                                 // the run's words are still written (zeros)
            for (int i = 0; i < C; ++i) *reinterpret_cast<uint4*>(dst + i * 32 + 4 * run) = make_uint4(0u, 0u, 0u, 0u);
        } else if ((blk + 1) * kBlockCoords <= L.size && dec[0] == (uint16_t)kDecZeroBit) {
            // 128 coordinates of level 0 are 128 zero bits; the last run of a block is followed by zero padding
            // up to the block's last word
            const uint32_t nbits = r.check_end ? r.end_bit - r.start_bit : 32u * (uint32_t)r.nwords - r.start_bit;
            if (r.check_end ? nbits == 128u : (nbits >= 128u && nbits < 160u)) {
                const uint32_t end = r.start_bit + nbits;
                const int w0 = (int)(r.start_bit >> 5), w1 = (int)(end >> 5);
                uint32_t any = stream_word(r, w0) >> (r.start_bit & 31u);
#pragma unroll
                for (int i = 1; i < 6; ++i) {
                    const uint32_t x = stream_word(r, w0 + i);
                    if (w0 + i < w1) any |= x;
                    else if (w0 + i == w1 && (end & 31u)) any |= x << (32u - (end & 31u));
                }
                if (any == 0u) {
                    walk = false;
                    for (int i = 0; i < C; ++i) *reinterpret_cast<uint4*>(dst + i * 32 + 4 * run) = make_uint4(0u, 0u, 0u, 0u);
                }
            }
        }
    }
    {
        const uint32_t m = __ballot_sync(0xffffffffu, walk);
        int at = 0;
        if ((threadIdx.x & 31) == 0 && m) at = atomicAdd(&ntodo, __popc(m));
        at = __shfl_sync(0xffffffffu, at, 0);
        if (walk) todo[at + __popc(m & ((1u << (threadIdx.x & 31)) - 1u))] = (uint8_t)threadIdx.x;
    }
    __syncthreads();
    if ((int)threadIdx.x < ntodo) {
        const int t = todo[threadIdx.x];
        int64_t blk;
        const RunRef r = run_ref(t, blk);
        uint32_t* dst = msg + blk * (int64_t)C * 32;
        const bool full = (blk + 1) * kBlockCoords <= L.size;
        switch (full ? C : -C) {
#define LQ_CASE(CC) case CC:  broken |= decode_run<CC, true>(r, dec, blk, t & 7, L.size, dst); break;  \
                    case -CC: broken |= decode_run<CC, false>(r, dec, blk, t & 7, L.size, dst); break;
            LQ_CASE(2) LQ_CASE(3) LQ_CASE(4) LQ_CASE(5) LQ_CASE(6) LQ_CASE(7) LQ_CASE(8) LQ_CASE(9)
#undef LQ_CASE
            default: break;
        }
    }
    if (broken) atomicOr(bad, 1u);
}

}  // namespace

cudaError_t launch_entropy_encode(const PlanDev& p, const uint32_t* packed, const uint32_t* enc_tables,
                                  uint32_t* offsets, uint32_t* out, int64_t capacity, uint16_t* run_offsets,
                                  EncodeScratch scratch, cudaStream_t s)
{
    if (p.num_tiles == 0) return cudaSuccess;
    const dim3 grid((unsigned)p.num_tiles * p.sub_tiles, (unsigned)p.num_workers);
    const dim3 chunks((unsigned)((p.total_blocks + 1023) / 1024), (unsigned)p.num_workers);
    entropy_encode_kernel<0><<<grid, kThreads, 0, s>>>(p, packed, enc_tables, offsets, out, capacity, nullptr, scratch.lane_bits);
    entropy_scan_sums_kernel<<<chunks, 1024, 0, s>>>(p, offsets, scratch.scan_part);
    entropy_scan_apply_kernel<<<chunks, 1024, 0, s>>>(p, offsets, scratch.scan_part);
    entropy_encode_kernel<1><<<grid, kThreads, 0, s>>>(p, packed, enc_tables, offsets, out, capacity, run_offsets, scratch.lane_bits);
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
