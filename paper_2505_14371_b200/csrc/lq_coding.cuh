// Decode table of the entropy stage (shared by the code that builds it and the kernels that read it).
// One entry per value of the next kDecBits = 13 stream bits (first bit in bit 0): a code word is at most
// kCodeMaxLen = 12 bits and a non-zero level is followed by its sign bit, so 13 bits always hold one whole
// coordinate.  entry = symbol (2 * level index + sign, bits 0..8) | bits taken (word + sign, 1..13) << 12;
// where no word matches (incomplete codes) the entry is kDecInvalid | 1 << 12: the flag (bit 9, which no valid entry
// sets) is sticky when entries are OR-ed together, and a walker still advances.
#pragma once
#include "lq_internal.cuh"

namespace lq {

constexpr int kDecBits = kCodeMaxLen + 1;
constexpr int kDecEntries = 1 << kDecBits;
constexpr uint32_t kDecInvalid = 1u << 9;
constexpr int kDecLenShift = 12;
constexpr uint32_t kDecZeroBit = 1u << kDecLenShift;         // the entry of "level 0 in one bit": symbol 0, one bit taken


// ---- host side of the stage (lq_coding.cu) ----
bool huffman_lengths_host(const double* w, int n, int max_len, uint8_t* len);
bool canonical_codes_host(const uint8_t* len, int n, int max_len, uint32_t* code);
void build_code_tables_host(const uint8_t* len, const uint32_t* code, int n, uint32_t* enc, uint16_t* dec);

// Scratch of the encoder, owned by the plan: the bits every lane of every block takes (filled by the sizing pass and
// read by the writing pass, so that a lane's coordinates are sized once) and the per-1024-blocks sums of the scan.
struct EncodeScratch {
    uint16_t* lane_bits;     // [K][total_blocks][32]
    uint32_t* scan_part;     // [K][ceil(total_blocks / 1024)]
};
cudaError_t launch_entropy_encode(const PlanDev& p, const uint32_t* packed, const uint32_t* enc_tables,
                                  uint32_t* offsets, uint32_t* out, int64_t capacity, uint16_t* run_offsets,
                                  EncodeScratch scratch, cudaStream_t s);
cudaError_t launch_entropy_decode(const PlanDev& p, const uint32_t* in, int64_t capacity, const uint32_t* offsets,
                                  const uint16_t* run_offsets, const uint16_t* dec_tables, uint32_t* packed, uint32_t* bad,
                                  cudaStream_t s);

}  // namespace lq
