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

}  // namespace lq
