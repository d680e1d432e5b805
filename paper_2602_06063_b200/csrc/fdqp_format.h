// Format variants of the 32 x 256 block container (the paper calls its dequantisation logic format-agnostic and names
// other group sizes and MXFP4 as formats the container is meant to take).  Every variant keeps the code section of
// the Q4NX block (4096 bytes: eight 32-row x 32-column tiles, two codes per byte); what follows differs:
//   Q4NX   : 256 bf16 scales, 256 bf16 offsets (one per row and group of 32)          -> 5120 bytes
//   group 64 : 128 + 128 (one per row and group of 64)                                 -> 4608 bytes
//   group 128:  64 +  64                                                               -> 4352 bytes
//   MXFP4  : codes are E2M1 elements; 256 E8M0 scale bytes (row r of group t at t*32 + r), no offsets -> 4352 bytes
// The variants need K % 256 == 0 (whole blocks).  Plain data, shared by host and device code.
#pragma once
#include <stdint.h>

namespace fdqp {

constexpr int kFmtQ4nx = 0, kFmtG64 = 1, kFmtG128 = 2, kFmtMxfp4 = 3, kFmtCount = 4;
constexpr int kCodeBytes = 4096;  // code section of a full block = start of the scale section

template <int FMT>
struct FmtTraits;
template <>
struct FmtTraits<kFmtQ4nx> {
    static constexpr int kBlock = 5120, kShift = 0, kOffSect = 4608;
    static constexpr bool kMx = false;
};
template <>
struct FmtTraits<kFmtG64> {
    static constexpr int kBlock = 4608, kShift = 1, kOffSect = 4096 + 256;
    static constexpr bool kMx = false;
};
template <>
struct FmtTraits<kFmtG128> {
    static constexpr int kBlock = 4352, kShift = 2, kOffSect = 4096 + 128;
    static constexpr bool kMx = false;
};
template <>
struct FmtTraits<kFmtMxfp4> {
    static constexpr int kBlock = 4352, kShift = 0, kOffSect = 0;
    static constexpr bool kMx = true;
};

constexpr int fmt_block_bytes(int fmt) {
    return fmt == kFmtQ4nx ? 5120 : fmt == kFmtG64 ? 4608 : (fmt == kFmtG128 || fmt == kFmtMxfp4) ? 4352 : 0;
}
constexpr int fmt_group(int fmt) { return fmt == kFmtG64 ? 64 : fmt == kFmtG128 ? 128 : (fmt == kFmtQ4nx || fmt == kFmtMxfp4) ? 32 : 0; }

// The MXFP4 element as an unsigned byte: 2 * value + 12 (0 .. 24), so that the unsigned integer MMA applies and the
// constant goes where the Q4NX offset goes (-12 * half the scale, times the group's sum of x).
constexpr int kMxBias = 12;  // w = (byte - 12) / 2 * scale

}  // namespace fdqp
