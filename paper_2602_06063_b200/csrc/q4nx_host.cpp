// Host-side Q4NX container: size, pack, unpack (Sec. "Dequantization Engine" of the paper:
// a 32 x 256 block = 32*256 int4 codes + 256 bf16 scales + 256 bf16 offsets = 5120 bytes).
//
// The container is written in storage order -- strip by strip, block by block, section by
// section -- with a running output cursor; element positions are never computed by a closed
// address formula here, so the packer is a different statement of the layout than the readers
// used to check it.
#include <cstdint>
#include <cstring>

#include "fdqp.h"

namespace {

constexpr int64_t kStripRows = 32;    // output features per strip
constexpr int64_t kGroup = 32;        // quantisation group along K
constexpr int64_t kBlockGroups = 8;   // groups per full block (256 input features)

inline bool shape_ok(int64_t K, int64_t N) {
    return K > 0 && N > 0 && (K % kGroup) == 0 && (N % kStripRows) == 0;
}

inline void put_u16(uint8_t*& cur, uint16_t v) {
    *cur++ = static_cast<uint8_t>(v & 0xff);
    *cur++ = static_cast<uint8_t>(v >> 8);
}

inline uint16_t get_u16(const uint8_t*& cur) {
    uint16_t v = static_cast<uint16_t>(cur[0] | (static_cast<uint16_t>(cur[1]) << 8));
    cur += 2;
    return v;
}

}  // namespace

extern "C" size_t q4nx_packed_bytes(int64_t K, int64_t N) {
    if (!shape_ok(K, N)) return 0;
    return static_cast<size_t>(N / kStripRows) * static_cast<size_t>(K / kGroup) * 640u;
}

extern "C" fdqp_status q4nx_pack(const uint8_t* codes, const uint16_t* scales_bf16, const uint16_t* offsets_bf16,
                                 int64_t K, int64_t N, void* out, size_t out_bytes) {
    if (!codes || !scales_bf16 || !offsets_bf16 || !out) return FDQP_ERR_ARG;
    if (!shape_ok(K, N)) return FDQP_ERR_SHAPE;
    if (out_bytes < q4nx_packed_bytes(K, N)) return FDQP_ERR_SIZE;
    const int64_t groups = K / kGroup;
    uint8_t* cur = static_cast<uint8_t*>(out);
    unsigned bad = 0;
    for (int64_t strip = 0; strip < N / kStripRows; ++strip) {
        const int64_t row0 = strip * kStripRows;
        for (int64_t g0 = 0; g0 < groups; g0 += kBlockGroups) {
            const int64_t g1 = (g0 + kBlockGroups < groups) ? g0 + kBlockGroups : groups;
            // code section: one 32-row x 32-column tile per group, rows in order, two codes per byte
            for (int64_t g = g0; g < g1; ++g) {
                for (int64_t r = 0; r < kStripRows; ++r) {
                    const uint8_t* src = codes + (row0 + r) * K + g * kGroup;
                    for (int p = 0; p < 16; ++p) {
                        const unsigned lo = src[2 * p], hi = src[2 * p + 1];
                        bad |= (lo | hi) & 0xf0u;
                        *cur++ = static_cast<uint8_t>((lo & 15u) | ((hi & 15u) << 4));
                    }
                }
            }
            // scale section, then offset section, same (group, row) order
            for (int64_t g = g0; g < g1; ++g)
                for (int64_t r = 0; r < kStripRows; ++r) put_u16(cur, scales_bf16[(row0 + r) * groups + g]);
            for (int64_t g = g0; g < g1; ++g)
                for (int64_t r = 0; r < kStripRows; ++r) put_u16(cur, offsets_bf16[(row0 + r) * groups + g]);
        }
    }
    return bad ? FDQP_ERR_ARG : FDQP_OK;
}

extern "C" fdqp_status q4nx_unpack(const void* packed, int64_t K, int64_t N, uint8_t* codes, uint16_t* scales_bf16,
                                   uint16_t* offsets_bf16) {
    if (!packed || !codes || !scales_bf16 || !offsets_bf16) return FDQP_ERR_ARG;
    if (!shape_ok(K, N)) return FDQP_ERR_SHAPE;
    const int64_t groups = K / kGroup;
    const uint8_t* cur = static_cast<const uint8_t*>(packed);
    for (int64_t strip = 0; strip < N / kStripRows; ++strip) {
        const int64_t row0 = strip * kStripRows;
        for (int64_t g0 = 0; g0 < groups; g0 += kBlockGroups) {
            const int64_t g1 = (g0 + kBlockGroups < groups) ? g0 + kBlockGroups : groups;
            for (int64_t g = g0; g < g1; ++g) {
                for (int64_t r = 0; r < kStripRows; ++r) {
                    uint8_t* dst = codes + (row0 + r) * K + g * kGroup;
                    for (int p = 0; p < 16; ++p) {
                        const uint8_t byte = *cur++;
                        dst[2 * p] = byte & 15u;
                        dst[2 * p + 1] = byte >> 4;
                    }
                }
            }
            for (int64_t g = g0; g < g1; ++g)
                for (int64_t r = 0; r < kStripRows; ++r) scales_bf16[(row0 + r) * groups + g] = get_u16(cur);
            for (int64_t g = g0; g < g1; ++g)
                for (int64_t r = 0; r < kStripRows; ++r) offsets_bf16[(row0 + r) * groups + g] = get_u16(cur);
        }
    }
    return FDQP_OK;
}

// ---- format variants (group sizes 64 / 128, MXFP4): same storage-order walk, sections per format -------------------

namespace {

inline int variant_group(int format) { return format == FDQP_FMT_G64 ? 64 : format == FDQP_FMT_G128 ? 128 : format == FDQP_FMT_MXFP4 ? 32 : 0; }

inline bool variant_shape_ok(int64_t K, int64_t N) { return K > 0 && N > 0 && (K % 256) == 0 && (N % kStripRows) == 0; }

}  // namespace

extern "C" size_t q4nx_packed_bytes_fmt(int format, int64_t K, int64_t N) {
    if (format == FDQP_FMT_Q4NX) return q4nx_packed_bytes(K, N);
    const int g = variant_group(format);
    if (g == 0 || !variant_shape_ok(K, N)) return 0;
    const size_t meta = format == FDQP_FMT_MXFP4 ? 256u : static_cast<size_t>(2 * 2 * 32 * (256 / g));
    return static_cast<size_t>(N / kStripRows) * static_cast<size_t>(K / 256) * (4096u + meta);
}

extern "C" fdqp_status q4nx_pack_fmt(int format, const uint8_t* codes, const void* scales, const uint16_t* offsets_bf16,
                                     int64_t K, int64_t N, void* out, size_t out_bytes) {
    if (format == FDQP_FMT_Q4NX)
        return q4nx_pack(codes, static_cast<const uint16_t*>(scales), offsets_bf16, K, N, out, out_bytes);
    const int g = variant_group(format);
    if (g == 0) return FDQP_ERR_ARG;
    const bool mx = format == FDQP_FMT_MXFP4;
    if (!codes || !scales || !out || (!mx && !offsets_bf16)) return FDQP_ERR_ARG;
    if (!variant_shape_ok(K, N)) return FDQP_ERR_SHAPE;
    if (out_bytes < q4nx_packed_bytes_fmt(format, K, N)) return FDQP_ERR_SIZE;
    const int64_t groups = K / g, per_block = 256 / g;
    const uint16_t* s16 = static_cast<const uint16_t*>(scales);
    const uint8_t* s8 = static_cast<const uint8_t*>(scales);
    uint8_t* cur = static_cast<uint8_t*>(out);
    unsigned bad = 0;
    for (int64_t strip = 0; strip < N / kStripRows; ++strip) {
        const int64_t row0 = strip * kStripRows;
        for (int64_t blk = 0; blk < K / 256; ++blk) {
            for (int64_t tile = 0; tile < 8; ++tile) {
                for (int64_t r = 0; r < kStripRows; ++r) {
                    const uint8_t* src = codes + (row0 + r) * K + blk * 256 + tile * 32;
                    for (int p = 0; p < 16; ++p) {
                        const unsigned lo = src[2 * p], hi = src[2 * p + 1];
                        bad |= (lo | hi) & 0xf0u;
                        *cur++ = static_cast<uint8_t>((lo & 15u) | ((hi & 15u) << 4));
                    }
                }
            }
            if (mx) {
                for (int64_t gi = 0; gi < per_block; ++gi)
                    for (int64_t r = 0; r < kStripRows; ++r) {
                        const uint8_t e = s8[(row0 + r) * groups + blk * per_block + gi];
                        bad |= (e == 255u) ? 0x100u : 0u;  // the scale format's NaN
                        *cur++ = e;
                    }
            } else {
                for (int64_t gi = 0; gi < per_block; ++gi)
                    for (int64_t r = 0; r < kStripRows; ++r) put_u16(cur, s16[(row0 + r) * groups + blk * per_block + gi]);
                for (int64_t gi = 0; gi < per_block; ++gi)
                    for (int64_t r = 0; r < kStripRows; ++r) put_u16(cur, offsets_bf16[(row0 + r) * groups + blk * per_block + gi]);
            }
        }
    }
    return bad ? FDQP_ERR_ARG : FDQP_OK;
}

extern "C" fdqp_status q4nx_unpack_fmt(int format, const void* packed, int64_t K, int64_t N, uint8_t* codes, void* scales,
                                       uint16_t* offsets_bf16) {
    if (format == FDQP_FMT_Q4NX) return q4nx_unpack(packed, K, N, codes, static_cast<uint16_t*>(scales), offsets_bf16);
    const int g = variant_group(format);
    if (g == 0) return FDQP_ERR_ARG;
    const bool mx = format == FDQP_FMT_MXFP4;
    if (!packed || !codes || !scales || (!mx && !offsets_bf16)) return FDQP_ERR_ARG;
    if (!variant_shape_ok(K, N)) return FDQP_ERR_SHAPE;
    const int64_t groups = K / g, per_block = 256 / g;
    uint16_t* s16 = static_cast<uint16_t*>(scales);
    uint8_t* s8 = static_cast<uint8_t*>(scales);
    const uint8_t* cur = static_cast<const uint8_t*>(packed);
    for (int64_t strip = 0; strip < N / kStripRows; ++strip) {
        const int64_t row0 = strip * kStripRows;
        for (int64_t blk = 0; blk < K / 256; ++blk) {
            for (int64_t tile = 0; tile < 8; ++tile) {
                for (int64_t r = 0; r < kStripRows; ++r) {
                    uint8_t* dst = codes + (row0 + r) * K + blk * 256 + tile * 32;
                    for (int p = 0; p < 16; ++p) {
                        const uint8_t byte = *cur++;
                        dst[2 * p] = byte & 15u;
                        dst[2 * p + 1] = byte >> 4;
                    }
                }
            }
            if (mx) {
                for (int64_t gi = 0; gi < per_block; ++gi)
                    for (int64_t r = 0; r < kStripRows; ++r) s8[(row0 + r) * groups + blk * per_block + gi] = *cur++;
            } else {
                for (int64_t gi = 0; gi < per_block; ++gi)
                    for (int64_t r = 0; r < kStripRows; ++r) s16[(row0 + r) * groups + blk * per_block + gi] = get_u16(cur);
                for (int64_t gi = 0; gi < per_block; ++gi)
                    for (int64_t r = 0; r < kStripRows; ++r) offsets_bf16[(row0 + r) * groups + blk * per_block + gi] = get_u16(cur);
            }
        }
    }
    return FDQP_OK;
}
