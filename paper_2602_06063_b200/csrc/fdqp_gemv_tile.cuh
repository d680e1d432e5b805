// Tile-level pieces of the streaming GEMV kernels, shared by the single-call kernel and the chained kernel:
// the split of a block range over persistent CTAs, the fixed-point preparation of the activations, and the load and
// multiply-accumulate of one 32 x 32 group-tile on the integer tensor-core instruction (Eq. 3 inside Eq. 15).
#pragma once
#include "fdqp_device.cuh"
#include "fdqp_format.h"
#include "fdqp_plan.h"

namespace fdqp {

// 32-bit arithmetic is exact (and an order of magnitude cheaper than a 64-bit division) while (G + 1)(T + 1) < 2^32.
__device__ __forceinline__ bool fits32(int64_t G, int64_t T) { return (((uint64_t)(G + 1) * (uint64_t)(T + 1)) >> 32) == 0; }
__device__ __forceinline__ int64_t div_floor(int64_t a, int64_t b, bool small) {
    return small ? (int64_t)((uint32_t)a / (uint32_t)b) : a / b;
}
__device__ __forceinline__ int64_t range_begin(int64_t ci, int64_t G, int64_t T) {
    if (fits32(G, T)) return (int64_t)(((uint32_t)ci * (uint32_t)T) / (uint32_t)G);
    return (ci * T) / G;
}
// index of the CTA whose range [range_begin(ci), range_begin(ci+1)) contains L
__device__ __forceinline__ int64_t cta_of(int64_t L, int64_t G, int64_t T) {
    if (fits32(G, T)) return (int64_t)((((uint32_t)L + 1u) * (uint32_t)G - 1u) / (uint32_t)T);
    return ((L + 1) * G - 1) / T;
}


// ---- activation preparation ------------------------------------------------------------------------
//
// One thread per (group-tile T, token, quarter q): eight consecutive activations of a 32-group.
//
// M <= 2 (SINGLE == true, "column" layout): the group as 31-bit fixed point relative to its largest exponent, in four
//   SIGNED base-256 digits, each digit plane in MMA fragment order ({bytes of even k, bytes of odd k}).  Per (tile,
//   token) a 136-byte record: [plane 3 (most significant): 4 x 8 B by q][plane 2][plane 1][plane 0][{sum x, unit}].
// M >= 3 (SINGLE == false): no fixed point -- the bf16 activations themselves, permuted into the B-fragment order of
//   the bf16 MMA (this thread's 16 bytes become (x0,x4), (x1,x5), (x2,x6), (x3,x7)), 64 bytes per (tile, token) at
//   xq[((T*M + tok)*4 + q)*4], and the group's sum of x at xsc[T*8 + tok].
// `tile` is the group-tile index in x, `slot` the tile's index in the destination (global: the same; shared
// memory: relative to the CTA's K slice).  Must be called by whole quads (the four q of a (tile, token)).
__device__ __forceinline__ uint4 xprep_load(const uint16_t* __restrict__ x, int K, int tile, int tok, int q, bool valid) {
    uint4 v = make_uint4(0, 0, 0, 0);
    if (valid) v = *reinterpret_cast<const uint4*>(x + (int64_t)tok * K + tile * kGroup + q * 8);
    return v;
}

// Eight bf16 sums, each rounded once from the exact sum (the residual stream of a decoder layer stays in bf16).
__device__ __forceinline__ uint4 add_bf16x8(uint4 a, uint4 b) {
    uint4 r;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(r.x) : "r"(a.x), "r"(b.x));
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(r.y) : "r"(a.y), "r"(b.y));
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(r.z) : "r"(a.z), "r"(b.z));
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(r.w) : "r"(a.w), "r"(b.w));
    return r;
}

// Returns true when the group had to be flagged (column layout only; the same value in the four lanes of a quad).
//
// Flagged groups.  The fixed point holds an activation exactly as long as it is an integer multiple of the group's
// unit 2^(e_g - 29) -- true for every bf16 within 2^22 of the group's largest magnitude.  A group with an element that
// is not (a value more than four million times smaller than an outlier beside it, a subnormal beside a normal
// number), or with a non-finite element, is FLAGGED instead of rounded: its record carries unit = 0 and sum = 0, so
// that the tensor-core path contributes exactly nothing for it, and the raw bf16 activations in k order in bytes
// 0..63 (where the planes would be).  The GEMV kernels then evaluate that group in fp32 straight from Eq. 3 (piece_exact_token below).
template <bool SINGLE>
__device__ __forceinline__ bool xprep_item(const uint4 v, int M, int slot, int tok, int q, bool valid,
                                           uint32_t* __restrict__ xq, float* __restrict__ xsc) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float f[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
    float psum = ((f[0] + f[1]) + (f[2] + f[3])) + ((f[4] + f[5]) + (f[6] + f[7]));
    psum += __shfl_xor_sync(0xffffffffu, psum, 1);
    psum += __shfl_xor_sync(0xffffffffu, psum, 2);
    if (!SINGLE) {
        if (!valid) return false;
        uint4 o;
        o.x = __byte_perm(w[0], w[2], 0x5410);  // (x0, x4)
        o.y = __byte_perm(w[0], w[2], 0x7632);  // (x1, x5)
        o.z = __byte_perm(w[1], w[3], 0x5410);  // (x2, x6)
        o.w = __byte_perm(w[1], w[3], 0x7632);  // (x3, x7)
        *reinterpret_cast<uint4*>(xq + ((int64_t)(slot * M + tok) * 4 + q) * 4) = o;
        if (q == 0) xsc[(int64_t)slot * 8 + tok] = psum;
        return false;
    }
    float amax = fmaxf(fmaxf(fmaxf(fabsf(f[0]), fabsf(f[1])), fmaxf(fabsf(f[2]), fabsf(f[3]))),
                       fmaxf(fmaxf(fabsf(f[4]), fabsf(f[5])), fmaxf(fabsf(f[6]), fabsf(f[7]))));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
    // exponent field of the group's largest magnitude, kept where both scale factors are normal floats
    constexpr int kFrac = 29;  // |fixed-point value| <= 2^30: four signed base-256 digits
    int emax = (int)(__float_as_uint(amax) >> 23);
    int inexact = emax == 255 ? 1 : 0;  // an infinity in the group (a NaN fails the comparison below)
    emax = emax < 32 ? 32 : (emax > 254 ? 254 : emax);
    const float to_fixed = __uint_as_float((uint32_t)(254 + kFrac - emax) << 23);  // 2^(127 + kFrac - emax)
    float unit = __uint_as_float((uint32_t)(emax - kFrac) << 23);                  // 2^(emax - 127 - kFrac)
    // I = the nearest integer to x / unit; bytes of (I + 0x80808080) ^ 0x80808080 are the signed digits of I in base
    // 256 (I = 2^24 d3 + 65536 d2 + 256 d1 + d0, each in [-128, 127]).
    uint32_t J[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float scaled = f[i] * to_fixed;  // exact (a power-of-two factor) unless it underflows
        const int I = __float2int_rn(scaled);
        // the element is held exactly iff rounding to an integer changed nothing (and nothing underflowed to zero)
        if ((float)I != scaled || (scaled == 0.f && f[i] != 0.f)) inexact = 1;
        J[i] = ((uint32_t)I + 0x80808080u) ^ 0x80808080u;
    }
    inexact |= __shfl_xor_sync(0xffffffffu, inexact, 1);
    inexact |= __shfl_xor_sync(0xffffffffu, inexact, 2);
    const bool flagged = inexact != 0;
    uint32_t plane[4][2];  // [0] most significant; {even k, odd k}
#pragma unroll
    for (int pl = 0; pl < 4; ++pl) {
        const uint32_t sel = (uint32_t)(3 - pl) | ((uint32_t)(7 - pl) << 4);  // byte 3 - pl of both operands
        const uint32_t e01 = __byte_perm(J[0], J[2], sel), e23 = __byte_perm(J[4], J[6], sel);
        const uint32_t o01 = __byte_perm(J[1], J[3], sel), o23 = __byte_perm(J[5], J[7], sel);
        plane[pl][0] = __byte_perm(e01, e23, 0x5410);
        plane[pl][1] = __byte_perm(o01, o23, 0x5410);
    }
    if (!valid) return false;
    if (flagged) {
        psum = 0.f;
        unit = 0.f;
    }
    constexpr int kRecWords = kColsRecBytes / 4;
    uint32_t* rec = xq + ((int64_t)slot * M + tok) * kRecWords;
    if (flagged) {  // raw activations 8q .. 8q+7 (records are 8-byte aligned)
        *reinterpret_cast<uint2*>(rec + q * 4) = make_uint2(v.x, v.y);
        *reinterpret_cast<uint2*>(rec + q * 4 + 2) = make_uint2(v.z, v.w);
    } else {
#pragma unroll
        for (int pl = 0; pl < 4; ++pl)
            *reinterpret_cast<uint2*>(rec + pl * 8 + q * 2) = make_uint2(plane[pl][0], plane[pl][1]);
    }
    if (q == 0) *reinterpret_cast<uint2*>(rec + kColsSumOff / 4) = make_uint2(__float_as_uint(psum), __float_as_uint(unit));
    return flagged;
}

// ---- one 32 x 32 group-tile -------------------------------------------------------------------------


// Kernel modes (see the header comment): derived constants.
template <int MODE>
struct ModeTraits {
    static constexpr bool kCols = MODE != 2;     // planes as MMA columns (M <= kColsMaxTokens)
    static constexpr int kAcc = kCols ? 1 : 2;   // accumulator columns per lane
    static constexpr bool kXRow = MODE == 3;     // offset term needs the sums of x of both tokens
    static constexpr int kAccM = MODE == 3 ? 2 : 1;
};

struct TileIn {
    uint32_t c[4];   // code words: word q of rows g, g+8, g+16, g+24
    uint32_t so[4];  // column modes: (d[g], d[g+8]), (d[g+16], d[g+24]); mode 2 also (m[g], m[g+8]), (m[g+16], m[g+24])
    uint32_t b[4];   // B fragments: column modes: {even k, odd k} of this lane's column; mode 2: the two k-steps' bf16 pairs
    float sc[2];     // column modes: {sum x, unit} of the lane's token; mode 2: sum of x of tokens 2q, 2q+1
    float xrow[2];   // mode 3: sum of x of tokens 0, 1 for this group
    uint32_t m_row;  // column modes: bf16 offset of row `lane` (low half)
};

// Per-lane pieces of the shared-memory addresses of the prepared activations.
struct LaneAddr {
    uint32_t xs, x_stride;   // base and bytes per tile of the prepared-x records
    uint32_t xb_off;         // column modes: this lane's B column inside the tile
    uint32_t sc_off;         // column modes: {sum x, unit} of the token whose columns this lane accumulates
    uint32_t x_lane, xsc_lane;  // mode 2: this lane's 16 bytes of activations / pair of sums inside tile 0
};

// Column modes: so_addr addresses the scale chunks only (lanes 0..15 matter); m_addr is this lane's own offset word.
// MXFP4: so_addr is the byte address of row g's scale of this tile, m_addr that of row `lane`'s; so[0..3] then hold,
// as fp32 bits, the scales 2^(e-127) of rows g, g+8, g+16, g+24 (a scale byte of 0, i.e. 2^-127, counts as 0 here),
// m_row that of row `lane`; the B fragments are re-ordered to the natural k order the element look-up produces.
__device__ __forceinline__ uint32_t lds_u8(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
// {even k, odd k} byte order of a B fragment pair -> {k 0..3, k 4..7}
__device__ __forceinline__ void mx_natural_order(uint32_t& b0, uint32_t& b1) {
    const uint32_t e = b0, o = b1;
    b0 = prmt(e, o, 0x5140u);
    b1 = prmt(e, o, 0x7362u);
}

template <int MODE, int FMT = kFmtQ4nx>
__device__ __forceinline__ void tile_load(TileIn& t, uint32_t code_addr, uint32_t so_addr, uint32_t m_addr, int tile,
                                          const LaneAddr& la) {
    using T = ModeTraits<MODE>;
    constexpr bool kMx = FmtTraits<FMT>::kMx;
    ldmatrix_x4(t.c, code_addr);
    if (kMx) {
#pragma unroll
        for (int k = 0; k < 4; ++k) t.so[k] = lds_u8(so_addr + 8u * k) << 23;
    }
    if (T::kCols) {
        if (kMx) {
            t.m_row = lds_u8(m_addr) << 23;
        } else {
            uint32_t dd[2];
            ldmatrix_x2_trans(dd, so_addr);
            t.so[0] = dd[0];
            t.so[1] = dd[1];
            asm volatile("ld.shared.u16 %0, [%1];" : "=r"(t.m_row) : "r"(m_addr));
        }
        const uint32_t tb = la.xs + (uint32_t)tile * la.x_stride;
        asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(t.b[0]), "=r"(t.b[1]) : "r"(tb + la.xb_off));
        const float2 v = lds64f(tb + la.sc_off);
        t.sc[0] = v.x;
        t.sc[1] = v.y;
        if (T::kXRow) {  // the sums of x of both tokens (each in its own record)
            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(t.xrow[0]) : "r"(tb + (uint32_t)kColsSumOff));
            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(t.xrow[1]) : "r"(tb + (uint32_t)(kColsRecBytes + kColsSumOff)));
        }
        if (kMx) mx_natural_order(t.b[0], t.b[1]);
    } else {
        if (!kMx) ldmatrix_x4_trans(t.so, so_addr);
        const uint4 r0 = lds128(la.x_lane + (uint32_t)tile * la.x_stride);
        t.b[0] = r0.x; t.b[1] = r0.y; t.b[2] = r0.z; t.b[3] = r0.w;
        const float2 xv = lds64f(la.xsc_lane + (uint32_t)tile * (uint32_t)kPlaneSumBytes);
        t.sc[0] = xv.x;
        t.sc[1] = xv.y;
    }
}

// Eight E2M1 codes of a word -> the unsigned bytes 2v + 12 (0 .. 24) of k 0..3 and k 4..7.  A 16-entry table as two
// byte permutes: a selector nibble with bit 3 set returns the selected byte's sign fill, which is 0 for these bytes, so
// the table of the non-negative codes answers only codes 0..7 and, with bit 3 flipped, that of the negative codes only
// codes 8..15.
// The two answers are disjoint (one of them is 0 in every byte), so they are not merged: each goes through the MMA and
// the accumulator adds them.
struct MxBytes {
    uint32_t pos_lo, pos_hi, neg_lo, neg_hi;
};
// The four table words live in registers for the whole kernel (loaded through an opaque move, so that the compiler
// does not re-create the constants in front of every permute).
struct MxTables {
    uint32_t pos0, pos1, neg0, neg1;
};
__device__ __forceinline__ MxTables mx_tables() {
    MxTables t;
    asm volatile("mov.b32 %0, 0x0F0E0D0C;" : "=r"(t.pos0));  // 12 + {0, 1, 2, 3}
    asm volatile("mov.b32 %0, 0x18141210;" : "=r"(t.pos1));  // 12 + {4, 6, 8, 12}
    asm volatile("mov.b32 %0, 0x090A0B0C;" : "=r"(t.neg0));  // 12 - {0, 1, 2, 3}
    asm volatile("mov.b32 %0, 0x00040608;" : "=r"(t.neg1));  // 12 - {4, 6, 8, 12}
    return t;
}
__device__ __forceinline__ MxBytes mx_codes_to_bytes(uint32_t w, const MxTables& tb) {
    const uint32_t wn = w ^ 0x88888888u;
    MxBytes r;
    r.pos_lo = prmt(tb.pos0, tb.pos1, w);
    r.neg_lo = prmt(tb.neg0, tb.neg1, wn);
    r.pos_hi = prmt(tb.pos0, tb.pos1, w >> 16);
    r.neg_hi = prmt(tb.neg0, tb.neg1, wn >> 16);
    return r;
}

// d += A . B (same shapes and types as imma below)
template <bool B_SIGNED>
__device__ __forceinline__ void imma_acc(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    if (B_SIGNED)
        asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <bool B_SIGNED>
__device__ __forceinline__ void imma(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                     uint32_t b1) {
    const int zero = 0;  // accumulator start value
    if (B_SIGNED)
        asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
            : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(zero));
    else
        asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
            : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(zero));
}

// Per-lane constants of the column modes: which two MMA columns the lane holds.  Columns 4*(tok%2) + {0,1,2,3} are
// digit planes 3, 2, 1, 0 of token tok (of the pair); lane q holds columns 2q, 2q+1:
//   q even: (plane 3, plane 2) -> 256 * s3 + s2, weighted 65536 * unit;   q odd: (plane 1, plane 0) -> 256 * s1 + s0,
//   weighted unit.
struct LaneConst {
    float w_unit;      // factor on `unit` (0 when the lane's token does not exist)
    uint32_t nib_mask, nib_magic;  // mode 2: 0x000F000F and 0x43004300, held in registers for the whole kernel
    MxTables mx;       // MXFP4 only: the element look-up tables
};

// D = A(16x16, bf16, row) * B(16x8, bf16, col) + D, fp32 accumulate (mode 2).
__device__ __forceinline__ void mma_bf16_acc(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// D = A * B (accumulator starts at zero: no registers to clear)
__device__ __forceinline__ void mma_bf16_zero(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                              uint32_t b1) {
    const float zero = 0.f;
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(zero));
}
// Two exact small integers as a bf16 pair: nibbles i and i + 4 of a code word.  (w >> 4i) & 0x000F000F | 0x43004300 is
// the pair (128 + n_i, 128 + n_{i+4}) -- in bf16 the ulp at 128 is 1 -- and the packed subtraction removes the 128.
// The AND and the OR are ONE three-input logic instruction (look-up table 0xEA = (a & b) | c).
__device__ __forceinline__ uint32_t nibble_pair_bf16(uint32_t w, int i, uint32_t mask, uint32_t magic) {
    uint32_t biased, r;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(biased) : "r"(w >> (4 * i)), "r"(mask), "r"(magic));
    asm("sub.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(biased), "r"(magic));
    return r;
}
// The same from two bytes (values up to 127) minus `bias`: bytes `sel` picks from {lo, hi} become the low bytes of the
// halves of 0x43.. patterns.
__device__ __forceinline__ uint32_t byte_pair_bf16(uint32_t packed, uint32_t sel, uint32_t bias_pair) {
    uint32_t r;
    asm("sub.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(prmt(packed, 0x43434343u, sel)), "r"(bias_pair));
    return r;
}

// acc[row][.] += d * unit * (sum_k q_k X_k) + m * (sum_k x_k), fp32 (Eq. 3 applied per group).
// `unit` (and 256 * unit) are powers of two, so d * unit is formed exactly by the mixed bf16 FMA.
// Column modes keep the offset term sum_g m_g * X_g in a lane-per-row layout (acc_m[tok], row = lane).
// MXFP4 (FMT): the element bytes 2v + 12 take the codes' place, half the power-of-two scale takes d's, and -12 times
// that takes m's.
template <int MODE, int FMT = kFmtQ4nx>
__device__ __forceinline__ void tile_compute(const TileIn& t, float (&acc)[4][ModeTraits<MODE>::kAcc],
                                             float (&acc_m)[ModeTraits<MODE>::kAccM], const LaneConst& lc) {
    using T = ModeTraits<MODE>;
    constexpr bool kMx = FmtTraits<FMT>::kMx;
    if (T::kCols) {
        const float mw = kMx ? -0.5f * (float)kMxBias * __uint_as_float(t.m_row) : bf16lo_mul_f32hi(t.m_row, 1.0f);
        if (T::kXRow) {
#pragma unroll
            for (int tk = 0; tk < T::kAccM; ++tk) acc_m[tk] = fmaf(mw, t.xrow[tk], acc_m[tk]);
        } else {
            acc_m[0] = fmaf(mw, t.sc[0], acc_m[0]);
        }
        const float uq = t.sc[1] * lc.w_unit;  // (MXFP4: w_unit carries the 1/2 of the elements' integer form)
#pragma unroll
        for (int h = 0; h < 2; ++h) {  // rows (g, g+8) then (g+16, g+24)
            const uint32_t w0 = t.c[2 * h], w1 = t.c[2 * h + 1];
            int d[4];
            if (kMx) {
                const MxBytes m0 = mx_codes_to_bytes(w0, lc.mx), m1 = mx_codes_to_bytes(w1, lc.mx);  // lo: k 0..3, hi: k 4..7
                imma<true>(d, m0.pos_lo, m1.pos_lo, m0.pos_hi, m1.pos_hi, t.b[0], t.b[1]);
                imma_acc<true>(d, m0.neg_lo, m1.neg_lo, m0.neg_hi, m1.neg_hi, t.b[0], t.b[1]);
            } else {
                const uint32_t e0 = w0 & 0x0F0F0F0Fu, o0 = (w0 >> 4) & 0x0F0F0F0Fu;  // even-k codes, odd-k codes
                const uint32_t e1 = w1 & 0x0F0F0F0Fu, o1 = (w1 >> 4) & 0x0F0F0F0Fu;
                imma<true>(d, e0, e1, o0, o1, t.b[0], t.b[1]);
            }
            const float dq[2] = {kMx ? __uint_as_float(t.so[2 * h]) * uq : bf16lo_mul_f32hi(t.so[h], uq),
                                 kMx ? __uint_as_float(t.so[2 * h + 1]) * uq : bf16hi_mul_f32hi(t.so[h], uq)};
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                // the lane's two digit columns combined in integers (exact, |.| < 2^24), one conversion
                const float s = __int2float_rn(d[2 * r] * 256 + d[2 * r + 1]);
                acc[2 * h + r][0] = fmaf(dq[r], s, acc[2 * h + r][0]);
            }
        }
        return;
    }
    // Mode 2 (M = 3 .. 8): codes and activations are both exact in bf16, the tokens are the MMA's eight columns, the
    // group's 32 inputs two k16 steps; sum_k q_k x_k accumulates in fp32 inside the tensor core.  k order inside a
    // step is a free permutation shared by both operands: code word nibbles (i, i + 4) pair with (x_i, x_{i+4}).
    float dv[4], mv[4];  // rows g, g+8, g+16, g+24
    if (kMx) {
#pragma unroll
        for (int i = 0; i < 4; ++i) dv[i] = 0.5f * __uint_as_float(t.so[i]);  // the element bytes hold twice the value
    } else {
        dv[0] = bf16lo_mul_f32hi(t.so[0], 1.0f);
        dv[1] = bf16hi_mul_f32hi(t.so[0], 1.0f);
        dv[2] = bf16lo_mul_f32hi(t.so[1], 1.0f);
        dv[3] = bf16hi_mul_f32hi(t.so[1], 1.0f);
        mv[0] = bf16lo_mul_f32hi(t.so[2], 1.0f);
        mv[1] = bf16hi_mul_f32hi(t.so[2], 1.0f);
        mv[2] = bf16lo_mul_f32hi(t.so[3], 1.0f);
        mv[3] = bf16hi_mul_f32hi(t.so[3], 1.0f);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {  // rows (g, g+8) then (g+16, g+24)
        const uint32_t w0 = t.c[2 * h], w1 = t.c[2 * h + 1];
        uint32_t a0[4], a1[4];  // rows g + 16h and g + 8 + 16h: pairs (n0,n4), (n1,n5), (n2,n6), (n3,n7)
        if (kMx) {
            // element bytes 2v + 12 in natural k order (lo: k 0..3, hi: k 4..7), interleaved to (k_i, k_{i+4}) pairs
            const MxBytes m0 = mx_codes_to_bytes(w0, lc.mx), m1 = mx_codes_to_bytes(w1, lc.mx);
            const uint32_t lo0 = m0.pos_lo | m0.neg_lo, hi0 = m0.pos_hi | m0.neg_hi;
            const uint32_t lo1 = m1.pos_lo | m1.neg_lo, hi1 = m1.pos_hi | m1.neg_hi;
            const uint32_t p0 = prmt(lo0, hi0, 0x5140u), p1 = prmt(lo0, hi0, 0x7362u);  // (k0,k4,k1,k5), (k2,k6,k3,k7)
            const uint32_t r0 = prmt(lo1, hi1, 0x5140u), r1 = prmt(lo1, hi1, 0x7362u);
            constexpr uint32_t kBias = 0x43004300u + (uint32_t)kMxBias * 0x00010001u;  // 128 + 12 in both halves
            a0[0] = byte_pair_bf16(p0, 0x4140u, kBias); a0[1] = byte_pair_bf16(p0, 0x4342u, kBias);
            a0[2] = byte_pair_bf16(p1, 0x4140u, kBias); a0[3] = byte_pair_bf16(p1, 0x4342u, kBias);
            a1[0] = byte_pair_bf16(r0, 0x4140u, kBias); a1[1] = byte_pair_bf16(r0, 0x4342u, kBias);
            a1[2] = byte_pair_bf16(r1, 0x4140u, kBias); a1[3] = byte_pair_bf16(r1, 0x4342u, kBias);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                a0[i] = nibble_pair_bf16(w0, i, lc.nib_mask, lc.nib_magic);
                a1[i] = nibble_pair_bf16(w1, i, lc.nib_mask, lc.nib_magic);
            }
        }
        float cc[4];  // (row g+16h, tok 2q), (same row, tok 2q+1), (row g+8+16h, tok 2q), (.., 2q+1)
        mma_bf16_zero(cc, a0[0], a1[0], a0[1], a1[1], t.b[0], t.b[1]);
        mma_bf16_acc(cc, a0[2], a1[2], a0[3], a1[3], t.b[2], t.b[3]);
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int i = 2 * h + r;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                acc[i][j] = fmaf(dv[i], cc[2 * r + j], acc[i][j]);
                if (!kMx) acc[i][j] = fmaf(mv[i], t.sc[j], acc[i][j]);
            }
        }
    }
}

// ---- flagged groups: evaluated in fp32 straight from Eq. 3 -----------------------------------------------------------
//
// For a group whose activations the fixed point cannot hold exactly (see xprep_item) the tensor-core path contributes
// zero; before a consumer warp hands a strip piece to the reducer it adds the true contribution of every flagged
// (group-tile, token) among the tiles it processed for that piece.  Lane r owns output row r of the strip and
// accumulates x_k * w_hat(r, k) over the group's 32 inputs in k order, w_hat = fmaf(d, q, m) being the once-rounded
// value of Eq. 3 (MXFP4: element times power-of-two scale, exact).  Error: 32 fp32 roundings relative to the partial
// sums per group, far inside the acceptance bound whatever the activations' range; non-finite activations propagate.
// The weights of those tiles have left the shared-memory ring by then and are read again from global memory: this
// path is rare by construction (no group of ordinary activations is flagged) and is kept out of line and out of the
// tile loop, which never looks at the flags.
//
// Geometry of a warp's share of a piece.  Processing-order position i = bl + pos0 (bl = block index inside the K
// slice); the warp owns the positions with (i mod CB) in [j0, j0 + BPW) and, of each block, group-tile tw.
struct ExactPiece {
    const uint8_t* blk0;   // global address of the strip's first block of this K slice
    int groups_total;      // K / 32
    int b_first;           // first block of the K slice
    int bl_lo, bl_hi;      // the piece's blocks (indices inside the slice)
    int pos0;              // i - bl
    int CB, j0, BPW, tw;
    uint32_t unit0, unit_tile_stride;  // shared-memory address of the token's unit for tile 0, and bytes per tile
    uint32_t raw0, raw_tile_stride;    // the same for the token's raw activations
    uint32_t piece_stride;             // distance between the four 16-byte pieces of the raw activations
};

template <int FMT>
__device__ __noinline__ float piece_exact_token(const ExactPiece e, int lane) {
    using F = FmtTraits<FMT>;
    float acc = 0.f;
    for (int bl = e.bl_lo; bl < e.bl_hi; ++bl) {
        const int i = bl + e.pos0;
        const int in_chunk = i % e.CB - e.j0;
        if (in_chunk < 0 || in_chunk >= e.BPW) continue;
        const int rest = e.groups_total - 8 * (e.b_first + bl);
        const int jb = rest < 8 ? rest : 8;  // groups of this block (short only at the end of K, Q4NX only)
        if (e.tw >= jb) continue;
        const int tile = bl * 8 + e.tw;
        float unit;
        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(unit) : "r"(e.unit0 + (uint32_t)tile * e.unit_tile_stride));
        if (unit != 0.f) continue;  // not flagged (same answer in every lane)
        const uint8_t* blk = e.blk0 + (int64_t)bl * F::kBlock;
        const uint4 c = __ldg(reinterpret_cast<const uint4*>(blk + e.tw * 512 + lane * 16));
        const uint32_t cw[4] = {c.x, c.y, c.z, c.w};
        float d, m = 0.f;
        if (F::kMx) {
            // half the scale: the element table below holds twice the E2M1 value (a scale byte of 0 counts as zero)
            d = 0.5f * __uint_as_float((uint32_t)__ldg(blk + kCodeBytes + e.tw * 32 + lane) << 23);
        } else {
            const int sect = FMT == kFmtQ4nx ? 512 * jb : kCodeBytes;
            const int osect = FMT == kFmtQ4nx ? 576 * jb : (int)F::kOffSect;
            const int word = ((e.tw >> F::kShift) * 32 + lane) * 2;
            d = __uint_as_float((uint32_t)__ldg(reinterpret_cast<const uint16_t*>(blk + sect + word)) << 16);
            m = __uint_as_float((uint32_t)__ldg(reinterpret_cast<const uint16_t*>(blk + osect + word)) << 16);
        }
        const uint32_t raw = e.raw0 + (uint32_t)tile * e.raw_tile_stride;
#pragma unroll 1
        for (int p4 = 0; p4 < 4; ++p4) {
            uint32_t xw[4];  // (the records are 8-byte aligned)
            asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(xw[0]), "=r"(xw[1]) : "r"(raw + (uint32_t)p4 * e.piece_stride));
            asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(xw[2]), "=r"(xw[3]) : "r"(raw + (uint32_t)p4 * e.piece_stride + 8u));
#pragma unroll
            for (int j = 0; j < 4; ++j) {  // byte j of code word p4: k = 8 p4 + 2j in the low nibble, k + 1 in the high one
                const uint32_t byte = (cw[p4] >> (8 * j)) & 0xffu;
                float w0, w1;
                if (F::kMx) {
                    const uint32_t q0 = byte & 15u, q1 = byte >> 4;
                    const float v0 = (float)((0xC8643210u >> (4u * (q0 & 7u))) & 15u) * d;  // 2|value|: 0 1 2 3 4 6 8 12
                    const float v1 = (float)((0xC8643210u >> (4u * (q1 & 7u))) & 15u) * d;
                    w0 = (q0 & 8u) ? -v0 : v0;
                    w1 = (q1 & 8u) ? -v1 : v1;
                } else {
                    w0 = fmaf(d, (float)(byte & 15u), m);
                    w1 = fmaf(d, (float)(byte >> 4), m);
                }
                acc = fmaf(bf16_lo_to_f32(xw[j]), w0, acc);
                acc = fmaf(bf16_hi_to_f32(xw[j]), w1, acc);
            }
        }
    }
    return acc;
}

// OR of a predicate over the `nthreads` threads that meet at named barrier `id` (one barrier instruction).
__device__ __forceinline__ bool named_barrier_or(int id, int nthreads, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.or.pred q, %2, %3, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred), "r"(id), "r"(nthreads)
        : "memory");
    return r != 0;
}

}  // namespace fdqp
