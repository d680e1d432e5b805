// Prefill-sized projection (M >= 9 token rows): dequantise Q4NX blocks into shared memory and contract on the
// 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM).
//
// The paper's prefill path dequantises a Q4NX block to bf16, writes it to DRAM and runs a tiled bf16 GEMM on it
// (Sec. "Dequantization Engine", Sec. "Tiling-based MM").  Here the DRAM round trip is removed: the dequantised tile
// only ever exists in shared memory, in the layout the tensor core reads.
//
// The basic form: one CTA computes a 256 (output features) x 256 (tokens) tile of y:
//   D[n][tok] = sum_k w16[k][n] * x[tok][k],   w16 = RNE_bf16( RN_fp32(d * q + m) )      (Eq. 3, then Eq. 14)
//   - UMMA shape 128 x N_inst x 16 (kind::f16, bf16 inputs, fp32 accumulate), two accumulators (rows 0..127 and
//     128..255 of the tile) of 256 TMEM columns each = all 512 columns;
//   - A = dequantised weights, [256 rows][64 k] bf16 per pipeline stage, K-major, 128-byte swizzle, written by sixteen
//     dequantisation warps (one 32-row strip and 32-wide group each) with plain shared-memory stores; each warp reads
//     its codes, scale and offset straight from global memory, eight k-steps ahead;
//   - B = x, [tokens][64 k] bf16 per stage, K-major, 128-byte swizzle, loaded by TMA (2-D tiled copy, no
//     multicast); rows beyond M and columns beyond K are zero-filled by the copy engine;
//   - one elected thread issues the MMAs; tcgen05.commit hands stages back and announces the finished accumulators;
//   - epilogue: the dequantisation warps read TMEM (tcgen05.ld 32x32b) and store fp32 y, 128 contiguous bytes
//     per warp store (bf16 epilogues go through shared memory).
// Up to 128 tokens: 128 x 128 tiles, two CTAs per SM, the converted weights kept in tensor memory (tcgen05.st) and read
// from there by the MMAs; up to 64 tokens a smaller form of that fits three CTAs per SM.  More than 256 tokens: a pair
// of SMs works on a 256 x 512 tile (cta_group::2).  Few tiles: K slices, summed by a second kernel.
// Every wait is bounded; TMEM is released on every path.
#include <cuda.h>

#include "fdqp_device.cuh"
#include "fdqp_format.h"
#include "fdqp_plan.h"

namespace fdqp {

constexpr int kPfRows = 256;      // output features per CTA tile
constexpr int kPfToks = 256;      // tokens per CTA tile
constexpr int kPfK = 64;          // k per pipeline stage (one 128-byte swizzle row of bf16)
constexpr int kPfStages = 3;
constexpr int kPfDequantWarps = 8;   // two-SM kernel: one (strip, group) of the CTA's 128 rows each
constexpr int kPfThreads = (2 + kPfDequantWarps) * 32;  // warp 0: TMA + TMEM owner, warp 1: MMA issuer
constexpr uint32_t kPfTmemCols = 512;

constexpr int kPfTmemAStages = 4, kPfTmemBStages = 6;  // the variant that keeps the weights in tensor memory
// Geometry of the one-SM kernel by tile height (see the kernel).
template <int ROWS>
struct Pf1 {
    static constexpr int kRows = ROWS;
    static constexpr int kToks = ROWS == 256 ? 256 : 128;             // tokens per CTA tile = rows of the x box
    static constexpr uint32_t kABytes = ROWS * kPfK * 2;
    static constexpr uint32_t kBBytes = kToks * kPfK * 2;
    static constexpr uint32_t kStageBytes = kABytes + kBBytes;
    static constexpr int kDequantWarps = ROWS / 16;                   // one (strip, group) of the tile each
    static constexpr int kThreads = (2 + kDequantWarps) * 32;
    static constexpr uint32_t kTmemCols = ROWS == 256 ? 512 : 128;
    static constexpr uint32_t kSmemBytes = kPfStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
    static constexpr int kCtasPerSm = ROWS == 256 ? 1 : 2;
    static constexpr uint32_t kSmemBytesTmemA = kPfTmemBStages * kBBytes + 1024 + 256;  // x stages only
    static constexpr uint32_t kSmemBytesTri = 4 * kBBytes + 1024 + 256;                // three CTAs per SM: four x stages
};

struct PrefillParams {
    const uint8_t* W;
    float* y;       // [M][N] result, or (Z > 1) Z partial results of that shape, one per K slice
    int* status;
    int M, K, N;
    uint16_t* y16;  // bf16 output of the epilogues other than kEpiNone (Z == 1 only; K-split calls leave it to the sum)
    int epi;
    int Z;          // K slices; slice z covers k-steps [z * ksteps_z, (z + 1) * ksteps_z)
    int ksteps_z;   // 64-wide k-steps per slice
    uint32_t x_box_bytes;  // one-SM kernel: bytes of one x box (64 k x the token rows that exist, rounded up to 16)
};

// ---- tcgen05 wrappers -----------------------------------------------------------------------------------------

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem desc] * B[smem desc]; issued by one thread for the whole CTA.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The same with A taken from tensor memory: lane i of a_tmem = row i of A, one 32-bit column = two consecutive k.
__device__ __forceinline__ void umma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 16 consecutive 32-bit columns of this thread's TMEM lane (the warp's lane quarter) <- 16 registers.
__device__ __forceinline__ void tmem_st_16cols(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
// Arrive on `bar` once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Shared-memory matrix descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);  // start address
    d |= (uint64_t)1 << 16;                        // leading-dimension byte offset (unused for this layout)
    d |= (uint64_t)(1024 >> 4) << 32;              // stride-dimension byte offset: next 8-row group
    d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                        // 128-byte swizzle
    return d;
}

// Instruction descriptor, kind::f16: D fp32, A and B bf16, both K-major, M = 128, N = n_inst.
__device__ __forceinline__ uint32_t umma_idesc(uint32_t n_inst) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((n_inst >> 3) << 17) | ((128u >> 4) << 24);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

__device__ __forceinline__ void tmem_ld_32cols(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,"
        "%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ---- dequantisation of one (strip, group) into the swizzled A tile ---------------------------------------------------

struct GroupRegs {
    uint4 codes;      // this lane's row: 32 codes of the group
    uint32_t d_bits;  // bf16 scale in the low half (MXFP4: the E8M0 scale byte)
    uint32_t m_bits;  // bf16 offset in the low half
    bool valid;
};

// g counts 32-column tiles along K; the format variants (whole blocks only) keep the tile's scale and offset at the
// index of the larger group it belongs to.
template <int FMT>
__device__ __forceinline__ GroupRegs group_load(const uint8_t* __restrict__ W, int K, int64_t strip, int g, int lane,
                                                bool strip_ok) {
    using F = FmtTraits<FMT>;
    GroupRegs r;
    const int groups = K / kGroup;
    r.valid = strip_ok && g < groups;
    r.codes = make_uint4(0, 0, 0, 0);
    r.d_bits = 0;
    r.m_bits = 0;
    if (FMT != kFmtQ4nx) {
        if (r.valid) {
            const int b = g >> 3, t = g & 7;
            const uint8_t* blk = W + (strip * (int64_t)(K / kBlockK) + b) * (int64_t)F::kBlock;
            r.codes = __ldg(reinterpret_cast<const uint4*>(blk + t * 512 + lane * 16));
            if (F::kMx) {
                r.d_bits = __ldg(blk + kCodeBytes + t * 32 + lane);
            } else {
                const int at = 2 * ((t >> F::kShift) * 32 + lane);
                r.d_bits = __ldg(reinterpret_cast<const unsigned short*>(blk + kCodeBytes + at));
                r.m_bits = __ldg(reinterpret_cast<const unsigned short*>(blk + F::kOffSect + at));
            }
        }
        return r;
    }
    if (r.valid) {
        const int b = g >> 3, t = g & 7;
        const int rest = groups - 8 * b;
        const int jb = rest < 8 ? rest : 8;
        const uint8_t* blk = W + strip * ((int64_t)kGroupBytes * groups) + (int64_t)b * kBlockBytes;
        r.codes = __ldg(reinterpret_cast<const uint4*>(blk + t * 512 + lane * 16));
        r.d_bits = __ldg(reinterpret_cast<const unsigned short*>(blk + 512 * jb + 2 * (t * 32 + lane)));
        r.m_bits = __ldg(reinterpret_cast<const unsigned short*>(blk + 576 * jb + 2 * (t * 32 + lane)));
    }
    return r;
}

// (low | high) half of a packed bf16 pair times bf16 d plus fp32 m, rounded once to fp32: exactly Eq. 3, because the
// product of an integer code <= 15 and a bf16 scale is exact inside the fused multiply-add.
__device__ __forceinline__ float dequant_lo(uint32_t q2, uint32_t d_bits, float m) {
    float r;
    asm("{\n\t.reg .b16 qlo, qhi, dlo, dhi;\n\tmov.b32 {qlo, qhi}, %1;\n\tmov.b32 {dlo, dhi}, %2;\n\t"
        "fma.rn.f32.bf16 %0, qlo, dlo, %3;\n\t}"
        : "=f"(r) : "r"(q2), "r"(d_bits), "f"(m));
    return r;
}
__device__ __forceinline__ float dequant_hi(uint32_t q2, uint32_t d_bits, float m) {
    float r;
    asm("{\n\t.reg .b16 qlo, qhi, dlo, dhi;\n\tmov.b32 {qlo, qhi}, %1;\n\tmov.b32 {dlo, dhi}, %2;\n\t"
        "fma.rn.f32.bf16 %0, qhi, dlo, %3;\n\t}"
        : "=f"(r) : "r"(q2), "r"(d_bits), "f"(m));
    return r;
}

// Writes row (strip_local*32 + lane), k in [32*gl, 32*gl + 32) of the A tile: w16 = RNE_bf16(RN_fp32(d*q + m)).
// Codes become bf16 pairs with one logic op per pair ((w >> 4i) & 0x000F000F | 0x43004300 = (128+q_i, 128+q_{i+4}));
// the bias is removed exactly by a packed bf16 subtract; no integer-to-float conversion instruction is used.
// An absent group arrives with codes, d and m all zero and therefore writes zeros.
//
// MXFP4: every element times its power-of-two scale is a bf16 number, so the tile is exact.  Eight E2M1 codes become
// bf16 through two byte tables (high and low byte of the magnitude's bf16 pattern, indexed by the code's low three bits
// with one permute per four codes each), the sign bits are moved to bit 7 of the high bytes by one more permute, the
// bytes are interleaved into bf16 pairs, and a packed bf16 multiply applies the scale 2^(e-127) (bf16 bits e << 7).
__device__ __forceinline__ uint32_t pf_prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// (x & 0x000F000F) | 0x43004300 as ONE three-input logic instruction (look-up table 0xEA = (a & b) | c): the bf16 pair
// (128 + nibble 0, 128 + nibble 4) of x; the packed subtraction removes the 128 exactly.
__device__ __forceinline__ uint32_t pf_nibble_pair(uint32_t x) {
    uint32_t biased, r;
    asm("lop3.b32 %0, %1, 0x000F000F, 0x43004300, 0xEA;" : "=r"(biased) : "r"(x));
    asm("sub.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(biased), "r"(0x43004300u));
    return r;
}

template <int FMT>
__device__ __forceinline__ void group_store(uint32_t a_tile, const GroupRegs& r, int strip_local, int gl, int lane) {
    const int row = strip_local * 32 + lane;
    const uint32_t row_base = a_tile + (uint32_t)((row >> 3) * 1024 + (row & 7) * 128);
    const uint32_t r7s = (uint32_t)(row & 7) << 4;
    const uint32_t words[4] = {r.codes.x, r.codes.y, r.codes.z, r.codes.w};
    if (FmtTraits<FMT>::kMx) {
        constexpr uint32_t kHi0 = 0x3F3F3F00u, kHi1 = 0x40404040u;  // bf16 of 0, .5, 1, 1.5 | 2, 3, 4, 6: high bytes
        constexpr uint32_t kLo0 = 0xC0800000u, kLo1 = 0xC0804000u;  //                                     low bytes
        const uint32_t e = r.valid ? r.d_bits : 127u;               // an absent group has zero codes: any scale does
        const uint32_t sc = e ? e << 7 : 0x0040u;                   // bf16 bits of 2^(e-127)
        const uint32_t sc2 = sc | (sc << 16);
#pragma unroll
        for (int wi = 0; wi < 4; ++wi) {  // 8 codes -> one 16-byte chunk
            const uint32_t w = words[wi];
            const uint32_t mag = w & 0x77777777u, w4 = w << 4;
            uint32_t hi_a = pf_prmt(kHi0, kHi1, mag), lo_a = pf_prmt(kLo0, kLo1, mag);              // codes 0..3
            uint32_t hi_b = pf_prmt(kHi0, kHi1, mag >> 16), lo_b = pf_prmt(kLo0, kLo1, mag >> 16);  // codes 4..7
            hi_a |= pf_prmt(w, w4, 0x1504u) & 0x80808080u;  // signs: bit 3 of nibble j -> bit 7 of byte j
            hi_b |= pf_prmt(w, w4, 0x3726u) & 0x80808080u;
            uint32_t o0 = pf_prmt(lo_a, hi_a, 0x5140u), o1 = pf_prmt(lo_a, hi_a, 0x7362u);
            uint32_t o2 = pf_prmt(lo_b, hi_b, 0x5140u), o3 = pf_prmt(lo_b, hi_b, 0x7362u);
            asm("mul.rn.bf16x2 %0, %0, %1;" : "+r"(o0) : "r"(sc2));
            asm("mul.rn.bf16x2 %0, %0, %1;" : "+r"(o1) : "r"(sc2));
            asm("mul.rn.bf16x2 %0, %0, %1;" : "+r"(o2) : "r"(sc2));
            asm("mul.rn.bf16x2 %0, %0, %1;" : "+r"(o3) : "r"(sc2));
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(row_base + (((uint32_t)(gl * 4 + wi) << 4) ^ r7s)),
                         "r"(o0), "r"(o1), "r"(o2), "r"(o3)
                         : "memory");
        }
        return;
    }
    const float m = __uint_as_float(r.m_bits << 16);
#pragma unroll
    for (int wi = 0; wi < 4; ++wi) {  // 8 codes -> one 16-byte chunk
        const uint32_t w = words[wi];
        float f[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t q2 = pf_nibble_pair(w >> (4 * i));  // bf16x2 (q_i, q_{i+4}), exact
            f[i] = dequant_lo(q2, r.d_bits, m);
            f[i + 4] = dequant_hi(q2, r.d_bits, m);
        }
        uint32_t o0, o1, o2, o3;
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o0) : "f"(f[1]), "f"(f[0]));  // {hi, lo}
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o1) : "f"(f[3]), "f"(f[2]));
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o2) : "f"(f[5]), "f"(f[4]));
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o3) : "f"(f[7]), "f"(f[6]));
        // 16-byte chunk (gl*4 + wi) of the 128-byte row, at its swizzled position
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(row_base + (((uint32_t)(gl * 4 + wi) << 4) ^ r7s)),
                     "r"(o0), "r"(o1), "r"(o2), "r"(o3)
                     : "memory");
    }
}

// The same 32 weights as 16 bf16 pairs in k order in registers (for the kernel that keeps the weights in tensor memory).
template <int FMT>
__device__ __forceinline__ void group_convert(const GroupRegs& r, uint32_t (&out)[16]) {
    const uint32_t words[4] = {r.codes.x, r.codes.y, r.codes.z, r.codes.w};
    if (FmtTraits<FMT>::kMx) {
        constexpr uint32_t kHi0 = 0x3F3F3F00u, kHi1 = 0x40404040u, kLo0 = 0xC0800000u, kLo1 = 0xC0804000u;
        const uint32_t e = r.valid ? r.d_bits : 127u;
        const uint32_t sc = e ? e << 7 : 0x0040u;
        const uint32_t sc2 = sc | (sc << 16);
#pragma unroll
        for (int wi = 0; wi < 4; ++wi) {
            const uint32_t w = words[wi];
            const uint32_t mag = w & 0x77777777u, w4 = w << 4;
            uint32_t hi_a = pf_prmt(kHi0, kHi1, mag), lo_a = pf_prmt(kLo0, kLo1, mag);
            uint32_t hi_b = pf_prmt(kHi0, kHi1, mag >> 16), lo_b = pf_prmt(kLo0, kLo1, mag >> 16);
            hi_a |= pf_prmt(w, w4, 0x1504u) & 0x80808080u;
            hi_b |= pf_prmt(w, w4, 0x3726u) & 0x80808080u;
            uint32_t o0 = pf_prmt(lo_a, hi_a, 0x5140u), o1 = pf_prmt(lo_a, hi_a, 0x7362u);
            uint32_t o2 = pf_prmt(lo_b, hi_b, 0x5140u), o3 = pf_prmt(lo_b, hi_b, 0x7362u);
            asm("mul.rn.bf16x2 %0, %0, %1;" : "+r"(o0) : "r"(sc2));
            asm("mul.rn.bf16x2 %0, %0, %1;" : "+r"(o1) : "r"(sc2));
            asm("mul.rn.bf16x2 %0, %0, %1;" : "+r"(o2) : "r"(sc2));
            asm("mul.rn.bf16x2 %0, %0, %1;" : "+r"(o3) : "r"(sc2));
            out[4 * wi] = o0;
            out[4 * wi + 1] = o1;
            out[4 * wi + 2] = o2;
            out[4 * wi + 3] = o3;
        }
        return;
    }
    const float m = __uint_as_float(r.m_bits << 16);
#pragma unroll
    for (int wi = 0; wi < 4; ++wi) {
        const uint32_t w = words[wi];
        float f[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t q2 = pf_nibble_pair(w >> (4 * i));
            f[i] = dequant_lo(q2, r.d_bits, m);
            f[i + 4] = dequant_hi(q2, r.d_bits, m);
        }
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(out[4 * wi]) : "f"(f[1]), "f"(f[0]));
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(out[4 * wi + 1]) : "f"(f[3]), "f"(f[2]));
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(out[4 * wi + 2]) : "f"(f[5]), "f"(f[4]));
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(out[4 * wi + 3]) : "f"(f[7]), "f"(f[6]));
    }
}

// ---- bf16 epilogues: the tile goes through shared memory so that global memory sees whole 128-byte lines --------------
//
// A thread owns one output feature (a TMEM lane) and many tokens, so 2-byte results written straight to y would reach
// memory as 64- or 32-byte pieces of a line per store (measured: twice the time of the fp32 store for half the bytes).
// The warps therefore write their results into the pipeline's shared memory (free once the accumulators are final) as a
// [token][column] bf16 tile, and then copy it out row by row, 16 bytes per lane.

// Copies rows [0, toks) of a [toks][cols] bf16 tile at shared address `stage` (cols * 2 in {128, 256, 512} bytes) to
// dst[t * ld16 + 0 .. valid_cols); warp wi of nwarps, 16-byte chunks, whole warps.
__device__ __forceinline__ void stage_copy_out(uint32_t stage, uint16_t* dst, int64_t ld16, int toks, int cols,
                                               int valid_cols, int wi, int nwarps, int lane) {
    const int cpr = cols / 8;   // 16-byte chunks per tile row: 8, 16 or 32
    const int rpi = 32 / cpr;   // tile rows one warp moves per step
    const int chunk = lane % cpr;
    for (int t = wi * rpi + lane / cpr; t < toks; t += nwarps * rpi) {
        if (chunk * 8 < valid_cols) {
            const uint4 v = lds128(stage + (uint32_t)(t * cols + chunk * 8) * 2u);
            *reinterpret_cast<uint4*>(dst + (int64_t)t * ld16 + chunk * 8) = v;
        }
    }
}

// ---- the kernel -------------------------------------------------------------------------------------------------------

#define PF_T0() do { } while (0)
#define PF_DT() 0

// ROWS: output features per CTA tile.  256: the tile described above, one CTA per SM.  128 (for M <= 128): a 128 x 128
// tile with half-size stages (16 KB + 16 KB), eight conversion warps and 128 TMEM columns, so that TWO CTAs share an SM:
// one CTA's start-up, epilogue and stage latencies overlap the other's main loop.
// ATMEM (with ROWS = 128 only): the converted weights go to tensor memory (tcgen05.st) instead of shared memory and the
// MMA takes its A operand from there, which removes the weights' store and re-read from the shared-memory traffic (at
// <= 128 tokens per MMA that traffic is what the tensor pipe waits for).  Shared memory then holds x stages only (six of
// them); TMEM holds the accumulators (128 columns) and four weight stages of 32 columns (64 k as bf16 pairs).
template <int FMT, int ROWS, bool ATMEM = false, bool TRI = false>
__global__ void __launch_bounds__(Pf1<ROWS>::kThreads, TRI ? 3 : Pf1<ROWS>::kCtasPerSm)
    fdqp_prefill_kernel(const __grid_constant__ CUtensorMap x_map, const PrefillParams p) {
    using P = Pf1<ROWS>;
    static_assert(!ATMEM || ROWS == 128, "weights in tensor memory: 128-row tiles only");
    constexpr int CH = P::kToks / 2;  // token columns per epilogue warp of a quarter
    static_assert(!TRI || ATMEM, "three CTAs per SM: the tensor-memory variant only");
    constexpr int NA = TRI ? 2 : (ATMEM ? kPfTmemAStages : kPfStages);    // weight stages
    constexpr int NB = TRI ? 4 : (ATMEM ? kPfTmemBStages : kPfStages);    // x stages
    constexpr uint32_t kBStride = ATMEM ? P::kBBytes : P::kStageBytes;  // bytes from one x stage to the next
    constexpr uint32_t kBOff = ATMEM ? 0u : P::kABytes;                  // x tile inside its stage
    constexpr uint32_t kRing = NB * kBStride;
    constexpr uint32_t kTmemCols = TRI ? 128u : (ATMEM ? 256u : P::kTmemCols);
    constexpr uint32_t kTmemA = TRI ? 64 : 128;  // ATMEM: first TMEM column of the weight stages
    extern __shared__ uint8_t smem_raw[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // tiles must start on a 1024-byte boundary (swizzle atom)
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t bars = base + kRing;
    // barriers: full_a[NA], full_b[NB], empty_a[NA], empty_b[NB], acc_done; then the TMEM base address slot
    auto full_a = [&](int s) { return bars + 8u * s; };
    auto full_b = [&](int s) { return bars + 8u * (NA + s); };
    auto empty_a = [&](int s) { return bars + 8u * (NA + NB + s); };
    auto empty_b = [&](int s) { return bars + 8u * (2 * NA + NB + s); };
    const uint32_t acc_done = bars + 8u * (2 * NA + 2 * NB);
    const uint32_t tmem_slot = acc_done + 8u;
    const uint32_t staged = tmem_slot + 8u;  // bf16 epilogues: every epilogue warp has written its part of the tile
    volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(smem + kRing + 8 * (2 * NA + 2 * NB + 1));

    const int tok_tiles = (p.M + P::kToks - 1) / P::kToks;
    const int tile_id = blockIdx.x / p.Z, z = blockIdx.x % p.Z;                    // K slices of one tile adjacent
    const int n_tile = tile_id / tok_tiles, tok_tile = tile_id % tok_tiles;        // token tiles of one n-tile adjacent
    const int n0 = n_tile * P::kRows, tok0 = tok_tile * P::kToks;
    const int toks = (p.M - tok0) < P::kToks ? (p.M - tok0) : P::kToks;
    const uint32_t n_inst = (uint32_t)((toks + 15) & ~15);
    const int ksteps_all = (p.K + kPfK - 1) / kPfK;
    const int ks0 = z * p.ksteps_z;                                                // first k-step of this slice
    const int ksteps = (ksteps_all - ks0) < p.ksteps_z ? (ksteps_all - ks0) : p.ksteps_z;
    float* const yout = p.y + (int64_t)z * p.M * p.N;

    if (tid == 0) {
        for (int s = 0; s < NA; ++s) {
            mbar_init(full_a(s), P::kDequantWarps);
            mbar_init(empty_a(s), 1);
        }
        for (int s = 0; s < NB; ++s) {
            mbar_init(full_b(s), 1);
            mbar_init(empty_b(s), 1);
        }
        mbar_init(acc_done, 1);
        mbar_init(staged, P::kDequantWarps);
        mbar_fence_init();
    }
    if (warp == 0) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_g;
    bool ok = true;

    if (warp == 0) {
        // =============================== TMA producer: x tiles ==============================================
        if (lane == 0) {
            for (int i = 0; i < ksteps && ok; ++i) {
                const int s = i % NB;
                if (i >= NB) ok = mbar_wait(empty_b(s), ((i / NB) - 1) & 1, p.status);
                if (!ok) break;
                mbar_arrive_expect_tx(full_b(s), p.x_box_bytes);
                tma_load_2d(base + s * kBStride + kBOff, &x_map, (ks0 + i) * kPfK, tok0, full_b(s));
            }
        }
    } else if (warp == 1) {
        // =============================== MMA issuer =========================================================
        // The whole warp runs the loop on warp-uniform values (so that the descriptors can live in uniform registers,
        // which is where the tensor-core instructions take them from); lane 0 issues.
        {
            const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot_g, 0);
            const uint32_t idesc = umma_idesc(n_inst);
            for (int i = 0; i < ksteps && ok; ++i) {
                const int sa = i % NA, sb = i % NB;
                const uint32_t pha = (i / NA) & 1, phb = (i / NB) & 1;
                ok = mbar_wait(full_a(sa), pha, p.status) && mbar_wait(full_b(sb), phb, p.status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_addr = base + sa * P::kStageBytes, b_addr = base + sb * kBStride + kBOff;
                if (lane != 0) continue;
                if (ATMEM) {
                    const uint64_t bdesc = umma_smem_desc(b_addr);
#pragma unroll
                    for (int k4 = 0; k4 < kPfK / 16; ++k4)  // eight TMEM columns (16 bf16) further along the weights' rows
                        umma_bf16_ta(tmem_base, tmem_base + kTmemA + (uint32_t)(sa * (kPfK / 2) + 8 * k4), bdesc + 2 * k4, idesc,
                                     (i | k4) != 0);
                } else {
#pragma unroll
                    for (int half = 0; half < ROWS / 128; ++half) {
                        const uint64_t adesc = umma_smem_desc(a_addr + half * (128 * kPfK * 2));
                        const uint64_t bdesc = umma_smem_desc(b_addr);
#pragma unroll
                        for (int k4 = 0; k4 < kPfK / 16; ++k4)  // 32 bytes (16 bf16) further along the swizzled row
                            umma_bf16(tmem_base + half * 256, adesc + 2 * k4, bdesc + 2 * k4, idesc, (i | k4) != 0);
                    }
                }
                umma_commit(empty_a(sa));  // the stages may be refilled once these MMAs have read them
                umma_commit(empty_b(sb));
            }
            if (lane == 0) {
                umma_commit(acc_done);
            }
        }
    } else {
        // =============================== dequantisation warps ================================================
        const int dw = warp - 2;
        // strip of the tile and group of the 64-k stage this warp converts (ATMEM: the strip is the warp's TMEM lane quarter)
        const int sl = ATMEM ? (warp & 3) : (dw >> 1), gl = ATMEM ? (dw >> 2) : (dw & 1);
        const int64_t strip = (int64_t)n_tile * (P::kRows / 32) + sl;
        const bool strip_ok = strip < p.N / kStripRows;
        // the loads of the next eight k-steps are in flight while this one is converted: a k-step lasts 0.6-0.7 us and a
        // load from HBM under this kernel's traffic about as long, with a long tail; three k-steps ahead left the
        // conversion waiting for its weights (measured: 5-7 % at up to 128 tokens).  Groups past K load as zeros.
        const int gbase = 2 * ks0 + gl;  // this warp's group in k-step i of the slice: gbase + 2 i
        // Eight register sets, each reloaded right after it has been converted.  (Rotating the sets with moves instead --
        // g0 = g1; g1 = g2; g2 = just-loaded -- makes the move wait for the load it follows, one trip to memory per k-step.)
        auto convert_step = [&](int i, const GroupRegs& g) -> bool {
            const int s = i % NA;
            if (i >= NA && !mbar_wait(empty_a(s), ((i / NA) - 1) & 1, p.status)) return false;
            if (ATMEM) {
                // this lane's row of the group, 16 bf16 pairs, into its TMEM lane; ordered against the MMAs that read the
                // stage before (the barrier wait above) and after (the arrive below) by the tensor-core fences
                uint32_t wreg[16];
                group_convert<FMT>(g, wreg);
                tc_fence_after();
                tmem_st_16cols(tmem_base + ((uint32_t)(sl * 32) << 16) + kTmemA + (uint32_t)(s * (kPfK / 2) + gl * 16), wreg);
                tc_fence_before();
            } else {
                group_store<FMT>(base + s * P::kStageBytes, g, sl, gl, lane);
                // make the generic-proxy stores visible to the tensor core's (async-proxy) reads, then signal
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(full_a(s));
            return true;
        };
        if (TRI) {
            GroupRegs g0 = group_load<FMT>(p.W, p.K, strip, gbase + 0, lane, strip_ok);
            GroupRegs g1 = group_load<FMT>(p.W, p.K, strip, gbase + 2, lane, strip_ok);
            GroupRegs g2 = group_load<FMT>(p.W, p.K, strip, gbase + 4, lane, strip_ok);
            GroupRegs g3 = group_load<FMT>(p.W, p.K, strip, gbase + 6, lane, strip_ok);
            for (int i = 0; i < ksteps && ok; i += 4) {
                ok = convert_step(i, g0);
                g0 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 4), lane, strip_ok);
                if (ok && i + 1 < ksteps) {
                    ok = convert_step(i + 1, g1);
                    g1 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 5), lane, strip_ok);
                }
                if (ok && i + 2 < ksteps) {
                    ok = convert_step(i + 2, g2);
                    g2 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 6), lane, strip_ok);
                }
                if (ok && i + 3 < ksteps) {
                    ok = convert_step(i + 3, g3);
                    g3 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 7), lane, strip_ok);
                }
            }
        } else {
        GroupRegs g0 = group_load<FMT>(p.W, p.K, strip, gbase + 0, lane, strip_ok);
        GroupRegs g1 = group_load<FMT>(p.W, p.K, strip, gbase + 2, lane, strip_ok);
        GroupRegs g2 = group_load<FMT>(p.W, p.K, strip, gbase + 4, lane, strip_ok);
        GroupRegs g3 = group_load<FMT>(p.W, p.K, strip, gbase + 6, lane, strip_ok);
        GroupRegs g4 = group_load<FMT>(p.W, p.K, strip, gbase + 8, lane, strip_ok);
        GroupRegs g5 = group_load<FMT>(p.W, p.K, strip, gbase + 10, lane, strip_ok);
        GroupRegs g6 = group_load<FMT>(p.W, p.K, strip, gbase + 12, lane, strip_ok);
        GroupRegs g7 = group_load<FMT>(p.W, p.K, strip, gbase + 14, lane, strip_ok);
        for (int i = 0; i < ksteps && ok; i += 8) {
            ok = convert_step(i, g0);
            g0 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 8), lane, strip_ok);
            if (ok && i + 1 < ksteps) {
                ok = convert_step(i + 1, g1);
                g1 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 9), lane, strip_ok);
            }
            if (ok && i + 2 < ksteps) {
                ok = convert_step(i + 2, g2);
                g2 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 10), lane, strip_ok);
            }
            if (ok && i + 3 < ksteps) {
                ok = convert_step(i + 3, g3);
                g3 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 11), lane, strip_ok);
            }
            if (ok && i + 4 < ksteps) {
                ok = convert_step(i + 4, g4);
                g4 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 12), lane, strip_ok);
            }
            if (ok && i + 5 < ksteps) {
                ok = convert_step(i + 5, g5);
                g5 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 13), lane, strip_ok);
            }
            if (ok && i + 6 < ksteps) {
                ok = convert_step(i + 6, g6);
                g6 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 14), lane, strip_ok);
            }
            if (ok && i + 7 < ksteps) {
                ok = convert_step(i + 7, g7);
                g7 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 15), lane, strip_ok);
            }
        }
        }
        // =============================== epilogue: TMEM -> y =================================================
        if (ok) ok = mbar_wait(acc_done, 0, p.status);
        ok = __all_sync(0xffffffffu, ok);
        const bool via_smem = p.epi != kEpiNone && p.Z == 1;  // bf16 epilogues (a K-split call leaves them to the sum)
        const bool geglu = p.epi == kEpiGegluBf16;
        const int cols = geglu ? P::kRows / 2 : P::kRows;       // bf16 values per token row of the staged tile
        if (ok) {
            tc_fence_after();
            const int quarter = warp & 3;        // TMEM lanes this warp may read
            // the four warps of a quarter (dw = quarter', quarter' + 4, + 8, + 12) take (accumulator, column half)
            const int half = ROWS == 256 ? (dw >> 2) & 1 : 0, chalf = ROWS == 256 ? dw >> 3 : dw >> 2;
            const int n_local = half * 128 + quarter * 32 + lane;
            const int n = n0 + n_local;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(half * 256 + chalf * CH);
            const int c_end = ((int)n_inst < chalf * CH + CH ? (int)n_inst : chalf * CH + CH) - chalf * CH;
            const int64_t ldy = p.N;
            float* yrow = yout + (int64_t)(tok0 + chalf * CH) * ldy + n;  // token row of this warp's column 0
            const int toks_h = toks - chalf * CH;                          // tokens of this column half that exist
            // staged tile: this lane's column, and the first token row of this warp
            const uint32_t scol = base + (uint32_t)((chalf * CH) * cols + (geglu ? (n_local >> 5) * 16 + (lane & 15) : n_local)) * 2u;
            for (int c = 0; c < c_end; c += 32) {
                uint32_t v[32];
                tmem_ld_32cols(taddr + c, v);
                if (!via_smem) {
                    if (n < p.N) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (c + j < toks_h) yrow[j * ldy] = __uint_as_float(v[j]);
                    }
                    yrow += 32 * ldy;
                } else {
                    if (!geglu) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            asm volatile("st.shared.u16 [%0], %1;" ::"r"(scol + (uint32_t)((c + j) * cols) * 2u),
                                         "h"(f32_to_bf16_rne(__uint_as_float(v[j])))
                                         : "memory");
                    } else {
                        // lanes 0..15 hold gate rows, lanes 16..31 the up rows of the same outputs: the low half finishes
                        // the even tokens, the high half the odd ones -- one exchange per token pair, every lane busy
                        const bool low = lane < 16;
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) {
                            const float a = __uint_as_float(v[2 * jj]), b = __uint_as_float(v[2 * jj + 1]);
                            const float got = __shfl_xor_sync(0xffffffffu, low ? b : a, 16);
                            const float gate = low ? a : got, up = low ? got : b;
                            asm volatile("st.shared.u16 [%0], %1;" ::"r"(scol + (uint32_t)((c + 2 * jj + (low ? 0 : 1)) * cols) * 2u),
                                         "h"(f32_to_bf16_rne(gelu_tanh(gate) * up))
                                         : "memory");
                        }
                    }
                }
            }
        }
        if (via_smem) {
            // every warp arrives (also one that gave up), then the tile leaves shared memory in whole lines
            __syncwarp();
            if (lane == 0) mbar_arrive(staged);
            if (ok && mbar_wait(staged, 0, p.status)) {
                const int64_t ld16 = geglu ? p.N / 2 : p.N;
                const int col0 = geglu ? n0 / 2 : n0;
                const int valid = (int)((ld16 - col0) < cols ? (ld16 - col0) : cols);
                stage_copy_out(base, p.y16 + (int64_t)tok0 * ld16 + col0, ld16, toks, cols, valid, dw, P::kDequantWarps, lane);
            }
        }
    }
    // =============================== teardown: every path releases TMEM =====================================
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---- the two-SM kernel (M > 256) ----------------------------------------------------------------------------------
//
// A cluster of two CTAs computes a 256 (output features) x 512 (tokens) tile with tcgen05.mma.cta_group::2: each CTA
// dequantises ITS 128 rows (16 KB per 64-k stage) and loads ITS half of the tokens of each MMA (2 x 128 tokens, 32 KB
// per stage); the tensor cores of the pair read both CTAs' shared memory, so every converted weight serves 512 tokens
// and every loaded activation serves 256 rows.  Accumulators: 128 lanes x 512 columns of each CTA's TMEM (rows of that
// CTA, all 512 tokens).  CTA 0 of the pair issues the MMAs; stage barriers it waits on live in CTA 0 and are signalled
// by both CTAs; tcgen05.commit releases the stage in both CTAs at once.

constexpr int kP2Rows = 128;      // output features per CTA (256 per pair)
constexpr int kP2Toks = 512;      // tokens per pair tile
constexpr int kP2TokBox = 128;    // tokens per CTA per MMA
constexpr int kP2Stages = 4;
constexpr uint32_t kP2ABytes = kP2Rows * kPfK * 2;        // 16 KB
constexpr uint32_t kP2BBoxBytes = kP2TokBox * kPfK * 2;   // 16 KB
constexpr uint32_t kP2StageBytes = kP2ABytes + 2 * kP2BBoxBytes;  // 48 KB
constexpr uint32_t kP2SmemBytes = kP2Stages * kP2StageBytes + 1024 + 256;

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory offset in CTA `rank` of the cluster (shared::cluster window).
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on a barrier of another CTA of the cluster.  The data this signals was written to the issuing CTA's own shared
// memory and already made visible to the async proxy (the tensor cores) by fence.proxy.async; a cluster-scope release
// here would add a full memory barrier per warp per stage (measured: the dominant stall).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Bounded wait whose success also orders the other CTA's writes before this thread's later operations.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, int* status) {
    const unsigned long long t0 = globaltimer_ns();
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
        if ((it & 63u) == 63u && globaltimer_ns() - t0 > kWaitLimitNs) {
            atomicExch(status, kStatusTimeout);
            __threadfence_system();
            return false;
        }
    }
}
__device__ __forceinline__ void tmem_alloc2(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma2_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on the barrier at this offset in BOTH CTAs once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
    asm volatile(
        "{\n\t.reg .b16 m;\n\tmov.b16 m, 3;\n\t"
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n\t}"
        ::"r"(bar)
        : "memory");
}
// This CTA's box of x into its own shared memory; the bytes are counted on CTA 0's barrier.
__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar_cta0) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cta0), "r"(c0), "r"(c1)
        : "memory");
}

template <int FMT>
__global__ void __launch_bounds__(kPfThreads, 1)
    fdqp_prefill_pair_kernel(const __grid_constant__ CUtensorMap x_map, const PrefillParams p) {
    extern __shared__ uint8_t smem_raw[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // same offset in both CTAs (same kernel, same dynamic size)
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t bars = base + kP2Stages * kP2StageBytes;
    auto full_a = [&](int s) { return bars + 8u * s; };                      // used in CTA 0: 16 warp arrivals
    auto full_b = [&](int s) { return bars + 8u * (kP2Stages + s); };        // used in CTA 0: 1 arrival + 64 KB
    auto empty = [&](int s) { return bars + 8u * (2 * kP2Stages + s); };     // each CTA its own, signalled by commit
    const uint32_t acc_done = bars + 8u * (3 * kP2Stages);
    const uint32_t tmem_slot = acc_done + 8u;
    const uint32_t staged = tmem_slot + 8u;  // bf16 epilogues: every epilogue warp has written its part of the tile
    volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(smem + kP2Stages * kP2StageBytes + 8 * (3 * kP2Stages + 1));

    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1;
    const int tok_tiles = (p.M + kP2Toks - 1) / kP2Toks;
    const int tile_id = pair / p.Z, z = pair % p.Z;
    const int n_tile = tile_id / tok_tiles, tok_tile = tile_id % tok_tiles;
    const int n0 = n_tile * (2 * kP2Rows) + (int)rank * kP2Rows, tok0 = tok_tile * kP2Toks;
    const int ksteps_all = (p.K + kPfK - 1) / kPfK;
    const int ks0 = z * p.ksteps_z;
    const int ksteps = (ksteps_all - ks0) < p.ksteps_z ? (ksteps_all - ks0) : p.ksteps_z;
    float* const yout = p.y + (int64_t)z * p.M * p.N;
    // tokens of the two MMAs of a k-step, rounded up to the instruction's granularity (16); the second MMA is dropped
    // when the tile has no more than 256 tokens.  Each CTA supplies half of an MMA's tokens.
    const int rem = p.M - tok0;
    const int n_mma0 = rem >= 256 ? 256 : ((rem + 15) & ~15);
    const int n_mma1 = rem <= 256 ? 0 : (rem - 256 >= 256 ? 256 : ((rem - 256 + 15) & ~15));
    const int n_mmas = n_mma1 > 0 ? 2 : 1;

    if (tid == 0) {
        for (int s = 0; s < kP2Stages; ++s) {
            mbar_init(full_a(s), 2 * kPfDequantWarps);
            mbar_init(full_b(s), 1);
            mbar_init(empty(s), 1);
        }
        mbar_init(acc_done, 1);
        mbar_init(staged, kPfDequantWarps);
        mbar_fence_init();
    }
    if (warp == 0) {
        tmem_alloc2(tmem_slot, kPfTmemCols);
        tmem_relinquish2();
    }
    tc_fence_before();
    cluster_sync_all();  // barriers of both CTAs initialised, TMEM allocated in both
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_g;
    bool ok = true;

    if (warp == 0) {
        // =============================== TMA producer: this CTA's token boxes ================================
        if (lane == 0) {
            for (int i = 0; i < ksteps && ok; ++i) {
                const int s = i % kP2Stages;
                if (i >= kP2Stages) ok = mbar_wait(empty(s), ((i / kP2Stages) - 1) & 1, p.status);
                if (!ok) break;
                if (rank == 0) mbar_arrive_expect_tx(full_b(s), 2 * n_mmas * kP2BBoxBytes);  // both CTAs' boxes
                const uint32_t bar0 = mapa_shared(full_b(s), 0);
                const uint32_t b_addr = base + s * kP2StageBytes + kP2ABytes;
                // MMA j covers tokens [256 j, 256 j + n_j): this CTA supplies n_j / 2 of them (a full 128-token box is
                // copied; what the MMA does not read is ignored, what lies beyond M arrives as zeros)
                tma2_load_2d(b_addr, &x_map, (ks0 + i) * kPfK, tok0 + (int)rank * (n_mma0 / 2), bar0);
                if (n_mmas == 2)
                    tma2_load_2d(b_addr + kP2BBoxBytes, &x_map, (ks0 + i) * kPfK, tok0 + 256 + (int)rank * (n_mma1 / 2), bar0);
            }
        }
    } else if (warp == 1) {
        // =============================== MMA issuer (CTA 0 only) ============================================
        if (lane == 0 && rank == 0) {
            // kind::f16: D fp32, A and B bf16, both K-major, M = 256 over the pair, N = tokens of the MMA
            const uint32_t idesc_mn = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 4) << 24);
            const uint32_t idesc[2] = {idesc_mn | ((uint32_t)(n_mma0 >> 3) << 17), idesc_mn | ((uint32_t)(n_mma1 >> 3) << 17)};
            for (int i = 0; i < ksteps && ok; ++i) {
                const int s = i % kP2Stages;
                const uint32_t ph = (i / kP2Stages) & 1;
                ok = mbar_wait_cluster(full_a(s), ph, p.status) && mbar_wait_cluster(full_b(s), ph, p.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_addr = base + s * kP2StageBytes, b_addr = a_addr + kP2ABytes;
                const uint64_t adesc = umma_smem_desc(a_addr);
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    if (j < n_mmas) {
                        const uint64_t bdesc = umma_smem_desc(b_addr + j * kP2BBoxBytes);
#pragma unroll
                        for (int k4 = 0; k4 < kPfK / 16; ++k4)
                            umma2_bf16(tmem_base + j * 256, adesc + 2 * k4, bdesc + 2 * k4, idesc[j], (i | k4) != 0);
                    }
                }
                umma2_commit_both(empty(s));
            }
            umma2_commit_both(acc_done);
        }
    } else {
        // =============================== dequantisation warps ================================================
        const int dw = warp - 2;
        const int sl = dw >> 1, gl = dw & 1;  // strip of this CTA's 128 rows, group of the 64-k stage
        const int64_t strip = (int64_t)(n0 / kStripRows) + sl;
        const bool strip_ok = strip < p.N / kStripRows;
        // software pipeline: the loads of the next three k-steps are in flight while this one is converted (eight, as in
        // the one-SM kernel, measured no faster here); groups past K load as zeros
        const int gbase = 2 * ks0 + gl;  // this warp's group in k-step i of the slice: gbase + 2 i
        // three register sets, each reloaded right after it has been converted (no rotation by moves: see the one-SM kernel)
        const uint32_t full_a0 = mapa_shared(full_a(0), 0);
        auto convert_step = [&](int i, const GroupRegs& g) -> bool {
            const int s = i % kP2Stages;
            if (i >= kP2Stages && !mbar_wait(empty(s), ((i / kP2Stages) - 1) & 1, p.status)) return false;
            group_store<FMT>(base + s * kP2StageBytes, g, sl, gl, lane);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(full_a0 + 8u * s);
            return true;
        };
        GroupRegs g0 = group_load<FMT>(p.W, p.K, strip, gbase + 0, lane, strip_ok);
        GroupRegs g1 = group_load<FMT>(p.W, p.K, strip, gbase + 2, lane, strip_ok);
        GroupRegs g2 = group_load<FMT>(p.W, p.K, strip, gbase + 4, lane, strip_ok);
        for (int i = 0; i < ksteps && ok; i += 3) {
            ok = convert_step(i, g0);
            g0 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 3), lane, strip_ok);
            if (ok && i + 1 < ksteps) {
                ok = convert_step(i + 1, g1);
                g1 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 4), lane, strip_ok);
            }
            if (ok && i + 2 < ksteps) {
                ok = convert_step(i + 2, g2);
                g2 = group_load<FMT>(p.W, p.K, strip, gbase + 2 * (i + 5), lane, strip_ok);
            }
        }
        // =============================== epilogue: this CTA's TMEM -> y ======================================
        if (ok) ok = mbar_wait(acc_done, 0, p.status);
        ok = __all_sync(0xffffffffu, ok);
        const bool via_smem = p.epi != kEpiNone && p.Z == 1;  // bf16 epilogues (a K-split call leaves them to the sum)
        const bool geglu = p.epi == kEpiGegluBf16;
        const int cols = geglu ? kP2Rows / 2 : kP2Rows;       // bf16 values per token row of the staged tile
        const int toks_all = (p.M - tok0) < kP2Toks ? (p.M - tok0) : kP2Toks;
        if (ok) {
            tc_fence_after();
            const int quarter = warp & 3;   // TMEM lanes this warp may read
            const int chalf = dw >> 2;      // columns [256 chalf, 256 chalf + 256): every (quarter, half) once
            const int n_local = quarter * 32 + lane;
            const int n = n0 + n_local;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(chalf * 256);
            const int toks = p.M - tok0 - chalf * 256;  // tokens of this column half that exist
            const int64_t ldy = p.N;
            float* yrow = yout + (int64_t)(tok0 + chalf * 256) * ldy + n;  // token row of column 0 of this half
            const uint32_t scol = base + (uint32_t)((chalf * 256) * cols + (geglu ? (n_local >> 5) * 16 + (lane & 15) : n_local)) * 2u;
            for (int c = 0; c < 256 && c < toks; c += 32) {
                uint32_t v[32];
                tmem_ld_32cols(taddr + c, v);
                if (!via_smem) {
                    if (n < p.N) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (c + j < toks) yrow[j * ldy] = __uint_as_float(v[j]);
                    }
                    yrow += 32 * ldy;
                } else {
                    if (!geglu) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            asm volatile("st.shared.u16 [%0], %1;" ::"r"(scol + (uint32_t)((c + j) * cols) * 2u),
                                         "h"(f32_to_bf16_rne(__uint_as_float(v[j])))
                                         : "memory");
                    } else {
                        // lanes 0..15 hold gate rows, lanes 16..31 the up rows of the same outputs: the low half finishes
                        // the even tokens, the high half the odd ones -- one exchange per token pair, every lane busy
                        const bool low = lane < 16;
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) {
                            const float a = __uint_as_float(v[2 * jj]), b = __uint_as_float(v[2 * jj + 1]);
                            const float got = __shfl_xor_sync(0xffffffffu, low ? b : a, 16);
                            const float gate = low ? a : got, up = low ? got : b;
                            asm volatile("st.shared.u16 [%0], %1;" ::"r"(scol + (uint32_t)((c + 2 * jj + (low ? 0 : 1)) * cols) * 2u),
                                         "h"(f32_to_bf16_rne(gelu_tanh(gate) * up))
                                         : "memory");
                        }
                    }
                }
            }
        }
        if (via_smem) {
            __syncwarp();
            if (lane == 0) mbar_arrive(staged);
            if (ok && mbar_wait(staged, 0, p.status)) {
                const int64_t ld16 = geglu ? p.N / 2 : p.N;
                const int col0 = geglu ? n0 / 2 : n0;
                const int valid = (int)((ld16 - col0) < cols ? (ld16 - col0) : cols);
                stage_copy_out(base, p.y16 + (int64_t)tok0 * ld16 + col0, ld16, toks_all, cols, valid, dw, kPfDequantWarps, lane);
            }
        }
    }
    // =============================== teardown: every path of both CTAs releases TMEM =========================
    tc_fence_before();
    cluster_sync_all();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc2(tmem_base, kPfTmemCols);
    }
}

// Second phase of a K-split call: y = sum over slices z (ascending) of the partial results; four outputs per thread.
__global__ void __launch_bounds__(256) fdqp_prefill_sum_kernel(const float4* __restrict__ ws, float4* __restrict__ y, int Z,
                                                                int64_t quads) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= quads) return;
    float4 acc = ws[i];
    for (int z = 1; z < Z; ++z) {
        const float4 v = ws[(int64_t)z * quads + i];
        acc.x += v.x;
        acc.y += v.y;
        acc.z += v.z;
        acc.w += v.w;
    }
    y[i] = acc;
}

// The same for the bf16 / gated-GELU epilogues: one output value per thread, whole warps on one (token, strip).
__global__ void __launch_bounds__(256) fdqp_prefill_sum_epi_kernel(const float* __restrict__ ws, uint16_t* __restrict__ y16,
                                                                    int epi, int Z, int M, int N) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t total = (int64_t)M * N;  // a multiple of 32
    if (idx >= total) return;
    float acc = ws[idx];
    for (int z = 1; z < Z; ++z) acc += ws[(int64_t)z * total + idx];
    const int tok = (int)(idx / N), n = (int)(idx - (int64_t)tok * N);
    store_output(nullptr, y16, epi, N, n >> 5, n & 31, tok, acc);
}

// ---- host side ----------------------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

template <int FMT>
static cudaError_t prefill_set_smem_limit_fmt() {
    cudaError_t e = cudaFuncSetAttribute(fdqp_prefill_kernel<FMT, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Pf1<256>::kSmemBytes);
    if (e) return e;
    if ((e = cudaFuncSetAttribute(fdqp_prefill_kernel<FMT, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Pf1<128>::kSmemBytes))) return e;
    if ((e = cudaFuncSetAttribute(fdqp_prefill_kernel<FMT, 128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Pf1<128>::kSmemBytesTmemA))) return e;
    if ((e = cudaFuncSetAttribute(fdqp_prefill_kernel<FMT, 128, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Pf1<128>::kSmemBytesTri))) return e;
    return cudaFuncSetAttribute(fdqp_prefill_pair_kernel<FMT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kP2SmemBytes);
}

cudaError_t prefill_set_smem_limit() {
    cudaError_t e;
    if ((e = prefill_set_smem_limit_fmt<kFmtQ4nx>())) return e;
    if ((e = prefill_set_smem_limit_fmt<kFmtG64>())) return e;
    if ((e = prefill_set_smem_limit_fmt<kFmtG128>())) return e;
    return prefill_set_smem_limit_fmt<kFmtMxfp4>();
}

template <int FMT>
static cudaError_t prefill_launch_kernels(const CUtensorMap& map, const PrefillParams& p, int pair, int a_tmem, int M, int N,
                                          int Z, cudaStream_t stream) {
    if (pair) {
        const int n_tiles = (N + 2 * kP2Rows - 1) / (2 * kP2Rows), tok_tiles = (M + kP2Toks - 1) / kP2Toks;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(2 * n_tiles * tok_tiles * Z));
        cfg.blockDim = dim3((unsigned)kPfThreads);
        cfg.dynamicSmemBytes = kP2SmemBytes;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, fdqp_prefill_pair_kernel<FMT>, map, p);
    }
    if (pair == 0 && M <= Pf1<128>::kToks) {  // small tiles, two CTAs per SM
        const int n_tiles = (N + 127) / 128;
        if (a_tmem == 2 && M <= 64)
            fdqp_prefill_kernel<FMT, 128, true, true><<<n_tiles * Z, Pf1<128>::kThreads, Pf1<128>::kSmemBytesTri, stream>>>(map, p);
        else if (a_tmem)
            fdqp_prefill_kernel<FMT, 128, true><<<n_tiles * Z, Pf1<128>::kThreads, Pf1<128>::kSmemBytesTmemA, stream>>>(map, p);
        else
            fdqp_prefill_kernel<FMT, 128><<<n_tiles * Z, Pf1<128>::kThreads, Pf1<128>::kSmemBytes, stream>>>(map, p);
        return cudaGetLastError();
    }
    const int n_tiles = (N + kPfRows - 1) / kPfRows, tok_tiles = (M + kPfToks - 1) / kPfToks;
    fdqp_prefill_kernel<FMT, 256><<<n_tiles * tok_tiles * Z, Pf1<256>::kThreads, Pf1<256>::kSmemBytes, stream>>>(map, p);
    return cudaGetLastError();
}

// x: [M][K] bf16 row-major (device).  Returns cudaErrorNotSupported if the tensor map cannot be built.
// pair != 0: the two-SM kernel (256 x 512 tiles per CTA pair), meant for M > 256.
// Z > 1: K is cut into Z slices (tiles x Z CTAs or CTA pairs), their partial results go to `ws` ([Z][M][N] floats) and a
// second kernel adds them in slice order into y.  For shapes with too few tiles to fill the GPU.
// x_row_bytes: distance between token rows of x (K * 2 for a dense [M][K] array; a multiple of 16).
// epi: kEpiNone writes fp32 y; the other epilogues write bf16 to y16 (see fdqp_plan.h).
// fmt: the container's format (fdqp_format.h).
// kernels_launched (may be null): receives 1, or 2 when the K slices needed the second kernel.
cudaError_t prefill_launch(const uint8_t* W, const uint16_t* x, int64_t x_row_bytes, float* y, uint16_t* y16, int epi, float* ws,
                           int* status, int M, int K, int N, int pair, int Z, int fmt, int a_tmem, cudaStream_t stream,
                           int* kernels_launched) {
    if (kernels_launched) *kernels_launched = 0;
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return cudaErrorNotSupported;
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};      // innermost first
    const cuuint64_t strides[1] = {(cuuint64_t)x_row_bytes};        // bytes between token rows
    // one-SM kernel: the box holds only the token rows the MMAs read (M rounded up to 16), not the whole tile's
    const int tile_toks = M <= Pf1<128>::kToks ? Pf1<128>::kToks : kPfToks;
    const int box_rows = pair ? kP2TokBox : (M < tile_toks ? (M + 15) / 16 * 16 : tile_toks);
    const cuuint32_t box[2] = {(cuuint32_t)kPfK, (cuuint32_t)box_rows};
    const cuuint32_t elem[2] = {1, 1};
    if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<uint16_t*>(x), dims, strides, box, elem,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    PrefillParams p;
    const int ksteps_all = (K + kPfK - 1) / kPfK;
    if (Z < 1 || Z > ksteps_all || !ws) Z = 1;
    p.W = W;
    p.y = Z > 1 ? ws : y;
    p.y16 = y16;
    p.epi = epi;
    p.status = status;
    p.M = M;
    p.K = K;
    p.N = N;
    p.ksteps_z = (ksteps_all + Z - 1) / Z;
    p.x_box_bytes = (uint32_t)box_rows * kPfK * 2;
    p.Z = (ksteps_all + p.ksteps_z - 1) / p.ksteps_z;  // no empty slice
    Z = p.Z;
    cudaError_t err;
    switch (fmt) {
        case kFmtQ4nx: err = prefill_launch_kernels<kFmtQ4nx>(map, p, pair, a_tmem, M, N, Z, stream); break;
        case kFmtG64: err = prefill_launch_kernels<kFmtG64>(map, p, pair, a_tmem, M, N, Z, stream); break;
        case kFmtG128: err = prefill_launch_kernels<kFmtG128>(map, p, pair, a_tmem, M, N, Z, stream); break;
        case kFmtMxfp4: err = prefill_launch_kernels<kFmtMxfp4>(map, p, pair, a_tmem, M, N, Z, stream); break;
        default: return cudaErrorInvalidValue;
    }
    if (err != cudaSuccess) return err;
    if (kernels_launched) *kernels_launched = Z > 1 ? 2 : 1;
    if (Z == 1) return err;
    if (epi != kEpiNone) {
        const int64_t total = (int64_t)M * N;
        fdqp_prefill_sum_epi_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(ws, y16, epi, Z, M, N);
        return cudaGetLastError();
    }
    const int64_t quads = (int64_t)M * N / 4;  // N is a multiple of 32
    fdqp_prefill_sum_kernel<<<(unsigned)((quads + 255) / 256), 256, 0, stream>>>(reinterpret_cast<const float4*>(ws),
                                                                                reinterpret_cast<float4*>(y), Z, quads);
    return cudaGetLastError();
}

}  // namespace fdqp
