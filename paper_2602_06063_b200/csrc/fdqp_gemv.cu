// Streaming GEMV kernels for FusedDQP at M = 1..8 tokens (Sec. "FusedDQP", Eq. 14 / 15, with the
// block-wise dequantisation of Eq. 3 fused in).
//
// Shape of the computation.  For every quantisation group (32 consecutive k of one output row n)
//     sum_k x_k * (d * q_k + m)  =  d * (sum_k q_k x_k)  +  m * (sum_k x_k)
// so the per-weight work is only "unpack a nibble and multiply-accumulate it with x"; scale d and
// offset m are applied once per group in fp32.  The inner sums run on the warp-level bf16 tensor-core
// instruction (mma.sync m16n8k16): A = 16 output rows x 16 k of codes, B = 16 k x 8 token columns of
// x, fp32 accumulate.  Codes are turned into bf16 with one logic op per pair
//     ((word >> 4i) & 0x000F000F) | 0x43004300  ->  bf16x2 (128 + q_i, 128 + q_{i+4})
// (exact); the +128 is cancelled by starting the accumulator at -128 * sum_k x_k, and the order of k
// inside a group is a free permutation as long as x is staged with the same one.
//
// Data movement.  The packed matrix is strip-major (32 output rows x all of K contiguous), so every
// CTA streams one contiguous byte range of HBM exactly once.  The producer warp issues one 1-D bulk
// async copy per Q4NX block (<= 5120 bytes), several lanes at a time, into a shared-memory ring of
// multi-block stages guarded by mbarriers; every consumer warp owns the same 32 x 32 group-tile of
// two blocks of a stage.  x (the CTA's K slice, all tokens) is staged once per CTA in the fragment
// order the MMA wants, together with the per-group sums of x.
//
// Work split.  The (K-slice, strip, block) space is cut into equal contiguous ranges, one per
// persistent CTA, so all SMs stream the same number of bytes whatever N and K are.  A strip whose
// blocks end up in several CTAs (or several K slices) is completed by whichever CTA arrives last at
// the strip's ticket: it sums the partial rows in a fixed order, so results are reproducible run to run.
// No CTA ever waits for another CTA.
#include "fdqp_device.cuh"
#include "fdqp_plan.h"

namespace fdqp {

__device__ __forceinline__ int64_t range_begin(int64_t ci, int64_t G, int64_t T) { return (ci * T) / G; }
// index of the CTA whose range [range_begin(ci), range_begin(ci+1)) contains L
__device__ __forceinline__ int64_t cta_of(int64_t L, int64_t G, int64_t T) { return ((L + 1) * G - 1) / T; }

__device__ __forceinline__ int slice_len(const GemvPlan& p, int z) {
    const int rest = p.nb - z * p.nbz;
    return rest < p.nbz ? rest : p.nbz;
}

// Partial-sum slot a CTA uses for its piece of strip s in slice z (the reader uses the same rule).
__device__ __forceinline__ float* piece_slot(const GemvPlan& p, int z, int64_t ci, int64_t s, int64_t unit_begin,
                                             bool whole_unit, int64_t cta_begin) {
    if (whole_unit) return p.ws_full + ((int64_t)z * p.S + s) * (kStripRows * kMaxTokens);
    const int which = (cta_begin >= unit_begin) ? 0 : 1;  // piece holds the CTA's first block, or its last
    return p.ws_edge + (((int64_t)z * p.Gz + ci) * 2 + which) * (kStripRows * kMaxTokens);
}

// Registers of one 32 x 32 group-tile in flight.
struct TileRegs {
    uint32_t c[4];   // code words: word q of rows g, g+8, g+16, g+24
    uint32_t so[4];  // (d[g], d[g+8]), (d[g+16], d[g+24]), (m[g], m[g+8]), (m[g+16], m[g+24]) as bf16 pairs
    uint4 xb;        // B fragments of the two k16 steps
    float xs[4];     // sum of x over the group for tokens 2q, 2q+1, and -128 times it
    float d0[4], d1[4];
};

#define FDQP_UNPACK(w, sh) ((((w) >> (sh)) & 0x000F000Fu) | 0x43004300u)

template <int NT>
__device__ __forceinline__ void tile_load(TileRegs& t, uint32_t code_addr, uint32_t so_addr, uint32_t x_addr,
                                          uint32_t xsum_addr) {
    ldmatrix_x4(t.c, code_addr);
    ldmatrix_x4_trans(t.so, so_addr);
    t.xb = lds128(x_addr);
    if (NT == 1) {
        const float2 v = lds64f(xsum_addr);  // {X, -128 X} of token 2q
        t.xs[0] = v.x;
        t.xs[1] = 0.f;
        t.xs[2] = v.y;
        t.xs[3] = 0.f;
    } else {
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                     : "=f"(t.xs[0]), "=f"(t.xs[1]), "=f"(t.xs[2]), "=f"(t.xs[3])
                     : "r"(xsum_addr));  // {X0, X1, -128 X0, -128 X1}
    }
}

__device__ __forceinline__ void tile_mma(TileRegs& t) {
    const float cinit[4] = {t.xs[2], t.xs[3], t.xs[2], t.xs[3]};  // -128 * sum x cancels the code bias
    {
        const uint32_t lo = t.c[0], hi = t.c[1];
        mma_bf16_16816(t.d0, FDQP_UNPACK(lo, 0), FDQP_UNPACK(hi, 0), FDQP_UNPACK(lo, 4), FDQP_UNPACK(hi, 4), t.xb.x,
                       t.xb.y, cinit);
        mma_bf16_16816(t.d0, FDQP_UNPACK(lo, 8), FDQP_UNPACK(hi, 8), FDQP_UNPACK(lo, 12), FDQP_UNPACK(hi, 12), t.xb.z,
                       t.xb.w, t.d0);
    }
    {
        const uint32_t lo = t.c[2], hi = t.c[3];
        mma_bf16_16816(t.d1, FDQP_UNPACK(lo, 0), FDQP_UNPACK(hi, 0), FDQP_UNPACK(lo, 4), FDQP_UNPACK(hi, 4), t.xb.x,
                       t.xb.y, cinit);
        mma_bf16_16816(t.d1, FDQP_UNPACK(lo, 8), FDQP_UNPACK(hi, 8), FDQP_UNPACK(lo, 12), FDQP_UNPACK(hi, 12), t.xb.z,
                       t.xb.w, t.d1);
    }
}

// acc[row][tok] += d * (sum_k q_k x_k) + m * (sum_k x_k), in fp32 (Eq. 3 applied per group)
template <int NT>
__device__ __forceinline__ void tile_scale(const TileRegs& t, float (&acc)[4][NT]) {
    const float dsc[4] = {bf16_lo_to_f32(t.so[0]), bf16_hi_to_f32(t.so[0]), bf16_lo_to_f32(t.so[1]),
                          bf16_hi_to_f32(t.so[1])};
    const float mof[4] = {bf16_lo_to_f32(t.so[2]), bf16_hi_to_f32(t.so[2]), bf16_lo_to_f32(t.so[3]),
                          bf16_hi_to_f32(t.so[3])};
    const float dd[4][2] = {{t.d0[0], t.d0[1]}, {t.d0[2], t.d0[3]}, {t.d1[0], t.d1[1]}, {t.d1[2], t.d1[3]}};
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            acc[i][j] = fmaf(dsc[i], dd[i][j], acc[i][j]);
            acc[i][j] = fmaf(mof[i], t.xs[j], acc[i][j]);
        }
}

// CW consumer warps (8 or 16); NT token columns kept per lane (1 when M == 1, else 2).
// A ring stage holds CB = CW / 4 blocks; warp w owns group-tile (w & 7) of blocks 2*(w >> 3) and
// 2*(w >> 3) + 1 of every stage.
template <int CW, int NT>
__global__ void __launch_bounds__((CW + 2) * 32, 1) fdqp_gemv_kernel(const __grid_constant__ GemvPlan p) {
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int CB = CW / 4;
    constexpr uint32_t kStageBytes = CB * kBlockBytes;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int M = p.M, K = p.K;

    const int z = blockIdx.x / p.Gz;
    const int64_t ci = blockIdx.x % p.Gz;
    const int b_first = z * p.nbz;
    const int len = slice_len(p, z);
    const int64_t T = (int64_t)p.S * len;
    const int64_t a = range_begin(ci, p.Gz, T), e = range_begin(ci + 1, p.Gz, T);
    const int nblk = (int)(e - a);
    if (nblk <= 0) return;
    const int64_t s_first = a / len;
    const int bl_first = (int)(a - s_first * len);           // block index inside the slice of the CTA's first block
    const int npieces = (int)((e - 1) / len - s_first) + 1;  // strips this CTA touches
    const int nchunk = (nblk + CB - 1) / CB;

    const uint32_t ring = smem_u32(smem);
    const uint32_t xs = ring + p.off_xs, zero_slot = ring + p.off_zero, xsum = ring + p.off_xsum;
    const uint32_t part = ring + p.off_part, bars = ring + p.off_bar;
    const int nstage = p.nstage;
    const uint32_t full0 = bars, empty0 = bars + 8u * nstage;
    const uint32_t red_full0 = bars + 16u * nstage, red_empty0 = red_full0 + 16u;

    for (int s = tid; s < nstage; s += blockDim.x) {
        mbar_init(full0 + 8u * s, 1);
        mbar_init(empty0 + 8u * s, CW);
    }
    if (tid < 2) {
        mbar_init(red_full0 + 8u * tid, CW);
        mbar_init(red_empty0 + 8u * tid, 1);
    }
    mbar_fence_init();
    __syncthreads();

    const int groups_total = K / kGroup;
    const int64_t strip_bytes = (int64_t)kGroupBytes * groups_total;

    if (warp == CW) {
        // =============================== producer ================================================
        // Lane j < CB copies block j of every stage; lane 0 owns the barrier traffic.
        uint64_t policy = 0;
        if (p.evict_first) policy = l2_policy_evict_first();
        int64_t ps = s_first;
        int pbl = bl_first + lane;  // only meaningful for lane < CB
        while (pbl >= len) { pbl -= len; ++ps; }
        int stage = 0;
        uint32_t phase = 0;  // parity of the stage's previous use
        bool alive = true;
        int c = 0;
        for (; c < nchunk && alive; ++c) {
            if (c >= nstage) {
                int ok = 1;
                if (lane == 0) ok = mbar_wait(empty0 + 8u * stage, phase ^ 1u, p.status) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { alive = false; break; }
            }
            const int i = c * CB + lane;
            uint32_t bytes = 0;
            if (lane < CB && i < nblk) {
                const int rest = groups_total - 8 * (b_first + pbl);
                bytes = (uint32_t)kGroupBytes * (uint32_t)(rest < 8 ? rest : 8);
            }
            const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
            if (lane == 0) mbar_arrive_expect_tx(full0 + 8u * stage, total);
            __syncwarp();
            if (bytes) {
                const uint8_t* src = p.W + ps * strip_bytes + (int64_t)(b_first + pbl) * kBlockBytes;
                const uint32_t dst = ring + stage * kStageBytes + lane * kBlockBytes;
                if (p.evict_first)
                    bulk_g2s_hint(dst, src, bytes, full0 + 8u * stage, policy);
                else
                    bulk_g2s(dst, src, bytes, full0 + 8u * stage);
            }
            pbl += CB;
            while (pbl >= len) { pbl -= len; ++ps; }
            if (++stage == nstage) { stage = 0; phase ^= 1u; }
        }
        // Do not leave while a copy into this CTA's shared memory may still be in flight.
        if (lane == 0) {
            const int issued = c;
            const int from = issued > nstage ? issued - nstage : 0;
            for (int k = from; k < issued; ++k)
                if (!mbar_wait(full0 + 8u * (k % nstage), (k / nstage) & 1, p.status)) break;
        }
        return;
    }

    // ---- consumers and reducer: stage this CTA's K slice of x (fragment order + per-group sums)
    {
        const int nthr = (CW + 1) * 32;
        const int t2 = warp < CW ? tid : tid - 32;  // skip the producer warp's ids
        const int kbeg = b_first * kBlockK;
        const int kend_full = (b_first + len) * kBlockK;
        const int kend = kend_full < K ? kend_full : K;
        const int ntiles = (kend - kbeg) / kGroup;
        uint8_t* xs_g = smem + p.off_xs;
        float* xsum_g = reinterpret_cast<float*>(smem + p.off_xsum);
        const int xsum_stride = (NT == 1) ? 2 : 4 * 4;  // floats per tile: {X,-128X} or 4 quads of {X0,X1,-128X0,-128X1}
        if (NT == 2)
            for (int i = t2; i < ntiles * 16; i += nthr) {
                const int tok = ((i >> 2) & 3) * 2 + (i & 1);  // slot i holds token 2q + (i & 1), q = (i >> 2) & 3
                if (tok >= M) xsum_g[i] = 0.f;
            }
        if (t2 < 16) reinterpret_cast<uint32_t*>(smem + p.off_zero)[t2] = 0u;
        const int items = ntiles * M * 4;
        for (int base = 0; base < items; base += nthr) {
            const int idx = base + t2;
            const bool valid = idx < items;
            float psum = 0.f;
            const int q = idx & 3, tm = idx >> 2;
            const int tok = tm % M, tile = tm / M;
            if (valid) {
                const uint4 v =
                    *reinterpret_cast<const uint4*>(p.x + (int64_t)tok * K + kbeg + tile * kGroup + q * 8);
                uint4 o;  // k order inside the lane's 8 values: 0,4,1,5,2,6,3,7
                o.x = __byte_perm(v.x, v.z, 0x5410);
                o.y = __byte_perm(v.x, v.z, 0x7632);
                o.z = __byte_perm(v.y, v.w, 0x5410);
                o.w = __byte_perm(v.y, v.w, 0x7632);
                *reinterpret_cast<uint4*>(xs_g + ((int64_t)tile * M + tok) * 64 + q * 16) = o;
                psum = ((bf16_lo_to_f32(v.x) + bf16_hi_to_f32(v.x)) + (bf16_lo_to_f32(v.y) + bf16_hi_to_f32(v.y))) +
                       ((bf16_lo_to_f32(v.z) + bf16_hi_to_f32(v.z)) + (bf16_lo_to_f32(v.w) + bf16_hi_to_f32(v.w)));
            }
            psum += __shfl_xor_sync(0xffffffffu, psum, 1);
            psum += __shfl_xor_sync(0xffffffffu, psum, 2);
            if (valid && q == 0) {
                if (NT == 1) {
                    xsum_g[tile * 2] = psum;
                    xsum_g[tile * 2 + 1] = -128.f * psum;
                } else {
                    float* dst = xsum_g + tile * xsum_stride + (tok >> 1) * 4 + (tok & 1);
                    dst[0] = psum;
                    dst[2] = -128.f * psum;
                }
            }
        }
        asm volatile("bar.sync 1, %0;" ::"r"(nthr) : "memory");
    }

    if (warp < CW) {
        // =============================== consumers ===============================================
        const int tw = warp & 7, j0 = (warp >> 3) * 2;
        const int g = lane >> 2, q = lane & 3;
        const uint32_t x_lane = (g < M) ? xs + g * 64 + q * 16 : zero_slot;
        const uint32_t x_stride = (g < M) ? (uint32_t)M * 64u : 0u;
        const uint32_t xsum_lane = (NT == 1) ? xsum : xsum + q * 16;
        const uint32_t xsum_stride = (NT == 1) ? 8u : 64u;
        // ldmatrix source rows: codes = row `lane` of the tile; scales/offsets = the four 16-byte
        // chunks of this tile's scale words and of its offset words, duplicated so that after the
        // transposed load every lane of a quad holds (d[g], d[g+8]), (d[g+16], d[g+24]), (m..), (m..)
        const uint32_t code_lane = tw * 512 + lane * 16;
        const int mat = lane >> 3;
        const uint32_t so_chunk = tw * 64 + (((mat & 1) * 2 + (lane & 1)) * 16);
        const uint32_t so_sect = mat >= 2 ? 576u : 512u;  // offsets section follows the scales section

        float acc[4][NT];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < NT; ++j) acc[i][j] = 0.f;

        int piece = 0;
        bool alive = true;
        // hand the warp's partial rows of the current strip piece to the reducer warp
        auto flush = [&]() {
            const int par = piece & 1;
            if (piece >= 2 && !mbar_wait(red_empty0 + 8u * par, ((piece >> 1) - 1) & 1, p.status)) alive = false;
            const uint32_t slot = part + (uint32_t)((par * CW + warp) * kStripRows * M) * 4u;
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    const int tok = 2 * q + j;
                    if (tok < M)
                        asm volatile("st.shared.f32 [%0], %1;" ::"r"(slot + (uint32_t)(tok * kStripRows + g + 8 * i) * 4u),
                                     "f"(acc[i][j])
                                     : "memory");
                    acc[i][j] = 0.f;
                }
            __syncwarp();
            if (lane == 0) mbar_arrive(red_full0 + 8u * par);
            ++piece;
        };

        int unit_first = -bl_first;          // index (relative to the CTA's first block) of block 0 of the current strip
        int unit_next = unit_first + len;    // ... and of the next strip
        int stage = 0;
        uint32_t phase = 0;
        for (int c = 0; c < nchunk && alive; ++c) {
            if (!mbar_wait(full0 + 8u * stage, phase, p.status)) { alive = false; break; }
            const uint32_t sbase = ring + stage * kStageBytes + j0 * kBlockBytes;
            const int i0 = c * CB + j0, i1 = i0 + 1;
            // block index inside the slice (for the staged x) and group count of both blocks
            int bl0 = i0 - unit_first, bl1;
            while (bl0 >= len) bl0 -= len;
            bl1 = bl0 + 1;
            if (bl1 >= len) bl1 -= len;
            const int r0 = groups_total - 8 * (b_first + bl0), r1 = groups_total - 8 * (b_first + bl1);
            const int jb0 = r0 < 8 ? r0 : 8, jb1 = r1 < 8 ? r1 : 8;
            const bool work = !(p.debug & 1);
            const bool act0 = work && (i0 < nblk) && (tw < jb0), act1 = work && (i1 < nblk) && (tw < jb1);
            TileRegs ta, tb;
            if (act0) {
                const int tile = bl0 * 8 + tw;
                tile_load<NT>(ta, sbase + code_lane, sbase + so_sect * jb0 + so_chunk, x_lane + tile * x_stride,
                              xsum_lane + tile * xsum_stride);
            }
            if (act1) {
                const int tile = bl1 * 8 + tw;
                tile_load<NT>(tb, sbase + kBlockBytes + code_lane, sbase + kBlockBytes + so_sect * jb1 + so_chunk,
                              x_lane + tile * x_stride, xsum_lane + tile * xsum_stride);
            }
            if (act0) tile_mma(ta);
            if (act1) tile_mma(tb);
            // all shared-memory reads of this stage are done: release it before the fp32 epilogue
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8u * stage);
            if (i0 < nblk) {
                while (i0 >= unit_next && alive) { flush(); unit_first = unit_next; unit_next += len; }
                if (act0) tile_scale<NT>(ta, acc);
            }
            if (i1 < nblk) {
                while (i1 >= unit_next && alive) { flush(); unit_first = unit_next; unit_next += len; }
                if (act1) tile_scale<NT>(tb, acc);
            }
            if (++stage == nstage) { stage = 0; phase ^= 1u; }
        }
        while (piece < npieces && alive) flush();
    } else {
        // =============================== reducer =================================================
        int64_t pa = a;
        for (int piece = 0; piece < npieces; ++piece) {
            const int64_t s = s_first + piece;
            const int64_t unit_begin = s * len, unit_end = unit_begin + len;
            const int64_t pe = unit_end < e ? unit_end : e;
            const int par = piece & 1;
            if (!mbar_wait(red_full0 + 8u * par, (piece >> 1) & 1, p.status)) break;
            float v[kMaxTokens];
#pragma unroll
            for (int t = 0; t < kMaxTokens; ++t) {
                v[t] = 0.f;
                if (t < M) {
#pragma unroll
                    for (int w = 0; w < CW; ++w) {
                        float f;
                        asm volatile("ld.shared.f32 %0, [%1];"
                                     : "=f"(f)
                                     : "r"(part + (uint32_t)(((par * CW + w) * M + t) * kStripRows + lane) * 4u)
                                     : "memory");
                        v[t] += f;
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(red_empty0 + 8u * par);

            const bool whole_unit = (pa == unit_begin) && (pe == unit_end);
            float* yrow = p.y + s * kStripRows + lane;
            if (whole_unit && p.Z == 1) {
#pragma unroll
                for (int t = 0; t < kMaxTokens; ++t)
                    if (t < M) yrow[(int64_t)t * p.N] = v[t];
            } else {
                float* slot = piece_slot(p, z, ci, s, unit_begin, whole_unit, a);
#pragma unroll
                for (int t = 0; t < kMaxTokens; ++t)
                    if (t < M) slot[t * kStripRows + lane] = v[t];
                __threadfence();
                __syncwarp();
                // how many pieces does strip s have over all slices?
                int total = 0;
                for (int zz = 0; zz < p.Z; ++zz) {
                    const int l2 = slice_len(p, zz);
                    const int64_t T2 = (int64_t)p.S * l2;
                    total += (int)(cta_of(s * l2 + l2 - 1, p.Gz, T2) - cta_of(s * l2, p.Gz, T2)) + 1;
                }
                int old = 0;
                if (lane == 0) old = atomicAdd(p.tickets + s, 1);
                old = __shfl_sync(0xffffffffu, old, 0);
                if (old == total - 1) {
                    // last piece to arrive: add all pieces of the strip in a fixed order
                    __threadfence();
#pragma unroll
                    for (int t = 0; t < kMaxTokens; ++t) v[t] = 0.f;
                    for (int zz = 0; zz < p.Z; ++zz) {
                        const int l2 = slice_len(p, zz);
                        const int64_t T2 = (int64_t)p.S * l2;
                        const int64_t u0 = s * l2;
                        const int64_t cf = cta_of(u0, p.Gz, T2), cl = cta_of(u0 + l2 - 1, p.Gz, T2);
                        for (int64_t c2 = cf; c2 <= cl; ++c2) {
                            const float* src = piece_slot(p, zz, c2, s, u0, cf == cl, range_begin(c2, p.Gz, T2));
#pragma unroll
                            for (int t = 0; t < kMaxTokens; ++t)
                                if (t < M) v[t] += __ldcg(src + t * kStripRows + lane);
                        }
                    }
#pragma unroll
                    for (int t = 0; t < kMaxTokens; ++t)
                        if (t < M) yrow[(int64_t)t * p.N] = v[t];
                    if (lane == 0) p.tickets[s] = 0;  // ready for the next launch on this stream
                }
            }
            pa = pe;
        }
    }
}

// ---- host-visible launchers ------------------------------------------------------------------

template <int CW, int NT>
static cudaError_t launch_one(const GemvPlan& p, cudaStream_t stream) {
    fdqp_gemv_kernel<CW, NT><<<p.Z * p.Gz, (CW + 2) * 32, p.smem_bytes, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t gemv_launch(const GemvPlan& p, int consumer_warps, cudaStream_t stream) {
    if (consumer_warps == 16) return p.M == 1 ? launch_one<16, 1>(p, stream) : launch_one<16, 2>(p, stream);
    return p.M == 1 ? launch_one<8, 1>(p, stream) : launch_one<8, 2>(p, stream);
}

cudaError_t gemv_set_smem_limit(int bytes) {
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(fdqp_gemv_kernel<8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
    if ((e = cudaFuncSetAttribute(fdqp_gemv_kernel<8, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
    if ((e = cudaFuncSetAttribute(fdqp_gemv_kernel<16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
    return cudaFuncSetAttribute(fdqp_gemv_kernel<16, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

}  // namespace fdqp
