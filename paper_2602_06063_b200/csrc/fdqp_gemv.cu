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
// (exact), the +128 is folded into the offset term (m - 128 d) * sum_k x_k, and the order of k inside
// a group is a free permutation as long as x is staged with the same one.
//
// Data movement.  The packed matrix is strip-major (32 output rows x all of K contiguous), so every
// CTA streams one contiguous byte range of HBM exactly once: a producer thread issues one 1-D bulk
// async copy per Q4NX block (<= 5120 bytes) into a shared-memory ring guarded by mbarriers; each of
// the 8 consumer warps of a warp group owns one 32 x 32 group-tile of the block.  x (the CTA's K
// slice, all tokens) is staged once per CTA in the fragment order the MMA wants, together with the
// per-group sums of x.
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

template <int CW, int NT>
__global__ void __launch_bounds__((CW + 2) * 32, 1) fdqp_gemv_kernel(const __grid_constant__ GemvPlan p) {
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int NBP = CW / 8;  // blocks in flight per CTA step: one per warp group
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

    const uint32_t ring = smem_u32(smem);
    const uint32_t xs = ring + p.off_xs, zero_slot = ring + p.off_zero, xsum = ring + p.off_xsum;
    const uint32_t part = ring + p.off_part, bars = ring + p.off_bar;
    const int nstage = p.nstage;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (nstage + s); };
    auto red_full = [&](int par) { return bars + 8u * (2 * nstage + par); };
    auto red_empty = [&](int par) { return bars + 8u * (2 * nstage + 2 + par); };

    if (tid == 0) {
        for (int s = 0; s < nstage; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 8);
        }
        for (int par = 0; par < 2; ++par) {
            mbar_init(red_full(par), CW);
            mbar_init(red_empty(par), 1);
        }
        mbar_fence_init();
    }
    __syncthreads();

    const int groups_total = K / kGroup;
    const int64_t strip_bytes = (int64_t)kGroupBytes * groups_total;
    auto block_groups = [&](int b) {
        const int rest = groups_total - 8 * b;
        return rest < 8 ? rest : 8;
    };

    // ---- producer state (warp CW, lane 0) and first fills: start the HBM stream before staging x
    const bool is_producer = (warp == CW) && (lane == 0);
    int64_t prod_s = 0;
    int prod_bl = 0, prod_i = 0, prod_stage = 0;
    uint64_t policy = 0;
    if (is_producer) {
        if (p.evict_first) policy = l2_policy_evict_first();
        prod_s = a / len;
        prod_bl = (int)(a - prod_s * len);
        const int first = nblk < nstage ? nblk : nstage;
        for (; prod_i < first; ++prod_i) {
            const int b = b_first + prod_bl;
            const uint32_t bytes = (uint32_t)(kGroupBytes * block_groups(b));
            const uint8_t* src = p.W + prod_s * strip_bytes + (int64_t)b * kBlockBytes;
            mbar_arrive_expect_tx(full_bar(prod_stage), bytes);
            if (p.evict_first)
                bulk_g2s_hint(ring + prod_stage * kBlockBytes, src, bytes, full_bar(prod_stage), policy);
            else
                bulk_g2s(ring + prod_stage * kBlockBytes, src, bytes, full_bar(prod_stage));
            if (++prod_bl == len) { prod_bl = 0; ++prod_s; }
            if (++prod_stage == nstage) prod_stage = 0;
        }
    }

    // ---- stage this CTA's K slice of x: fragment order for the MMA, plus per-group sums
    {
        const int kbeg = b_first * kBlockK;
        const int kend_full = (b_first + len) * kBlockK;
        const int kend = kend_full < K ? kend_full : K;
        const int ntiles = (kend - kbeg) / kGroup;
        uint8_t* xs_g = smem + p.off_xs;
        float* xsum_g = reinterpret_cast<float*>(smem + p.off_xsum);
        for (int i = tid; i < ntiles * kMaxTokens; i += blockDim.x)
            if ((i & 7) >= M) xsum_g[i] = 0.f;
        if (tid < 16) reinterpret_cast<uint32_t*>(smem + p.off_zero)[tid] = 0u;
        const int items = ntiles * M * 4;
        for (int base = 0; base < items; base += blockDim.x) {
            const int idx = base + tid;
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
            if (valid && q == 0) xsum_g[tile * kMaxTokens + tok] = psum;
        }
    }
    __syncthreads();

    if (warp < CW) {
        // =============================== consumers ===============================================
        const int wg = warp >> 3, tw = warp & 7;
        const int g = lane >> 2, q = lane & 3;
        const uint32_t x_lane = (g < M) ? xs + g * 64 + q * 16 : zero_slot;
        const uint32_t x_stride = (g < M) ? (uint32_t)M * 64u : 0u;
        const uint32_t xsum_lane = xsum + q * 8;
        // ldmatrix source rows: codes = row `lane` of the tile; scales/offsets = the four 16-byte
        // chunks of this tile's scale words and of its offset words, duplicated so that after the
        // transposed load every lane of a quad holds (d[g], d[g+8]), (d[g+16], d[g+24]), (m..), (m..)
        const uint32_t code_lane = tw * 512 + lane * 16;
        const int mat = lane >> 3;
        const uint32_t so_chunk = tw * 64 + (((mat & 1) * 2 + (lane & 1)) * 16);
        const bool so_is_offset = mat >= 2;

        float acc[4][NT];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < NT; ++j) acc[i][j] = 0.f;

        int i_rel = wg;                 // index of this group's next block relative to `a`
        int stage = wg % nstage;        // its ring stage
        uint32_t phase = (wg / nstage) & 1;
        int piece = 0;
        bool alive = true;
        int64_t pa = a;
        while (pa < e && alive) {
            const int64_t s = pa / len;
            const int64_t unit_end = (s + 1) * len;
            const int64_t pe = unit_end < e ? unit_end : e;
            int bl = (int)(a + i_rel - s * len);  // block index inside the slice for i_rel (valid when inside piece)
            const int i_end = (int)(pe - a);
            for (; i_rel < i_end; i_rel += NBP, bl += NBP) {
                const int b = b_first + bl;
                const int jb = block_groups(b);
                if (!mbar_wait(full_bar(stage), phase, p.status)) { alive = false; break; }
                if (tw < jb) {
                    const uint32_t sbase = ring + stage * kBlockBytes;
                    uint32_t c[4], so[4];
                    ldmatrix_x4(c, sbase + code_lane);
                    ldmatrix_x4_trans(so, sbase + (so_is_offset ? 576u : 512u) * jb + so_chunk);
                    const int tile = bl * 8 + tw;
                    const uint4 xb = lds128(x_lane + tile * x_stride);
                    const float2 xs2 = lds64f(xsum_lane + tile * (kMaxTokens * 4));
                    const float zero4[4] = {0.f, 0.f, 0.f, 0.f};
                    float d0[4], d1[4];
                    {
                        const uint32_t lo = c[0], hi = c[1];
                        mma_bf16_16816(d0, (lo & 0x000F000Fu) | 0x43004300u, (hi & 0x000F000Fu) | 0x43004300u,
                                       ((lo >> 4) & 0x000F000Fu) | 0x43004300u, ((hi >> 4) & 0x000F000Fu) | 0x43004300u,
                                       xb.x, xb.y, zero4);
                        mma_bf16_16816(d0, ((lo >> 8) & 0x000F000Fu) | 0x43004300u,
                                       ((hi >> 8) & 0x000F000Fu) | 0x43004300u,
                                       ((lo >> 12) & 0x000F000Fu) | 0x43004300u,
                                       ((hi >> 12) & 0x000F000Fu) | 0x43004300u, xb.z, xb.w, d0);
                    }
                    {
                        const uint32_t lo = c[2], hi = c[3];
                        mma_bf16_16816(d1, (lo & 0x000F000Fu) | 0x43004300u, (hi & 0x000F000Fu) | 0x43004300u,
                                       ((lo >> 4) & 0x000F000Fu) | 0x43004300u, ((hi >> 4) & 0x000F000Fu) | 0x43004300u,
                                       xb.x, xb.y, zero4);
                        mma_bf16_16816(d1, ((lo >> 8) & 0x000F000Fu) | 0x43004300u,
                                       ((hi >> 8) & 0x000F000Fu) | 0x43004300u,
                                       ((lo >> 12) & 0x000F000Fu) | 0x43004300u,
                                       ((hi >> 12) & 0x000F000Fu) | 0x43004300u, xb.z, xb.w, d1);
                    }
                    // per-group scale and offset, fp32: rows g, g+8, g+16, g+24
                    const float dsc[4] = {bf16_lo_to_f32(so[0]), bf16_hi_to_f32(so[0]), bf16_lo_to_f32(so[1]),
                                          bf16_hi_to_f32(so[1])};
                    const float mof[4] = {bf16_lo_to_f32(so[2]), bf16_hi_to_f32(so[2]), bf16_lo_to_f32(so[3]),
                                          bf16_hi_to_f32(so[3])};
                    const float dd[4][2] = {{d0[0], d0[1]}, {d0[2], d0[3]}, {d1[0], d1[1]}, {d1[2], d1[3]}};
                    const float xsv[2] = {xs2.x, xs2.y};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float cc = fmaf(dsc[i], -128.f, mof[i]);  // offset with the +128 code bias folded in
#pragma unroll
                        for (int j = 0; j < NT; ++j) {
                            acc[i][j] = fmaf(dsc[i], dd[i][j], acc[i][j]);
                            acc[i][j] = fmaf(cc, xsv[j], acc[i][j]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_bar(stage));
                stage += NBP;
                if (stage >= nstage) { stage -= nstage; phase ^= 1u; }
            }
            if (!alive) break;
            // ---- end of this strip piece: hand the warp's partial rows to the reducer warp
            const int par = piece & 1;
            if (piece >= 2 && !mbar_wait(red_empty(par), ((piece >> 1) - 1) & 1, p.status)) { alive = false; break; }
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
            if (lane == 0) mbar_arrive(red_full(par));
            ++piece;
            pa = pe;
        }
    } else if (warp == CW) {
        // =============================== producer ================================================
        if (lane == 0) {
            bool alive = true;
            for (; prod_i < nblk && alive; ++prod_i) {
                // the stage was last used by block prod_i - nstage; wait until its 8 warps released it
                if (!mbar_wait(empty_bar(prod_stage), ((prod_i / nstage) - 1) & 1, p.status)) { alive = false; break; }
                const int b = b_first + prod_bl;
                const uint32_t bytes = (uint32_t)(kGroupBytes * block_groups(b));
                const uint8_t* src = p.W + prod_s * strip_bytes + (int64_t)b * kBlockBytes;
                mbar_arrive_expect_tx(full_bar(prod_stage), bytes);
                if (p.evict_first)
                    bulk_g2s_hint(ring + prod_stage * kBlockBytes, src, bytes, full_bar(prod_stage), policy);
                else
                    bulk_g2s(ring + prod_stage * kBlockBytes, src, bytes, full_bar(prod_stage));
                if (++prod_bl == len) { prod_bl = 0; ++prod_s; }
                if (++prod_stage == nstage) prod_stage = 0;
            }
            // Do not leave while a copy into this CTA's shared memory may still be in flight.
            const int issued = prod_i;
            const int from = issued > nstage ? issued - nstage : 0;
            for (int i = from; i < issued; ++i)
                if (!mbar_wait(full_bar(i % nstage), (i / nstage) & 1, p.status)) break;
        }
    } else {
        // =============================== reducer =================================================
        int piece = 0;
        int64_t pa = a;
        while (pa < e) {
            const int64_t s = pa / len;
            const int64_t unit_begin = s * len, unit_end = unit_begin + len;
            const int64_t pe = unit_end < e ? unit_end : e;
            const int par = piece & 1;
            if (!mbar_wait(red_full(par), (piece >> 1) & 1, p.status)) break;
            float v[kMaxTokens];
#pragma unroll
            for (int t = 0; t < kMaxTokens; ++t) {
                v[t] = 0.f;
                if (t < M) {
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
            if (lane == 0) mbar_arrive(red_empty(par));

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
            ++piece;
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
