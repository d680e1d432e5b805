// Plain CUDA-core kernels: the dequantisation engine (Sec. "Dequantization Engine", Eq. 3; bound by its writes) and a
// straightforward dequantise-then-multiply projection (Eq. 14) that serves as the library's self-check path
// ("path" = 1; not tuned).  Both read the container with plain loads.
#include "fdqp_device.cuh"
#include "fdqp_format.h"
#include "fdqp_plan.h"

#include <cuda_bf16.h>

#include <type_traits>

namespace fdqp {

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t h) { return __uint_as_float(((uint32_t)h) << 16); }

// Format variants (whole blocks only): group 64 / 128 read their scale and offset at the larger group's index; MXFP4
// multiplies the E2M1 element by its power-of-two scale (exact).
__device__ __forceinline__ float e8m0_to_f32(uint32_t e) { return __uint_as_float(e ? e << 23 : 0x00400000u); }  // 2^(e-127)
__device__ __forceinline__ float e2m1_to_f32(uint32_t q) {
    const uint32_t mag = q & 7u;  // 0, 0.5, 1, 1.5, 2, 3, 4, 6: exponent field mag >> 1, mantissa bit mag & 1
    const float v = mag < 2u ? 0.5f * (float)mag : __uint_as_float(((126u + (mag >> 1)) << 23) | ((mag & 1u) << 22));
    return (q & 8u) ? -v : v;
}

// The dequantisation engine: a CTA of eight warps dequantises the same 32-wide group of EIGHT consecutive strips (a 32 k x 256 n
// tile), transposes it through shared memory and writes every k row of the tile as one contiguous run of 256 outputs
// (512 bytes of bf16, 1 KB of fp32), 16 bytes per lane.  A warp writing its strip directly produces 64-byte pieces (bf16)
// and measured 62 % of the copy bandwidth; this one is bound by the writes.  Same arithmetic, same bits.
template <int FMT, bool OUT_BF16>
__global__ void __launch_bounds__(256) fdqp_dequant_tile_kernel(const uint8_t* __restrict__ W, void* __restrict__ out, int K,
                                                                int N) {
    using F = FmtTraits<FMT>;
    using T = typename std::conditional<OUT_BF16, uint16_t, float>::type;
    __shared__ __align__(16) T tile[32][256 + (OUT_BF16 ? 8 : 4)];  // [k][n], rows padded against bank conflicts
    __shared__ float e2m1[16];  // MXFP4: the sixteen element values
    if (F::kMx) {
        if (threadIdx.x < 16) e2m1[threadIdx.x] = e2m1_to_f32(threadIdx.x);
        __syncthreads();
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int groups = K / kGroup;
    const int gk = blockIdx.x % groups;                 // consecutive CTAs walk along K: their reads stay inside a block
    const int64_t s0 = (int64_t)(blockIdx.x / groups) * 8;
    const int64_t s = s0 + warp;
    const int strips = N / kStripRows;
    if (s < strips) {
        const int b = gk >> 3, t = gk & 7;
        const uint8_t* blk;
        float d, m = 0.f;
        if (FMT == kFmtQ4nx) {
            const int rest = groups - 8 * b;
            const int jb = rest < 8 ? rest : 8;
            blk = W + s * ((int64_t)kGroupBytes * groups) + (int64_t)b * kBlockBytes;
            d = bf16_bits_to_f32(*reinterpret_cast<const uint16_t*>(blk + 512 * jb + 2 * (t * 32 + lane)));
            m = bf16_bits_to_f32(*reinterpret_cast<const uint16_t*>(blk + 576 * jb + 2 * (t * 32 + lane)));
        } else {
            blk = W + (s * (K / kBlockK) + b) * (int64_t)F::kBlock;
            if (F::kMx) {
                d = e8m0_to_f32(blk[kCodeBytes + t * 32 + lane]);
            } else {
                d = bf16_bits_to_f32(*reinterpret_cast<const uint16_t*>(blk + kCodeBytes + 2 * ((t >> F::kShift) * 32 + lane)));
                m = bf16_bits_to_f32(*reinterpret_cast<const uint16_t*>(blk + F::kOffSect + 2 * ((t >> F::kShift) * 32 + lane)));
            }
        }
        const uint4 cv = *reinterpret_cast<const uint4*>(blk + t * 512 + lane * 16);
        const uint32_t words[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const uint32_t q = (words[i >> 3] >> (4 * (i & 7))) & 15u;
            const float w = F::kMx ? e2m1[q] * d : fmaf(d, (float)q, m);  // one rounding (Eq. 3); MXFP4 exact
            if (OUT_BF16)
                tile[i][warp * 32 + lane] = (T)__bfloat16_as_ushort(__float2bfloat16_rn(w));
            else
                tile[i][warp * 32 + lane] = (T)w;
        }
    }
    __syncthreads();
    // every k row of the tile: 256 outputs = 32 (bf16) or 64 (fp32) 16-byte pieces
    constexpr int kPieces = 256 * (int)sizeof(T) / 16;   // per row
    constexpr int kPer = 16 / (int)sizeof(T);            // outputs per piece
    const int64_t n0 = s0 * kStripRows;
    for (int idx = threadIdx.x; idx < 32 * kPieces; idx += 256) {
        const int row = idx / kPieces, piece = idx % kPieces;
        const int64_t n = n0 + piece * kPer;
        if (n < N) {  // N is a multiple of 32, so a piece is entirely inside or outside
            const uint4 v = *reinterpret_cast<const uint4*>(&tile[row][piece * kPer]);
            *reinterpret_cast<uint4*>(reinterpret_cast<T*>(out) + (int64_t)(gk * kGroup + row) * N + n) = v;
        }
    }
}

// One warp per strip, lane = output row, up to 8 tokens per pass (blockIdx.y picks the token chunk).
__global__ void __launch_bounds__(128) fdqp_plain_kernel(const uint8_t* __restrict__ W, const uint16_t* __restrict__ x,
                                                         float* __restrict__ y, int M, int K, int N) {
    const int lane = threadIdx.x & 31;
    const int64_t s = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (s >= N / kStripRows) return;
    const int m0 = blockIdx.y * kMaxTokens;
    const int mc = (M - m0) < kMaxTokens ? (M - m0) : kMaxTokens;
    const int groups = K / kGroup;
    const uint8_t* strip = W + s * ((int64_t)kGroupBytes * groups);
    float acc[kMaxTokens];
#pragma unroll
    for (int t = 0; t < kMaxTokens; ++t) acc[t] = 0.f;
    for (int gk = 0; gk < groups; ++gk) {
        const int b = gk >> 3, t = gk & 7;
        const int rest = groups - 8 * b;
        const int jb = rest < 8 ? rest : 8;
        const uint8_t* blk = strip + (int64_t)b * kBlockBytes;
        const uint4 cv = *reinterpret_cast<const uint4*>(blk + t * 512 + lane * 16);
        const float d = bf16_bits_to_f32(*reinterpret_cast<const uint16_t*>(blk + 512 * jb + 2 * (t * 32 + lane)));
        const float m = bf16_bits_to_f32(*reinterpret_cast<const uint16_t*>(blk + 576 * jb + 2 * (t * 32 + lane)));
        const uint32_t words[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float w = fmaf(d, (float)((words[i >> 3] >> (4 * (i & 7))) & 15u), m);
#pragma unroll
            for (int tk = 0; tk < kMaxTokens; ++tk)
                if (tk < mc) acc[tk] = fmaf(bf16_bits_to_f32(x[(int64_t)(m0 + tk) * K + gk * kGroup + i]), w, acc[tk]);
        }
    }
#pragma unroll
    for (int tk = 0; tk < kMaxTokens; ++tk)
        if (tk < mc) y[(int64_t)(m0 + tk) * N + s * kStripRows + lane] = acc[tk];
}

// Self-test of the give-up path every kernel of the library shares: one warp waits on a barrier that nothing ever
// arrives on, with the same bounded wait and a short limit, records the timeout and returns normally.
__global__ void __launch_bounds__(32) fdqp_wait_selftest_kernel(int* status, unsigned long long limit_ns) {
    __shared__ __align__(8) uint64_t bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) mbar_init(b, 1);
    mbar_fence_init();
    __syncwarp();
    mbar_wait_for(b, 0, status, limit_ns);
}

cudaError_t wait_selftest_launch(int* status, unsigned long long limit_ns, cudaStream_t stream) {
    fdqp_wait_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_ns);
    return cudaGetLastError();
}

template <int FMT>
static cudaError_t dequant_fmt_launch_t(const uint8_t* W, void* out, bool out_bf16, int K, int N, cudaStream_t stream) {
    const int64_t ctas = (int64_t)((N / kStripRows + 7) / 8) * (K / kGroup);
    if (out_bf16)
        fdqp_dequant_tile_kernel<FMT, true><<<(unsigned)ctas, 256, 0, stream>>>(W, out, K, N);
    else
        fdqp_dequant_tile_kernel<FMT, false><<<(unsigned)ctas, 256, 0, stream>>>(W, out, K, N);
    return cudaGetLastError();
}

cudaError_t dequant_launch(const uint8_t* W, void* out, bool out_bf16, int K, int N, cudaStream_t stream) {
    return dequant_fmt_launch_t<kFmtQ4nx>(W, out, out_bf16, K, N, stream);
}

cudaError_t dequant_fmt_launch(int fmt, const uint8_t* W, void* out, bool out_bf16, int K, int N, cudaStream_t stream) {
    switch (fmt) {
        case kFmtQ4nx: return dequant_launch(W, out, out_bf16, K, N, stream);
        case kFmtG64: return dequant_fmt_launch_t<kFmtG64>(W, out, out_bf16, K, N, stream);
        case kFmtG128: return dequant_fmt_launch_t<kFmtG128>(W, out, out_bf16, K, N, stream);
        case kFmtMxfp4: return dequant_fmt_launch_t<kFmtMxfp4>(W, out, out_bf16, K, N, stream);
    }
    return cudaErrorInvalidValue;
}

cudaError_t plain_launch(const uint8_t* W, const uint16_t* x, float* y, int M, int K, int N, cudaStream_t stream) {
    const int strips = N / kStripRows;
    dim3 grid((unsigned)((strips + 3) / 4), (unsigned)((M + kMaxTokens - 1) / kMaxTokens));
    fdqp_plain_kernel<<<grid, 128, 0, stream>>>(W, x, y, M, K, N);
    return cudaGetLastError();
}

// ---- read-stream reference ------------------------------------------------------------------------------------------
//
// What the weight stream of the projection kernels could reach at most: one persistent CTA per SM pulls its share of a
// buffer through a shared-memory ring with the same 1-D bulk copies (40 KB per stage, evict-first) and drops the data.
// A measurement aid: the copy bandwidth counts a read and a write per byte, this one only reads.
constexpr int kStreamStages = 5;
constexpr uint32_t kStreamChunk = 8u * kBlockBytes;  // one ring stage of the projection kernels

__global__ void __launch_bounds__(32, 1) fdqp_stream_read_kernel(const uint8_t* __restrict__ buf, int64_t chunks, int* status) {
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t ring = smem_u32(smem);
    const uint32_t bars = ring + kStreamStages * kStreamChunk;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStreamStages; ++s) mbar_init(bars + 8u * s, 1);
        mbar_fence_init();
    }
    __syncwarp();
    if (threadIdx.x != 0) return;
    // this CTA's chunks: c0, c0 + 1, ... (equal contiguous shares)
    const int64_t c0 = chunks * blockIdx.x / gridDim.x, c1 = chunks * (blockIdx.x + 1) / gridDim.x;
    const int64_t n = c1 - c0;
    const uint64_t policy = l2_policy_evict_first();
    auto issue = [&](int64_t k) {
        const uint32_t bar = bars + 8u * (uint32_t)(k % kStreamStages);
        mbar_arrive_expect_tx(bar, kStreamChunk);
        bulk_g2s_hint(ring + (uint32_t)(k % kStreamStages) * kStreamChunk, buf + (c0 + k) * (int64_t)kStreamChunk, kStreamChunk, bar, policy);
    };
    for (int64_t k = 0; k < n && k < kStreamStages; ++k) issue(k);
    for (int64_t k = 0; k < n; ++k) {
        if (!mbar_wait(bars + 8u * (uint32_t)(k % kStreamStages), (uint32_t)(k / kStreamStages) & 1u, status)) break;
        if (k + kStreamStages < n) issue(k + kStreamStages);
    }
}

cudaError_t stream_read_launch(const uint8_t* buf, int64_t bytes, int sm_count, int* status, cudaStream_t stream) {
    static bool attr_set = false;
    constexpr int kSmem = kStreamStages * (int)kStreamChunk + 64;
    cudaError_t e;
    if (!attr_set) {
        if ((e = cudaFuncSetAttribute(fdqp_stream_read_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem))) return e;
        attr_set = true;
    }
    const int64_t chunks = bytes / (int64_t)kStreamChunk;
    if (chunks < 1) return cudaSuccess;
    fdqp_stream_read_kernel<<<sm_count, 32, kSmem, stream>>>(buf, chunks, status);
    return cudaGetLastError();
}

}  // namespace fdqp
