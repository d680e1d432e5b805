// Plain CUDA-core kernels: the dequantisation engine (Sec. "Dequantization Engine", Eq. 3) and a
// straightforward dequantise-then-multiply projection (Eq. 14) that serves as the library's
// self-check path ("path" = 1).  Neither is tuned; both read the container with plain loads.
#include "fdqp_device.cuh"
#include "fdqp_format.h"
#include "fdqp_plan.h"

#include <cuda_bf16.h>

namespace fdqp {

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t h) { return __uint_as_float(((uint32_t)h) << 16); }

// One warp per (strip, group): lane = output row.  out is [K][N]; the 32 lanes of a warp write 32
// consecutive n for each k, so every store is one full 128-byte (fp32) or 64-byte (bf16) line.
template <bool OUT_BF16>
__global__ void __launch_bounds__(256) fdqp_dequant_kernel(const uint8_t* __restrict__ W, void* __restrict__ out, int K,
                                                           int N) {
    const int lane = threadIdx.x & 31;
    const int groups = K / kGroup;
    const int64_t unit = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t total = (int64_t)(N / kStripRows) * groups;
    if (unit >= total) return;
    const int64_t s = unit / groups;
    const int gk = (int)(unit % groups);
    const int b = gk >> 3, t = gk & 7;
    const int rest = groups - 8 * b;
    const int jb = rest < 8 ? rest : 8;
    const uint8_t* blk = W + s * ((int64_t)kGroupBytes * groups) + (int64_t)b * kBlockBytes;
    const uint4 cv = *reinterpret_cast<const uint4*>(blk + t * 512 + lane * 16);
    const float d = bf16_bits_to_f32(*reinterpret_cast<const uint16_t*>(blk + 512 * jb + 2 * (t * 32 + lane)));
    const float m = bf16_bits_to_f32(*reinterpret_cast<const uint16_t*>(blk + 576 * jb + 2 * (t * 32 + lane)));
    const uint32_t words[4] = {cv.x, cv.y, cv.z, cv.w};
    const int64_t n = s * kStripRows + lane;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const float qf = (float)((words[i >> 3] >> (4 * (i & 7))) & 15u);
        const float w = fmaf(d, qf, m);  // d*q is exact, so this is the single rounding Eq. 3 asks for
        const int64_t at = (int64_t)(gk * kGroup + i) * N + n;
        if (OUT_BF16)
            reinterpret_cast<__nv_bfloat16*>(out)[at] = __float2bfloat16_rn(w);
        else
            reinterpret_cast<float*>(out)[at] = w;
    }
}

// The same engine for the format variants (whole blocks only): group 64 / 128 read their scale and offset at the larger
// group's index; MXFP4 multiplies the E2M1 element by its power-of-two scale (exact).
__device__ __forceinline__ float e8m0_to_f32(uint32_t e) { return __uint_as_float(e ? e << 23 : 0x00400000u); }  // 2^(e-127)
__device__ __forceinline__ float e2m1_to_f32(uint32_t q) {
    const uint32_t mag = q & 7u;  // 0, 0.5, 1, 1.5, 2, 3, 4, 6: exponent field mag >> 1, mantissa bit mag & 1
    const float v = mag < 2u ? 0.5f * (float)mag : __uint_as_float(((126u + (mag >> 1)) << 23) | ((mag & 1u) << 22));
    return (q & 8u) ? -v : v;
}

template <int FMT, bool OUT_BF16>
__global__ void __launch_bounds__(256) fdqp_dequant_fmt_kernel(const uint8_t* __restrict__ W, void* __restrict__ out, int K,
                                                               int N) {
    using F = FmtTraits<FMT>;
    const int lane = threadIdx.x & 31;
    const int groups = K / kGroup;  // 32-column tiles
    const int64_t unit = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t total = (int64_t)(N / kStripRows) * groups;
    if (unit >= total) return;
    const int64_t s = unit / groups;
    const int gk = (int)(unit % groups);
    const int b = gk >> 3, t = gk & 7;
    const uint8_t* blk = W + (s * (K / kBlockK) + b) * (int64_t)F::kBlock;
    const uint4 cv = *reinterpret_cast<const uint4*>(blk + t * 512 + lane * 16);
    float d, m = 0.f;
    if (F::kMx) {
        d = e8m0_to_f32(blk[kCodeBytes + t * 32 + lane]);
    } else {
        d = bf16_bits_to_f32(*reinterpret_cast<const uint16_t*>(blk + kCodeBytes + 2 * ((t >> F::kShift) * 32 + lane)));
        m = bf16_bits_to_f32(*reinterpret_cast<const uint16_t*>(blk + F::kOffSect + 2 * ((t >> F::kShift) * 32 + lane)));
    }
    const uint32_t words[4] = {cv.x, cv.y, cv.z, cv.w};
    const int64_t n = s * kStripRows + lane;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const uint32_t q = (words[i >> 3] >> (4 * (i & 7))) & 15u;
        const float w = F::kMx ? e2m1_to_f32(q) * d : fmaf(d, (float)q, m);
        const int64_t at = (int64_t)(gk * kGroup + i) * N + n;
        if (OUT_BF16)
            reinterpret_cast<__nv_bfloat16*>(out)[at] = __float2bfloat16_rn(w);
        else
            reinterpret_cast<float*>(out)[at] = w;
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

cudaError_t dequant_launch(const uint8_t* W, void* out, bool out_bf16, int K, int N, cudaStream_t stream) {
    const int64_t units = (int64_t)(N / kStripRows) * (K / kGroup);
    const unsigned grid = (unsigned)((units + 7) / 8);
    if (out_bf16)
        fdqp_dequant_kernel<true><<<grid, 256, 0, stream>>>(W, out, K, N);
    else
        fdqp_dequant_kernel<false><<<grid, 256, 0, stream>>>(W, out, K, N);
    return cudaGetLastError();
}

template <int FMT>
static cudaError_t dequant_fmt_launch_t(const uint8_t* W, void* out, bool out_bf16, int K, int N, cudaStream_t stream) {
    const int64_t units = (int64_t)(N / kStripRows) * (K / kGroup);
    const unsigned grid = (unsigned)((units + 7) / 8);
    if (out_bf16)
        fdqp_dequant_fmt_kernel<FMT, true><<<grid, 256, 0, stream>>>(W, out, K, N);
    else
        fdqp_dequant_fmt_kernel<FMT, false><<<grid, 256, 0, stream>>>(W, out, K, N);
    return cudaGetLastError();
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

}  // namespace fdqp
