// Device-side helpers shared by the FusedDQP kernels: mbarrier, bulk async copies,
// ldmatrix / mma.sync wrappers and the bounded wait every spin in this library uses.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace fdqp {

// Status word values written by kernels (match fdqp_status in fdqp.h).
constexpr int kStatusTimeout = 8;

// A wait that has not succeeded after this long gives up, records kStatusTimeout and lets
// the kernel drain instead of hanging the device.
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// ---- mbarrier -------------------------------------------------------------------------

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// The same test, but the thread may stay suspended for up to about a microsecond (it resumes at once when the phase
// completes): a waiting warp then spends few issue slots on polling.
__device__ __forceinline__ bool mbar_try_wait_suspended(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(1000u)
        : "memory");
    return ok != 0;
}

// Bounded wait on a phase parity.  Returns false (after recording the timeout in *status) if
// the barrier did not flip within `limit_ns`.
__device__ __forceinline__ bool mbar_wait_for(uint32_t bar, uint32_t parity, int* status, unsigned long long limit_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = globaltimer_ns();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait_suspended(bar, parity)) return true;
        if ((it & 63u) == 0u && globaltimer_ns() - t0 > limit_ns) {
            atomicExch(status, kStatusTimeout);
            __threadfence_system();
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* status) {
    return mbar_wait_for(bar, parity, status, kWaitLimitNs);
}

// ---- bulk async copy global -> shared (1-D, no multicast) ---------------------------------

__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// dst, src 16-byte aligned; bytes a multiple of 16.  Completion is signalled on `bar` as
// transaction bytes.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar,
                                              uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            dst),
        "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}

// ---- warp matrix helpers ---------------------------------------------------------------------

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t (&r)[2], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}

// D = A(16x16, bf16, row) * B(16x8, bf16, col) + C, fp32 accumulate.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1, const float (&c)[4]) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%10,%11,%12,%13};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

__device__ __forceinline__ float2 lds64f(uint32_t addr) {
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
    return v;
}

// Mixed-precision FMA (bf16 x bf16 + f32 -> f32): one FMA-pipe instruction that reads a 16-bit half of a
// 32-bit register, so widening a packed bf16 pair costs no integer/logic instruction.
// a = low / high half of `packed`, b = HIGH half of `w` (the bf16 truncation of an fp32 value, exact when that
// value is a power of two or already bf16).
__device__ __forceinline__ float bf16lo_mul_f32hi(uint32_t packed, float w) {
    float r;
    asm("{\n\t.reg .b16 alo, ahi, wlo, whi;\n\t"
        "mov.b32 {alo, ahi}, %1;\n\tmov.b32 {wlo, whi}, %2;\n\t"
        "fma.rn.f32.bf16 %0, alo, whi, %3;\n\t}"
        : "=f"(r)
        : "r"(packed), "f"(w), "f"(0.f));
    return r;
}
__device__ __forceinline__ float bf16hi_mul_f32hi(uint32_t packed, float w) {
    float r;
    asm("{\n\t.reg .b16 alo, ahi, wlo, whi;\n\t"
        "mov.b32 {alo, ahi}, %1;\n\tmov.b32 {wlo, whi}, %2;\n\t"
        "fma.rn.f32.bf16 %0, ahi, whi, %3;\n\t}"
        : "=f"(r)
        : "r"(packed), "f"(w), "f"(0.f));
    return r;
}

// Round-to-nearest-even bf16 bits of an fp32 (one conversion instruction).
__device__ __forceinline__ uint16_t f32_to_bf16_rne(float f) {
    uint16_t r;
    asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(r) : "f"(f));
    return r;
}

// GELU, tanh form: 0.5 g (1 + tanh(z)), z = sqrt(2/pi) (g + 0.044715 g^3), written as g / (1 + exp(-2 z)): the same
// function, two fast-math instructions instead of a tanh call; saturates to g and to -0 exactly.
__device__ __forceinline__ float gelu_tanh(float g) {
    const float z2 = 1.5957691216057308f * (g + 0.044715f * g * g * g);  // 2 z
    return __fdividef(g, 1.0f + __expf(-z2));
}

// The stored bits of one finished value under a bf16 epilogue; `up` is the partner row's value (gated GELU only).
__device__ __forceinline__ uint16_t epilogue_bf16(int epi, float v, float up) {
    return f32_to_bf16_rne(epi == 1 ? v : gelu_tanh(v) * up);
}

// One finished output value per lane: row `lane` of 32-row strip s, token row t.  All 32 lanes must call it together.
__device__ __forceinline__ void store_output(float* y, uint16_t* y16, int epi, int64_t N, int64_t s, int lane, int t,
                                             float v) {
    if (epi == 0) {
        y[(int64_t)t * N + s * 32 + lane] = v;
    } else if (epi == 1) {
        y16[(int64_t)t * N + s * 32 + lane] = epilogue_bf16(1, v, 0.f);
    } else {
        const float up = __shfl_xor_sync(0xffffffffu, v, 16);
        if (lane < 16) y16[(int64_t)t * (N / 2) + s * 16 + lane] = epilogue_bf16(2, v, up);
    }
}

__device__ __forceinline__ float bf16_lo_to_f32(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16_hi_to_f32(uint32_t packed) { return __uint_as_float(packed & 0xffff0000u); }

}  // namespace fdqp
