// Decode attention over a KV cache, chunk by chunk with an online softmax (the paper's FlowKV, Sec. "FlowKV": the
// decoding-step attention  o = sum_j softmax_j(scale * q . k_j) v_j  evaluated one key/value chunk at a time, with
// grouped-query attention and, for local layers, a sliding window -- FlowKV-SWA).
//
// The paper pipelines key chunks through one compute tile and value chunks through a second one.  Here the unit of work
// is a (KV head, range of positions) pair per CTA, so that all SMs stream the cache at once whatever the head count is:
//   - grid (splits, KV heads); a CTA's four warps each own every fourth 16-position tile of the CTA's range and run
//     their own cp.async ring (three stages of a 16 x d key tile and a 16 x d value tile, 16-byte chunks XOR-swizzled so
//     that ldmatrix reads are conflict-free);
//   - scores: S^T[16 positions][8 query heads] = K_tile (16 x d) . Q^T (d x 8) on mma.sync m16n8k16 (bf16, fp32
//     accumulate); the query heads of the KV head's group are the B operand and stay in registers (up to 8 per group);
//   - online softmax per query head in the exp2 domain (running maximum m, running sum l), probabilities rounded to
//     bf16 and moved into B-operand layout with eight shuffles;
//   - O^T[d][8 heads] += V_tile^T (d x 16, ldmatrix.trans) . P (16 x 8), fp32 accumulators in registers;
//   - the four warps' (m, l, O) are merged through shared memory and written as one partial per (split, head);
//     flowkv_merge_kernel combines the splits' partials in split order and normalises.
//   - short ranges (a sliding window, a young cache) are one launch: the splits of a KV head form a thread-block cluster
//     of up to 16 CTAs, every CTA leaves its partial in its own shared memory and, after a cluster barrier, each CTA
//     combines one slice of the head's outputs across all partials through distributed shared memory, in split order.
// Each cache byte is read once.  Everything is deterministic (fixed merge orders).
#include "fdqp_device.cuh"

namespace fdqp {

constexpr int kKvWarps = 4;
constexpr int kKvTile = 16;     // positions per warp tile
constexpr int kKvStages = 3;
constexpr int kKvMaxGroup = 8;  // query heads per KV head
constexpr int kKvMergeThreads = 1024;
constexpr int kKvMaxSplitsDev = 160;  // upper bound of the split count the merge kernel handles (a multiple of 32)
constexpr int kKvMaxCluster = 16;     // splits of the one-launch variant: one thread-block cluster per KV head

struct FlowKvParams {
    const uint16_t* q;  // [H][d]
    const uint16_t* K;  // [G][pitch][d]
    const uint16_t* V;
    float* ws;          // [H][splits][d + 4]: partial O (unnormalised), running maximum, running sum, 2 unused
    float* out;         // [H][d]: written by the one-launch variant only
    int H, G, L, pitch;
    int j0;             // first position attended to (0, or L - window)
    int chunk;          // positions per split (a multiple of kKvWarps * kKvTile)
    int splits;
    float scale_log2e;  // scale * log2(e): scores go through exp2
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int bytes = valid ? 16 : 0;  // 0: nothing is read, the 16 bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// a float of CTA `rank`'s shared memory, at the address `local` has in this CTA's
__device__ __forceinline__ float ld_cluster_f32(uint32_t local, uint32_t rank) {
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

// CLUSTER: the grid's x dimension is one cluster (splits <= kKvMaxCluster); the kernel writes `out` itself.
template <int D, bool CLUSTER>
__global__ void __launch_bounds__(kKvWarps * 32, 1) flowkv_decode_kernel(const FlowKvParams p) {
    constexpr int kRowBytes = D * 2;
    constexpr int kChunksPerRow = kRowBytes / 16;            // 32 (d = 256) or 16 (d = 128)
    constexpr int kTileBytes = kKvTile * kRowBytes;          // one 16-position tile of K or of V
    constexpr int kStageBytes = 2 * kTileBytes;              // K tile then V tile
    constexpr int kCopies = kKvTile * kChunksPerRow / 32;    // 16-byte copies per lane per tile and matrix
    extern __shared__ __align__(128) uint8_t smem[];
    // Launched with programmatic stream serialisation: the next launch may be set up while this grid runs; this grid
    // touches nothing (q, the cache and the workspace may all come from earlier launches) before those have completed.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g4 = lane >> 2, q4 = lane & 3;
    const int split = blockIdx.x, kvh = blockIdx.y;
    const int R = p.H / p.G;  // query heads of this KV head
    const int jb = p.j0 + split * p.chunk;
    const int je = (jb + p.chunk) < p.L ? (jb + p.chunk) : p.L;
    const int ntiles_cta = (je - jb + kKvTile - 1) / kKvTile;
    const int my_tiles = ntiles_cta > warp ? (ntiles_cta - warp + kKvWarps - 1) / kKvWarps : 0;
    const uint8_t* Kg = reinterpret_cast<const uint8_t*>(p.K) + (size_t)kvh * p.pitch * kRowBytes;
    const uint8_t* Vg = reinterpret_cast<const uint8_t*>(p.V) + (size_t)kvh * p.pitch * kRowBytes;
    const uint32_t ring = smem_u32(smem) + warp * (kKvStages * kStageBytes);

    // the copies of tile t (this warp's t-th tile) into ring stage t % kKvStages
    auto issue = [&](int t) {
        if (t < my_tiles) {
            const int j_tile = jb + (warp + t * kKvWarps) * kKvTile;
            const uint32_t dst = ring + (t % kKvStages) * kStageBytes;
#pragma unroll
            for (int i = 0; i < kCopies; ++i) {
                const int id = lane + 32 * i, row = id / kChunksPerRow, c = id % kChunksPerRow;
                const int j = j_tile + row;
                const bool ok = j < je;
                const size_t src = (size_t)(ok ? j : jb) * kRowBytes + (size_t)c * 16;
                const uint32_t off = (uint32_t)(row * kRowBytes + (((c & ~7) | ((c ^ row) & 7)) << 4));
                cp_async16(dst + off, Kg + src, ok);
                cp_async16(dst + kTileBytes + off, Vg + src, ok);
            }
        }
        cp_async_commit();  // one group per call, empty or not: the wait below counts groups
    };

    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};  // heads 2 q4 and 2 q4 + 1
    float o[D / 16][4];                                               // O^T: dims 16 dt + g4 (+8) x heads 2 q4 (+1)
#pragma unroll
    for (int dt = 0; dt < D / 16; ++dt) o[dt][0] = o[dt][1] = o[dt][2] = o[dt][3] = 0.f;

#pragma unroll
    for (int t = 0; t < kKvStages - 1; ++t) issue(t);

    // ---- Q^T as B fragments (loaded while the first tiles are on their way): lane (g4, q4) holds head g4, dims 16 kk + 2 q4 (+1) and + 8 (+9)
    uint32_t qf[D / 16][2];
    {
        const uint16_t* qh = p.q + (size_t)(kvh * R + (g4 < R ? g4 : 0)) * D;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t lo = *reinterpret_cast<const uint32_t*>(qh + kk * 16 + 2 * q4);
            const uint32_t hi = *reinterpret_cast<const uint32_t*>(qh + kk * 16 + 2 * q4 + 8);
            qf[kk][0] = g4 < R ? lo : 0u;
            qf[kk][1] = g4 < R ? hi : 0u;
        }
    }


    // ldmatrix source rows/chunks of this lane: matrix mi = lane / 8
    const int mi = lane >> 3, r8 = lane & 7;
    const int k_row = (mi & 1) * 8 + r8, k_cadd = mi >> 1;   // K (not transposed): matrices (rows 0-7 | 8-15) x (dims +0 | +8)
    const int v_row = (mi >> 1) * 8 + r8, v_cadd = mi & 1;   // V (transposed): matrices (keys 0-7 | 8-15) x (dims +0 | +8)

    for (int t = 0; t < my_tiles; ++t) {
        cp_async_wait<kKvStages - 2>();
        __syncwarp();
        const uint32_t kt = ring + (t % kKvStages) * kStageBytes, vt = kt + kTileBytes;
        const int j_tile = jb + (warp + t * kKvWarps) * kKvTile;

        // ---- scores S^T = K . Q^T
        float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            uint32_t a[4];
            const int c = kk * 2 + k_cadd;
            ldmatrix_x4(a, kt + (uint32_t)(k_row * kRowBytes + (((c & ~7) | ((c ^ k_row) & 7)) << 4)));
            mma_bf16_16816(s, a[0], a[1], a[2], a[3], qf[kk][0], qf[kk][1], s);
        }
        // the next tile's copies can start now: the stage they go to was read two iterations ago
        issue(t + kKvStages - 1);

        // ---- online softmax, per head (columns 2 q4, 2 q4 + 1), positions g4 and g4 + 8 of the tile
        const bool v_lo = j_tile + g4 < je, v_hi = j_tile + g4 + 8 < je;
        float sc[4];
        sc[0] = v_lo ? s[0] * p.scale_log2e : -INFINITY;
        sc[1] = v_lo ? s[1] * p.scale_log2e : -INFINITY;
        sc[2] = v_hi ? s[2] * p.scale_log2e : -INFINITY;
        sc[3] = v_hi ? s[3] * p.scale_log2e : -INFINITY;
        float tmax[2] = {fmaxf(sc[0], sc[2]), fmaxf(sc[1], sc[3])};
#pragma unroll
        for (int sh = 4; sh <= 16; sh <<= 1) {
            tmax[0] = fmaxf(tmax[0], __shfl_xor_sync(0xffffffffu, tmax[0], sh));
            tmax[1] = fmaxf(tmax[1], __shfl_xor_sync(0xffffffffu, tmax[1], sh));
        }
        float alpha[2], pr[4], psum[2];
#pragma unroll
        for (int c2 = 0; c2 < 2; ++c2) {
            const float m_new = fmaxf(m_run[c2], tmax[c2]);  // finite: the tile holds at least one valid position
            alpha[c2] = exp2f(m_run[c2] - m_new);
            pr[c2] = exp2f(sc[c2] - m_new);
            pr[2 + c2] = exp2f(sc[2 + c2] - m_new);
            psum[c2] = pr[c2] + pr[2 + c2];
            m_run[c2] = m_new;
        }
#pragma unroll
        for (int sh = 4; sh <= 16; sh <<= 1) {
            psum[0] += __shfl_xor_sync(0xffffffffu, psum[0], sh);
            psum[1] += __shfl_xor_sync(0xffffffffu, psum[1], sh);
        }
        l_run[0] = l_run[0] * alpha[0] + psum[0];
        l_run[1] = l_run[1] * alpha[1] + psum[1];

        // ---- P into B-operand layout: lane (g4, q4) needs head g4, positions 2 q4, 2 q4 + 1, 2 q4 + 8, 2 q4 + 9
        uint32_t pb[2];
        {
            const int src_a = ((2 * q4) << 2) | (g4 >> 1), src_b = ((2 * q4 + 1) << 2) | (g4 >> 1);
            const bool odd = g4 & 1;
            const float a0 = __shfl_sync(0xffffffffu, pr[0], src_a), a1 = __shfl_sync(0xffffffffu, pr[1], src_a);
            const float a2 = __shfl_sync(0xffffffffu, pr[2], src_a), a3 = __shfl_sync(0xffffffffu, pr[3], src_a);
            const float b0 = __shfl_sync(0xffffffffu, pr[0], src_b), b1 = __shfl_sync(0xffffffffu, pr[1], src_b);
            const float b2 = __shfl_sync(0xffffffffu, pr[2], src_b), b3 = __shfl_sync(0xffffffffu, pr[3], src_b);
            pb[0] = pack_bf16x2(odd ? a1 : a0, odd ? b1 : b0);  // positions 2 q4, 2 q4 + 1
            pb[1] = pack_bf16x2(odd ? a3 : a2, odd ? b3 : b2);  // positions 2 q4 + 8, 2 q4 + 9
            if (g4 >= R) pb[0] = pb[1] = 0u;
        }

        // ---- O^T = O^T * alpha + V^T . P
#pragma unroll
        for (int dt = 0; dt < D / 16; ++dt) {
            uint32_t a[4];
            const int c = dt * 2 + v_cadd;
            ldmatrix_x4_trans(a, vt + (uint32_t)(v_row * kRowBytes + (((c & ~7) | ((c ^ v_row) & 7)) << 4)));
            o[dt][0] *= alpha[0];
            o[dt][1] *= alpha[1];
            o[dt][2] *= alpha[0];
            o[dt][3] *= alpha[1];
            mma_bf16_16816(o[dt], a[0], a[1], a[2], a[3], pb[0], pb[1], o[dt]);
        }
    }
    cp_async_wait<0>();
    __syncthreads();  // every warp is done with its ring: the shared memory is reused for the merge

    // ---- merge the four warps' states and write this CTA's partial: part[warp][head][d] + stats[warp][head][2]
    float* part = reinterpret_cast<float*>(smem);
    float* stats = part + kKvWarps * kKvMaxGroup * D;
    if (g4 == 0) {  // lanes 0..3 hold the stats of heads 2 q4, 2 q4 + 1
        stats[(warp * kKvMaxGroup + 2 * q4) * 2] = m_run[0];
        stats[(warp * kKvMaxGroup + 2 * q4) * 2 + 1] = l_run[0];
        stats[(warp * kKvMaxGroup + 2 * q4 + 1) * 2] = m_run[1];
        stats[(warp * kKvMaxGroup + 2 * q4 + 1) * 2 + 1] = l_run[1];
    }
#pragma unroll
    for (int dt = 0; dt < D / 16; ++dt) {
        float* base = part + (size_t)(warp * kKvMaxGroup + 2 * q4) * D + dt * 16;
        base[g4] = o[dt][0];
        base[D + g4] = o[dt][1];
        base[g4 + 8] = o[dt][2];
        base[D + g4 + 8] = o[dt][3];
    }
    __syncthreads();
    // this CTA's partial: to the workspace, or (one-launch variant) to shared memory behind the warps' partials
    float* cl_o = stats + kKvWarps * kKvMaxGroup * 2;  // [R][D]
    float* cl_st = cl_o + kKvMaxGroup * D;             // [R][2]: running maximum, running sum
    for (int idx = tid; idx < R * D; idx += kKvWarps * 32) {
        const int h = idx / D, i = idx % D;
        float m = -INFINITY;
#pragma unroll
        for (int w = 0; w < kKvWarps; ++w) m = fmaxf(m, stats[(w * kKvMaxGroup + h) * 2]);
        float acc = 0.f, l = 0.f;
#pragma unroll
        for (int w = 0; w < kKvWarps; ++w) {
            const float mw = stats[(w * kKvMaxGroup + h) * 2];
            const float f = mw == -INFINITY ? 0.f : exp2f(mw - m);
            acc += part[(size_t)(w * kKvMaxGroup + h) * D + i] * f;
            l += stats[(w * kKvMaxGroup + h) * 2 + 1] * f;
        }
        if (CLUSTER) {
            cl_o[idx] = acc;
            if (i == 0) {
                cl_st[h * 2] = m;
                cl_st[h * 2 + 1] = l;
            }
        } else {
            float* dst = p.ws + ((size_t)(kvh * R + h) * p.splits + split) * (D + 4);
            dst[i] = acc;
            if (i == 0) {
                dst[D] = m;
                dst[D + 1] = l;
            }
        }
    }
    if (CLUSTER) {
        // every CTA of the cluster has its partial in place; CTA `split` combines outputs split, split + S, ... of the
        // head group (a thread per output) over all S partials in split order and normalises
        cluster_sync();
        const int S = p.splits;
        const uint32_t o_addr = smem_u32(cl_o), st_addr = smem_u32(cl_st);
        for (int idx = split * (kKvWarps * 32) + tid; idx < R * D; idx += S * (kKvWarps * 32)) {
            const int h = idx / D;
            float ms[kKvMaxCluster], ls[kKvMaxCluster], os[kKvMaxCluster];
            float m = -INFINITY;
#pragma unroll
            for (int s2 = 0; s2 < kKvMaxCluster; ++s2) {
                const bool on = s2 < S;
                ms[s2] = on ? ld_cluster_f32(st_addr + (uint32_t)(h * 8), (uint32_t)s2) : -INFINITY;
                ls[s2] = on ? ld_cluster_f32(st_addr + (uint32_t)(h * 8 + 4), (uint32_t)s2) : 0.f;
                os[s2] = on ? ld_cluster_f32(o_addr + (uint32_t)idx * 4u, (uint32_t)s2) : 0.f;
                m = fmaxf(m, ms[s2]);
            }
            float acc = 0.f, l = 0.f;
#pragma unroll
            for (int s2 = 0; s2 < kKvMaxCluster; ++s2) {
                const float f = ms[s2] == -INFINITY ? 0.f : exp2f(ms[s2] - m);
                acc += os[s2] * f;
                l += ls[s2] * f;
            }
            p.out[(size_t)kvh * R * D + idx] = acc / l;
        }
        cluster_sync();  // nobody leaves while its shared memory may still be read
    }
}

// out[h][i] = sum_s O_s[i] 2^(m_s - m*) / sum_s l_s 2^(m_s - m*) in a fixed order; one block per query head.
template <int D>
__global__ void __launch_bounds__(kKvMergeThreads) flowkv_merge_kernel(const float* __restrict__ ws, float* __restrict__ out, int splits) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int h = blockIdx.x, i = threadIdx.x;
    const float* base = ws + (size_t)h * splits * (D + 4);
    __shared__ float factor[kKvMaxSplitsDev];  // 2^(m_s - m*) per split
    __shared__ float l_total;
    constexpr int kCols = D / 4, kParts = kKvMergeThreads / kCols;
    __shared__ float4 partial[kParts][kCols];
    if (i < 32) {  // warp 0: the splits' statistics, a few per lane, all loads independent
        constexpr int kPer = kKvMaxSplitsDev / 32;
        float ms[kPer], ls[kPer];
        float m = -INFINITY;
#pragma unroll
        for (int k = 0; k < kPer; ++k) {
            const int s = i + 32 * k;
            ms[k] = s < splits ? base[(size_t)s * (D + 4) + D] : -INFINITY;
            ls[k] = s < splits ? base[(size_t)s * (D + 4) + D + 1] : 0.f;
            m = fmaxf(m, ms[k]);
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        float l = 0.f;
#pragma unroll
        for (int k = 0; k < kPer; ++k) {
            const int s = i + 32 * k;
            const float f = ms[k] == -INFINITY ? 0.f : exp2f(ms[k] - m);
            if (s < splits) factor[s] = f;
            l += ls[k] * f;
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
        if (i == 0) l_total = l;
    }
    __syncthreads();
    // the sum over splits: four columns per thread, the splits dealt round-robin to kParts thread groups (all of a
    // thread's loads are independent), then the groups' sums added in group order
    const int c = i % kCols, part = i / kCols;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int s = part; s < splits; s += kParts) {
        const float4 v = *reinterpret_cast<const float4*>(base + (size_t)s * (D + 4) + 4 * c);
        const float f = factor[s];
        acc.x += v.x * f;
        acc.y += v.y * f;
        acc.z += v.z * f;
        acc.w += v.w * f;
    }
    partial[part][c] = acc;
    __syncthreads();
    if (i < kCols) {
        float4 t = partial[0][i];
#pragma unroll
        for (int q = 1; q < kParts; ++q) {
            const float4 v = partial[q][i];
            t.x += v.x;
            t.y += v.y;
            t.z += v.z;
            t.w += v.w;
        }
        const float l = l_total;
        *reinterpret_cast<float4*>(out + (size_t)h * D + 4 * i) = make_float4(t.x / l, t.y / l, t.z / l, t.w / l);
    }
}

// ---- host side ------------------------------------------------------------------------------------------------------

template <int D>
constexpr int flowkv_smem_bytes() {
    constexpr int kRing = kKvWarps * kKvStages * 2 * kKvTile * D * 2;
    constexpr int kMerge = (kKvWarps * kKvMaxGroup * D + kKvWarps * kKvMaxGroup * 2 + kKvMaxGroup * D + kKvMaxGroup * 2) * 4;
    return kRing > kMerge ? kRing : kMerge;
}

template <int D>
static cudaError_t flowkv_launch_d(const FlowKvParams& p, float* out, cudaStream_t stream) {
    constexpr int kSmem = flowkv_smem_bytes<D>();
    static bool attr_set = false;  // per process; the attribute is per device function
    cudaError_t e;
    if (!attr_set) {
        if ((e = cudaFuncSetAttribute(flowkv_decode_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem))) return e;
        attr_set = true;
    }
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.splits, (unsigned)p.G);
    cfg.blockDim = dim3(kKvWarps * 32);
    cfg.dynamicSmemBytes = kSmem;
    cfg.stream = stream;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if ((e = cudaLaunchKernelEx(&cfg, flowkv_decode_kernel<D, false>, p))) return e;
    cfg.gridDim = dim3((unsigned)p.H);
    cfg.blockDim = dim3(kKvMergeThreads);
    cfg.dynamicSmemBytes = 0;
    const float* ws = p.ws;
    const int splits = p.splits;
    return cudaLaunchKernelEx(&cfg, flowkv_merge_kernel<D>, ws, out, splits);
}

// The one-launch variant: grid (S, G) in clusters of S CTAs.  `*usable` is set to the number of such clusters the
// device can hold at once (0: this cluster size cannot be launched here; the caller then takes the two-launch route).
template <int D>
static cudaError_t flowkv_cluster_config(int S, cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attrs) {
    constexpr int kSmem = flowkv_smem_bytes<D>();
    static bool attr_set = false;
    cudaError_t e;
    if (!attr_set) {
        if ((e = cudaFuncSetAttribute(flowkv_decode_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem))) return e;
        if ((e = cudaFuncSetAttribute(flowkv_decode_kernel<D, true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1))) return e;
        attr_set = true;
    }
    attrs[0].id = cudaLaunchAttributeClusterDimension;
    attrs[0].val.clusterDim.x = (unsigned)S;
    attrs[0].val.clusterDim.y = 1;
    attrs[0].val.clusterDim.z = 1;
    attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[1].val.programmaticStreamSerializationAllowed = 1;
    *cfg = cudaLaunchConfig_t{};
    cfg->blockDim = dim3(kKvWarps * 32);
    cfg->dynamicSmemBytes = kSmem;
    cfg->attrs = attrs;
    cfg->numAttrs = 2;
    return cudaSuccess;
}

template <int D>
static cudaError_t flowkv_cluster_usable(int S, int G, int* usable) {
    static int cached[kKvMaxCluster + 1];  // 0: not asked yet; else 1 + the number of co-resident clusters
    if (!cached[S]) {
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attrs[2];
        cudaError_t e = flowkv_cluster_config<D>(S, &cfg, attrs);
        if (e) return e;
        cfg.gridDim = dim3((unsigned)S, (unsigned)G);
        cfg.numAttrs = 1;  // the cluster shape alone
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, flowkv_decode_kernel<D, true>, &cfg);
        if (e) {
            (void)cudaGetLastError();
            n = 0;
        }
        cached[S] = 1 + n;
    }
    *usable = cached[S] - 1;
    return cudaSuccess;
}

template <int D>
static cudaError_t flowkv_launch_cluster_d(const FlowKvParams& p, cudaStream_t stream) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attrs[2];
    cudaError_t e = flowkv_cluster_config<D>(p.splits, &cfg, attrs);
    if (e) return e;
    cfg.gridDim = dim3((unsigned)p.splits, (unsigned)p.G);
    cfg.stream = stream;
    return cudaLaunchKernelEx(&cfg, flowkv_decode_kernel<D, true>, p);
}

// ws must hold H * max_splits * (d + 4) floats; max_splits <= kKvMaxSplitsDev.
cudaError_t flowkv_launch(const uint16_t* q, const uint16_t* K, const uint16_t* V, float* out, float* ws, int max_splits, int H,
                          int G, int d, int L, int pitch, int window, float scale, int sm_count, int cluster_max_positions,
                          int* launches, cudaStream_t stream) {
    if (d != 128 && d != 256) return cudaErrorInvalidValue;
    FlowKvParams p;
    p.q = q;
    p.K = K;
    p.V = V;
    p.ws = ws;
    p.out = out;
    p.H = H;
    p.G = G;
    p.L = L;
    p.pitch = pitch;
    p.j0 = (window > 0 && window < L) ? L - window : 0;
    const int n = L - p.j0;
    const int gran = kKvWarps * kKvTile;
    p.scale_log2e = scale * 1.4426950408889634f;
    if (n <= cluster_max_positions) {
        // one launch: S splits (a power of two, at most 16) of equal length, one cluster per KV head
        int S = 1;
        while (S < kKvMaxCluster && S * gran < n) S *= 2;
        int usable = 0;
        cudaError_t e = d == 256 ? flowkv_cluster_usable<256>(S, G, &usable) : flowkv_cluster_usable<128>(S, G, &usable);
        if (e) return e;
        if (usable >= 1) {
            p.splits = S;
            p.chunk = ((n + S - 1) / S + gran - 1) / gran * gran;
            *launches = 1;
            return d == 256 ? flowkv_launch_cluster_d<256>(p, stream) : flowkv_launch_cluster_d<128>(p, stream);
        }
    }
    // CTAs over all KV heads: as many as are resident at once (one per SM at d = 256, whose rings take 192 KB; two at
    // d = 128), never more -- a CTA that has to wait for a free SM would double the time.
    const int resident = sm_count * (d == 128 ? 2 : 1);
    int want = resident / G;
    if (want > max_splits) want = max_splits;
    if (want < 1) want = 1;
    int chunk = ((n + want - 1) / want + gran - 1) / gran * gran;
    p.chunk = chunk;
    p.splits = (n + chunk - 1) / chunk;
    if (p.splits > kKvMaxSplitsDev) return cudaErrorInvalidValue;
    *launches = 2;
    if (d == 256) return flowkv_launch_d<256>(p, out, stream);
    return flowkv_launch_d<128>(p, out, stream);
}

}  // namespace fdqp
