// A chain of FusedDQP projections in ONE persistent launch (M = 1 .. 8 tokens).
//
// The paper keeps every kernel of a decoder layer resident on its tile array and pipelines them: the projections
// stream their Q4NX blocks while the vector kernels between them run, and the intermediate vectors never leave the
// chip (Sec. "Mapping Gemma3 decoding"; Sec. "FusedDQP": the activation vector is broadcast while every tile streams
// its own blocks).  On this GPU the same idea is one grid of persistent CTAs, one per SM, that walks a LIST of
// projections (Eq. 14 / 15 with Eq. 3 fused, exactly as the single-call kernel computes them):
//   * the producer warp of a CTA runs through the block ranges of all steps without pause, so the shared-memory ring
//     already holds the first stages of step i + 1 while the consumers finish step i -- launch latency, barrier
//     set-up and the first trip to HBM are paid once per chain instead of once per projection;
//   * a step whose input is the previous step's output (the down projection after gate|up with its gated-GELU
//     epilogue; a projection after the normalised sum of the residual stream) waits -- bounded, like every wait in
//     this library -- until a counter in global memory says that all strips of that step have been stored; steps
//     with independent inputs wait for nothing;
//   * strips shared between CTAs and K slices are finished by whichever piece arrives last at the strip's ticket
//     (fixed summation order: results are reproducible run to run); no CTA waits for another CTA to do that.
// All CTAs of the grid are resident at once (one per SM, grid <= SM count), which is what makes the dependency
// wait safe; the last CTA to leave puts the counters back to zero for the next launch.
#include "fdqp_gemv_tile.cuh"

namespace fdqp {

namespace {

constexpr int kCW = 16;                 // consumer warps
constexpr int kNR = 2;                  // reducer warps
constexpr int kThreads = (kCW + 1 + kNR) * 32;
constexpr uint32_t kBB = kBlockBytes;
constexpr int kPrepBatch = 8;           // activations items (8 values each) a consumer thread prepares per step, at most

// The part of a step one CTA works on (same arithmetic in every warp role).
struct StepGeom {
    int z, b_first, len, nblk, bl_first, npieces, nt, bl_tail, nchunk;
    int64_t ci, a, e, s_first, s_last;
    int64_t a_true;  // where the CTA's range really begins in this slice's numbering (negative: in an earlier slice or step)
};

__device__ __forceinline__ int chain_slice_len(const ChainStep& st, int z) {
    const int rest = st.nb - z * st.nbz;
    return rest < st.nbz ? rest : st.nbz;
}

// Blocks of slice z of a step that CTA `cta` works on.  Two ways of cutting a chain into CTA ranges:
//   per step (cp.wide == 0): every slice of every step is cut into equal ranges over its own Gz CTAs, so that all CTAs
//     work on the same step at the same time -- what a step that waits for the previous one needs;
//   chain-wide (cp.wide != 0, only when no step waits for another): the blocks of all steps and slices are laid end
//     to end and cut into `grid` equal ranges, so that a CTA streams ONE contiguous share of the whole chain: it
//     prepares activations only for the steps it touches and shares at most two strips with its neighbours.
// (The divisions are done ONCE per CTA and unit, by one thread each, into a table in shared memory: unit_range; every
// warp role then derives what it needs from the table entry with multiplications only: unit_geom.)
__device__ __forceinline__ int4 unit_range(const ChainPlan& cp, const ChainStep& st, int z, int cta) {
    const int len = chain_slice_len(st, z);
    const int64_t T = (int64_t)st.S * len;
    int64_t a, e, a_true;
    if (cp.wide) {
        const int64_t B = (int64_t)st.B + (int64_t)z * st.S * st.nbz;  // slices before z are all nbz long
        const int64_t A = range_begin(cta, gridDim.x, cp.Wtot) - B, E = range_begin(cta + 1, gridDim.x, cp.Wtot) - B;
        a = A < 0 ? 0 : (A > T ? T : A);
        e = E < 0 ? 0 : (E > T ? T : E);
        a_true = A < -1 ? -1 : A;  // only "before this slice or not" matters (see chain_piece_slot)
    } else {
        if (cta / st.Gz != z) return make_int4(0, 0, 0, 0);  // another slice's CTA (or one this step cannot use)
        const int ci = cta % st.Gz;
        a = st.strip_aligned ? range_begin(ci, st.Gz, st.S) * len : range_begin(ci, st.Gz, T);
        e = st.strip_aligned ? range_begin(ci + 1, st.Gz, st.S) * len : range_begin(ci + 1, st.Gz, T);
        a_true = a;
    }
    if (e <= a) return make_int4(0, 0, 0, 0);
    // strips of the first and the last block; the sign of .z tells whether the range began before this slice
    const int s_first = (int)(a / len), s_last = (int)((e - 1) / len);
    return make_int4((int)a, (int)e, a_true < 0 ? -1 - s_first : s_first, s_last);
}

__device__ __forceinline__ StepGeom unit_geom(const ChainPlan& cp, const ChainStep& st, int z, int cta, int kCB, int4 t) {
    StepGeom g;
    g.z = z;
    g.ci = cp.wide ? cta : cta % st.Gz;
    g.b_first = z * st.nbz;
    g.len = chain_slice_len(st, z);
    g.a = t.x;
    g.e = t.y;
    g.nblk = t.y - t.x;
    g.bl_first = g.npieces = g.nt = g.bl_tail = g.nchunk = 0;
    g.s_first = g.s_last = 0;
    g.a_true = g.a;
    if (g.nblk <= 0) {
        g.nblk = 0;
        return g;
    }
    g.s_first = t.z < 0 ? -1 - t.z : t.z;
    g.s_last = t.w;
    if (t.z < 0) g.a_true = -1;
    g.bl_first = (int)(g.a - g.s_first * g.len);
    g.npieces = (int)(g.s_last - g.s_first) + 1;
    // processing order: the blocks of a partial last strip come first, then the rest of the range in order
    const int64_t tail_begin = g.s_last * g.len > g.a ? g.s_last * g.len : g.a;
    g.nt = (g.npieces >= 2 && g.e < (g.s_last + 1) * g.len) ? (int)(g.e - tail_begin) : 0;
    g.bl_tail = (int)(tail_begin - g.s_last * g.len);
    g.nchunk = (g.nblk + kCB - 1) / kCB;
    return g;
}

// First and last CTA that hold blocks of strip s in slice zz of a step, and where CTA c's range begins (in the
// slice's own block numbering, possibly negative in the chain-wide cut).
__device__ __forceinline__ void strip_ctas(const ChainPlan& cp, const ChainStep& st, int zz, int64_t s, int64_t* cf, int64_t* cl) {
    const int l2 = chain_slice_len(st, zz);
    const int64_t u0 = s * l2;
    if (cp.wide) {
        const int64_t B = (int64_t)st.B + (int64_t)zz * st.S * st.nbz;
        *cf = cta_of(B + u0, gridDim.x, cp.Wtot);
        *cl = cta_of(B + u0 + l2 - 1, gridDim.x, cp.Wtot);
    } else if (st.strip_aligned) {
        *cf = *cl = 0;
    } else {
        const int64_t T2 = (int64_t)st.S * l2;
        *cf = cta_of(u0, st.Gz, T2);
        *cl = cta_of(u0 + l2 - 1, st.Gz, T2);
    }
}
__device__ __forceinline__ int64_t cta_range_begin(const ChainPlan& cp, const ChainStep& st, int zz, int64_t c) {
    const int l2 = chain_slice_len(st, zz);
    if (cp.wide) return range_begin(c, gridDim.x, cp.Wtot) - ((int64_t)st.B + (int64_t)zz * st.S * st.nbz);
    return range_begin(c, st.Gz, (int64_t)st.S * l2);
}

// Partial-sum slot of a CTA's piece of strip s in slice z (writer and reader use the same rule).  ci: the CTA's index
// inside the slice (per-step cut) or in the grid (chain-wide cut, where a CTA has at most two partial pieces in the
// whole chain: the strip its range begins in and the strip it ends in).
__device__ __forceinline__ float* chain_piece_slot(const ChainPlan& cp, const ChainStep& st, int z, int64_t ci, int64_t s,
                                                   int64_t unit_begin, bool whole_unit, int64_t cta_begin) {
    if (whole_unit) return cp.ws_full + ((int64_t)st.full_off + (int64_t)z * st.S + s) * (kStripRows * kMaxTokens);
    const int which = (cta_begin >= unit_begin) ? 0 : 1;  // piece holds the CTA's first block, or its last
    const int64_t slot = cp.wide ? ci * 2 + which : (int64_t)st.edge_off + ((int64_t)z * st.Gz + ci) * 2 + which;
    return cp.ws_edge + slot * (kStripRows * kMaxTokens);
}

__device__ __forceinline__ uint4 ldcg128(const void* p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Bounded wait until *counter >= target (acquire).  false after the time limit, with the timeout recorded.
__device__ __forceinline__ bool wait_counter(const int* counter, int target, int* status) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= target) return true;
    const unsigned long long t0 = globaltimer_ns();
    for (uint32_t it = 1;; ++it) {
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
        if (v >= target) return true;
        if ((it & 63u) == 0u && globaltimer_ns() - t0 > kWaitLimitNs) {
            atomicExch(status, kStatusTimeout);
            __threadfence_system();
            return false;
        }
        __nanosleep(64);  // one poller per CTA, all on one address: leave the line to the CTAs that still count
    }
}

}  // namespace

// MODE as in the single-call kernel (1: M = 1, 3: M = 2, 2: M = 3 .. 8); BPW: blocks per consumer warp and ring stage
// (2 or 4); EPI: built with the bf16 epilogues and the fused RMS normalisation.  Q4NX only; 16 consumer warps, a
// producer warp, two reducer warps.
template <int MODE, int BPW, bool EPI>
__global__ void __launch_bounds__(kThreads, 1) fdqp_chain_kernel(const __grid_constant__ ChainPlan cp) {
    extern __shared__ __align__(128) uint8_t smem[];
    using MT = ModeTraits<MODE>;
    constexpr int NT = MT::kAcc;
    constexpr int FMT = kFmtQ4nx;
    constexpr int kBPW = BPW;
    constexpr int kCB = (kCW / 8) * kBPW;   // blocks per ring stage
    constexpr uint32_t kStageBytes = kCB * kBB;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int M = MODE == 1 ? 1 : (MODE == 3 ? 2 : cp.M);
    const int nstage = cp.nstage;

    const uint32_t ring = smem_u32(smem);
    const uint32_t xs = ring + cp.off_xs, xsc = ring + cp.off_xsum;
    const uint32_t part = ring + cp.off_part, bars = ring + cp.off_bar;
    const uint32_t full0 = bars, empty0 = bars + 8u * nstage;
    const uint32_t red_full0 = bars + 16u * nstage, red_empty0 = red_full0 + 16u;
    // fused RMS normalisation: one sum of squares per (group-tile, token), then one factor per token
    float* const norm_q = reinterpret_cast<float*>(smem + cp.off_norm);
    float* const norm_r = norm_q + kPrepBatch * kCW * 32 / 4;

    for (int s = tid; s < nstage; s += blockDim.x) {
        mbar_init(full0 + 8u * s, 1);
        mbar_init(empty0 + 8u * s, kCW);
    }
    if (tid < 2) {
        mbar_init(red_full0 + 8u * tid, kCW);
        mbar_init(red_empty0 + 8u * tid, 1);
    }
    // this CTA's block range in every (step, K slice) unit: one thread per unit does the divisions
    int4* const geo = reinterpret_cast<int4*>(smem + cp.off_geo);
    for (int ui = tid; ui < cp.nunits; ui += blockDim.x) geo[ui] = unit_range(cp, cp.step[cp.unit_step[ui]], cp.unit_slice[ui], blockIdx.x);
    mbar_fence_init();
    __syncthreads();
    // The next launch in the stream may begin as soon as SM slots free up: it streams weights (which nothing in this
    // library writes) and waits for this grid to complete before it touches activations, outputs or workspace.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == kCW) {
        // =============================== producer ================================================
        // One pass over the block ranges of all steps; lane j < kCB copies block j of every stage.
        const uint64_t policy = l2_policy_evict_first();
        int stage = 0, issued = 0;
        uint32_t phase = 0;
        bool alive = true;
        for (int ui = 0; ui < cp.nunits && alive; ++ui) {
            const int4 gt = geo[ui];
            if (gt.y <= gt.x) continue;  // nothing of this unit for this CTA
            const int si = cp.unit_step[ui], uz = cp.unit_slice[ui];
            const ChainStep& st = cp.step[si];
            const StepGeom g = unit_geom(cp, st, uz, blockIdx.x, kCB, gt);
            const int groups_total = st.K / kGroup;
            const int64_t strip_bytes = (int64_t)kGroupBytes * groups_total;
            for (int c = 0; c < g.nchunk; ++c) {
                if (issued >= nstage) {
                    int ok = 1;
                    if (lane == 0) ok = mbar_wait(empty0 + 8u * stage, phase ^ 1u, cp.status) ? 1 : 0;
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { alive = false; break; }
                }
                const int i = c * kCB + lane;  // position in processing order
                uint32_t bytes = 0;
                int64_t ps = 0;
                int pbl = 0;
                if (lane < kCB && i < g.nblk) {
                    // block i of the processing order -> (strip, block inside the slice)
                    const uint32_t rel = (uint32_t)g.bl_first + (uint32_t)(i < g.nt ? (g.nblk - g.nt + i) : (i - g.nt));
                    const uint32_t so = rel / (uint32_t)g.len;
                    ps = g.s_first + so;
                    pbl = (int)(rel - so * (uint32_t)g.len);
                    const int rest = groups_total - 8 * (g.b_first + pbl);
                    bytes = (uint32_t)kGroupBytes * (uint32_t)(rest < 8 ? rest : 8);
                }
                const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
                if (lane == 0) mbar_arrive_expect_tx(full0 + 8u * stage, total);
                __syncwarp();
                // Blocks that follow each other in the container AND in the stage go out as ONE copy (strips follow each other
                // in memory, so that is usually the whole stage): the memory system serves 20-40 KB copies faster than 5 KB ones
                // (bare read stream: 7.28 against 6.93 TB/s).  A run ends after a short block (its slot in the stage is not filled).
                const uint8_t* src = st.W + ps * strip_bytes + (int64_t)(g.b_first + pbl) * kBB;
                const uint64_t src_prev = __shfl_up_sync(0xffffffffu, (uint64_t)(uintptr_t)src, 1);
                const uint32_t bytes_prev = __shfl_up_sync(0xffffffffu, bytes, 1);
                const bool first_of_run = bytes != 0 && (lane == 0 || bytes_prev != kBB || (uint64_t)(uintptr_t)src != src_prev + kBB);
                const uint32_t firsts = __ballot_sync(0xffffffffu, first_of_run), filled = __ballot_sync(0xffffffffu, bytes != 0);
                const uint32_t later = firsts & ~((2u << lane) - 1u);                       // runs that begin after this lane
                const int run_end = later ? __ffs(later) - 1 : 32 - __clz(filled | 1u);    // one past the run's last lane
                const uint32_t bytes_last = __shfl_sync(0xffffffffu, bytes, (run_end - 1) & 31);
                if (first_of_run) {
                    const uint32_t run_bytes = (uint32_t)(run_end - 1 - lane) * kBB + bytes_last;
                    const uint32_t dst = ring + stage * kStageBytes + lane * kBB;
                    if (cp.evict_first)
                        bulk_g2s_hint(dst, src, run_bytes, full0 + 8u * stage, policy);
                    else
                        bulk_g2s(dst, src, run_bytes, full0 + 8u * stage);
                }
                if (++stage == nstage) { stage = 0; phase ^= 1u; }
                ++issued;
            }
        }
        // Do not leave while a copy into this CTA's shared memory may still be in flight.
        if (lane == 0) {
            const int from = issued > nstage ? issued - nstage : 0;
            for (int k = from; k < issued; ++k)
                if (!mbar_wait(full0 + 8u * (k % nstage), (k / nstage) & 1, cp.status)) break;
        }
    } else if (warp < kCW) {
        // =============================== consumers ===============================================
        const int tw = warp & 7, j0 = (warp >> 3) * kBPW;
        const int g8 = lane >> 2, q = lane & 3;
        LaneAddr la;
        LaneConst lc{};
        la.xs = xs;
        la.x_stride = (uint32_t)M * (uint32_t)(MT::kCols ? kColsRecBytes : kPlaneRecBytes);
        {
            const int gtok = g8 < M ? g8 : M - 1;
            la.x_lane = xs + (uint32_t)(gtok * 4 + q) * 16u;
            la.xsc_lane = xsc + q * 8;
            const int tok_b = g8 >> 2, pl = g8 & 3;
            la.xb_off = tok_b < M ? (uint32_t)(tok_b * kColsRecBytes + pl * 32 + q * 8) : 0u;  // (no such token: weight 0 below)
            const int tok_d = q >> 1;
            la.sc_off = (uint32_t)((tok_d < M ? tok_d : 0) * kColsRecBytes + kColsSumOff);
            lc.w_unit = tok_d < M ? ((q & 1) ? 1.f : 65536.f) : 0.f;
            asm volatile("mov.b32 %0, 0x000F000F;" : "=r"(lc.nib_mask));
            asm volatile("mov.b32 %0, 0x43004300;" : "=r"(lc.nib_magic));
        }
        // ldmatrix source rows (see the single-call kernel): codes = row `lane` of the tile; scales / offsets = the
        // 16-byte chunks of the tile's scale and offset words
        const uint32_t code_lane = tw * 512 + lane * 16;
        const int mat = lane >> 3;
        const uint32_t so_chunk = tw * 64 + (((mat & 1) * 2 + (lane & 1)) * 16);
        const uint32_t so_sect = (!MT::kCols && mat >= 2) ? 576u : 512u;
        const uint32_t m_lane = tw * 64 + lane * 2;
        const uint32_t so_full = ((!MT::kCols && mat >= 2) ? 4608u : (uint32_t)kCodeBytes) + so_chunk;
        const uint32_t m_full = 4608u + m_lane;

        float acc_m[MT::kAccM];
#pragma unroll
        for (int tk = 0; tk < MT::kAccM; ++tk) acc_m[tk] = 0.f;
        float acc[4][NT];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < NT; ++j) acc[i][j] = 0.f;

        int stage = 0;
        uint32_t phase = 0;
        int pieceG = 0;  // pieces handed to the reducers so far, over all steps (selects the hand-over buffer)
        bool alive = true;

        // Everything up to here touched only this CTA's shared memory.  x may come from the previous launch.
        asm volatile("griddepcontrol.wait;" ::: "memory");

        for (int ui = 0; ui < cp.nunits; ++ui) {
            const int4 gt = geo[ui];
            if (gt.y <= gt.x) continue;  // nothing of this unit for this CTA
            const int si = cp.unit_step[ui], uz = cp.unit_slice[ui];
            const ChainStep& st = cp.step[si];
            const StepGeom g = unit_geom(cp, st, uz, blockIdx.x, kCB, gt);  // (the same answer in every warp of the CTA)
            const int K = st.K;
            const int groups_total = K / kGroup;
            const int64_t strip_bytes = (int64_t)kGroupBytes * groups_total;
            // The step's input may be the previous step's output: wait until every strip of that step is stored.
            if (st.wait_prev && warp == 0 && lane == 0) wait_counter(cp.done + (si - 1), cp.step[si - 1].S, cp.status);
            // Every consumer warp has finished the tiles of the unit before: its activations may be overwritten.
            asm volatile("bar.sync 1, %0;" ::"n"(kCW * 32) : "memory");

            // ---- this CTA's K slice of x, prepared straight into shared memory ----
            bool saw_flagged = false;
            {
                const int kbeg = g.b_first * kBlockK;
                const int kend_full = (g.b_first + g.len) * kBlockK;
                const int ntiles_all = ((kend_full < K ? kend_full : K) - kbeg) / kGroup;
                // A range inside one strip, or in the end of one strip and the beginning of the next, touches only its own
                // blocks' share of x (a long-K projection cut over many CTAs): up to two tile ranges [lo1, hi1), [lo2, hi2).
                // The normalisation needs the whole row.
                int lo1 = 0, hi1 = ntiles_all, lo2 = 0, hi2 = 0;
                if (!(EPI && st.norm)) {
                    if (g.npieces == 1) {
                        lo1 = g.bl_first * 8;
                        hi1 = (g.bl_first + g.nblk) * 8;
                    } else if (g.npieces == 2 && g.nblk - (g.len - g.bl_first) <= g.bl_first) {
                        hi1 = (g.nblk - (g.len - g.bl_first)) * 8;  // the second strip's first blocks
                        lo2 = g.bl_first * 8;                        // the first strip's last blocks
                        hi2 = g.len * 8;
                    }
                    hi1 = hi1 < ntiles_all ? hi1 : ntiles_all;
                    hi2 = hi2 < ntiles_all ? hi2 : ntiles_all;
                    if (hi2 < lo2) hi2 = lo2;
                }
                const int n1 = hi1 - lo1, ntiles = n1 + (hi2 - lo2);
                // tile (relative to the K slice) of the t-th tile prepared
                auto tile_rel = [&](int t) { return t < n1 ? lo1 + t : lo2 + (t - n1); };
                const int tile0 = kbeg / kGroup;
                const int items = ntiles * M * 4;  // <= kPrepBatch * kCW * 32 (the plan guarantees it)
                uint32_t* xs_g = reinterpret_cast<uint32_t*>(smem + cp.off_xs);
                float* xsc_g = reinterpret_cast<float*>(smem + cp.off_xsum);
                uint4 v[kPrepBatch];
#pragma unroll
                for (int u = 0; u < kPrepBatch; ++u) {
                    const int idx = u * kCW * 32 + tid;
                    v[u] = make_uint4(0, 0, 0, 0);
                    if (idx < items) {
                        const int tm = idx >> 2, tile = tile0 + tile_rel(tm / M), tok = tm % M, qq = idx & 3;
                        v[u] = ldcg128(st.x + (int64_t)tok * K + tile * kGroup + qq * 8);
                    }
                }
                if (EPI && st.norm) {
                    // RMS normalisation (the whole row is in this CTA: the plan gives such a step one K slice).
                    // Pass 1: optional residual addition, sum of squares per (tile, token).
#pragma unroll
                    for (int u = 0; u < kPrepBatch; ++u) {
                        const int idx = u * kCW * 32 + tid;
                        if (u * kCW * 32 < items) {  // warp-uniform
                            const bool valid = idx < items;
                            const int tm = idx >> 2, tile = tile0 + (valid ? tm / M : 0), tok = valid ? tm % M : 0, qq = idx & 3;
                            if (st.residual && valid) {
                                v[u] = add_bf16x8(v[u], ldcg128(st.residual + (int64_t)tok * K + tile * kGroup + qq * 8));
                                if (st.h_out && blockIdx.x == 0)
                                    *reinterpret_cast<uint4*>(st.h_out + (int64_t)tok * K + tile * kGroup + qq * 8) = v[u];
                            }
                            const uint32_t xw[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                            float ss = 0.f;
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float f0 = __uint_as_float(xw[i] << 16), f1 = __uint_as_float(xw[i] & 0xffff0000u);
                                ss = fmaf(f0, f0, ss);
                                ss = fmaf(f1, f1, ss);
                            }
                            ss += __shfl_xor_sync(0xffffffffu, ss, 1);
                            ss += __shfl_xor_sync(0xffffffffu, ss, 2);
                            if (valid && qq == 0) norm_q[tm] = ss;  // tm = (tile - tile0) * M + tok
                        }
                    }
                    asm volatile("bar.sync 1, %0;" ::"n"(kCW * 32) : "memory");
                    // one warp per token adds the row's groups in a fixed order: the same factor in every run
                    if (warp < M) {
                        float tot = 0.f;
                        for (int t2 = lane; t2 < ntiles; t2 += 32) tot += norm_q[t2 * M + warp];
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
                        if (lane == 0) norm_r[warp] = rsqrtf(tot / (float)K + st.eps);
                    }
                    asm volatile("bar.sync 1, %0;" ::"n"(kCW * 32) : "memory");
                    // Pass 2: x <- bf16(x * r * (1 + gamma))
#pragma unroll
                    for (int u = 0; u < kPrepBatch; ++u) {
                        const int idx = u * kCW * 32 + tid;
                        if (idx < items) {
                            const int tm = idx >> 2, tile = tile0 + tm / M, tok = tm % M, qq = idx & 3;
                            const float r = norm_r[tok];
                            const uint4 gm = *reinterpret_cast<const uint4*>(st.gamma + tile * kGroup + qq * 8);
                            const uint32_t xw[4] = {v[u].x, v[u].y, v[u].z, v[u].w}, gw[4] = {gm.x, gm.y, gm.z, gm.w};
                            uint32_t o[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float f0 = __uint_as_float(xw[i] << 16), f1 = __uint_as_float(xw[i] & 0xffff0000u);
                                const float g0 = 1.0f + __uint_as_float(gw[i] << 16), g1 = 1.0f + __uint_as_float(gw[i] & 0xffff0000u);
                                o[i] = (uint32_t)f32_to_bf16_rne(f0 * r * g0) | ((uint32_t)f32_to_bf16_rne(f1 * r * g1) << 16);
                            }
                            v[u] = make_uint4(o[0], o[1], o[2], o[3]);
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < kPrepBatch; ++u) {
                    const int idx = u * kCW * 32 + tid;
                    if (u * kCW * 32 < items) {  // warp-uniform: whole quads run the shuffles together
                        const bool valid = idx < items;
                        const int tm = idx >> 2;
                        if (xprep_item<MT::kCols>(v[u], M, valid ? tile_rel(tm / M) : 0, valid ? tm % M : 0, idx & 3, valid, xs_g, xsc_g))
                            saw_flagged = true;
                    }
                }
            }
            // all of x is in place; the same barrier instruction tells every consumer whether a group was flagged
            const bool any_flagged = named_barrier_or(1, kCW * 32, saw_flagged);

            // ---- strip bookkeeping in processing order (see the single-call kernel) ----
            const int nblk = g.nblk, len = g.len;
            int unit_first = g.nt > 0 ? -g.bl_tail : -g.bl_first;
            int unit_next = g.nt > 0 ? g.nt : unit_first + len;
            int first_fix = g.nt > 0 ? g.bl_first : 0;
            int piece_lo = 0, piece = 0;
            auto next_unit = [&]() {
                piece_lo = unit_next;
                unit_first = unit_next - first_fix;
                first_fix = 0;
                unit_next = unit_first + len;
            };
            // hand the warp's partial rows of the current strip piece to a reducer warp
            auto flush = [&]() {
                if (MT::kCols && any_flagged && alive) {
                    // flagged groups among the tiles this warp processed for the piece: the fp32 path adds them
                    const int hi = unit_next < nblk ? unit_next : nblk;
                    if (hi > piece_lo) {
                        const int64_t s_cur = g.nt > 0 ? (piece == 0 ? g.s_last : g.s_first + piece - 1) : g.s_first + piece;
                        ExactPiece ep;
                        ep.blk0 = st.W + s_cur * strip_bytes + (int64_t)g.b_first * kBB;
                        ep.groups_total = groups_total;
                        ep.b_first = g.b_first;
                        ep.bl_lo = piece_lo - unit_first;
                        ep.bl_hi = hi - unit_first;
                        ep.pos0 = unit_first;
                        ep.CB = kCB;
                        ep.j0 = j0;
                        ep.BPW = kBPW;
                        ep.tw = tw;
                        ep.raw_tile_stride = la.x_stride;
                        ep.unit_tile_stride = la.x_stride;
                        ep.piece_stride = 16u;
#pragma unroll
                        for (int tk = 0; tk < MT::kAccM; ++tk) {
                            ep.unit0 = xs + (uint32_t)(tk * kColsRecBytes + kColsUnitOff);
                            ep.raw0 = xs + (uint32_t)(tk * kColsRecBytes);
                            acc_m[tk] += piece_exact_token<FMT>(ep, lane);
                        }
                    }
                }
                const int par = pieceG & 1;
                if (alive && pieceG >= 2 && !mbar_wait(red_empty0 + 8u * par, ((pieceG >> 1) - 1) & 1, cp.status)) alive = false;
                constexpr int PT = MT::kCols ? kColsPartTerms : 1;
                const uint32_t slot = part + (uint32_t)((par * kCW + warp) * PT * kStripRows * M) * 4u;
                if (MT::kCols) {
                    const int tok = q >> 1;
                    if (tok < M) {
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            asm volatile("st.shared.f32 [%0], %1;" ::"r"(slot + (uint32_t)((((q & 1) * M + tok) * kStripRows) + g8 + 8 * i) * 4u),
                                         "f"(acc[i][0])
                                         : "memory");
                    }
#pragma unroll
                    for (int tk = 0; tk < MT::kAccM; ++tk) {
                        asm volatile("st.shared.f32 [%0], %1;" ::"r"(slot + (uint32_t)((2 * M + tk) * kStripRows + lane) * 4u), "f"(acc_m[tk])
                                     : "memory");
                        acc_m[tk] = 0.f;
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[i][0] = 0.f;
                } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int j = 0; j < NT; ++j) {
                            const int tok = 2 * q + j;
                            if (tok < M)
                                asm volatile("st.shared.f32 [%0], %1;" ::"r"(slot + (uint32_t)(tok * kStripRows + g8 + 8 * i) * 4u),
                                             "f"(acc[i][j])
                                             : "memory");
                            acc[i][j] = 0.f;
                        }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(red_full0 + 8u * par);
                ++piece;
                ++pieceG;
            };

            const bool all_full = (groups_total & 7) == 0;
            auto interior_limit = [&]() { return all_full ? (unit_next < nblk ? unit_next : nblk) : -1; };
            int lim = interior_limit();
            for (int c = 0; c < g.nchunk; ++c) {
                const int i0 = c * kCB + j0;
                if (i0 < nblk && i0 >= unit_next) {
                    while (i0 >= unit_next) { flush(); next_unit(); }
                    lim = interior_limit();
                }
                if (alive && !mbar_wait(full0 + 8u * stage, phase, cp.status)) alive = false;
                if (alive) {
                    const uint32_t sbase = ring + stage * kStageBytes + j0 * kBB;
                    if (i0 + kBPW - 1 < lim) {
                        // interior stage: the warp's blocks inside the range and the current strip, every block full
                        const int tile = (i0 - unit_first) * 8 + tw;
#pragma unroll
                        for (int pr = 0; pr < kBPW / 2; ++pr) {  // two tiles in flight at a time
                            const uint32_t sb = sbase + pr * 2 * kBB;
                            TileIn ta, tb;
                            tile_load<MODE, FMT>(ta, sb + code_lane, sb + so_full, sb + m_full, tile + 16 * pr, la);
                            tile_load<MODE, FMT>(tb, sb + kBB + code_lane, sb + kBB + so_full, sb + kBB + m_full, tile + 16 * pr + 8, la);
                            tile_compute<MODE, FMT>(ta, acc, acc_m, lc);
                            if (pr == kBPW / 2 - 1) {
                                // every shared-memory read of this stage has been issued and consumed in order: hand it back
                                __syncwarp();
                                if (lane == 0) mbar_arrive(empty0 + 8u * stage);
                            }
                            tile_compute<MODE, FMT>(tb, acc, acc_m, lc);
                        }
                    } else if (all_full && i0 + kBPW <= nblk && unit_next > i0 && unit_next - first_fix + len >= i0 + kBPW) {
                        // exactly one strip boundary inside the warp's blocks, every block full and inside the range: the
                        // blocks before it, the hand-off of the finished strip piece, the blocks after it -- two tiles in
                        // flight wherever two neighbours are on the same side
                        const int pb = unit_next - i0;  // first block of the next strip piece, 1 .. BPW - 1
#pragma unroll 1
                        for (int jj = 0; jj < kBPW;) {
                            if (jj == pb) {
                                flush();
                                next_unit();
                                lim = interior_limit();
                            }
                            const uint32_t sb = sbase + jj * kBB;
                            const int tile = (i0 + jj - unit_first) * 8 + tw;
                            TileIn ta;
                            tile_load<MODE, FMT>(ta, sb + code_lane, sb + so_full, sb + m_full, tile, la);
                            if (jj + 1 < kBPW && jj + 1 != pb) {
                                TileIn tb;
                                tile_load<MODE, FMT>(tb, sb + kBB + code_lane, sb + kBB + so_full, sb + kBB + m_full, tile + 8, la);
                                tile_compute<MODE, FMT>(ta, acc, acc_m, lc);
                                tile_compute<MODE, FMT>(tb, acc, acc_m, lc);
                                jj += 2;
                            } else {
                                tile_compute<MODE, FMT>(ta, acc, acc_m, lc);
                                jj += 1;
                            }
                        }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(empty0 + 8u * stage);
                    } else {
                        // general stage (range end, several boundaries, short last block): one block at a time
                        for (int jj = 0; jj < kBPW; ++jj) {
                            const int i = i0 + jj;
                            if (i >= nblk) break;
                            if (i >= unit_next) {
                                while (i >= unit_next) { flush(); next_unit(); }
                                lim = interior_limit();
                            }
                            const int bl = i - unit_first;
                            const int rest = groups_total - 8 * (g.b_first + bl);
                            const int jb = rest < 8 ? rest : 8;
                            if (tw < jb) {
                                const uint32_t sb = sbase + jj * kBB;
                                TileIn ta;
                                tile_load<MODE, FMT>(ta, sb + code_lane, sb + so_sect * jb + so_chunk, sb + 576u * jb + m_lane, bl * 8 + tw, la);
                                tile_compute<MODE, FMT>(ta, acc, acc_m, lc);
                            }
                        }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(empty0 + 8u * stage);
                    }
                }
                if (++stage == nstage) { stage = 0; phase ^= 1u; }
            }
            while (piece < g.npieces) { flush(); next_unit(); }
        }
    } else {
        // =============================== reducers ================================================
        const int r = warp - kCW - 1;
        int pieceG = 0, stored_strips = 0;
        bool alive = true;
        asm volatile("griddepcontrol.wait;" ::: "memory");  // before any global write of this grid
        for (int ui = 0; ui < cp.nunits; ++ui) {
            const int si = cp.unit_step[ui], uz = cp.unit_slice[ui];
            const ChainStep& st = cp.step[si];
            const StepGeom g = unit_geom(cp, st, uz, blockIdx.x, kCB, geo[ui]);
            const int len = g.len;
            for (int piece = 0; piece < g.npieces; ++piece) {
                const int G = pieceG + piece;  // index over all steps: hand-over buffer and owner alternate with it
                if ((G % kNR) != r) continue;
                // pieces in processing order: the partial last strip first (if any), then the strips in order
                const int64_t s = g.nt > 0 ? (piece == 0 ? g.s_last : g.s_first + piece - 1) : g.s_first + piece;
                const int64_t unit_begin = s * len, unit_end = unit_begin + len;
                const int64_t pa = unit_begin > g.a ? unit_begin : g.a;
                const int64_t pe = unit_end < g.e ? unit_end : g.e;
                const int par = G & 1;
                if (alive && !mbar_wait(red_full0 + 8u * par, (G >> 1) & 1, cp.status)) alive = false;
                if (!alive) break;
                const float* part_g = reinterpret_cast<const float*>(smem + cp.off_part);
                float v[kMaxTokens];
#pragma unroll
                for (int t = 0; t < kMaxTokens; ++t) {
                    v[t] = 0.f;
                    if (t < M) {
                        constexpr int PT = MT::kCols ? kColsPartTerms : 1;
#pragma unroll
                        for (int w = 0; w < kCW; ++w)
#pragma unroll
                            for (int h = 0; h < PT; ++h)
                                v[t] += part_g[(((par * kCW + w) * PT + h) * M + t) * kStripRows + lane];
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(red_empty0 + 8u * par);

                const bool whole_unit = (pa == unit_begin) && (pe == unit_end);
                bool stored = false;
                if (st.Z == 1 && whole_unit) {
#pragma unroll
                    for (int t = 0; t < kMaxTokens; ++t)
                        if (t < M) {
                            if (!EPI) st.y[(int64_t)t * st.N + s * kStripRows + lane] = v[t];
                            else store_output(st.y, st.y16, st.epi, st.N, s, lane, t, v[t]);
                        }
                    stored = true;
                } else {
                    float* slot = chain_piece_slot(cp, st, g.z, g.ci, s, unit_begin, whole_unit, g.a_true);
#pragma unroll
                    for (int t = 0; t < kMaxTokens; ++t)
                        if (t < M) slot[t * kStripRows + lane] = v[t];
                    __syncwarp();
                    // how many pieces does strip s have over all slices?
                    int total = 0;
                    for (int zz = 0; zz < st.Z; ++zz) {
                        int64_t cf, cl;
                        strip_ctas(cp, st, zz, s, &cf, &cl);
                        total += (int)(cl - cf) + 1;
                    }
                    // release this warp's partial rows and acquire everybody else's in one round trip
                    int old = 0;
                    if (lane == 0)
                        asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(cp.tickets + st.ticket_off + s) : "memory");
                    old = __shfl_sync(0xffffffffu, old, 0);
                    if (old == total - 1) {
                        // last piece to arrive: add all pieces of the strip in a fixed order
#pragma unroll
                        for (int t = 0; t < kMaxTokens; ++t) v[t] = 0.f;
                        for (int zz = 0; zz < st.Z; ++zz) {
                            const int64_t u0 = s * chain_slice_len(st, zz);
                            int64_t cf, cl;
                            strip_ctas(cp, st, zz, s, &cf, &cl);
                            for (int64_t c2 = cf; c2 <= cl; ++c2) {
                                const float* src = chain_piece_slot(cp, st, zz, c2, s, u0, cf == cl, cta_range_begin(cp, st, zz, c2));
#pragma unroll
                                for (int t = 0; t < kMaxTokens; ++t)
                                    if (t < M) v[t] += __ldcg(src + t * kStripRows + lane);
                            }
                        }
#pragma unroll
                        for (int t = 0; t < kMaxTokens; ++t)
                            if (t < M) {
                                if (!EPI) st.y[(int64_t)t * st.N + s * kStripRows + lane] = v[t];
                                else store_output(st.y, st.y16, st.epi, st.N, s, lane, t, v[t]);
                            }
                        if (lane == 0) cp.tickets[st.ticket_off + s] = 0;  // ready for the next launch on this stream
                        stored = true;
                    }
                }
                if (stored) ++stored_strips;
            }
            pieceG += g.npieces;
            // Strips whose outputs this warp put into global memory, counted for the step that waits on this one: one
            // addition per warp and step (not per strip: every CTA of the grid polls this counter).
            if (st.signal && stored_strips > 0 && (ui + 1 == cp.nunits || cp.unit_step[ui + 1] != si)) {
                __syncwarp();
                if (lane == 0) asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(cp.done + si), "r"(stored_strips) : "memory");
                stored_strips = 0;
            }
            if (ui + 1 == cp.nunits || cp.unit_step[ui + 1] != si) stored_strips = 0;
        }
    }

    // The last CTA to leave puts the dependency counters back to zero for the next launch (every wait of every CTA
    // has ended by the time its threads meet here).
    if (!cp.has_deps) return;  // (kernel-uniform) no step of this launch counted anything
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const int old = atomicAdd(cp.exit_count, 1);
        if (old == (int)gridDim.x - 1) {
            for (int i = 0; i < cp.nsteps; ++i) cp.done[i] = 0;
            *cp.exit_count = 0;
            __threadfence();
        }
    }
}

template <int MODE>
static cudaError_t chain_set_smem_limit_mode(int bytes) {
    const cudaFuncAttribute a = cudaFuncAttributeMaxDynamicSharedMemorySize;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(fdqp_chain_kernel<MODE, 2, false>, a, bytes))) return e;
    if ((e = cudaFuncSetAttribute(fdqp_chain_kernel<MODE, 2, true>, a, bytes))) return e;
    if ((e = cudaFuncSetAttribute(fdqp_chain_kernel<MODE, 4, false>, a, bytes))) return e;
    return cudaFuncSetAttribute(fdqp_chain_kernel<MODE, 4, true>, a, bytes);
}

cudaError_t chain_set_smem_limit(int bytes) {
    cudaError_t e;
    if ((e = chain_set_smem_limit_mode<1>(bytes))) return e;
    if ((e = chain_set_smem_limit_mode<2>(bytes))) return e;
    return chain_set_smem_limit_mode<3>(bytes);
}

template <int MODE>
static cudaError_t chain_launch_mode(const cudaLaunchConfig_t& cfg, const ChainPlan& cp, bool epi) {
    if (cp.bpw == 4)
        return epi ? cudaLaunchKernelEx(&cfg, fdqp_chain_kernel<MODE, 4, true>, cp) : cudaLaunchKernelEx(&cfg, fdqp_chain_kernel<MODE, 4, false>, cp);
    return epi ? cudaLaunchKernelEx(&cfg, fdqp_chain_kernel<MODE, 2, true>, cp) : cudaLaunchKernelEx(&cfg, fdqp_chain_kernel<MODE, 2, false>, cp);
}

// launch_mode: bit 0 = programmatic stream serialisation (the next launch may start its weight stream early),
// bit 1 = cooperative launch (the runtime refuses the launch unless all CTAs can be resident at once).
cudaError_t chain_launch(const ChainPlan& cp, int grid, bool epi, int launch_mode, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)kThreads);
    cfg.dynamicSmemBytes = cp.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (launch_mode & 1) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    if (launch_mode & 2) {
        attr[n].id = cudaLaunchAttributeCooperative;
        attr[n].val.cooperative = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = (unsigned)n;
    if (cp.M == 1) return chain_launch_mode<1>(cfg, cp, epi);
    if (cp.M == 2) return chain_launch_mode<3>(cfg, cp, epi);
    return chain_launch_mode<2>(cfg, cp, epi);
}

}  // namespace fdqp
