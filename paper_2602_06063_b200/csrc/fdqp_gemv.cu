// Streaming GEMV kernels for FusedDQP at M = 1..8 tokens (Sec. "FusedDQP", Eq. 14 / 15, with the
// block-wise dequantisation of Eq. 3 fused in).
//
// Shape of the computation.  For every quantisation group (32 consecutive k of one output row n)
//     sum_k x_k * (d * q_k + m)  =  d * (sum_k q_k x_k)  +  m * (sum_k x_k)
// so the per-weight work is only "unpack a nibble and multiply-accumulate it with x"; scale d and
// offset m are applied once per group in fp32.
//
// The inner sums sum_k q_k x_k run on the warp-level integer tensor-core instruction
// (mma.sync m16n8k32, u8 x s8/u8 -> s32): the 4-bit codes become bytes with two logic ops per four
// codes (w & 0x0F0F0F0F, (w >> 4) & 0x0F0F0F0F -- B200 issues integer/logic instructions at half the
// fp32 rate, so this unpack is the budget that matters), and the activations of a group are held as
// fixed point relative to the group's largest exponent (|value| <= 2^22), split into three byte planes
// (x = 2^e_g * (65536 p2 + 256 p1 + p0), p2 signed, p1 and p0 unsigned; exact for every element
// within 2^14 of the group's largest, rounded to 2^-22 of it otherwise).  One MMA covers a whole
// group of 16 output rows; its s32 result is exact.  The order of k inside a group is a free
// permutation as long as both operands use the same one (even k in the low half, odd k in the high).
// The plane sums are recombined in int32 (they fit) and converted to fp32 once per value.
// For M <= 2 most of the MMA's eight token columns would be idle, so the three planes of a token ride in
// three columns (as signed digits; column 3 / 7 is zero): one MMA per 16 rows yields all three plane sums
// of up to TWO tokens (kernel modes: 1 = one token, 3 = two tokens).  Mode 2 (M = 3..8) issues one MMA per plane
// with the eight tokens as columns; measured on B200 it beats two column-mode MMAs from M = 3 on.
//
// The plane split of x is done by every GEMV CTA itself when its K slice is short (one work item per
// consumer thread at most), else once per call by a small preparation kernel, after which every GEMV
// CTA brings its K slice of the prepared x into shared memory with bulk async copies.
//
// Data movement.  The packed matrix is strip-major (32 output rows x all of K contiguous), so every
// CTA streams one contiguous byte range of HBM exactly once.  The producer warp issues one 1-D bulk
// async copy per Q4NX block (<= 5120 bytes), several lanes at a time, into a shared-memory ring of
// multi-block stages guarded by mbarriers; every consumer warp owns the same 32 x 32 group-tile of
// two or four blocks of a stage.
//
// Work split.  The (K-slice, strip, block) space is cut into equal contiguous ranges, one per
// persistent CTA, so all SMs stream the same number of bytes whatever N and K are.  A strip whose
// blocks end up in several CTAs (or several K slices) is completed by whichever CTA arrives last at
// the strip's ticket: it sums the partial rows in a fixed order, so results are reproducible run to
// run (K slices, used only when the prepared x of the whole K would not fit beside the ring, are
// strip-aligned and added by fdqp_splitk_sum_kernel instead).  A CTA handles the shared strip at the END of its range FIRST, so that the exchange through
// global memory is off its critical path and its last piece is a whole strip written directly.
// No CTA ever waits for another CTA.
#include "fdqp_gemv_tile.cuh"

namespace fdqp {

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


// Stand-alone preparation of a whole x, for calls whose K slice is too large to prepare inside every GEMV CTA.
template <bool SINGLE>
__global__ void __launch_bounds__(128) fdqp_xprep_kernel(const uint16_t* __restrict__ x, uint32_t* __restrict__ xq,
                                                          float* __restrict__ xsc, int M, int K) {
    // The GEMV kernel that follows is launched with programmatic stream serialisation: it may start now and
    // stream weights; it waits (griddepcontrol.wait) before touching what this kernel writes.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");  // x may be the previous launch's output
    const int items = (K / kGroup) * M * 4;
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    const bool valid = idx < items;
    const int q = idx & 3, tm = idx >> 2;
    const int tok = valid ? tm % M : 0, tile = valid ? tm / M : 0;
    xprep_item<SINGLE>(xprep_load(x, K, tile, tok, q, valid), M, tile, tok, q, valid, xq, xsc);
}

// CW consumer warps (8 or 16); MODE as above (1: M = 1, 3: M = 2, 2: M = 3..8); EPI: built with the bf16 epilogues
// and the fused RMS normalisation (the plain build keeps its stores and its preparation free of their branches).
// A ring stage holds CB = (CW / 8) * BPW blocks; warp w owns group-tile (w & 7) of the BPW (2 or 4) consecutive
// blocks starting at BPW * (w >> 3) of every stage.  More blocks per stage = fewer barrier round trips per tile.
// Warps CW+1 .. CW+NR are reducers (NR = CW / 8): reducer r completes the strip pieces with piece % NR == r.
// FMT: the container's format (fdqp_format.h).  The variants differ in the block size, in where a tile's scale and
// offset sit (one per 64 or 128 inputs: tiles share them) and, for MXFP4, in how codes and scales become numbers; they
// hold whole blocks only.
template <int CW, int MODE, int BPW, bool EPI, int FMT = kFmtQ4nx>
__global__ void __launch_bounds__((CW + 1 + CW / 8) * 32, CW == 8 ? 2 : 1)
    fdqp_gemv_kernel(const __grid_constant__ GemvPlan p) {
    extern __shared__ __align__(128) uint8_t smem[];
    using MT = ModeTraits<MODE>;
    using F = FmtTraits<FMT>;
    constexpr int NT = MT::kAcc;
    constexpr int CB = (CW / 8) * BPW;
    constexpr int NR = CW / 8;
    constexpr uint32_t kBB = F::kBlock;  // bytes of a full block
    constexpr uint32_t kStageBytes = CB * kBB;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int M = MODE == 1 ? 1 : (MODE == 3 ? 2 : p.M), K = p.K;  // compile-time in the column modes

    const int z = blockIdx.x / p.Gz;
    const int64_t ci = blockIdx.x % p.Gz;
    const int b_first = z * p.nbz;
    const int len = slice_len(p, z);
    const int64_t T = (int64_t)p.S * len;
    // contiguous range of the slice's blocks: equal block counts, or whole strips when the plan asks for that
    const int64_t a = p.strip_aligned ? range_begin(ci, p.Gz, p.S) * len : range_begin(ci, p.Gz, T);
    const int64_t e = p.strip_aligned ? range_begin(ci + 1, p.Gz, p.S) * len : range_begin(ci + 1, p.Gz, T);
    const int nblk = (int)(e - a);
    if (nblk <= 0) return;
    const bool small = fits32(p.Gz, T);
    const int64_t s_first = div_floor(a, len, small), s_last = div_floor(e - 1, len, small);
    const int bl_first = (int)(a - s_first * len);    // block index inside the slice of the CTA's first block
    const int npieces = (int)(s_last - s_first) + 1;  // strips this CTA touches
    // Processing order: the blocks of a partial last strip come first, then the rest of the range in order.
    const int64_t tail_begin = s_last * len > a ? s_last * len : a;
    const int nt = (npieces >= 2 && e < (s_last + 1) * len) ? (int)(e - tail_begin) : 0;
    const int bl_tail = (int)(tail_begin - s_last * len);
    const int nchunk = (nblk + CB - 1) / CB;

    const uint32_t ring = smem_u32(smem);
    const uint32_t xs = ring + p.off_xs, xsc = ring + p.off_xsum;
    const uint32_t part = ring + p.off_part, bars = ring + p.off_bar;
    const int nstage = p.nstage;
    const uint32_t full0 = bars, empty0 = bars + 8u * nstage;
    const uint32_t red_full0 = bars + 16u * nstage, red_empty0 = red_full0 + 16u, x_bar = red_full0 + 32u;

    for (int s = tid; s < nstage; s += blockDim.x) {
        mbar_init(full0 + 8u * s, 1);
        mbar_init(empty0 + 8u * s, CW);
    }
    if (tid < 2) {
        mbar_init(red_full0 + 8u * tid, CW);
        mbar_init(red_empty0 + 8u * tid, 1);
    }
    if (tid == 2) mbar_init(x_bar, 1);
    // fused RMS normalisation: one sum of squares per (group-tile, token) quad, up to 128 of them
    float* const norm_q = reinterpret_cast<float*>(smem + p.off_bar + (2u * (uint32_t)nstage + 6u) * 8u);
    mbar_fence_init();
    __syncthreads();
    // The next launch in the stream may begin as soon as SM slots free up: it streams weights (which nothing in this
    // library writes) and waits for this grid to complete before it touches activations, outputs or workspace.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int groups_total = K / kGroup;
    const int64_t strip_bytes = FMT == kFmtQ4nx ? (int64_t)kGroupBytes * groups_total : (int64_t)kBB * (groups_total / 8);

    if (warp == CW) {
        // =============================== producer ================================================
        // Lane j < CB copies block j of every stage; lane 0 owns the barrier traffic.
        uint64_t policy = 0;
        if (p.evict_first) policy = l2_policy_evict_first();
        const uint32_t len_magic = (uint32_t)(0x100000000ull / (uint32_t)len) + 1u;
        const bool magic_ok = ((uint64_t)(nblk + len) * (uint64_t)len) < 0x80000000ull && len > 1;
        int stage = 0;
        uint32_t phase = 0;  // parity of the stage's current use
        bool alive = true;
        int c = 0;
        for (; c < nchunk && alive; ++c) {
            if (c >= nstage) {
                int ok = 1;
                if (lane == 0) ok = mbar_wait(empty0 + 8u * stage, phase ^ 1u, p.status) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { alive = false; break; }
            }
            const int i = c * CB + lane;  // position in processing order
            uint32_t bytes = 0;
            int64_t ps = 0;
            int pbl = 0;
            if (lane < CB && i < nblk) {
                // block i of the processing order -> (strip, block inside the slice)
                const uint32_t rel = (uint32_t)bl_first + (uint32_t)(i < nt ? (nblk - nt + i) : (i - nt));
                uint32_t so = __umulhi(rel, len_magic);  // rel / len: exact while rel * len < 2^32
                if (!magic_ok) so = rel / (uint32_t)len;
                ps = s_first + so;
                pbl = (int)(rel - so * (uint32_t)len);
                const int rest = groups_total - 8 * (b_first + pbl);
                bytes = FMT == kFmtQ4nx ? (uint32_t)kGroupBytes * (uint32_t)(rest < 8 ? rest : 8) : kBB;
            }
            const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
            if (lane == 0) mbar_arrive_expect_tx(full0 + 8u * stage, total);
            __syncwarp();
            // Blocks that follow each other in the container AND in the stage go out as ONE copy (strips follow each other
            // in memory, so that is usually the whole stage): the memory system serves 20-40 KB copies faster than 5 KB ones
            // (bare read stream: 7.28 against 6.93 TB/s).  A run ends after a short block (its slot in the stage is not filled).
            const uint8_t* src = p.W + ps * strip_bytes + (int64_t)(b_first + pbl) * kBB;
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
                if (p.evict_first)
                    bulk_g2s_hint(dst, src, run_bytes, full0 + 8u * stage, policy);
                else
                    bulk_g2s(dst, src, run_bytes, full0 + 8u * stage);
            }
            if (++stage == nstage) { stage = 0; phase ^= 1u; }
        }
        // Do not leave while a copy into this CTA's shared memory may still be in flight.
        if (lane == 0) {
            if (!p.prep_inline) mbar_wait(x_bar, 0, p.status);
            const int issued = c;
            const int from = issued > nstage ? issued - nstage : 0;
            for (int k = from; k < issued; ++k)
                if (!mbar_wait(full0 + 8u * (k % nstage), (k / nstage) & 1, p.status)) break;
        }
        return;
    }

    if (warp < CW) {
        // =============================== consumers ===============================================
        const int tw = warp & 7, j0 = (warp >> 3) * BPW;
        const int g = lane >> 2, q = lane & 3;
        // B fragments.  Mode 2: column g is token g (any valid token for unused columns: their results are never
        // stored).  Column modes: column g is plane 2 - g%4 of token g/4 (zeros for g%4 == 3 and for a token that
        // does not exist); this lane accumulates the columns of token q/2.
        LaneAddr la;
        LaneConst lc{};
        la.xs = xs;
        la.x_stride = (uint32_t)M * (uint32_t)(MT::kCols ? kColsRecBytes : kPlaneRecBytes);
        {
            const int gtok = g < M ? g : M - 1;
            la.x_lane = xs + (uint32_t)(gtok * 4 + q) * 16u;
            la.xsc_lane = xsc + q * 8;
            const int tok_b = g >> 2, pl = g & 3;
            la.xb_off = tok_b < M ? (uint32_t)(tok_b * kColsRecBytes + pl * 32 + q * 8) : 0u;  // (no such token: weight 0 below)
            const int tok_d = q >> 1;
            la.sc_off = (uint32_t)((tok_d < M ? tok_d : 0) * kColsRecBytes + kColsSumOff);
            lc.w_unit = (tok_d < M ? ((q & 1) ? 1.f : 65536.f) : 0.f) * (F::kMx ? 0.5f : 1.f);
            if (F::kMx) lc.mx = mx_tables();
            // (opaque moves: the compiler keeps the two constants in registers instead of re-creating them per use)
            asm volatile("mov.b32 %0, 0x000F000F;" : "=r"(lc.nib_mask));
            asm volatile("mov.b32 %0, 0x43004300;" : "=r"(lc.nib_magic));
        }
        float acc_m[MT::kAccM];  // column modes: offset term of row `lane`, per token
#pragma unroll
        for (int tk = 0; tk < MT::kAccM; ++tk) acc_m[tk] = 0.f;
        // ldmatrix source rows: codes = row `lane` of the tile; scales/offsets = the four 16-byte
        // chunks of this tile's scale words and of its offset words, duplicated so that after the
        // transposed load every lane of a quad holds (d[g], d[g+8]), (d[g+16], d[g+24]), (m..), (m..)
        const uint32_t code_lane = tw * 512 + lane * 16;
        const int mat = lane >> 3;
        const uint32_t so_chunk = (tw >> F::kShift) * 64 + (((mat & 1) * 2 + (lane & 1)) * 16);
        const uint32_t so_sect = (!MT::kCols && mat >= 2) ? 576u : 512u;  // offsets section follows the scales section
        const uint32_t m_lane = (tw >> F::kShift) * 64 + lane * 2;         // column modes: this lane's own offset word
        // the same two addresses inside a full block of the format (MXFP4: scale bytes of row g and of row `lane`)
        const uint32_t so_full = F::kMx ? (uint32_t)kCodeBytes + tw * 32 + g
                                        : ((!MT::kCols && mat >= 2) ? (uint32_t)F::kOffSect : (uint32_t)kCodeBytes) + so_chunk;
        const uint32_t m_full = F::kMx ? (uint32_t)kCodeBytes + tw * 32 + lane : (uint32_t)F::kOffSect + m_lane;

        float acc[4][NT];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < NT; ++j) acc[i][j] = 0.f;

        // Strip bookkeeping in processing order: position of block 0 of the current strip, position where
        // the next strip starts, the in-slice index of the first block after the leading tail piece, and the position
        // where the current piece began.
        int unit_first = nt > 0 ? -bl_tail : -bl_first;
        int unit_next = nt > 0 ? nt : unit_first + len;
        int first_fix = nt > 0 ? bl_first : 0;
        int piece_lo = 0;
        auto next_unit = [&]() {
            piece_lo = unit_next;
            unit_first = unit_next - first_fix;
            first_fix = 0;
            unit_next = unit_first + len;
        };
        bool any_flagged = false;  // set once x is prepared: some group of the K slice takes the fp32 path

        // where this lane's partial sums go in the reducer's buffer (parity 0; parity 1 lies part_par_bytes further)
        constexpr int PT = MT::kCols ? kColsPartTerms : 1;
        const uint32_t part_par_bytes = (uint32_t)(CW * PT * kStripRows * M) * 4u;
        const uint32_t part_warp = part + (uint32_t)(warp * PT * kStripRows * M) * 4u;
        const uint32_t st_acc = part_warp + (uint32_t)(MT::kCols ? ((q & 1) * M + (q >> 1)) * kStripRows + g : 2 * q * kStripRows + g) * 4u;
        const uint32_t st_m = part_warp + (uint32_t)(2 * M * kStripRows + lane) * 4u;
        int piece = 0;
        bool alive = true;
        // hand the warp's partial rows of the current strip piece to the reducer warp
        auto flush = [&]() {
            if (MT::kCols && any_flagged && alive) {
                // flagged groups among the tiles this warp processed for the piece: their contribution comes from the
                // fp32 path (the tensor-core path added exactly zero for them)
                const int hi = unit_next < nblk ? unit_next : nblk;
                if (hi > piece_lo) {
                    const int64_t s_cur = nt > 0 ? (piece == 0 ? s_last : s_first + piece - 1) : s_first + piece;
                    ExactPiece ep;
                    ep.blk0 = p.W + s_cur * strip_bytes + (int64_t)b_first * kBB;
                    ep.groups_total = groups_total;
                    ep.b_first = b_first;
                    ep.bl_lo = piece_lo - unit_first;
                    ep.bl_hi = hi - unit_first;
                    ep.pos0 = unit_first;
                    ep.CB = CB;
                    ep.j0 = j0;
                    ep.BPW = BPW;
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
            const int par = piece & 1;
            if (piece >= 2 && !mbar_wait(red_empty0 + 8u * par, ((piece >> 1) - 1) & 1, p.status)) alive = false;
            const uint32_t pslot = par ? part_par_bytes : 0u;
            if (MT::kCols) {
                // Lanes q and q^1 hold the two column halves of each row's sum for token q/2, lane r holds row r's
                // offset terms: all three go to the reducer as they are ([term][token][row]); it adds them.
                if ((q >> 1) < M) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        asm volatile("st.shared.f32 [%0], %1;" ::"r"(st_acc + pslot + 32u * i), "f"(acc[i][0]) : "memory");
                }
#pragma unroll
                for (int tk = 0; tk < MT::kAccM; ++tk) {
                    asm volatile("st.shared.f32 [%0], %1;" ::"r"(st_m + pslot + (uint32_t)(tk * kStripRows * 4)), "f"(acc_m[tk]) : "memory");
                    acc_m[tk] = 0.f;
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[i][0] = 0.f;
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < NT; ++j) {
                        if (2 * q + j < M)
                            asm volatile("st.shared.f32 [%0], %1;" ::"r"(st_acc + pslot + (uint32_t)((j * kStripRows + 8 * i) * 4)), "f"(acc[i][j])
                                         : "memory");
                        acc[i][j] = 0.f;
                    }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(red_full0 + 8u * par);
            ++piece;
        };

        // Everything up to here touched only this CTA's shared memory.  x may come from the previous launch.
        asm volatile("griddepcontrol.wait;" ::: "memory");
        bool saw_flagged = false;
        if (p.prep_inline) {
            // prepare this CTA's K slice of x straight into shared memory (cheap, and the first weights are still
            // on their way from HBM)
            const int kbeg = b_first * kBlockK;
            const int kend_full = (b_first + len) * kBlockK;
            const int tile0 = kbeg / kGroup, ntiles = ((kend_full < K ? kend_full : K) - kbeg) / kGroup;
            const int items = ntiles * M * 4;
            uint32_t* xs_g = reinterpret_cast<uint32_t*>(smem + p.off_xs);
            float* xsc_g = reinterpret_cast<float*>(smem + p.off_xsum);
            constexpr int kBatch = 8;  // loads in flight per thread: one trip to L2 / HBM for typical decode shapes
            for (int base = 0; base < items; base += kBatch * CW * 32) {
                uint4 v[kBatch];
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const int idx = base + u * CW * 32 + tid;
                    const bool valid = idx < items;
                    const int tm = idx >> 2;
                    v[u] = xprep_load(p.x, K, tile0 + (valid ? tm / M : 0), valid ? tm % M : 0, idx & 3, valid);
                }
                if (EPI && p.norm) {
                    // RMS normalisation in place (the plan guarantees one item per thread at most and the whole row in
                    // this CTA): sum of squares per token over all quads, then x <- bf16(x * r * (1 + gamma))
                    const bool valid = tid < items;
                    const int tm = tid >> 2, tok = valid ? tm % M : 0, tile = valid ? tm / M : 0;
                    const uint4 gm = xprep_load(p.gamma, K, tile0 + tile, 0, tid & 3, valid);
                    if (p.residual) {
                        // the residual addition first; every CTA needs the sum, the grid's first CTA also stores it
                        v[0] = add_bf16x8(v[0], xprep_load(p.residual, K, tile0 + tile, tok, tid & 3, valid));
                        if (p.h_out && blockIdx.x == 0 && valid)
                            *reinterpret_cast<uint4*>(p.h_out + (int64_t)tok * K + (tile0 + tile) * kGroup + (tid & 3) * 8) = v[0];
                    }
                    const uint32_t xw[4] = {v[0].x, v[0].y, v[0].z, v[0].w}, gw[4] = {gm.x, gm.y, gm.z, gm.w};
                    float f[8], ss = 0.f;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        f[2 * i] = __uint_as_float(xw[i] << 16);
                        f[2 * i + 1] = __uint_as_float(xw[i] & 0xffff0000u);
                        ss = fmaf(f[2 * i], f[2 * i], ss);
                        ss = fmaf(f[2 * i + 1], f[2 * i + 1], ss);
                    }
                    ss += __shfl_xor_sync(0xffffffffu, ss, 1);
                    ss += __shfl_xor_sync(0xffffffffu, ss, 2);
                    if (valid && (tid & 3) == 0) norm_q[tm] = ss;  // tm = tile * M + tok
                    asm volatile("bar.sync 1, %0;" ::"n"(CW * 32) : "memory");
                    // the row's quads in a fixed order (four interleaved chains): the same sum in every thread and run
                    float t4[4] = {0.f, 0.f, 0.f, 0.f};
                    int t2 = 0;
                    for (; t2 + 4 <= ntiles; t2 += 4) {
#pragma unroll
                        for (int c4 = 0; c4 < 4; ++c4) t4[c4] += norm_q[(t2 + c4) * M + tok];
                    }
                    for (; t2 < ntiles; ++t2) t4[0] += norm_q[t2 * M + tok];
                    const float tot = (t4[0] + t4[1]) + (t4[2] + t4[3]);
                    const float r = rsqrtf(tot / (float)K + p.eps);
                    uint32_t o[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float g0 = 1.0f + __uint_as_float(gw[i] << 16), g1 = 1.0f + __uint_as_float(gw[i] & 0xffff0000u);
                        o[i] = (uint32_t)f32_to_bf16_rne(f[2 * i] * r * g0) | ((uint32_t)f32_to_bf16_rne(f[2 * i + 1] * r * g1) << 16);
                    }
                    v[0] = make_uint4(o[0], o[1], o[2], o[3]);
                }
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const int idx = base + u * CW * 32 + tid;
                    if (base + u * CW * 32 < items) {  // warp-uniform: whole quads run the shuffles together
                        const bool valid = idx < items;
                        const int tm = idx >> 2;
                        if (xprep_item<MT::kCols>(v[u], M, valid ? tm / M : 0, valid ? tm % M : 0, idx & 3, valid, xs_g, xsc_g))
                            saw_flagged = true;
                    }
                }
            }
        } else {
            if (!mbar_wait(x_bar, 0, p.status)) alive = false;
            // the preparation kernel's records: does this CTA's K slice hold a flagged group (unit == 0)?
            if (MT::kCols) {
                const int kend_full = (b_first + len) * kBlockK;
                const int nrec = (((kend_full < K ? kend_full : K) - b_first * kBlockK) / kGroup) * M;
                for (int r = tid; r < nrec && alive; r += CW * 32) {
                    float unit;
                    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(unit) : "r"(xs + (uint32_t)(r * kColsRecBytes + kColsUnitOff)));
                    if (unit == 0.f) saw_flagged = true;
                }
            }
        }
        // all of x is in place; one barrier instruction also tells every consumer whether any group of the slice was
        // flagged for the fp32 path (none in ordinary activations: the tile loop then never looks)
        any_flagged = named_barrier_or(1, CW * 32, saw_flagged);
        // An "interior" stage -- both of the warp's blocks inside the range and the current strip, every block
        // full -- needs no bookkeeping beyond two tile indices.  `lim` is the first position that is not interior.
        const bool all_full = (groups_total & 7) == 0;
        auto interior_limit = [&]() { return all_full ? (unit_next < nblk ? unit_next : nblk) : -1; };
        int lim = interior_limit();
        int stage = 0;
        uint32_t phase = 0;
        for (int c = 0; c < nchunk && alive; ++c) {
            const int i0 = c * CB + j0;
            if (i0 < nblk && i0 >= unit_next) {
                while (i0 >= unit_next && alive) { flush(); next_unit(); }
                lim = interior_limit();
            }
            if (!mbar_wait(full0 + 8u * stage, phase, p.status)) { alive = false; break; }
            const uint32_t sbase = ring + stage * kStageBytes + j0 * kBB;
            if (i0 + BPW - 1 < lim) {
                const int tile = (i0 - unit_first) * 8 + tw;
#pragma unroll
                for (int pr = 0; pr < BPW / 2; ++pr) {  // two tiles in flight at a time
                    const uint32_t sb = sbase + pr * 2 * kBB;
                    TileIn ta, tb;
                    tile_load<MODE, FMT>(ta, sb + code_lane, sb + so_full, sb + m_full, tile + 16 * pr, la);
                    tile_load<MODE, FMT>(tb, sb + kBB + code_lane, sb + kBB + so_full, sb + kBB + m_full, tile + 16 * pr + 8, la);
                    tile_compute<MODE, FMT>(ta, acc, acc_m, lc);
                    if (pr == BPW / 2 - 1) {
                        // every shared-memory read of this stage has been issued and consumed in order: hand it back
                        __syncwarp();
                        if (lane == 0) mbar_arrive(empty0 + 8u * stage);
                    }
                    tile_compute<MODE, FMT>(tb, acc, acc_m, lc);
                }
            } else if (all_full && i0 + BPW <= nblk && unit_next > i0 && unit_next - first_fix + len >= i0 + BPW) {
                // exactly one strip boundary inside the warp's blocks, every block full and inside the range: the blocks
                // before it, the hand-off of the finished strip piece, the blocks after it -- two tiles in flight
                // wherever two neighbours are on the same side
                const int pb = unit_next - i0;  // first block of the next strip piece, 1 .. BPW - 1
                auto one = [&](int jj) {
                    const uint32_t sb = sbase + jj * kBB;
                    TileIn ta;
                    tile_load<MODE, FMT>(ta, sb + code_lane, sb + so_full, sb + m_full, (i0 + jj - unit_first) * 8 + tw, la);
                    tile_compute<MODE, FMT>(ta, acc, acc_m, lc);
                };
                auto two = [&](int jj) {
                    const uint32_t sb = sbase + jj * kBB;
                    const int tile = (i0 + jj - unit_first) * 8 + tw;
                    TileIn ta, tb;
                    tile_load<MODE, FMT>(ta, sb + code_lane, sb + so_full, sb + m_full, tile, la);
                    tile_load<MODE, FMT>(tb, sb + kBB + code_lane, sb + kBB + so_full, sb + kBB + m_full, tile + 8, la);
                    tile_compute<MODE, FMT>(ta, acc, acc_m, lc);
                    tile_compute<MODE, FMT>(tb, acc, acc_m, lc);
                };
                auto hand_over = [&]() {
                    flush();
                    next_unit();
                    lim = interior_limit();
                };
                if (BPW == 4) {
                    if (pb == 2) {
                        two(0);
                        hand_over();
                        two(2);
                    } else if (pb == 1) {
                        one(0);
                        hand_over();
                        two(1);
                        one(3);
                    } else {
                        two(0);
                        one(2);
                        hand_over();
                        one(3);
                    }
                } else {  // two blocks per warp: the boundary is between them
                    one(0);
                    hand_over();
                    one(1);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8u * stage);
            } else {
                // general stage (range end, several boundaries, short last block): one block at a time
                for (int jj = 0; jj < BPW; ++jj) {
                    const int i = i0 + jj;
                    if (i >= nblk) break;
                    if (i >= unit_next) {
                        while (i >= unit_next && alive) { flush(); next_unit(); }
                        lim = interior_limit();
                    }
                    const int bl = i - unit_first;
                    const int rest = groups_total - 8 * (b_first + bl);
                    const int jb = rest < 8 ? rest : 8;
                    if (tw < jb) {
                        const uint32_t sb = sbase + jj * kBB;
                        const int tile = bl * 8 + tw;
                        TileIn ta;
                        if (FMT == kFmtQ4nx)  // the only format with short last blocks
                            tile_load<MODE, FMT>(ta, sb + code_lane, sb + so_sect * jb + so_chunk, sb + 576u * jb + m_lane, tile, la);
                        else
                            tile_load<MODE, FMT>(ta, sb + code_lane, sb + so_full, sb + m_full, tile, la);
                        tile_compute<MODE, FMT>(ta, acc, acc_m, lc);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8u * stage);
            }
            if (++stage == nstage) { stage = 0; phase ^= 1u; }
        }
        while (piece < npieces && alive) { flush(); next_unit(); }
    } else {
        // =============================== reducer =================================================
        // The prepared activations of this CTA's K slice: one barrier, a few large copies.  They are written by
        // the preparation kernel this launch may overlap with, hence the dependency wait first.
        asm volatile("griddepcontrol.wait;" ::: "memory");  // before any global write of this grid
        if (warp == CW + 1 && lane == 0 && !p.prep_inline) {
            const int kbeg = b_first * kBlockK;
            const int kend_full = (b_first + len) * kBlockK;
            const int kend = kend_full < K ? kend_full : K;
            const uint32_t tile0 = (uint32_t)(kbeg / kGroup), ntiles = (uint32_t)((kend - kbeg) / kGroup);
            constexpr uint32_t kRec = MT::kCols ? kColsRecBytes : kPlaneRecBytes;
            // (a bulk copy moves multiples of 16 bytes: an odd number of 136-byte records is rounded up into the slack
            // both buffers keep behind the records)
            const uint32_t rec_bytes = (ntiles * (uint32_t)M * kRec + 15u) & ~15u, sc_bytes = MT::kCols ? 0u : ntiles * (uint32_t)kPlaneSumBytes;
            mbar_arrive_expect_tx(x_bar, rec_bytes + sc_bytes);
            const uint8_t* src = reinterpret_cast<const uint8_t*>(p.xq) + (size_t)tile0 * M * kRec;
            for (uint32_t off = 0; off < rec_bytes; off += 32768u) {
                const uint32_t n = rec_bytes - off < 32768u ? rec_bytes - off : 32768u;
                bulk_g2s(xs + off, src + off, n, x_bar);
            }
            if constexpr (!MT::kCols) {
                const uint8_t* s2 = reinterpret_cast<const uint8_t*>(p.xsc) + (size_t)tile0 * kPlaneSumBytes;
                for (uint32_t off = 0; off < sc_bytes; off += 32768u) {
                    const uint32_t n = sc_bytes - off < 32768u ? sc_bytes - off : 32768u;
                    bulk_g2s(xsc + off, s2 + off, n, x_bar);
                }
            }
        }
        for (int piece = warp - CW - 1; piece < npieces; piece += NR) {
            // pieces in processing order: the partial last strip first (if any), then the strips in order
            const int64_t s = nt > 0 ? (piece == 0 ? s_last : s_first + piece - 1) : s_first + piece;
            const int64_t unit_begin = s * len, unit_end = unit_begin + len;
            const int64_t pa = unit_begin > a ? unit_begin : a;
            const int64_t pe = unit_end < e ? unit_end : e;
            const int par = piece & 1;
            if (!mbar_wait(red_full0 + 8u * par, (piece >> 1) & 1, p.status)) break;
            const float* part_g = reinterpret_cast<const float*>(smem + p.off_part);
            float v[kMaxTokens];
#pragma unroll
            for (int t = 0; t < kMaxTokens; ++t) {
                v[t] = 0.f;
                if (t < M) {
                    constexpr int PT = MT::kCols ? kColsPartTerms : 1;
#pragma unroll
                    for (int w = 0; w < CW; ++w)
#pragma unroll
                        for (int h = 0; h < PT; ++h)
                            v[t] += part_g[(((par * CW + w) * PT + h) * M + t) * kStripRows + lane];
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(red_empty0 + 8u * par);

            const bool whole_unit = (pa == unit_begin) && (pe == unit_end);
            if (p.Z > 1) {
                // K slices: ranges are strip-aligned, every (slice, strip) has one owner; the slices are added by
                // fdqp_splitk_sum_kernel after this grid (fixed order, no arrival counters)
                float* slot = p.ws_full + ((int64_t)z * p.S + s) * (kStripRows * kMaxTokens);
#pragma unroll
                for (int t = 0; t < kMaxTokens; ++t)
                    if (t < M) slot[t * kStripRows + lane] = v[t];
            } else if (whole_unit) {
                if (!EPI) {  // EPI: the bf16 / gated-GELU epilogues are compiled in (plan.epi says which)
                    float* yrow = p.y + s * kStripRows + lane;
#pragma unroll
                    for (int t = 0; t < kMaxTokens; ++t)
                        if (t < M) yrow[(int64_t)t * p.N] = v[t];
                } else {
#pragma unroll
                    for (int t = 0; t < kMaxTokens; ++t)
                        if (t < M) store_output(p.y, p.y16, p.epi, p.N, s, lane, t, v[t]);
                }
            } else {
                float* slot = piece_slot(p, z, ci, s, unit_begin, whole_unit, a);
#pragma unroll
                for (int t = 0; t < kMaxTokens; ++t)
                    if (t < M) slot[t * kStripRows + lane] = v[t];
                __syncwarp();
                // how many pieces does strip s have over all slices?
                int total = p.Z;  // strip-aligned ranges: one whole piece per slice
                if (!p.strip_aligned) {
                    total = 0;
                    for (int zz = 0; zz < p.Z; ++zz) {
                        const int l2 = slice_len(p, zz);
                        const int64_t T2 = (int64_t)p.S * l2;
                        total += (int)(cta_of(s * l2 + l2 - 1, p.Gz, T2) - cta_of(s * l2, p.Gz, T2)) + 1;
                    }
                }
                // release this warp's partial rows and acquire everybody else's in one round trip
                int old = 0;
                if (lane == 0)
                    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(p.tickets + s) : "memory");
                old = __shfl_sync(0xffffffffu, old, 0);
                if (old == total - 1) {
                    // last piece to arrive: add all pieces of the strip in a fixed order
#pragma unroll
                    for (int t = 0; t < kMaxTokens; ++t) v[t] = 0.f;
                    for (int zz = 0; zz < p.Z; ++zz) {
                        const int l2 = slice_len(p, zz);
                        const int64_t T2 = (int64_t)p.S * l2;
                        const int64_t u0 = s * l2;
                        const int64_t cf = p.strip_aligned ? 0 : cta_of(u0, p.Gz, T2);
                        const int64_t cl = p.strip_aligned ? 0 : cta_of(u0 + l2 - 1, p.Gz, T2);
                        for (int64_t c2 = cf; c2 <= cl; ++c2) {
                            const float* src = piece_slot(p, zz, c2, s, u0, cf == cl, range_begin(c2, p.Gz, T2));
#pragma unroll
                            for (int t = 0; t < kMaxTokens; ++t)
                                if (t < M) v[t] += __ldcg(src + t * kStripRows + lane);
                        }
                    }
                    if (!EPI) {  // EPI: the bf16 / gated-GELU epilogues are compiled in (plan.epi says which)
                        float* yrow = p.y + s * kStripRows + lane;
#pragma unroll
                        for (int t = 0; t < kMaxTokens; ++t)
                            if (t < M) yrow[(int64_t)t * p.N] = v[t];
                    } else {
#pragma unroll
                        for (int t = 0; t < kMaxTokens; ++t)
                            if (t < M) store_output(p.y, p.y16, p.epi, p.N, s, lane, t, v[t]);
                    }
                    if (lane == 0) p.tickets[s] = 0;  // ready for the next launch on this stream
                }
            }
        }
    }
}

// Second phase of a K-split projection: y[tok][n] = sum over slices z (ascending) of the slice partials.
// ws is [Z][S][kMaxTokens][32]; one thread per (tok, n).
__global__ void __launch_bounds__(256) fdqp_splitk_sum_kernel(const float* __restrict__ ws, float* __restrict__ y,
                                                               uint16_t* __restrict__ y16, int epi, int Z, int S, int M, int N) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");  // the GEMV grid's partials
    // whole warps stay together (store_output shuffles): M * N is a multiple of 32
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (int64_t)M * N) return;
    const int tok = (int)(idx / N), n = (int)(idx - (int64_t)tok * N);
    const int s = n >> 5, r = n & 31;
    float acc = 0.f;
    for (int z = 0; z < Z; ++z) acc += ws[(((int64_t)z * S + s) * kMaxTokens + tok) * kStripRows + r];
    store_output(y, y16, epi, N, s, r, tok, acc);
}


// RMS normalisation on its own (the calls whose activation preparation does not happen inside a GEMV CTA): one CTA per
// token row, out[m][k] = bf16(x * rsqrt(mean(x^2) + eps) * (1 + gamma[k])).
// residual (may be null): x + residual, rounded once to bf16, is what gets normalised; h_out (may be null) receives it.
__global__ void __launch_bounds__(256) fdqp_rmsnorm_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ residual,
                                                            uint16_t* __restrict__ h_out, const uint16_t* __restrict__ gamma,
                                                            float eps, uint16_t* __restrict__ out, int K) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");  // x may be the previous launch's output
    __shared__ float part[8];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint16_t* xr = x + (int64_t)blockIdx.x * K;
    const uint16_t* rr = residual ? residual + (int64_t)blockIdx.x * K : nullptr;
    uint16_t* orow = out + (int64_t)blockIdx.x * K;
    float ss = 0.f;
    for (int k = tid * 8; k < K; k += 256 * 8) {  // K is a multiple of 32
        uint4 w = *reinterpret_cast<const uint4*>(xr + k);
        if (rr) {
            w = add_bf16x8(w, *reinterpret_cast<const uint4*>(rr + k));
            if (h_out) *reinterpret_cast<uint4*>(h_out + (int64_t)blockIdx.x * K + k) = w;
        }
        const uint32_t xw[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float a = __uint_as_float(xw[i] << 16), b = __uint_as_float(xw[i] & 0xffff0000u);
            ss = fmaf(a, a, ss);
            ss = fmaf(b, b, ss);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) part[warp] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += part[w];
    const float r = rsqrtf(tot / (float)K + eps);
    for (int k = tid * 8; k < K; k += 256 * 8) {
        uint4 w = *reinterpret_cast<const uint4*>(xr + k);
        if (rr) w = add_bf16x8(w, *reinterpret_cast<const uint4*>(rr + k));  // the same sum as in the first pass
        const uint4 g = *reinterpret_cast<const uint4*>(gamma + k);
        const uint32_t xw[4] = {w.x, w.y, w.z, w.w}, gw[4] = {g.x, g.y, g.z, g.w};
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float a = __uint_as_float(xw[i] << 16), b = __uint_as_float(xw[i] & 0xffff0000u);
            const float g0 = 1.0f + __uint_as_float(gw[i] << 16), g1 = 1.0f + __uint_as_float(gw[i] & 0xffff0000u);
            o[i] = (uint32_t)f32_to_bf16_rne(a * r * g0) | ((uint32_t)f32_to_bf16_rne(b * r * g1) << 16);
        }
        *reinterpret_cast<uint4*>(orow + k) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

cudaError_t rmsnorm_launch(const uint16_t* x, const uint16_t* residual, uint16_t* h_out, const uint16_t* gamma, float eps,
                           uint16_t* out, int M, int K, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)M);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fdqp_rmsnorm_kernel, x, residual, h_out, gamma, eps, out, K);
}

// ---- host-visible launchers ------------------------------------------------------------------

template <int CW, int MODE, int BPW>
static cudaError_t launch_one(const GemvPlan& p, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.Z * p.Gz));
    cfg.blockDim = dim3((unsigned)((CW + 1 + CW / 8) * 32));
    cfg.dynamicSmemBytes = p.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;  // may overlap the launch before it (see the kernel)
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return (p.epi == kEpiNone && !p.norm) ? cudaLaunchKernelEx(&cfg, fdqp_gemv_kernel<CW, MODE, BPW, false>, p)
                             : cudaLaunchKernelEx(&cfg, fdqp_gemv_kernel<CW, MODE, BPW, true>, p);
}

cudaError_t xprep_launch(const uint16_t* x, uint32_t* xq, float* xsc, int M, int K, cudaStream_t stream) {
    const int items = (K / kGroup) * M * 4;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((items + 127) / 128));
    cfg.blockDim = dim3(128);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return M <= kColsMaxTokens ? cudaLaunchKernelEx(&cfg, fdqp_xprep_kernel<true>, x, xq, xsc, M, K)
                  : cudaLaunchKernelEx(&cfg, fdqp_xprep_kernel<false>, x, xq, xsc, M, K);
}

cudaError_t splitk_sum_launch(const float* ws, float* y, uint16_t* y16, int epi, int Z, int S, int M, int N,
                              cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(((int64_t)M * N + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fdqp_splitk_sum_kernel, ws, y, y16, epi, Z, S, M, N);
}

// consumer_warps: 8 or 16; p.bpw (blocks per warp per stage): 2 or 4.  Kernel mode by M (see the header).
// The format variants: 16 consumer warps, fp32 output.
template <int FMT>
static cudaError_t launch_fmt(const GemvPlan& p, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.Z * p.Gz));
    cfg.blockDim = dim3((unsigned)((16 + 1 + 2) * 32));
    cfg.dynamicSmemBytes = p.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    const bool b4 = p.bpw == 4;
    if (p.M == 1)
        return b4 ? cudaLaunchKernelEx(&cfg, fdqp_gemv_kernel<16, 1, 4, false, FMT>, p)
                  : cudaLaunchKernelEx(&cfg, fdqp_gemv_kernel<16, 1, 2, false, FMT>, p);
    if (p.M > kColsMaxTokens)
        return b4 ? cudaLaunchKernelEx(&cfg, fdqp_gemv_kernel<16, 2, 4, false, FMT>, p)
                  : cudaLaunchKernelEx(&cfg, fdqp_gemv_kernel<16, 2, 2, false, FMT>, p);
    return b4 ? cudaLaunchKernelEx(&cfg, fdqp_gemv_kernel<16, 3, 4, false, FMT>, p)
              : cudaLaunchKernelEx(&cfg, fdqp_gemv_kernel<16, 3, 2, false, FMT>, p);
}

cudaError_t gemv_launch(const GemvPlan& p, int consumer_warps, cudaStream_t stream) {
    if (p.fmt != kFmtQ4nx) {
        if (consumer_warps != 16 || p.epi != kEpiNone || p.norm) return cudaErrorInvalidValue;
        if (p.fmt == kFmtG64) return launch_fmt<kFmtG64>(p, stream);
        if (p.fmt == kFmtG128) return launch_fmt<kFmtG128>(p, stream);
        if (p.fmt == kFmtMxfp4) return launch_fmt<kFmtMxfp4>(p, stream);
        return cudaErrorInvalidValue;
    }
    const bool w16 = consumer_warps == 16, b4 = p.bpw == 4;
    if (p.M == 1) {
        if (w16) return b4 ? launch_one<16, 1, 4>(p, stream) : launch_one<16, 1, 2>(p, stream);
        return b4 ? launch_one<8, 1, 4>(p, stream) : launch_one<8, 1, 2>(p, stream);
    }
    if (p.M > kColsMaxTokens) {
        if (w16) return b4 ? launch_one<16, 2, 4>(p, stream) : launch_one<16, 2, 2>(p, stream);
        return b4 ? launch_one<8, 2, 4>(p, stream) : launch_one<8, 2, 2>(p, stream);
    }
    if (w16) return b4 ? launch_one<16, 3, 4>(p, stream) : launch_one<16, 3, 2>(p, stream);
    return b4 ? launch_one<8, 3, 4>(p, stream) : launch_one<8, 3, 2>(p, stream);
}

template <int CW, int MODE>
static cudaError_t set_smem_limit_mode(int bytes) {
    const cudaFuncAttribute a = cudaFuncAttributeMaxDynamicSharedMemorySize;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(fdqp_gemv_kernel<CW, MODE, 2, false>, a, bytes))) return e;
    if ((e = cudaFuncSetAttribute(fdqp_gemv_kernel<CW, MODE, 4, false>, a, bytes))) return e;
    if ((e = cudaFuncSetAttribute(fdqp_gemv_kernel<CW, MODE, 2, true>, a, bytes))) return e;
    return cudaFuncSetAttribute(fdqp_gemv_kernel<CW, MODE, 4, true>, a, bytes);
}

template <int FMT>
static cudaError_t set_smem_limit_fmt(int bytes) {
    const cudaFuncAttribute a = cudaFuncAttributeMaxDynamicSharedMemorySize;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(fdqp_gemv_kernel<16, 1, 2, false, FMT>, a, bytes))) return e;
    if ((e = cudaFuncSetAttribute(fdqp_gemv_kernel<16, 1, 4, false, FMT>, a, bytes))) return e;
    if ((e = cudaFuncSetAttribute(fdqp_gemv_kernel<16, 2, 2, false, FMT>, a, bytes))) return e;
    if ((e = cudaFuncSetAttribute(fdqp_gemv_kernel<16, 2, 4, false, FMT>, a, bytes))) return e;
    if ((e = cudaFuncSetAttribute(fdqp_gemv_kernel<16, 3, 2, false, FMT>, a, bytes))) return e;
    return cudaFuncSetAttribute(fdqp_gemv_kernel<16, 3, 4, false, FMT>, a, bytes);
}

cudaError_t gemv_set_smem_limit(int bytes) {
    cudaError_t e;
    if ((e = set_smem_limit_fmt<kFmtG64>(bytes))) return e;
    if ((e = set_smem_limit_fmt<kFmtG128>(bytes))) return e;
    if ((e = set_smem_limit_fmt<kFmtMxfp4>(bytes))) return e;
    if ((e = set_smem_limit_mode<8, 1>(bytes))) return e;
    if ((e = set_smem_limit_mode<16, 1>(bytes))) return e;
    if ((e = set_smem_limit_mode<8, 2>(bytes))) return e;
    if ((e = set_smem_limit_mode<16, 2>(bytes))) return e;
    if ((e = set_smem_limit_mode<8, 3>(bytes))) return e;
    return set_smem_limit_mode<16, 3>(bytes);
}

}  // namespace fdqp
