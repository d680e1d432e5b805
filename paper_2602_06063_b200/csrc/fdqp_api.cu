// C ABI of the FusedDQP library: context, argument checks, launch planning and dispatch.
// Every operation of the projection runs in the CUDA kernels; nothing here computes on the host
// and there is no fallback when the device is not an sm_100 part.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "fdqp.h"
#include "fdqp_format.h"
#include "fdqp_plan.h"

namespace fdqp {
cudaError_t gemv_launch(const GemvPlan& p, int consumer_warps, cudaStream_t stream);
cudaError_t gemv_set_smem_limit(int bytes);
cudaError_t splitk_sum_launch(const float* ws, float* y, uint16_t* y16, int epi, int Z, int S, int M, int N,
                              cudaStream_t stream);
cudaError_t xprep_launch(const uint16_t* x, uint32_t* xq, float* xsc, int M, int K, cudaStream_t stream);
cudaError_t dequant_launch(const uint8_t* W, void* out, bool out_bf16, int K, int N, cudaStream_t stream);
cudaError_t dequant_fmt_launch(int fmt, const uint8_t* W, void* out, bool out_bf16, int K, int N, cudaStream_t stream);
cudaError_t prefill_set_smem_limit();
cudaError_t prefill_launch(const uint8_t* W, const uint16_t* x, int64_t x_row_bytes, float* y, uint16_t* y16, int epi, float* ws,
                           int* status, int M, int K, int N, int pair, int Z, int fmt, int a_tmem, cudaStream_t stream,
                           int* kernels_launched);
cudaError_t rmsnorm_launch(const uint16_t* x, const uint16_t* residual, uint16_t* h_out, const uint16_t* gamma, float eps,
                           uint16_t* out, int M, int K, cudaStream_t stream);
cudaError_t flowkv_launch(const uint16_t* q, const uint16_t* K, const uint16_t* V, float* out, float* ws, int max_splits, int H,
                          int G, int d, int L, int pitch, int window, float scale, int sm_count, int cluster_max_positions,
                          int* launches, cudaStream_t stream);
cudaError_t plain_launch(const uint8_t* W, const uint16_t* x, float* y, int M, int K, int N, cudaStream_t stream);
cudaError_t stream_read_launch(const uint8_t* buf, int64_t bytes, int sm_count, int* status, cudaStream_t stream);
cudaError_t wait_selftest_launch(int* status, unsigned long long limit_ns, cudaStream_t stream);
cudaError_t chain_set_smem_limit(int bytes);
cudaError_t chain_launch(const ChainPlan& cp, int grid, bool epi, int launch_mode, cudaStream_t stream);
}  // namespace fdqp

using namespace fdqp;

constexpr int kFlowKvClusterPositions = 2048;  // default of the "flowkv_cluster" parameter

struct fdqp_ctx {
    int device = 0;
    int sm_count = 0;
    int smem_optin = 0;
    int64_t max_M = 0, max_K = 0, max_N = 0;
    float* ws_edge = nullptr;
    float* ws_full = nullptr;
    float* pf_ws = nullptr;      // partial results of K-split tensor-core calls
    float* kv_ws = nullptr;      // decode attention: per (query head, split) partial results
    uint16_t* x_norm = nullptr;  // normalised activations of calls whose RMS normalisation cannot be fused (max_M x max_K)
    uint8_t* x_spread = nullptr; // small x copied with its rows further apart (see kSpreadBelowBytes)
    size_t pf_ws_bytes = 0;
    int* tickets = nullptr;
    uint32_t* xq = nullptr;      // prepared activations of the call in flight
    float* xsc = nullptr;
    int* status_host = nullptr;  // pinned, mapped
    int* status_dev = nullptr;   // device alias of status_host
    void* x_stage = nullptr;     // fdqp_run_host staging (allocated on its first use)
    float* y_stage = nullptr;
    int64_t launches = 0;
    std::string last_err;
    // overrides (-1 = automatic)
    int64_t p_path = -1, p_ctas_per_sm = -1, p_cw = -1, p_stages = -1, p_split_k = -1, p_evict = -1, p_prep = -1, p_aligned = -1, p_bpw = -1, p_pair = -1, p_pf_split = -1;
    // fdqp_run_chain: partial rows of shared strips (2 per CTA and step), of whole strip-slices, arrival counters per
    // (step, strip), and the per-step completion counters followed by the exit counter
    float* chain_edge = nullptr;
    float* chain_full = nullptr;
    int* chain_tickets = nullptr;
    int* chain_done = nullptr;
    size_t chain_ticket_cap = 0;
    int64_t p_chain_launch = 1, p_chain_steps = kMaxChainSteps, p_chain_wide = 1, p_chain_dep = 0;
    int64_t p_flowkv_cluster = kFlowKvClusterPositions;  // ranges up to this many positions take the one-launch attention
    int64_t p_direct_y = 1;  // fdqp_run_host*: small results are stored straight into device-addressable host memory
    int64_t p_atmem = 1;  // tensor-core kernel up to 128 tokens: keep the converted weights in tensor memory
};

namespace {

constexpr int kMaxStages = 40;
// Measured on B200: while all of x is smaller than 128 KB, the tensor-core kernels (every CTA re-reads the same few rows
// of x by TMA at every k-step) run 1.45x slower; with the same rows placed further apart, so that they cover at least
// 256 KB of addresses, the slow-down is gone.  Such an x is therefore copied into a spread-out staging buffer first.
constexpr int64_t kSpreadBelowBytes = 128 << 10;
constexpr int64_t kSpreadToBytes = 256 << 10;
constexpr size_t kSpreadBufBytes = (size_t)kSpreadToBytes + 256 * 128;  // row distance rounds up to 128 bytes, M <= 256 here
constexpr int64_t kPrefillMinK = 256;          // shortest reduction the dispatch gives to the tensor-core kernels
constexpr size_t kDirectHostBytes = 1u << 20;  // results up to this size go straight to addressable host memory
constexpr int kKvMaxHeads = 64, kKvMaxSplits = 148, kKvMaxDim = 256;  // decode attention workspace
constexpr size_t kPrefillWsCap = 128u << 20;  // bytes of partial results a context keeps for K-split tensor-core calls
constexpr int kMinStages = 3;  // ring depth below which another K slice is preferred
// fdqp_run_chain: shared memory a step's prepared activations may take (K is cut into slices beyond it), activation
// items (8 values) one CTA prepares per step at most, and the partial-row slots for steps with K slices
constexpr uint32_t kChainXsCap = 64u << 10;
constexpr int kChainPrepItems = 8 * 16 * 32;
constexpr size_t kChainFullSlots = 16384;

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) == cudaSuccess && (prev == dev || cudaSetDevice(dev) == cudaSuccess)) ok = true;
        if (prev == dev) prev = -1;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

fdqp_status cuda_fail(fdqp_ctx* ctx, cudaError_t e, const char* what) {
    if (ctx) ctx->last_err = std::string(what) + ": " + cudaGetErrorString(e);
    cudaGetLastError();  // clear the sticky-less error state
    return e == cudaErrorMemoryAllocation ? FDQP_ERR_NOMEM : FDQP_ERR_CUDA;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline uint32_t round_up(uint32_t v, uint32_t a) { return (v + a - 1) / a * a; }

fdqp_status check_shape(const fdqp_ctx* ctx, int64_t M, int64_t K, int64_t N) {
    if (M < 1 || K <= 0 || N <= 0 || (K % kGroup) != 0 || (N % kStripRows) != 0) return FDQP_ERR_SHAPE;
    if (M > ctx->max_M || K > ctx->max_K || N > ctx->max_N) return FDQP_ERR_SIZE;
    return FDQP_OK;
}

// More than 256 token rows: a pair of SMs works on a 256 x 512 tile (every converted weight serves 512 tokens).
bool use_pair(const fdqp_ctx* ctx, int64_t M) { return ctx->p_pair >= 0 ? ctx->p_pair != 0 : M > 256; }

// Time model of a tensor-core call cut into Z K slices (microseconds, without the launch and the optional spreading
// copy; constants measured on B200).  A CTA (pair) costs about c per 64-wide k-step when its SM is full: c = 0.64 up to
// 64 tokens rising to 0.72 at 128 (128-row tiles, two CTAs per SM), 0.78 (256-row tiles, one CTA per SM), 0.95 (two-SM
// kernel).  The busiest SM runs n = ceil(CTAs / SMs) of them, two at a time where two fit; a CTA that has the SM to
// itself runs its k-steps in about 0.7 of that time.  Z > 1 adds the second kernel (2-3 us on the stream: it overlaps the first one's tail) and the partial results:
// written by the slices, read and summed by the second kernel.
double prefill_time_model(const fdqp_ctx* ctx, int64_t M, int64_t K, int64_t N, int64_t Z) {
    const bool pair = use_pair(ctx, M);
    const bool small = !pair && M <= 128;
    const int64_t tiles = pair ? ((N + 255) / 256) * ((M + 511) / 512)
                               : (small ? (N + 127) / 128 : ((N + 255) / 256) * ((M + 255) / 256));
    const int64_t units = pair ? ctx->sm_count / 2 : ctx->sm_count;
    const int64_t n = (tiles * Z + units - 1) / units;
    const double rounds = small ? (double)(n / 2) + ((n & 1) ? 0.7 : 0.0) : (double)n;
    const double c = pair ? 0.95 : (M <= 64 ? 0.64 : (M <= 128 ? 0.64 + 0.08 * (double)(M - 64) / 64.0 : 0.78));
    const int64_t kz = ((K + 63) / 64 + Z - 1) / Z;
    double t = rounds * (double)kz * c;
    if (Z > 1) t += 2.5 + (double)(2 * Z + 1) * (double)M * (double)N * 4.0 / 5.0e6;
    return t;
}

// K slices of a tensor-core call: the count the time model likes best (a larger count has to win by 8 %), while every
// slice keeps at least eight 64-wide k-steps and the partial results fit the context's workspace.  Few tiles (27B down:
// 42 of 128 rows) get as many slices as fill the SMs once; a tile count just above a multiple of the slots (12B-like
// K = 5376, N = 43008 at M = 32: 336 CTAs on 296 slots) gets the slices that even out the last round (85 -> 70 us).
int prefill_slices(const fdqp_ctx* ctx, int64_t M, int64_t K, int64_t N) {
    const int64_t ksteps = (K + 63) / 64;
    int64_t zmax = kMaxSplit;
    if (zmax > ksteps / 8) zmax = ksteps / 8;
    const int64_t fit = (int64_t)(ctx->pf_ws_bytes / ((size_t)M * (size_t)N * 4));
    if (zmax > fit) zmax = fit;
    if (zmax < 1) zmax = 1;
    if (ctx->p_pf_split > 0) return (int)(ctx->p_pf_split < zmax ? ctx->p_pf_split : zmax);
    int64_t best = 1;
    double t_best = prefill_time_model(ctx, M, K, N, 1);
    for (int64_t Z = 2; Z <= zmax; ++Z) {
        const double t = prefill_time_model(ctx, M, K, N, Z);
        if (t < 0.95 * t_best) {
            best = Z;
            t_best = t;
        }
    }
    return (int)best;
}

// Up to 128 tokens the one-SM kernel keeps the converted weights in tensor memory (mode 1, two CTAs per SM).  Up to 64
// tokens a variant with half the accumulator columns, two weight stages and a four-deep weight prefetch (64 registers)
// fits three CTAs per SM (mode 2): 6 % faster when the call has at least three CTAs per SM to run (LM head 181 -> 170 us),
// slower when it has not (12B gate|up at M = 32: 44 -> 47 us), so the automatic choice asks for that many.
int prefill_tmem_mode(const fdqp_ctx* ctx, int64_t M, int64_t K, int64_t N) {
    if (ctx->p_atmem != 1) return (int)ctx->p_atmem;
    if (M > 64) return 1;
    const int64_t ctas = ((N + 127) / 128) * prefill_slices(ctx, M, K, N);
    return ctas >= 3 * (int64_t)ctx->sm_count ? 2 : 1;
}

// M >= 9: the tensor-core kernels, or the GEMV kernel eight token rows at a time -- whichever a small cost model
// (microseconds, constants measured on B200) says is faster.
//   GEMV: every chunk streams the whole matrix, at about 5.5 TB/s for 1-2 rows, 3.9 for 3-4, 3.2 for 5-8, plus ~8 us
//   (back-to-back chunks of a small matrix: 2 x 15 us for 16 MB).
//   Tensor-core kernels: prefill_time_model above.
bool use_prefill(const fdqp_ctx* ctx, int64_t M, int64_t K, int64_t N) {
    if (M <= kMaxTokens || ctx->p_path == 2) return false;
    if (ctx->p_path == 3) return true;
    // The tensor-core kernels multiply by bf16-rounded weights (relative error up to 2^-8 per weight).  Against the
    // acceptance bound 2e-3 * sum|x w| that is safe only where the K terms' rounding errors average out: with K = 32 two
    // of 40,000 outputs were seen just outside it.  Short reductions therefore stay on the GEMV kernels (fp32 weights).
    if (K < kPrefillMinK) return false;
    const double mb = 0.625 * (double)K * (double)N / 1.0e6;  // packed weights, bytes per microsecond = TB/s * 1e6
    const int64_t last = M % kMaxTokens;                       // rows of the ragged last chunk (0: none)
    const double last_rate = last <= 2 ? 5.5 : (last <= 4 ? 3.9 : 3.2);
    const double t_gemv = (double)(M / kMaxTokens) * (8.0 + mb / 3.2) + (last ? 8.0 + mb / last_rate : 0.0);
    double t_tensor = 5.0 + prefill_time_model(ctx, M, K, N, prefill_slices(ctx, M, K, N));
    if (prefill_tmem_mode(ctx, M, K, N) == 2) t_tensor *= 0.94;  // three CTAs per SM
    if (M * K * 2 < kSpreadBelowBytes) t_tensor += 3.0;                                   // the spreading copy
    return t_tensor < t_gemv;
}

// Shared-memory carve-up for a given configuration; returns the ring depth that fits (0 if none).
struct SmemLayout {
    uint32_t stage_bytes, xs_bytes, xsum_bytes, part_bytes, fixed;
    int nstage;
};

SmemLayout smem_layout(const fdqp_ctx* ctx, int M, int nbz, int cw, int ctas_per_sm, int bpw, int fmt) {
    SmemLayout L;
    L.stage_bytes = (uint32_t)(cw / 8) * (uint32_t)bpw * (uint32_t)fmt_block_bytes(fmt);
    const uint32_t tiles = (uint32_t)nbz * 8u;
    L.xs_bytes = tiles * (uint32_t)(M <= kColsMaxTokens ? kColsRecBytes : kPlaneRecBytes) * (uint32_t)M;  // prepared activations of the K slice
    L.xsum_bytes = M <= kColsMaxTokens ? 0u : tiles * (uint32_t)kPlaneSumBytes;  // per-token sums of x (M >= 3 only)
    L.part_bytes = 2u * (uint32_t)cw * kStripRows * (uint32_t)M * 4u * (M <= kColsMaxTokens ? (uint32_t)kColsPartTerms : 1u);
    L.fixed = round_up(L.xs_bytes, 128) + round_up(L.xsum_bytes, 128) + round_up(L.part_bytes, 128) +
              (2u * kMaxStages + 6u) * 8u + 512u + 128u;
    const uint32_t per_cta = (uint32_t)ctx->smem_optin / (uint32_t)ctas_per_sm - (ctas_per_sm > 1 ? 1024u : 0u);
    L.nstage = per_cta > L.fixed ? (int)((per_cta - L.fixed) / L.stage_bytes) : 0;
    if (L.nstage > kMaxStages) L.nstage = kMaxStages;
    return L;
}

// Fill the launch plan of one GEMV launch (M <= 8).  Returns false if no ring fits.
bool plan_gemv(const fdqp_ctx* ctx, int M, int K, int N, int* consumer_warps, GemvPlan* p, int fmt = kFmtQ4nx) {
    std::memset(p, 0, sizeof(*p));
    p->fmt = fmt;
    p->M = M;
    p->K = K;
    p->N = N;
    p->S = N / kStripRows;
    p->nb = (K + kBlockK - 1) / kBlockK;
    // measured on B200: one 19-warp CTA per SM (one start-up per SM, all of its shared memory) is the better shape at
    // every size; two 10-warp CTAs per SM remain available as a launch parameter
    int ctas_per_sm = ctx->p_ctas_per_sm > 0 ? (int)ctx->p_ctas_per_sm : 1;
    if (ctas_per_sm > kMaxCtasPerSm) ctas_per_sm = kMaxCtasPerSm;
    if (fmt != kFmtQ4nx) ctas_per_sm = 1;  // the variants are built for the 16-consumer-warp shape only
    int cw = 16, Z = 1, nbz = p->nb, bpw = 2;
    SmemLayout L{};
    for (;; --ctas_per_sm) {
        // register file: one 19-warp CTA or two 10-warp CTAs fit an SM
        cw = ctas_per_sm > 1 ? 8 : ((ctx->p_cw == 8 || ctx->p_cw == 16) ? (int)ctx->p_cw : 16);
        if (fmt != kFmtQ4nx) cw = 16;
        // K slices: as few as leave a ring of at least kMinStages stages beside the staged activations
        Z = ctx->p_split_k > 0 ? (int)ctx->p_split_k : 1;
        for (;; Z *= 2) {
            if (Z > p->nb) Z = p->nb;
            nbz = (p->nb + Z - 1) / Z;
            // four blocks per warp per stage halve the barrier traffic per tile
            const int64_t blocks_per_cta = (int64_t)p->S * p->nb / ((int64_t)ctx->sm_count * ctas_per_sm);
            // (measured: LM head 68 against 91 us at M = 1, 101 against 119 us at M = 8; never when the larger stage would
            // force a K split)
            bpw = ctx->p_bpw == 2 || ctx->p_bpw == 4 ? (int)ctx->p_bpw : (blocks_per_cta >= 4 ? 4 : 2);
            L = smem_layout(ctx, M, nbz, cw, ctas_per_sm, bpw, fmt);
            if (bpw == 4 && ctx->p_bpw != 4 && L.nstage < kMinStages) {
                // The larger stages do not fit beside this slice's activations.  Another K slice keeps them (measured on
                // the 27B down projection, K = 21504: M = 4 23.3 us with four slices against 32.7 us with two slices
                // and the smaller stages; M = 3 23.1 against 27.2, M = 8 24.9 against 29.4); the smaller stages are
                // what is left when K cannot be cut further.
                if (ctx->p_split_k <= 0 && Z * 2 <= kMaxSplit && Z * 2 <= p->nb) continue;
                bpw = 2;
                L = smem_layout(ctx, M, nbz, cw, ctas_per_sm, bpw, fmt);
            }
            if (L.nstage >= kMinStages || Z >= kMaxSplit || Z >= p->nb) break;
        }
        if (L.nstage >= 2 || ctas_per_sm == 1) break;
    }
    if (L.nstage < 2) return false;
    // K slices are strip-aligned, so the busiest CTA of a slice works on ceil(strips / CTAs of the slice) whole strip
    // slices: with few strips per CTA the number of slices decides how uneven that is (27B down, 168 strips: 3 x 42 blocks
    // with two slices, 5 x 21 with four, 10 x 11 with eight; measured at M = 3: 26.0 / 23.0 / 23.8 us).  Once K has to be
    // cut, take the count, up to four times the necessary one, whose busiest CTA has the least to do.
    if (Z > 1 && ctx->p_split_k <= 0) {
        const int grid_all = ctx->sm_count * ctas_per_sm;
        auto busiest = [&](int z) {
            const int nbz_c = (p->nb + z - 1) / z;
            const int z_eff = (p->nb + nbz_c - 1) / nbz_c;
            int gz = grid_all / z_eff;
            if (gz < 1) gz = 1;
            if (gz > p->S) gz = (int)p->S;
            return (int64_t)((p->S + gz - 1) / gz) * nbz_c;
        };
        int best = Z;
        for (int cand = Z * 2; cand <= Z * 4 && cand <= kMaxSplit && cand <= p->nb; cand *= 2)
            if (busiest(cand) < busiest(best)) best = cand;
        if (best != Z) {
            Z = best;
            nbz = (p->nb + Z - 1) / Z;
            L = smem_layout(ctx, M, nbz, cw, ctas_per_sm, bpw, fmt);  // (a shorter slice: at least as many stages)
        }
    }
    Z = (p->nb + nbz - 1) / nbz;  // drop slices that would be empty
    p->Z = Z;
    p->nbz = nbz;
    int grid = ctx->sm_count * ctas_per_sm;
    const int64_t total_blocks = (int64_t)p->S * p->nb;
    if (grid > total_blocks) grid = (int)total_blocks;
    int Gz = grid / Z;
    if (Gz < 1) Gz = 1;
    // Equal block counts per CTA keep every SM streaming, but a strip shared by two CTAs is finished through
    // global memory (~2 us on the critical path unless the CTA also owns whole strips to do afterwards).  Cutting at
    // strip boundaries avoids that at the price of imbalance.  Estimate both (us) and take the cheaper.
    {
        // Time to stream the busiest CTA's blocks (us): an SM alone pulls a 5 KB block in about 0.085 us (60 GB/s), all SMs
        // together are held to the HBM rate (0.79 ns per block over the whole grid) -- so when few CTAs have work, or the
        // work is uneven, the busiest one is not slowed down by the others' share.
        const double t_sm = 0.085 * ctas_per_sm, t_all = (double)(total_blocks / Z) * 5120.0 / 6.5e6;
        const int64_t blocks_bal = (total_blocks / Z + Gz - 1) / Gz;
        // (measured: ranges cut inside strips also stream 3-4 % slower -- strip boundaries then fall at odd places inside
        // the stages, and more stages take the bookkeeping path)
        const double stream_bal = (double)blocks_bal * t_sm > t_all ? (double)blocks_bal * t_sm : t_all;
        const double cost_bal = stream_bal * 1.04 + (blocks_bal >= 2 * (int64_t)nbz ? 1.0 : 2.0);
        const int Ga = Gz < p->S ? Gz : p->S;
        const int64_t blocks_al = (int64_t)((p->S + Ga - 1) / Ga) * nbz;
        // (when the grid as a whole is held to the HBM rate, what the busiest CTA has beyond the average it streams
        // alone, at its own rate, after the others have finished)
        const double beyond = (double)blocks_al - (double)(total_blocks / Z) / (double)Ga;
        const double held = t_all + (beyond > 0 ? beyond : 0) * t_sm;
        const double stream_al = (double)blocks_al * t_sm > held ? (double)blocks_al * t_sm : held;
        const double cost_al = stream_al + (Z > 1 ? 2.0 : 0.4);
        // K slices are always strip-aligned: every (slice, strip) then has one owner and the slices are added by a
        // second small kernel instead of through arrival counters
        const bool aligned = Z > 1 || (ctx->p_aligned >= 0 ? ctx->p_aligned != 0 : cost_al < cost_bal);
        p->strip_aligned = aligned ? 1 : 0;
        if (aligned) Gz = Ga;
    }
    p->Gz = Gz;
    int nstage = L.nstage;
    if (ctx->p_stages > 0 && ctx->p_stages < nstage) nstage = (int)ctx->p_stages;
    p->nstage = nstage;
    p->bpw = bpw;
    p->off_xs = (uint32_t)nstage * L.stage_bytes;
    p->off_xsum = p->off_xs + round_up(L.xs_bytes, 128);
    p->off_part = p->off_xsum + round_up(L.xsum_bytes, 128);
    p->off_bar = p->off_part + round_up(L.part_bytes, 128);
    p->smem_bytes = p->off_bar + (2u * (uint32_t)nstage + 6u) * 8u + 512u;  // barriers, then the fused normalisation's sums
    p->evict_first = ctx->p_evict >= 0 ? (ctx->p_evict != 0) : 1;
    // work items (8 activations each) per CTA if x is prepared in-kernel; beyond this a preparation kernel is cheaper
    p->prep_inline = ctx->p_prep >= 0 ? (int)(ctx->p_prep != 0) : ((int64_t)nbz * 8 * M * 4 <= (int64_t)2 * cw * 32);
    p->ws_edge = ctx->ws_edge;
    p->ws_full = ctx->ws_full;
    p->tickets = ctx->tickets;
    p->xq = ctx->xq;
    p->xsc = ctx->xsc;
    p->status = ctx->status_dev;
    *consumer_warps = cw;
    return true;
}

}  // namespace

extern "C" const char* fdqp_status_string(fdqp_status s) {
    switch (s) {
        case FDQP_OK: return "ok";
        case FDQP_ERR_ARG: return "bad argument";
        case FDQP_ERR_SHAPE: return "bad shape (M >= 1, K and N positive multiples of 32)";
        case FDQP_ERR_ALIGN: return "pointer not 16-byte aligned";
        case FDQP_ERR_SIZE: return "size beyond buffer or context maxima";
        case FDQP_ERR_ARCH: return "device is not compute capability 10.x";
        case FDQP_ERR_CUDA: return "CUDA runtime error";
        case FDQP_ERR_NOMEM: return "out of memory";
        case FDQP_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    }
    return "unknown status";
}

extern "C" fdqp_status fdqp_create(fdqp_ctx** out, int device, int64_t max_M, int64_t max_K, int64_t max_N) {
    if (!out) return FDQP_ERR_ARG;
    *out = nullptr;
    if (max_M < 1 || max_K <= 0 || max_N <= 0 || (max_K % kGroup) != 0 || (max_N % kStripRows) != 0)
        return FDQP_ERR_SHAPE;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
        cudaGetLastError();
        return FDQP_ERR_CUDA;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return FDQP_ERR_CUDA;
    if (prop.major != 10) return FDQP_ERR_ARCH;  // sm_100a code only; no other path exists
    DeviceGuard guard(device);
    if (!guard.ok) return FDQP_ERR_CUDA;
    fdqp_ctx* ctx = new (std::nothrow) fdqp_ctx();
    if (!ctx) return FDQP_ERR_NOMEM;
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    ctx->smem_optin = (int)prop.sharedMemPerBlockOptin;
    ctx->max_M = max_M;
    ctx->max_K = max_K;
    ctx->max_N = max_N;
    const int64_t S = max_N / kStripRows;
    const size_t slot = sizeof(float) * kStripRows * kMaxTokens;
    cudaError_t e;
    fdqp_status st = FDQP_OK;
    do {
        if ((e = cudaMalloc(&ctx->ws_edge, slot * 2 * (size_t)ctx->sm_count * kMaxCtasPerSm))) { st = cuda_fail(nullptr, e, ""); break; }
        if ((e = cudaMalloc(&ctx->ws_full, slot * (size_t)kMaxSplit * (size_t)S))) { st = cuda_fail(nullptr, e, ""); break; }
        if ((e = cudaMalloc(&ctx->tickets, sizeof(int) * (size_t)S))) { st = cuda_fail(nullptr, e, ""); break; }
        if ((e = cudaMalloc(&ctx->kv_ws, (size_t)kKvMaxHeads * kKvMaxSplits * (kKvMaxDim + 4) * 4))) { st = cuda_fail(nullptr, e, ""); break; }
        if ((e = cudaMalloc(&ctx->x_norm, (size_t)max_M * (size_t)max_K * 2))) { st = cuda_fail(nullptr, e, ""); break; }
        if (max_M > kMaxTokens) {
            // K-split tensor-core calls (shapes with few output tiles): up to kMaxSplit partial results, capped
            const size_t want = (size_t)kMaxSplit * (size_t)max_M * (size_t)max_N * 4;
            ctx->pf_ws_bytes = want < kPrefillWsCap ? want : kPrefillWsCap;
            if ((e = cudaMalloc(&ctx->pf_ws, ctx->pf_ws_bytes))) { st = cuda_fail(nullptr, e, ""); break; }
            if ((e = cudaMalloc(&ctx->x_spread, kSpreadBufBytes))) { st = cuda_fail(nullptr, e, ""); break; }
        }
        if ((e = cudaMemset(ctx->tickets, 0, sizeof(int) * (size_t)S))) { st = cuda_fail(nullptr, e, ""); break; }
        const size_t tiles = (size_t)(max_K / kGroup), toks = (size_t)(max_M < kMaxTokens ? max_M : kMaxTokens);
        if ((e = cudaMalloc(&ctx->xq, tiles * toks * kColsRecBytes + 16))) { st = cuda_fail(nullptr, e, ""); break; }
        if ((e = cudaMalloc(&ctx->xsc, tiles * 64))) { st = cuda_fail(nullptr, e, ""); break; }
        if ((e = cudaMemset(ctx->xq, 0, tiles * toks * kColsRecBytes + 16))) { st = cuda_fail(nullptr, e, ""); break; }
        if ((e = cudaMemset(ctx->xsc, 0, tiles * 64))) { st = cuda_fail(nullptr, e, ""); break; }
        if ((e = cudaHostAlloc(&ctx->status_host, sizeof(int), cudaHostAllocMapped))) { st = cuda_fail(nullptr, e, ""); break; }
        *ctx->status_host = 0;
        if ((e = cudaHostGetDevicePointer(&ctx->status_dev, ctx->status_host, 0))) { st = cuda_fail(nullptr, e, ""); break; }
        {
            const size_t slot_b = sizeof(float) * kStripRows * kMaxTokens;
            ctx->chain_ticket_cap = (size_t)16 * (size_t)S < 65536 ? 65536 : (size_t)16 * (size_t)S;
            if ((e = cudaMalloc(&ctx->chain_edge, slot_b * 2 * (size_t)ctx->sm_count * kChainEdgeSteps))) { st = cuda_fail(nullptr, e, ""); break; }
            if ((e = cudaMalloc(&ctx->chain_full, slot_b * kChainFullSlots))) { st = cuda_fail(nullptr, e, ""); break; }
            if ((e = cudaMalloc(&ctx->chain_tickets, sizeof(int) * ctx->chain_ticket_cap))) { st = cuda_fail(nullptr, e, ""); break; }
            if ((e = cudaMalloc(&ctx->chain_done, sizeof(int) * (kMaxChainSteps + 1)))) { st = cuda_fail(nullptr, e, ""); break; }
            if ((e = cudaMemset(ctx->chain_tickets, 0, sizeof(int) * ctx->chain_ticket_cap))) { st = cuda_fail(nullptr, e, ""); break; }
            if ((e = cudaMemset(ctx->chain_done, 0, sizeof(int) * (kMaxChainSteps + 1)))) { st = cuda_fail(nullptr, e, ""); break; }
        }
        if ((e = chain_set_smem_limit(ctx->smem_optin))) { st = cuda_fail(nullptr, e, ""); break; }
        if ((e = gemv_set_smem_limit(ctx->smem_optin))) { st = cuda_fail(nullptr, e, ""); break; }
        if ((e = prefill_set_smem_limit())) { st = cuda_fail(nullptr, e, ""); break; }
        if ((e = cudaDeviceSynchronize())) { st = cuda_fail(nullptr, e, ""); break; }
    } while (false);
    if (st != FDQP_OK) {
        fdqp_destroy(ctx);
        return st;
    }
    *out = ctx;
    return FDQP_OK;
}

extern "C" fdqp_status fdqp_destroy(fdqp_ctx* ctx) {
    if (!ctx) return FDQP_OK;
    DeviceGuard guard(ctx->device);
    if (ctx->ws_edge) cudaFree(ctx->ws_edge);
    if (ctx->ws_full) cudaFree(ctx->ws_full);
    if (ctx->pf_ws) cudaFree(ctx->pf_ws);
    if (ctx->x_spread) cudaFree(ctx->x_spread);
    if (ctx->x_norm) cudaFree(ctx->x_norm);
    if (ctx->kv_ws) cudaFree(ctx->kv_ws);
    if (ctx->tickets) cudaFree(ctx->tickets);
    if (ctx->chain_edge) cudaFree(ctx->chain_edge);
    if (ctx->chain_full) cudaFree(ctx->chain_full);
    if (ctx->chain_tickets) cudaFree(ctx->chain_tickets);
    if (ctx->chain_done) cudaFree(ctx->chain_done);
    if (ctx->xq) cudaFree(ctx->xq);
    if (ctx->xsc) cudaFree(ctx->xsc);
    if (ctx->x_stage) cudaFree(ctx->x_stage);
    if (ctx->y_stage) cudaFree(ctx->y_stage);
    if (ctx->status_host) cudaFreeHost(ctx->status_host);
    cudaGetLastError();
    delete ctx;
    return FDQP_OK;
}

namespace {

// The projection with its epilogue: `out` is fp32 [M][N] (kEpiNone), bf16 [M][N] (kEpiBf16) or bf16 [M][N/2]
// (kEpiGegluBf16).
// gamma != nullptr: x is RMS-normalised first, x <- bf16(x * rsqrt(mean_k x^2 + eps) * (1 + gamma)) per token row --
// inside the GEMV kernel's activation preparation when that runs in-kernel on the whole row, else by a kernel of its own.
fdqp_status run_impl(fdqp_ctx* ctx, const void* x_bf16, const void* gamma_bf16, float eps, const void* W_q4nx, void* out,
                     int epi, int64_t M, int64_t K, int64_t N, void* cuda_stream, int fmt = kFmtQ4nx,
                     const void* residual_bf16 = nullptr, void* h_out_bf16 = nullptr) {
    if (!ctx || !x_bf16 || !W_q4nx || !out) return FDQP_ERR_ARG;
    if ((residual_bf16 || h_out_bf16) && !gamma_bf16) return FDQP_ERR_ARG;
    if (h_out_bf16 && !residual_bf16) return FDQP_ERR_ARG;
    if (h_out_bf16 && (h_out_bf16 == x_bf16 || h_out_bf16 == residual_bf16)) return FDQP_ERR_ARG;  // read by every CTA
    if ((residual_bf16 && !aligned16(residual_bf16)) || (h_out_bf16 && !aligned16(h_out_bf16))) return FDQP_ERR_ALIGN;
    if (fmt < 0 || fmt >= kFmtCount) return FDQP_ERR_ARG;
    if (fmt != kFmtQ4nx && (K % kBlockK) != 0) return FDQP_ERR_SHAPE;           // the variants hold whole blocks only
    if (fmt != kFmtQ4nx && (epi != kEpiNone || gamma_bf16)) return FDQP_ERR_ARG;  // ... and have the fp32 store only
    if (gamma_bf16 && !aligned16(gamma_bf16)) return FDQP_ERR_ALIGN;
    if (gamma_bf16 && !(eps >= 0.f)) return FDQP_ERR_ARG;
    if (epi != kEpiNone && epi != kEpiBf16 && epi != kEpiGegluBf16) return FDQP_ERR_ARG;
    fdqp_status st = check_shape(ctx, M, K, N);
    if (st != FDQP_OK) return st;
    if (!aligned16(x_bf16) || !aligned16(W_q4nx) || !aligned16(out)) return FDQP_ERR_ALIGN;
    if ((epi != kEpiNone || gamma_bf16 || fmt != kFmtQ4nx) && ctx->p_path == 1) return FDQP_ERR_ARG;  // the plain self-check kernel does none of these
    float* y = epi == kEpiNone ? static_cast<float*>(out) : nullptr;
    uint16_t* y16 = epi == kEpiNone ? nullptr : static_cast<uint16_t*>(out);
    const int64_t n_out = epi == kEpiGegluBf16 ? N / 2 : N;  // output values per token row
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FDQP_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const uint8_t* W = static_cast<const uint8_t*>(W_q4nx);
    const uint16_t* x = static_cast<const uint16_t*>(x_bf16);
    const uint16_t* gamma = static_cast<const uint16_t*>(gamma_bf16);
    const uint16_t* residual = static_cast<const uint16_t*>(residual_bf16);
    uint16_t* h_out = static_cast<uint16_t*>(h_out_bf16);
    cudaError_t e;
    bool fuse_norm = false;
    if (gamma) {
        // fused when the call is one GEMV launch that prepares the whole row of x inside every CTA
        GemvPlan probe;
        int cw = 0;
        fuse_norm = M <= kMaxTokens && !use_prefill(ctx, M, K, N) && plan_gemv(ctx, (int)M, (int)K, (int)N, &cw, &probe) &&
                    probe.prep_inline && probe.Z == 1 && (K / kGroup) * M * 4 <= (int64_t)cw * 32;
        if (!fuse_norm) {
            if ((e = rmsnorm_launch(x, residual, h_out, gamma, eps, ctx->x_norm, (int)M, (int)K, stream)))
                return cuda_fail(ctx, e, "RMS normalisation launch");
            ctx->launches += 1;
            x = ctx->x_norm;
        }
    }
    if (ctx->p_path == 1) {
        if ((e = plain_launch(W, x, y, (int)M, (int)K, (int)N, stream))) return cuda_fail(ctx, e, "plain kernel launch");
        ctx->launches += 1;
        return FDQP_OK;
    }
    if (use_prefill(ctx, M, K, N)) {
        // prefill-sized M: dequantise into shared memory, contract with tcgen05 (accumulators in TMEM)
        const uint16_t* xt = x;
        int64_t x_row_bytes = K * 2;
        if (M * K * 2 < kSpreadBelowBytes && ctx->x_spread) {
            x_row_bytes = ((kSpreadToBytes + M - 1) / M + 127) / 128 * 128;
            if ((e = cudaMemcpy2DAsync(ctx->x_spread, (size_t)x_row_bytes, x, (size_t)K * 2, (size_t)K * 2, (size_t)M,
                                       cudaMemcpyDeviceToDevice, stream)))
                return cuda_fail(ctx, e, "x spreading copy");
            xt = reinterpret_cast<const uint16_t*>(ctx->x_spread);
        }
        int kernels = 0;
        if ((e = prefill_launch(W, xt, x_row_bytes, y, y16, epi, ctx->pf_ws, ctx->status_dev, (int)M, (int)K, (int)N,
                                use_pair(ctx, M) ? 1 : 0, prefill_slices(ctx, M, K, N), fmt, prefill_tmem_mode(ctx, M, K, N), stream,
                                &kernels)))
            return cuda_fail(ctx, e, "prefill kernel launch");
        ctx->launches += kernels;
        return FDQP_OK;
    }
    // Token rows are processed eight at a time by the streaming GEMV kernel.
    for (int64_t m0 = 0; m0 < M; m0 += kMaxTokens) {
        const int mc = (int)((M - m0) < kMaxTokens ? (M - m0) : kMaxTokens);
        GemvPlan plan;
        int cw = 0;
        if (!plan_gemv(ctx, mc, (int)K, (int)N, &cw, &plan, fmt)) return FDQP_ERR_SIZE;
        plan.W = W;
        plan.x = x + m0 * K;
        plan.y = y ? y + m0 * N : nullptr;
        plan.y16 = y16 ? y16 + m0 * n_out : nullptr;
        plan.epi = epi;
        if (fuse_norm) {
            plan.norm = 1;
            plan.gamma = gamma;
            plan.eps = eps;
            plan.residual = residual;
            plan.h_out = h_out;
        }
        if (!plan.prep_inline) {
            if ((e = xprep_launch(plan.x, ctx->xq, ctx->xsc, mc, (int)K, stream)))
                return cuda_fail(ctx, e, "x preparation launch");
            ctx->launches += 1;
        }
        if ((e = gemv_launch(plan, cw, stream))) return cuda_fail(ctx, e, "gemv kernel launch");
        ctx->launches += 1;
        if (plan.Z > 1) {
            if ((e = splitk_sum_launch(ctx->ws_full, plan.y, plan.y16, epi, plan.Z, plan.S, mc, (int)N, stream)))
                return cuda_fail(ctx, e, "split-K sum launch");
            ctx->launches += 1;
        }
    }
    return FDQP_OK;
}

}  // namespace

extern "C" fdqp_status fdqp_run(fdqp_ctx* ctx, const void* x_bf16, const void* W_q4nx, float* y, int64_t M, int64_t K,
                                int64_t N, void* cuda_stream) {
    return run_impl(ctx, x_bf16, nullptr, 0.f, W_q4nx, y, kEpiNone, M, K, N, cuda_stream);
}

extern "C" fdqp_status fdqp_run_fmt(fdqp_ctx* ctx, int format, const void* x_bf16, const void* W_packed, float* y, int64_t M,
                                    int64_t K, int64_t N, void* cuda_stream) {
    return run_impl(ctx, x_bf16, nullptr, 0.f, W_packed, y, kEpiNone, M, K, N, cuda_stream, format);
}

extern "C" fdqp_status fdqp_run_epilogue(fdqp_ctx* ctx, const void* x_bf16, const void* W_q4nx, void* out, int epilogue,
                                         int64_t M, int64_t K, int64_t N, void* cuda_stream) {
    return run_impl(ctx, x_bf16, nullptr, 0.f, W_q4nx, out, epilogue, M, K, N, cuda_stream);
}

extern "C" fdqp_status fdqp_run_rmsnorm_epilogue(fdqp_ctx* ctx, const void* x_bf16, const void* gamma_bf16, float eps,
                                                 const void* W_q4nx, void* out, int epilogue, int64_t M, int64_t K, int64_t N,
                                                 void* cuda_stream) {
    if (!gamma_bf16) return FDQP_ERR_ARG;
    return run_impl(ctx, x_bf16, gamma_bf16, eps, W_q4nx, out, epilogue, M, K, N, cuda_stream);
}

extern "C" fdqp_status fdqp_run_add_rmsnorm_epilogue(fdqp_ctx* ctx, const void* x_bf16, const void* residual_bf16,
                                                     void* h_out_bf16, const void* gamma_bf16, float eps, const void* W_q4nx,
                                                     void* out, int epilogue, int64_t M, int64_t K, int64_t N,
                                                     void* cuda_stream) {
    if (!gamma_bf16 || !residual_bf16) return FDQP_ERR_ARG;
    return run_impl(ctx, x_bf16, gamma_bf16, eps, W_q4nx, out, epilogue, M, K, N, cuda_stream, kFmtQ4nx, residual_bf16,
                    h_out_bf16);
}

extern "C" fdqp_status fdqp_stream_read(fdqp_ctx* ctx, const void* buf, int64_t bytes, void* cuda_stream) {
    if (!ctx || !buf || bytes < 0) return FDQP_ERR_ARG;
    if (!aligned16(buf)) return FDQP_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FDQP_ERR_CUDA;
    const cudaError_t e = stream_read_launch(static_cast<const uint8_t*>(buf), bytes, ctx->sm_count, ctx->status_dev,
                                             static_cast<cudaStream_t>(cuda_stream));
    if (e) return cuda_fail(ctx, e, "read-stream kernel launch");
    ctx->launches += 1;
    return FDQP_OK;
}

extern "C" fdqp_status fdqp_flowkv_decode(fdqp_ctx* ctx, const void* q_bf16, const void* K_bf16, const void* V_bf16, float* out,
                                          int64_t H, int64_t G, int64_t d, int64_t L, int64_t pitch, int64_t window,
                                          float scale, void* cuda_stream) {
    if (!ctx || !q_bf16 || !K_bf16 || !V_bf16 || !out) return FDQP_ERR_ARG;
    if (H < 1 || G < 1 || (H % G) != 0 || H / G > 8 || (d != 128 && d != 256) || L < 1 || pitch < L) return FDQP_ERR_SHAPE;
    if (H > kKvMaxHeads || pitch > (int64_t)1 << 30) return FDQP_ERR_SIZE;
    if (!aligned16(q_bf16) || !aligned16(K_bf16) || !aligned16(V_bf16) || !aligned16(out)) return FDQP_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FDQP_ERR_CUDA;
    int launches = 0;
    const cudaError_t e = flowkv_launch(static_cast<const uint16_t*>(q_bf16), static_cast<const uint16_t*>(K_bf16),
                                        static_cast<const uint16_t*>(V_bf16), out, ctx->kv_ws, kKvMaxSplits, (int)H, (int)G, (int)d,
                                        (int)L, (int)pitch, (int)window, scale, ctx->sm_count, (int)ctx->p_flowkv_cluster,
                                        &launches, static_cast<cudaStream_t>(cuda_stream));
    if (e) return cuda_fail(ctx, e, "decode attention launch");
    ctx->launches += launches;
    return FDQP_OK;
}

extern "C" fdqp_status fdqp_run_host_async(fdqp_ctx* ctx, const void* x_host_bf16, const void* W_q4nx, float* y_host,
                                           int64_t M, int64_t K, int64_t N, void* cuda_stream) {
    if (!ctx || !x_host_bf16 || !W_q4nx || !y_host) return FDQP_ERR_ARG;
    fdqp_status st = check_shape(ctx, M, K, N);
    if (st != FDQP_OK) return st;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FDQP_ERR_CUDA;
    cudaError_t e;
    if (!ctx->x_stage) {
        if ((e = cudaMalloc(&ctx->x_stage, (size_t)ctx->max_M * ctx->max_K * 2))) return cuda_fail(ctx, e, "x staging");
        if ((e = cudaMalloc(&ctx->y_stage, (size_t)ctx->max_M * ctx->max_N * 4))) return cuda_fail(ctx, e, "y staging");
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // Decode-sized x in page-locked host memory that the device can address is read from there by the activation
    // preparation kernel (a few kilobytes over the bus, once), instead of being copied to the device first: the copy
    // engine's start-up costs more than the kernel.  The GEMV kernels themselves then never touch x.
    const void* x_dev = ctx->x_stage;
    bool direct_x = false;
    if (M <= kMaxTokens && (size_t)M * K * 2 <= kDirectHostBytes && ctx->p_direct_y != 0 && ctx->p_path != 1) {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, x_host_bf16) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer &&
            aligned16(attr.devicePointer)) {
            x_dev = attr.devicePointer;
            direct_x = true;
        } else {
            cudaGetLastError();
        }
    }
    if (!direct_x && (e = cudaMemcpyAsync(ctx->x_stage, x_host_bf16, (size_t)M * K * 2, cudaMemcpyHostToDevice, stream)))
        return cuda_fail(ctx, e, "x copy");
    // Small results in page-locked host memory that the device can address are stored there by the kernels themselves
    // (posted writes over the bus, a few microseconds for tens of kilobytes): no copy-out to launch and wait for.
    // y is write-only for every kernel.  Otherwise: the staging buffer and a copy.
    float* y_dev = ctx->y_stage;
    if ((size_t)M * N * 4 <= kDirectHostBytes && ctx->p_direct_y != 0) {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, y_host) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer &&
            aligned16(attr.devicePointer))
            y_dev = static_cast<float*>(attr.devicePointer);
        else
            cudaGetLastError();
    }
    const int64_t saved_prep = ctx->p_prep;
    if (direct_x) ctx->p_prep = 0;  // x is read once, by the preparation kernel
    st = fdqp_run(ctx, x_dev, W_q4nx, y_dev, M, K, N, cuda_stream);
    ctx->p_prep = saved_prep;
    if (st != FDQP_OK) return st;
    if (y_dev == ctx->y_stage && (e = cudaMemcpyAsync(y_host, ctx->y_stage, (size_t)M * N * 4, cudaMemcpyDeviceToHost, stream)))
        return cuda_fail(ctx, e, "y copy");
    return FDQP_OK;
}

extern "C" fdqp_status fdqp_run_host(fdqp_ctx* ctx, const void* x_host_bf16, const void* W_q4nx, float* y_host,
                                     int64_t M, int64_t K, int64_t N, void* cuda_stream) {
    const fdqp_status st = fdqp_run_host_async(ctx, x_host_bf16, W_q4nx, y_host, M, K, N, cuda_stream);
    if (st != FDQP_OK) return st;
    const cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream));
    if (e) return cuda_fail(ctx, e, "stream sync");
    return fdqp_last_status(ctx);
}

extern "C" fdqp_status fdqp_dequant(fdqp_ctx* ctx, const void* W_q4nx, void* out, int out_is_bf16, int64_t K, int64_t N,
                                    void* cuda_stream) {
    if (!ctx || !W_q4nx || !out || (out_is_bf16 != 0 && out_is_bf16 != 1)) return FDQP_ERR_ARG;
    fdqp_status st = check_shape(ctx, 1, K, N);
    if (st != FDQP_OK) return st;
    if (!aligned16(W_q4nx) || !aligned16(out)) return FDQP_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FDQP_ERR_CUDA;
    cudaError_t e = dequant_launch(static_cast<const uint8_t*>(W_q4nx), out, out_is_bf16 != 0, (int)K, (int)N,
                                   static_cast<cudaStream_t>(cuda_stream));
    if (e) return cuda_fail(ctx, e, "dequant kernel launch");
    ctx->launches += 1;
    return FDQP_OK;
}

extern "C" fdqp_status fdqp_dequant_fmt(fdqp_ctx* ctx, int format, const void* W_packed, void* out, int out_is_bf16,
                                        int64_t K, int64_t N, void* cuda_stream) {
    if (format == kFmtQ4nx) return fdqp_dequant(ctx, W_packed, out, out_is_bf16, K, N, cuda_stream);
    if (!ctx || !W_packed || !out || (out_is_bf16 != 0 && out_is_bf16 != 1) || format < 0 || format >= kFmtCount)
        return FDQP_ERR_ARG;
    fdqp_status st = check_shape(ctx, 1, K, N);
    if (st != FDQP_OK) return st;
    if ((K % kBlockK) != 0) return FDQP_ERR_SHAPE;
    if (!aligned16(W_packed) || !aligned16(out)) return FDQP_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FDQP_ERR_CUDA;
    cudaError_t e = dequant_fmt_launch(format, static_cast<const uint8_t*>(W_packed), out, out_is_bf16 != 0, (int)K, (int)N,
                                       static_cast<cudaStream_t>(cuda_stream));
    if (e) return cuda_fail(ctx, e, "dequant kernel launch");
    ctx->launches += 1;
    return FDQP_OK;
}

extern "C" fdqp_status fdqp_last_status(fdqp_ctx* ctx) {
    if (!ctx) return FDQP_ERR_ARG;
    const int v = *static_cast<volatile int*>(ctx->status_host);
    return v == 0 ? FDQP_OK : static_cast<fdqp_status>(v);
}

extern "C" fdqp_status fdqp_selftest_bounded_wait(fdqp_ctx* ctx, int64_t limit_us, void* cuda_stream) {
    if (!ctx || limit_us < 1 || limit_us > 100000) return FDQP_ERR_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FDQP_ERR_CUDA;
    cudaError_t e = wait_selftest_launch(ctx->status_dev, (unsigned long long)limit_us * 1000ull, static_cast<cudaStream_t>(cuda_stream));
    if (e) return cuda_fail(ctx, e, "bounded-wait self-test launch");
    ctx->launches += 1;
    return FDQP_OK;
}

extern "C" const char* fdqp_last_cuda_error(fdqp_ctx* ctx) { return ctx ? ctx->last_err.c_str() : ""; }

extern "C" fdqp_status fdqp_set_param(fdqp_ctx* ctx, const char* key, int64_t value) {
    if (!ctx || !key) return FDQP_ERR_ARG;
    const int64_t v = value < 0 ? -1 : value;
    if (!std::strcmp(key, "path")) {
        if (v > 3) return FDQP_ERR_ARG;
        ctx->p_path = v;
    } else if (!std::strcmp(key, "ctas_per_sm")) {
        if (v == 0 || v > kMaxCtasPerSm) return FDQP_ERR_ARG;
        ctx->p_ctas_per_sm = v;
    } else if (!std::strcmp(key, "consumer_warps")) {
        if (v != -1 && v != 8 && v != 16) return FDQP_ERR_ARG;
        ctx->p_cw = v;
    } else if (!std::strcmp(key, "stages")) {
        if (v == 0 || v == 1) return FDQP_ERR_ARG;
        ctx->p_stages = v;
    } else if (!std::strcmp(key, "split_k")) {
        if (v != -1 && v != 1 && v != 2 && v != 4 && v != 8) return FDQP_ERR_ARG;
        ctx->p_split_k = v;
    } else if (!std::strcmp(key, "prefill_split_k")) {
        if (v == 0 || v > kMaxSplit) return FDQP_ERR_ARG;
        ctx->p_pf_split = v;
    } else if (!std::strcmp(key, "host_direct_y")) {
        if (v != 0 && v != 1) return FDQP_ERR_ARG;
        ctx->p_direct_y = v;
    } else if (!std::strcmp(key, "prefill_a_tmem")) {
        if (v != 0 && v != 1 && v != 2) return FDQP_ERR_ARG;
        ctx->p_atmem = v;
    } else if (!std::strcmp(key, "prefill_pair")) {
        if (v > 1) return FDQP_ERR_ARG;
        ctx->p_pair = v;
    } else if (!std::strcmp(key, "l2_evict_first")) {
        if (v > 1) return FDQP_ERR_ARG;
        ctx->p_evict = v;
    } else if (!std::strcmp(key, "blocks_per_warp")) {
        if (v != -1 && v != 2 && v != 4) return FDQP_ERR_ARG;
        ctx->p_bpw = v;
    } else if (!std::strcmp(key, "strip_aligned")) {
        if (v > 1) return FDQP_ERR_ARG;
        ctx->p_aligned = v;
    } else if (!std::strcmp(key, "chain_launch")) {
        if (v > 3) return FDQP_ERR_ARG;
        ctx->p_chain_launch = v < 0 ? 1 : v;
    } else if (!std::strcmp(key, "flowkv_cluster")) {
        if (v > (int64_t)1 << 20) return FDQP_ERR_ARG;
        ctx->p_flowkv_cluster = v < 0 ? kFlowKvClusterPositions : v;
    } else if (!std::strcmp(key, "chain_dependent")) {
        if (v > 1) return FDQP_ERR_ARG;
        ctx->p_chain_dep = v < 0 ? 0 : v;
    } else if (!std::strcmp(key, "chain_wide")) {
        if (v > 1) return FDQP_ERR_ARG;
        ctx->p_chain_wide = v < 0 ? 1 : v;
    } else if (!std::strcmp(key, "chain_steps")) {
        if (v == 0 || v > kMaxChainSteps) return FDQP_ERR_ARG;
        ctx->p_chain_steps = v < 0 ? kMaxChainSteps : v;
    } else if (!std::strcmp(key, "prep_inline")) {
        if (v > 1) return FDQP_ERR_ARG;
        ctx->p_prep = v;
    } else {
        return FDQP_ERR_ARG;
    }
    return FDQP_OK;
}

extern "C" int64_t fdqp_launch_count(fdqp_ctx* ctx) { return ctx ? ctx->launches : 0; }

extern "C" fdqp_status fdqp_describe(fdqp_ctx* ctx, int64_t M, int64_t K, int64_t N, char* buf, size_t buf_bytes) {
    if (!ctx || !buf || buf_bytes == 0) return FDQP_ERR_ARG;
    fdqp_status st = check_shape(ctx, M, K, N);
    if (st != FDQP_OK) return st;
    if (ctx->p_path == 1) {
        std::snprintf(buf, buf_bytes, "fdqp_plain_kernel grid=(%lld,%lld) block=128", (long long)((N / 32 + 3) / 4),
                      (long long)((M + 7) / 8));
        return FDQP_OK;
    }
    if (use_prefill(ctx, M, K, N)) {
        const int Z = prefill_slices(ctx, M, K, N);
        if (use_pair(ctx, M))
            std::snprintf(buf, buf_bytes,
                          "fdqp_prefill_pair_kernel grid=%lld cluster=2 block=320 tile=256x512 per pair stages=4 tmem_cols=512 "
                          "split_k=%d%s",
                          (long long)(2 * ((N + 255) / 256) * ((M + 511) / 512) * Z), Z, Z > 1 ? " + fdqp_prefill_sum_kernel" : "");
        else if (M <= 128) {
            const int mode = prefill_tmem_mode(ctx, M, K, N);
            const bool tri = mode == 2 && M <= 64;
            std::snprintf(buf, buf_bytes,
                          "fdqp_prefill_kernel<128> grid=%lld block=320 tile=128x128 %s CTAs per SM %s split_k=%d%s",
                          (long long)(((N + 127) / 128) * Z), tri ? "three" : "two",
                          tri ? "weights in TMEM (2 stages) x_stages=4 tmem_cols=128"
                              : (mode ? "weights in TMEM (4 stages) x_stages=6 tmem_cols=256" : "stages=3 tmem_cols=128"),
                          Z, Z > 1 ? " + fdqp_prefill_sum_kernel" : "");
        }
        else
            std::snprintf(buf, buf_bytes,
                          "fdqp_prefill_kernel grid=%lld block=576 tile=256x256 stages=3 tmem_cols=512 split_k=%d%s",
                          (long long)(((N + 255) / 256) * ((M + 255) / 256) * Z), Z, Z > 1 ? " + fdqp_prefill_sum_kernel" : "");
        return FDQP_OK;
    }
    GemvPlan plan;
    int cw = 0;
    const int mc = (int)(M < kMaxTokens ? M : kMaxTokens);
    if (!plan_gemv(ctx, mc, (int)K, (int)N, &cw, &plan)) return FDQP_ERR_SIZE;
    std::snprintf(buf, buf_bytes,
                  "%sfdqp_gemv_kernel<%d,%d> calls=%lld grid=%d block=%d smem=%u stages=%d split_k=%d ctas_per_slice=%d "
                  "evict_first=%d strip_aligned=%d blocks_per_warp=%d",
                  plan.prep_inline ? "" : "fdqp_xprep_kernel + ", cw, mc == 1 ? 1 : (mc > kColsMaxTokens ? 2 : (mc == 2 ? 3 : 1)), (long long)((M + kMaxTokens - 1) / kMaxTokens), plan.Z * plan.Gz, (cw + 1 + cw / 8) * 32,
                  plan.smem_bytes, plan.nstage, plan.Z, plan.Gz, plan.evict_first, plan.strip_aligned, plan.bpw);
    return FDQP_OK;
}

// ---- a chain of projections in one persistent launch -----------------------------------------------------------------

extern "C" fdqp_status fdqp_run_chain(fdqp_ctx* ctx, const fdqp_chain_step* steps, int64_t n_steps, int64_t M,
                                      void* cuda_stream) {
    if (!ctx || !steps || n_steps < 1) return FDQP_ERR_ARG;
    if (M < 1) return FDQP_ERR_SHAPE;
    if (M > kMaxTokens) return FDQP_ERR_SIZE;
    for (int64_t i = 0; i < n_steps; ++i) {
        const fdqp_chain_step& u = steps[i];
        if (!u.x_bf16 || !u.W_q4nx || !u.out) return FDQP_ERR_ARG;
        if (u.epilogue != kEpiNone && u.epilogue != kEpiBf16 && u.epilogue != kEpiGegluBf16) return FDQP_ERR_ARG;
        if ((u.residual_bf16 || u.h_out_bf16) && !u.gamma_bf16) return FDQP_ERR_ARG;
        if (u.h_out_bf16 && !u.residual_bf16) return FDQP_ERR_ARG;
        if (u.h_out_bf16 && (u.h_out_bf16 == u.x_bf16 || u.h_out_bf16 == u.residual_bf16)) return FDQP_ERR_ARG;
        if (u.gamma_bf16 && !(u.eps >= 0.f)) return FDQP_ERR_ARG;
        if (u.depends_on_previous != 0 && (u.depends_on_previous != 1 || i == 0)) return FDQP_ERR_ARG;
        const fdqp_status st = check_shape(ctx, M, u.K, u.N);
        if (st != FDQP_OK) return st;
        if (!aligned16(u.x_bf16) || !aligned16(u.W_q4nx) || !aligned16(u.out) || (u.gamma_bf16 && !aligned16(u.gamma_bf16)) ||
            (u.residual_bf16 && !aligned16(u.residual_bf16)) || (u.h_out_bf16 && !aligned16(u.h_out_bf16)))
            return FDQP_ERR_ALIGN;
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FDQP_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int grid = ctx->sm_count;
    const int m = (int)M;
    const bool cols = m <= kColsMaxTokens;
    const uint32_t rec = (uint32_t)(cols ? kColsRecBytes : kPlaneRecBytes);
    // blocks of a K slice whose prepared activations fit the shared-memory budget and one preparation pass
    int cap_blocks = (int)(kChainXsCap / (8u * rec * (uint32_t)m));
    if (cap_blocks > kChainPrepItems / (8 * m * 4)) cap_blocks = kChainPrepItems / (8 * m * 4);
    if (cap_blocks < 1) return FDQP_ERR_SIZE;
    // plan every launch before the first one goes out, so that an error launches nothing; where the steps of a launch
    // need more counters or partial-row slots than the workspace holds, the chain is cut into shorter launches
    std::vector<ChainPlan> plans;
    std::vector<char> plan_epi;
    // plans of the launches that cover steps [seg_begin, seg_end), appended to `plans`
    auto plan_all = [&](const int64_t seg_begin, const int64_t seg_end, const int per_launch) -> fdqp_status {
    for (int64_t first = seg_begin; first < seg_end; first += per_launch) {
        const int n = (int)((seg_end - first) < per_launch ? (seg_end - first) : per_launch);
        ChainPlan cp;
        std::memset(&cp, 0, sizeof(cp));
        cp.nsteps = n;
        cp.M = m;
        cp.ws_edge = ctx->chain_edge;
        cp.ws_full = ctx->chain_full;
        cp.tickets = ctx->chain_tickets;
        cp.done = ctx->chain_done;
        cp.exit_count = ctx->chain_done + kMaxChainSteps;
        cp.status = ctx->status_dev;
        cp.evict_first = ctx->p_evict >= 0 ? (ctx->p_evict != 0) : 1;
        uint32_t xs_bytes = 0, xsum_bytes = 0;
        size_t ticket_off = 0, edge_off = 0, full_off = 0, blocks = 0;
        bool epi = false, dependent = false;
        for (int i = 0; i < n; ++i) {
            const fdqp_chain_step& u = steps[first + i];
            ChainStep& c = cp.step[i];
            c.W = static_cast<const uint8_t*>(u.W_q4nx);
            c.x = static_cast<const uint16_t*>(u.x_bf16);
            c.y = u.epilogue == kEpiNone ? static_cast<float*>(u.out) : nullptr;
            c.y16 = u.epilogue == kEpiNone ? nullptr : static_cast<uint16_t*>(u.out);
            c.gamma = static_cast<const uint16_t*>(u.gamma_bf16);
            c.residual = static_cast<const uint16_t*>(u.residual_bf16);
            c.h_out = static_cast<uint16_t*>(u.h_out_bf16);
            c.eps = u.eps;
            c.epi = u.epilogue;
            c.norm = u.gamma_bf16 ? 1 : 0;
            if (c.epi != kEpiNone || c.norm) epi = true;
            c.K = (int)u.K;
            c.N = (int)u.N;
            c.S = c.N / kStripRows;
            c.nb = (c.K + kBlockK - 1) / kBlockK;
            int Z = (c.nb + cap_blocks - 1) / cap_blocks;
            c.nbz = (c.nb + Z - 1) / Z;
            Z = (c.nb + c.nbz - 1) / c.nbz;
            c.Z = Z;
            if (c.norm && Z > 1) return FDQP_ERR_SIZE;  // the normalisation needs the whole row in every CTA
            if (Z > grid) return FDQP_ERR_SIZE;
            const int len_last = c.nb - (Z - 1) * c.nbz;
            int64_t Gz = grid / Z;
            if (Gz > (int64_t)c.S * len_last) Gz = (int64_t)c.S * len_last;
            if (Gz < 1) Gz = 1;
            // whole strips per CTA when that costs at most 3 % of imbalance (nothing is exchanged between CTAs then) --
            // or, for a step another one waits on, when the extra blocks of the busiest CTA (0.125 us each) cost less
            // than the exchange of shared strips that the waiting step would have to sit out (about 2 us)
            c.strip_aligned = 0;
            if (c.S >= Gz) {
                const int64_t per = (c.S + Gz - 1) / Gz;
                const double extra_blocks = ((double)per - (double)c.S / (double)Gz) * (double)c.nbz;
                const bool waited_on = first + i + 1 < seg_end && steps[first + i + 1].depends_on_previous != 0;
                if ((double)per * (double)Gz <= 1.03 * (double)c.S || (waited_on && extra_blocks * 0.125 < 2.0)) c.strip_aligned = 1;
            }
            if (ctx->p_aligned >= 0 && (ctx->p_aligned == 0 || c.S >= Gz)) c.strip_aligned = ctx->p_aligned != 0;
            c.Gz = (int)Gz;
            c.wait_prev = (u.depends_on_previous && i > 0) ? 1 : 0;  // across launches the stream order is the dependency
            if (c.wait_prev) {
                cp.step[i - 1].signal = 1;
                dependent = true;
            }
            c.B = (uint32_t)blocks;
            blocks += (size_t)c.S * c.nb;
            for (int z = 0; z < Z; ++z) {
                if (cp.nunits >= kMaxChainUnits) return FDQP_ERR_SIZE;
                cp.unit_step[cp.nunits] = (uint8_t)i;
                cp.unit_slice[cp.nunits] = (uint8_t)z;
                ++cp.nunits;
            }
            c.ticket_off = (uint32_t)ticket_off;
            c.edge_off = (uint32_t)edge_off;
            c.full_off = (uint32_t)full_off;
            ticket_off += (size_t)c.S;
            edge_off += (size_t)2 * Z * c.Gz;
            if (Z > 1) full_off += (size_t)Z * c.S;
            const uint32_t xb = (uint32_t)c.nbz * 8u * rec * (uint32_t)m;
            if (xb > xs_bytes) xs_bytes = xb;
            if (!cols && (uint32_t)c.nbz * 8u * (uint32_t)kPlaneSumBytes > xsum_bytes) xsum_bytes = (uint32_t)c.nbz * 8u * (uint32_t)kPlaneSumBytes;
        }
        // No step of this launch waits for another one: cut the whole chain, not every step, into equal CTA ranges.
        cp.Wtot = (uint32_t)blocks;
        cp.has_deps = dependent ? 1 : 0;
        cp.wide = (!dependent && blocks >= (size_t)grid && blocks < (1u << 31) && ctx->p_chain_wide != 0) ? 1 : 0;
        if (ticket_off > ctx->chain_ticket_cap || full_off > kChainFullSlots ||
            (cp.wide ? (size_t)2 * grid : edge_off) > (size_t)2 * ctx->sm_count * kChainEdgeSteps)
            return FDQP_ERR_SIZE;
        const uint32_t part_bytes = 2u * 16u * kStripRows * (uint32_t)m * 4u * (cols ? (uint32_t)kColsPartTerms : 1u);
        const uint32_t norm_bytes = (uint32_t)(kChainPrepItems / 4) * 4u + 64u;
        const uint32_t geo_bytes = (uint32_t)cp.nunits * 16u;  // the CTA's block range per (step, K slice) unit
        const uint32_t fixed = round_up(xs_bytes, 128) + round_up(xsum_bytes, 128) + round_up(part_bytes, 128) +
                               round_up(norm_bytes, 128) + round_up(geo_bytes, 128) + (2u * kMaxStages + 4u) * 8u + 128u;
        // four blocks per warp and stage (half the barrier round trips per tile) while the ring keeps three stages
        int bpw = ctx->p_bpw == 2 || ctx->p_bpw == 4 ? (int)ctx->p_bpw : 4;
        uint32_t stage_bytes = 2u * (uint32_t)bpw * kBlockBytes;
        int nstage = (uint32_t)ctx->smem_optin > fixed ? (int)(((uint32_t)ctx->smem_optin - fixed) / stage_bytes) : 0;
        if (bpw == 4 && ctx->p_bpw != 4 && nstage < kMinStages) {
            bpw = 2;
            stage_bytes = 2u * (uint32_t)bpw * kBlockBytes;
            nstage = (uint32_t)ctx->smem_optin > fixed ? (int)(((uint32_t)ctx->smem_optin - fixed) / stage_bytes) : 0;
        }
        cp.bpw = bpw;
        if (nstage > kMaxStages) nstage = kMaxStages;
        if (ctx->p_stages > 0 && ctx->p_stages < nstage) nstage = (int)ctx->p_stages;
        if (nstage < 2) return FDQP_ERR_SIZE;
        cp.nstage = nstage;
        cp.off_xs = (uint32_t)nstage * stage_bytes;
        cp.off_xsum = cp.off_xs + round_up(xs_bytes, 128);
        cp.off_part = cp.off_xsum + round_up(xsum_bytes, 128);
        cp.off_norm = cp.off_part + round_up(part_bytes, 128);
        cp.off_geo = cp.off_norm + round_up(norm_bytes, 128);
        cp.off_bar = cp.off_geo + round_up(geo_bytes, 128);
        cp.smem_bytes = cp.off_bar + (2u * (uint32_t)nstage + 4u) * 8u;
        plans.push_back(cp);
        plan_epi.push_back(epi ? 1 : 0);
    }
    return FDQP_OK;
    };
    // A step that consumes the previous step's output begins a new launch by default (the stream order is the
    // dependency): a launch without dependencies is cut into CTA ranges as one sequence, which is the fast form, and a
    // step alone in its launch goes out as a single call.  Measured on the Gemma3-4B MLP block (normalise -> gate|up ->
    // gated GELU -> down): 20.2 us at M = 1 and 30.5 us at M = 8 this way, 24.5 / 49.0 us with both steps in one launch
    // and the second waiting on the first's completion counter -- that form is kept ("chain_dependent" = 1).
    struct Action { int single; size_t index; };  // a single call of steps[index], or the launch plans[index]
    std::vector<Action> actions;
    for (int64_t seg_begin = 0; seg_begin < n_steps;) {
        int64_t seg_end = seg_begin + 1;
        while (seg_end < n_steps && (ctx->p_chain_dep != 0 || steps[seg_end].depends_on_previous == 0)) ++seg_end;
        if (ctx->p_chain_dep == 0 && seg_end - seg_begin == 1) {
            actions.push_back(Action{1, (size_t)seg_begin});
        } else {
            const size_t before = plans.size();
            fdqp_status planned = FDQP_ERR_SIZE;
            for (int per_launch = (int)ctx->p_chain_steps; per_launch >= 1; per_launch = per_launch > 1 ? (per_launch + 1) / 2 : 0) {
                plans.resize(before);
                plan_epi.resize(before);
                planned = plan_all(seg_begin, seg_end, per_launch);
                if (planned != FDQP_ERR_SIZE) break;
            }
            if (planned != FDQP_OK) return planned;
            for (size_t i = before; i < plans.size(); ++i) actions.push_back(Action{0, i});
        }
        seg_begin = seg_end;
    }
    for (const Action& a : actions) {
        if (a.single) {
            const fdqp_chain_step& u = steps[a.index];
            const fdqp_status st = run_impl(ctx, u.x_bf16, u.gamma_bf16, u.eps, u.W_q4nx, u.out, u.epilogue, M, u.K, u.N, cuda_stream,
                                            kFmtQ4nx, u.residual_bf16, u.h_out_bf16);
            if (st != FDQP_OK) return st;
        } else {
            const cudaError_t e = chain_launch(plans[a.index], grid, plan_epi[a.index] != 0, (int)ctx->p_chain_launch, stream);
            if (e) return cuda_fail(ctx, e, "chain kernel launch");
            ctx->launches += 1;
        }
    }
    return FDQP_OK;
}

// ---- projection without any allocation -------------------------------------------------------------------------
//
// fdqp_run_noalloc serves callers that must not allocate device memory when they run a projection: a server that
// handed all device memory to its own pool at start-up, a real-time loop that cannot afford the device-wide
// synchronisation an allocation may imply, a plug-in that is forbidden to allocate after initialisation.  It is the
// streaming GEMV kernel with its scratch -- the partial-row slots of strips shared between CTAs, the strips' arrival
// counters and the status word -- in a fixed array that is part of the loaded library image.

namespace {

constexpr int kNoAllocMaxCtas = 320;                  // partial-row slots: two per persistent CTA
constexpr int64_t kNoAllocMaxN = 262144;              // arrival counters: one per 32-row strip
constexpr int64_t kNoAllocMaxK = 1 << 20;             // far beyond what shared memory holds without a K split
constexpr size_t kNoAllocEdgeBytes = (size_t)kNoAllocMaxCtas * 2 * kStripRows * kMaxTokens * sizeof(float);
constexpr size_t kNoAllocTicketBytes = (size_t)(kNoAllocMaxN / kStripRows) * sizeof(int);
constexpr size_t kNoAllocScratchBytes = kNoAllocEdgeBytes + kNoAllocTicketBytes + 256;  // + status word

struct NoAllocDevice {
    bool ready = false;
    unsigned char* scratch = nullptr;  // device address of g_noalloc_scratch on this device
    int sm_count = 0;
    int smem_optin = 0;
};

constexpr int kNoAllocMaxDevices = 64;
NoAllocDevice g_noalloc_devices[kNoAllocMaxDevices];
std::mutex g_noalloc_mutex;

}  // namespace

// 688,384 bytes, held by every device that loads the library until the process exits.  In host code this name is
// only a handle for the runtime; the device address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

extern "C" fdqp_status fdqp_run_noalloc(const void* x_bf16, const void* W_q4nx, float* y, int64_t M, int64_t K, int64_t N,
                                        void* cuda_stream) {
    if (!x_bf16 || !W_q4nx || !y) return FDQP_ERR_ARG;
    if (M < 1 || K <= 0 || N <= 0 || (K % kGroup) != 0 || (N % kStripRows) != 0) return FDQP_ERR_SHAPE;
    if (M > kMaxTokens || N > kNoAllocMaxN || K > kNoAllocMaxK) return FDQP_ERR_SIZE;
    if (!aligned16(x_bf16) || !aligned16(W_q4nx) || !aligned16(y)) return FDQP_ERR_ALIGN;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNoAllocMaxDevices) {
        cudaGetLastError();
        return FDQP_ERR_CUDA;
    }
    NoAllocDevice info;
    {
        // First call on this device: look the device up and resolve the scratch array's address, with the device current.
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        NoAllocDevice& d = g_noalloc_devices[dev];
        if (!d.ready) {
            int major = 0;
            if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) { cudaGetLastError(); return FDQP_ERR_CUDA; }
            if (major != 10) return FDQP_ERR_ARCH;
            if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
                cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
                cudaGetLastError();
                return FDQP_ERR_CUDA;
            }
            if (gemv_set_smem_limit(d.smem_optin) != cudaSuccess) { cudaGetLastError(); return FDQP_ERR_CUDA; }
            void* ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) { cudaGetLastError(); return FDQP_ERR_CUDA; }
            d.scratch = static_cast<unsigned char*>(ptr);
            d.ready = true;
        }
        info = d;
    }
    // Plan with the ordinary planner on a stack context: no K split (its workspace would not be modest) and the
    // activations prepared inside the kernel (no staging buffer).
    fdqp_ctx tmp;
    tmp.device = dev;
    tmp.sm_count = info.sm_count;
    tmp.smem_optin = info.smem_optin;
    tmp.max_M = kMaxTokens;
    tmp.max_K = K;
    tmp.max_N = kNoAllocMaxN;
    tmp.p_split_k = 1;
    tmp.p_prep = 1;
    tmp.ws_edge = reinterpret_cast<float*>(info.scratch);
    tmp.tickets = reinterpret_cast<int*>(info.scratch + kNoAllocEdgeBytes);
    tmp.status_dev = reinterpret_cast<int*>(info.scratch + kNoAllocEdgeBytes + kNoAllocTicketBytes);
    GemvPlan plan;
    int cw = 0;
    if (!plan_gemv(&tmp, (int)M, (int)K, (int)N, &cw, &plan)) return FDQP_ERR_SIZE;  // the K slice of x must fit shared memory
    if (plan.Z != 1 || plan.Z * plan.Gz > kNoAllocMaxCtas) return FDQP_ERR_SIZE;
    plan.W = static_cast<const uint8_t*>(W_q4nx);
    plan.x = static_cast<const uint16_t*>(x_bf16);
    plan.y = y;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // The array keeps whatever the last call left: the arrival counters must start at zero.
    if (cudaMemsetAsync(plan.tickets, 0, sizeof(int) * (size_t)plan.S, stream) != cudaSuccess) { cudaGetLastError(); return FDQP_ERR_CUDA; }
    if (gemv_launch(plan, cw, stream) != cudaSuccess) { cudaGetLastError(); return FDQP_ERR_CUDA; }
    return FDQP_OK;
}

// The status word of fdqp_run_noalloc lives in the scratch array (there is no context to hold it).  One blocking 4-byte
// copy from the current device; allocates nothing.
extern "C" fdqp_status fdqp_noalloc_last_status(void) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNoAllocMaxDevices) {
        cudaGetLastError();
        return FDQP_ERR_CUDA;
    }
    unsigned char* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_devices[dev].ready) return FDQP_OK;  // no call on this device yet
        scratch = g_noalloc_devices[dev].scratch;
    }
    int v = 0;
    if (cudaMemcpy(&v, scratch + kNoAllocEdgeBytes + kNoAllocTicketBytes, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return FDQP_ERR_CUDA;
    }
    return v == 0 ? FDQP_OK : static_cast<fdqp_status>(v);
}
