// Launch plan of the streaming GEMV kernels: the quantities the host fixes per call and the
// kernel re-derives per CTA.  Plain data, shared by the host dispatcher and the device code.
#pragma once
#include <stdint.h>

namespace fdqp {

constexpr int kStripRows = 32;      // output features per strip
constexpr int kGroup = 32;          // quantisation group along K
constexpr int kBlockK = 256;        // input features per full Q4NX block
constexpr int kBlockBytes = 5120;   // bytes of a full block (Sec. "Dequantization Engine")
constexpr int kGroupBytes = 640;    // bytes a block spends per group: 512 codes + 64 scales + 64 offsets
constexpr int kMaxTokens = 8;       // token rows one GEMV launch handles
// What a kernel writes for a finished output value (values of fdqp_epilogue in fdqp.h).
constexpr int kEpiNone = 0;       // fp32 y [M][N]
constexpr int kEpiBf16 = 1;       // bf16 y [M][N]
constexpr int kEpiGegluBf16 = 2;  // bf16 [M][N/2]: gelu(row r) * (row r + 16) of every 32-row strip
// Up to this many tokens the GEMV lays the byte planes of a token out as MMA columns; above it, one MMA per plane.
constexpr int kColsMaxTokens = 2;
// Column modes hand three partial terms per (row, token) to the reducer (two column halves + the offset term).
constexpr int kColsPartTerms = 3;
// Prepared activations in shared memory (written by xprep_item, read by the tile loop):
//   column modes (M <= 2): one 136-byte record per (group-tile, token) -- four signed byte planes of the 31-bit fixed
//   point (4 x 32 bytes) and {sum of x, unit} at 128;
//   M >= 3: the bf16 activations themselves in MMA fragment order, 64 bytes per (group-tile, token), and the sums of x
//   of the (up to eight) tokens, 32 bytes per group-tile.
constexpr int kColsRecBytes = 136, kColsSumOff = 128, kColsUnitOff = 132;
constexpr int kPlaneRecBytes = 64, kPlaneSumBytes = 32;
constexpr int kMaxSplit = 8;        // K slices
constexpr int kMaxCtasPerSm = 2;

struct GemvPlan {
    const uint8_t* W;     // device, packed Q4NX
    const uint16_t* x;    // device, [M][K] bf16 bits
    const uint32_t* xq;   // device, prepared activations of a call whose x is prepared by fdqp_xprep_kernel (layout above)
    const float* xsc;     // device, M >= 3: per group-tile the sums of x by token, [K/32][8]
    float* y;             // device, fp32 output [M][N] (epilogue kEpiNone)
    uint16_t* y16;        // device, bf16 output (other epilogues)
    int epi;
    const uint16_t* gamma;  // RMS normalisation of x fused into the in-kernel activation preparation (norm != 0):
    float eps;              //   x <- bf16(x * rsqrt(mean(x^2) + eps) * (1 + gamma)), per token row
    int norm;
    const uint16_t* residual;  // with norm: x + residual (bf16, one rounding) is what gets normalised ...
    uint16_t* h_out;           // ... and, when not null, is also written here by the grid's first CTA ([M][K] bf16)
    float* ws_edge;       // device, [grid][2][32*kMaxTokens] partial sums of strips shared between CTAs
    float* ws_full;       // device, [Z][S][32*kMaxTokens] partial sums of whole strip-slices (Z > 1)
    int* tickets;         // device, [S] arrival counters, zero between launches
    int* status;          // host-mapped sticky status word
    int fmt;              // container format (fdqp_format.h); 0 = Q4NX
    int M, K, N;
    int S;                // strips = N / 32
    int nb;               // blocks per strip = ceil(K / 256)
    int Z;                // K slices
    int nbz;              // blocks per slice = ceil(nb / Z); every slice is non-empty
    int Gz;               // CTAs per slice; grid = Z * Gz
    int nstage;           // ring depth in stages of (consumer warps / 8) * bpw blocks
    int bpw;              // blocks each consumer warp handles per stage (2 or 4)
    int evict_first;      // weight copies carry an evict-first L2 hint
    int strip_aligned;    // 1: CTA ranges are cut at strip boundaries (no strip is shared between CTAs of a slice)
    int prep_inline;      // 1: every CTA prepares its K slice of x itself; 0: a preparation kernel ran before
    uint32_t off_xs;      // shared-memory offsets (bytes): prepared-x records, per-token scalars,
    uint32_t off_xsum;    //   partial rows, barriers
    uint32_t off_part;
    uint32_t off_bar;
    uint32_t smem_bytes;
};

// ---- a chain of projections in one persistent launch (fdqp_chain.cu) ---------------------------------------------
constexpr int kMaxChainSteps = 160;  // projections one launch walks (a longer chain is cut into several launches)
constexpr int kMaxChainUnits = 240;  // (step, K slice) pairs of one launch
constexpr int kChainEdgeSteps = 64;  // partial-row slots for strips shared between CTAs: two per CTA for this many steps

struct ChainStep {
    const uint8_t* W;          // device, packed Q4NX
    const uint16_t* x;         // device, [M][K] bf16 bits (may be written by the previous step: wait_prev)
    float* y;                  // device, fp32 output [M][N] (epilogue kEpiNone)
    uint16_t* y16;             // device, bf16 output (other epilogues)
    const uint16_t* gamma;     // RMS normalisation of x in the activation preparation (norm != 0)
    const uint16_t* residual;  // with norm: x + residual is what gets normalised ...
    uint16_t* h_out;           // ... and, when not null, is also written here by the grid's first CTA
    float eps;
    int epi, norm;
    int K, N;
    int S;                     // strips = N / 32
    int nb;                    // blocks per strip = ceil(K / 256)
    int Z, nbz;                // K slices and blocks per slice (the prepared x of a slice must fit shared memory)
    int Gz;                    // CTAs per slice (Z * Gz <= grid; the rest of the grid idles during this step)
    int strip_aligned;         // 1: CTA ranges are cut at strip boundaries
    uint32_t B;                // chain-wide cut: position of this step's first block in the chain's block sequence
    int wait_prev;             // 1: the step's input is the previous step's output: wait for all of its strips
    int signal;                // 1: the next step waits on this one: count the stored strips in done[step]
    uint32_t ticket_off;       // this step's arrival counters inside ChainPlan::tickets
    uint32_t edge_off;         // this step's slots inside ChainPlan::ws_edge (2 per CTA) ...
    uint32_t full_off;         // ... and inside ChainPlan::ws_full (Z * S, used when Z > 1)
};

struct ChainPlan {
    int nsteps, M;
    float* ws_edge;            // device, partial rows of strips shared between CTAs
    float* ws_full;            // device, partial rows of whole strip-slices (steps with K slices)
    int* tickets;              // device, arrival counters per (step, strip), zero between launches
    int* done;                 // device, [kMaxChainSteps] strips stored per step, zero between launches
    int* exit_count;           // device, CTAs that have finished (the last one resets `done`)
    int* status;               // host-mapped sticky status word
    int nstage, evict_first;
    int bpw;                   // blocks per consumer warp and ring stage (2 or 4; a stage holds twice as many blocks)
    int has_deps;              // 1: some step waits for the one before it (the completion counters are in use)
    int wide;                  // 1: chain-wide cut into CTA ranges (no step waits for another), 0: every step cut on its own
    uint32_t Wtot;             // chain-wide cut: blocks of all steps together
    int nunits;                // (step, K slice) pairs in processing order
    uint8_t unit_step[kMaxChainUnits], unit_slice[kMaxChainUnits];
    uint32_t off_xs, off_xsum, off_part, off_norm, off_geo, off_bar, smem_bytes;  // shared-memory carve-up (bytes)
    ChainStep step[kMaxChainSteps];
};

}  // namespace fdqp
