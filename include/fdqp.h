/*
 * fdqp.h -- C ABI of the FusedDQP library for NVIDIA B200 (sm_100a).
 *
 * FusedDQP is the decode-time projection of the paper "Mapping Gemma3 onto an
 * Edge Dataflow Architecture": a matrix-vector (or thin matrix-matrix) product
 * whose weight matrix is stored in the 4-bit Q4NX container and is dequantised
 * inside the same kernel that multiplies it (Sec. "FusedDQP", Eq. 14 and 15),
 * using the block-wise rule of Eq. 3 (Sec. "Dequantization Engine").
 *
 * Naming used by every entry point
 *   x      activations, [M][K] row-major, bf16           (M token rows)
 *   w_hat  logical dequantised weights, w_hat[k][n]       (K inputs, N outputs)
 *   y      result, [M][N] row-major, fp32:  y[m][n] = sum_k x[m][k] * w_hat[k][n]
 * The paper writes the same product as Y = W x A with W of size "M x K"; its M
 * (output features) is N here, and M here counts tokens.
 *
 * Q4NX container ("layout v1").  The paper fixes the content and size of a
 * block -- 32 x 256 int4 codes, 256 bf16 scales, 256 bf16 minimum-value
 * offsets, 5120 bytes, group size 32 -- and that blocks are consumed left to
 * right along K.  The remaining byte-level choices are this library's:
 *   - a block covers 32 output features (a "strip", s = n / 32, r = n % 32)
 *     by 256 input features (b = k / 256); groups of 32 run along K;
 *   - strips are stored one after another, and the blocks of a strip follow
 *     each other, so a strip is one contiguous run of 20*K bytes;
 *   - a block with j groups (j = 8, or (K/32) % 8 for the last block of a strip
 *     when K is not a multiple of 256) is 640*j bytes:
 *         [codes 512*j] [scales 64*j] [offsets 64*j];
 *   - with c = k % 256, t = c / 32, i = c % 32: the code of (r, c) is in byte
 *     t*512 + r*16 + i/2, low nibble for even i; the group's scale is the
 *     little-endian bf16 word 512*j + 2*(t*32 + r), its offset the word at
 *     576*j + 2*(t*32 + r).
 * K and N must be positive multiples of 32.  Codes are unsigned 0..15.
 *
 * Dequantisation (Eq. 3):  w_hat = d * code + m, evaluated with d and m widened
 * exactly from bf16 and ONE rounding to fp32.  fdqp_dequant returns exactly that
 * value (or its round-to-nearest-even bf16).  fdqp_run accumulates in fp32 in an
 * unspecified but run-to-run reproducible order; for M >= 9 the weights pass
 * through bf16 before a tensor-core contraction.  Acceptance bound for y against
 * an fp64 evaluation: |y - y_ref| <= 2e-3 * sum_k |x*w_hat| + 1e-5.
 * What the kernels guarantee for every finite input, and where the acceptance
 * bound follows from it:
 *   - M <= 8 (GEMV kernels): the activations enter the arithmetic EXACTLY (no
 *     rounding of x, whatever the dynamic range inside a 32-group: see fdqp_run);
 *     a group contributes d * (sum_k code_k x_k) + m * (sum_k x_k), the sums exact
 *     or fp32-accumulated, combined in fp32.  So |y - y_ref| <= 2^-17 * sum_k
 *     |x_k| (|d * code_k| + |m|) + 1e-5, which is inside the acceptance bound
 *     unless more than 99.5 % of that sum cancels inside d * code + m (weights
 *     that are exactly zero through m = -d * code under the largest activations).
 *   - M >= 9 (tensor-core kernels): additionally each w_hat is rounded to bf16
 *     (2^-9 relative), so the bound holds when the K rounding errors average
 *     out; the dispatch keeps reductions shorter than K = 256 on the GEMV kernels.
 * Non-finite activations give non-finite outputs in their token row.
 *
 * Conventions
 *   - "host" / "device" on every pointer says where the memory must live.
 *   - No entry point throws; each returns an fdqp_status (FDQP_OK == 0).
 *   - Device work is enqueued on the caller's CUDA stream (a cudaStream_t passed
 *     as void*; NULL is the legacy default stream) and is asynchronous unless
 *     stated otherwise.
 *   - There is no CPU fallback: without an sm_100 device fdqp_create fails.
 */
#ifndef FDQP_H
#define FDQP_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define FDQP_API __attribute__((visibility("default")))
#else
#define FDQP_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fdqp_ctx fdqp_ctx; /* opaque, owned by the library */

typedef enum {
    FDQP_OK = 0,
    FDQP_ERR_ARG = 1,     /* null pointer, bad flag, code > 15 */
    FDQP_ERR_SHAPE = 2,   /* M < 1, K or N not a positive multiple of 32 */
    FDQP_ERR_ALIGN = 3,   /* a device pointer is not 16-byte aligned */
    FDQP_ERR_SIZE = 4,    /* output buffer too small, or shape beyond the context's maxima */
    FDQP_ERR_ARCH = 5,    /* device is not compute capability 10.x */
    FDQP_ERR_CUDA = 6,    /* a CUDA runtime call failed; see fdqp_last_cuda_error */
    FDQP_ERR_NOMEM = 7,   /* allocation failed */
    FDQP_ERR_TIMEOUT = 8  /* a bounded wait inside a kernel ran out (sticky, see fdqp_last_status) */
} fdqp_status;

/* ---- Q4NX container (host side; Sec. "Dequantization Engine") ------------- */

/* Bytes of a packed K x N matrix: K*N*5/8 (a 32 x 256 block is 5120 bytes).
 * Returns 0 if K or N is not a positive multiple of 32. */
FDQP_API size_t q4nx_packed_bytes(int64_t K, int64_t N);

/* Pack codes, scales and offsets into the container described above.
 *   codes        host, [N][K], one code per byte, each 0..15 (else FDQP_ERR_ARG)
 *   scales_bf16  host, [N][K/32], raw bf16 bits of d
 *   offsets_bf16 host, [N][K/32], raw bf16 bits of m
 *   out          host, out_bytes >= q4nx_packed_bytes(K, N) (else FDQP_ERR_SIZE)
 * Lossless; the caller keeps ownership of every buffer.  How float weights are
 * turned into (code, d, m) is outside this library. */
FDQP_API fdqp_status q4nx_pack(const uint8_t* codes, const uint16_t* scales_bf16, const uint16_t* offsets_bf16,
                      int64_t K, int64_t N, void* out, size_t out_bytes);

/* Inverse of q4nx_pack (all buffers host, sized as above). */
FDQP_API fdqp_status q4nx_unpack(const void* packed, int64_t K, int64_t N, uint8_t* codes, uint16_t* scales_bf16,
                        uint16_t* offsets_bf16);

/* ---- format variants of the block container ---------------------------------- */

/* The paper describes its dequantisation logic as format-agnostic and the block
 * container as able to take other group sizes and MXFP4.  Every variant keeps the
 * 32 x 256 block and its 4096-byte code section (addressed exactly as in Q4NX);
 * the metadata that follows differs.  With r = n % 32 and c = k % 256:
 *   FDQP_FMT_Q4NX  : the container above (group 32, 5120-byte blocks)
 *   FDQP_FMT_G64   : Eq. 3 with one bf16 scale and offset per 64 inputs:
 *                    scale u16 at 4096 + 2*((c/64)*32 + r), offsets 256 bytes
 *                    further on; 4608-byte blocks (4.5 bits per weight)
 *   FDQP_FMT_G128  : one per 128 inputs: scale at 4096 + 2*((c/128)*32 + r),
 *                    offsets 128 bytes on; 4352-byte blocks (4.25 bits)
 *   FDQP_FMT_MXFP4 : the code is an E2M1 element (bit 3 sign, bits 2..1 exponent,
 *                    bit 0 mantissa: 0, 0.5, 1, 1.5, 2, 3, 4, 6 and negatives), a
 *                    group of 32 shares the E8M0 scale 2^(e-127), e = 0..254, one
 *                    byte at 4096 + (c/32)*32 + r; no offsets; 4352-byte blocks.
 *                    w_hat = element * 2^(e-127), exact in fp32.
 * The variants need K % 256 == 0 and N % 32 == 0 (whole blocks). */
typedef enum { FDQP_FMT_Q4NX = 0, FDQP_FMT_G64 = 1, FDQP_FMT_G128 = 2, FDQP_FMT_MXFP4 = 3 } fdqp_format;

/* Bytes of a packed K x N matrix in `format`; 0 for a shape the format cannot hold. */
FDQP_API size_t q4nx_packed_bytes_fmt(int format, int64_t K, int64_t N);

/* q4nx_pack / q4nx_unpack for any format.  With g the format's group size:
 *   codes    host, [N][K], one code per byte, 0..15
 *   scales   host, [N][K/g]: raw bf16 bits (uint16) for the Eq. 3 formats, the E8M0
 *            byte (uint8, 255 = NaN is refused with FDQP_ERR_ARG) for MXFP4
 *   offsets_bf16  host, [N][K/g] raw bf16 bits; ignored (may be null) for MXFP4
 * Errors as q4nx_pack. */
FDQP_API fdqp_status q4nx_pack_fmt(int format, const uint8_t* codes, const void* scales, const uint16_t* offsets_bf16,
                          int64_t K, int64_t N, void* out, size_t out_bytes);
FDQP_API fdqp_status q4nx_unpack_fmt(int format, const void* packed, int64_t K, int64_t N, uint8_t* codes, void* scales,
                            uint16_t* offsets_bf16);

/* ---- context --------------------------------------------------------------- */

/* Create a context on CUDA device `device` for projections up to max_M x max_K x
 * max_N.  Allocates (device) the split-K workspace and its arrival counters, and, when
 * max_M > 8, up to 128 MB for the partial results of K-split tensor-core calls; the
 * staging buffers of fdqp_run_host are allocated by its first call.  Reads the SM count
 * and shared-memory limits.
 * A context serves one stream at a time: its workspace is not re-entrant.
 * Errors: FDQP_ERR_ARG (null), FDQP_ERR_SHAPE, FDQP_ERR_ARCH (not sm_100),
 * FDQP_ERR_CUDA, FDQP_ERR_NOMEM.  On error *ctx is NULL. */
FDQP_API fdqp_status fdqp_create(fdqp_ctx** ctx, int device, int64_t max_M, int64_t max_K, int64_t max_N);

/* Free everything fdqp_create allocated.  The caller must have synchronised the
 * streams that used the context.  NULL is accepted. */
FDQP_API fdqp_status fdqp_destroy(fdqp_ctx* ctx);

/* ---- the projection (Sec. "FusedDQP", Eq. 14 / 15, with Eq. 3 fused) ------- */

/* y = x * dequant(W).
 *   x_bf16  device, [M][K] bf16, 16-byte aligned
 *   W_q4nx  device, q4nx_packed_bytes(K, N) bytes, 16-byte aligned
 *   y       device, [M][N] fp32, 16-byte aligned; fully overwritten (no accumulate, no bias)
 * Dispatch: M = 1 and 2..8 run the streaming GEMV kernels (weights fetched once
 * from HBM through a shared-memory ring, nibbles unpacked in registers, scale and
 * offset applied in fp32, split-K across CTAs reduced in a fixed order); M >= 9
 * runs either the dequantise-into-shared-memory tensor-core path (tcgen05,
 * accumulators in TMEM; a one-SM kernel up to 256 token rows, a two-SM kernel
 * above; K cut into slices when a shape has few output tiles) or the GEMV kernel
 * eight token rows at a time, whichever a small cost model expects to be faster
 * (GEMV chunks up to about 16-24 rows, or more when N is small).  Reductions
 * shorter than K = 256 always take the GEMV kernels: the tensor-core path
 * multiplies by bf16-rounded weights, whose rounding errors need a long K to
 * average out inside the acceptance bound.
 * How the GEMV kernels hold x.  M <= 2: each 32-group as 31-bit fixed point
 * relative to its largest exponent, in four signed byte planes that ride in the
 * columns of one integer tensor-core MMA per 16 rows -- exact for every bf16
 * within 2^22 of the group's largest magnitude.  A group with anything else (a
 * value more than four million times smaller than its neighbour, a subnormal
 * beside a normal number, an infinity, a NaN) is not rounded: it is flagged,
 * contributes nothing through the tensor cores and is evaluated in fp32, weight
 * by weight as Eq. 3 writes it, inside the same kernel.  M = 3 .. 8: codes and
 * activations are both exact in bf16 and go through the bf16 tensor-core MMA with
 * fp32 accumulation; nothing is rounded and nothing needs a flag.
 * Asynchronous on `cuda_stream`; no allocation and no host synchronisation.  W, x
 * and y must stay valid until the stream has passed the call.  Two calls that
 * share a context must be ordered on one stream.
 * Errors (nothing is launched): FDQP_ERR_ARG, FDQP_ERR_SHAPE, FDQP_ERR_ALIGN,
 * FDQP_ERR_SIZE (beyond the maxima given to fdqp_create), FDQP_ERR_CUDA. */
FDQP_API fdqp_status fdqp_run(fdqp_ctx* ctx, const void* x_bf16, const void* W_q4nx, float* y, int64_t M, int64_t K,
                     int64_t N, void* cuda_stream);

/* Epilogues of fdqp_run_epilogue. */
typedef enum {
    FDQP_EPI_NONE = 0,       /* out = y, fp32 [M][N]: the same as fdqp_run */
    FDQP_EPI_BF16 = 1,       /* out = y rounded to nearest-even bf16, [M][N] */
    FDQP_EPI_GEGLU_BF16 = 2  /* out = gelu(gate) * up as bf16, [M][N/2] (see below) */
} fdqp_epilogue;

/* The projection followed, in the same kernels, by the step that comes after it in a
 * decoder layer.  The paper runs the GELU-and-multiply step as a kernel of its own
 * after the gate and up projections (its section on mapping the decoder) and gives
 * no formula; this entry point fuses it into the projection's store, with GELU in
 * its tanh form 0.5 g (1 + tanh(sqrt(2/pi) (g + 0.044715 g^3))), evaluated in fp32
 * on the fp32 projection results.
 *   FDQP_EPI_GEGLU_BF16: W holds the gate and up matrices fused along N with their
 *   rows interleaved sixteen by sixteen: rows 32j .. 32j+15 of W are gate features
 *   16j .. 16j+15, rows 32j+16 .. 32j+31 are the up features of the same outputs
 *   (a row order for the caller to apply before q4nx_pack).  Output value
 *   out[m][16j + r] = bf16(gelu(y[m][32j + r]) * y[m][32j + 16 + r]), r = 0..15.
 *   out     device, 16-byte aligned; fp32 or bf16 as the epilogue says; fully overwritten
 * Everything else (arguments, dispatch, asynchrony, errors) as fdqp_run; additionally
 * FDQP_ERR_ARG for an unknown epilogue, or for a bf16 epilogue while the "path"
 * parameter selects the plain self-check kernel. */
FDQP_API fdqp_status fdqp_run_epilogue(fdqp_ctx* ctx, const void* x_bf16, const void* W_q4nx, void* out, int epilogue,
                              int64_t M, int64_t K, int64_t N, void* cuda_stream);

/* fdqp_run_epilogue preceded, in the same launch where possible, by the RMS
 * normalisation that comes before a projection in a decoder layer (the paper runs
 * it as a vector kernel of its own and gives no formula; this is the form with
 * scale 1 + weight, evaluated in fp32 and handed on as bf16):
 *   x_n[m][k] = bf16( x[m][k] * rsqrt(mean_k x[m][k]^2 + eps) * (1 + gamma[k]) ),
 *   out = epilogue( x_n * dequant(W) ).
 *   gamma_bf16  device, [K] bf16, 16-byte aligned; eps >= 0
 * The normalisation is fused into the GEMV kernel's activation preparation when the
 * call is a single GEMV launch that prepares the whole row of x inside every CTA
 * (about M * K <= 4096, e.g. every K = 2560 projection at M = 1); otherwise a small
 * kernel writes x_n to a staging buffer of the context first.  x is not modified.
 * Everything else as fdqp_run_epilogue; FDQP_ERR_ARG also for a null gamma or eps < 0. */
FDQP_API fdqp_status fdqp_run_rmsnorm_epilogue(fdqp_ctx* ctx, const void* x_bf16, const void* gamma_bf16, float eps,
                                      const void* W_q4nx, void* out, int epilogue, int64_t M, int64_t K, int64_t N,
                                      void* cuda_stream);

/* fdqp_run_rmsnorm_epilogue with the residual addition that precedes the
 * normalisation in a decoder layer (the paper pairs the two in its vector kernels):
 *   h[m][k]   = bf16( x[m][k] + residual[m][k] )          one rounding of the exact sum
 *   x_n[m][k] = bf16( h[m][k] * rsqrt(mean_k h[m][k]^2 + eps) * (1 + gamma[k]) )
 *   out       = epilogue( x_n * dequant(W) )
 *   residual_bf16  device, [M][K] bf16, 16-byte aligned
 *   h_out_bf16     device, [M][K] bf16, 16-byte aligned, or null: receives h (the
 *                  updated residual stream).  Must not be x or residual themselves:
 *                  every CTA of the fused launch reads those (FDQP_ERR_ARG).
 * Fused into the GEMV launch under the same condition as the normalisation alone
 * (then the grid's first CTA stores h); otherwise the separate normalisation kernel
 * does the addition.  Everything else as fdqp_run_rmsnorm_epilogue. */
FDQP_API fdqp_status fdqp_run_add_rmsnorm_epilogue(fdqp_ctx* ctx, const void* x_bf16, const void* residual_bf16,
                                          void* h_out_bf16, const void* gamma_bf16, float eps, const void* W_q4nx,
                                          void* out, int epilogue, int64_t M, int64_t K, int64_t N, void* cuda_stream);

/* Measurement aid (the paper has no counterpart): reads the first floor(bytes / 40960) * 40960 bytes of `buf` (device,
 * 16-byte aligned) once, one persistent CTA per SM pulling its contiguous share through a shared-memory ring with the
 * bulk copies the projection kernels stream their weights with, and drops the data.  Timed by the caller, it gives the
 * read rate that stream can reach at most on this device (a copy's bandwidth counts a read and a write per byte).
 * Asynchronous on `cuda_stream`; writes nothing but the status word on a timed-out wait.
 * Errors: FDQP_ERR_ARG, FDQP_ERR_ALIGN, FDQP_ERR_CUDA. */
FDQP_API fdqp_status fdqp_stream_read(fdqp_ctx* ctx, const void* buf, int64_t bytes, void* cuda_stream);

/* Decode attention over a KV cache (the paper's FlowKV, and FlowKV-SWA for local
 * layers): the attention of ONE new token at decoding step L,
 *     out[h] = sum_j softmax_j( scale * q[h] . K[g][j] ) V[g][j],   g = h / (H / G),
 * over positions j = 0 .. L-1, or only the last `window` of them (window > 0 and
 * < L: sliding-window attention); evaluated chunk by chunk with a running maximum
 * and a running sum, K and V each read once.  (The paper's equation for the
 * decoding step omits the scale; it is an argument here.)  Short ranges (a sliding
 * window, a young cache; see the "flowkv_cluster" parameter) are one kernel
 * launch, longer ones two.
 *   q_bf16  device, [H][d] bf16
 *   K_bf16, V_bf16  device, [G][pitch][d] bf16: position j of KV head g at
 *           (g * pitch + j) * d; pitch >= L is the cache's capacity in positions
 *   out     device, [H][d] fp32, fully overwritten
 *   H % G == 0, H / G <= 8, H <= 64, d in {128, 256}; all pointers 16-byte aligned
 * Probabilities pass through bf16 before they weight the values (tensor-core
 * operand); bound against an fp64 evaluation, per element:
 *     |out - ref| <= 6e-3 * sum_j p_j |V[g][j]| + 1e-5.
 * Asynchronous on `cuda_stream`; no allocation; uses the context's workspace, so
 * calls sharing a context must be ordered on one stream.
 * Errors: FDQP_ERR_ARG, FDQP_ERR_SHAPE, FDQP_ERR_SIZE, FDQP_ERR_ALIGN, FDQP_ERR_CUDA. */
FDQP_API fdqp_status fdqp_flowkv_decode(fdqp_ctx* ctx, const void* q_bf16, const void* K_bf16, const void* V_bf16, float* out,
                               int64_t H, int64_t G, int64_t d, int64_t L, int64_t pitch, int64_t window, float scale,
                               void* cuda_stream);

/* One step of fdqp_run_chain: a projection as fdqp_run_add_rmsnorm_epilogue describes it (x, optional RMS
 * normalisation with optional residual addition, W, epilogue, out), with M common to the chain. */
typedef struct {
    const void* x_bf16;        /* device, [M][K] bf16, 16-byte aligned */
    const void* W_q4nx;        /* device, q4nx_packed_bytes(K, N) bytes, 16-byte aligned */
    void* out;                 /* device, 16-byte aligned: fp32 [M][N], bf16 [M][N] or bf16 [M][N/2] as `epilogue` says */
    int64_t K, N;
    int epilogue;              /* fdqp_epilogue */
    int depends_on_previous;   /* 1: x_bf16 (or residual_bf16) is the `out` / h_out of the PREVIOUS step of this chain */
    const void* gamma_bf16;    /* not null: RMS-normalise x first (scale 1 + gamma), device [K] bf16 */
    float eps;
    const void* residual_bf16; /* with gamma: h = bf16(x + residual) is what gets normalised; device [M][K] bf16 or null */
    void* h_out_bf16;          /* with residual: receives h, device [M][K] bf16, or null */
} fdqp_chain_step;

/* A chain of projections at M = 1 .. 8 token rows in as few launches as possible: ONE persistent kernel walks up to
 * 160 steps (longer chains, and chains whose steps together need more arrival counters or partial-row slots than the
 * context's workspace holds, are cut into several launches).  The paper keeps all kernels of a decoder layer resident
 * and pipelined on its tile array, the vectors between them staying on chip (its section on mapping the decoder;
 * Sec. "FusedDQP"); here the weight stream of step i + 1 is already filling shared memory while step i finishes, so
 * launch latency and the first trip to HBM are paid once per chain.  Each step computes exactly what
 * fdqp_run_add_rmsnorm_epilogue computes for the same arguments (Eq. 14 / 15 with Eq. 3 fused; same acceptance
 * bound; results reproducible run to run, though the summation order may differ from the single call's).
 *   depends_on_previous = 1  the step starts its activations only after every output of the previous step is in
 *                            global memory.  Example: gate|up with FDQP_EPI_GEGLU_BF16 followed by the down projection
 *                            on its output.  A dependency on any EARLIER step than the previous one is not tracked.
 *                            By default such a step begins a new launch (the stream order is the dependency; a step
 *                            alone in its launch goes out as the single call it is equivalent to), which measured
 *                            faster than the alternative the "chain_dependent" parameter selects: the step stays in
 *                            the same launch and waits on a counter of the previous step's stored outputs (a bounded
 *                            wait: FDQP_ERR_TIMEOUT in fdqp_last_status if it runs out).
 *   depends_on_previous = 0  the step's inputs must not be written by any step of the chain.
 * A step's outputs must not alias the inputs of another step unless that step depends on it.
 * Limits: 1 <= M <= 8; Q4NX only; a normalised step that shares its launch with others needs its whole row prepared in
 * one piece (M * K <= 13056 for M <= 2, M * K <= 32768 above: every K = 2560 projection qualifies); shapes within the
 * context's maxima.
 * Asynchronous on `cuda_stream`; no allocation; uses the context's chain workspace, so calls that share a context
 * must be ordered on one stream.
 * Errors (found before anything is launched): FDQP_ERR_ARG (null pointers, n_steps < 1, unknown epilogue, dependency flag on the
 * first step, residual without gamma), FDQP_ERR_SHAPE, FDQP_ERR_ALIGN, FDQP_ERR_SIZE (beyond the context's maxima,
 * M > 8, a normalised step whose row does not fit one K slice, workspace exhausted), FDQP_ERR_CUDA. */
FDQP_API fdqp_status fdqp_run_chain(fdqp_ctx* ctx, const fdqp_chain_step* steps, int64_t n_steps, int64_t M,
                                    void* cuda_stream);

/* Same projection with HOST activations and result: copies x (host, [M][K] bf16)
 * to the context's device staging buffer, runs fdqp_run, copies y back to `y_host`
 * (host, [M][N] fp32) and synchronises the stream before returning.  W stays a
 * device pointer (weights are resident model state).  Pinned host memory makes
 * the copies asynchronous but is not required.  Page-locked buffers the device can
 * address (e.g. cudaHostAlloc) of at most 1 MiB are used in place ("host_direct_y"
 * parameter, default 1): the kernels store y there themselves, and up to eight
 * token rows of x are read from there by the activation-preparation kernel; no
 * copy is issued for them. */
FDQP_API fdqp_status fdqp_run_host(fdqp_ctx* ctx, const void* x_host_bf16, const void* W_q4nx, float* y_host,
                          int64_t M, int64_t K, int64_t N, void* cuda_stream);

/* fdqp_run_host without the final synchronisation: the copy of x, the projection
 * and the copy of y are enqueued on `cuda_stream` and the call returns.  x_host and
 * y_host (host; pinned memory for the copies to be asynchronous) must stay valid
 * and untouched until the stream has passed the call; y_host holds the result once
 * the caller has synchronised the stream, after which fdqp_last_status tells whether
 * a kernel gave up.  Several calls may be queued on one stream (they share the
 * context's staging buffers in stream order); calls on different streams must not
 * share a context.  Errors as fdqp_run. */
FDQP_API fdqp_status fdqp_run_host_async(fdqp_ctx* ctx, const void* x_host_bf16, const void* W_q4nx, float* y_host,
                                int64_t M, int64_t K, int64_t N, void* cuda_stream);

/* The same projection for callers that must not allocate device memory at the time of the call -- a server that
 * gave all device memory to its own pool at start-up, a real-time loop that cannot take the device-wide
 * synchronisation an allocation may bring, a plug-in that may not allocate after initialisation.  (The paper has no
 * counterpart: this is a packaging of fdqp_run's GEMV kernel, not another operation.)
 *   x_bf16, W_q4nx, y   device pointers, 16-byte aligned, as for fdqp_run; runs on the CURRENT device
 *   limits              M <= 8; N <= 262144; and the prepared activations must fit shared memory without
 *                       splitting K (about M*K <= 32768, e.g. K <= 3840 at M = 8); beyond them FDQP_ERR_SIZE.
 *                       A bounded wait that ran out inside the kernel is reported by fdqp_noalloc_last_status.
 * It takes no context and calls no cudaMalloc / cudaFree or any other allocating routine.  Its scratch -- the
 * partial-row slots of strips shared between CTAs, their arrival counters, a status word -- is a 688,384-byte
 * array inside the library image, resident on every device that loads the library until the process exits.
 * The first call on a device looks up the device's limits and the array's device address; make that first call
 * before any stream capture.  Every call clears the arrival counters it is going to use (a cudaMemsetAsync on
 * the stream) and then launches the kernel; the rest of the array keeps the previous call's contents.
 * All calls on a device share the one array: calls whose kernels could overlap on the GPU (different streams,
 * no dependency between them) race and give wrong results -- keep them on one stream or order them.
 * Asynchronous on `cuda_stream`.  Errors (nothing is launched): FDQP_ERR_ARG, FDQP_ERR_SHAPE, FDQP_ERR_ALIGN,
 * FDQP_ERR_SIZE, FDQP_ERR_ARCH, FDQP_ERR_CUDA. */
FDQP_API fdqp_status fdqp_run_noalloc(const void* x_bf16, const void* W_q4nx, float* y, int64_t M, int64_t K,
                                      int64_t N, void* cuda_stream);

/* Did a kernel of fdqp_run_noalloc give up on a bounded wait?  That entry point has no context to keep a status in,
 * so its kernels record FDQP_ERR_TIMEOUT in a word of the scratch array; this call copies that word back from the
 * CURRENT device (one blocking 4-byte device-to-host copy: call it after synchronising the stream; it allocates
 * nothing).  FDQP_OK when no kernel gave up, or when fdqp_run_noalloc has not run on this device yet;
 * FDQP_ERR_TIMEOUT once one did -- sticky until the process exits, and the y of that call is undefined (the next
 * call clears the arrival counters it uses, so later calls are unaffected).  FDQP_ERR_CUDA if the copy fails.
 * (The paper has no counterpart.) */
FDQP_API fdqp_status fdqp_noalloc_last_status(void);

/* ---- the dequantisation engine (Sec. "Dequantization Engine", Eq. 3) ------- */

/* Write the dequantised matrix w_hat[k][n] to `out` (device, [K][N] row-major,
 * 16-byte aligned): fp32 when out_is_bf16 == 0, else bf16 = RNE(fp32 value).
 * Bit-exact by definition (one rounding to fp32).  Asynchronous on the stream. */
FDQP_API fdqp_status fdqp_dequant(fdqp_ctx* ctx, const void* W_q4nx, void* out, int out_is_bf16, int64_t K, int64_t N,
                         void* cuda_stream);

/* fdqp_run and fdqp_dequant for a matrix packed in `format` (fdqp_format).  Same
 * arguments, results, acceptance bound (dequantised values bit-exact; y within
 * 2e-3 * sum_k |x_k w_hat_k| + 1e-5 of the fp64 product), asynchrony and errors as
 * fdqp_run / fdqp_dequant; FDQP_FMT_Q4NX is exactly those calls.  Dispatch on M as
 * in fdqp_run: the streaming GEMV kernels up to eight token rows, the tensor-core
 * kernels (which dequantise the format into shared memory) above.  In the GEMV
 * kernels an MXFP4 scale byte of 0 (2^-127, below 1e-38) counts as a scale of zero;
 * the tensor-core kernels and the dequantisation engine use it exactly.  FDQP_ERR_ARG for an unknown
 * format, FDQP_ERR_SHAPE when K is not a multiple of 256. */
FDQP_API fdqp_status fdqp_run_fmt(fdqp_ctx* ctx, int format, const void* x_bf16, const void* W_packed, float* y, int64_t M,
                         int64_t K, int64_t N, void* cuda_stream);
FDQP_API fdqp_status fdqp_dequant_fmt(fdqp_ctx* ctx, int format, const void* W_packed, void* out, int out_is_bf16, int64_t K,
                             int64_t N, void* cuda_stream);

/* ---- status, tuning, introspection ---------------------------------------- */

/* Sticky device-side status: FDQP_ERR_TIMEOUT once any kernel of this context gave
 * up on a bounded wait (its output is then undefined), else FDQP_OK.  Reads a
 * host-mapped word: call it after synchronising the stream; it synchronises
 * nothing itself.  Cleared only by fdqp_destroy. */
FDQP_API fdqp_status fdqp_last_status(fdqp_ctx* ctx);

/* Exercises the give-up path that every device-side wait of the library shares
 * (all of them are bounded; a wait that runs out records FDQP_ERR_TIMEOUT in the
 * context's status word and the kernel returns normally, freeing what it holds):
 * enqueues one warp that waits on a barrier nothing arrives on, with that same
 * wait and a limit of `limit_us` microseconds (1 .. 100000).  After the caller has
 * synchronised the stream, fdqp_last_status(ctx) is FDQP_ERR_TIMEOUT (sticky for
 * this context); the device and other contexts are unaffected.  Nothing faults
 * and nothing is left running.  Errors: FDQP_ERR_ARG (null ctx, limit out of
 * range), FDQP_ERR_CUDA. */
FDQP_API fdqp_status fdqp_selftest_bounded_wait(fdqp_ctx* ctx, int64_t limit_us, void* cuda_stream);

/* Text of the last CUDA runtime error seen by this context ("" if none).  The
 * pointer stays valid until the next failing call or fdqp_destroy. */
FDQP_API const char* fdqp_last_cuda_error(fdqp_ctx* ctx);

/* Human-readable name of a status code (static storage). */
FDQP_API const char* fdqp_status_string(fdqp_status s);

/* Override a launch parameter; value < 0 restores the built-in choice.  Keys:
 *   "path"          0 = dispatch on M (default), 1 = force the plain CUDA-core kernel,
 *                   2 = run M >= 9 through the GEMV kernel eight token rows at a time,
 *                   3 = run every M >= 9 through the tensor-core prefill kernel (also K < 256, which the
 *                   dispatch keeps off it: with so few terms the bf16 rounding of the weights does not average
 *                   out and single outputs can land a few per cent outside the acceptance bound)
 *   "ctas_per_sm"   persistent CTAs per SM for the GEMV kernels (1 or 2; 2 implies 8 consumer warps)
 *   "consumer_warps" 8 or 16 consumer warps per CTA
 *   "stages"        shared-memory ring depth in stages (a stage holds consumer_warps / 8 * blocks_per_warp blocks)
 *   "blocks_per_warp" 2 or 4 Q4NX blocks per consumer warp per stage
 *   "split_k"       number of K slices (1, 2, 4 or 8)
 *   "l2_evict_first" 1 = weight copies carry an evict-first L2 hint
 *   "strip_aligned" 1 = CTA work ranges are cut at strip boundaries, 0 = equal block counts per CTA
 *   "prep_inline"   1 = every GEMV CTA prepares its slice of x itself, 0 = a preparation kernel runs first
 *   "chain_launch"  fdqp_run_chain: bit 0 = programmatic stream serialisation (default on), bit 1 = cooperative launch
 *   "chain_steps"   fdqp_run_chain: most steps per launch (1 .. 160, default 160)
 *   "chain_dependent" fdqp_run_chain: 0 (default) = a step with depends_on_previous begins a new launch; 1 = it stays in
 *                   the launch and waits on the previous step's completion counter
 *   "chain_wide"    fdqp_run_chain: 1 (default) = a launch none of whose steps depends on another is cut into CTA ranges
 *                   as one sequence of blocks, 0 = every step is cut on its own
 *   "flowkv_cluster" fdqp_flowkv_decode: ranges of up to this many positions (default 2048; 0 = never) run as ONE launch,
 *                   the splits of a KV head as a thread-block cluster merged through distributed shared memory;
 *                   longer ranges take the two-launch route (split kernel + merge kernel)
 *   "prefill_split_k" 1..8 K slices for the tensor-core kernels (their partial results are added by a second
 *                   kernel); default: as many as fill the SMs when a shape has few output tiles
 *   "prefill_pair"  1 = prefill-sized calls use the two-SM kernel (256 x 512 tile per CTA pair), 0 = the one-SM kernel
 *                   (256 x 256 tile; 128 x 128 tiles, two CTAs per SM, up to 128 token rows); default: two-SM kernel
 *                   when M > 256
 *   "host_direct_y" fdqp_run_host*: 1 (default) = small x and y in device-addressable page-locked host memory are
 *                   read / written in place by the kernels, 0 = always through the staging buffers and copies
 *   "prefill_a_tmem" one-SM tensor-core kernel up to 128 token rows: 1 (default) = the converted weights are kept in
 *                   tensor memory and read from there by the MMAs (two CTAs per SM; up to 64 token rows three smaller
 *                   CTAs per SM when the call has that many to run), 2 = the three-CTA form whenever M <= 64,
 *                   0 = weights in shared memory; same results bit for bit
 * Unknown key or unusable value: FDQP_ERR_ARG.  Meant for benchmarks and tests. */
FDQP_API fdqp_status fdqp_set_param(fdqp_ctx* ctx, const char* key, int64_t value);

/* Number of kernels this context has launched since it was created. */
FDQP_API int64_t fdqp_launch_count(fdqp_ctx* ctx);

/* Describe the launch fdqp_run would make for (M, K, N) into `buf` (host,
 * NUL-terminated, truncated to buf_bytes): kernel name, grid, block, shared
 * memory, stages, split.  Launches nothing. */
FDQP_API fdqp_status fdqp_describe(fdqp_ctx* ctx, int64_t M, int64_t K, int64_t N, char* buf, size_t buf_bytes);

#ifdef __cplusplus
}
#endif
#endif /* FDQP_H */
