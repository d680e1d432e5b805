/*
 * Seeded synthetic inputs for Q4NX projections.
 *
 * This module only draws numbers: a counter-based generator (every element is
 * a pure function of (seed, stream, index), so any thread count gives the same
 * bits) and the value recipes for codes, scales, offsets and activations.  It
 * holds none of the projection's arithmetic and is used by both the CPU oracle's
 * tests and the CUDA path's tests, so both see identical inputs.
 *
 * Recipe:
 *   r(seed, stream, i) = mix64(key(seed, stream) + i * GOLDEN)
 *   code   = r >> 60                                   uniform 0..15
 *   z      = sqrt(-2 ln u1) * cos(2 pi u2)             Box-Muller, fp64
 *            u1 = ((r1 >> 11) + 1) * 2^-53, u2 = (r2 >> 11) * 2^-53
 *   scale  = bf16(|sigma_d * z|),  offset = bf16(sigma_m * z),  x = bf16(a * z)
 *   bf16() = round-to-nearest-even of the fp32 rounding of the fp64 value.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#define GOLDEN 0x9E3779B97F4A7C15ull

static uint64_t mix64(uint64_t z) {
    z += GOLDEN;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static uint64_t stream_key(uint64_t seed, uint64_t stream) {
    return mix64(mix64(seed) ^ (stream * 0xD6E8FEB86659FD93ull));
}

static uint64_t draw(uint64_t key, uint64_t i) { return mix64(key + i * GOLDEN); }

static uint16_t to_bf16(double v) {
    float f = (float)v;
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

static double normal_at(uint64_t k1, uint64_t k2, uint64_t i) {
    double u1 = (double)((draw(k1, i) >> 11) + 1) * (1.0 / 9007199254740992.0);
    double u2 = (double)(draw(k2, i) >> 11) * (1.0 / 9007199254740992.0);
    return sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925286766559 * u2);
}

/* raw 64-bit draws, for tests that build structured inputs */
void synth_u64(uint64_t seed, uint64_t stream, int64_t count, uint64_t *out) {
    uint64_t k = stream_key(seed, stream);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) out[i] = draw(k, (uint64_t)i);
}

/* codes[count], one 4-bit code per byte; stream 0 */
void synth_codes(uint64_t seed, int64_t count, uint8_t *out) {
    uint64_t k = stream_key(seed, 0);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) out[i] = (uint8_t)(draw(k, (uint64_t)i) >> 60);
}

/* bf16(|sigma * z|); streams 1, 2 */
void synth_scales(uint64_t seed, int64_t count, double sigma, uint16_t *out) {
    uint64_t k1 = stream_key(seed, 1), k2 = stream_key(seed, 2);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) out[i] = to_bf16(fabs(sigma * normal_at(k1, k2, (uint64_t)i)));
}

/* bf16(sigma * z); streams 3, 4 */
void synth_offsets(uint64_t seed, int64_t count, double sigma, uint16_t *out) {
    uint64_t k1 = stream_key(seed, 3), k2 = stream_key(seed, 4);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) out[i] = to_bf16(sigma * normal_at(k1, k2, (uint64_t)i));
}

/* bf16(amp * z); streams 5, 6 */
void synth_x(uint64_t seed, int64_t count, double amp, uint16_t *out) {
    uint64_t k1 = stream_key(seed, 5), k2 = stream_key(seed, 6);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) out[i] = to_bf16(amp * normal_at(k1, k2, (uint64_t)i));
}
