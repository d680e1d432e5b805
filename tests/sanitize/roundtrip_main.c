/* Round-trip driver for the host-side sanitizer test: the library's packer (q4nx_host.cpp) and the oracle's reader and
 * arithmetic (oracle_q4nx.c) are compiled together with -fsanitize=address,undefined and driven over shapes with ragged
 * tail blocks, every format variant and exact-fit buffers, so that an out-of-bounds access or undefined behaviour in
 * either aborts the process.  Deterministic inputs from a small LCG; exits 0 when every comparison holds. */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "fdqp.h"

size_t oracle_packed_bytes(int64_t K, int64_t N);
int oracle_unpack(const uint8_t *packed, int64_t K, int64_t N, uint8_t *codes, uint16_t *scales, uint16_t *offsets);
int oracle_dequant(const uint8_t *codes, const uint16_t *scales, const uint16_t *offsets, int64_t K, int64_t N, int64_t n0,
                   int64_t n1, float *w32, uint16_t *w16);
int oracle_project_packed(const uint16_t *x_bf16, const uint8_t *packed, int64_t M, int64_t K, int64_t N, int64_t n0,
                          int64_t n1, int use_w16, int nthreads, double *y, double *abs_sum);
size_t oracle_fmt_packed_bytes(int fmt, int64_t K, int64_t N);
int oracle_fmt_unpack(int fmt, const uint8_t *packed, int64_t K, int64_t N, uint8_t *codes, uint16_t *scales,
                      uint16_t *offsets);

static uint32_t lcg_state = 12345u;
static uint32_t lcg(void) {
    lcg_state = lcg_state * 1664525u + 1013904223u;
    return lcg_state >> 8;
}

#define CHECK(cond)                                                          \
    do {                                                                     \
        if (!(cond)) {                                                       \
            fprintf(stderr, "%s:%d: check failed: %s\n", __FILE__, __LINE__, #cond); \
            exit(1);                                                         \
        }                                                                    \
    } while (0)

static void q4nx_case(int64_t K, int64_t N) {
    const int64_t G = K / 32;
    uint8_t *codes = malloc((size_t)(N * K)), *codes2 = malloc((size_t)(N * K)), *codes3 = malloc((size_t)(N * K));
    uint16_t *sc = malloc((size_t)(N * G) * 2), *of = malloc((size_t)(N * G) * 2);
    uint16_t *sc2 = malloc((size_t)(N * G) * 2), *of2 = malloc((size_t)(N * G) * 2);
    uint16_t *sc3 = malloc((size_t)(N * G) * 2), *of3 = malloc((size_t)(N * G) * 2);
    for (int64_t i = 0; i < N * K; ++i) codes[i] = (uint8_t)(lcg() & 15u);
    for (int64_t i = 0; i < N * G; ++i) {
        sc[i] = (uint16_t)(0x3c00u + (lcg() & 0xffu));  /* positive scales around 2^-7 */
        of[i] = (uint16_t)(((lcg() & 1u) << 15) | 0x3b00u | (lcg() & 0xffu));
    }
    const size_t bytes = q4nx_packed_bytes(K, N);
    CHECK(bytes == (size_t)(K * N * 5 / 8));
    CHECK(bytes == oracle_packed_bytes(K, N));
    uint8_t *packed = malloc(bytes);  /* exact fit: one byte too many written is an ASan report */
    CHECK(q4nx_pack(codes, sc, of, K, N, packed, bytes) == FDQP_OK);
    CHECK(q4nx_pack(codes, sc, of, K, N, packed, bytes - 1) == FDQP_ERR_SIZE);
    CHECK(oracle_unpack(packed, K, N, codes2, sc2, of2) == 0);
    CHECK(q4nx_unpack(packed, K, N, codes3, sc3, of3) == FDQP_OK);
    CHECK(!memcmp(codes, codes2, (size_t)(N * K)) && !memcmp(codes, codes3, (size_t)(N * K)));
    CHECK(!memcmp(sc, sc2, (size_t)(N * G) * 2) && !memcmp(sc, sc3, (size_t)(N * G) * 2));
    CHECK(!memcmp(of, of2, (size_t)(N * G) * 2) && !memcmp(of, of3, (size_t)(N * G) * 2));
    /* the oracle's arithmetic over the same buffers: every output column, two token rows */
    float *w32 = malloc((size_t)(K * N) * 4);
    uint16_t *w16 = malloc((size_t)(K * N) * 2);
    CHECK(oracle_dequant(codes, sc, of, K, N, 0, N, w32, w16) == 0);
    uint16_t *x = malloc((size_t)(2 * K) * 2);
    for (int64_t i = 0; i < 2 * K; ++i) x[i] = (uint16_t)(((lcg() & 1u) << 15) | 0x3f00u | (lcg() & 0x7fu));
    double *y = malloc((size_t)(2 * N) * 8), *a = malloc((size_t)(2 * N) * 8);
    CHECK(oracle_project_packed(x, packed, 2, K, N, 0, N, 0, 1, y, a) == 0);
    for (int64_t i = 0; i < 2 * N; ++i) CHECK(a[i] >= (y[i] < 0 ? -y[i] : y[i]) * (1.0 - 1e-12));
    /* a bad code is refused, nothing past the buffers is touched */
    codes[N * K - 1] = 16;
    CHECK(q4nx_pack(codes, sc, of, K, N, packed, bytes) == FDQP_ERR_ARG);
    free(codes); free(codes2); free(codes3); free(sc); free(of); free(sc2); free(of2); free(sc3); free(of3);
    free(packed); free(w32); free(w16); free(x); free(y); free(a);
}

static void fmt_case(int fmt, int64_t K, int64_t N) {
    const int64_t g = fmt == FDQP_FMT_G64 ? 64 : (fmt == FDQP_FMT_G128 ? 128 : 32), G = K / g;
    const int mx = fmt == FDQP_FMT_MXFP4;
    uint8_t *codes = malloc((size_t)(N * K)), *codes2 = malloc((size_t)(N * K)), *codes3 = malloc((size_t)(N * K));
    uint16_t *of = malloc((size_t)(N * G) * 2), *of2 = malloc((size_t)(N * G) * 2), *of3 = malloc((size_t)(N * G) * 2);
    uint16_t *sc16 = malloc((size_t)(N * G) * 2), *sc2 = malloc((size_t)(N * G) * 2), *sc3 = malloc((size_t)(N * G) * 2);
    uint8_t *sc8 = malloc((size_t)(N * G)), *sc8b = malloc((size_t)(N * G));
    for (int64_t i = 0; i < N * K; ++i) codes[i] = (uint8_t)(lcg() & 15u);
    for (int64_t i = 0; i < N * G; ++i) {
        sc16[i] = (uint16_t)(0x3c00u + (lcg() & 0xffu));
        sc8[i] = (uint8_t)(118u + lcg() % 5u);
        of[i] = (uint16_t)(0x3b00u | (lcg() & 0xffu));
    }
    const size_t bytes = q4nx_packed_bytes_fmt(fmt, K, N);
    CHECK(bytes != 0 && bytes == oracle_fmt_packed_bytes(fmt, K, N));
    uint8_t *packed = malloc(bytes);
    CHECK(q4nx_pack_fmt(fmt, codes, mx ? (const void *)sc8 : (const void *)sc16, mx ? NULL : of, K, N, packed, bytes) == FDQP_OK);
    CHECK(oracle_fmt_unpack(fmt, packed, K, N, codes2, sc2, mx ? NULL : of2) == 0);
    CHECK(!memcmp(codes, codes2, (size_t)(N * K)));
    for (int64_t i = 0; i < N * G; ++i) CHECK(sc2[i] == (mx ? (uint16_t)sc8[i] : sc16[i]));
    if (!mx) CHECK(!memcmp(of, of2, (size_t)(N * G) * 2));
    CHECK(q4nx_unpack_fmt(fmt, packed, K, N, codes3, mx ? (void *)sc8b : (void *)sc3, mx ? NULL : of3) == FDQP_OK);
    CHECK(!memcmp(codes, codes3, (size_t)(N * K)));
    if (mx) CHECK(!memcmp(sc8, sc8b, (size_t)(N * G)));
    else CHECK(!memcmp(sc16, sc3, (size_t)(N * G) * 2) && !memcmp(of, of3, (size_t)(N * G) * 2));
    free(codes); free(codes2); free(codes3); free(of); free(of2); free(of3); free(sc16); free(sc2); free(sc3);
    free(sc8); free(sc8b); free(packed);
}

int main(void) {
    const int64_t shapes[][2] = {{32, 32}, {64, 32}, {224, 64}, {256, 32}, {288, 96}, {1152, 64}, {2560, 32}, {544, 160}};
    for (size_t i = 0; i < sizeof(shapes) / sizeof(shapes[0]); ++i) q4nx_case(shapes[i][0], shapes[i][1]);
    for (int fmt = FDQP_FMT_G64; fmt <= FDQP_FMT_MXFP4; ++fmt) {
        fmt_case(fmt, 256, 32);
        fmt_case(fmt, 768, 96);
    }
    CHECK(q4nx_packed_bytes(250, 32) == 0 && q4nx_packed_bytes(256, 31) == 0 && q4nx_packed_bytes(0, 32) == 0);
    CHECK(q4nx_packed_bytes_fmt(FDQP_FMT_G64, 288, 32) == 0);
    puts("sanitized round trips ok");
    return 0;
}
