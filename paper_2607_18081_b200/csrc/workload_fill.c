/*
 * Seeded synthetic-tensor filler for the benchmark and test workloads.
 *
 * Fills a buffer with N(0, std) samples rounded (nearest-even) to fp16 or bf16 bit
 * patterns.  Counter based: element pair p of a tensor with 64-bit key K is a pure
 * function of (K, p), so any slice can be regenerated and threads need no shared
 * state.  This file holds no arithmetic of the selective FFN itself; it only makes
 * inputs, which the CUDA library and its CPU yardstick both read.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static inline uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

static inline uint16_t f32_to_f16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t sign = (u >> 16) & 0x8000u;
    uint32_t a = u & 0x7FFFFFFFu;
    if (a >= 0x47800000u) return (uint16_t)(sign | 0x7C00u);          /* overflow -> inf */
    if (a < 0x38800000u) {                                            /* subnormal half */
        if (a < 0x33000000u) return (uint16_t)sign;                   /* < 2^-25 -> 0 */
        uint32_t e = a >> 23;                                         /* 102..112 */
        uint32_t m = (a & 0x7FFFFFu) | 0x800000u;
        uint32_t shift = 126u - e;                                    /* 14..24 */
        uint32_t q = m >> shift, rem = m & ((1u << shift) - 1u), half = 1u << (shift - 1);
        if (rem > half || (rem == half && (q & 1u))) q++;
        return (uint16_t)(sign | q);
    }
    uint32_t v = a - 0x38000000u;                                     /* rebias 127 -> 15 */
    v += 0xFFFu + ((v >> 13) & 1u);
    return (uint16_t)(sign | (v >> 13));
}

/* dtype: 1 = fp16, 2 = bf16.  n elements; first = index of the first element (even). */
void wl_fill_normal(uint16_t *out, uint64_t first, uint64_t n, uint64_t key, float std,
                    int dtype, int threads) {
    const float two_pi = 6.28318530717958647692f;
    uint64_t pairs = (n + 1) / 2;
    if (threads < 1) threads = 1;
#pragma omp parallel for num_threads(threads) schedule(static)
    for (uint64_t q = 0; q < pairs; ++q) {
        uint64_t p = first / 2 + q;
        uint64_t h1 = mix64(key ^ mix64(2 * p));
        uint64_t h2 = mix64(key ^ mix64(2 * p + 1));
        float u1 = (float)((h1 >> 40) + 1) * (1.0f / 16777216.0f);   /* (0, 1] */
        float u2 = (float)(h2 >> 40) * (1.0f / 16777216.0f);         /* [0, 1) */
        float r = std * sqrtf(-2.0f * logf(u1));
        float a = r * cosf(two_pi * u2), b = r * sinf(two_pi * u2);
        uint64_t i = 2 * q;
        out[i] = dtype == 1 ? f32_to_f16_rne(a) : f32_to_bf16_rne(a);
        if (i + 1 < n) out[i + 1] = dtype == 1 ? f32_to_f16_rne(b) : f32_to_bf16_rne(b);
    }
}
