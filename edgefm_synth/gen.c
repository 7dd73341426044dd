/*
 * Seeded synthetic-input generator shared by the CPU oracle's tests and the CUDA path's tests.
 *
 * It holds none of the decoder's arithmetic: it only turns (seed, tensor id, element index) into
 * a reproducible bf16 sample of N(0, std^2).  Counter based, so every element is independent of
 * generation order and of the number of threads.
 *
 *   key   = mix64(seed * GOLDEN + tensor_id)
 *   z     = mix64(key + (i + 1) * GOLDEN)
 *   u1    = ((z >> 32) + 1) / 2^32      in (0, 1]
 *   u2    = (z & 0xffffffff) / 2^32     in [0, 1)
 *   value = bf16_rne( (float)( std * sqrt(-2 ln u1) * cos(2 pi u2) ) )     (Box-Muller, cosine branch)
 */
#include <math.h>
#include <stdint.h>

#define GOLDEN 0x9E3779B97F4A7C15ULL

static inline uint64_t mix64(uint64_t z) {
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ULL;
    z ^= z >> 27; z *= 0x94D049BB133111EBULL;
    z ^= z >> 31;
    return z;
}

static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    __builtin_memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u); /* quiet NaN */
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

uint64_t synth_key(uint64_t seed, uint64_t tensor_id) { return mix64(seed * GOLDEN + tensor_id); }

uint64_t synth_u64(uint64_t seed, uint64_t tensor_id, uint64_t i) {
    return mix64(synth_key(seed, tensor_id) + (i + 1) * GOLDEN);
}

/* out[j] = sample for element index (offset + j), j in [0, n). */
void synth_normal_bf16(uint64_t seed, uint64_t tensor_id, uint64_t offset, uint64_t n, double std,
                       uint16_t *out) {
    const uint64_t key = synth_key(seed, tensor_id);
    const double two_pi = 6.283185307179586476925286766559;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < (int64_t)n; ++j) {
        uint64_t z = mix64(key + (offset + (uint64_t)j + 1) * GOLDEN);
        double u1 = ((double)(z >> 32) + 1.0) * (1.0 / 4294967296.0);
        double u2 = (double)(z & 0xffffffffULL) * (1.0 / 4294967296.0);
        double g = sqrt(-2.0 * log(u1)) * cos(two_pi * u2);
        out[j] = f32_to_bf16_rne((float)(std * g));
    }
}
