/* Seeded synthetic-input generator (fast path, plain C + OpenMP).
 *
 * This file holds NO arithmetic of the inference method: it only turns
 * (seed, tensor uid, flat index) into a reproducible pseudo-random weight.
 * It is the compiled twin of tpi_synth/gen.py (same integers, same bits) and
 * serves both the CPU oracle's tests and the GPU harness as an input source.
 *
 * Recipe (counter based, integer exact until the last step):
 *   key = mix64(seed XOR uid)
 *   r1  = mix64(key + 2*idx), r2 = mix64(key + 2*idx + 1)
 *   S   = sum of the eight 16-bit fields of r1 and r2      (Irwin-Hall, n = 8)
 *   z   = (S - 262140) / 53509.91992145008                 (fp64, one division)
 *   w   = (float)(offset + scale * z)
 * and, for bf16 storage, round-to-nearest-even of w to its upper 16 bits.
 * mix64 is the published splitmix64 finaliser.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>

static inline uint64_t mix64(uint64_t x) {
    x += 0x9E3779B97F4A7C15ULL;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ULL;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBULL;
    return x ^ (x >> 31);
}

static inline float draw(uint64_t key, uint64_t idx, double offset, double scale) {
    uint64_t r1 = mix64(key + 2 * idx), r2 = mix64(key + 2 * idx + 1);
    uint32_t s = 0;
    for (int k = 0; k < 4; ++k) {
        s += (uint32_t)((r1 >> (16 * k)) & 0xFFFF);
        s += (uint32_t)((r2 >> (16 * k)) & 0xFFFF);
    }
    double z = ((double)s - 262140.0) / 53509.91992145008;
    return (float)(offset + scale * z);
}

static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u); /* values here are finite and small */
    return (uint16_t)(u >> 16);
}

/* Fill dst[0..count) with elements start .. start+count-1 of the tensor.
 * as_bf16 = 0: dst is float[count]; 1: dst is uint16_t[count] (bf16 bits). */
void tpi_synth_fill(uint64_t seed, uint64_t uid, uint64_t start, uint64_t count,
                    double offset, double scale, int as_bf16, void *dst) {
    const uint64_t key = mix64(seed ^ uid);
    if (as_bf16) {
        uint16_t *o = (uint16_t *)dst;
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < (int64_t)count; ++i)
            o[i] = f32_to_bf16_rne(draw(key, start + (uint64_t)i, offset, scale));
    } else {
        float *o = (float *)dst;
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < (int64_t)count; ++i)
            o[i] = draw(key, start + (uint64_t)i, offset, scale);
    }
}
