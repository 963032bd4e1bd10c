/*
 * Seeded synthetic tensor generator shared by the CPU oracle's tests and the
 * GPU path's tests/benchmarks.  It holds no arithmetic of the verify step: it
 * only fills buffers with reproducible pseudo-random values.
 *
 * Generator: counter-based.  Value j of stream `seed` is drawn from two
 * SplitMix64 outputs (counters 2j and 2j+1) turned into uniforms in (0,1] and
 * [0,1) and pushed through the cosine branch of the Box-Muller transform, all
 * in double precision, then rounded once (round-to-nearest-even) to the
 * storage type.  Every element is addressable by its index, so a sub-range of
 * a tensor can be regenerated without the rest.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

static inline uint64_t splitmix64_at(uint64_t seed, uint64_t counter) {
    uint64_t z = seed + (counter + 1ull) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static inline double normal_at(uint64_t seed, uint64_t j) {
    const double two_pi = 6.283185307179586476925286766559;
    uint64_t a = splitmix64_at(seed, 2ull * j);
    uint64_t b = splitmix64_at(seed, 2ull * j + 1ull);
    double u1 = ((double)(a >> 11) + 1.0) * (1.0 / 9007199254740992.0); /* (0,1] */
    double u2 = (double)(b >> 11) * (1.0 / 9007199254740992.0);         /* [0,1) */
    return sqrt(-2.0 * log(u1)) * cos(two_pi * u2);
}

/* out[j] = mean + std * z_j, j in [first, first+count), stored as float32. */
void wl_fill_normal_f32(float *out, uint64_t first, uint64_t count,
                        uint64_t seed, double mean, double std) {
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < (int64_t)count; ++j)
        out[j] = (float)(mean + std * normal_at(seed, first + (uint64_t)j));
}

/* Same values rounded to IEEE binary16, written as raw 16-bit patterns. */
void wl_fill_normal_f16(uint16_t *out, uint64_t first, uint64_t count,
                        uint64_t seed, double mean, double std) {
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < (int64_t)count; ++j) {
        _Float16 h = (_Float16)(mean + std * normal_at(seed, first + (uint64_t)j));
        uint16_t bits;
        __builtin_memcpy(&bits, &h, 2);
        out[j] = bits;
    }
}

/* out[j] = SplitMix64 output number (first + j) of stream `seed`. */
void wl_fill_u64(uint64_t *out, uint64_t first, uint64_t count, uint64_t seed) {
    for (uint64_t j = 0; j < count; ++j) out[j] = splitmix64_at(seed, first + j);
}
