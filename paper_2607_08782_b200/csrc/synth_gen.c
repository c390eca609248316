/*
 * Seeded synthetic-input generator (host, plain C + OpenMP).
 *
 * Holds no arithmetic of the MoE layer itself: it only produces reproducible
 * pseudo-random numbers that both the CUDA library and the CPU oracle receive
 * as inputs.  The generator is counter based, so element i of a stream can be
 * produced independently of every other element:
 *
 *   mix64(z)            the public splitmix64 finaliser
 *   rnd(seed,stream,i)  = mix64(mix64(seed + stream*0xD1B54A32D192ED03) + i)
 *   u(i)                = (rnd >> 11) * 2^-53                  in [0,1)
 *   normal pair j       = sqrt(-2 ln(1-u(2j))) * {cos,sin}(2 pi u(2j+1))
 *                         -> elements 2j and 2j+1 of the stream (Box-Muller, fp64)
 *
 * bf16 outputs are the fp32 value rounded to nearest-even on its bit pattern.
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

static inline uint64_t stream_key(uint64_t seed, uint64_t stream) {
    return mix64(seed + stream * 0xD1B54A32D192ED03ull);
}

static inline double uniform01(uint64_t key, uint64_t i) {
    return (double)(mix64(key + i) >> 11) * (1.0 / 9007199254740992.0);
}

/* Element i of the standard-normal stream (pair j = i/2 shares one radius). */
static inline double normal_at(uint64_t key, uint64_t i) {
    const uint64_t j = i >> 1;
    const double u0 = uniform01(key, 2 * j);
    const double u1 = uniform01(key, 2 * j + 1);
    const double r = sqrt(-2.0 * log(1.0 - u0));
    const double a = 6.283185307179586476925286766559 * u1;
    return (i & 1) ? r * sin(a) : r * cos(a);
}

static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/* out[k] = rnd(seed, stream, offset + k) */
void synth_u64(uint64_t seed, uint64_t stream, uint64_t offset, int64_t n, uint64_t* out) {
    const uint64_t key = stream_key(seed, stream);
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < n; ++k) out[k] = mix64(key + offset + (uint64_t)k);
}

/* out[k] = u(offset + k) as fp64 */
void synth_uniform_f64(uint64_t seed, uint64_t stream, uint64_t offset, int64_t n, double* out) {
    const uint64_t key = stream_key(seed, stream);
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < n; ++k) out[k] = uniform01(key, offset + (uint64_t)k);
}

/* out[k] = scale * normal(offset + k) as fp64 */
void synth_normal_f64(uint64_t seed, uint64_t stream, uint64_t offset, int64_t n, double scale, double* out) {
    const uint64_t key = stream_key(seed, stream);
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < n; ++k) out[k] = scale * normal_at(key, offset + (uint64_t)k);
}

/* out[k] = bf16_rne(fp32(scale * normal(offset + k))) as raw 16-bit patterns */
void synth_normal_bf16(uint64_t seed, uint64_t stream, uint64_t offset, int64_t n, double scale, uint16_t* out) {
    const uint64_t key = stream_key(seed, stream);
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < n; ++k) out[k] = f32_to_bf16_rne((float)(scale * normal_at(key, offset + (uint64_t)k)));
}
