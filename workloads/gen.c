/*
 * Seeded synthetic-input generator: counter-based normal deviates.
 *
 * This file holds no arithmetic of the MoE layer. It only fills arrays with
 * reproducible pseudo-random numbers, so that the CPU oracle and the CUDA path
 * are fed bit-identical inputs.
 *
 * Element i of a stream with seed s comes from one 64-bit hash of the pair
 * index i/2 (splitmix64 finaliser applied to a hashed seed plus the counter);
 * the two halves of the hash are the two uniforms of a Box-Muller transform
 * whose cosine branch gives element 2p and whose sine branch gives 2p+1.
 * Any element can therefore be produced independently of all others, in any
 * order and with any number of threads.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static inline uint64_t sm64(uint64_t z)
{
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

/* exported so that Python can derive permutations / uniforms from the same hash */
uint64_t wl_hash(uint64_t seed, uint64_t counter) { return sm64(sm64(seed) + counter); }

static inline void normal_pair(uint64_t seed_h, uint64_t pair, double *z0, double *z1)
{
    uint64_t r = sm64(seed_h + pair);
    double u1 = ((double)(r >> 32) + 1.0) * (1.0 / 4294967296.0);     /* (0,1] */
    double u2 = (double)(r & 0xFFFFFFFFull) * (1.0 / 4294967296.0);   /* [0,1) */
    double rad = sqrt(-2.0 * log(u1));
    double ang = 6.283185307179586476925286766559 * u2;
    *z0 = rad * cos(ang);
    *z1 = rad * sin(ang);
}

static inline uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;                 /* inputs are finite: no NaN handling needed */
    return (uint16_t)(u >> 16);
}

/* elements [start, start+n) of the bf16 stream (start must be even): lets a caller produce a huge
 * tensor piece by piece, or only the pieces it needs */
void wl_normal_bf16_range(uint16_t *out, int64_t start, int64_t n, uint64_t seed, double mean, double std)
{
    uint64_t sh = sm64(seed);
    int64_t p0 = start / 2, npairs = (n + 1) / 2;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < npairs; ++p) {
        double z0, z1;
        normal_pair(sh, (uint64_t)(p0 + p), &z0, &z1);
        out[2 * p] = f32_to_bf16_rne((float)(mean + std * z0));
        if (2 * p + 1 < n) out[2 * p + 1] = f32_to_bf16_rne((float)(mean + std * z1));
    }
}

/* out[i] = mean + std * z_i, i in [0,n), stored as fp32 */
void wl_normal_f32(float *out, int64_t n, uint64_t seed, double mean, double std)
{
    uint64_t sh = sm64(seed);
    int64_t npairs = (n + 1) / 2;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < npairs; ++p) {
        double z0, z1;
        normal_pair(sh, (uint64_t)p, &z0, &z1);
        out[2 * p] = (float)(mean + std * z0);
        if (2 * p + 1 < n) out[2 * p + 1] = (float)(mean + std * z1);
    }
}

/* same stream, rounded to fp32 and then to bf16 (round to nearest even), stored as raw uint16 */
void wl_normal_bf16(uint16_t *out, int64_t n, uint64_t seed, double mean, double std)
{
    uint64_t sh = sm64(seed);
    int64_t npairs = (n + 1) / 2;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < npairs; ++p) {
        double z0, z1;
        normal_pair(sh, (uint64_t)p, &z0, &z1);
        out[2 * p] = f32_to_bf16_rne((float)(mean + std * z0));
        if (2 * p + 1 < n) out[2 * p + 1] = f32_to_bf16_rne((float)(mean + std * z1));
    }
}

/* out[t*E + e] += bias[e]  (the per-expert load-skew bias of the skewed configs) */
void wl_add_row_bias_f32(float *out, int64_t T, int64_t E, const float *bias)
{
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t)
        for (int64_t e = 0; e < E; ++e) out[t * E + e] += bias[e];
}
