/*
 * Seeded synthetic inputs: permutations and payloads.
 *
 * This file holds input generators only; it contains none of the routing
 * method's arithmetic and is the one piece both the CUDA tests/bench and the
 * oracle tests draw their inputs from.
 *
 * Random numbers: the SplitMix64 sequence (Steele, Lea, Flood 2014; Vigna's
 * public-domain formulation) seeded with the given seed; bounded draws use the
 * multiply-high method with rejection (Lemire 2019), so they are unbiased.
 */
#include <stdint.h>
#include <stddef.h>

typedef struct { uint64_t s; } rng_t;

static uint64_t next64(rng_t *r) {
    uint64_t z = (r->s += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

/* uniform integer in [0, bound), bound >= 1 */
static uint64_t below(rng_t *r, uint64_t bound) {
    unsigned __int128 m = (unsigned __int128)next64(r) * bound;
    uint64_t lo = (uint64_t)m;
    if (lo < bound) {
        uint64_t thresh = (0 - bound) % bound;
        while (lo < thresh) {
            m = (unsigned __int128)next64(r) * bound;
            lo = (uint64_t)m;
        }
    }
    return (uint64_t)(m >> 64);
}

/* Uniform random permutation (Fisher-Yates / Durstenfeld): for i = N-1..1 swap with j in [0, i]. */
void gen_fisher_yates(uint32_t *p, uint64_t N, uint64_t seed) {
    rng_t r = { seed };
    for (uint64_t i = 0; i < N; ++i) p[i] = (uint32_t)i;
    for (uint64_t i = N - 1; i >= 1; --i) {
        uint64_t j = below(&r, i + 1);
        uint32_t t = p[i]; p[i] = p[j]; p[j] = t;
    }
}

/* batch of permutations of N with seeds seed0, seed0+1, ... */
void gen_fisher_yates_batch(uint32_t *p, uint64_t N, uint64_t batch, uint64_t seed0) {
    for (uint64_t b = 0; b < batch; ++b) gen_fisher_yates(p + b * N, N, seed0 + b);
}

/* Uniform random single-cycle permutation (Sattolo): swap with j in [0, i-1]. */
void gen_sattolo(uint32_t *p, uint64_t N, uint64_t seed) {
    rng_t r = { seed };
    for (uint64_t i = 0; i < N; ++i) p[i] = (uint32_t)i;
    for (uint64_t i = N - 1; i >= 1; --i) {
        uint64_t j = below(&r, i);
        uint32_t t = p[i]; p[i] = p[j]; p[j] = t;
    }
}

/* fp32 payload, uniform in [0, 1): top 24 random bits times 2^-24 */
void gen_payload_f32(float *x, uint64_t N, uint64_t seed) {
    rng_t r = { seed };
    for (uint64_t i = 0; i < N; ++i) x[i] = (float)(next64(&r) >> 40) * (1.0f / 16777216.0f);
}

/* 64-bit payload: element index in the low half, seeded random bits in the high half */
void gen_payload_u64(uint64_t *x, uint64_t N, uint64_t seed) {
    rng_t r = { seed };
    for (uint64_t i = 0; i < N; ++i) x[i] = (next64(&r) & 0xFFFFFFFF00000000ull) | (uint32_t)i;
}
