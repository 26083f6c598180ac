/*
 * Seeded synthetic input generator (test/bench infrastructure).
 *
 * Counter-based: element i of a stream depends only on (key, i), so any
 * sub-range can be produced independently and in parallel.  The generator
 * draws numbers and rounds them to the storage type; it contains none of the
 * MoE layer's arithmetic.
 *
 *   mix      : the splitmix64 output function (Steele, Lea, Flood 2014)
 *   uniform  : 53-bit mantissa from the top bits of a mixed counter
 *   normal   : Box-Muller on a pair of uniforms; elements 2p and 2p+1 take the
 *              cosine and the sine branch of pair p
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

uint64_t dsmoe_gen_key(uint64_t seed, const char *name) {
    /* FNV-1a over the tensor name, folded with the seed through the mixer */
    uint64_t h = 0xCBF29CE484222325ull;
    for (const unsigned char *p = (const unsigned char *)name; *p; ++p) {
        h ^= *p;
        h *= 0x100000001B3ull;
    }
    return mix64(mix64(seed) ^ h);
}

static inline void normal_pair(uint64_t key, uint64_t pair, double *c, double *s) {
    uint64_t r1 = mix64(key + (2 * pair + 1) * 0x9E3779B97F4A7C15ull);
    uint64_t r2 = mix64(key + (2 * pair + 2) * 0x9E3779B97F4A7C15ull);
    double u1 = ((double)(r1 >> 11) + 1.0) * (1.0 / 9007199254740992.0); /* (0,1] */
    double u2 = (double)(r2 >> 11) * (1.0 / 9007199254740992.0);         /* [0,1) */
    double rad = sqrt(-2.0 * log(u1));
    double ang = 6.283185307179586476925286766559 * u2;
    *c = rad * cos(ang);
    *s = rad * sin(ang);
}

static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x40); /* NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* out[i] = scale * N(0,1) for i in [first, first+count), as fp32 */
void dsmoe_gen_normal_f32(uint64_t key, uint64_t first, uint64_t count, double scale, float *out) {
#pragma omp parallel for schedule(static)
    for (int64_t p = (int64_t)(first / 2); p <= (int64_t)((first + count - 1) / 2); ++p) {
        if (count == 0) continue;
        double c, s;
        normal_pair(key, (uint64_t)p, &c, &s);
        uint64_t i0 = 2 * (uint64_t)p, i1 = i0 + 1;
        if (i0 >= first && i0 < first + count) out[i0 - first] = (float)(scale * c);
        if (i1 >= first && i1 < first + count) out[i1 - first] = (float)(scale * s);
    }
}

/* same stream, rounded once (nearest-even) to bfloat16 bit patterns */
void dsmoe_gen_normal_bf16(uint64_t key, uint64_t first, uint64_t count, double scale, uint16_t *out) {
#pragma omp parallel for schedule(static)
    for (int64_t p = (int64_t)(first / 2); p <= (int64_t)((first + count - 1) / 2); ++p) {
        if (count == 0) continue;
        double c, s;
        normal_pair(key, (uint64_t)p, &c, &s);
        uint64_t i0 = 2 * (uint64_t)p, i1 = i0 + 1;
        if (i0 >= first && i0 < first + count) out[i0 - first] = f32_to_bf16_rne((float)(scale * c));
        if (i1 >= first && i1 < first + count) out[i1 - first] = f32_to_bf16_rne((float)(scale * s));
    }
}

/* uniform doubles in [0,1) (used for seeded permutations and token sampling) */
void dsmoe_gen_uniform_f64(uint64_t key, uint64_t first, uint64_t count, double *out) {
    for (uint64_t i = 0; i < count; ++i) {
        uint64_t r = mix64(key + (first + i + 1) * 0x9E3779B97F4A7C15ull);
        out[i] = (double)(r >> 11) * (1.0 / 9007199254740992.0);
    }
}

void dsmoe_bf16_to_f32(const uint16_t *in, uint64_t count, float *out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)count; ++i) {
        uint32_t u = (uint32_t)in[i] << 16;
        memcpy(&out[i], &u, 4);
    }
}

void dsmoe_f32_to_bf16(const float *in, uint64_t count, uint16_t *out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)count; ++i) out[i] = f32_to_bf16_rne(in[i]);
}
