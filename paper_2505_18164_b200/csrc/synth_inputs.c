/* Seeded synthetic tensors and prompts.
 *
 * This file holds no model arithmetic: it only fills buffers with reproducible
 * pseudo-random values.  Every element is a pure function of (seed, tensor
 * ordinal, element index), so any slice of any tensor can be regenerated alone
 * and the result does not depend on the thread count.
 *
 * Generator: a 64-bit finaliser-style mixer (the splitmix64 output function)
 * applied to a counter, two uniforms per pair of elements, Box-Muller in fp64.
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

static inline uint64_t tensor_key(uint64_t seed, uint64_t ordinal) {
    return mix64(mix64(seed) ^ (ordinal * 0xD1B54A32D192ED03ull + 0x8CB92BA72F3D8DD7ull));
}

/* standard normal pair for pair index j of a keyed tensor */
static inline void normal_pair(uint64_t key, uint64_t j, double *z0, double *z1) {
    uint64_t h1 = mix64(key ^ mix64(2 * j));
    uint64_t h2 = mix64(key ^ mix64(2 * j + 1));
    double u1 = (double)((h1 >> 11) + 1) * (1.0 / 9007199254740992.0); /* (0,1] */
    double u2 = (double)(h2 >> 11) * (1.0 / 9007199254740992.0);       /* [0,1) */
    double r = sqrt(-2.0 * log(u1));
    double a = 6.283185307179586476925286766559 * u2;
    *z0 = r * cos(a);
    *z1 = r * sin(a);
}

static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40); /* NaN */
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/* Fill out[0..n) with elements [first, first+n) of tensor `ordinal`:
 * value = fp32(std * z), z ~ N(0,1).  dtype 0: float32 out, 1: bfloat16
 * (uint16, round-to-nearest-even of the fp32 value). */
void synth_normal(uint64_t seed, uint64_t ordinal, double std, int dtype,
                  uint64_t first, uint64_t n, void *out) {
    const uint64_t key = tensor_key(seed, ordinal);
    float *of = (float *)out;
    uint16_t *oh = (uint16_t *)out;
    const uint64_t j0 = first / 2, j1 = (first + n + 1) / 2;
#pragma omp parallel for schedule(static)
    for (uint64_t j = j0; j < j1; ++j) {
        double z[2];
        normal_pair(key, j, &z[0], &z[1]);
        for (int h = 0; h < 2; ++h) {
            uint64_t e = 2 * j + (uint64_t)h;
            if (e < first || e >= first + n) continue;
            float v = (float)(std * z[h]);
            if (dtype == 0) of[e - first] = v;
            else oh[e - first] = f32_to_bf16_rne(v);
        }
    }
}

/* Fill out[0..n) with a constant (1.0 for norm gains, 0.0 for norm offsets). */
void synth_const(double value, int dtype, uint64_t n, void *out) {
    float v = (float)value;
    if (dtype == 0) { float *o = (float *)out; for (uint64_t i = 0; i < n; ++i) o[i] = v; }
    else { uint16_t *o = (uint16_t *)out; uint16_t b = f32_to_bf16_rne(v); for (uint64_t i = 0; i < n; ++i) o[i] = b; }
}

/* Token ids uniform over [0, vocab): stream `stream` of seed `seed`. */
void synth_tokens(uint64_t seed, uint64_t stream, int32_t vocab, uint64_t n, int32_t *out) {
    const uint64_t key = tensor_key(seed, 0x746f6b656e73ull + stream);
    for (uint64_t i = 0; i < n; ++i) {
        uint64_t h = mix64(key ^ mix64(i));
        double u = (double)(h >> 11) * (1.0 / 9007199254740992.0);
        int32_t t = (int32_t)(u * (double)vocab);
        out[i] = t >= vocab ? vocab - 1 : t;
    }
}
