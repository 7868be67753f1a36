/*
 * Seeded synthetic-input generators (host, plain C + OpenMP).
 *
 * These routines only manufacture inputs: bf16 weight tensors, token ids,
 * uniforms, Gaussian noise.  They hold none of the verification arithmetic
 * (no transformer maths, no softmax, no acceptance rule).  Both the CUDA
 * library's callers and the CPU checker are fed from here so that they see
 * bit-identical arrays.
 *
 * Generator: a counter-based construction.  Element i of stream s under
 * seed z is a pure function of (z, s, i): the 64-bit word
 *     r = splitmix64_finalise( (z * C1) ^ (s * C2) ^ (i * C3 + C4) )
 * applied twice (two rounds of the SplitMix64 output permutation, Steele,
 * Lea & Flood 2014), so any element can be produced independently and the
 * result does not depend on the thread count.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

static inline uint64_t sm64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ULL;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

static inline uint64_t ctr_word(uint64_t seed, uint64_t stream, uint64_t idx) {
    uint64_t a = sm64(seed * 0xD6E8FEB86659FD93ULL + 0x2545F4914F6CDD1DULL);
    uint64_t b = sm64(a ^ (stream * 0xA0761D6478BD642FULL));
    return sm64(sm64(b ^ (idx * 0xE7037ED1A0B428DBULL)));
}

/* fp32 -> bf16, round to nearest, ties to even (finite inputs only). */
static inline uint16_t f32_to_bf16_rne(float f) {
    union { float f; uint32_t u; } v;
    v.f = f;
    uint32_t lsb = (v.u >> 16) & 1u;
    v.u += 0x7FFFu + lsb;
    return (uint16_t)(v.u >> 16);
}

/* Two independent standard normals from one 64-bit word (Box-Muller, in
 * double; the radius uniform is kept away from 0). */
static inline void normal_pair(uint64_t r, double *z0, double *z1) {
    uint32_t hi = (uint32_t)(r >> 32), lo = (uint32_t)r;
    double u1 = ((double)hi + 0.5) * (1.0 / 4294967296.0);
    double u2 = ((double)lo + 0.5) * (1.0 / 4294967296.0);
    double rad = sqrt(-2.0 * log(u1));
    double ang = 6.283185307179586476925286766559 * u2;
    *z0 = rad * cos(ang);
    *z1 = rad * sin(ang);
}

/* out[i] = bf16( std * N(0,1) ), i in [0, n). */
void synth_normal_bf16(uint16_t *out, int64_t n, uint64_t seed, uint64_t stream, double std) {
    int64_t pairs = (n + 1) / 2;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < pairs; ++p) {
        double z0, z1;
        normal_pair(ctr_word(seed, stream, (uint64_t)p), &z0, &z1);
        out[2 * p] = f32_to_bf16_rne((float)(std * z0));
        if (2 * p + 1 < n) out[2 * p + 1] = f32_to_bf16_rne((float)(std * z1));
    }
}

/* out[i] = (float)( std * N(0,1) ). */
void synth_normal_f32(float *out, int64_t n, uint64_t seed, uint64_t stream, double std) {
    int64_t pairs = (n + 1) / 2;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < pairs; ++p) {
        double z0, z1;
        normal_pair(ctr_word(seed, stream, (uint64_t)p), &z0, &z1);
        out[2 * p] = (float)(std * z0);
        if (2 * p + 1 < n) out[2 * p + 1] = (float)(std * z1);
    }
}

/* out[i] = (r >> 40) * 2^-24: uniform on [0,1), exactly representable in fp32. */
void synth_uniform_f32(float *out, int64_t n, uint64_t seed, uint64_t stream) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        uint64_t r = ctr_word(seed, stream, (uint64_t)i);
        out[i] = (float)(r >> 40) * (1.0f / 16777216.0f);
    }
}

/* Uniform token ids on [0, vocab). */
void synth_tokens_i32(int32_t *out, int64_t n, uint64_t seed, uint64_t stream, int32_t vocab) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        uint64_t r = ctr_word(seed, stream, (uint64_t)i);
        out[i] = (int32_t)(((r >> 32) * (uint64_t)vocab) >> 32);
    }
}

/* Uniform integers on [lo, hi] (inclusive). */
void synth_ints_i32(int32_t *out, int64_t n, uint64_t seed, uint64_t stream, int32_t lo, int32_t hi) {
    uint64_t span = (uint64_t)(hi - lo) + 1u;
    for (int64_t i = 0; i < n; ++i) {
        uint64_t r = ctr_word(seed, stream, (uint64_t)i);
        out[i] = lo + (int32_t)(((r >> 32) * span) >> 32);
    }
}

/* bf16 <-> fp32 array helpers (pure format conversion). */
void synth_bf16_to_f32(const uint16_t *in, float *out, int64_t n) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        union { float f; uint32_t u; } v;
        v.u = (uint32_t)in[i] << 16;
        out[i] = v.f;
    }
}

void synth_f32_to_bf16(const float *in, uint16_t *out, int64_t n) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) out[i] = f32_to_bf16_rne(in[i]);
}
