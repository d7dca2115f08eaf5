/*
 * Seeded synthetic-input generator shared by the CPU oracle's tests and the
 * CUDA path's tests / bench.  It produces INPUTS only (weight tensors as bf16
 * bit patterns, prompt token ids); it contains no arithmetic of the decoding
 * method itself.
 *
 * Every element is a pure function of (seed, tensor_id, element index), so a
 * tensor can be generated in any order, on any number of threads, and is
 * identical on every machine:
 *
 *   u64  = mix(mix(seed, tensor_id) + index * GOLDEN)
 *   z    = QUANTILE[u64 >> 48]            (65536 mid-point quantiles of N(0,1))
 *   w    = bf16_rne( (float)z * std * scale )
 *
 * The quantile table makes the draw a 16-bit discretisation of the normal
 * distribution (tails end at +-4.3 sigma); its spacing is finer than bf16's
 * 8-bit mantissa almost everywhere, so after rounding the weights are
 * indistinguishable from rounded N(0, std^2) draws.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

#define SYNTH_GOLDEN 0x9E3779B97F4A7C15ull

static inline uint64_t mix64(uint64_t z) {
    z += SYNTH_GOLDEN;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static inline uint64_t stream_key(uint64_t seed, uint64_t tensor_id) {
    return mix64(mix64(seed) ^ (tensor_id * 0xD1B54A32D192ED03ull));
}

/* Inverse of the standard normal CDF: rational initial guess refined by
 * Newton steps on erfc (double precision, then rounded to float). */
static double inv_norm_cdf(double p) {
    /* initial guess: logistic-type approximation, good enough for Newton */
    double x;
    if (p < 0.5) {
        double t = sqrt(-2.0 * log(p));
        x = -(t - (2.515517 + 0.802853 * t + 0.010328 * t * t) /
                      (1.0 + 1.432788 * t + 0.189269 * t * t + 0.001308 * t * t * t));
    } else {
        double t = sqrt(-2.0 * log(1.0 - p));
        x = t - (2.515517 + 0.802853 * t + 0.010328 * t * t) /
                    (1.0 + 1.432788 * t + 0.189269 * t * t + 0.001308 * t * t * t);
    }
    for (int it = 0; it < 4; ++it) {
        double cdf = 0.5 * erfc(-x * 0.70710678118654752440);
        double pdf = 0.39894228040143267794 * exp(-0.5 * x * x);
        x -= (cdf - p) / pdf;
    }
    return x;
}

static float g_quantile[65536];
static int g_quantile_ready = 0;

void synth_init(void) {
    if (g_quantile_ready) return;
    for (int i = 0; i < 65536; ++i)
        g_quantile[i] = (float)inv_norm_cdf(((double)i + 0.5) / 65536.0);
    g_quantile_ready = 1;
}

static inline uint16_t f32_to_bf16_rne(float f) {
    union { float f; uint32_t u; } v;
    v.f = f;
    uint32_t u = v.u;
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/* out[i] = bf16( N(0,1)-quantile draw * std * scale ), i in [0, n) */
void synth_normal_bf16(uint64_t seed, uint64_t tensor_id, int64_t n, float std, float scale,
                       uint16_t *out) {
    synth_init();
    const uint64_t key = stream_key(seed, tensor_id);
    const float s = std * scale;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        uint64_t h = mix64(key + (uint64_t)i * SYNTH_GOLDEN);
        out[i] = f32_to_bf16_rne(g_quantile[h >> 48] * s);
    }
}

/* out[i] = bf16( 1 + spread * draw ): norm gains; spread = 0 gives exactly 1.0 */
void synth_gain_bf16(uint64_t seed, uint64_t tensor_id, int64_t n, float spread, uint16_t *out) {
    synth_init();
    const uint64_t key = stream_key(seed, tensor_id);
    for (int64_t i = 0; i < n; ++i) {
        uint64_t h = mix64(key + (uint64_t)i * SYNTH_GOLDEN);
        out[i] = f32_to_bf16_rne(1.0f + spread * g_quantile[h >> 48]);
    }
}

/* out[i] uniform in [0, vocab) */
void synth_tokens(uint64_t seed, uint64_t stream_id, int64_t n, int32_t vocab, int32_t *out) {
    const uint64_t key = stream_key(seed, stream_id);
    for (int64_t i = 0; i < n; ++i) {
        uint64_t h = mix64(key + (uint64_t)i * SYNTH_GOLDEN);
        out[i] = (int32_t)(((h >> 32) * (uint64_t)vocab) >> 32);
    }
}

/* one uniform integer in [0, bound) for (seed, stream_id, index) */
int32_t synth_uniform_int(uint64_t seed, uint64_t stream_id, int64_t index, int32_t bound) {
    const uint64_t key = stream_key(seed, stream_id);
    uint64_t h = mix64(key + (uint64_t)index * SYNTH_GOLDEN);
    return (int32_t)(((h >> 32) * (uint64_t)bound) >> 32);
}
