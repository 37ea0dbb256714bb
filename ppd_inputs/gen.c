/*
 * Seeded synthetic inputs for the PPD decode path: a random-init LLaMA-shaped weight
 * blob (bf16) and uniform-random prompt token ids.
 *
 * This module only draws numbers.  It holds none of the decoder's arithmetic and is the
 * one piece of code that both the CPU oracle and the CUDA library consume (each receives
 * the finished blob as an input).
 *
 * Recipe (the synthetic stand-in for the paper's LLaMA-family checkpoints, which are not
 * available): every matrix, the embedding table E and the unembedding W_H are drawn
 * i.i.d. N(0, sigma^2) with sigma = 0.02; the two matrices that write into the residual
 * stream (W_o and W_d) are additionally multiplied by resid_scale (0.1 by default) so
 * that early-layer predictions often agree with the final argmax; norm gains are 1.
 * Values are rounded to bf16 (round-to-nearest-even) and stored as uint16.
 *
 * Blob order, all row-major [out][in]:
 *   E[V][D]
 *   for each layer: g1[D] Wq[D][D] Wk[D][D] Wv[D][D] Wo[D][D] g2[D] Wg[F][D] Wu[F][D] Wd[D][F]
 *   g_final[D]  W_H[V][D]
 *
 * The generator is counter based: element i of tensor t depends only on (seed, t, i), so
 * the result does not depend on the thread count.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

typedef struct {
    int32_t n_layers, d_model, d_ffn, vocab;
} ppd_inputs_shape;

static inline uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u); /* finite inputs only */
    return (uint16_t)(u >> 16);
}

/* Two independent standard normals from one 64-bit draw (Box-Muller, double precision). */
static inline void normal_pair(uint64_t r, double* z0, double* z1) {
    const double two_pi = 6.283185307179586476925286766559;
    double u1 = ((double)(uint32_t)(r >> 32) + 1.0) * (1.0 / 4294967296.0); /* (0,1] */
    double u2 = (double)(uint32_t)r * (1.0 / 4294967296.0);                /* [0,1) */
    double rad = sqrt(-2.0 * log(u1));
    *z0 = rad * cos(two_pi * u2);
    *z1 = rad * sin(two_pi * u2);
}

static void fill_normal(uint16_t* dst, size_t n, uint64_t seed, uint64_t tensor_id, double scale) {
    const uint64_t key = mix64(mix64(seed) ^ (tensor_id * 0xD1B54A32D192ED03ull));
    const size_t n_pairs = (n + 1) / 2;
#pragma omp parallel for schedule(static)
    for (size_t j = 0; j < n_pairs; ++j) {
        double z0, z1;
        normal_pair(mix64(key + j), &z0, &z1);
        dst[2 * j] = f32_to_bf16_rne((float)(scale * z0));
        if (2 * j + 1 < n) dst[2 * j + 1] = f32_to_bf16_rne((float)(scale * z1));
    }
}

static void fill_ones(uint16_t* dst, size_t n) {
    for (size_t i = 0; i < n; ++i) dst[i] = 0x3F80u; /* bf16(1.0) */
}

size_t ppd_inputs_blob_elems(const ppd_inputs_shape* s) {
    const size_t D = (size_t)s->d_model, F = (size_t)s->d_ffn, V = (size_t)s->vocab;
    const size_t per_layer = D + 4 * D * D + D + 3 * F * D;
    return V * D + (size_t)s->n_layers * per_layer + D + V * D;
}

/* Fills dst[0 .. blob_elems) with the bf16 blob.  Returns 0, or -1 on a bad shape. */
int ppd_inputs_gen_weights(const ppd_inputs_shape* s, uint64_t seed, double sigma,
                           double resid_scale, uint16_t* dst) {
    if (!s || !dst || s->n_layers < 1 || s->d_model < 1 || s->d_ffn < 1 || s->vocab < 1) return -1;
    const size_t D = (size_t)s->d_model, F = (size_t)s->d_ffn, V = (size_t)s->vocab;
    uint16_t* p = dst;
    uint64_t t = 0;
    fill_normal(p, V * D, seed, t++, sigma); p += V * D;
    for (int l = 0; l < s->n_layers; ++l) {
        fill_ones(p, D); p += D;
        fill_normal(p, D * D, seed, t++, sigma); p += D * D;               /* Wq */
        fill_normal(p, D * D, seed, t++, sigma); p += D * D;               /* Wk */
        fill_normal(p, D * D, seed, t++, sigma); p += D * D;               /* Wv */
        fill_normal(p, D * D, seed, t++, sigma * resid_scale); p += D * D; /* Wo */
        fill_ones(p, D); p += D;
        fill_normal(p, F * D, seed, t++, sigma); p += F * D;               /* Wg */
        fill_normal(p, F * D, seed, t++, sigma); p += F * D;               /* Wu */
        fill_normal(p, D * F, seed, t++, sigma * resid_scale); p += D * F; /* Wd */
    }
    fill_ones(p, D); p += D;
    fill_normal(p, V * D, seed, t++, sigma); p += V * D;
    return 0;
}

/* Uniform token ids in [0, vocab). */
int ppd_inputs_gen_prompt(int32_t vocab, uint64_t seed, int32_t n, int32_t* dst) {
    if (vocab < 1 || n < 0 || (n > 0 && !dst)) return -1;
    const uint64_t key = mix64(mix64(seed) ^ 0x70726F6D7074ull);
    for (int32_t i = 0; i < n; ++i) {
        uint64_t r = mix64(key + (uint64_t)i);
        dst[i] = (int32_t)(((r >> 32) * (uint64_t)vocab) >> 32);
    }
    return 0;
}
