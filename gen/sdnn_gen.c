/*
 * Seeded synthetic workloads for the sparse-DNN hot path: sparsity patterns,
 * weight values, biases, binary inputs and targets.
 *
 * This file holds NO arithmetic of the method (no products, activations,
 * gradients).  It only produces the arrays that both the CPU oracle and the
 * CUDA library receive as inputs, so the two sides see bit-identical data.
 *
 * Every number is a pure function of a 64-bit key (counter-based): the key is
 * built from (master seed, stream id, a, b) and slot t of the key is the t-th
 * output of the splitmix64 sequence started at that key.  Nothing depends on
 * thread count or call order.
 *
 * Workload shapes follow the paper's experimental grid (Section 6: N in
 * {1024, 4096, 16384, 65536} neurons per layer, L in {120, 480, 1920} layers,
 * 60000 binary input vectors); the patterns themselves are synthetic
 * stand-ins for the RadiX-Net topologies used there.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define GOLDEN 0x9E3779B97F4A7C15ULL

static inline uint64_t mix64(uint64_t z) {
    z += GOLDEN;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

static inline uint64_t make_key(uint64_t seed, uint64_t stream, uint64_t a, uint64_t b) {
    uint64_t h = mix64(seed ^ mix64(stream));
    h = mix64(h ^ a);
    h = mix64(h ^ b);
    return h;
}

static inline uint64_t draw(uint64_t key, uint64_t t) { return mix64(key + t * GOLDEN); }

/* exported so tests can pin the generator itself */
uint64_t sdnn_gen_draw(uint64_t seed, uint64_t stream, uint64_t a, uint64_t b, uint64_t t) {
    return draw(make_key(seed, stream, a, b), t);
}

/* k distinct values (ascending) out of the table cand[0..m) (or 0..m-1 when cand == NULL),
 * drawn by rejection from the stream of `key`. */
static void draw_row(uint64_t key, int32_t m, int32_t k, const int32_t *cand, int32_t *out) {
    int32_t have = 0;
    uint64_t t = 0;
    while (have < k) {
        int32_t pick = (int32_t)(draw(key, t++) % (uint64_t)m);
        int32_t c = cand ? cand[pick] : pick;
        int32_t pos = have, dup = 0;
        for (int32_t q = 0; q < have; ++q) {
            if (out[q] == c) { dup = 1; break; }
        }
        if (dup) continue;
        while (pos > 0 && out[pos - 1] > c) { out[pos] = out[pos - 1]; --pos; }
        out[pos] = c;
        ++have;
    }
}

/* Uniform pattern: every row holds k distinct columns drawn uniformly from [0, n). */
void sdnn_gen_pattern_uniform(uint64_t seed, uint64_t stream, int64_t layer, int32_t n, int32_t k,
                              int32_t *col /* [n*k] */) {
#pragma omp parallel for schedule(static)
    for (int32_t i = 0; i < n; ++i)
        draw_row(make_key(seed, stream, (uint64_t)layer, (uint64_t)i), n, k, NULL, col + (int64_t)i * k);
}

/* Seeded permutation of [0, n) (Fisher-Yates driven by one key per layer). */
void sdnn_gen_permutation(uint64_t seed, uint64_t stream, int64_t layer, int32_t n, int32_t *perm) {
    uint64_t key = make_key(seed, stream, (uint64_t)layer, 0x70657261ULL);
    for (int32_t i = 0; i < n; ++i) perm[i] = i;
    for (int32_t i = n - 1; i > 0; --i) {
        int32_t j = (int32_t)(draw(key, (uint64_t)i) % (uint64_t)(i + 1));
        int32_t tmp = perm[i]; perm[i] = perm[j]; perm[j] = tmp;
    }
}

/* Banded-permuted pattern: rows [w*r, w*(r+1)) draw their k distinct columns from the
 * window { perm[w*r + t] : 0 <= t < w } of a per-layer permutation. */
void sdnn_gen_pattern_windowed(uint64_t seed, uint64_t stream, int64_t layer, int32_t n, int32_t k,
                               int32_t window, const int32_t *perm, int32_t *col) {
#pragma omp parallel for schedule(static)
    for (int32_t i = 0; i < n; ++i) {
        int32_t base = (i / window) * window;
        int32_t m = (base + window <= n) ? window : (n - base);
        draw_row(make_key(seed, stream, (uint64_t)layer, (uint64_t)i), m, k, perm + base, col + (int64_t)i * k);
    }
}

/* iid N(0, sigma^2), Box-Muller in double, rounded once to fp32. */
void sdnn_gen_normal(uint64_t seed, uint64_t stream, int64_t a, int64_t count, double sigma, float *out) {
    const uint64_t key = make_key(seed, stream, (uint64_t)a, 0x6e6f726dULL);
    const double two_pi = 6.283185307179586476925286766559;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < count; ++p) {
        uint64_t r1 = draw(key, (uint64_t)(2 * p)), r2 = draw(key, (uint64_t)(2 * p + 1));
        double u1 = ((double)(r1 >> 11) + 1.0) * 0x1.0p-53; /* (0, 1] */
        double u2 = (double)(r2 >> 11) * 0x1.0p-53;         /* [0, 1) */
        out[p] = (float)(sigma * sqrt(-2.0 * log(u1)) * cos(two_pi * u2));
    }
}

/* iid Bernoulli(prob) as 0.0f / 1.0f. */
void sdnn_gen_bernoulli(uint64_t seed, uint64_t stream, int64_t a, int64_t count, double prob, float *out) {
    const uint64_t key = make_key(seed, stream, (uint64_t)a, 0x6265726eULL);
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < count; ++p) {
        double u = (double)(draw(key, (uint64_t)p) >> 11) * 0x1.0p-53;
        out[p] = (u < prob) ? 1.0f : 0.0f;
    }
}

/* iid uniform on [0, 1) with 24 random bits (exact in fp32). */
void sdnn_gen_uniform(uint64_t seed, uint64_t stream, int64_t a, int64_t count, float *out) {
    const uint64_t key = make_key(seed, stream, (uint64_t)a, 0x756e6966ULL);
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < count; ++p)
        out[p] = (float)(draw(key, (uint64_t)p) >> 40) * 0x1.0p-24f;
}
