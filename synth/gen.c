/*
 * Seeded synthetic-input generator (counter-based, so any element or row can be
 * produced on its own, in any order, on any number of threads, with the same value).
 *
 * This file holds NO arithmetic of the method under test (no softmax, entropy,
 * LayerNorm, head or sampler code): it only draws random numbers and rounds them.
 * Both the CPU oracle's callers and the CUDA path's callers feed on its arrays.
 *
 * Random source: a 64-bit counter hash built from the SplitMix64 finaliser
 * (Steele, Lea, Flood 2014; Vigna's public-domain constants). Value j of stream s
 * under seed k is mix(mix(k ^ s*GOLDEN) + j*GOLDEN).  Gaussians: Box-Muller in fp64.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#define GOLDEN 0x9E3779B97F4A7C15ULL

static inline uint64_t mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

static inline uint64_t stream_key(uint64_t seed, uint64_t stream) {
    return mix64(seed ^ (stream * GOLDEN) ^ 0xA5A5A5A55A5A5A5AULL);
}

static inline uint64_t draw_u64(uint64_t key, uint64_t j) { return mix64(key + (j + 1) * GOLDEN); }

/* uniform in the open interval (0,1), 53 bits */
static inline double draw_u01(uint64_t key, uint64_t j) {
    return ((double)(draw_u64(key, j) >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}

/* Box-Muller pair number p of a stream: two independent N(0,1) */
static inline void draw_pair(uint64_t key, uint64_t p, double* z0, double* z1) {
    double u1 = draw_u01(key, 2 * p), u2 = draw_u01(key, 2 * p + 1);
    double r = sqrt(-2.0 * log(u1));
    double a = 6.283185307179586476925 * u2;
    *z0 = r * cos(a);
    *z1 = r * sin(a);
}

static inline double draw_normal(uint64_t key, uint64_t e) {
    double z0, z1;
    draw_pair(key, e >> 1, &z0, &z1);
    return (e & 1) ? z1 : z0;
}

/* float -> bf16 bits, round to nearest even (NaN kept quiet) */
static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/* out[i] = (float)(scale * N(0,1)) for elements start .. start+count-1 of the stream */
void synth_normal_f32(uint64_t seed, uint64_t stream, uint64_t start, uint64_t count, double scale,
                      float* out) {
    const uint64_t key = stream_key(seed, stream);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)count; ++i)
        out[i] = (float)(scale * draw_normal(key, start + (uint64_t)i));
}

/* same, rounded to bf16 (bits) */
void synth_normal_bf16(uint64_t seed, uint64_t stream, uint64_t start, uint64_t count, double scale,
                       uint16_t* out) {
    const uint64_t key = stream_key(seed, stream);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)count; ++i)
        out[i] = f32_to_bf16_rne((float)(scale * draw_normal(key, start + (uint64_t)i)));
}

/*
 * Feature rows [row0, row0+nrows) of an n x d matrix, bf16 bits, row-major.
 * Each row is one of two kinds, chosen per row from the row's own hash:
 *   kind A with probability p_a, else kind B, where a kind is
 *     0 flat    : d iid N(0,1)
 *     1 peaked  : d iid N(0,1), then one uniformly chosen channel j set to 20*|x_j|
 *     2 heavy   : d iid Student-t(3): g / sqrt(chi2_3 / 3), chi2_3 = g1^2 - 2 ln u
 * mode 0: "alternate" (even rows kind_a, odd rows kind_b; p_a ignored)
 * mode 1: Bernoulli(p_a) per row.
 * kinds_out (may be NULL) receives the kind of each generated row.
 */
void synth_feat_rows(uint64_t seed, uint64_t stream, int32_t mode, double p_a, int32_t kind_a,
                     int32_t kind_b, int64_t row0, int64_t nrows, int32_t d, uint16_t* out,
                     uint8_t* kinds_out) {
    const uint64_t key_g = stream_key(seed, stream);          /* gaussians, pair-indexed */
    const uint64_t key_u = stream_key(seed, stream + 1);      /* extra uniforms (heavy rows) */
    const uint64_t key_r = stream_key(seed, stream + 2);      /* per-row decisions */
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t r = 0; r < nrows; ++r) {
        const uint64_t row = (uint64_t)(row0 + r);
        int kind;
        if (mode == 0) kind = (row & 1) ? kind_b : kind_a;
        else kind = (draw_u01(key_r, 2 * row) < p_a) ? kind_a : kind_b;
        if (kinds_out) kinds_out[r] = (uint8_t)kind;
        uint16_t* o = out + (size_t)r * (size_t)d;
        const uint64_t e0 = row * (uint64_t)d;               /* element index of channel 0 */
        if (kind == 2) {
            for (int32_t c = 0; c < d; ++c) {
                double g, g1;
                draw_pair(key_g, e0 + (uint64_t)c, &g, &g1);  /* one pair per element */
                double chi = g1 * g1 - 2.0 * log(draw_u01(key_u, e0 + (uint64_t)c));
                o[c] = f32_to_bf16_rne((float)(g / sqrt(chi / 3.0)));
            }
        } else {
            int32_t jpk = -1;
            if (kind == 1) {
                jpk = (int32_t)(draw_u01(key_r, 2 * row + 1) * (double)d);
                if (jpk >= d) jpk = d - 1;
            }
            for (int32_t c = 0; c < d; ++c) {
                double x = draw_normal(key_g, e0 + (uint64_t)c);
                if (c == jpk) x = 20.0 * fabs(x);
                o[c] = f32_to_bf16_rne((float)x);
            }
        }
    }
}

/* bf16 bits <-> float helpers for the Python side (exact widening; RNE narrowing) */
void synth_bf16_to_f32(const uint16_t* in, uint64_t count, float* out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)count; ++i) {
        uint32_t u = (uint32_t)in[i] << 16;
        memcpy(&out[i], &u, 4);
    }
}

void synth_f32_to_bf16(const float* in, uint64_t count, uint16_t* out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)count; ++i) out[i] = f32_to_bf16_rne(in[i]);
}
