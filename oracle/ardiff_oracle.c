/*
 * ORACLE -- test infrastructure, not product code.
 *
 * Plain, slow, fp64 CPU statement of what the entropy-gated few-step head computes.
 * Only the tests, the smoke check and the benchmark's cpu_baseline / reference leg may
 * call it; the CUDA path shares no code, header, table or helper with this file.
 * Loops run in the order the definitions are written; the only parallelism is an OpenMP
 * "for" over tokens (tokens are independent).
 *
 * Part 1, the gate: per-token Shannon entropy of the softmax-normalised shallow-feature
 * row (the paper's entropy indicator, Eq. for L_entropy in "Entropy-Informed Speculative
 * Decoding" and the supplementary "Entropy Calculation Logic", with H = -L_entropy as in
 * Algorithm 1 "H^s <- -L_entropy"), the threshold test of Algorithm 1
 * ("if H^s < tau_ent": drop), and the ascending list of surviving token ids.
 *
 * Part 2, the head: x_0-side sampling "x = Diff_theta(x_t | t, z)" (Preliminary,
 * AR+Diffusion Hybrid Paradigm) with an MLP head conditioned on the AR feature z and on
 * t, run for K Euler flow steps from shared start noise (Algorithm 1, "Initialize").
 * The paper fixes only "MLP-based", "conditioned on t and z" and "few steps"; the
 * AdaLN residual-MLP structure, the sinusoidal time embedding and the Euler update are
 * this build's stated reading (parity unpinned with respect to the paper for those
 * details: nothing the paper prints can confirm them; the function is pinned instead by
 * closed forms, invariants, a library restatement and brute force in the CPU tests).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline double bf16_to_f64(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* ------------------------------------------------------------------------------------
 * Gate.  Omega = softmax(row);  H = -sum_c Omega_c ln Omega_c  (natural log; terms with
 * Omega_c = 0 contribute 0);  keep = (H >= tau), i.e. drop iff H < tau (Algorithm 1).
 * The softmax is the textbook max-subtracted form: Omega_c = exp(x_c - m) / S.
 * A row that holds a NaN, a +inf, or only -inf gives H = NaN and is dropped.
 * ---------------------------------------------------------------------------------- */
static double row_entropy(const uint16_t* row, int32_t d) {
    double m = -INFINITY;
    int has_nan = 0;
    for (int32_t c = 0; c < d; ++c) {
        double x = bf16_to_f64(row[c]);
        if (x != x) has_nan = 1;
        if (x > m) m = x;
    }
    if (has_nan) return NAN;
    double S = 0.0;
    for (int32_t c = 0; c < d; ++c) S += exp(bf16_to_f64(row[c]) - m);
    double H = 0.0;
    for (int32_t c = 0; c < d; ++c) {
        double p = exp(bf16_to_f64(row[c]) - m) / S;
        if (p > 0.0) H -= p * log(p);
        else if (p != p) return NAN;
    }
    return H;
}

void oracle_entropy(const uint16_t* feat, int64_t n, int32_t d, double* H) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) H[i] = row_entropy(feat + (size_t)i * (size_t)d, d);
}

/* H [n] out (may be NULL), mask [n] out (1 = keep), idx [n] out (first *count valid) */
void oracle_gate(const uint16_t* feat, int64_t n, int32_t d, float tau, double* H, uint8_t* mask,
                 int32_t* idx, int32_t* count) {
    double* Hloc = H ? H : (double*)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    oracle_entropy(feat, n, d, Hloc);
    const double t = (double)tau;
    int32_t k = 0;
    for (int64_t i = 0; i < n; ++i) {
        uint8_t keep = (Hloc[i] >= t) ? 1 : 0; /* false for NaN */
        mask[i] = keep;
        if (keep) idx[k++] = (int32_t)i;
    }
    *count = k;
    if (!H) free(Hloc);
}

/*
 * Block-prefix gate: the early stop of Algorithm 1, Step 1, as it is written. Token i owns the
 * r consecutive rows i*r .. i*r+r-1 of feat; its indicator is the mean of their row entropies
 * (H^s = -L_entropy, the mean over the R rows -- and heads -- of the entropy-loss equation).
 * Tokens come in draft blocks of gamma (the last block may be shorter). Scanning a block in
 * order, the first token with H^s < tau ends speculation: it and every later token of the block
 * are dropped ("draft_tokens[1 : i-1]", "break"). len[b] = tokens kept in block b.
 */
void oracle_gate_blocks(const uint16_t* feat, int64_t n, int32_t r, int32_t d, int32_t gamma, float tau,
                        double* Hs, uint8_t* mask, int32_t* idx, int32_t* count, int32_t* len) {
    double* Hrow = (double*)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1) * (size_t)r);
    oracle_entropy(feat, n * r, d, Hrow);
    for (int64_t i = 0; i < n; ++i) {
        double acc = 0.0;
        for (int32_t j = 0; j < r; ++j) acc += Hrow[(size_t)i * (size_t)r + (size_t)j];
        Hs[i] = acc / (double)r;
    }
    free(Hrow);
    const double t = (double)tau;
    int32_t k = 0;
    for (int64_t b0 = 0, b = 0; b0 < n; b0 += gamma, ++b) {
        const int64_t b1 = (b0 + gamma < n) ? b0 + gamma : n;
        int speculate = 1;
        int32_t kept = 0;
        for (int64_t i = b0; i < b1; ++i) {
            if (speculate && !(Hs[i] >= t)) speculate = 0; /* H < tau, or NaN */
            mask[i] = (uint8_t)speculate;
            if (speculate) { idx[k++] = (int32_t)i; ++kept; }
        }
        len[b] = kept;
    }
    *count = k;
}

/* Threshold from entropy statistics ("Entropy-Based Early Stopping", the tau equation):
 * tau = 0.3 * mean(H) - 0.1 * std(H), std taken over the whole set (divisor n). */
void oracle_tau_calibrate(const double* H, int64_t n, double* mean, double* std, double* tau) {
    double m = 0.0;
    for (int64_t i = 0; i < n; ++i) m += H[i];
    m /= (double)n;
    double v = 0.0;
    for (int64_t i = 0; i < n; ++i) v += (H[i] - m) * (H[i] - m);
    v /= (double)n;
    *mean = m;
    *std = sqrt(v);
    *tau = 0.3 * m - 0.1 * sqrt(v);
}

/* Accepted draft length per block (Algorithm 1, Step 4):
 * n_b = min({i-1 : r_i > ratio_i} U {len_b}), i counted from 1 inside the block. len_b is
 * len(draft_tokens) as Step 1 left it: block_len[b] drafts when the early stop truncated the block
 * (block_len == NULL: nothing was truncated, the whole block reaches Step 4). */
void oracle_accept_prefix(const float* r, const float* ratio, int64_t n, int32_t gamma, const int32_t* block_len,
                          int32_t* nacc) {
    for (int64_t b0 = 0, b = 0; b0 < n; b0 += gamma, ++b) {
        int64_t b1 = (b0 + gamma < n) ? b0 + gamma : n;
        if (block_len) {
            const int64_t lb = block_len[b] > 0 ? block_len[b] : 0;
            if (b0 + lb < b1) b1 = b0 + lb;
        }
        int32_t acc = (int32_t)(b1 - b0);
        for (int64_t i = b0; i < b1; ++i) {
            if (r[i] > ratio[i]) { acc = (int32_t)(i - b0); break; }
        }
        nacc[b] = acc;
    }
}

/* ------------------------------------------------------------------------------------
 * Head.  All parameters are bf16 bit patterns widened exactly to double; noise and the
 * time schedule are float32 widened to double; nothing is rounded in between.
 * Linear layers use the [out][in] layout: y_o = b_o + sum_i W[o][i] x_i.
 * ---------------------------------------------------------------------------------- */
typedef struct {
    int32_t C, Dc, W, L, F;
    const uint16_t *Wc, *bc;     /* [W][Dc], [W]      c = Wc z + bc                      */
    const uint16_t *Wt1, *bt1;   /* [W][F],  [W]      time MLP layer 1                   */
    const uint16_t *Wt2, *bt2;   /* [W][W],  [W]      time MLP layer 2                   */
    const uint16_t *Win, *bin;   /* [W][C],  [W]      h = Win x + bin                    */
    const uint16_t *Wmod, *bmod; /* [L][3W][W], [L][3W]  rows: shift | scale | gate      */
    const uint16_t *W1, *b1;     /* [L][W][W], [L][W]                                    */
    const uint16_t *W2, *b2;     /* [L][W][W], [L][W]                                    */
    const uint16_t *Wfm, *bfm;   /* [2W][W], [2W]     rows: shift | scale                */
    const uint16_t *Wout, *bout; /* [C][W],  [C]                                         */
} oracle_head_params;

static inline double silu(double a) { return a / (1.0 + exp(-a)); }

static void linear(const uint16_t* Wm, const uint16_t* b, int32_t n_out, int32_t n_in,
                   const double* x, double* y) {
    for (int32_t o = 0; o < n_out; ++o) {
        double acc = bf16_to_f64(b[o]);
        const uint16_t* w = Wm + (size_t)o * (size_t)n_in;
        for (int32_t i = 0; i < n_in; ++i) acc += bf16_to_f64(w[i]) * x[i];
        y[o] = acc;
    }
}

/* LN(h) = (h - mean) / sqrt(var + 1e-6), biased variance over the W channels, no affine */
static void layer_norm(const double* h, int32_t W, double* out) {
    double mean = 0.0;
    for (int32_t i = 0; i < W; ++i) mean += h[i];
    mean /= (double)W;
    double var = 0.0;
    for (int32_t i = 0; i < W; ++i) var += (h[i] - mean) * (h[i] - mean);
    var /= (double)W;
    const double r = 1.0 / sqrt(var + 1e-6);
    for (int32_t i = 0; i < W; ++i) out[i] = (h[i] - mean) * r;
}

/* temb = Wt2 SiLU(Wt1 e + bt1) + bt2,  e = [cos(1000 t w_f) | sin(1000 t w_f)], f < F/2,
 * w_f = 10000^(-f / (F/2)) */
static void time_embedding(const oracle_head_params* P, double t, double* temb, double* tmpW,
                           double* e) {
    const int32_t half = P->F / 2;
    for (int32_t f = 0; f < half; ++f) {
        double w = pow(10000.0, -(double)f / (double)half);
        e[f] = cos(1000.0 * t * w);
        e[half + f] = sin(1000.0 * t * w);
    }
    linear(P->Wt1, P->bt1, P->W, P->F, e, tmpW);
    for (int32_t i = 0; i < P->W; ++i) tmpW[i] = silu(tmpW[i]);
    linear(P->Wt2, P->bt2, P->W, P->W, tmpW, temb);
}

/* One survivor token: K steps of the head, each followed by the sampler update
 *   x <- ax_k x + av_k v + an_k z_k        (coef = {ax_0, av_0, an_0, ax_1, ...}, z_k = step noise or none).
 * The Euler flow update is the case ax = 1, av = t_{k+1} - t_k, an = 0. */
static void head_token(const oracle_head_params* P, const uint16_t* z_bits, const double* temb_all,
                       const double* coef, const float* step_noise_tok, size_t step_stride, int32_t K, double* x,
                       double* buf) {
    const int32_t C = P->C, Dc = P->Dc, W = P->W, L = P->L;
    double* z = buf;              /* Dc */
    double* c = z + Dc;           /* W  */
    double* s = c + W;            /* W  */
    double* h = s + W;            /* W  */
    double* mod = h + W;          /* 3W */
    double* u = mod + 3 * W;      /* W  */
    double* a = u + W;            /* W  */
    double* r = a + W;            /* W  */
    double* v = r + W;            /* C  */
    for (int32_t i = 0; i < Dc; ++i) z[i] = bf16_to_f64(z_bits[i]);
    linear(P->Wc, P->bc, W, Dc, z, c);
    for (int32_t k = 0; k < K; ++k) {
        const double* temb = temb_all + (size_t)k * (size_t)W;
        for (int32_t i = 0; i < W; ++i) s[i] = silu(c[i] + temb[i]);
        linear(P->Win, P->bin, W, C, x, h);
        for (int32_t b = 0; b < L; ++b) {
            linear(P->Wmod + (size_t)b * 3 * W * W, P->bmod + (size_t)b * 3 * W, 3 * W, W, s, mod);
            const double *sh = mod, *sc = mod + W, *g = mod + 2 * W;
            layer_norm(h, W, u);
            for (int32_t i = 0; i < W; ++i) u[i] = u[i] * (1.0 + sc[i]) + sh[i];
            linear(P->W1 + (size_t)b * W * W, P->b1 + (size_t)b * W, W, W, u, a);
            for (int32_t i = 0; i < W; ++i) a[i] = silu(a[i]);
            linear(P->W2 + (size_t)b * W * W, P->b2 + (size_t)b * W, W, W, a, r);
            for (int32_t i = 0; i < W; ++i) h[i] += g[i] * r[i];
        }
        linear(P->Wfm, P->bfm, 2 * W, W, s, mod);
        layer_norm(h, W, u);
        for (int32_t i = 0; i < W; ++i) u[i] = u[i] * (1.0 + mod[W + i]) + mod[i];
        linear(P->Wout, P->bout, C, W, u, v);
        const double ax = coef[3 * k], av = coef[3 * k + 1], an = coef[3 * k + 2];
        for (int32_t i = 0; i < C; ++i) {
            double xn = ax * x[i] + av * v[i];
            if (step_noise_tok) xn += an * (double)step_noise_tok[(size_t)k * step_stride + (size_t)i];
            x[i] = xn;
        }
    }
}

/*
 * cond  [n][Dc] bf16 bits, noise [n][C] float32, t_sched [K+1] float32,
 * idx [count] token ids (any order), out [n][C] double: only rows idx[j] are written.
 * K = 0 copies the noise rows.
 */
static void head_sample_coef(const oracle_head_params* P, const uint16_t* cond, const float* noise,
                             const float* t_sched, int32_t K, const double* coef, const float* step_noise,
                             int64_t n, const int32_t* idx, int32_t count, double* out) {
    const int32_t C = P->C, Dc = P->Dc, W = P->W;
    double* temb_all = (double*)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1) * (size_t)W);
    {
        double* tmpW = (double*)malloc(sizeof(double) * (size_t)W);
        double* e = (double*)malloc(sizeof(double) * (size_t)P->F);
        for (int32_t k = 0; k < K; ++k)
            time_embedding(P, (double)t_sched[k], temb_all + (size_t)k * (size_t)W, tmpW, e);
        free(tmpW);
        free(e);
    }
    const size_t per_tok = (size_t)Dc + (size_t)W * 10 + (size_t)C;
#pragma omp parallel
    {
        double* buf = (double*)malloc(sizeof(double) * per_tok);
#pragma omp for schedule(dynamic, 1)
        for (int32_t j = 0; j < count; ++j) {
            const size_t tok = (size_t)idx[j];
            double* x = out + tok * (size_t)C;
            for (int32_t i = 0; i < C; ++i) x[i] = (double)noise[tok * (size_t)C + i];
            head_token(P, cond + tok * (size_t)Dc, temb_all, coef,
                       step_noise ? step_noise + tok * (size_t)C : NULL, (size_t)n * (size_t)C, K, x, buf);
        }
        free(buf);
    }
    free(temb_all);
}

/* K Euler flow steps: x <- x + (t_{k+1} - t_k) v. */
void oracle_head_sample(const oracle_head_params* P, const uint16_t* cond, const float* noise,
                        const float* t_sched, int32_t K, const int32_t* idx, int32_t count,
                        double* out) {
    double* coef = (double*)malloc(sizeof(double) * 3 * (size_t)(K > 0 ? K : 1));
    for (int32_t k = 0; k < K; ++k) {
        coef[3 * k] = 1.0;
        coef[3 * k + 1] = (double)t_sched[k + 1] - (double)t_sched[k];
        coef[3 * k + 2] = 0.0;
    }
    head_sample_coef(P, cond, noise, t_sched, K, coef, NULL, 0, idx, count, out);
    free(coef);
}

/*
 * Other samplers on the same head (the paper's heads are also run as eps-prediction DDPM heads,
 * "x_t = sqrt(abar_t) x + sqrt(1 - abar_t) eps", and as x_0-prediction consistency students,
 * "x_0 = Diff_theta(x_t | t, z)"): every such step is linear in (x, head output, fresh noise), so
 * the caller passes the three coefficients per step. t_sched [K] are the times fed to the head;
 * coef [3K] float32 (widened); step_noise [K][n][C] float32 or NULL.
 */
void oracle_head_sample_coef(const oracle_head_params* P, const uint16_t* cond, const float* noise,
                             const float* t_sched, int32_t K, const float* coef, const float* step_noise,
                             int64_t n, const int32_t* idx, int32_t count, double* out) {
    double* c = (double*)malloc(sizeof(double) * 3 * (size_t)(K > 0 ? K : 1));
    for (int32_t i = 0; i < 3 * K; ++i) c[i] = (double)coef[i];
    head_sample_coef(P, cond, noise, t_sched, K, c, step_noise, n, idx, count, out);
    free(c);
}

/* exposed for the tests that pin the pieces separately */
void oracle_layer_norm(const double* h, int32_t W, double* out) { layer_norm(h, W, out); }

void oracle_time_embedding(const oracle_head_params* P, float t, double* temb) {
    double* tmpW = (double*)malloc(sizeof(double) * (size_t)P->W);
    double* e = (double*)malloc(sizeof(double) * (size_t)P->F);
    time_embedding(P, (double)t, temb, tmpW, e);
    free(tmpW);
    free(e);
}
