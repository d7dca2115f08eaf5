/*
 * CPU oracle (see del_oracle.h for its role, precision and pins).
 *
 * Paper passages followed:
 *   Sec. 2 "Auto-regressive decoding": h^l = Transformer_l(h^{l-1}), token = argmax LM-Head(h^L)
 *   Sec. 2 "Speculative decoding", greedy special case: accept while draft top-1 == target top-1,
 *          1..gamma+1 tokens per round
 *   Sec. 2 "Early-exit self-speculative decoding": draft = first E layers + LM head, verify with
 *          all layers, KV cache shared
 *   Sec. 4.1 Eq. 1 (tokens-per-layer, in its sum form), cost d*l + L
 *   Sec. 4.2 shadow tokens, u_r, c_r^l, decayed sum S, Eq. 2 (alpha_l)
 *   Sec. 4.3 selection by argmax of TPL, initialisation from the prefill
 *   Sec. 4.4 dynamic draft-exiting: confidence = probability of the top-1 token, tcs / fcs, Eq. 3
 *   Algorithm 1 (the loop with its confidence break, DEL_Update)
 *   App. B.2 hyper-parameters: window 32, omega 0.95
 * The decoder block itself is the standard pre-norm Llama block (RMSNorm, rotary embedding with
 * rotate-half pairing, grouped-query causal attention, SwiGLU), which the paper takes as given.
 */
#include "del_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

struct ora_seq {
    ora_shape sh;
    ora_weights w;
    int32_t T;          /* committed positions in the KV cache */
    int32_t x_in;       /* token to be fed at position T */
    int32_t E, gamma;   /* choice for the next round */
    int32_t fixed_E, fixed_gamma;
    int32_t fs_mode;    /* 1: fixed exit layer, speculation length steered by the +-1 controller (baseline FS) */
    double *Sc;         /* [L], index l-1; Sc[L-1] (layer L) tracked too: it must equal Sn */
    double Sn;
    double *Stcs, *Sfcs; /* [L] decayed confidence sums over matched / mismatched shadow tokens (Sec. 4.4) */
    double *tau;        /* [L] thresholds of Eq. 3 from the current statistics */
    double *conf;       /* [L][rows] confidence of every shadow token of the last round / prefill window */
    int32_t exit_mode;  /* 1: the draft loop runs up to g_max steps and stops on a low confidence */
    double temperature, top_p; /* speculative sampling (temperature <= 0: greedy) */
    uint64_t seed;
    float *qlog, *plog; /* [g_max + 1][V] logits of the exit head per draft / of the target per row, last round */
    ora_sample_info sinfo;
    float *K, *V;       /* [L][max_seq][n_kv*hd] */
    float *H;           /* [L+1][rows][d] hidden stack */
    int32_t rows;       /* rows per layer in H */
    float *rope_cos, *rope_sin; /* [max_seq][hd/2] */
};

static inline float bf16_to_float(uint16_t b) {
    union { uint32_t u; float f; } v;
    v.u = (uint32_t)b << 16;
    return v.f;
}

int ora_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* dot product accumulated in double: 32 partial sums over k mod 32, then a fixed-order final sum, so
 * the order depends only on K.  The operands are floats widened to double; float*float is exact in
 * double, hence the fused multiply-add used here rounds exactly like multiply-then-add. */
static double dot_dd(const double *a, const double *b, int32_t K) {
    double acc[32];
    for (int j = 0; j < 32; ++j) acc[j] = 0.0;
    int32_t k0 = 0;
    for (; k0 + 32 <= K; k0 += 32)
        for (int j = 0; j < 32; ++j) acc[j] = __builtin_fma(a[k0 + j], b[k0 + j], acc[j]);
    double s = 0.0;
    for (int j = 0; j < 32; ++j) s += acc[j];
    for (; k0 < K; ++k0) s += a[k0] * b[k0];
    return s;
}

static double dot_ff(const float *a, const float *b, int32_t K) {
    double acc[32];
    for (int j = 0; j < 32; ++j) acc[j] = 0.0;
    int32_t k0 = 0;
    for (; k0 + 32 <= K; k0 += 32)
        for (int j = 0; j < 32; ++j) acc[j] = __builtin_fma((double)a[k0 + j], (double)b[k0 + j], acc[j]);
    double s = 0.0;
    for (int j = 0; j < 32; ++j) s += acc[j];
    for (; k0 < K; ++k0) s += (double)a[k0] * (double)b[k0];
    return s;
}

/* Y[r][o] = W[o] . X[r]   (W bf16 [N][K], X float [m][K], Y float [m][N]).  Each (r, o) is one dot
 * product in the order of dot_dd; rows and weights are widened to double once, which changes no bit. */
static void matmul_rows(const uint16_t *W, int32_t N, int32_t K, const float *X, int32_t m, float *Y) {
    double *Xd = (double *)malloc((size_t)m * K * sizeof(double));
    for (size_t i = 0; i < (size_t)m * K; ++i) Xd[i] = (double)X[i];
#pragma omp parallel
    {
        double *wd = (double *)malloc((size_t)K * sizeof(double));
#pragma omp for schedule(static)
        for (int32_t o = 0; o < N; ++o) {
            const uint16_t *wr = W + (size_t)o * K;
            for (int32_t k = 0; k < K; ++k) wd[k] = (double)bf16_to_float(wr[k]);
            for (int32_t r = 0; r < m; ++r) Y[(size_t)r * N + o] = (float)dot_dd(wd, Xd + (size_t)r * K, K);
        }
        free(wd);
    }
    free(Xd);
}

/* RMSNorm: out = x / sqrt(mean(x^2) + eps) * gain */
void ora_rmsnorm(const float *x, const uint16_t *gain, int32_t d, float eps, float *out) {
    double ss = dot_ff(x, x, d);
    double inv = 1.0 / sqrt(ss / (double)d + (double)eps);
    for (int32_t k = 0; k < d; ++k) out[k] = (float)((double)x[k] * inv * (double)bf16_to_float(gain[k]));
}

/* Rotary embedding, rotate-half pairing (j, j + hd/2), angle = pos * theta^(-2j/hd) */
static void rope_tables(float *c, float *s, int32_t max_seq, int32_t hd, float theta) {
    int32_t half = hd / 2;
    for (int32_t p = 0; p < max_seq; ++p)
        for (int32_t j = 0; j < half; ++j) {
            double inv_freq = pow((double)theta, -2.0 * (double)j / (double)hd);
            double ang = (double)p * inv_freq;
            c[(size_t)p * half + j] = (float)cos(ang);
            s[(size_t)p * half + j] = (float)sin(ang);
        }
}

static void rope_apply(float *x, int32_t n_heads, int32_t hd, const float *c, const float *s) {
    int32_t half = hd / 2;
    for (int32_t h = 0; h < n_heads; ++h) {
        float *v = x + (size_t)h * hd;
        for (int32_t j = 0; j < half; ++j) {
            double a = v[j], b = v[j + half];
            double cj = c[j], sj = s[j];
            v[j] = (float)(a * cj - b * sj);
            v[j + half] = (float)(b * cj + a * sj);
        }
    }
}

void ora_rope(float *x, int32_t n_heads, int32_t head_dim, int32_t pos, float theta) {
    int32_t half = head_dim / 2;
    float *c = (float *)malloc(sizeof(float) * half), *s = (float *)malloc(sizeof(float) * half);
    for (int32_t j = 0; j < half; ++j) {
        double ang = (double)pos * pow((double)theta, -2.0 * (double)j / (double)head_dim);
        c[j] = (float)cos(ang);
        s[j] = (float)sin(ang);
    }
    rope_apply(x, n_heads, head_dim, c, s);
    free(c);
    free(s);
}

void ora_softmax(const float *x, int32_t n, double *p) {
    double mx = x[0];
    for (int32_t i = 1; i < n; ++i)
        if (x[i] > mx) mx = x[i];
    double sum = 0.0;
    for (int32_t i = 0; i < n; ++i) {
        p[i] = exp((double)x[i] - mx);
        sum += p[i];
    }
    for (int32_t i = 0; i < n; ++i) p[i] /= sum;
}

float ora_silu(float x) { return (float)((double)x / (1.0 + exp(-(double)x))); }

ora_seq *ora_seq_create(const ora_shape *shape, const ora_weights *w) {
    ora_seq *s = (ora_seq *)calloc(1, sizeof(ora_seq));
    s->sh = *shape;
    s->w = *w;
    const ora_shape *sh = &s->sh;
    size_t kvd = (size_t)sh->n_kv_heads * sh->head_dim;
    s->K = (float *)calloc((size_t)sh->n_layers * sh->max_seq * kvd, sizeof(float));
    s->V = (float *)calloc((size_t)sh->n_layers * sh->max_seq * kvd, sizeof(float));
    s->rows = sh->g_max + 1 > sh->init_window ? sh->g_max + 1 : sh->init_window;
    s->H = (float *)calloc((size_t)(sh->n_layers + 1) * s->rows * sh->d_model, sizeof(float));
    s->Sc = (double *)calloc(sh->n_layers, sizeof(double));
    s->Stcs = (double *)calloc(sh->n_layers, sizeof(double));
    s->Sfcs = (double *)calloc(sh->n_layers, sizeof(double));
    s->tau = (double *)calloc(sh->n_layers, sizeof(double));
    s->conf = (double *)calloc((size_t)sh->n_layers * s->rows, sizeof(double));
    s->rope_cos = (float *)malloc(sizeof(float) * (size_t)sh->max_seq * (sh->head_dim / 2));
    s->rope_sin = (float *)malloc(sizeof(float) * (size_t)sh->max_seq * (sh->head_dim / 2));
    rope_tables(s->rope_cos, s->rope_sin, sh->max_seq, sh->head_dim, sh->rope_theta);
    s->fixed_E = 0;
    s->fixed_gamma = 0;
    s->E = sh->e_min;
    s->gamma = sh->g_min;
    return s;
}

void ora_seq_destroy(ora_seq *s) {
    if (!s) return;
    free(s->K); free(s->V); free(s->H); free(s->Sc); free(s->rope_cos); free(s->rope_sin);
    free(s->Stcs); free(s->Sfcs); free(s->tau); free(s->conf); free(s->qlog); free(s->plog);
    free(s);
}

void ora_set_policy(ora_seq *s, int32_t fixed_E, int32_t fixed_gamma) {
    s->fixed_E = fixed_E;
    s->fixed_gamma = fixed_gamma;
    s->fs_mode = 0;
    if (fixed_E > 0) { s->E = fixed_E; s->gamma = fixed_gamma; }
}

void ora_set_policy_fs(ora_seq *s, int32_t fixed_E, int32_t gamma0) {
    ora_set_policy(s, fixed_E, gamma0);
    s->fs_mode = 1;
}

/* The FS baseline of Sec. 5.1: one more draft next time if every draft of this round was accepted, one
 * fewer if any was rejected.  The paper gives no bounds; here the length stays within [max(1, g_min),
 * g_max] (at 0 nothing could ever be accepted again) and a round without drafts changes nothing. */
int32_t ora_fs_next_gamma(int32_t gamma, int32_t g, int32_t n, int32_t g_min, int32_t g_max) {
    const int32_t lo = g_min > 1 ? g_min : 1;
    if (g < 1) return gamma;
    if (n == g) return gamma + 1 > g_max ? g_max : gamma + 1;
    return gamma - 1 < lo ? lo : gamma - 1;
}

int32_t ora_committed_len(const ora_seq *s) { return s->T; }

void ora_get_stats(const ora_seq *s, double *Sc, double *Sn, int32_t *E, int32_t *gamma) {
    if (Sc) memcpy(Sc, s->Sc, sizeof(double) * s->sh.n_layers);
    if (Sn) *Sn = s->Sn;
    if (E) *E = s->E;
    if (gamma) *gamma = s->gamma;
}

/* Eq. 3: midpoint of the decayed mean confidence of matched and of mismatched shadow tokens.  The paper
 * does not say what a mean over no tokens is; here the mean over no matched tokens is 1 and the mean
 * over no mismatched tokens is 0 (the two ends of the range of a probability). */
double ora_threshold(double Stcs, double Sc, double Sfcs, double Smis) {
    double mean_true = 1.0, mean_false = 0.0;
    if (Sc > 0.0) mean_true = Stcs / Sc;
    if (Smis > 0.0) mean_false = Sfcs / Smis;
    double sum = mean_true + mean_false;
    return 0.5 * sum;
}

/* S(u - c) = S(u) - S(c): S is linear */
static void refresh_tau(ora_seq *s) {
    for (int32_t l = 0; l < s->sh.n_layers; ++l)
        s->tau[l] = ora_threshold(s->Stcs[l], s->Sc[l], s->Sfcs[l], s->Sn - s->Sc[l]);
}

void ora_set_stats(ora_seq *s, const double *Sc, double Sn, int32_t E, int32_t gamma) {
    memcpy(s->Sc, Sc, sizeof(double) * s->sh.n_layers);
    s->Sn = Sn; s->E = E; s->gamma = gamma;
    refresh_tau(s);
}

void ora_set_exit_mode(ora_seq *s, int32_t mode) { s->exit_mode = mode ? 1 : 0; }

void ora_get_conf_stats(const ora_seq *s, double *Stcs, double *Sfcs, double *tau) {
    if (Stcs) memcpy(Stcs, s->Stcs, sizeof(double) * s->sh.n_layers);
    if (Sfcs) memcpy(Sfcs, s->Sfcs, sizeof(double) * s->sh.n_layers);
    if (tau) memcpy(tau, s->tau, sizeof(double) * s->sh.n_layers);
}

void ora_set_conf_stats(ora_seq *s, const double *Stcs, const double *Sfcs) {
    memcpy(s->Stcs, Stcs, sizeof(double) * s->sh.n_layers);
    memcpy(s->Sfcs, Sfcs, sizeof(double) * s->sh.n_layers);
    refresh_tau(s);
}

void ora_get_conf(const ora_seq *s, double *conf, int32_t n_cols) {
    for (int32_t l = 0; l < s->sh.n_layers; ++l)
        for (int32_t i = 0; i < n_cols; ++i) conf[(size_t)l * n_cols + i] = s->conf[(size_t)l * s->rows + i];
}

static float *hidden_at(const ora_seq *s, int32_t layer, int32_t row) {
    return s->H + ((size_t)layer * s->rows + row) * s->sh.d_model;
}
const float *ora_hidden(const ora_seq *s, int32_t layer, int32_t row) { return hidden_at(s, layer, row); }

static float *k_at(const ora_seq *s, int32_t layer1, int32_t pos) {
    size_t kvd = (size_t)s->sh.n_kv_heads * s->sh.head_dim;
    return s->K + ((size_t)(layer1 - 1) * s->sh.max_seq + pos) * kvd;
}
static float *v_at(const ora_seq *s, int32_t layer1, int32_t pos) {
    size_t kvd = (size_t)s->sh.n_kv_heads * s->sh.head_dim;
    return s->V + ((size_t)(layer1 - 1) * s->sh.max_seq + pos) * kvd;
}
const float *ora_k_row(const ora_seq *s, int32_t layer, int32_t pos) { return k_at(s, layer, pos); }
const float *ora_v_row(const ora_seq *s, int32_t layer, int32_t pos) { return v_at(s, layer, pos); }

/* h^0 = embedding row of the token (Sec. 2) */
void ora_embed(const ora_seq *s, int32_t token, float *h) {
    const uint16_t *e = s->w.tok_emb + (size_t)token * s->sh.d_model;
    for (int32_t k = 0; k < s->sh.d_model; ++k) h[k] = bf16_to_float(e[k]);
}

/* causal attention of one query row at position pos over cached keys 0..pos, all heads */
static void attend_row(const ora_seq *s, int32_t layer1, const float *q, int32_t pos, float *out) {
    const ora_shape *sh = &s->sh;
    const int32_t hd = sh->head_dim, group = sh->n_heads / sh->n_kv_heads;
    const double scale = 1.0 / sqrt((double)hd);
#pragma omp parallel
    {
        float *sc = (float *)malloc(sizeof(float) * (size_t)(pos + 1));
        double *p = (double *)malloc(sizeof(double) * (size_t)(pos + 1));
        double *acc = (double *)malloc(sizeof(double) * (size_t)hd);
#pragma omp for schedule(static)
        for (int32_t h = 0; h < sh->n_heads; ++h) {
            const int32_t kvh = h / group;
            const float *qh = q + (size_t)h * hd;
            for (int32_t j = 0; j <= pos; ++j)
                sc[j] = (float)(dot_ff(qh, k_at(s, layer1, j) + (size_t)kvh * hd, hd) * scale);
            ora_softmax(sc, pos + 1, p);
            for (int32_t e = 0; e < hd; ++e) acc[e] = 0.0;
            for (int32_t j = 0; j <= pos; ++j) {
                const float *vj = v_at(s, layer1, j) + (size_t)kvh * hd;
                for (int32_t e = 0; e < hd; ++e) acc[e] += p[j] * (double)vj[e];
            }
            for (int32_t e = 0; e < hd; ++e) out[(size_t)h * hd + e] = (float)acc[e];
        }
        free(sc); free(p); free(acc);
    }
}

/* One pre-norm Llama block over m rows at positions pos0..pos0+m-1 (row i sees keys <= pos0+i). */
void ora_layer_rows(ora_seq *s, int32_t layer1, const float *h_in, int32_t pos0, int32_t m, float *h_out) {
    const ora_shape *sh = &s->sh;
    const int32_t d = sh->d_model, hd = sh->head_dim, F = sh->d_ffn;
    const int32_t nq = sh->n_heads * hd, nk = sh->n_kv_heads * hd, half = hd / 2;
    const int32_t li = layer1 - 1;
    const int32_t CH = 32;
    float *a = (float *)malloc(sizeof(float) * (size_t)CH * d);
    float *q = (float *)malloc(sizeof(float) * (size_t)CH * nq);
    float *k = (float *)malloc(sizeof(float) * (size_t)CH * nk);
    float *v = (float *)malloc(sizeof(float) * (size_t)CH * nk);
    float *o = (float *)malloc(sizeof(float) * (size_t)CH * nq);
    float *y = (float *)malloc(sizeof(float) * (size_t)CH * d);
    float *h1 = (float *)malloc(sizeof(float) * (size_t)CH * d);
    float *gt = (float *)malloc(sizeof(float) * (size_t)CH * F);
    float *up = (float *)malloc(sizeof(float) * (size_t)CH * F);
    for (int32_t r0 = 0; r0 < m; r0 += CH) {
        const int32_t mc = (m - r0 < CH) ? m - r0 : CH;
        const float *hin = h_in + (size_t)r0 * d;
        float *hout = h_out + (size_t)r0 * d;
        for (int32_t r = 0; r < mc; ++r) ora_rmsnorm(hin + (size_t)r * d, s->w.attn_norm[li], d, sh->rms_eps, a + (size_t)r * d);
        matmul_rows(s->w.wq[li], nq, d, a, mc, q);
        matmul_rows(s->w.wk[li], nk, d, a, mc, k);
        matmul_rows(s->w.wv[li], nk, d, a, mc, v);
        for (int32_t r = 0; r < mc; ++r) {
            const int32_t pos = pos0 + r0 + r;
            const float *c = s->rope_cos + (size_t)pos * half, *sn = s->rope_sin + (size_t)pos * half;
            rope_apply(q + (size_t)r * nq, sh->n_heads, hd, c, sn);
            rope_apply(k + (size_t)r * nk, sh->n_kv_heads, hd, c, sn);
            memcpy(k_at(s, layer1, pos), k + (size_t)r * nk, sizeof(float) * nk);
            memcpy(v_at(s, layer1, pos), v + (size_t)r * nk, sizeof(float) * nk);
        }
        for (int32_t r = 0; r < mc; ++r) attend_row(s, layer1, q + (size_t)r * nq, pos0 + r0 + r, o + (size_t)r * nq);
        matmul_rows(s->w.wo[li], d, nq, o, mc, y);
        for (size_t i = 0; i < (size_t)mc * d; ++i) h1[i] = hin[i] + y[i];
        for (int32_t r = 0; r < mc; ++r) ora_rmsnorm(h1 + (size_t)r * d, s->w.ffn_norm[li], d, sh->rms_eps, a + (size_t)r * d);
        matmul_rows(s->w.w_gate[li], F, d, a, mc, gt);
        matmul_rows(s->w.w_up[li], F, d, a, mc, up);
        for (size_t i = 0; i < (size_t)mc * F; ++i) gt[i] = ora_silu(gt[i]) * up[i];
        matmul_rows(s->w.w_down[li], d, F, gt, mc, y);
        for (size_t i = 0; i < (size_t)mc * d; ++i) hout[i] = h1[i] + y[i];
    }
    free(a); free(q); free(k); free(v); free(o); free(y); free(h1); free(gt); free(up);
}

/* Exit head at any layer: shared final RMSNorm, LM head, greedy choice (Sec. 2; Sec. 4.2 applies the
 * same head to every layer's hidden state).  Lowest token id wins ties. */
/* Confidence score of Sec. 4.4: the softmax probability of the top-1 token, 1 / sum_v exp(z_v - z_max). */
double ora_confidence(const float *logits, int32_t V) {
    double mx = logits[0];
    for (int32_t t = 1; t < V; ++t)
        if (logits[t] > mx) mx = logits[t];
    double sum = 0.0;
    for (int32_t t = 0; t < V; ++t) sum += exp((double)logits[t] - mx);
    return 1.0 / sum;
}

static void exit_head_conf(const ora_seq *s, const float *h, int32_t *token, float *margin, double *conf) {
    float *lg = (float *)malloc(sizeof(float) * s->sh.vocab);
    ora_exit_head(s, h, token, margin, lg);
    *conf = ora_confidence(lg, s->sh.vocab);
    free(lg);
}

void ora_exit_head(const ora_seq *s, const float *h, int32_t *token, float *margin, float *logits_or_null) {
    const ora_shape *sh = &s->sh;
    const int32_t d = sh->d_model, V = sh->vocab;
    float *a = (float *)malloc(sizeof(float) * d);
    float *lg = logits_or_null ? logits_or_null : (float *)malloc(sizeof(float) * V);
    ora_rmsnorm(h, s->w.final_norm, d, sh->rms_eps, a);
    matmul_rows(s->w.lm_head, V, d, a, 1, lg);
    int32_t best = 0;
    for (int32_t t = 1; t < V; ++t)
        if (lg[t] > lg[best]) best = t;
    float second = -INFINITY;
    for (int32_t t = 0; t < V; ++t)
        if (t != best && lg[t] > second) second = lg[t];
    if (token) *token = best;
    if (margin) *margin = lg[best] - second;
    if (!logits_or_null) free(lg);
    free(a);
}

/* Greedy verification: length of the longest prefix of drafts equal to the target's tokens (Sec. 2). */
int32_t ora_accept_len(const int32_t *drafts, const int32_t *verified, int32_t g) {
    int32_t n = 0;
    while (n < g && drafts[n] == verified[n]) ++n;
    return n;
}

/* ---------------------------------------------------------------- speculative sampling (Sec. 2) */

/* finaliser of the splitmix64 generator (a bijective 64-bit mixer) */
static uint64_t mix64(uint64_t x) {
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27; x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}

double ora_uniform(uint64_t seed, int64_t pos, int32_t purpose) {
    const uint64_t ctr = (uint64_t)pos * 4u + (uint64_t)purpose + 1u;
    const uint64_t x = mix64(seed ^ mix64(ctr * 0x9E3779B97F4A7C15ull));
    return (double)(x >> 11) * (1.0 / 9007199254740992.0);      /* 53 bits */
}

typedef struct { double p; int32_t id; } prob_id;
static int by_prob_desc(const void *a, const void *b) {
    const prob_id *x = (const prob_id *)a, *y = (const prob_id *)b;
    if (x->p > y->p) return -1;
    if (x->p < y->p) return 1;
    return x->id < y->id ? -1 : (x->id > y->id ? 1 : 0);
}

void ora_nucleus(const float *logits, int32_t V, double temperature, double top_p, double *probs) {
    double mx = logits[0];
    for (int32_t t = 1; t < V; ++t)
        if (logits[t] > mx) mx = logits[t];
    double Z = 0.0;
    for (int32_t t = 0; t < V; ++t) { probs[t] = exp(((double)logits[t] - mx) / temperature); Z += probs[t]; }
    for (int32_t t = 0; t < V; ++t) probs[t] /= Z;
    if (top_p >= 1.0) return;
    prob_id *o = (prob_id *)malloc(sizeof(prob_id) * (size_t)V);
    for (int32_t t = 0; t < V; ++t) { o[t].p = probs[t]; o[t].id = t; }
    qsort(o, (size_t)V, sizeof(prob_id), by_prob_desc);
    double before = 0.0;                /* mass of the tokens ahead in the descending order */
    int32_t k = 0;
    while (k < V && before < top_p) { before += o[k].p; ++k; }
    for (int32_t j = k; j < V; ++j) probs[o[j].id] = 0.0;
    free(o);
    double K = 0.0;
    for (int32_t t = 0; t < V; ++t) K += probs[t];
    for (int32_t t = 0; t < V; ++t) probs[t] /= K;
}

int32_t ora_sample_cdf(const double *probs, int32_t V, double u) {
    double c = 0.0;
    int32_t last = 0;
    for (int32_t t = 0; t < V; ++t) {
        if (probs[t] <= 0.0) continue;
        c += probs[t];
        last = t;
        if (u < c) return t;
    }
    return last;                        /* u beyond the rounded total: the last token with mass */
}

double ora_residual(const double *p, const double *q, int32_t V, double *r) {
    double R = 0.0;
    for (int32_t t = 0; t < V; ++t) { r[t] = p[t] > q[t] ? p[t] - q[t] : 0.0; R += r[t]; }
    if (R <= 0.0) { memcpy(r, p, sizeof(double) * (size_t)V); return 0.0; }
    for (int32_t t = 0; t < V; ++t) r[t] /= R;
    return R;
}

void ora_set_sampling(ora_seq *s, double temperature, double top_p, uint64_t seed) {
    s->temperature = temperature;
    s->top_p = top_p;
    s->seed = seed;
    if (temperature > 0.0 && !s->qlog) {
        const size_t n = (size_t)(s->sh.g_max + 1) * s->sh.vocab;
        s->qlog = (float *)calloc(n, sizeof(float));
        s->plog = (float *)calloc(n, sizeof(float));
    }
}

void ora_get_sample_info(const ora_seq *s, ora_sample_info *out) { *out = s->sinfo; }

const float *ora_round_logits(const ora_seq *s, int32_t which, int32_t row) {
    return (which ? s->plog : s->qlog) + (size_t)row * s->sh.vocab;
}

/* One step of S(a) = sum_i omega^(r-i-1) a[i], written as the recursion S <- omega*S + a (Sec. 4.2). */
double ora_decay_step(double S, double omega, double a) {
    double t = omega * S;
    return t + a;
}

/* Eq. 1 in its sum form: (sum_{k=0..d} alpha^k) / (d*l + L) */
double ora_tpl(double alpha, int32_t l, int32_t d, int32_t L) {
    double term = 1.0, sum = 1.0;
    for (int32_t k = 1; k <= d; ++k) {
        term = term * alpha;
        sum = sum + term;
    }
    return sum / (double)(d * l + L);
}

/* Sec. 4.3: (E, gamma) = argmax TPL over the given ranges; first maximum in l-major order. */
void ora_select(const double *Sc, double Sn, int32_t L, int32_t e_min, int32_t e_max, int32_t g_min,
                int32_t g_max, int32_t *E, int32_t *gamma) {
    double best = -1.0;
    int32_t bE = e_min, bg = g_min;
    for (int32_t l = e_min; l <= e_max; ++l) {
        double alpha = Sc[l - 1] / Sn;
        for (int32_t d = g_min; d <= g_max; ++d) {
            double t = ora_tpl(alpha, l, d, L);
            if (t > best) { best = t; bE = l; bg = d; }
        }
    }
    *E = bE;
    *gamma = bg;
}

static void choose_next(ora_seq *s, int32_t g, int32_t n) {
    const ora_shape *sh = &s->sh;
    if (s->fixed_E > 0 && s->fs_mode) {
        s->E = s->fixed_E;
        s->gamma = ora_fs_next_gamma(s->gamma, g, n, sh->g_min, sh->g_max);
        return;
    }
    if (s->fixed_E > 0) { s->E = s->fixed_E; s->gamma = s->fixed_gamma; return; }
    ora_select(s->Sc, s->Sn, sh->n_layers, sh->e_min, sh->e_max, sh->g_min, sh->g_max, &s->E, &s->gamma);
}

int32_t ora_prefill(ora_seq *s, const int32_t *prompt, int32_t P, int32_t *shadow, float *margin,
                    ora_round_info *info) {
    const ora_shape *sh = &s->sh;
    const int32_t d = sh->d_model, L = sh->n_layers;
    const int32_t W = P < sh->init_window ? P : sh->init_window;
    float *ha = (float *)malloc(sizeof(float) * (size_t)P * d);
    float *hb = (float *)malloc(sizeof(float) * (size_t)P * d);
    for (int32_t t = 0; t < P; ++t) ora_embed(s, prompt[t], ha + (size_t)t * d);
    for (int32_t j = 0; j < W; ++j) memcpy(hidden_at(s, 0, j), ha + (size_t)(P - W + j) * d, sizeof(float) * d);
    for (int32_t l = 1; l <= L; ++l) {
        ora_layer_rows(s, l, ha, 0, P, hb);
        for (int32_t j = 0; j < W; ++j) memcpy(hidden_at(s, l, j), hb + (size_t)(P - W + j) * d, sizeof(float) * d);
        float *t = ha; ha = hb; hb = t;
    }
    free(ha); free(hb);
    /* shadow tokens of every layer over the window; agreement with layer L seeds the statistics */
    int32_t *sd = (int32_t *)malloc(sizeof(int32_t) * (size_t)L * W);
    for (int32_t l = 1; l <= L; ++l)
        for (int32_t j = 0; j < W; ++j) {
            float mg;
            exit_head_conf(s, hidden_at(s, l, j), &sd[(size_t)(l - 1) * W + j], &mg, &s->conf[(size_t)(l - 1) * s->rows + j]);
            if (shadow) shadow[(size_t)(l - 1) * sh->init_window + j] = sd[(size_t)(l - 1) * W + j];
            if (margin) margin[(size_t)(l - 1) * sh->init_window + j] = mg;
        }
    for (int32_t l = 1; l <= L; ++l) {
        int32_t c = 0;
        double tcs = 0.0, fcs = 0.0;
        for (int32_t j = 0; j < W; ++j) {
            const int match = sd[(size_t)(l - 1) * W + j] == sd[(size_t)(L - 1) * W + j];
            const double cf = s->conf[(size_t)(l - 1) * s->rows + j];
            c += match;
            if (match) tcs += cf; else fcs += cf;
        }
        s->Sc[l - 1] = (double)c;
        s->Stcs[l - 1] = tcs;
        s->Sfcs[l - 1] = fcs;
    }
    s->Sn = (double)W;
    refresh_tau(s);
    s->T = P;
    s->x_in = sd[(size_t)(L - 1) * W + (W - 1)];
    free(sd);
    if (s->temperature > 0.0) {
        /* the first generated token is drawn from the target's filtered distribution at the last prompt position */
        double *pp = (double *)malloc(sizeof(double) * (size_t)sh->vocab);
        ora_exit_head(s, hidden_at(s, L, W - 1), NULL, NULL, s->plog);
        ora_nucleus(s->plog, sh->vocab, s->temperature, s->top_p, pp);
        s->x_in = ora_sample_cdf(pp, sh->vocab, ora_uniform(s->seed, P, 2));
        free(pp);
    }
    choose_next(s, 0, 0);
    if (info) {
        memset(info, 0, sizeof(*info));
        info->n_emitted = 1;
        info->emitted[0] = s->x_in;
        info->next_E = s->E;
        info->next_gamma = s->gamma;
        info->Sn = s->Sn;
        info->next_tau = s->tau[s->E - 1];
    }
    return s->x_in;
}

int ora_round(ora_seq *s, int32_t remaining, ora_round_info *info, int32_t *shadow, float *margin,
              int32_t *counts) {
    const ora_shape *sh = &s->sh;
    const int32_t d = sh->d_model, L = sh->n_layers, stride = sh->g_max + 1;
    const int32_t E = s->E;
    /* Algorithm 1: with dynamic draft-exiting the loop runs up to d_max steps, otherwise gamma steps */
    int32_t g_cap = s->exit_mode ? sh->g_max : s->gamma;
    if (remaining < 1) return -1;
    if (g_cap > remaining - 1) g_cap = remaining - 1;
    if (g_cap > ORA_MAX_GAMMA || g_cap + 1 > s->rows || s->T + g_cap + 1 > sh->max_seq) return -2;
    int32_t drafts[ORA_MAX_GAMMA];
    double draft_conf[ORA_MAX_GAMMA + 1];
    const double tau_E = s->tau[E - 1];
    int32_t in = s->x_in, g = 0, stopped = 0;
    const int samp = s->temperature > 0.0;
    const int32_t V = sh->vocab;
    double *pp = NULL, *qq = NULL, *rr = NULL;
    if (samp) {
        pp = (double *)malloc(sizeof(double) * (size_t)V);
        qq = (double *)malloc(sizeof(double) * (size_t)V);
        rr = (double *)malloc(sizeof(double) * (size_t)V);
        memset(&s->sinfo, 0, sizeof(s->sinfo));
    }
    /* draft: tokens through layers 1..E + exit head (Algorithm 1, draft loop); a token whose confidence is
     * below the threshold ends the loop and is not appended */
    for (int32_t i = 0; i < g_cap; ++i) {
        int32_t tok;
        ora_embed(s, in, hidden_at(s, 0, i));
        for (int32_t l = 1; l <= E; ++l) ora_layer_rows(s, l, hidden_at(s, l - 1, i), s->T + i, 1, hidden_at(s, l, i));
        if (samp) {
            /* the confidence stays the top-1 probability at temperature 1 (Sec. 4.4); the token is drawn from the
             * exit head's filtered distribution */
            float *lg = s->qlog + (size_t)i * V;
            ora_exit_head(s, hidden_at(s, E, i), &tok, NULL, lg);
            draft_conf[i] = ora_confidence(lg, V);
            if (s->exit_mode && draft_conf[i] < tau_E) { stopped = 1; break; }
            ora_nucleus(lg, V, s->temperature, s->top_p, qq);
            s->sinfo.u_draft[i] = ora_uniform(s->seed, (int64_t)s->T + 1 + i, 0);
            tok = ora_sample_cdf(qq, V, s->sinfo.u_draft[i]);
            s->sinfo.q_x[i] = qq[tok];
        } else {
            exit_head_conf(s, hidden_at(s, E, i), &tok, NULL, &draft_conf[i]);
            if (s->exit_mode && draft_conf[i] < tau_E) { stopped = 1; break; }
        }
        drafts[g++] = tok;
        in = tok;
    }
    /* verify: the last input through layers 1..E, then all g+1 rows through layers E+1..L, reusing the
     * exit layer's cached hidden states and the KV cache written while drafting */
    ora_embed(s, in, hidden_at(s, 0, g));
    for (int32_t l = 1; l <= E; ++l) ora_layer_rows(s, l, hidden_at(s, l - 1, g), s->T + g, 1, hidden_at(s, l, g));
    for (int32_t l = E + 1; l <= L; ++l) ora_layer_rows(s, l, hidden_at(s, l - 1, 0), s->T, g + 1, hidden_at(s, l, 0));
    /* shadow tokens: exit head on every layer's hidden state of every row (Sec. 4.2) */
    int32_t *sd = (int32_t *)malloc(sizeof(int32_t) * (size_t)L * stride);
    for (int32_t l = 1; l <= L; ++l)
        for (int32_t i = 0; i <= g; ++i) {
            float mg;
            exit_head_conf(s, hidden_at(s, l, i), &sd[(size_t)(l - 1) * stride + i], &mg, &s->conf[(size_t)(l - 1) * s->rows + i]);
            if (shadow) shadow[(size_t)(l - 1) * stride + i] = sd[(size_t)(l - 1) * stride + i];
            if (margin) margin[(size_t)(l - 1) * stride + i] = mg;
        }
    const int32_t *verified = sd + (size_t)(L - 1) * stride;
    int32_t n, last_token;
    if (samp) {
        /* Sec. 2: draft i is accepted with probability min(1, p(x)/q(x)); after the first rejection the token
         * comes from the normalised max(0, p - q) of that position, after g acceptances from p at position g */
        for (int32_t i = 0; i <= g; ++i) ora_exit_head(s, hidden_at(s, L, i), NULL, NULL, s->plog + (size_t)i * V);
        n = 0;
        int rejected = 0;
        while (n < g) {
            const int32_t x = drafts[n];
            ora_nucleus(s->plog + (size_t)n * V, V, s->temperature, s->top_p, pp);
            ora_nucleus(s->qlog + (size_t)n * V, V, s->temperature, s->top_p, qq);
            const double u = ora_uniform(s->seed, (int64_t)s->T + 1 + n, 1);
            s->sinfo.u_accept[n] = u;
            s->sinfo.p_x[n] = pp[x];
            s->sinfo.n_tests = n + 1;
            const double ratio = pp[x] / qq[x];
            if (u < (ratio < 1.0 ? ratio : 1.0)) ++n;
            else { rejected = 1; break; }
        }
        s->sinfo.u_final = ora_uniform(s->seed, (int64_t)s->T + 1 + n, 2);
        s->sinfo.from_residual = rejected;
        if (rejected) {
            ora_residual(pp, qq, V, rr);
            last_token = ora_sample_cdf(rr, V, s->sinfo.u_final);
        } else {
            ora_nucleus(s->plog + (size_t)g * V, V, s->temperature, s->top_p, pp);
            last_token = ora_sample_cdf(pp, V, s->sinfo.u_final);
        }
        free(pp); free(qq); free(rr);
    } else {
        n = ora_accept_len(drafts, verified, g);
        last_token = verified[n];
    }
    /* matches within the valid context i = 0..n, decayed statistics (Eq. 2); the number of valid
     * positions is n + 1 */
    for (int32_t l = 1; l <= L; ++l) {
        int32_t c = 0;
        double tcs = 0.0, fcs = 0.0;    /* confidence sums over matched / mismatched shadow tokens (Sec. 4.4) */
        for (int32_t i = 0; i <= n; ++i) {
            const int match = sd[(size_t)(l - 1) * stride + i] == verified[i];
            const double cf = s->conf[(size_t)(l - 1) * s->rows + i];
            c += match;
            if (match) tcs += cf; else fcs += cf;
        }
        if (counts) counts[l - 1] = c;
        s->Sc[l - 1] = ora_decay_step(s->Sc[l - 1], sh->omega, (double)c);
        s->Stcs[l - 1] = ora_decay_step(s->Stcs[l - 1], sh->omega, tcs);
        s->Sfcs[l - 1] = ora_decay_step(s->Sfcs[l - 1], sh->omega, fcs);
    }
    s->Sn = ora_decay_step(s->Sn, sh->omega, (double)(n + 1));
    refresh_tau(s);
    if (info) {
        memset(info, 0, sizeof(*info));
        info->E = E; info->gamma = s->gamma; info->g = g;
        info->n_accept = n; info->n_emitted = n + 1;
        for (int32_t i = 0; i < g; ++i) info->drafts[i] = drafts[i];
        for (int32_t i = 0; i < n; ++i) info->emitted[i] = drafts[i];   /* (greedy: equal to the target's tokens) */
        info->emitted[n] = last_token;
        info->loaded_layers = g * E + L;
        info->stopped = stopped;
        info->tau = tau_E;
        for (int32_t i = 0; i < g + stopped; ++i) info->draft_conf[i] = draft_conf[i];
    }
    s->T += n + 1;
    s->x_in = last_token;
    free(sd);
    choose_next(s, g, n);
    if (info) { info->next_E = s->E; info->next_gamma = s->gamma; info->Sn = s->Sn; info->next_tau = s->tau[s->E - 1]; }
    return 0;
}
