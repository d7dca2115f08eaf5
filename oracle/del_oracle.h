/*
 * CPU oracle for the greedy self-speculative decode round with dynamic exit
 * layer selection (DEL).  TEST INFRASTRUCTURE ONLY: it exists to check the
 * CUDA library and to be timed as the CPU baseline; the product never calls it.
 * It shares no code with the CUDA path.
 *
 * Precision: weights are bf16 bit patterns (expanded exactly to float);
 * activations, the KV cache and logits are stored as float; every reduction
 * (dot products, mean of squares, softmax sums, attention-weighted sums) is
 * accumulated in double in a fixed order that does not depend on how many rows
 * are processed together.  The acceptance statistics and the selection run in
 * double with no fused multiply-add.
 *
 * Pinned by tests/test_oracle_*.py against: an independent non-cached forward
 * pass, closed forms for RMSNorm / softmax / SiLU / RoPE, greedy speculative ==
 * greedy auto-regressive for every (E, gamma), the paper's worked example of a
 * round, brute-force shadow tokens from truncated models, the decayed-sum
 * definition, exhaustive evaluation of the tokens-per-layer formula, and for
 * dynamic draft-exiting: the softmax definition of the confidence, Eq. 3 from
 * explicit histories, and the two limits of the threshold (never / always stop).
 * Speculative sampling: the uniform numbers by a Kolmogorov-Smirnov test, the
 * filtered distribution by scipy / numpy on the same rows and its limits, the
 * inverse CDF by numpy's searchsorted, acceptance and residual by the identity
 * that makes speculative sampling exact and by a Monte-Carlo run, the round by
 * a replay of its decisions from the logits it exposes.
 * Parity unpinned: the absolute values of logits of the random model (no
 * published activations exist) and any distribution-level behaviour that would
 * need the paper's trained checkpoints.
 */
#ifndef DEL_ORACLE_H
#define DEL_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ORA_MAX_GAMMA 32

typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
    float rms_eps, rope_theta;
    int32_t max_seq;
    int32_t e_min, e_max, g_min, g_max, init_window;
    double omega;
} ora_shape;

/* bf16 bit patterns, matrices [out, in] row-major; per-layer arrays have n_layers entries */
typedef struct {
    const uint16_t *tok_emb, *final_norm, *lm_head;
    const uint16_t *const *attn_norm, *const *wq, *const *wk, *const *wv, *const *wo;
    const uint16_t *const *ffn_norm, *const *w_gate, *const *w_up, *const *w_down;
} ora_weights;

typedef struct {
    int32_t E, gamma;        /* the (E, gamma) this round ran with */
    int32_t g;               /* drafts actually made (gamma clipped near the end of generation) */
    int32_t n_accept;        /* accepted drafts, 0..g */
    int32_t n_emitted;       /* n_accept + 1 */
    int32_t drafts[ORA_MAX_GAMMA];
    int32_t emitted[ORA_MAX_GAMMA + 1];
    int32_t next_E, next_gamma;
    int32_t loaded_layers;   /* g * E + L : the paper's cost of the round */
    double Sn;               /* decayed number of valid positions after this round */
    /* dynamic draft-exiting (Sec. 4.4) */
    int32_t stopped;         /* 1: the draft loop ended on a confidence below the threshold */
    int32_t pad_;
    double tau;              /* threshold of the exit layer the draft loop used */
    double next_tau;         /* threshold of the next round's exit layer */
    double draft_conf[ORA_MAX_GAMMA + 1]; /* confidence of every drafted token, the one that ended the loop included */
} ora_round_info;

typedef struct ora_seq ora_seq;

ora_seq *ora_seq_create(const ora_shape *shape, const ora_weights *w);
void ora_seq_destroy(ora_seq *s);

/* Fix the policy: (E, gamma) stay as given (gamma = 0 is vanilla auto-regressive decoding).
 * E <= 0 restores the dynamic selection. */
void ora_set_policy(ora_seq *s, int32_t fixed_E, int32_t fixed_gamma);

/* Baseline FS(E-gamma) of Sec. 5.1: fixed exit layer, the speculation length starts at gamma0 and moves by
 * +1 after a round whose drafts were all accepted, by -1 after a round with a rejection. */
void ora_set_policy_fs(ora_seq *s, int32_t fixed_E, int32_t gamma0);
int32_t ora_fs_next_gamma(int32_t gamma, int32_t g, int32_t n, int32_t g_min, int32_t g_max);

/* Prefill over the prompt, initial statistics from the last init_window positions, first token and
 * first (E, gamma).  shadow/margin (may be NULL): [n_layers][init_window] row-major, layer 1 first,
 * only the first W = min(init_window, n_prompt) columns are written.  Returns the first token. */
int32_t ora_prefill(ora_seq *s, const int32_t *prompt, int32_t n_prompt, int32_t *shadow, float *margin,
                    ora_round_info *info);

/* One speculative round; remaining = tokens still to be generated (>= 1).
 * shadow/margin/counts may be NULL; shadow and margin are [n_layers][g_max + 1], counts [n_layers]. */
int ora_round(ora_seq *s, int32_t remaining, ora_round_info *info, int32_t *shadow, float *margin,
              int32_t *counts);

/* Dynamic draft-exiting (Sec. 4.4, Algorithm 1): mode 1 lets the draft loop run up to g_max steps and end
 * it at the first token whose confidence is below the exit layer's threshold (that token is dropped);
 * mode 0 (default) drafts exactly gamma tokens.  The confidence statistics are tracked in both modes. */
void ora_set_exit_mode(ora_seq *s, int32_t mode);
/* decayed confidence sums and thresholds, [n_layers] each, index l-1 */
void ora_get_conf_stats(const ora_seq *s, double *Stcs, double *Sfcs, double *tau);
void ora_set_conf_stats(ora_seq *s, const double *Stcs, const double *Sfcs);
/* confidence of the shadow tokens of the last round (or of the prefill window): [n_layers][n_cols] */
void ora_get_conf(const ora_seq *s, double *conf, int32_t n_cols);

/* state access */
int32_t ora_committed_len(const ora_seq *s);
void ora_get_stats(const ora_seq *s, double *Sc /*[n_layers], index l-1*/, double *Sn, int32_t *E, int32_t *gamma);
void ora_set_stats(ora_seq *s, const double *Sc, double Sn, int32_t E, int32_t gamma);
/* hidden state h^l (l = 0 is the embedding) of row i of the last round / of window column i after prefill */
const float *ora_hidden(const ora_seq *s, int32_t layer, int32_t row);
/* cached key / value row of 1-based layer at a position, n_kv_heads * head_dim floats */
const float *ora_k_row(const ora_seq *s, int32_t layer, int32_t pos);
const float *ora_v_row(const ora_seq *s, int32_t layer, int32_t pos);

/* building blocks, exposed so that tests can pin each of them */
void ora_embed(const ora_seq *s, int32_t token, float *h);
void ora_rmsnorm(const float *x, const uint16_t *gain_bf16, int32_t d, float eps, float *out);
void ora_rope(float *x, int32_t n_heads, int32_t head_dim, int32_t pos, float theta);
void ora_softmax(const float *x, int32_t n, double *p);
float ora_silu(float x);
/* rows at consecutive positions pos0..pos0+m-1 through 1-based layer; writes K,V at those positions */
void ora_layer_rows(ora_seq *s, int32_t layer, const float *h_in, int32_t pos0, int32_t m, float *h_out);
/* shared final RMSNorm + LM head + greedy choice (lowest id on ties); margin = top1 - top2 logit */
void ora_exit_head(const ora_seq *s, const float *h, int32_t *token, float *margin, float *logits_or_null);

/* top-1 softmax probability of a logit row */
double ora_confidence(const float *logits, int32_t V);
/* Eq. 3 for one layer; Smis = decayed number of mismatched shadow tokens */
double ora_threshold(double Stcs, double Sc, double Sfcs, double Smis);
int32_t ora_accept_len(const int32_t *drafts, const int32_t *verified, int32_t g);
double ora_decay_step(double S, double omega, double a);
double ora_tpl(double alpha, int32_t l, int32_t d, int32_t L);
void ora_select(const double *Sc /*index l-1*/, double Sn, int32_t L, int32_t e_min, int32_t e_max, int32_t g_min,
                int32_t g_max, int32_t *E, int32_t *gamma);
int ora_num_threads(void);

/* ---- speculative sampling (Sec. 2: accept a draft with probability min(1, p/q), otherwise resample from
 * the normalised max(0, p - q); one more token from p when every draft was accepted), with the temperature
 * and nucleus (top-p) filtering of Sec. 5 / the inference setup applied to both distributions. */

/* Uniform number in [0, 1) of a counter-based generator: a function of (seed, absolute position of the token
 * being decided, purpose) only, so that no generator state has to be carried.  purpose 0: drawing the draft
 * token, 1: the acceptance test of that draft, 2: the token that ends the round (residual or extra token). */
double ora_uniform(uint64_t seed, int64_t pos, int32_t purpose);
/* probs[i] = softmax(logits / temperature) restricted to the nucleus and renormalised.  The nucleus is the
 * shortest prefix, in order of descending probability (equal probabilities: lower token id first), whose mass
 * reaches top_p: a token is kept iff the mass strictly before it is < top_p.  top_p >= 1 keeps everything. */
void ora_nucleus(const float *logits, int32_t V, double temperature, double top_p, double *probs);
/* inverse CDF in token-id order: the first token whose cumulative probability exceeds u */
int32_t ora_sample_cdf(const double *probs, int32_t V, double u);
/* r = max(0, p - q) normalised to sum 1; returns the mass before normalisation (0: r is set to p) */
double ora_residual(const double *p, const double *q, int32_t V, double *r);

/* temperature <= 0 switches sampling off (greedy verification, the default).  Call before ora_prefill: the
 * first token is drawn too (purpose 2 at position n_prompt). */
void ora_set_sampling(ora_seq *s, double temperature, double top_p, uint64_t seed);

typedef struct {
    int32_t n_tests;                    /* acceptance tests made: min(n_accept + 1, g) */
    int32_t from_residual;              /* 1: the round's last token came from the residual distribution */
    double u_draft[ORA_MAX_GAMMA];      /* uniform numbers used */
    double u_accept[ORA_MAX_GAMMA];
    double u_final;
    double q_x[ORA_MAX_GAMMA];          /* filtered draft probability of each drafted token */
    double p_x[ORA_MAX_GAMMA];          /* filtered target probability of each tested draft */
} ora_sample_info;
/* record of the last round (sampling on) */
void ora_get_sample_info(const ora_seq *s, ora_sample_info *out);
/* logits of the last round: which = 0 the exit head's row of draft i (i < g, plus the dropped one when the
 * loop stopped), which = 1 the target's row i (i <= g); valid until the next round */
const float *ora_round_logits(const ora_seq *s, int32_t which, int32_t row);

#ifdef __cplusplus
}
#endif
#endif
