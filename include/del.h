/*
 * libdel — the hot path of one greedy self-speculative decode round with dynamic exit-layer
 * selection (DEL) on a Llama-style decoder, as hand-written CUDA kernels for sm_100a.
 *
 * The calls follow the paper's statement of the method:
 *   Sec. 2 ("Early-exit self-speculative decoding"): draft gamma tokens with the first E layers plus the
 *          LM head, verify them with the full model, reusing the KV cache written while drafting;
 *   Sec. 2 ("Speculative decoding", greedy case): keep the longest prefix of drafts whose tokens equal
 *          the target model's top-1 tokens, plus the target's next token (1..gamma+1 tokens per round);
 *   Sec. 4.2: run the LM head over every layer's cached hidden states of the round ("shadow tokens"),
 *          count matches with the target's tokens inside the valid context, keep decayed sums;
 *   Sec. 4.1 (Eq. 1) and Sec. 4.3: pick the next (E, gamma) maximising expected tokens per loaded layer;
 *   Sec. 4.4 and Eq. 3: confidence of a token = its softmax probability; decayed confidence sums over
 *          matched and mismatched shadow tokens give each layer a threshold;
 *   Algorithm 1: the loop, with its confidence break when a sequence is in exit mode (del_set_exit_mode);
 *   Sec. 2 ("Speculative decoding", general case) with the temperature and top-p of the inference setup:
 *          speculative sampling for a sequence that asks for it (del_set_sampling).
 *
 * Conventions
 *   - Plain C ABI.  Every pointer is either HOST or DEVICE memory as stated per field/argument.
 *   - Return value 0 on success, a negative DEL_E* code otherwise; nothing throws or aborts.
 *   - The library never allocates device memory: weights, KV pages, page table and the workspace are
 *     allocated by the caller, stay owned by the caller and must outlive the context.  Weights are
 *     never written.  KV pages, the page table and the workspace are written only by work enqueued on
 *     the stream given to del_init.  The context itself (host bookkeeping, pinned staging buffers,
 *     events) is owned by the library and freed by del_destroy.
 *   - All device work is enqueued on that one stream.  Calls documented "async" return without
 *     synchronising; the others synchronise the stream before returning.
 *   - One context serves max_batch independent sequences (0 <= seq < max_batch), each with its own
 *     committed length, acceptance statistics and (E, gamma).
 *   - Layers are 1-based (layer 0 = embedding output); gamma = 0 is a legal speculation length and
 *     makes a round one plain auto-regressive step.
 */
#ifndef DEL_H
#define DEL_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DEL_MAX_GAMMA 31          /* largest g_max accepted by del_init */
#define DEL_MAX_ROWS 64           /* most rows (over all sequences) one layer pass may carry */

enum {
    DEL_OK = 0,
    DEL_EINVAL = -1,              /* bad shape, bad argument, E or gamma out of range */
    DEL_ENOSPC = -2,              /* KV pages or max_seq exhausted, workspace too small */
    DEL_ESTATE = -3,              /* call order wrong (e.g. verify before draft, round before prefill) */
    DEL_ETIMEOUT = -4,            /* a bounded device-side wait expired (kernel reported it); see below */
    DEL_ECUDA = -5                /* a CUDA call failed; see del_last_cuda_error */
};

typedef struct del_ctx del_ctx;   /* opaque, owned by the library */

/* Model shape, cache geometry and DEL hyper-parameters.
 * Requirements checked by del_init: head_dim in {64, 128}; n_heads % n_kv_heads == 0;
 * d_model % 32 == 0; vocab % 32 == 0; d_ffn % 16 == 0; page_size == 16; max_seq % page_size == 0;
 * 1 <= e_min <= e_max < n_layers; 0 <= g_min <= g_max <= DEL_MAX_GAMMA;
 * max_batch * (g_max + 1) <= DEL_MAX_ROWS; 1 <= init_window <= 32. */
typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
    float rms_eps, rope_theta;    /* rope_theta is informational: the tables below are what is used */
    int32_t max_batch, max_seq, page_size, n_pages;
    int32_t e_min, e_max, g_min, g_max;   /* search ranges of the selection (Sec. 4.3) */
    int32_t init_window;          /* prompt positions that seed the statistics (App. B.2: 32) */
    double omega;                 /* decay of the acceptance statistics (App. B.2: 0.95) */
} del_shape;

/* All tensors bf16 in DEVICE memory, matrices row-major [out_features, in_features].  The per-layer
 * members are HOST arrays of n_layers DEVICE pointers (index l-1 for layer l); the arrays themselves
 * are read only during del_init. */
typedef struct {
    const void *tok_emb;          /* [vocab, d_model] */
    const void *final_norm;       /* [d_model] gains of the final RMSNorm (shared by every exit) */
    const void *lm_head;          /* [vocab, d_model] */
    const void *const *attn_norm; /* [d_model] */
    const void *const *wq;        /* [n_heads*head_dim, d_model] */
    const void *const *wk;        /* [n_kv_heads*head_dim, d_model] */
    const void *const *wv;        /* [n_kv_heads*head_dim, d_model] */
    const void *const *wo;        /* [d_model, n_heads*head_dim] */
    const void *const *ffn_norm;  /* [d_model] */
    const void *const *w_gate;    /* [d_ffn, d_model] */
    const void *const *w_up;      /* [d_ffn, d_model] */
    const void *const *w_down;    /* [d_model, d_ffn] */
    const float *rope_cos;        /* DEVICE fp32 [max_seq, head_dim/2]: cos(pos * theta^(-2j/head_dim)) */
    const float *rope_sin;        /* DEVICE fp32 [max_seq, head_dim/2]; pairing is (j, j + head_dim/2) */
} del_weights;

/* Paged KV cache in DEVICE memory.  The library assigns pages to sequences and writes page_table.
 *   k_pages: bf16 [n_pages][n_layers][n_kv_heads][page_size][head_dim]   (keys after rotary embedding)
 *   v_pages: bf16 [n_pages][n_layers][n_kv_heads][head_dim][page_size]   (values, transposed per page)
 *   page_table: int32 [max_batch][max_seq / page_size]
 * The pages must hold finite values when handed over (e.g. zeros): slots of a page that are not written yet are
 * masked with a probability of exactly 0, and 0 times a NaN bit pattern would still be NaN. */
typedef struct {
    void *k_pages, *v_pages;
    int32_t *page_table;
} del_kv;

/* Result of one round for one sequence (HOST memory). */
typedef struct {
    int32_t E, gamma;             /* the setting the round ran with */
    int32_t g;                    /* drafts made: gamma clipped to the tokens still wanted minus one */
    int32_t n_accept;             /* accepted drafts, 0..g */
    int32_t n_emitted;            /* n_accept + 1; 0 if the sequence was not live */
    int32_t tokens[DEL_MAX_GAMMA + 1];   /* the n_emitted tokens committed by the round */
    int32_t next_E, next_gamma;   /* choice for the next round */
    int32_t status;               /* 0, or a DEL_E* code reported by a kernel */
    int32_t stopped;              /* 1: the draft loop ended on a confidence below tau (that token was dropped) */
    double tau;                   /* threshold of layer E the draft loop compared with (exit mode), else 0 */
    double next_tau;              /* Eq. 3 for layer next_E from the updated statistics */
} del_round_out;

/* Bytes of DEVICE workspace del_init needs for this shape (256-byte aligned base expected). */
size_t del_workspace_bytes(const del_shape *shape);

/* Creates a context.  shape, weights, kv: HOST structs (copied).  workspace: DEVICE, ws_bytes >=
 * del_workspace_bytes(shape); its contents are clobbered.  cuda_stream: a cudaStream_t (0 = default
 * stream).  Errors: DEL_EINVAL (shape requirements, null pointers), DEL_ENOSPC (workspace too small,
 * n_pages cannot hold even one sequence), DEL_ECUDA. */
int del_init(del_ctx **ctx, const del_shape *shape, const del_weights *weights, const del_kv *kv,
             void *workspace, size_t ws_bytes, void *cuda_stream);

/* Prefill (Algorithm 1, "Require"; Sec. 4.3 last sentence; App. B.2): runs all layers over the prompt
 * (HOST int32 [n_prompt], 1 <= n_prompt, n_prompt + max_new_tokens + g_max + 1 <= max_seq), fills the KV
 * cache, computes every layer's shadow tokens over the last min(init_window, n_prompt) positions,
 * seeds the statistics with their agreement with the last layer, emits the first token and picks the
 * first (E, gamma).  max_new_tokens (>= 1) counts that first token; later rounds clip gamma so that
 * exactly max_new_tokens tokens are produced.  Any previous state of `seq` is released first.
 * Synchronises.  first_out (HOST, may be NULL): n_emitted = 1, tokens[0], next_E, next_gamma. */
int del_prefill(del_ctx *ctx, int seq, const int32_t *prompt, int n_prompt, int max_new_tokens,
                del_round_out *first_out);

/* Draft phase (Sec. 2 early-exit drafting; Algorithm 1 draft loop): gamma tokens, each through embedding,
 * layers 1..E, shared final RMSNorm, LM head, argmax.  gamma is clipped like in del_round.  Async, except
 * for a sequence in exit mode (del_set_exit_mode): then gamma is the most the loop may draft, the host reads
 * each token's confidence (one synchronisation per token) and the loop ends at the first one below the
 * threshold.  Errors: DEL_EINVAL (E outside [1, n_layers-1], gamma outside [0, g_max]),
 * DEL_ESTATE (no prefill, sequence finished, previous round not completed), DEL_ENOSPC. */
int del_draft(del_ctx *ctx, int seq, int E, int gamma);

/* Verify phase (Sec. 2; Algorithm 1 "Verify D by M_p"): the last input token through layers 1..E, then
 * the g+1 positions through layers E+1..L starting from the exit layer's cached hidden states; KV
 * written for all g+1 positions; every layer's hidden state of every position kept.  Async.
 * DEL_ESTATE unless del_draft came before. */
int del_verify(del_ctx *ctx, int seq);

/* Shadow tokens, acceptance and statistics (Sec. 4.2, Algorithm 1 DEL_Update up to the alpha update):
 * one LM-head pass over the stacked hidden states of all layers and positions with a fused argmax,
 * longest-matching-prefix acceptance, per-layer match counts over the n_accept+1 valid positions,
 * decayed sums.  Commits the accepted tokens.  Synchronises (the host learns n_accept).
 * out (HOST, may be NULL) gets everything except next_E / next_gamma. */
int del_layer_accept(del_ctx *ctx, int seq, del_round_out *out);

/* Selection (Eq. 1 in its sum form, Sec. 4.3): argmax over E in [e_min, e_max], gamma in
 * [g_min, g_max] of (sum_{k<=gamma} alpha_E^k) / (gamma*E + L), first maximum in E-major order.
 * Synchronises; writes the choice to *E and *gamma (HOST, may be NULL) and keeps it for del_round. */
int del_select(del_ctx *ctx, int seq, int32_t *E, int32_t *gamma);

/* One whole round for every live sequence at once (each with its own E, gamma and state): draft,
 * verify, layer_accept and select with layer passes shared by the sequences, and one host round trip
 * at the end: the last kernel posts the results in pinned host memory and the call returns as soon as
 * they are there (that kernel may still be retiring; anything enqueued on the stream afterwards is
 * ordered behind it, and every other call of this library synchronises before it reads device state).
 * out: HOST array [max_batch]; entries of sequences that are not live get n_emitted = 0.  Returns
 * DEL_ESTATE if no sequence is live. */
int del_round(del_ctx *ctx, del_round_out *out);

/* Fix the policy of a sequence: del_round uses (E, gamma) as given instead of the selection
 * (gamma = 0: plain auto-regressive decoding).  E <= 0 restores the dynamic choice. */
int del_set_policy(del_ctx *ctx, int seq, int E, int gamma);

/* The paper's baseline FS(E-gamma) on the same round (Sec. 5.1): fixed exit layer E, the speculation length
 * starts at gamma0 (>= 1) and moves by +1 after a round whose drafts were all accepted and by -1 after a
 * round with a rejection, within [max(1, g_min), g_max].  (The baseline LS(E-gamma) is del_set_policy.)
 * del_set_policy with E <= 0 ends it. */
int del_set_policy_fs(del_ctx *ctx, int seq, int E, int gamma0);

/* Dynamic draft-exiting (Sec. 4.4, Algorithm 1) for a sequence: mode 1 lets the draft loop run for up to
 * g_max tokens (del_round) or the given gamma (del_draft) and ends it at the first token whose
 * confidence (top-1 softmax probability of the exit head, fp32) is below the threshold of layer E from
 * Eq. 3; that token is not appended, and its pass through layers 1..E is reused by the verify phase.
 * The kernel that finalises a drafted token takes the decision and posts it in pinned host memory; the host polls for
 * it before it enqueues the next draft step, so a round then has one host round trip per drafted token instead of one per round.  mode 0 (default) drafts exactly gamma tokens.  The
 * confidence statistics and thresholds are maintained in both modes. */
int del_set_exit_mode(del_ctx *ctx, int seq, int mode);

/* Speculative sampling (Sec. 2) for a sequence slot, with temperature and nucleus (top-p) filtering applied to
 * the draft and to the target distribution alike.  temperature > 0 switches it on (top_p > 0 then), <= 0 back
 * to greedy verification (the default).  While it is on:
 *   - draft i is drawn from softmax(exit-head logits / temperature) restricted to its nucleus and renormalised
 *     (the nucleus: tokens in order of descending probability, equal ones by ascending id, kept while the mass
 *     before them is < top_p), by inverse CDF in token-id order;
 *   - it is accepted when u < min(1, p(x) / q(x)), p and q the filtered target / draft probabilities; the first
 *     rejected position gets its token from the normalised max(0, p - q); after g acceptances one more token
 *     comes from the target's filtered row g; the first token of del_prefill is drawn from the target's row of
 *     the last prompt position;
 *   - shadow tokens, confidences, statistics and the (E, gamma) selection are unchanged (greedy tokens of
 *     every layer compared with the last layer's; the valid context is rows 0..n_accept).
 * The uniform numbers are a function of (seed, absolute position of the token decided, purpose: 0 draft draw,
 * 1 acceptance test, 2 last token of the round) only: the splitmix64 finaliser applied twice, 53 bits.
 * The setting belongs to the slot and survives del_prefill / del_release.  The logit rows the decisions need
 * are stored by the LM-head kernels that run anyway.  vocab must be a multiple of 4 and <= 262144.  Errors: DEL_EINVAL, DEL_ESTATE (a round is half done). */
int del_set_sampling(del_ctx *ctx, int seq, double temperature, double top_p, uint64_t seed);

/* Record of the last sampled round (synchronises; any pointer may be NULL): acceptance tests made, whether
 * the last token came from the residual distribution, and the filtered draft / target probability of draft i
 * (HOST float [32] each; p_x is valid for the tested drafts only). */
int del_get_sample_info(del_ctx *ctx, int seq, int32_t *n_tests, int32_t *from_residual, float *q_x, float *p_x);

/* Test reader: logits row (HOST float [vocab]) of the last sampled round: which = 0 the exit head's row of
 * draft `row`, which = 1 the target's row `row` (0..g).  Synchronises. */
int del_get_round_logits(del_ctx *ctx, int seq, int which, int row, float *out);

/* Test reader: shadow tokens and their confidences of the first n_cols slots (1 <= n_cols <= 64) of every layer:
 * after del_prefill the whole initialisation window (n_cols = min(init_window, n_prompt)), which del_get_shadow
 * and del_get_conf, sized for a round, cut at g_max + 1 columns.  HOST [n_layers][n_cols] each, either may be
 * NULL.  Synchronises. */
int del_get_window(del_ctx *ctx, int seq, int n_cols, int32_t *shadow, float *conf);

/* Test hook: the sampling kernels' device functions on one caller-supplied pair of rows (HOST float [vocab],
 * vocab <= the model's).  out (HOST int32 [4]): the token drawn from the filtered draft row with u_draft; 1 if
 * u_accept accepts it; the token the residual distribution gives with u_final; the token the filtered target
 * row gives with u_final.  prob (HOST double [2]): filtered q(x), p(x).  stat (HOST int32 [8], may be NULL):
 * per row (draft, target) the key of the smallest kept weight, ties kept, ties present, 0.  Uses sequence 0's
 * sampling buffers as scratch.  Synchronises. */
int del_sample_probe(del_ctx *ctx, const float *p_logits, const float *q_logits, int vocab, double temperature, double top_p,
                     double u_draft, double u_accept, double u_final, int32_t *out, double *prob, int32_t *stat);

/* Confidence statistics (Sec. 4.4).  HOST double [n_layers] each, entry l-1 for layer l: decayed sums of
 * the confidences of matched / mismatched shadow tokens, and the thresholds of Eq. 3 (a mean over no
 * tokens counts as 1 for matched and 0 for mismatched ones).  Any pointer of the getter may be NULL.
 * Synchronise. */
int del_get_conf_stats(del_ctx *ctx, int seq, double *Stcs, double *Sfcs, double *tau);
int del_set_conf_stats(del_ctx *ctx, int seq, const double *Stcs, const double *Sfcs);
/* Confidences of the last round: shadow_conf fp32 [n_layers][g_max + 1] (shadow tokens of
 * del_layer_accept), draft_conf fp32 [g_max + 1] (draft i at entry i, the dropped one included).
 * HOST, either may be NULL.  Synchronises. */
int del_get_conf(del_ctx *ctx, int seq, float *shadow_conf, float *draft_conf);

/* Acceptance statistics, for resuming and for tests.  Sc: HOST double [n_layers], entry l-1 is the
 * decayed match count of layer l; Sn: decayed number of valid positions.  Synchronise. */
int del_get_stats(del_ctx *ctx, int seq, double *Sc, double *Sn, int32_t *E, int32_t *gamma);
int del_set_stats(del_ctx *ctx, int seq, const double *Sc, double Sn, int32_t E, int32_t gamma);

/* Introspection for tests; all synchronise and copy to HOST memory.
 *   del_get_shadow: int32 [n_layers][g_max + 1] shadow tokens and int32 [n_layers] match counts of the
 *                   last del_layer_accept of `seq` (either pointer may be NULL).
 *   del_get_hidden: fp32 [d_model], hidden state of `layer` (0..n_layers) at row `row` of the last pass.
 *   del_debug_logits: fp32 [vocab], logits of the exit head applied to that hidden state, computed by a
 *                   separate unfused kernel.
 *   del_get_kv:     fp32 [n_kv_heads*head_dim] key and value rows of `layer` (1-based) at position pos. */
int del_get_shadow(del_ctx *ctx, int seq, int32_t *shadow, int32_t *counts);
/* int32 [g_max]: the draft tokens of the sequence's last draft phase (first g entries are meaningful). */
int del_get_drafts(del_ctx *ctx, int seq, int32_t *drafts);
/* Overrides the token that the next round feeds first (used when resuming from a known stream). */
int del_force_token(del_ctx *ctx, int seq, int32_t token);
int del_get_hidden(del_ctx *ctx, int seq, int layer, int row, float *out);
int del_debug_logits(del_ctx *ctx, int seq, int layer, int row, float *out);
int del_get_kv(del_ctx *ctx, int seq, int layer, int pos, float *k_out, float *v_out);

/* DEL_ETIMEOUT.  The tensor-core kernels (stacked LM head, prefill GEMMs) wait on shared-memory barriers for
 * their own asynchronous copies and tensor-core instructions.  Every such wait gives up after 2^26 polls
 * (of the order of seconds to a minute, depending on the clock), records a non-zero code in the workspace's
 * error word, lets the kernel wind down (tensor memory freed) and return.  The call that next reads results
 * (del_prefill, del_layer_accept, del_select, del_round) then returns DEL_ETIMEOUT, clears the word, and the
 * context stays usable: the sequence's round did not complete and should be re-prefilled.
 * del_debug_inject_error writes `code` (non-zero) into that word with a stream-ordered copy from the host, as
 * an expired wait would have: a test hook for the error path that makes no kernel wait. */
int del_debug_inject_error(del_ctx *ctx, int code);

/* Committed length (prompt + emitted tokens) of a sequence, or a negative code. */
int del_committed_len(del_ctx *ctx, int seq);
/* Frees the sequence's KV pages and marks it empty. */
int del_release(del_ctx *ctx, int seq);
/* Kernel launches enqueued since del_init (for launch accounting). */
int64_t del_launch_count(const del_ctx *ctx);
/* Bytes the library itself copied host->device (plans, page-table entries, prompts) and
 * device->host (round results) since del_init. */
int del_get_traffic(const del_ctx *ctx, int64_t *h2d_bytes, int64_t *d2h_bytes);
/* Switches of the launch machinery (bit 0: programmatic dependent launch, bit 1: reserved,
 * bit 2: tcgen05 LM head instead of the streaming one, bit 3: record CUDA
 * events around every launch, bit 4: one weight-streaming CTA per SM, bit 5: prefill every prompt
 * position through the decode kernels instead of the tensor-core GEMMs, bit 6: the decode attention kernel in
 * passes of 64 rows instead of the flash-style prefill attention, bit 7: the stacked LM head runs only over the
 * layers the selection can pick (e_min..e_max) and the last one; shadow tokens, counts and statistics of the other
 * layers are then not maintained, bit 8: the mma.sync flash-style prefill attention also where the tcgen05 one
 * (head dimension 128) would run, bit 9: the decode attention kernel does not request the O-projection's weights into
 * L2).  Returns the previous flags. */
int del_set_flags(del_ctx *ctx, int flags);

/* With flag bit 3 set, per kernel class (0 QKV, 1 attention, 2 O-proj, 3 gate/up, 4 down, 5 draft LM
 * head, 6 stacked LM head, 7 other): summed device time in ms, launches, and algorithmic bytes (weights
 * or KV the launches had to read).  HOST arrays of 8 (any may be NULL); reset != 0 clears the sums. */
int del_get_kernel_times(del_ctx *ctx, double *ms, int64_t *launches, double *bytes, int reset);

/* Exit-head arg-max without any allocation (the paper has no counterpart: this entry point exists for
 * callers that cannot call cudaMalloc — a serving loop whose device memory pool is frozen after
 * start-up, a plug-in that receives tensors but no allocator, a process that has filled the GPU).
 * Needs no context.  x: DEVICE bf16 [rows][d_model], hidden rows already multiplied by the final norm's
 * gain (the norm's 1/rms is positive and cannot change the arg-max); lm_head: DEVICE bf16
 * [vocab][d_model]; tokens: DEVICE int32 [rows], token id of the largest logit per row (lowest id on
 * ties).  Async on cuda_stream.  The kernel's scratch (per-CTA arg-max partials) lives in a fixed
 * array inside the library image, DEL_STATIC_SCRATCH_BYTES per GPU that loads the library, held until
 * the process exits.  Limits: 1 <= rows <= DEL_MAX_ROWS, vocab % 16 == 0, d_model >= 256 and % 8 == 0;
 * anything larger than the fixed array can serve returns DEL_EINVAL.  No cudaMalloc / cudaFree or
 * allocating library routine is called.  All calls on a device share the array: calls that overlap on
 * the GPU (different streams) race, calls on one stream are safe; what a call reads from the array it
 * has written first.  The first call on each device looks up the array's device address: make that
 * call before any stream capture begins.  A row whose logits are all NaN has no largest one: its entry of
 * tokens is then 0x7fffffff, which is no token id. */
#define DEL_STATIC_SCRATCH_BYTES ((1 << 19) + 4096)
int del_head_argmax_static(const void *x, const void *lm_head, int rows, int vocab, int d_model, int32_t *tokens,
                           void *cuda_stream);

const char *del_strerror(int code);
/* Text of the last CUDA error seen by this context ("" if none). */
const char *del_last_cuda_error(const del_ctx *ctx);
void del_destroy(del_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif
