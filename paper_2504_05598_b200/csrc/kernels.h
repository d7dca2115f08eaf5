// Internal launch interface between the host-side round scheduler (del_api.cu) and the kernels.
#pragma once

#include "common.cuh"

// cudaFuncSetAttribute acts on the current device only: a kernel's dynamic shared-memory limit is raised once per
// device (a process may drive contexts on several GPUs).  `done` is the caller's static per-kernel record.
#define DEL_MAX_DEVICES 64
struct SmemAttrOnce {
    bool done[DEL_MAX_DEVICES] = {};
    template <typename K> cudaError_t set(K kern, int bytes) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < DEL_MAX_DEVICES && done[dev]) return cudaSuccess;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess && dev >= 0 && dev < DEL_MAX_DEVICES) done[dev] = true;
        return e;
    }
};

enum { EPI_QKV = 0, EPI_OPROJ = 1, EPI_GATEUP = 2, EPI_DOWN = 3, EPI_LMHEAD = 4 };

struct GemmArgs {
    Dims D;
    Buffers B;
    PassPlan plan;             // rows of the pass, by value: read from the constant bank, no dependent load
    int32_t layer;             // 1-based layer the op belongs to (LMHEAD: the exit layer)
    int32_t K;                 // in-features
    int32_t n_items;           // work items: tile pairs (QKV, GATEUP) or 16-row tiles
    const bf16 *X;             // activations (see rowgemm.cu for the indexing per epilogue)
    const bf16 *XL;            // their low parts (layer GEMMs; the LM head takes single bf16 rows)
    int32_t row0;              // layer GEMMs: first row of the pass this launch handles (a launch takes up to 32 rows)
    const bf16 *W0, *W1, *W2;
    const bf16 *gain_a, *gain_b;
    int32_t ctas_per_sm;       // weight-streaming CTAs per SM for passes of up to 8 rows: 1 or 2 (0: 2)
    int32_t *tile_ctr;         // per-launch zeroed counter for dynamic tile claims (nullptr: static round-robin)
    int32_t x_by_row;          // LMHEAD: activations are X[c] (stacked rows) instead of XE[seq][slot]
    const float *row_scale;    // LMHEAD with x_by_row: log2(e) / rms per row (nullptr: taken from B.SSE)
    float *logits_out;         // LMHEAD: also store the normalised logits, row c at logits_out[c * V] with x_by_row,
                               // else at logits_out[(seq * DEL_SAMPLE_ROWS + slot) * V]  (nullptr: not stored)
};

cudaError_t launch_rowgemm(int epi, const GemmArgs &a, int m, int n_sms, cudaStream_t st, bool pdl);
// CTAs an LM-head launch of m rows uses (= number of arg-max partials it leaves per row)
int rowgemm_lmhead_grid(int n_items, int m, int n_sms, int ctas_per_sm);

struct AttnArgs {
    Dims D;
    Buffers B;
    PassPlan plan;
    int32_t layer;
    int32_t n_splits;          // key-range splits per (segment, kv head)
    int32_t max_rows;          // largest segment (rows), decides the number of query tiles
    // Per segment: cache positions below this one were written before the host last synchronised with the stream
    // (positions committed in earlier rounds), so the kernel may read them before it waits for its producer.
    // Everything later may come from a launch that is still running (the wait of a launch covers its whole chain
    // of predecessors, but nothing bounds how far ahead of that wait a dependent launch may start).  0: nothing.
    int32_t early_pos[DEL_SEQ_MAX];
    // Weights that the launches after this one stream (the O-projection's, the head of gate / up): requested into L2
    // by this kernel's CTAs once their own cache reads are on their way, so that HBM works while attention, which is
    // bound by latency, runs.
    AttnPrefetch pf;
};
cudaError_t launch_attention(const AttnArgs &a, int n_seg, cudaStream_t st, bool pdl);
int attention_splits(int pages, int n_units, int tiles_par, int n_sms);

// control kernels
struct CtlArgs {
    Dims D;
    Buffers B;
    PassPlan plan;
    const bf16 *tok_emb, *gain0, *final_gain, *lm_head;
    const int32_t *tok_src;    // token buffer the embedding reads (B.TOK or B.PROMPT)
    int32_t n_part;            // LM-head partials to reduce
    int32_t draft_index;       // which draft the finalised token is
    int32_t e_min, e_max, g_min, g_max;
    int32_t mode;              // accept: 0 = round, 1 = prefill initialisation
    int32_t do_select;
    int32_t n_rows;            // rows of the stacked LM-head problem
    int32_t n_vtiles;
    double omega;
    // draft loop with the confidence break: the finalise kernel also posts (confidence, stamp) per sequence in
    // host memory that the device can write, so that the host sees it without a copy and a stream synchronisation
    volatile float *post_conf;          // [DEL_SEQ_MAX] device-visible host memory, or nullptr
    volatile uint32_t *post_stamp;      // [DEL_SEQ_MAX]
    // the break of Algorithm 1's draft loop is decided here: per sequence the threshold of its exit layer (0: the
    // sequence does not use draft-exiting), and where the decision (1: confidence below the threshold) is posted
    volatile uint32_t *post_stop;       // [DEL_SEQ_MAX]
    double exit_tau[DEL_SEQ_MAX];
    uint32_t stamp;
    // end of a round: the update kernel also posts every sequence's result (with the device error word as its
    // status) and a stamp there
    volatile int32_t *post_out;         // [DEL_SEQ_MAX][sizeof(del_round_out) / 4], or nullptr
    volatile uint32_t *post_done;       // [DEL_SEQ_MAX]
};

// rows of the stacked LM head: (seq, layer, slot) per row, plus per-sequence bookkeeping of the update.
// The launchers below take a HOST pointer and pass the plan by value in the kernel parameters.
struct UpdatePlan {
    int32_t n_seq, n_rows;
    // layers whose hidden rows go through the stacked LM head: all L, or (trimmed) only the candidates of the
    // selection e_min..e_max plus the last layer; lay_n of them, layer of index j = j < lay_n - 1 ? lay_first + j : L
    int32_t lay_first, lay_n;
    struct {
        int32_t seq, row0, g, E;     // rows row0 + (l-1)*(g+1) + i ; E = draft layer of the round
        int32_t n_valid_init;        // prefill: window width W (rows per layer = W)
        int32_t sampling;            // 1: accept length and last token come from B.SMP (speculative sampling)
        int32_t pad[2];
    } s[DEL_SEQ_MAX];
};

// 1-based layer of stacked-layer index j
__host__ __device__ inline int plan_layer(const UpdatePlan *up, int L, int j) { return j < up->lay_n - 1 ? up->lay_first + j : L; }

cudaError_t launch_embed(const CtlArgs &a, int m, cudaStream_t st, bool pdl);
cudaError_t launch_draft_finalize_embed(const CtlArgs &a, int m, bool embed_next, cudaStream_t st, bool pdl);
cudaError_t launch_prep_rows(const CtlArgs &a, const UpdatePlan *up, int n_rows, cudaStream_t st, bool pdl);
cudaError_t launch_shadow_reduce(const CtlArgs &a, const UpdatePlan *up, const float *pv, const int32_t *pi, const float *ps,
                                 int n_part, int pstride, int cstride, int row_base, int n_rows, cudaStream_t st, bool pdl);
cudaError_t launch_refresh_tau(const CtlArgs &a, int seq, cudaStream_t st);
cudaError_t launch_update(const CtlArgs &a, const UpdatePlan *up, void *out_dev, int n_seq, cudaStream_t st, bool pdl);
cudaError_t launch_select(const CtlArgs &a, const UpdatePlan *up, void *out_dev, int n_seq, cudaStream_t st, bool pdl);
cudaError_t launch_debug_logits(const CtlArgs &a, int layer, int seq, int slot, float *out_dev, cudaStream_t st);
cudaError_t launch_gather_kv(const CtlArgs &a, int layer, int seq, int pos, float *k_out, float *v_out, cudaStream_t st);

// Speculative sampling (sampling.cu).  One entry per sequence that samples in this launch.
struct SampleSeq {
    int32_t seq, slot, g, pad;   // slot: the draft index (draft kernel); g: drafts of the round (verify kernel)
    int64_t pos0;                // committed positions T: draft i is the token at position T + 1 + i
    double inv_T, top_p;
    unsigned long long seed;
};
struct SampleArgs {
    Dims D;
    Buffers B;
    int32_t n, pad;
    SampleSeq s[DEL_SEQ_MAX];
};
// draft i of every listed sequence: filtered distribution of its exit-head row, token drawn, stored as draft i
cudaError_t launch_sample_draft(const SampleArgs &a, cudaStream_t st, bool pdl);
// filtered-distribution statistics of the target rows 0..g of every listed sequence
cudaError_t launch_sample_stats(const SampleArgs &a, int max_rows, cudaStream_t st, bool pdl);
// acceptance tests and the token that ends the round (or, with g = 0 and pos0 = n_prompt - 1, the first token)
cudaError_t launch_sample_verify(const SampleArgs &a, cudaStream_t st, bool pdl);
// test hook: one (target, draft) pair of logit rows in device memory -> out[0..2] = drafted token, accepted?, last
// token; prob[0..1] = filtered q(x), p(x); stat[0..1] = RowStat of q, p
cudaError_t launch_sample_probe(const float *p_logits, const float *q_logits, int V, double inv_T, double top_p, double u_draft,
                                double u_accept, double u_final, int32_t *out, double *prob, RowStat *stat, cudaStream_t st);
int sample_max_vocab();

// Stacked LM head on tcgen05 / TMEM with fused arg-max (lmhead_tc.cu).  The tensor maps are 128-byte
// opaque blobs (CUtensorMap) kept by the host context.
int lmhead_tc_make_map(void *map_out, const void *base, uint64_t rows, uint64_t d, uint32_t box_rows);
int lmhead_tc_vtiles(int V);
// sel (may be null): stacked rows [row_lo, row_lo + n) whose normalised logits are also stored, row r at dst[(r - row_lo) * V]
struct LogitSel { int32_t row_lo, n; float *dst; };
cudaError_t launch_lmhead_tc(const void *map_x, const void *map_w, float *part_v, int32_t *part_i, float *part_s,
                             const float *row_scale, int n_rows, int V, int d, int32_t *err, const LogitSel *sel, int n_sel,
                             int n_sms, cudaStream_t st, bool pdl);

// Prompt prefill on tcgen05 (prefill_tc.cu): tiled GEMMs over up to PF_ROWS prompt positions of one sequence
// with the layer's element-wise work fused into the epilogues.  All buffers hold PF_ROWS rows.
#define PF_ROWS 512
enum { PF_QKV = 0, PF_OPROJ = 1, PF_GATEUP = 2, PF_DOWN = 3 };
struct PfArgs {
    Dims D;
    int32_t M, K;              // valid rows of the chunk, in-features of this GEMM
    int32_t n_ntiles;          // output tiles of this GEMM (prefill_tc_ntiles)
    int32_t n_ssp;             // partial sums of squares per row (= output tiles of a d-wide GEMM)
    int32_t layer, seq, pos0;  // 1-based layer; the rows are positions pos0 .. pos0 + M - 1 of sequence seq
    float *H;                  // [PF_ROWS][d] residual stream, updated in place
    bf16 *XS, *XSL;            // [PF_ROWS][d] h * attention-norm gain (high / low part): input of QKV, written by DOWN
    float *SSP;                // [PF_ROWS][n_ssp] sums of squares of h per output tile of DOWN (QKV's 1/rms)
    bf16 *Q, *QL, *ATT, *ATTL; // [PF_ROWS][nh * hd] queries, attention output (each as high / low part)
    bf16 *XM, *XML;            // [PF_ROWS][d] h_mid * ffn-norm gain (high / low part), written by OPROJ
    float *SSPM;               // [PF_ROWS][n_ssp]
    bf16 *ACT, *ACTL;          // [PF_ROWS][F] (high / low part)
    const bf16 *gain;          // OPROJ: ffn-norm gain; DOWN: the next layer's attention-norm gain
    bf16 *KP, *VP;             // paged cache
    const int32_t *PT;
    const float *rope_cos, *rope_sin;
    int32_t *err;
    // rows at positions >= win0 belong to the window that seeds the acceptance statistics: their hidden state
    // after every layer is also stored in the hidden stack (slot = position - win0)
    float *stackH;
    int32_t win0;
    int32_t bn_narrow;         // tile width of O-proj and down (prefill_tc_narrow)
};
int prefill_tc_ntiles(int epi, const Dims &D);
int prefill_tc_narrow(const Dims &D);          // tile width of O-proj and down for this shape
int prefill_tc_nssp(const Dims &D);            // partial sums of squares per row (one per 128 columns)

// Causal attention of a prefill chunk (prefill_attn.cu): rows 0..M-1 of Q (positions pos0 + row of sequence seq)
// against the paged cache of `layer` (which already holds the chunk's own keys and values) -> ATT.
struct PfAttnArgs {
    Dims D;
    const bf16 *Q, *QL;        // [M][nh * hd] queries, high and low part
    bf16 *ATT, *ATTL;          // [M][nh * hd] output, high and low part
    const bf16 *KP, *VP;
    const int32_t *PT;
    int32_t M, layer, seq, pos0;
};
cudaError_t launch_prefill_attention(const PfAttnArgs &a, cudaStream_t st, bool pdl);
// The same on tcgen05 / TMEM / TMA (prefill_attn_tc.cu), for head dimension 128.  map_qh / map_ql: the chunk's query
// buffers (lmhead_tc_make_map, boxes of 128 rows); map_k / map_v: 5-d maps of the paged cache.
bool prefill_attention_tc_supported(const Dims &D);
int prefill_attention_tc_make_maps(void *map_k, void *map_v, const void *k_pages, const void *v_pages, const Dims &D, int n_pages);
cudaError_t launch_prefill_attention_tc(const void *map_qh, const void *map_ql, const void *map_k, const void *map_v,
                                        const PfAttnArgs &a, int32_t *err, cudaStream_t st, bool pdl);
cudaError_t launch_prefill_gemm(int epi, const void *map_a, const void *map_a_lo, const void *map_b0, const void *map_b1,
                                const void *map_b2, const PfArgs &p, int n_sms, cudaStream_t st, bool pdl);
cudaError_t launch_prefill_embed(const PfArgs &p, const bf16 *tok_emb, const int32_t *prompt, const bf16 *gain0, cudaStream_t st);
