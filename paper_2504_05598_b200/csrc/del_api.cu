// Host side of libdel: the C ABI of include/del.h, the round scheduler (which rows go through which
// layers in which order), paged-KV bookkeeping and the launch sequence.  No device memory is allocated
// here: every buffer is carved out of the caller's workspace.
#include "../../include/del.h"
#include "kernels.h"

#include <algorithm>
#include <chrono>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

namespace {

constexpr int PLAN_RING = 192;
constexpr int CTR_RING = 4096;
constexpr int FLAG_PDL = 1, FLAG_GRAPH = 2, FLAG_TC = 4, FLAG_TIMING = 8, FLAG_ONECTA = 16, FLAG_NO_BULK_PREFILL = 32,
              FLAG_DECODE_ATTN_PREFILL = 64, FLAG_TRIM_ROWS = 128, FLAG_MMA_SYNC_PREFILL_ATTN = 256, FLAG_NO_WEIGHT_PREFETCH = 512;
enum { CLS_QKV = 0, CLS_ATTN, CLS_OPROJ, CLS_GATEUP, CLS_DOWN, CLS_LMHEAD, CLS_LMSTACK, CLS_OTHER, CLS_N };

struct SeqHost {
    bool active = false;
    int T = 0;               // committed positions
    int remaining = 0;       // tokens still to emit
    int E = 0, gamma = 0;    // choice for the next round
    int fixed_E = 0, fixed_gamma = 0;
    int fs_mode = 0;         // fixed E with the +-1 speculation-length controller
    int phase = 0;           // 0 idle, 1 drafted, 2 verified
    int cur_E = 0, cur_g = 0, cur_gamma = 0;
    int exit_mode = 0;       // 1: the draft loop stops on a low confidence (checked by the host per step)
    int cur_stopped = 0;
    double tau = 0.0;        // Eq. 3 threshold of the exit layer the next round uses
    double cur_tau = 0.0;
    std::vector<int> pages;
};

struct Carve {
    size_t off = 0;
    template <typename T> T *take(void *base, size_t n) {
        off = (off + 255) & ~(size_t)255;
        T *p = base ? reinterpret_cast<T *>(reinterpret_cast<char *>(base) + off) : nullptr;
        off += n * sizeof(T);
        return p;
    }
};

}  // namespace

struct del_ctx {
    del_shape sh;
    Dims D;
    Buffers B;
    int R_max = 0, n_vtiles = 0;
    const bf16 *tok_emb, *final_norm, *lm_head;
    std::vector<const bf16 *> attn_norm, wq, wk, wv, wo, ffn_norm, w_gate, w_up, w_down;
    cudaStream_t st = nullptr;
    int n_sms = 148;
    int flags = FLAG_PDL | FLAG_TC;
    bool in_round = false;               // the passes being enqueued belong to a decode round (not to a prefill)
    SeqHost seq[DEL_SEQ_MAX];
    std::vector<int> free_pages;
    std::vector<int32_t> pt_host;
    // plans
    int ctr_cur = 0;                     // next free slot of the tile-claim counter ring
    PassPlan *plan_host = nullptr;       // host ring of pass plans (passed to kernels by value)
    int plan_cur = 0;
    UpdatePlan *up_host = nullptr;                         // [2] pinned; passed to the kernels by value
    del_round_out *out_host = nullptr, *out_dev = nullptr; // [B]
    void *stage_host = nullptr;                            // small pinned scratch
    float *dbg_dev = nullptr;                              // [V] debug logits / kv rows
    alignas(64) unsigned char map_x[128], map_w[128];     // tensor maps of the stacked rows and of W_lm
    // bulk prefill on the tensor cores: chunk buffers in the workspace, tensor maps of them and of every layer's weights
    struct TMap { alignas(64) unsigned char b[128]; };
    PfArgs pf;                                            // buffer pointers (the per-launch fields are filled in later)
    TMap pf_xs, pf_att, pf_xm, pf_act;                    // activation buffers, high parts ...
    TMap pf_xsl, pf_attl, pf_xml, pf_actl;                // ... and low parts
    TMap pf_q, pf_ql, kv_k, kv_v;                         // tcgen05 prefill attention: query buffers, paged cache
    bool pfa_ok = false;
    std::vector<TMap> pf_wq, pf_wk, pf_wv, pf_wo, pf_wg, pf_wu, pf_wd;
    bool pf_ok = false;
    // mailbox of the draft loop's confidence check: pinned host memory that the finalise kernel writes directly
    volatile float *post_conf = nullptr;
    volatile uint32_t *post_stamp = nullptr;
    volatile uint32_t *post_stop = nullptr;               // the draft loop's break, decided by the finalise kernel
    volatile int32_t *post_out = nullptr;                 // round results posted by the update kernel
    volatile uint32_t *post_done = nullptr;
    uint32_t post_seq = 0;
    bool tc_ok = false;
    // speculative sampling per sequence slot (temperature <= 0: greedy); kept across prefills of the slot
    struct Sampling { double temperature = 0.0, top_p = 1.0; unsigned long long seed = 0; } samp[DEL_SEQ_MAX];
    int64_t launches = 0, h2d_bytes = 0, d2h_bytes = 0;
    // optional per-launch timing (FLAG_TIMING): events around every launch, summed per kernel class
    struct TimeRec { int cls, ev; double bytes; };
    std::vector<cudaEvent_t> ev_pool;
    std::vector<TimeRec> recs;
    int ev_used = 0, cur_cls = CLS_OTHER;
    double cur_bytes = 0.0;
    double cls_ms[CLS_N] = {0}, cls_bytes[CLS_N] = {0};
    int64_t cls_n[CLS_N] = {0};
    char err[256] = {0};
    cudaError_t last = cudaSuccess;
};

namespace {

size_t carve_all(const del_shape &s, void *base, Dims &D, Buffers &B, int &R_max, int &n_vtiles,
                 del_round_out **out_dev, float **dbg_dev, PfArgs *pf) {
    D.L = s.n_layers; D.d = s.d_model; D.nh = s.n_heads; D.nkv = s.n_kv_heads; D.hd = s.head_dim; D.F = s.d_ffn; D.V = s.vocab;
    D.B = s.max_batch;
    // slots of the hidden stack per sequence: what a round needs (g_max + 1 rows, the prefill window), raised to
    // a full pass so that the prefill streams the weights once per DEL_ROWS_MAX prompt positions
    D.S = std::max(std::max(s.g_max + 1, s.init_window), DEL_ROWS_MAX);
    D.max_seq = s.max_seq; D.page_size = s.page_size; D.pages_per_seq = s.max_seq / s.page_size;
    D.n_sst = s.d_model / 16;
    D.eps = s.rms_eps;
    R_max = s.n_layers * std::max(D.S, std::min(s.max_batch * (s.g_max + 1), DEL_ROWS_MAX));
    n_vtiles = (s.vocab + 127) / 128;
    const size_t L1 = (size_t)D.L + 1, BS = (size_t)D.B * D.S, qd = (size_t)D.nh * D.hd;
    Carve c;
    B.H = c.take<float>(base, L1 * BS * D.d);
    B.XS = c.take<bf16>(base, L1 * BS * D.d);
    B.XSL = c.take<bf16>(base, L1 * BS * D.d);
    B.SS = c.take<float>(base, L1 * BS * D.n_sst);
    B.XE = c.take<bf16>(base, BS * D.d);
    B.Q = c.take<bf16>(base, DEL_ROWS_MAX * qd);
    B.ATT = c.take<bf16>(base, DEL_ROWS_MAX * qd);
    B.ATTL = c.take<bf16>(base, DEL_ROWS_MAX * qd);
    B.HM = c.take<float>(base, (size_t)DEL_ROWS_MAX * D.d);
    B.XM = c.take<bf16>(base, (size_t)DEL_ROWS_MAX * D.d);
    B.XML = c.take<bf16>(base, (size_t)DEL_ROWS_MAX * D.d);
    B.SSM = c.take<float>(base, (size_t)DEL_ROWS_MAX * D.n_sst);
    B.ACT = c.take<bf16>(base, (size_t)DEL_ROWS_MAX * D.F);
    B.ACTL = c.take<bf16>(base, (size_t)DEL_ROWS_MAX * D.F);
    B.APO = c.take<float>(base, (size_t)DEL_ROWS_MAX * D.nh * 16 * D.hd);
    B.APML = c.take<float>(base, (size_t)DEL_ROWS_MAX * D.nh * 16 * 2);
    B.ACNT = c.take<int32_t>(base, (size_t)DEL_SEQ_MAX * D.nkv);
    B.LPV = c.take<float>(base, (size_t)1024 * DEL_ROWS_MAX);
    B.LPI = c.take<int32_t>(base, (size_t)1024 * DEL_ROWS_MAX);
    B.LPS = c.take<float>(base, (size_t)1024 * DEL_ROWS_MAX);
    B.RK = c.take<float>(base, (size_t)DEL_ROWS_MAX);
    B.TPV = c.take<float>(base, (size_t)(R_max + 128) * n_vtiles);
    B.TPI = c.take<int32_t>(base, (size_t)(R_max + 128) * n_vtiles);
    B.TPS = c.take<float>(base, (size_t)(R_max + 128) * n_vtiles);
    B.RS = c.take<float>(base, (size_t)(R_max + 128));
    B.SSE = c.take<float>(base, BS * D.n_sst);
    B.DCONF = c.take<float>(base, (size_t)D.B * (D.S + 1));
    B.SCONF = c.take<float>(base, (size_t)D.B * D.L * D.S);
    B.STCS = c.take<double>(base, (size_t)D.B * D.L);
    B.SFCS = c.take<double>(base, (size_t)D.B * D.L);
    B.TAU = c.take<double>(base, (size_t)D.B * D.L);
    B.QLOG = c.take<float>(base, (size_t)D.B * DEL_SAMPLE_ROWS * D.V);
    B.PLOG = c.take<float>(base, (size_t)D.B * DEL_SAMPLE_ROWS * D.V);
    B.QSTAT = c.take<RowStat>(base, (size_t)D.B * DEL_SAMPLE_ROWS);
    B.PSTAT = c.take<RowStat>(base, (size_t)D.B * DEL_SAMPLE_ROWS);
    B.SMP = c.take<SampleOut>(base, (size_t)D.B);
    B.PROMPT_ALL = c.take<int32_t>(base, (size_t)D.max_seq);
    B.XN = c.take<bf16>(base, (size_t)(R_max + 128) * D.d);
    B.SHADOW = c.take<int32_t>(base, (size_t)D.B * D.L * D.S);
    B.COUNTS = c.take<int32_t>(base, (size_t)D.B * D.L);
    B.TOK = c.take<int32_t>(base, (size_t)D.B * (D.S + 1));
    B.SC = c.take<double>(base, (size_t)D.B * D.L);
    B.ST = c.take<SeqState>(base, (size_t)D.B);
    B.TCNT = c.take<int32_t>(base, CTR_RING);
    *out_dev = c.take<del_round_out>(base, (size_t)D.B);
    B.ERR = c.take<int32_t>(base, 64);           // right behind the results: one copy brings both to the host
    *dbg_dev = c.take<float>(base, (size_t)std::max(D.V, 2 * D.nkv * D.hd));
    // chunk buffers of the bulk prefill (PF_ROWS prompt positions)
    PfArgs pfa;
    memset(&pfa, 0, sizeof(pfa));
    pfa.n_ssp = prefill_tc_nssp(D);
    pfa.H = c.take<float>(base, (size_t)PF_ROWS * D.d);
    pfa.XS = c.take<bf16>(base, (size_t)PF_ROWS * D.d);
    pfa.XSL = c.take<bf16>(base, (size_t)PF_ROWS * D.d);
    pfa.SSP = c.take<float>(base, (size_t)PF_ROWS * pfa.n_ssp);
    pfa.Q = c.take<bf16>(base, (size_t)PF_ROWS * qd);
    pfa.QL = c.take<bf16>(base, (size_t)PF_ROWS * qd);
    pfa.ATT = c.take<bf16>(base, (size_t)PF_ROWS * qd);
    pfa.ATTL = c.take<bf16>(base, (size_t)PF_ROWS * qd);
    pfa.XM = c.take<bf16>(base, (size_t)PF_ROWS * D.d);
    pfa.XML = c.take<bf16>(base, (size_t)PF_ROWS * D.d);
    pfa.SSPM = c.take<float>(base, (size_t)PF_ROWS * pfa.n_ssp);
    pfa.ACT = c.take<bf16>(base, (size_t)PF_ROWS * D.F);
    pfa.ACTL = c.take<bf16>(base, (size_t)PF_ROWS * D.F);
    if (pf) *pf = pfa;
    return (c.off + 255) & ~(size_t)255;
}

int validate(const del_shape *s) {
    if (!s) return DEL_EINVAL;
    if (s->n_layers < 2 || s->n_layers > 512) return DEL_EINVAL;
    if (s->head_dim != 64 && s->head_dim != 128) return DEL_EINVAL;
    if (s->n_heads < 1 || s->n_kv_heads < 1 || s->n_heads % s->n_kv_heads) return DEL_EINVAL;
    if (s->d_model < 256 || s->d_model % 32) return DEL_EINVAL;
    if (s->n_heads * s->head_dim < 256) return DEL_EINVAL;
    if (s->vocab < 32 || s->vocab % 32) return DEL_EINVAL;
    if (s->d_ffn < 256 || s->d_ffn % 16) return DEL_EINVAL;
    if (s->page_size != 16 || s->max_seq < 16 || s->max_seq % 16) return DEL_EINVAL;
    if (s->max_batch < 1 || s->max_batch > DEL_SEQ_MAX) return DEL_EINVAL;
    if (s->e_min < 1 || s->e_min > s->e_max || s->e_max >= s->n_layers) return DEL_EINVAL;
    if (s->g_min < 0 || s->g_min > s->g_max || s->g_max > DEL_MAX_GAMMA) return DEL_EINVAL;
    if (s->max_batch * (s->g_max + 1) > DEL_ROWS_MAX) return DEL_EINVAL;
    if (s->init_window < 1 || s->init_window > 32) return DEL_EINVAL;
    if (!(s->omega >= 0.0 && s->omega <= 1.0)) return DEL_EINVAL;
    if (s->n_pages < 1) return DEL_EINVAL;
    return DEL_OK;
}

int fail(del_ctx *c, cudaError_t e) {
    c->last = e;
    snprintf(c->err, sizeof(c->err), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return DEL_ECUDA;
}
#define CK(call)                                   \
    do {                                           \
        cudaError_t e__ = (call);                  \
        if (e__ != cudaSuccess) return fail(c, e__); \
    } while (0)
int timing_begin(del_ctx *c) {
    if (!(c->flags & FLAG_TIMING)) return -1;
    while ((int)c->ev_pool.size() < 2 * (c->ev_used + 1)) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) return -1;
        c->ev_pool.push_back(e);
    }
    const int i = c->ev_used++;
    cudaEventRecord(c->ev_pool[2 * i], c->st);
    return i;
}
void timing_end(del_ctx *c, int i) {
    if (i >= 0) {
        cudaEventRecord(c->ev_pool[2 * i + 1], c->st);
        c->recs.push_back({c->cur_cls, i, c->cur_bytes});
    }
    c->cur_cls = CLS_OTHER;
    c->cur_bytes = 0.0;
}
// call after the stream has been synchronised
void timing_collect(del_ctx *c) {
    for (const auto &r : c->recs) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, c->ev_pool[2 * r.ev], c->ev_pool[2 * r.ev + 1]) == cudaSuccess) {
            c->cls_ms[r.cls] += ms;
            c->cls_bytes[r.cls] += r.bytes;
            c->cls_n[r.cls] += 1;
        }
    }
    c->recs.clear();
    c->ev_used = 0;
}
#define LAUNCH(call)                               \
    do {                                           \
        const int t__ = timing_begin(c);           \
        cudaError_t e__ = (call);                  \
        if (e__ != cudaSuccess) return fail(c, e__); \
        ++c->launches;                             \
        timing_end(c, t__);                        \
    } while (0)
#define TAG(cls, bytes) (c->cur_cls = (cls), c->cur_bytes = (double)(bytes))

bool pdl(const del_ctx *c) { return (c->flags & FLAG_PDL) != 0; }

// ---- plan ring: plans are written into pinned host memory and copied to the device ring in one go
struct PlanBatch {
    del_ctx *c;
    int first, count = 0;
    explicit PlanBatch(del_ctx *ctx) : c(ctx), first(ctx->plan_cur) {}
    PassPlan *add(int *index) {
        *index = first + count;
        return &c->plan_host[first + count++];
    }
};

int plan_begin(del_ctx *c, int need) {
    if (need > PLAN_RING) return DEL_EINVAL;
    if (c->plan_cur + need > PLAN_RING) {
        c->plan_cur = 0;
    }
    return DEL_OK;
}
int plan_commit(del_ctx *c, const PlanBatch &b) {
    if (b.count == 0) return DEL_OK;
    c->plan_cur = b.first + b.count;
    return DEL_OK;
}

// rows of one pass: for every listed sequence `nrows` consecutive slots starting at slot0
struct RowSpec { int seq, slot0, nrows; };

void fill_plan(const del_ctx *c, PassPlan *p, const std::vector<RowSpec> &specs, bool prompt_tokens) {
    memset(p, 0, sizeof(*p));
    int m = 0, ns = 0;
    for (const RowSpec &r : specs) {
        const SeqHost &s = c->seq[r.seq];
        p->seg[ns++] = Segment{r.seq, m, r.nrows, s.T + r.slot0};
        for (int i = 0; i < r.nrows; ++i) {
            const int slot = r.slot0 + i, pos = s.T + slot;
            p->rows[m++] = RowDesc{r.seq, slot, pos, prompt_tokens ? pos : r.seq * (c->D.S + 1) + slot};
        }
    }
    p->m = m;
    p->n_seg = ns;
}

int ensure_pages(del_ctx *c, int sq, int positions) {
    SeqHost &s = c->seq[sq];
    const int need = (positions + 15) / 16;
    if (positions > c->D.max_seq) return DEL_ENOSPC;
    if ((int)s.pages.size() >= need) return DEL_OK;
    const int first_new = (int)s.pages.size();
    if ((int)c->free_pages.size() < need - first_new) return DEL_ENOSPC;
    while ((int)s.pages.size() < need) {
        const int pg = c->free_pages.back();
        c->free_pages.pop_back();
        c->pt_host[(size_t)sq * c->D.pages_per_seq + s.pages.size()] = pg;
        s.pages.push_back(pg);
    }
    // the source is pageable host memory: the copy is staged before the call returns
    CK(cudaMemcpyAsync(c->B.PT + (size_t)sq * c->D.pages_per_seq + first_new,
                       c->pt_host.data() + (size_t)sq * c->D.pages_per_seq + first_new,
                       sizeof(int32_t) * (need - first_new), cudaMemcpyHostToDevice, c->st));
    c->h2d_bytes += sizeof(int32_t) * (need - first_new);
    return DEL_OK;
}

void release_seq(del_ctx *c, int sq) {
    SeqHost &s = c->seq[sq];
    for (int pg : s.pages) c->free_pages.push_back(pg);
    s = SeqHost();
}

// next zeroed tile-claim counter; the ring is cleared (in stream order) each time it wraps
int32_t *next_counter(del_ctx *c) {
    if (c->ctr_cur == CTR_RING) {
        cudaMemsetAsync(c->B.TCNT, 0, sizeof(int32_t) * CTR_RING, c->st);
        c->ctr_cur = 0;
    }
    return c->B.TCNT + c->ctr_cur++;
}

GemmArgs gemm_base(del_ctx *c, int plan_idx, int layer) {
    GemmArgs a;
    memset(&a, 0, sizeof(a));
    a.tile_ctr = next_counter(c);
    a.ctas_per_sm = (c->flags & FLAG_ONECTA) ? 1 : 2;
    a.D = c->D;
    a.B = c->B;
    a.plan = c->plan_host[plan_idx];
    a.layer = layer;
    return a;
}

CtlArgs ctl_base(const del_ctx *c, int plan_idx) {
    CtlArgs a;
    memset(&a, 0, sizeof(a));
    a.D = c->D;
    a.B = c->B;
    if (plan_idx >= 0) a.plan = c->plan_host[plan_idx];
    a.tok_emb = c->tok_emb;
    a.gain0 = c->attn_norm[0];
    a.final_gain = c->final_norm;
    a.lm_head = c->lm_head;
    a.tok_src = c->B.TOK;
    a.e_min = c->sh.e_min; a.e_max = c->sh.e_max; a.g_min = c->sh.g_min; a.g_max = c->sh.g_max;
    a.omega = c->sh.omega;
    a.n_vtiles = c->n_vtiles;
    return a;
}

struct PassInfo {
    int plan_idx, m, n_seg, max_rows, max_kv;
};

PassInfo pass_info(const del_ctx *c, int plan_idx) {
    const PassPlan &p = c->plan_host[plan_idx];
    PassInfo pi{plan_idx, p.m, p.n_seg, 0, 0};
    for (int i = 0; i < p.n_seg; ++i) {
        pi.max_rows = std::max(pi.max_rows, p.seg[i].nrows);
        pi.max_kv = std::max(pi.max_kv, p.seg[i].pos0 + p.seg[i].nrows);
    }
    return pi;
}

// one decoder layer over the rows of a pass
int run_layer(del_ctx *c, const PassInfo &pi, int l, bool write_exit) {
    const Dims &D = c->D;
    const bool P = pdl(c);
    {
        GemmArgs a = gemm_base(c, pi.plan_idx, l);
        a.K = D.d;
        a.n_items = (D.nh + 2 * D.nkv) * (D.hd / 16);
        a.X = c->B.XS; a.XL = c->B.XSL;
        a.W0 = c->wq[l - 1]; a.W1 = c->wk[l - 1]; a.W2 = c->wv[l - 1];
        for (a.row0 = 0; a.row0 < pi.m; a.row0 += DEL_GEMM_ROWS) {
            if (a.row0) a.tile_ctr = next_counter(c);
            TAG(CLS_QKV, 2.0 * (D.nh + 2 * D.nkv) * D.hd * D.d);
            LAUNCH(launch_rowgemm(EPI_QKV, a, pi.m, c->n_sms, c->st, P));
        }
    }
    {
        AttnArgs a;
        memset(&a, 0, sizeof(a));
        a.D = D; a.B = c->B; a.plan = c->plan_host[pi.plan_idx]; a.layer = l;
        const int pages = (pi.max_kv + 15) / 16;
        const int R = pi.max_rows * (D.nh / D.nkv), n_mt = (R + 15) / 16;
        const int ns = attention_splits(pages, pi.n_seg * D.nkv, n_mt >= 3 ? 4 : n_mt, c->n_sms);
        a.n_splits = ns;
        a.max_rows = pi.max_rows;
        if (c->in_round) {          // what earlier rounds committed is final (the host has synchronised since)
            for (int i = 0; i < pi.n_seg; ++i) a.early_pos[i] = c->seq[c->plan_host[pi.plan_idx].seg[i].seq].T;
            // pages a warp walks: with more than two, attention's own later reads would queue behind the weights
            // (13B shape at 3 k context, 8 pages per warp: 2.3 % slower with the request than without)
            const int walkers = ns * (8 / (n_mt >= 3 ? 4 : n_mt));
            if (!(c->flags & FLAG_NO_WEIGHT_PREFETCH) && pages <= 2 * walkers) {
                // HBM idles while attention runs: the O-projection's weights go to L2 meanwhile (measured at the 7B
                // shape: + 0.9 % tokens/s; asking for the head of gate / up as well, 60 MB in all, gains nothing)
                a.pf.ptr[0] = c->wo[l - 1];
                a.pf.bytes[0] = (uint32_t)std::min((size_t)D.d * D.nh * D.hd * sizeof(bf16), (size_t)64 << 20);
                a.pf.n = 1;
            }
        }
        {
            double kvb = 0.0;
            const PassPlan &pp = c->plan_host[pi.plan_idx];
            for (int i = 0; i < pp.n_seg; ++i) kvb += 4.0 * (pp.seg[i].pos0 + pp.seg[i].nrows) * D.nkv * D.hd;
            TAG(CLS_ATTN, kvb);
        }
        LAUNCH(launch_attention(a, pi.n_seg, c->st, P));
    }
    {
        GemmArgs a = gemm_base(c, pi.plan_idx, l);
        a.K = D.nh * D.hd;
        a.n_items = D.d / 16;
        a.X = c->B.ATT; a.XL = c->B.ATTL;
        a.W0 = c->wo[l - 1];
        a.gain_a = c->ffn_norm[l - 1];
        for (a.row0 = 0; a.row0 < pi.m; a.row0 += DEL_GEMM_ROWS) {
            if (a.row0) a.tile_ctr = next_counter(c);
            TAG(CLS_OPROJ, 2.0 * D.d * D.nh * D.hd);
            LAUNCH(launch_rowgemm(EPI_OPROJ, a, pi.m, c->n_sms, c->st, P));
        }
    }
    {
        GemmArgs a = gemm_base(c, pi.plan_idx, l);
        a.K = D.d;
        a.n_items = D.F / 8;
        a.X = c->B.XM; a.XL = c->B.XML;
        a.W0 = c->w_gate[l - 1]; a.W1 = c->w_up[l - 1];
        for (a.row0 = 0; a.row0 < pi.m; a.row0 += DEL_GEMM_ROWS) {
            if (a.row0) a.tile_ctr = next_counter(c);
            TAG(CLS_GATEUP, 4.0 * D.F * D.d);
            LAUNCH(launch_rowgemm(EPI_GATEUP, a, pi.m, c->n_sms, c->st, P));
        }
    }
    {
        GemmArgs a = gemm_base(c, pi.plan_idx, l);
        a.K = D.F;
        a.n_items = D.d / 16;
        a.X = c->B.ACT; a.XL = c->B.ACTL;
        a.W0 = c->w_down[l - 1];
        a.gain_a = l < D.L ? c->attn_norm[l] : nullptr;
        a.gain_b = write_exit ? c->final_norm : nullptr;
        for (a.row0 = 0; a.row0 < pi.m; a.row0 += DEL_GEMM_ROWS) {
            if (a.row0) a.tile_ctr = next_counter(c);
            TAG(CLS_DOWN, 2.0 * D.d * D.F);
            LAUNCH(launch_rowgemm(EPI_DOWN, a, pi.m, c->n_sms, c->st, P));
        }
    }
    return DEL_OK;
}

// sequences of a call with their round parameters
struct Job { int seq, E, g; int stopped = 0; };

// ---- draft (a1-a3): g tokens per sequence, layers 1..E, exit head, arg-max, next embedding
int plans_needed_draft(const std::vector<Job> &jobs) {
    int gmax = 0;
    for (const Job &j : jobs) gmax = std::max(gmax, j.g);
    return gmax * ((int)jobs.size() + 2);
}

// plans of one draft step: all drafting rows, and per distinct exit layer the rows that go on beyond it
struct DraftStep { int full_idx = -1; std::vector<int> sub_idx; int samp_idx = -1; };

bool samples(const del_ctx *c, int sq) { return c->samp[sq].temperature > 0.0; }

SampleSeq sample_seq(const del_ctx *c, int sq, int slot, int g, int64_t pos0) {
    SampleSeq s;
    memset(&s, 0, sizeof(s));
    s.seq = sq; s.slot = slot; s.g = g; s.pos0 = pos0;
    s.inv_T = 1.0 / c->samp[sq].temperature;
    s.top_p = c->samp[sq].top_p;
    s.seed = c->samp[sq].seed;
    return s;
}

std::vector<int> exit_layers(const std::vector<Job> &jobs) {
    // distinct exit layers, ascending: the rows of a pass thin out as sequences reach their exit
    std::vector<int> Es;
    for (const Job &j : jobs) Es.push_back(j.E);
    std::sort(Es.begin(), Es.end());
    Es.erase(std::unique(Es.begin(), Es.end()), Es.end());
    return Es;
}

// `act`: the sequences that draft token i
void plan_draft_step(del_ctx *c, PlanBatch &pb, const std::vector<Job> &act, const std::vector<int> &Es, int i, DraftStep &st) {
    std::vector<RowSpec> full;
    for (const Job &j : act) full.push_back(RowSpec{j.seq, i, 1});
    fill_plan(c, pb.add(&st.full_idx), full, false);
    for (size_t e = 0; e < Es.size(); ++e) {
        if (e == 0) { st.sub_idx.push_back(st.full_idx); continue; }
        std::vector<RowSpec> sub;
        for (const Job &j : act)
            if (j.E >= Es[e]) sub.push_back(RowSpec{j.seq, i, 1});
        int idx = -1;
        if (!sub.empty()) fill_plan(c, pb.add(&idx), sub, false);
        st.sub_idx.push_back(idx);
    }
    // sequences that sample: their drawn token is embedded as the next row by a launch of its own
    std::vector<RowSpec> smp;
    for (const Job &j : act)
        if (samples(c, j.seq)) smp.push_back(RowSpec{j.seq, i + 1, 1});
    if (!smp.empty()) fill_plan(c, pb.add(&st.samp_idx), smp, false);
}

// layers 1..E of every drafting row, the exit head in one pass over W_lm, arg-max + confidence, next embedding
int launch_draft_step(del_ctx *c, const DraftStep &st, const std::vector<int> &Es, int i, uint32_t stamp = 0) {
    const bool P = pdl(c);
    const PassInfo full = pass_info(c, st.full_idx);
    if (i == 0) {
        CtlArgs ca = ctl_base(c, full.plan_idx);
        LAUNCH(launch_embed(ca, full.m, c->st, P));
    }
    int l = 1;
    for (size_t e = 0; e < Es.size(); ++e) {
        if (st.sub_idx[e] < 0) break;
        const PassInfo pi = pass_info(c, st.sub_idx[e]);
        for (; l <= Es[e]; ++l) {
            int rc = run_layer(c, pi, l, l == Es[e]);
            if (rc) return rc;
        }
    }
    GemmArgs a = gemm_base(c, full.plan_idx, 0);
    a.K = c->D.d;
    a.n_items = c->D.V / 16;
    a.X = c->B.XE;
    a.W0 = c->lm_head;
    if (st.samp_idx >= 0) a.logits_out = c->B.QLOG;      // the whole row of each draft is kept for the sampling kernels
    TAG(CLS_LMHEAD, 2.0 * c->D.V * c->D.d);
    LAUNCH(launch_rowgemm(EPI_LMHEAD, a, full.m, c->n_sms, c->st, P));
    CtlArgs ca = ctl_base(c, full.plan_idx);
    ca.n_part = rowgemm_lmhead_grid(a.n_items, full.m, c->n_sms, a.ctas_per_sm);
    if (stamp != 0 && c->post_conf != nullptr) {
        ca.post_conf = c->post_conf;
        ca.post_stamp = c->post_stamp;
        ca.post_stop = c->post_stop;
        for (int sq = 0; sq < c->D.B; ++sq) ca.exit_tau[sq] = c->seq[sq].exit_mode ? c->seq[sq].cur_tau : 0.0;
        ca.stamp = stamp;
    }
    LAUNCH(launch_draft_finalize_embed(ca, full.m, true, c->st, P));
    if (st.samp_idx >= 0) {
        // speculative sampling: the draft is drawn from the filtered exit-head distribution (it replaces the
        // arg-max token stored above) and embedded as the next row
        const PassPlan &sp = c->plan_host[st.samp_idx];
        SampleArgs sa;
        memset(&sa, 0, sizeof(sa));
        sa.D = c->D; sa.B = c->B;
        for (int r = 0; r < sp.m; ++r) {
            const int sq = sp.rows[r].seq;
            sa.s[sa.n++] = sample_seq(c, sq, i, 0, c->seq[sq].T);
        }
        LAUNCH(launch_sample_draft(sa, c->st, P));
        CtlArgs ce = ctl_base(c, st.samp_idx);
        LAUNCH(launch_embed(ce, sp.m, c->st, P));
    }
    return DEL_OK;
}

int enqueue_draft(del_ctx *c, const std::vector<Job> &jobs) {
    int gmax = 0;
    for (const Job &j : jobs) gmax = std::max(gmax, j.g);
    if (gmax == 0) return DEL_OK;
    int rc = plan_begin(c, plans_needed_draft(jobs));
    if (rc) return rc;
    PlanBatch pb(c);
    const std::vector<int> Es = exit_layers(jobs);
    std::vector<DraftStep> steps(gmax);
    for (int i = 0; i < gmax; ++i) {
        std::vector<Job> act;
        for (const Job &j : jobs)
            if (i < j.g) act.push_back(j);
        plan_draft_step(c, pb, act, Es, i, steps[i]);
    }
    rc = plan_commit(c, pb);
    if (rc) return rc;
    for (int i = 0; i < gmax; ++i) {
        rc = launch_draft_step(c, steps[i], Es, i);
        if (rc) return rc;
    }
    return DEL_OK;
}

// Draft loop of Algorithm 1 with its confidence break.  On entry job.g is the most tokens the sequence
// may draft; on return it is the number it kept, and job.stopped tells whether a low confidence ended
// the loop (the dropped token's pass through layers 1..E then serves as the verify phase's last row).
// The host reads each new token's confidence, so there is one synchronisation per step.
int draft_with_exit(del_ctx *c, std::vector<Job> &jobs) {
    std::vector<int> cap(jobs.size());
    int gmax = 0;
    for (size_t k = 0; k < jobs.size(); ++k) {
        cap[k] = jobs[k].g;
        jobs[k].g = 0;
        jobs[k].stopped = 0;
        gmax = std::max(gmax, cap[k]);
    }
    const std::vector<int> Es = exit_layers(jobs);
    float *conf_host = reinterpret_cast<float *>(c->stage_host) + 2048;
    std::vector<char> stop_dev(jobs.size(), 0);
    for (int i = 0; i < gmax; ++i) {
        std::vector<Job> act;
        std::vector<size_t> who;
        for (size_t k = 0; k < jobs.size(); ++k)
            if (!jobs[k].stopped && i < cap[k]) { act.push_back(jobs[k]); who.push_back(k); }
        if (act.empty()) break;
        int rc = plan_begin(c, (int)Es.size() + 2);
        if (rc) return rc;
        PlanBatch pb(c);
        DraftStep st;
        plan_draft_step(c, pb, act, Es, i, st);
        rc = plan_commit(c, pb);
        if (rc) return rc;
        const uint32_t stamp = ++c->post_seq ? c->post_seq : ++c->post_seq;     // never 0
        rc = launch_draft_step(c, st, Es, i, stamp);
        if (rc) return rc;
        // The finalise kernel posts each sequence's confidence in pinned host memory; the host polls the stamp
        // (about a second at most), so the next step can be enqueued while that kernel is still writing the
        // next embedding.  Without the mailbox, or if the stamp does not arrive: copy + synchronise.
        bool posted = c->post_conf != nullptr && !(c->flags & FLAG_TIMING);
        if (posted) {
            const auto t0 = std::chrono::steady_clock::now();
            for (size_t k : who) {
                const int sq = jobs[k].seq;
                if (!c->seq[sq].exit_mode) continue;
                while (c->post_stamp[sq] != stamp) {
                    if (std::chrono::steady_clock::now() - t0 > std::chrono::seconds(1)) { posted = false; break; }
                }
                if (!posted) break;
                conf_host[k] = c->post_conf[sq];
                stop_dev[k] = c->post_stop[sq] != 0;
                c->d2h_bytes += sizeof(float) + 2 * sizeof(uint32_t);
            }
        }
        if (!posted) {
            bool any = false;
            for (size_t k : who)
                if (c->seq[jobs[k].seq].exit_mode) {
                    CK(cudaMemcpyAsync(conf_host + k, c->B.DCONF + (size_t)jobs[k].seq * (c->D.S + 1) + i + 1, sizeof(float),
                                       cudaMemcpyDeviceToHost, c->st));
                    c->d2h_bytes += sizeof(float);
                    any = true;
                }
            if (any) CK(cudaStreamSynchronize(c->st));
        }
        for (size_t k : who) {
            const SeqHost &s = c->seq[jobs[k].seq];
            // Algorithm 1: break, token dropped.  The finalise kernel has taken the decision (same comparison: the fp32
            // confidence widened against the fp64 threshold); the copy fall-back repeats it here.
            const bool stop = posted ? stop_dev[k] : (s.exit_mode && (double)conf_host[k] < s.cur_tau);
            if (stop) jobs[k].stopped = 1;
            else jobs[k].g = i + 1;
        }
    }
    return DEL_OK;
}

// ---- a whole prompt (positions 0 .. n_pos-1 of sequence sq) through the tensor-core GEMMs: the KV cache of
// every position, and every layer's hidden state of the positions from win0 on (the window that seeds the
// statistics) into the hidden stack; chunks of PF_ROWS positions, attention in passes of DEL_ROWS_MAX query rows
int prefill_bulk(del_ctx *c, int sq, int n_pos, int win0) {
    const Dims &D = c->D;
    const bool P = pdl(c);
    for (int p0 = 0; p0 < n_pos; p0 += PF_ROWS) {
        PfArgs a = c->pf;
        a.M = std::min(PF_ROWS, n_pos - p0);
        a.seq = sq;
        a.pos0 = p0;
        a.stackH = c->B.H;
        a.win0 = win0;
        const bool has_window = p0 + a.M > win0;      // then the last layer is needed in full
        cudaError_t e = launch_prefill_embed(a, c->tok_emb, c->B.PROMPT_ALL, c->attn_norm[0], c->st);
        if (e != cudaSuccess) return fail(c, e);
        ++c->launches;
        for (int l = 1; l <= D.L; ++l) {
            a.layer = l;
            a.K = D.d;
            a.n_ntiles = prefill_tc_ntiles(PF_QKV, D);
            LAUNCH(launch_prefill_gemm(PF_QKV, c->pf_xs.b, c->pf_xsl.b, c->pf_wq[l - 1].b, c->pf_wk[l - 1].b, c->pf_wv[l - 1].b, a, c->n_sms, c->st, P));
            if (l == D.L && !has_window) break;       // of the last layer only the keys and values are needed
            if (!(c->flags & FLAG_DECODE_ATTN_PREFILL)) {
                // one flash-style pass over the chunk's rows and all keys up to each row's position
                PfAttnArgs pa;
                memset(&pa, 0, sizeof(pa));
                pa.D = D;
                pa.Q = a.Q; pa.QL = a.QL; pa.ATT = a.ATT; pa.ATTL = a.ATTL;
                pa.KP = c->B.KP; pa.VP = c->B.VP; pa.PT = c->B.PT;
                pa.M = a.M; pa.layer = l; pa.seq = sq; pa.pos0 = p0;
                if (c->pfa_ok && !(c->flags & FLAG_MMA_SYNC_PREFILL_ATTN))
                    LAUNCH(launch_prefill_attention_tc(c->pf_q.b, c->pf_ql.b, c->kv_k.b, c->kv_v.b, pa, c->B.ERR, c->st, P));
                else
                    LAUNCH(launch_prefill_attention(pa, c->st, P));
            } else
            for (int r0 = 0; r0 < a.M; r0 += DEL_ROWS_MAX) {
                AttnArgs at;
                memset(&at, 0, sizeof(at));
                at.D = D;
                at.B = c->B;
                at.B.Q = a.Q + (size_t)r0 * D.nh * D.hd;
                at.B.ATT = a.ATT + (size_t)r0 * D.nh * D.hd;
                at.B.ATTL = a.ATTL + (size_t)r0 * D.nh * D.hd;
                const int nr = std::min(DEL_ROWS_MAX, a.M - r0);
                at.plan.m = nr;
                at.plan.n_seg = 1;
                at.plan.seg[0] = Segment{sq, 0, nr, p0 + r0};
                at.layer = l;
                const int pages = (p0 + r0 + nr + 15) / 16;
                const int R = nr * (D.nh / D.nkv), n_mt = (R + 15) / 16;
                at.n_splits = attention_splits(pages, D.nkv, n_mt >= 3 ? 4 : n_mt, c->n_sms);
                at.max_rows = nr;
                LAUNCH(launch_attention(at, 1, c->st, P));
            }
            a.K = D.nh * D.hd;
            a.n_ntiles = prefill_tc_ntiles(PF_OPROJ, D);
            a.gain = c->ffn_norm[l - 1];
            LAUNCH(launch_prefill_gemm(PF_OPROJ, c->pf_att.b, c->pf_attl.b, c->pf_wo[l - 1].b, nullptr, nullptr, a, c->n_sms, c->st, P));
            a.K = D.d;
            a.n_ntiles = prefill_tc_ntiles(PF_GATEUP, D);
            LAUNCH(launch_prefill_gemm(PF_GATEUP, c->pf_xm.b, c->pf_xml.b, c->pf_wg[l - 1].b, c->pf_wu[l - 1].b, nullptr, a, c->n_sms, c->st, P));
            a.K = D.F;
            a.n_ntiles = prefill_tc_ntiles(PF_DOWN, D);
            a.gain = l < D.L ? c->attn_norm[l] : nullptr;      // the next layer's attention norm
            LAUNCH(launch_prefill_gemm(PF_DOWN, c->pf_act.b, c->pf_actl.b, c->pf_wd[l - 1].b, nullptr, nullptr, a, c->n_sms, c->st, P));
        }
    }
    return DEL_OK;
}

// ---- verify (a4-a5)
int enqueue_verify(del_ctx *c, const std::vector<Job> &jobs) {
    int rc = plan_begin(c, (int)jobs.size() + 2);
    if (rc) return rc;
    PlanBatch pb(c);
    std::vector<int> Es;
    for (const Job &j : jobs) Es.push_back(j.E);
    std::sort(Es.begin(), Es.end());
    Es.erase(std::unique(Es.begin(), Es.end()), Es.end());
    // segment k covers layers (Es[k-1], Es[k]] ; the last one (Es.back(), L]
    std::vector<int> idx(Es.size() + 1);
    std::vector<int> embed_rows;
    for (size_t k = 0; k <= Es.size(); ++k) {
        const int l_first = k == 0 ? 1 : Es[k - 1] + 1;
        std::vector<RowSpec> specs;
        for (const Job &j : jobs) {
            // a sequence whose draft loop stopped on a low confidence already has row g through layer E
            if (l_first <= j.E) { if (!j.stopped) specs.push_back(RowSpec{j.seq, j.g, 1}); }
            else specs.push_back(RowSpec{j.seq, 0, j.g + 1});
        }
        idx[k] = -1;
        if (!specs.empty()) fill_plan(c, pb.add(&idx[k]), specs, false);
    }
    // sequences that drafted nothing still need their input token embedded
    int embed_idx = -1;
    {
        std::vector<RowSpec> specs;
        for (const Job &j : jobs)
            if (j.g == 0 && !j.stopped) specs.push_back(RowSpec{j.seq, 0, 1});
        if (!specs.empty()) fill_plan(c, pb.add(&embed_idx), specs, false);
    }
    rc = plan_commit(c, pb);
    if (rc) return rc;
    if (embed_idx >= 0) {
        CtlArgs ca = ctl_base(c, embed_idx);
        LAUNCH(launch_embed(ca, c->plan_host[embed_idx].m, c->st, pdl(c)));
    }
    int l = 1;
    for (size_t k = 0; k <= Es.size(); ++k) {
        const int l_last = k < Es.size() ? Es[k] : c->D.L;
        if (idx[k] < 0) { l = l_last + 1; continue; }
        const PassInfo pi = pass_info(c, idx[k]);
        for (; l <= l_last; ++l) {
            rc = run_layer(c, pi, l, false);
            if (rc) return rc;
        }
    }
    return DEL_OK;
}

// ---- speculative sampling at the end of a round (Sec. 2): logits of the target's rows (one more pass over
// W_lm per sampling sequence, on the normalised rows the stacked head already prepared), their filtered
// distributions, the acceptance tests and the last token.  mode 1 (prefill): only the first token is drawn,
// from the row of the last prompt position.
// first stacked row and number of rows of the target (last layer) of sequence u of an update
void target_rows(const del_ctx *c, const UpdatePlan *up, int u, int g, int mode, int W, size_t &row, int &m) {
    const int per = mode ? W : g + 1;
    m = mode ? 1 : g + 1;
    (void)c;
    row = (size_t)up->s[u].row0 + (size_t)(up->lay_n - 1) * per + (mode ? W - 1 : 0);
}

int enqueue_sampling(del_ctx *c, const std::vector<Job> &jobs, const UpdatePlan *up, int mode, int W, bool have_logits) {
    std::vector<int> who;
    for (size_t u = 0; u < jobs.size(); ++u)
        if (samples(c, jobs[u].seq)) who.push_back((int)u);
    if (who.empty()) return DEL_OK;
    const bool P = pdl(c);
    std::vector<int> pidx(who.size(), -1);
    if (!have_logits) {
        int rc = plan_begin(c, (int)who.size());
        if (rc) return rc;
        PlanBatch pb(c);
        for (size_t k = 0; k < who.size(); ++k) {
            PassPlan *p = pb.add(&pidx[k]);
            memset(p, 0, sizeof(*p));
            p->m = mode ? 1 : jobs[who[k]].g + 1;
        }
        rc = plan_commit(c, pb);
        if (rc) return rc;
    }
    SampleArgs sa;
    memset(&sa, 0, sizeof(sa));
    sa.D = c->D; sa.B = c->B;
    int max_rows = 0;
    for (size_t k = 0; k < who.size(); ++k) {
        const Job &j = jobs[who[k]];
        size_t row;
        int m;
        target_rows(c, up, who[k], j.g, mode, W, row, m);
        if (!have_logits) {
            // the stacked head did not keep the target's logits (streaming head): one more pass over W_lm
            GemmArgs a = gemm_base(c, pidx[k], 0);
            a.K = c->D.d;
            a.n_items = c->D.V / 16;
            a.X = c->B.XN + row * c->D.d;
            a.W0 = c->lm_head;
            a.x_by_row = 1;
            a.row_scale = c->B.RS + row;
            a.logits_out = c->B.PLOG + (size_t)j.seq * DEL_SAMPLE_ROWS * c->D.V;
            TAG(CLS_LMHEAD, 2.0 * c->D.V * c->D.d);
            LAUNCH(launch_rowgemm(EPI_LMHEAD, a, m, c->n_sms, c->st, P));
        }
        sa.s[sa.n++] = sample_seq(c, j.seq, 0, mode ? 0 : j.g, mode ? c->seq[j.seq].T - 1 : c->seq[j.seq].T);
        max_rows = std::max(max_rows, m);
    }
    LAUNCH(launch_sample_stats(sa, max_rows, c->st, P));
    LAUNCH(launch_sample_verify(sa, c->st, P));
    return DEL_OK;
}

// ---- stacked LM head + arg-max over all layers' hidden rows (a6), then accept / counts (a7-a8)
int enqueue_update(del_ctx *c, const std::vector<Job> &jobs, int mode, int W, bool do_select, uint32_t post_stamp = 0) {
    UpdatePlan *up = &c->up_host[0];
    memset(up, 0, sizeof(*up));
    // rows of the stacked head: every layer, or only the layers the selection can pick plus the last one
    const bool trim = (c->flags & FLAG_TRIM_ROWS) != 0;
    up->lay_first = trim ? c->sh.e_min : 1;
    up->lay_n = trim ? c->sh.e_max - c->sh.e_min + 2 : c->D.L;
    int rows = 0;
    for (const Job &j : jobs) {
        auto &e = up->s[up->n_seq++];
        e.seq = j.seq; e.row0 = rows; e.g = j.g; e.E = j.E; e.n_valid_init = W;
        e.sampling = samples(c, j.seq) ? 1 : 0;
        rows += up->lay_n * (mode ? W : j.g + 1);
    }
    up->n_rows = rows;
    if (rows > c->R_max) return DEL_EINVAL;
    const bool P = pdl(c);
    CtlArgs ca = ctl_base(c, -1);
    ca.mode = mode;
    ca.n_rows = rows;
    if (post_stamp != 0 && c->post_out != nullptr) {
        ca.post_out = c->post_out;
        ca.post_done = c->post_done;
        ca.stamp = post_stamp;
    }
    LAUNCH(launch_prep_rows(ca, up, rows, c->st, P));
    if ((c->flags & FLAG_TC) && c->tc_ok) {
        // one pass over W_lm on the tensor cores, arg-max fused; partials [row][vocabulary tile]
        const int nvt = lmhead_tc_vtiles(c->D.V);
        TAG(CLS_LMSTACK, 2.0 * c->D.V * c->D.d);
        // sequences that sample: the epilogue also stores the logits of the target's rows
        LogitSel sel[DEL_SEQ_MAX];
        int n_sel = 0;
        for (size_t u = 0; u < jobs.size(); ++u)
            if (samples(c, jobs[u].seq)) {
                size_t row;
                int m;
                target_rows(c, up, (int)u, jobs[u].g, mode, W, row, m);
                sel[n_sel++] = LogitSel{(int32_t)row, m, c->B.PLOG + (size_t)jobs[u].seq * DEL_SAMPLE_ROWS * c->D.V};
            }
        LAUNCH(launch_lmhead_tc(c->map_x, c->map_w, c->B.TPV, c->B.TPI, c->B.TPS, c->B.RS, rows, c->D.V, c->D.d, c->B.ERR,
                                sel, n_sel, c->n_sms, c->st, P));
        LAUNCH(launch_shadow_reduce(ca, up, c->B.TPV, c->B.TPI, c->B.TPS, nvt, 1, nvt, 0, rows, c->st, P));
        int rs = enqueue_sampling(c, jobs, up, mode, W, true);
        if (rs) return rs;
        ca.do_select = do_select;             // the selection runs at the end of the update kernel
        LAUNCH(launch_update(ca, up, c->out_dev, up->n_seq, c->st, P));
        return DEL_OK;
    }
    // streaming LM head in chunks of 64 stacked rows
    const int n_chunks = (rows + DEL_ROWS_MAX - 1) / DEL_ROWS_MAX;
    int rc = plan_begin(c, n_chunks);
    if (rc) return rc;
    PlanBatch pb(c);
    std::vector<int> pidx(n_chunks);
    for (int k = 0; k < n_chunks; ++k) {
        PassPlan *p = pb.add(&pidx[k]);
        memset(p, 0, sizeof(*p));
        p->m = std::min(DEL_ROWS_MAX, rows - k * DEL_ROWS_MAX);
    }
    rc = plan_commit(c, pb);
    if (rc) return rc;
    for (int k = 0; k < n_chunks; ++k) {
        const int m = c->plan_host[pidx[k]].m;
        GemmArgs a = gemm_base(c, pidx[k], 0);
        a.K = c->D.d;
        a.n_items = c->D.V / 16;
        a.X = c->B.XN + (size_t)k * DEL_ROWS_MAX * c->D.d;
        a.W0 = c->lm_head;
        a.x_by_row = 1;
        a.row_scale = c->B.RS + (size_t)k * DEL_ROWS_MAX;
        TAG(CLS_LMSTACK, 2.0 * c->D.V * c->D.d);
        LAUNCH(launch_rowgemm(EPI_LMHEAD, a, m, c->n_sms, c->st, P));
        const int n_part = rowgemm_lmhead_grid(a.n_items, m, c->n_sms, a.ctas_per_sm);
        LAUNCH(launch_shadow_reduce(ca, up, c->B.LPV, c->B.LPI, c->B.LPS, n_part, DEL_ROWS_MAX, 1, k * DEL_ROWS_MAX, m,
                                    c->st, P));
    }
    rc = enqueue_sampling(c, jobs, up, mode, W, false);
    if (rc) return rc;
    ca.do_select = do_select;
    LAUNCH(launch_update(ca, up, c->out_dev, up->n_seq, c->st, P));
    return DEL_OK;
}

int read_out(del_ctx *c) {
    // the results of all sequences and the device error word behind them, in one copy
    const size_t span = (size_t)(reinterpret_cast<const char *>(c->B.ERR) - reinterpret_cast<const char *>(c->out_dev)) + sizeof(int32_t);
    CK(cudaMemcpyAsync(c->out_host, c->out_dev, span, cudaMemcpyDeviceToHost, c->st));
    c->d2h_bytes += span;
    const int32_t *err_host = reinterpret_cast<const int32_t *>(reinterpret_cast<const char *>(c->out_host) + span - sizeof(int32_t));
    CK(cudaStreamSynchronize(c->st));
    timing_collect(c);
    if (*err_host != 0) {
        // a bounded device-side wait expired; clear the word so that the context stays usable
        snprintf(c->err, sizeof(c->err), "device wait expired (code %d)", *err_host);
        cudaMemsetAsync(c->B.ERR, 0, sizeof(int32_t), c->st);
        return DEL_ETIMEOUT;
    }
    return DEL_OK;
}

// thresholds of a sequence recomputed on the device from its statistics; the host copy of the
// threshold of the current exit layer follows
int refresh_tau(del_ctx *c, int sq) {
    CtlArgs ca = ctl_base(c, -1);
    cudaError_t e = launch_refresh_tau(ca, sq, c->st);
    if (e != cudaSuccess) return fail(c, e);
    CK(cudaStreamSynchronize(c->st));
    if (c->seq[sq].E >= 1) {
        double t = 0.0;
        CK(cudaMemcpy(&t, c->B.TAU + (size_t)sq * c->D.L + (c->seq[sq].E - 1), sizeof(double), cudaMemcpyDeviceToHost));
        c->seq[sq].tau = t;
    }
    return DEL_OK;
}

// threshold of an arbitrary layer (the caller fixed E itself); synchronises
double exit_threshold(del_ctx *c, int sq, int E) {
    double t = 0.0;
    if (cudaStreamSynchronize(c->st) != cudaSuccess) return 0.0;
    if (cudaMemcpy(&t, c->B.TAU + (size_t)sq * c->D.L + (E - 1), sizeof(double), cudaMemcpyDeviceToHost) != cudaSuccess) return 0.0;
    return t;
}

int clip_gamma(const SeqHost &s, int gamma) { return std::max(0, std::min(gamma, s.remaining - 1)); }

bool seq_ok(const del_ctx *c, int sq) { return c && sq >= 0 && sq < c->D.B; }

}  // namespace

// =====================================================================================  C ABI
extern "C" {

size_t del_workspace_bytes(const del_shape *shape) {
    if (validate(shape) != DEL_OK) return 0;
    Dims D; Buffers B; int R, nv; del_round_out *o; float *dbg;
    return carve_all(*shape, nullptr, D, B, R, nv, &o, &dbg, nullptr);
}

int del_init(del_ctx **out, const del_shape *shape, const del_weights *w, const del_kv *kv, void *workspace,
             size_t ws_bytes, void *cuda_stream) {
    if (!out || !w || !kv || !workspace) return DEL_EINVAL;
    int rc = validate(shape);
    if (rc) return rc;
    if (!w->tok_emb || !w->final_norm || !w->lm_head || !w->attn_norm || !w->wq || !w->wk || !w->wv || !w->wo ||
        !w->ffn_norm || !w->w_gate || !w->w_up || !w->w_down || !w->rope_cos || !w->rope_sin)
        return DEL_EINVAL;
    if (!kv->k_pages || !kv->v_pages || !kv->page_table) return DEL_EINVAL;
    if (ws_bytes < del_workspace_bytes(shape)) return DEL_ENOSPC;
    del_ctx *c = new (std::nothrow) del_ctx();
    if (!c) return DEL_ENOSPC;
    c->sh = *shape;
    carve_all(*shape, workspace, c->D, c->B, c->R_max, c->n_vtiles, &c->out_dev, &c->dbg_dev, &c->pf);
    c->B.KP = (bf16 *)kv->k_pages; c->B.VP = (bf16 *)kv->v_pages; c->B.PT = kv->page_table;
    c->B.rope_cos = w->rope_cos; c->B.rope_sin = w->rope_sin;
    c->tok_emb = (const bf16 *)w->tok_emb; c->final_norm = (const bf16 *)w->final_norm; c->lm_head = (const bf16 *)w->lm_head;
    const int L = shape->n_layers;
    auto grab = [&](std::vector<const bf16 *> &dst, const void *const *src) {
        dst.resize(L);
        for (int l = 0; l < L; ++l) {
            dst[l] = (const bf16 *)src[l];
            if (!dst[l]) return false;
        }
        return true;
    };
    if (!grab(c->attn_norm, w->attn_norm) || !grab(c->wq, w->wq) || !grab(c->wk, w->wk) || !grab(c->wv, w->wv) ||
        !grab(c->wo, w->wo) || !grab(c->ffn_norm, w->ffn_norm) || !grab(c->w_gate, w->w_gate) || !grab(c->w_up, w->w_up) ||
        !grab(c->w_down, w->w_down)) {
        delete c;
        return DEL_EINVAL;
    }
    c->st = (cudaStream_t)cuda_stream;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaHostAlloc((void **)&c->plan_host, sizeof(PassPlan) * PLAN_RING, cudaHostAllocDefault);
    if (e == cudaSuccess) e = cudaHostAlloc((void **)&c->up_host, sizeof(UpdatePlan) * 2, cudaHostAllocDefault);
    if (e == cudaSuccess) e = cudaHostAlloc((void **)&c->out_host, sizeof(del_round_out) * DEL_SEQ_MAX + 1024, cudaHostAllocDefault);
    if (e == cudaSuccess) e = cudaHostAlloc((void **)&c->stage_host, 1 << 16, cudaHostAllocDefault);
    if (e == cudaSuccess) {
        // mailbox for the draft loop's confidence check (device-writable pinned memory); optional
        void *mb = nullptr;
        const size_t mb_bytes = 4 * DEL_SEQ_MAX * sizeof(uint32_t) + DEL_SEQ_MAX * sizeof(del_round_out);
        if (cudaHostAlloc(&mb, mb_bytes, cudaHostAllocMapped) == cudaSuccess) {
            memset(mb, 0, mb_bytes);
            void *dp = nullptr;
            if (cudaHostGetDevicePointer(&dp, mb, 0) == cudaSuccess && dp == mb) {
                c->post_conf = reinterpret_cast<volatile float *>(mb);
                c->post_stamp = reinterpret_cast<volatile uint32_t *>(mb) + DEL_SEQ_MAX;
                c->post_done = reinterpret_cast<volatile uint32_t *>(mb) + 2 * DEL_SEQ_MAX;
                c->post_stop = reinterpret_cast<volatile uint32_t *>(mb) + 3 * DEL_SEQ_MAX;
                c->post_out = reinterpret_cast<volatile int32_t *>(reinterpret_cast<uint32_t *>(mb) + 4 * DEL_SEQ_MAX);
            } else {
                cudaFreeHost(mb);
            }
        } else {
            cudaGetLastError();
        }
    }
    // zero the workspace (counters, statistics) and the KV pages (stale bit patterns must stay finite)
    if (e == cudaSuccess) e = cudaMemsetAsync(workspace, 0, del_workspace_bytes(shape), c->st);
    const size_t kv_bytes = (size_t)shape->n_pages * L * shape->n_kv_heads * 16 * shape->head_dim * sizeof(bf16);
    if (e == cudaSuccess) e = cudaMemsetAsync(kv->k_pages, 0, kv_bytes, c->st);
    if (e == cudaSuccess) e = cudaMemsetAsync(kv->v_pages, 0, kv_bytes, c->st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->st);
    if (e != cudaSuccess) {
        del_destroy(c);
        return DEL_ECUDA;
    }
    c->tc_ok = (shape->d_model % 64 == 0) && lmhead_tc_vtiles(shape->vocab) <= 1024 &&   // partials one block reduces
               lmhead_tc_make_map(c->map_x, c->B.XN, (uint64_t)c->R_max + 128, (uint64_t)shape->d_model, 128) == 0 &&
               lmhead_tc_make_map(c->map_w, c->lm_head, (uint64_t)shape->vocab, (uint64_t)shape->d_model, 256) == 0;
    {
        // tensor maps of the bulk prefill: activations in boxes of 128 rows, weights of 256 (gate / up: 128)
        const uint64_t d = shape->d_model, qd = (uint64_t)shape->n_heads * shape->head_dim,
                       kvd = (uint64_t)shape->n_kv_heads * shape->head_dim, F = shape->d_ffn;
        bool ok = lmhead_tc_make_map(c->pf_xs.b, c->pf.XS, PF_ROWS, d, 128) == 0 &&
                  lmhead_tc_make_map(c->pf_att.b, c->pf.ATT, PF_ROWS, qd, 128) == 0 &&
                  lmhead_tc_make_map(c->pf_xm.b, c->pf.XM, PF_ROWS, d, 128) == 0 &&
                  lmhead_tc_make_map(c->pf_act.b, c->pf.ACT, PF_ROWS, F, 128) == 0 &&
                  lmhead_tc_make_map(c->pf_xsl.b, c->pf.XSL, PF_ROWS, d, 128) == 0 &&
                  lmhead_tc_make_map(c->pf_attl.b, c->pf.ATTL, PF_ROWS, qd, 128) == 0 &&
                  lmhead_tc_make_map(c->pf_xml.b, c->pf.XML, PF_ROWS, d, 128) == 0 &&
                  lmhead_tc_make_map(c->pf_actl.b, c->pf.ACTL, PF_ROWS, F, 128) == 0;
        auto maps = [&](std::vector<del_ctx::TMap> &dst, const std::vector<const bf16 *> &w, uint64_t rows, uint64_t cols, uint32_t box) {
            dst.resize(L);
            for (int l = 0; l < L && ok; ++l) ok = lmhead_tc_make_map(dst[l].b, w[l], rows, cols, box) == 0;
        };
        maps(c->pf_wq, c->wq, qd, d, 256);
        maps(c->pf_wk, c->wk, kvd, d, 256);
        maps(c->pf_wv, c->wv, kvd, d, 256);
        const uint32_t bn_narrow = (uint32_t)prefill_tc_narrow(c->D);
        maps(c->pf_wo, c->wo, d, qd, bn_narrow);
        maps(c->pf_wg, c->w_gate, F, d, 128);
        maps(c->pf_wu, c->w_up, F, d, 128);
        maps(c->pf_wd, c->w_down, d, F, bn_narrow);
        c->pf.bn_narrow = (int32_t)bn_narrow;
        c->pf_ok = ok;
        c->pfa_ok = ok && prefill_attention_tc_supported(c->D) &&
                    lmhead_tc_make_map(c->pf_q.b, c->pf.Q, PF_ROWS, qd, 128) == 0 &&
                    lmhead_tc_make_map(c->pf_ql.b, c->pf.QL, PF_ROWS, qd, 128) == 0 &&
                    prefill_attention_tc_make_maps(c->kv_k.b, c->kv_v.b, c->B.KP, c->B.VP, c->D, shape->n_pages) == 0;
        c->pf.D = c->D;
        c->pf.KP = c->B.KP; c->pf.VP = c->B.VP; c->pf.PT = c->B.PT;
        c->pf.rope_cos = c->B.rope_cos; c->pf.rope_sin = c->B.rope_sin;
        c->pf.err = c->B.ERR;
    }
    c->pt_host.assign((size_t)c->D.B * c->D.pages_per_seq, 0);
    for (int p = shape->n_pages - 1; p >= 0; --p) c->free_pages.push_back(p);
    *out = c;
    return DEL_OK;
}

void del_destroy(del_ctx *c) {
    if (!c) return;
    if (c->plan_host) cudaFreeHost(c->plan_host);
    if (c->up_host) cudaFreeHost(c->up_host);
    if (c->out_host) cudaFreeHost(c->out_host);
    if (c->stage_host) cudaFreeHost(c->stage_host);
    if (c->post_conf) cudaFreeHost(const_cast<float *>(c->post_conf));
    for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
    delete c;
}

int del_release(del_ctx *c, int sq) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    release_seq(c, sq);
    return DEL_OK;
}

int del_prefill(del_ctx *c, int sq, const int32_t *prompt, int n_prompt, int max_new_tokens, del_round_out *first_out) {
    if (!seq_ok(c, sq) || !prompt || n_prompt < 1 || max_new_tokens < 1) return DEL_EINVAL;
    c->in_round = false;
    for (int i = 0; i < n_prompt; ++i)
        if (prompt[i] < 0 || prompt[i] >= c->D.V) return DEL_EINVAL;
    if (n_prompt + max_new_tokens + c->sh.g_max + 1 > c->D.max_seq) return DEL_ENOSPC;
    release_seq(c, sq);
    SeqHost &s = c->seq[sq];
    int rc = ensure_pages(c, sq, n_prompt + 1);
    if (rc) { release_seq(c, sq); return rc; }
    CK(cudaMemcpyAsync(c->B.PROMPT_ALL, prompt, sizeof(int32_t) * n_prompt, cudaMemcpyHostToDevice, c->st));
    c->h2d_bytes += sizeof(int32_t) * n_prompt;
    SeqState st0;
    memset(&st0, 0, sizeof(st0));
    memcpy(c->stage_host, &st0, sizeof(st0));
    CK(cudaMemcpyAsync(c->B.ST + sq, c->stage_host, sizeof(SeqState), cudaMemcpyHostToDevice, c->st));
    const int S = c->D.S, W = std::min(c->sh.init_window, n_prompt);
    // chunks of <= S positions; the last chunk is exactly the window so that its hidden states stay
    // in slots 0..W-1 of the stack
    std::vector<std::pair<int, int>> chunks;
    // long prompts go through the tensor-core prefill as a whole; short ones through the decode kernels
    if (c->pf_ok && !(c->flags & FLAG_NO_BULK_PREFILL) && n_prompt - W >= 64) {
        rc = prefill_bulk(c, sq, n_prompt, n_prompt - W);
        if (rc) return rc;
    } else {
        for (int p0 = 0; p0 < n_prompt - W; p0 += S) chunks.push_back({p0, std::min(S, n_prompt - W - p0)});
        chunks.push_back({n_prompt - W, W});
    }
    s.T = 0;
    for (auto ch : chunks) {
        rc = plan_begin(c, 1);
        if (rc) return rc;
        PlanBatch pb(c);
        int idx;
        s.T = ch.first;                      // rows are addressed relative to the committed length
        fill_plan(c, pb.add(&idx), {RowSpec{sq, 0, ch.second}}, true);
        rc = plan_commit(c, pb);
        if (rc) return rc;
        CtlArgs ca = ctl_base(c, idx);
        ca.tok_src = c->B.PROMPT_ALL;
        LAUNCH(launch_embed(ca, ch.second, c->st, pdl(c)));
        const PassInfo pi = pass_info(c, idx);
        for (int l = 1; l <= c->D.L; ++l) {
            rc = run_layer(c, pi, l, false);
            if (rc) return rc;
        }
    }
    s.T = n_prompt;
    s.active = true;
    s.remaining = max_new_tokens;
    s.phase = 0;
    rc = enqueue_update(c, {Job{sq, 0, 0}}, 1, W, true);
    if (rc) return rc;
    rc = read_out(c);
    if (rc) return rc;
    const del_round_out &o = c->out_host[sq];
    s.remaining -= 1;
    s.E = o.next_E;
    s.gamma = o.next_gamma;
    s.tau = o.next_tau;
    if (first_out) {
        memset(first_out, 0, sizeof(*first_out));
        first_out->n_emitted = 1;
        first_out->tokens[0] = o.tokens[0];
        first_out->next_E = o.next_E;
        first_out->next_gamma = o.next_gamma;
        first_out->next_tau = o.next_tau;
    }
    return DEL_OK;
}

int del_draft(del_ctx *c, int sq, int E, int gamma) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    SeqHost &s = c->seq[sq];
    if (E < 1 || E >= c->D.L || gamma < 0 || gamma > c->sh.g_max) return DEL_EINVAL;
    if (!s.active || s.remaining < 1 || s.phase != 0) return DEL_ESTATE;
    c->in_round = true;
    const int g = clip_gamma(s, gamma);
    int rc = ensure_pages(c, sq, s.T + g + 1);
    if (rc) return rc;
    std::vector<Job> jobs{Job{sq, E, g}};
    s.cur_tau = s.exit_mode ? exit_threshold(c, sq, E) : 0.0;
    if (s.exit_mode) rc = draft_with_exit(c, jobs);
    else rc = enqueue_draft(c, jobs);
    if (rc) return rc;
    s.cur_E = E; s.cur_g = jobs[0].g; s.cur_stopped = jobs[0].stopped; s.cur_gamma = gamma; s.phase = 1;
    return DEL_OK;
}

int del_verify(del_ctx *c, int sq) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    SeqHost &s = c->seq[sq];
    if (!s.active || s.phase != 1) return DEL_ESTATE;
    c->in_round = true;
    int rc = enqueue_verify(c, {Job{sq, s.cur_E, s.cur_g, s.cur_stopped}});
    if (rc) return rc;
    s.phase = 2;
    return DEL_OK;
}

static void finish_round(del_ctx *c, int sq, del_round_out *dst, bool with_next) {
    SeqHost &s = c->seq[sq];
    const del_round_out &o = c->out_host[sq];
    s.T += o.n_emitted;
    s.remaining -= o.n_emitted;
    s.phase = 0;
    if (with_next) { s.E = o.next_E; s.gamma = o.next_gamma; s.tau = o.next_tau; }
    if (dst) {
        *dst = o;
        dst->E = s.cur_E; dst->gamma = s.cur_gamma; dst->g = s.cur_g;
        dst->status = 0;
        dst->stopped = s.cur_stopped;
        dst->tau = s.cur_tau;
        if (!with_next) { dst->next_E = 0; dst->next_gamma = 0; dst->next_tau = 0.0; }
    }
}

int del_layer_accept(del_ctx *c, int sq, del_round_out *out) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    SeqHost &s = c->seq[sq];
    if (!s.active || s.phase != 2) return DEL_ESTATE;
    int rc = enqueue_update(c, {Job{sq, s.cur_E, s.cur_g}}, 0, 0, false);
    if (rc) return rc;
    rc = read_out(c);
    if (rc) return rc;
    finish_round(c, sq, out, false);
    return DEL_OK;
}

int del_select(del_ctx *c, int sq, int32_t *E, int32_t *gamma) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    SeqHost &s = c->seq[sq];
    if (!s.active) return DEL_ESTATE;
    UpdatePlan *up = &c->up_host[1];
    memset(up, 0, sizeof(*up));
    up->n_seq = 1;
    up->s[0].seq = sq;
    up->s[0].g = s.cur_g;            // the +-1 controller looks at the round just accepted
    CtlArgs ca = ctl_base(c, -1);
    LAUNCH(launch_select(ca, up, c->out_dev, 1, c->st, pdl(c)));
    int rc = read_out(c);
    if (rc) return rc;
    s.E = c->out_host[sq].next_E;
    s.gamma = c->out_host[sq].next_gamma;
    s.tau = c->out_host[sq].next_tau;
    if (E) *E = s.E;
    if (gamma) *gamma = s.gamma;
    return DEL_OK;
}

int del_round(del_ctx *c, del_round_out *out) {
    if (!c || !out) return DEL_EINVAL;
    c->in_round = true;
    std::vector<Job> jobs;
    bool any_exit = false;
    for (int sq = 0; sq < c->D.B; ++sq) {
        SeqHost &s = c->seq[sq];
        memset(&out[sq], 0, sizeof(out[sq]));
        if (!s.active || s.remaining < 1) continue;
        if (s.phase != 0) return DEL_ESTATE;
        const int E = s.fixed_E > 0 ? s.fixed_E : s.E;
        const int gamma = (s.fixed_E > 0 && !s.fs_mode) ? s.fixed_gamma : s.gamma;
        // Algorithm 1: with draft-exiting the loop may run up to d_max tokens, otherwise gamma tokens
        const int g = clip_gamma(s, s.exit_mode ? c->sh.g_max : gamma);
        int rc = ensure_pages(c, sq, s.T + g + 1);
        if (rc) return rc;
        s.cur_E = E; s.cur_g = g; s.cur_gamma = gamma; s.cur_stopped = 0;
        s.cur_tau = s.exit_mode ? (s.fixed_E > 0 ? exit_threshold(c, sq, E) : s.tau) : 0.0;
        any_exit = any_exit || s.exit_mode;
        jobs.push_back(Job{sq, E, g});
    }
    if (jobs.empty()) return DEL_ESTATE;
    int rc = any_exit ? draft_with_exit(c, jobs) : enqueue_draft(c, jobs);
    if (rc) return rc;
    for (const Job &j : jobs) { c->seq[j.seq].cur_g = j.g; c->seq[j.seq].cur_stopped = j.stopped; }
    rc = enqueue_verify(c, jobs);
    if (rc) return rc;
    // The update kernel posts every sequence's result and a stamp in pinned host memory; polling that is a
    // shorter way home than a copy and a stream synchronisation.  Timing mode and the fall-back use the copy.
    const bool mailbox = c->post_out != nullptr && !(c->flags & FLAG_TIMING);
    const uint32_t stamp = ++c->post_seq ? c->post_seq : ++c->post_seq;
    rc = enqueue_update(c, jobs, 0, 0, true, mailbox ? stamp : 0);
    if (rc) return rc;
    bool posted = mailbox;
    if (posted) {
        const auto t0 = std::chrono::steady_clock::now();
        constexpr int NWORD = (int)(sizeof(del_round_out) / sizeof(int32_t));
        for (const Job &j : jobs) {
            while (c->post_done[j.seq] != stamp) {
                if (std::chrono::steady_clock::now() - t0 > std::chrono::seconds(2)) { posted = false; break; }
            }
            if (!posted) break;
            int32_t *dst = reinterpret_cast<int32_t *>(&c->out_host[j.seq]);
            for (int w = 0; w < NWORD; ++w) dst[w] = c->post_out[(size_t)j.seq * NWORD + w];
            c->d2h_bytes += sizeof(del_round_out);
            if (c->out_host[j.seq].status != 0) posted = false;      // let the copy path report and clear the error
        }
    }
    if (!posted) {
        rc = read_out(c);
        if (rc) return rc;
    }
    for (const Job &j : jobs) finish_round(c, j.seq, &out[j.seq], true);
    return DEL_OK;
}

static int set_policy(del_ctx *c, int sq, int E, int gamma, int fs) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    if (E > 0 && (E >= c->D.L || gamma < 0 || gamma > c->sh.g_max)) return DEL_EINVAL;
    if (fs && (E < 1 || gamma < 1)) return DEL_EINVAL;
    SeqHost &s = c->seq[sq];
    s.fixed_E = E > 0 ? E : 0;
    s.fixed_gamma = E > 0 ? gamma : 0;
    s.fs_mode = fs;
    if (fs) s.gamma = gamma;
    CK(cudaStreamSynchronize(c->st));
    SeqState st;
    CK(cudaMemcpy(&st, c->B.ST + sq, sizeof(st), cudaMemcpyDeviceToHost));
    st.fixed_E = s.fixed_E;
    st.fixed_gamma = s.fixed_gamma;
    st.fs_mode = fs;
    if (fs) st.gamma = gamma;
    CK(cudaMemcpy(c->B.ST + sq, &st, sizeof(st), cudaMemcpyHostToDevice));
    return DEL_OK;
}

int del_set_policy(del_ctx *c, int sq, int E, int gamma) { return set_policy(c, sq, E, gamma, 0); }
int del_set_policy_fs(del_ctx *c, int sq, int E, int gamma0) { return set_policy(c, sq, E, gamma0, 1); }

int del_get_stats(del_ctx *c, int sq, double *Sc, double *Sn, int32_t *E, int32_t *gamma) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    CK(cudaStreamSynchronize(c->st));
    if (Sc) CK(cudaMemcpy(Sc, c->B.SC + (size_t)sq * c->D.L, sizeof(double) * c->D.L, cudaMemcpyDeviceToHost));
    SeqState st;
    CK(cudaMemcpy(&st, c->B.ST + sq, sizeof(st), cudaMemcpyDeviceToHost));
    if (Sn) *Sn = st.Sn;
    if (E) *E = c->seq[sq].E;
    if (gamma) *gamma = c->seq[sq].gamma;
    return DEL_OK;
}

int del_set_stats(del_ctx *c, int sq, const double *Sc, double Sn, int32_t E, int32_t gamma) {
    if (!seq_ok(c, sq) || !Sc) return DEL_EINVAL;
    CK(cudaStreamSynchronize(c->st));
    CK(cudaMemcpy(c->B.SC + (size_t)sq * c->D.L, Sc, sizeof(double) * c->D.L, cudaMemcpyHostToDevice));
    SeqState st;
    CK(cudaMemcpy(&st, c->B.ST + sq, sizeof(st), cudaMemcpyDeviceToHost));
    st.Sn = Sn; st.E = E; st.gamma = gamma;
    CK(cudaMemcpy(c->B.ST + sq, &st, sizeof(st), cudaMemcpyHostToDevice));
    c->seq[sq].E = E;
    c->seq[sq].gamma = gamma;
    return refresh_tau(c, sq);
}

int del_set_exit_mode(del_ctx *c, int sq, int mode) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    c->seq[sq].exit_mode = mode ? 1 : 0;
    return DEL_OK;
}

int del_set_sampling(del_ctx *c, int sq, double temperature, double top_p, uint64_t seed) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    if (temperature > 0.0 && !(top_p > 0.0)) return DEL_EINVAL;
    if (temperature > 0.0 && (c->D.V > sample_max_vocab() || c->D.V % 4 != 0)) return DEL_EINVAL;
    if (c->seq[sq].phase != 0) return DEL_ESTATE;
    c->samp[sq].temperature = temperature > 0.0 ? temperature : 0.0;
    c->samp[sq].top_p = top_p;
    c->samp[sq].seed = seed;
    return DEL_OK;
}

int del_get_sample_info(del_ctx *c, int sq, int32_t *n_tests, int32_t *from_residual, float *q_x, float *p_x) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    SampleOut so;
    CK(cudaStreamSynchronize(c->st));
    CK(cudaMemcpy(&so, c->B.SMP + sq, sizeof(so), cudaMemcpyDeviceToHost));
    if (n_tests) *n_tests = so.n_tests;
    if (from_residual) *from_residual = so.from_residual;
    if (q_x) memcpy(q_x, so.q_x, sizeof(so.q_x));
    if (p_x) memcpy(p_x, so.p_x, sizeof(so.p_x));
    return DEL_OK;
}

int del_get_round_logits(del_ctx *c, int sq, int which, int row, float *out) {
    if (!seq_ok(c, sq) || !out || row < 0 || row >= DEL_SAMPLE_ROWS) return DEL_EINVAL;
    const float *src = (which ? c->B.PLOG : c->B.QLOG) + ((size_t)sq * DEL_SAMPLE_ROWS + row) * c->D.V;
    CK(cudaStreamSynchronize(c->st));
    CK(cudaMemcpy(out, src, sizeof(float) * c->D.V, cudaMemcpyDeviceToHost));
    return DEL_OK;
}

int del_sample_probe(del_ctx *c, const float *p_logits, const float *q_logits, int vocab, double temperature, double top_p,
                     double u_draft, double u_accept, double u_final, int32_t *out, double *prob, int32_t *stat) {
    if (!c || !p_logits || !q_logits || !out || !prob || vocab < 1 || vocab > c->D.V || vocab % 4 != 0 || !(temperature > 0.0) || !(top_p > 0.0))
        return DEL_EINVAL;
    // scratch: the two logit buffers of sequence 0 hold the rows, its statistics slots the results
    float *zp = c->B.PLOG, *zq = c->B.QLOG;
    int32_t *o_dev = reinterpret_cast<int32_t *>(c->B.SMP);
    double *pr_dev = reinterpret_cast<double *>(c->B.PSTAT);
    RowStat *st_dev = c->B.QSTAT;
    CK(cudaStreamSynchronize(c->st));
    CK(cudaMemcpy(zp, p_logits, sizeof(float) * vocab, cudaMemcpyHostToDevice));
    CK(cudaMemcpy(zq, q_logits, sizeof(float) * vocab, cudaMemcpyHostToDevice));
    cudaError_t e = launch_sample_probe(zp, zq, vocab, 1.0 / temperature, top_p, u_draft, u_accept, u_final, o_dev, pr_dev, st_dev, c->st);
    if (e != cudaSuccess) return fail(c, e);
    CK(cudaStreamSynchronize(c->st));
    CK(cudaMemcpy(out, o_dev, sizeof(int32_t) * 4, cudaMemcpyDeviceToHost));
    CK(cudaMemcpy(prob, pr_dev, sizeof(double) * 2, cudaMemcpyDeviceToHost));
    if (stat) {
        RowStat rs[2];
        CK(cudaMemcpy(rs, st_dev, sizeof(rs), cudaMemcpyDeviceToHost));
        for (int k = 0; k < 2; ++k) {
            stat[4 * k + 0] = (int32_t)rs[k].kstar;
            stat[4 * k + 1] = rs[k].tie_keep;
            stat[4 * k + 2] = rs[k].cnt_eq;
            stat[4 * k + 3] = 0;
        }
    }
    return DEL_OK;
}

int del_get_conf_stats(del_ctx *c, int sq, double *Stcs, double *Sfcs, double *tau) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    CK(cudaStreamSynchronize(c->st));
    const size_t off = (size_t)sq * c->D.L, nb = sizeof(double) * c->D.L;
    if (Stcs) CK(cudaMemcpy(Stcs, c->B.STCS + off, nb, cudaMemcpyDeviceToHost));
    if (Sfcs) CK(cudaMemcpy(Sfcs, c->B.SFCS + off, nb, cudaMemcpyDeviceToHost));
    if (tau) CK(cudaMemcpy(tau, c->B.TAU + off, nb, cudaMemcpyDeviceToHost));
    return DEL_OK;
}

int del_set_conf_stats(del_ctx *c, int sq, const double *Stcs, const double *Sfcs) {
    if (!seq_ok(c, sq) || !Stcs || !Sfcs) return DEL_EINVAL;
    CK(cudaStreamSynchronize(c->st));
    const size_t off = (size_t)sq * c->D.L, nb = sizeof(double) * c->D.L;
    CK(cudaMemcpy(c->B.STCS + off, Stcs, nb, cudaMemcpyHostToDevice));
    CK(cudaMemcpy(c->B.SFCS + off, Sfcs, nb, cudaMemcpyHostToDevice));
    return refresh_tau(c, sq);
}

int del_get_conf(del_ctx *c, int sq, float *shadow_conf, float *draft_conf) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    CK(cudaStreamSynchronize(c->st));
    const int L = c->D.L, S = c->D.S, G = c->sh.g_max + 1;
    if (shadow_conf) {
        std::vector<float> tmp((size_t)L * S);
        CK(cudaMemcpy(tmp.data(), c->B.SCONF + (size_t)sq * L * S, sizeof(float) * L * S, cudaMemcpyDeviceToHost));
        for (int l = 0; l < L; ++l)
            for (int i = 0; i < G; ++i) shadow_conf[l * G + i] = tmp[(size_t)l * S + i];
    }
    if (draft_conf)
        CK(cudaMemcpy(draft_conf, c->B.DCONF + (size_t)sq * (S + 1) + 1, sizeof(float) * G, cudaMemcpyDeviceToHost));
    return DEL_OK;
}

int del_get_window(del_ctx *c, int sq, int n_cols, int32_t *shadow, float *conf) {
    if (!seq_ok(c, sq) || n_cols < 1 || n_cols > c->D.S) return DEL_EINVAL;
    CK(cudaStreamSynchronize(c->st));
    const int L = c->D.L, S = c->D.S;
    if (shadow) {
        std::vector<int32_t> tmp((size_t)L * S);
        CK(cudaMemcpy(tmp.data(), c->B.SHADOW + (size_t)sq * L * S, sizeof(int32_t) * L * S, cudaMemcpyDeviceToHost));
        for (int l = 0; l < L; ++l)
            for (int i = 0; i < n_cols; ++i) shadow[l * n_cols + i] = tmp[(size_t)l * S + i];
    }
    if (conf) {
        std::vector<float> tmp((size_t)L * S);
        CK(cudaMemcpy(tmp.data(), c->B.SCONF + (size_t)sq * L * S, sizeof(float) * L * S, cudaMemcpyDeviceToHost));
        for (int l = 0; l < L; ++l)
            for (int i = 0; i < n_cols; ++i) conf[l * n_cols + i] = tmp[(size_t)l * S + i];
    }
    return DEL_OK;
}

int del_get_shadow(del_ctx *c, int sq, int32_t *shadow, int32_t *counts) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    CK(cudaStreamSynchronize(c->st));
    const int L = c->D.L, S = c->D.S, G = c->sh.g_max + 1;
    if (shadow) {
        std::vector<int32_t> tmp((size_t)L * S);
        CK(cudaMemcpy(tmp.data(), c->B.SHADOW + (size_t)sq * L * S, sizeof(int32_t) * L * S, cudaMemcpyDeviceToHost));
        for (int l = 0; l < L; ++l)
            for (int i = 0; i < G; ++i) shadow[l * G + i] = tmp[(size_t)l * S + i];
    }
    if (counts) CK(cudaMemcpy(counts, c->B.COUNTS + (size_t)sq * L, sizeof(int32_t) * L, cudaMemcpyDeviceToHost));
    return DEL_OK;
}

int del_get_drafts(del_ctx *c, int sq, int32_t *drafts) {
    if (!seq_ok(c, sq) || !drafts) return DEL_EINVAL;
    CK(cudaStreamSynchronize(c->st));
    if (c->sh.g_max > 0)
        CK(cudaMemcpy(drafts, c->B.TOK + (size_t)sq * (c->D.S + 1) + 1, sizeof(int32_t) * c->sh.g_max, cudaMemcpyDeviceToHost));
    return DEL_OK;
}

int del_force_token(del_ctx *c, int sq, int32_t token) {
    if (!seq_ok(c, sq) || token < 0 || token >= c->D.V) return DEL_EINVAL;
    CK(cudaStreamSynchronize(c->st));
    CK(cudaMemcpy(c->B.TOK + (size_t)sq * (c->D.S + 1), &token, sizeof(int32_t), cudaMemcpyHostToDevice));
    return DEL_OK;
}

int del_get_hidden(del_ctx *c, int sq, int layer, int row, float *out) {
    if (!seq_ok(c, sq) || !out || layer < 0 || layer > c->D.L || row < 0 || row >= c->D.S) return DEL_EINVAL;
    CK(cudaStreamSynchronize(c->st));
    const size_t sr = ((size_t)layer * c->D.B + sq) * c->D.S + row;
    CK(cudaMemcpy(out, c->B.H + sr * c->D.d, sizeof(float) * c->D.d, cudaMemcpyDeviceToHost));
    return DEL_OK;
}

int del_debug_logits(del_ctx *c, int sq, int layer, int row, float *out) {
    if (!seq_ok(c, sq) || !out || layer < 0 || layer > c->D.L || row < 0 || row >= c->D.S) return DEL_EINVAL;
    CtlArgs ca = ctl_base(c, -1);
    LAUNCH(launch_debug_logits(ca, layer, sq, row, c->dbg_dev, c->st));
    CK(cudaStreamSynchronize(c->st));
    CK(cudaMemcpy(out, c->dbg_dev, sizeof(float) * c->D.V, cudaMemcpyDeviceToHost));
    return DEL_OK;
}

int del_get_kv(del_ctx *c, int sq, int layer, int pos, float *k_out, float *v_out) {
    if (!seq_ok(c, sq) || layer < 1 || layer > c->D.L || pos < 0) return DEL_EINVAL;
    if (pos >= (int)c->seq[sq].pages.size() * 16) return DEL_EINVAL;
    const int n = c->D.nkv * c->D.hd;
    CtlArgs ca = ctl_base(c, -1);
    LAUNCH(launch_gather_kv(ca, layer, sq, pos, c->dbg_dev, c->dbg_dev + n, c->st));
    CK(cudaStreamSynchronize(c->st));
    if (k_out) CK(cudaMemcpy(k_out, c->dbg_dev, sizeof(float) * n, cudaMemcpyDeviceToHost));
    if (v_out) CK(cudaMemcpy(v_out, c->dbg_dev + n, sizeof(float) * n, cudaMemcpyDeviceToHost));
    return DEL_OK;
}

int del_debug_inject_error(del_ctx *c, int code) {
    if (!c || code == 0) return DEL_EINVAL;
    int32_t *src = reinterpret_cast<int32_t *>(c->stage_host) + 4096;     // pinned: the copy is stream-ordered
    *src = code;
    CK(cudaMemcpyAsync(c->B.ERR, src, sizeof(int32_t), cudaMemcpyHostToDevice, c->st));
    CK(cudaStreamSynchronize(c->st));
    return DEL_OK;
}

int del_committed_len(del_ctx *c, int sq) {
    if (!seq_ok(c, sq)) return DEL_EINVAL;
    return c->seq[sq].active ? c->seq[sq].T : DEL_ESTATE;
}

int64_t del_launch_count(const del_ctx *c) { return c ? c->launches : 0; }

int del_get_traffic(const del_ctx *c, int64_t *h2d_bytes, int64_t *d2h_bytes) {
    if (!c) return DEL_EINVAL;
    if (h2d_bytes) *h2d_bytes = c->h2d_bytes;
    if (d2h_bytes) *d2h_bytes = c->d2h_bytes;
    return DEL_OK;
}

int del_get_kernel_times(del_ctx *c, double *ms, int64_t *launches, double *bytes, int reset) {
    if (!c) return DEL_EINVAL;
    for (int i = 0; i < CLS_N; ++i) {
        if (ms) ms[i] = c->cls_ms[i];
        if (launches) launches[i] = c->cls_n[i];
        if (bytes) bytes[i] = c->cls_bytes[i];
        if (reset) { c->cls_ms[i] = 0; c->cls_n[i] = 0; c->cls_bytes[i] = 0; }
    }
    return DEL_OK;
}

int del_set_flags(del_ctx *c, int flags) {
    if (!c) return DEL_EINVAL;
    const int old = c->flags;
    c->flags = flags;
    return old;
}

const char *del_strerror(int code) {
    switch (code) {
        case DEL_OK: return "ok";
        case DEL_EINVAL: return "invalid argument or shape";
        case DEL_ENOSPC: return "out of KV pages, sequence length or workspace";
        case DEL_ESTATE: return "call order wrong for the sequence's state";
        case DEL_ETIMEOUT: return "a bounded device-side wait expired";
        case DEL_ECUDA: return "CUDA error (see del_last_cuda_error)";
    }
    return "unknown error";
}

const char *del_last_cuda_error(const del_ctx *c) { return c ? c->err : ""; }

}  // extern "C"
