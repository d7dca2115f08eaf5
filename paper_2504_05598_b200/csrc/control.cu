// Small kernels around the weight-streaming ones: token embedding, arg-max finalisation of the draft
// head, row preparation and arg-max reduction of the stacked LM head, prefix acceptance with the
// acceptance-statistics update, the (E, gamma) selection, and two test-only readers.
#include "../../include/del.h"
#include "kernels.h"

namespace {

constexpr int CTL_THREADS = 256;

__device__ __forceinline__ void write_embedding(const CtlArgs &a, int token, int seq, int slot) {
    // h^0 = embedding row; also the bf16 input of layer 1's attention norm and its partial sums of squares.
    // A thread owns 8 consecutive features; two neighbouring threads make one 16-feature partial.
    const int d = a.D.d;
    const bf16 *e = a.tok_emb + (size_t)token * d;
    const size_t sr = stack_row(a.D, 0, seq, slot);
    for (int o0 = 0; o0 < d; o0 += 2 * 8 * CTL_THREADS) {
        uint4 ev[2], gv[2];
        int o[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            o[r] = o0 + (r * CTL_THREADS + threadIdx.x) * 8;
            ev[r] = ldg_stream16_pred(e + o[r], o[r] < d);
            gv[r] = ldg_stream16_pred(a.gain0 + o[r], o[r] < d);
        }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const uint32_t ew[4] = {ev[r].x, ev[r].y, ev[r].z, ev[r].w}, gw[4] = {gv[r].x, gv[r].y, gv[r].z, gv[r].w};
            float h[8], ss = 0.f;
            uint32_t xs[4], xl[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                h[2 * q] = __uint_as_float(ew[q] << 16);
                h[2 * q + 1] = __uint_as_float(ew[q] & 0xffff0000u);
                split_bf16x2(h[2 * q] * __uint_as_float(gw[q] << 16), h[2 * q + 1] * __uint_as_float(gw[q] & 0xffff0000u), xs[q], xl[q]);
                ss += h[2 * q] * h[2 * q] + h[2 * q + 1] * h[2 * q + 1];
            }
            ss += __shfl_xor_sync(0xffffffffu, ss, 1);
            if (o[r] < d) {
                float4 *hp = reinterpret_cast<float4 *>(a.B.H + sr * d + o[r]);
                hp[0] = make_float4(h[0], h[1], h[2], h[3]);
                hp[1] = make_float4(h[4], h[5], h[6], h[7]);
                *reinterpret_cast<uint4 *>(a.B.XS + sr * d + o[r]) = make_uint4(xs[0], xs[1], xs[2], xs[3]);
                *reinterpret_cast<uint4 *>(a.B.XSL + sr * d + o[r]) = make_uint4(xl[0], xl[1], xl[2], xl[3]);
                if ((threadIdx.x & 1) == 0) a.B.SS[sr * a.D.n_sst + (o[r] >> 4)] = ss;
            }
        }
    }
}

__global__ void __launch_bounds__(CTL_THREADS) embed_kernel(const __grid_constant__ CtlArgs a) {
    pdl_launch();
    pdl_wait();
    const RowDesc rd = a.plan.rows[blockIdx.x];
    const int token = a.tok_src[rd.tok];
    write_embedding(a, token, rd.seq, rd.slot);
}

// block-wide arg-max with ties to the lowest index; result valid in thread 0
__device__ __forceinline__ void block_argmax(float &v, int &idx) {
    __shared__ float sv[CTL_THREADS / 32];
    __shared__ int si[CTL_THREADS / 32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float v2 = __shfl_xor_sync(0xffffffffu, v, o);
        const int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
        if (v2 > v || (v2 == v && i2 < idx)) { v = v2; idx = i2; }
    }
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = v; si[threadIdx.x >> 5] = idx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < CTL_THREADS / 32; ++w)
            if (sv[w] > v || (sv[w] == v && si[w] < idx)) { v = sv[w]; idx = si[w]; }
    }
}

// block-wide sum in a fixed order; result valid in thread 0
__device__ __forceinline__ float block_sum(float v) {
    __shared__ float ssum[CTL_THREADS / 32];
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) ssum[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
    if (threadIdx.x == 0)
        for (int w = 0; w < CTL_THREADS / 32; ++w) t += ssum[w];
    return t;
}

// Partials (maximum, index, exp sum) of one row reduced to the token and its confidence score (Sec. 4.4:
// the probability of the top-1 token) = 1 / sum_p s_p * exp2(k * (v_p - M)), M the overall maximum,
// k = log2(e) / rms of the row.  All partials are loaded once (up to PMAX per thread stay in registers).
// Results valid in thread 0.
constexpr int PMAX = 4;                              // CTL_THREADS * PMAX = 1024 partials
__device__ __forceinline__ void reduce_partials(const float *pv, const int32_t *pi, const float *ps, int n_part, size_t pstride,
                                                const float *kp, int &token, float &conf) {
    __shared__ float s_max;
    float vv[PMAX], sv[PMAX];
    int iv[PMAX];
#pragma unroll
    for (int q = 0; q < PMAX; ++q) {
        const int p = threadIdx.x + q * CTL_THREADS;
        const bool ok = p < n_part;
        vv[q] = ok ? ldg_cg_f32(pv + (size_t)p * pstride) : -INFINITY;
        sv[q] = ok ? ldg_cg_f32(ps + (size_t)p * pstride) : 0.f;
        iv[q] = ok ? pi[(size_t)p * pstride] : 0x7fffffff;
    }
    const float k = ldg_cg_f32(kp);
    float v = -INFINITY;
    int idx = 0x7fffffff;
#pragma unroll
    for (int q = 0; q < PMAX; ++q)
        if (vv[q] > v || (vv[q] == v && iv[q] < idx)) { v = vv[q]; idx = iv[q]; }
    block_argmax(v, idx);
    if (threadIdx.x == 0) s_max = v;
    __syncthreads();
    const float M = s_max;
    float acc = 0.f;
#pragma unroll
    for (int q = 0; q < PMAX; ++q) acc += sv[q] * exp2f(k * (vv[q] - M));
    const float total = block_sum(acc);
    token = idx;
    conf = 1.f / total;
}

// Draft head, last step: reduce the per-CTA arg-max partials of the streaming LM head into the draft
// token, store it, and write the embedding of that token as the next row of the sequence.
__global__ void __launch_bounds__(CTL_THREADS) draft_finalize_embed_kernel(const __grid_constant__ CtlArgs a, int embed_next) {
    __shared__ int s_tok;
    pdl_launch();
    pdl_wait();
    const int c = blockIdx.x;
    const RowDesc rd = a.plan.rows[c];
    int idx;
    float conf;
    reduce_partials(a.B.LPV + c, a.B.LPI + c, a.B.LPS + c, a.n_part, DEL_ROWS_MAX, a.B.RK + c, idx, conf);
    if (threadIdx.x == 0) {
        s_tok = idx;
        a.B.TOK[rd.seq * (a.D.S + 1) + rd.slot + 1] = idx;
        a.B.DCONF[rd.seq * (a.D.S + 1) + rd.slot + 1] = conf;
        if (a.post_conf != nullptr) {
            a.post_conf[rd.seq] = conf;
            a.post_stop[rd.seq] = (a.exit_tau[rd.seq] > 0.0 && (double)conf < a.exit_tau[rd.seq]) ? 1u : 0u;
            __threadfence_system();              // the confidence is in host memory before the stamp that announces it
            a.post_stamp[rd.seq] = a.stamp;
        }
    }
    __syncthreads();
    if (embed_next) write_embedding(a, s_tok, rd.seq, rd.slot + 1);
}

__device__ __forceinline__ bool locate_row(const UpdatePlan *up, int L, int mode, int rr, int &seq, int &layer, int &slot) {
    for (int u = 0; u < up->n_seq; ++u) {
        const int per = mode ? up->s[u].n_valid_init : up->s[u].g + 1;
        const int r = rr - up->s[u].row0;
        if (r >= 0 && r < per * up->lay_n) {
            seq = up->s[u].seq;
            const int j = r / per;
            layer = plan_layer(up, L, j);
            slot = r - j * per;
            return true;
        }
    }
    return false;
}

// Stacked LM head input: row (seq, layer, slot) of the hidden stack times the final norm's gain, as
// bf16.  The norm's 1/rms is a positive per-row scalar and cannot change the arg-max, so it is left out
// of the product; it is stored (times log2 e) for the confidence score, which does depend on it.
__global__ void __launch_bounds__(CTL_THREADS) prep_rows_kernel(const CtlArgs a, const __grid_constant__ UpdatePlan up_v) {
    const UpdatePlan *up = &up_v;
    pdl_launch();
    pdl_wait();
    int seq, layer, slot;
    if (!locate_row(up, a.D.L, a.mode, blockIdx.x, seq, layer, slot)) return;
    const int d = a.D.d;
    const float *h = a.B.H + stack_row(a.D, layer, seq, slot) * d;
    bf16 *x = a.B.XN + (size_t)blockIdx.x * d;
    float sq = 0.f;
    // 8 consecutive features per thread and step (d is a multiple of 32): two 16-byte loads of h, one of the gains
    for (int o = threadIdx.x * 8; o < d; o += CTL_THREADS * 8) {
        const uint4 h0 = ldg_act16(h + o), h1 = ldg_act16(h + o + 4);
        const uint4 gv = ldg_stream16_pred(a.final_gain + o, true);
        const float hv[8] = {__uint_as_float(h0.x), __uint_as_float(h0.y), __uint_as_float(h0.z), __uint_as_float(h0.w),
                             __uint_as_float(h1.x), __uint_as_float(h1.y), __uint_as_float(h1.z), __uint_as_float(h1.w)};
        const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w};
        uint32_t xo[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            xo[q] = pack_bf16(hv[2 * q] * __uint_as_float(gw[q] << 16), hv[2 * q + 1] * __uint_as_float(gw[q] & 0xffff0000u));
            sq += hv[2 * q] * hv[2 * q] + hv[2 * q + 1] * hv[2 * q + 1];
        }
        *reinterpret_cast<uint4 *>(x + o) = make_uint4(xo[0], xo[1], xo[2], xo[3]);
    }
    const float total = block_sum(sq);
    if (threadIdx.x == 0) a.B.RS[blockIdx.x] = rsqrtf(total / (float)d + a.D.eps) * 1.4426950408889634f;
}

// Reduce the vocabulary-tile partials of one stacked row into its shadow token.
__global__ void __launch_bounds__(CTL_THREADS) shadow_reduce_kernel(const CtlArgs a, const __grid_constant__ UpdatePlan up_v, const float *pv,
                                                                    const int32_t *pi, const float *ps, int n_part, int pstride,
                                                                    int cstride, int row_base) {
    const UpdatePlan *up = &up_v;
    pdl_launch();
    pdl_wait();
    const int c = blockIdx.x;
    int idx;
    float conf;
    reduce_partials(pv + (size_t)c * cstride, pi + (size_t)c * cstride, ps + (size_t)c * cstride, n_part, pstride,
                    a.B.RS + row_base + c, idx, conf);
    if (threadIdx.x == 0) {
        int seq, layer, slot;
        if (locate_row(up, a.D.L, a.mode, row_base + c, seq, layer, slot)) {
            a.B.SHADOW[((size_t)seq * a.D.L + (layer - 1)) * a.D.S + slot] = idx;
            a.B.SCONF[((size_t)seq * a.D.L + (layer - 1)) * a.D.S + slot] = conf;
        }
    }
}

// Eq. 3 for one layer: midpoint of the decayed mean confidences of matched and mismatched shadow tokens
// (a mean over no tokens counts as 1 for the matched and as 0 for the mismatched ones).
__device__ __forceinline__ double threshold(double Stcs, double Sc, double Sfcs, double Sn) {
    const double Smis = __dsub_rn(Sn, Sc);
    const double mean_true = Sc > 0.0 ? __ddiv_rn(Stcs, Sc) : 1.0;
    const double mean_false = Smis > 0.0 ? __ddiv_rn(Sfcs, Smis) : 0.0;
    return __dmul_rn(0.5, __dadd_rn(mean_true, mean_false));
}

// Thresholds of every layer from the statistics as they stand (after the statistics were set from outside).
__global__ void refresh_tau_kernel(const CtlArgs a, int seq) {
    const int L = a.D.L;
    for (int l = threadIdx.x; l < L; l += blockDim.x)
        a.B.TAU[seq * L + l] = threshold(a.B.STCS[seq * L + l], a.B.SC[seq * L + l], a.B.SFCS[seq * L + l], a.B.ST[seq].Sn);
}

// (E, gamma) = argmax of (sum_{k<=gamma} alpha_E^k) / (gamma*E + L), first maximum in E-major order.
// Called by all threads of a block of at least 64 threads; u = index of the sequence in the update plan.
__device__ __forceinline__ void select_body(const CtlArgs &a, const UpdatePlan *up, del_round_out *out, int u) {
    __shared__ double s_best[64];
    __shared__ int s_g[64];
    const int seq = up->s[u].seq, L = a.D.L;
    SeqState *st = a.B.ST + seq;
    int E = a.e_min, G = a.g_min;
    if (st->fixed_E > 0 && st->fs_mode) {
        // baseline FS (Sec. 5.1): one more draft after a round whose drafts were all accepted, one fewer after
        // a rejection, within [max(1, g_min), g_max]; a round without drafts changes nothing
        E = st->fixed_E;
        G = st->gamma;
        const int g = up->s[u].g, n = out[seq].n_accept;
        const int lo = a.g_min > 1 ? a.g_min : 1;
        if (a.mode == 0 && g >= 1) G = (n == g) ? min(G + 1, a.g_max) : max(G - 1, lo);
    } else if (st->fixed_E > 0) {
        E = st->fixed_E;
        G = st->fixed_gamma;
    } else {
        const double Sn = st->Sn;
        double bestE = -1.0;
        for (int l0 = a.e_min; l0 <= a.e_max; l0 += 64) {
            const int l = l0 + threadIdx.x;
            double best = -1.0;
            int bg = a.g_min;
            if (threadIdx.x < 64 && l <= a.e_max) {
                const double alpha = __ddiv_rn(a.B.SC[seq * L + l - 1], Sn);
                double term = 1.0, sum = 1.0;
                for (int dd = 0; dd <= a.g_max; ++dd) {
                    if (dd > 0) { term = __dmul_rn(term, alpha); sum = __dadd_rn(sum, term); }
                    if (dd >= a.g_min) {
                        const double tpl = __ddiv_rn(sum, (double)(dd * l + L));
                        if (tpl > best) { best = tpl; bg = dd; }
                    }
                }
            }
            if (threadIdx.x < 64) { s_best[threadIdx.x] = best; s_g[threadIdx.x] = bg; }
            __syncthreads();
            if (threadIdx.x == 0) {
                for (int j = 0; j < 64 && l0 + j <= a.e_max; ++j)
                    if (s_best[j] > bestE) { bestE = s_best[j]; E = l0 + j; G = s_g[j]; }
            }
            __syncthreads();
        }
    }
    if (threadIdx.x == 0) {
        st->E = E;
        st->gamma = G;
        out[seq].next_E = E;
        out[seq].next_gamma = G;
        out[seq].next_tau = a.B.TAU[seq * L + E - 1];
    }
}

__global__ void __launch_bounds__(64) select_kernel(const CtlArgs a, const __grid_constant__ UpdatePlan up_v, del_round_out *out) {
    pdl_launch();
    pdl_wait();
    select_body(a, &up_v, out, blockIdx.x);
}

// Prefix acceptance, per-layer match counts over the valid context and decayed statistics
// (S <- omega * S + a, no fused multiply-add so that the host oracle's doubles are reproduced).
__global__ void __launch_bounds__(128) update_kernel(const CtlArgs a, const __grid_constant__ UpdatePlan up_v, del_round_out *out) {
    const UpdatePlan *up = &up_v;
    __shared__ int s_n;
    pdl_launch();
    pdl_wait();
    const int u = blockIdx.x;
    const int seq = up->s[u].seq, g = up->s[u].g, L = a.D.L, S = a.D.S;
    const int32_t *sh = a.B.SHADOW + (size_t)seq * L * S;
    const int32_t *verified = sh + (size_t)(L - 1) * S;
    const float *cf = a.B.SCONF + (size_t)seq * L * S;
    int32_t *tok = a.B.TOK + seq * (S + 1);
    del_round_out *o = out + seq;
    if (a.mode == 1) {
        const int W = up->s[u].n_valid_init;
        for (int j = threadIdx.x; j < up->lay_n; j += blockDim.x) {
            const int l = plan_layer(up, L, j) - 1;
            int c = 0;
            double tcs = 0.0, fcs = 0.0;
            for (int j = 0; j < W; ++j) {
                const bool match = sh[(size_t)l * S + j] == verified[j];
                c += match;
                if (match) tcs = __dadd_rn(tcs, (double)cf[(size_t)l * S + j]);
                else fcs = __dadd_rn(fcs, (double)cf[(size_t)l * S + j]);
            }
            a.B.COUNTS[seq * L + l] = c;
            a.B.SC[seq * L + l] = (double)c;
            a.B.STCS[seq * L + l] = tcs;
            a.B.SFCS[seq * L + l] = fcs;
            a.B.TAU[seq * L + l] = threshold(tcs, (double)c, fcs, (double)W);
        }
        if (threadIdx.x == 0) {
            // first token: the target's greedy token, or (speculative sampling) the one drawn from its row
            const int32_t first = up->s[u].sampling ? a.B.SMP[seq].last_token : verified[W - 1];
            a.B.ST[seq].Sn = (double)W;
            tok[0] = first;
            o->n_accept = 0;
            o->n_emitted = 1;
            o->tokens[0] = first;
        }
        if (a.do_select) {
            __syncthreads();
            select_body(a, up, out, u);
        }
        return;
    }
    const bool samp = up->s[u].sampling != 0;
    if (threadIdx.x == 0) {
        // greedy: the longest prefix of drafts equal to the target's tokens; speculative sampling: the accept
        // length and the last token decided by the sampling kernels (Sec. 2)
        int n = 0;
        if (samp) n = a.B.SMP[seq].n_accept;
        else while (n < g && tok[1 + n] == verified[n]) ++n;
        s_n = n;
        o->n_accept = n;
        o->n_emitted = n + 1;
        for (int i = 0; i < n; ++i) o->tokens[i] = tok[1 + i];
        o->tokens[n] = samp ? a.B.SMP[seq].last_token : verified[n];
        a.B.ST[seq].Sn = __dadd_rn(__dmul_rn(a.omega, a.B.ST[seq].Sn), (double)(n + 1));
    }
    __syncthreads();
    const int n = s_n;
    const double Sn_new = a.B.ST[seq].Sn;            // written by thread 0 before the barrier
    for (int j = threadIdx.x; j < up->lay_n; j += blockDim.x) {
        const int l = plan_layer(up, L, j) - 1;      // (trimmed: the statistics of the other layers are left alone)
        int c = 0;
        double tcs = 0.0, fcs = 0.0;                 // confidence sums over matched / mismatched shadow tokens (Sec. 4.4)
        for (int i = 0; i <= n; ++i) {
            const bool match = sh[(size_t)l * S + i] == verified[i];
            c += match;
            if (match) tcs = __dadd_rn(tcs, (double)cf[(size_t)l * S + i]);
            else fcs = __dadd_rn(fcs, (double)cf[(size_t)l * S + i]);
        }
        a.B.COUNTS[seq * L + l] = c;
        const double Sc = __dadd_rn(__dmul_rn(a.omega, a.B.SC[seq * L + l]), (double)c);
        const double St = __dadd_rn(__dmul_rn(a.omega, a.B.STCS[seq * L + l]), tcs);
        const double Sf = __dadd_rn(__dmul_rn(a.omega, a.B.SFCS[seq * L + l]), fcs);
        a.B.SC[seq * L + l] = Sc;
        a.B.STCS[seq * L + l] = St;
        a.B.SFCS[seq * L + l] = Sf;
        a.B.TAU[seq * L + l] = threshold(St, Sc, Sf, Sn_new);
    }
    __syncthreads();
    if (threadIdx.x == 0) tok[0] = samp ? a.B.SMP[seq].last_token : verified[n];      // next round's input token
    if (a.do_select) select_body(a, up, out, u);     // (the statistics above are visible after the barrier)
    if (a.post_out != nullptr) {
        // the finished result goes to device-writable host memory, then the stamp that announces it
        __syncthreads();
        constexpr int NWORD = (int)(sizeof(del_round_out) / sizeof(int32_t));
        const int32_t *src = reinterpret_cast<const int32_t *>(o);
        volatile int32_t *dst = a.post_out + (size_t)seq * NWORD;
        constexpr int STATUS_WORD = (int)(offsetof(del_round_out, status) / sizeof(int32_t));
        for (int w = threadIdx.x; w < NWORD; w += blockDim.x)
            dst[w] = w == STATUS_WORD ? *reinterpret_cast<volatile int32_t *>(a.B.ERR) : src[w];
        __threadfence_system();
        __syncthreads();
        if (threadIdx.x == 0) a.post_done[seq] = a.stamp;
    }
}

// Test-only: logits of the exit head on one hidden row, straightforward one-warp-per-vocab-row dots.
__global__ void __launch_bounds__(CTL_THREADS) debug_logits_kernel(const CtlArgs a, int layer, int seq, int slot, float *out) {
    __shared__ float s_red[CTL_THREADS / 32];
    __shared__ float s_r;
    const int d = a.D.d;
    const float *h = a.B.H + stack_row(a.D, layer, seq, slot) * d;
    float ss = 0.f;
    for (int o = threadIdx.x; o < d; o += CTL_THREADS) ss += h[o] * h[o];
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < CTL_THREADS / 32; ++w) t += s_red[w];
        s_r = rsqrtf(t / (float)d + a.D.eps);
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int v = blockIdx.x * (CTL_THREADS / 32) + warp; v < a.D.V; v += gridDim.x * (CTL_THREADS / 32)) {
        const bf16 *w = a.lm_head + (size_t)v * d;
        float acc = 0.f;
        for (int o = lane; o < d; o += 32) {
            const float x = bf16_to_f(__float2bfloat16_rn(h[o] * bf16_to_f(a.final_gain[o])));
            acc += bf16_to_f(w[o]) * x;
        }
        acc = warp_sum(acc);
        if (lane == 0) out[v] = acc * s_r;
    }
}

__global__ void gather_kv_kernel(const CtlArgs a, int layer, int seq, int pos, float *k_out, float *v_out) {
    const int hd = a.D.hd, n = a.D.nkv * hd;
    const int pg = a.B.PT[seq * a.D.pages_per_seq + (pos >> 4)], sl = pos & 15;
    for (int e = threadIdx.x; e < n; e += blockDim.x) {
        const int kvh = e / hd, dim = e - kvh * hd;
        const size_t base = (((size_t)pg * a.D.L + (layer - 1)) * a.D.nkv + kvh) * 16 * hd;
        k_out[e] = bf16_to_f(a.B.KP[base + (size_t)sl * hd + dim]);
        v_out[e] = bf16_to_f(a.B.VP[base + (size_t)dim * 16 + sl]);
    }
}

template <typename... KArgs, typename... Args>
cudaError_t launch(void (*kern)(KArgs...), int grid, int block, cudaStream_t st, bool pdl, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

}  // namespace

cudaError_t launch_embed(const CtlArgs &a, int m, cudaStream_t st, bool pdl) {
    return launch(embed_kernel, m, CTL_THREADS, st, pdl, a);
}
cudaError_t launch_draft_finalize_embed(const CtlArgs &a, int m, bool embed_next, cudaStream_t st, bool pdl) {
    return launch(draft_finalize_embed_kernel, m, CTL_THREADS, st, pdl, a, (int)embed_next);
}
cudaError_t launch_prep_rows(const CtlArgs &a, const UpdatePlan *up, int n_rows, cudaStream_t st, bool pdl) {
    return launch(prep_rows_kernel, n_rows, CTL_THREADS, st, pdl, a, *up);
}
cudaError_t launch_shadow_reduce(const CtlArgs &a, const UpdatePlan *up, const float *pv, const int32_t *pi, const float *ps,
                                 int n_part, int pstride, int cstride, int row_base, int n_rows, cudaStream_t st, bool pdl) {
    return launch(shadow_reduce_kernel, n_rows, CTL_THREADS, st, pdl, a, *up, pv, pi, ps, n_part, pstride, cstride, row_base);
}
cudaError_t launch_refresh_tau(const CtlArgs &a, int seq, cudaStream_t st) {
    return launch(refresh_tau_kernel, 1, 128, st, false, a, seq);
}
cudaError_t launch_update(const CtlArgs &a, const UpdatePlan *up, void *out_dev, int n_seq, cudaStream_t st, bool pdl) {
    return launch(update_kernel, n_seq, 128, st, pdl, a, *up, (del_round_out *)out_dev);
}
cudaError_t launch_select(const CtlArgs &a, const UpdatePlan *up, void *out_dev, int n_seq, cudaStream_t st, bool pdl) {
    return launch(select_kernel, n_seq, 64, st, pdl, a, *up, (del_round_out *)out_dev);
}
cudaError_t launch_debug_logits(const CtlArgs &a, int layer, int seq, int slot, float *out_dev, cudaStream_t st) {
    return launch(debug_logits_kernel, 296, CTL_THREADS, st, false, a, layer, seq, slot, out_dev);
}
cudaError_t launch_gather_kv(const CtlArgs &a, int layer, int seq, int pos, float *k_out, float *v_out, cudaStream_t st) {
    return launch(gather_kv_kernel, 1, 256, st, false, a, layer, seq, pos, k_out, v_out);
}
