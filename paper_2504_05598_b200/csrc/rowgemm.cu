// Weight-streaming skinny GEMM  Y[m, N] = X[m, K] * W[N, K]^T  for m <= 64 activation rows, with the
// layer's element-wise work fused into its epilogues.  It is bound by HBM: every weight byte is read
// exactly once per pass, straight from global memory into tensor-core fragments.
//
// Mapping.  A tile is 16 weight rows (output features; two groups of 8, see tile_rows) over the whole K.  The 8 warps of a
// CTA split K in 32-element steps (warp w takes steps w, w+8, ...), so at any time the CTA reads 512
// contiguous bytes of each of the 16 rows.  Per step a thread issues one 16-byte load for row g and one
// for row g+8 (g = lane/4) at column offset 8*(lane%4): the eight bf16 values feed two m16n8k16 MMAs.
// The tensor core sums over k, so any permutation of k applied to both operands gives the same
// product; the activation fragment is therefore loaded with the same 16-byte pattern from the row's
// bf16 vector, and no shared-memory staging or ldmatrix is needed.  Loads are issued in bursts of U
// k-steps (all loads of a burst before its first MMA); the two resident CTAs per SM overlap each
// other's bursts, and the first burst of weights is issued before the kernel waits for its producer
// (programmatic dependent launch).
// Partial sums of the 8 warps are added in a fixed order through shared memory: results do not depend
// on the grid size or on how many rows share the pass.
//
// Activation precision.  The layer GEMMs take every activation as a pair of bf16 values (high + low part, 16
// bits of mantissa; the weights are exact bf16 anyway), so that the product carries fp32-like accuracy.  The
// low parts cost no extra tensor-core instruction for up to four rows: the eight columns of an MMA's n-tile
// hold the high parts of rows 0..3 and the low parts of the same rows, and the two column halves are added
// after the cross-warp reduction.  In general a launch of NT n-tiles serves 4 * NT rows (at most 32; a pass
// of more rows is two launches).  The LM head takes single bf16 rows (8 * NT of them).
//
// Epilogues (one per use in the decoder layer):
//   QKV    scale by the row's 1/rms, rotary embedding on q and k, q -> Q buffer, k and v -> paged cache
//   OPROJ  + residual -> HM, XM = bf16(HM * ffn gain), partial sums of squares
//   GATEUP scale by 1/rms, silu(gate) * up -> ACT
//   DOWN   + residual -> hidden stack, XS/XE = bf16(h * next gain), partial sums of squares
//   LMHEAD running arg-max over the vocabulary tiles of this CTA (1/rms > 0 cannot change it)
// RMSNorm is split: the producer stores bf16(h * gain) and per-tile sums of h^2, the consumer scales
// its accumulators by rsqrt(mean(h^2) + eps) (the scale is a per-row scalar, so it commutes with W).
#include "kernels.h"

namespace {


// bytes of the reduction buffer, result tile, row scales and arg-max state (16-byte multiple)
__host__ __device__ constexpr size_t small_smem_bytes(int nt, int nw) {
    return (sizeof(float4) * nw * nt * 32 + sizeof(float) * (nt * 8 * 16 + 4 * nt * 8) + 15) & ~(size_t)15;
}

// The 16 weight rows of a tile are two groups of 8 (MMA rows g and g+8), which need not be adjacent:
//   QKV, q and k tiles: rows j..j+7 of a head and their rotary partners j+hd/2..  (one thread then holds
//        both members of every rotation pair); v tiles: 16 consecutive rows
//   GATEUP: 8 rows of W_gate and the same 8 rows of W_up (SiLU(gate)*up stays inside the tile)
//   others: 16 consecutive rows
template <int EPI>
__device__ __forceinline__ void tile_rows(const GemmArgs &a, int item, const bf16 *&lo, const bf16 *&hi) {
    if (EPI == EPI_QKV) {
        const int h8 = a.D.hd >> 4;                 // tiles per head
        const int nq = a.D.nh * h8, nk = a.D.nkv * h8;
        if (item < nq + nk) {
            const bf16 *W = item < nq ? a.W0 : a.W1;
            const int it = item < nq ? item : item - nq;
            const int head = it / h8, jb = it - head * h8;
            lo = W + (size_t)(head * a.D.hd + jb * 8) * a.K;
            hi = lo + (size_t)(a.D.hd >> 1) * a.K;
            return;
        }
        lo = a.W2 + (size_t)(16 * (item - nq - nk)) * a.K;
        hi = lo + (size_t)8 * a.K;
        return;
    }
    if (EPI == EPI_GATEUP) {
        lo = a.W0 + (size_t)(8 * item) * a.K;
        hi = a.W1 + (size_t)(8 * item) * a.K;
        return;
    }
    lo = a.W0 + (size_t)(16 * item) * a.K;
    hi = lo + (size_t)8 * a.K;
}

// NW warps split K: 8 (two CTAs per SM for up to 32 columns), or 16 in one CTA per SM for launches with no more
// tiles than SMs and a long K, where a second CTA per SM would find no tile and the tile's bursts run in a row
template <int NT, int U, int EPI, int NW>
__global__ void __launch_bounds__(NW * 32, (NW == 8 && NT <= 4 ? 2 : 1)) rowgemm_kernel(const __grid_constant__ GemmArgs a) {
    constexpr int NTHREADS = NW * 32;
    constexpr int NC = NT * 8;                      // MMA columns
    constexpr bool HL = EPI != EPI_LMHEAD;          // columns [0, NR): high parts of NR rows, [NR, NC): their low parts
    constexpr int NR = HL ? NC / 2 : NC;            // activation rows handled
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float4 *red = reinterpret_cast<float4 *>(smem_raw);                       // [NW warps][NT][32]
    float *res = reinterpret_cast<float *>(smem_raw + sizeof(float4) * NW * NT * 32);  // [NC][16]
    float *rscale = res + NC * 16;                                      // [NC]
    float *best_v = rscale + NC;                                              // [NC]
    int *best_i = reinterpret_cast<int *>(best_v + NC);                       // [NC]
    float *best_s = best_v + 2 * NC;                                          // [NC] exp sums relative to best_v

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int K = a.K;
    const int n_ksteps = (K + 31) >> 5;
    const int nkw = (n_ksteps + NW - 1) / NW;       // k-steps per warp and tile (the last ones may be empty)
    __shared__ int s_claim[2];                      // tile claimed for the turn after next (double-buffered)

    uint4 wa[U], wb[U];
    uint4 xv[U][NT];
    const bf16 *xrow[NT];

    const bf16 *base = nullptr, *base_hi = nullptr;     // this thread's row g / row g+8 of the current tile
    auto tile_base = [&](int item) {
        tile_rows<EPI>(a, item, base, base_hi);
        base += (size_t)g * K + 8 * t;
        base_hi += (size_t)g * K + 8 * t;
    };
    // one burst: U k-steps of this warp, all loads issued before the first use
    // (the load sequences are kept free of branches: the compiler batches them only in straight-line code)
    auto load_w = [&](int u0, bool live) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int k0 = (warp + NW * (u0 + u)) << 5;
            const bool ok = live && (u0 + u < nkw) && (k0 + 8 * t < K);
            wa[u] = ldg_stream16_pred(base + k0, ok);
            wb[u] = ldg_stream16_pred(base_hi + k0, ok);
        }
    };
    auto load_x = [&](int u0, bool live) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int k0 = ((warp + NW * (u0 + u)) << 5) + 8 * t;
            const bool ok = live && (u0 + u < nkw) && (k0 < K);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) xv[u][nt] = ldg_act16_pred(xrow[nt] + k0, ok && xrow[nt] != nullptr);
        }
    };

    // the first burst of weights goes out before the producer kernel has finished
    // Tiles: two static turns per CTA (b, b + grid), further tiles claimed from a per-launch counter so that
    // fast CTAs take more and all CTAs finish together.  Results do not depend on who computes a tile.
    const int grid = (int)gridDim.x;
    int cur_item = blockIdx.x;
    int nxt_item = cur_item + grid < a.n_items ? cur_item + grid : -1;
    int claimed = -1;                               // thread 0: the claim in flight
    auto claim = [&]() {
        if (tid == 0 && a.tile_ctr != nullptr && nxt_item >= 0) claimed = 2 * grid + atomicAdd(a.tile_ctr, 1);
    };
    tile_base(cur_item);
    load_w(0, true);
    claim();
    pdl_launch();
    pdl_wait();

    const PassPlan *plan = &a.plan;
    const int row0 = HL ? a.row0 : 0;               // rows row0 .. row0 + NR - 1 of the pass
    const int m = plan->m;
    // activation row pointers of this thread's columns
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int col = nt * 8 + g;
        const bool low = HL && col >= NR;
        const int c = row0 + (low ? col - NR : col);
        xrow[nt] = nullptr;
        if (c < m) {
            size_t r;
            if (EPI == EPI_QKV) r = stack_row(a.D, a.layer - 1, plan->rows[c].seq, plan->rows[c].slot);
            else if (EPI == EPI_LMHEAD) r = a.x_by_row ? (size_t)c : (size_t)plan->rows[c].seq * a.D.S + plan->rows[c].slot;
            else r = c;
            xrow[nt] = (low ? a.XL : a.X) + r * (size_t)K;
        }
    }
    load_x(0, true);

    // per-row 1/rms from the producer's partial sums of squares: the loads of this warp's first row go
    // out now, their sum is taken after the first burst of MMAs (it is needed in the first epilogue only)
    constexpr int SSN = 12;                         // 32 * 12 partials = rows of up to 6144 features
    float ssv[SSN];
    auto ss_ptr = [&](int c) -> const float * {
        if (EPI == EPI_GATEUP) return a.B.SSM + (size_t)c * a.D.n_sst;
        return a.B.SS + stack_row(a.D, a.layer - 1, plan->rows[c].seq, plan->rows[c].slot) * a.D.n_sst;
    };
    if (EPI == EPI_QKV || EPI == EPI_GATEUP) {
        const bool v0 = warp < NR && row0 + warp < m;
        const float *ss = v0 ? ss_ptr(row0 + warp) : a.B.SSM;
#pragma unroll
        for (int q = 0; q < SSN; ++q) {
            const int i = lane + 32 * q;
            ssv[q] = (v0 && i < a.D.n_sst) ? ldg_cg_f32(ss + i) : 0.f;
        }
    }
    if (EPI == EPI_LMHEAD) {
        for (int c = tid; c < NC; c += NTHREADS) { best_v[c] = -INFINITY; best_i[c] = 0x7fffffff; best_s[c] = 0.f; }
    }
    // no barrier here: rscale / best_* are first read in an epilogue, after the two barriers of tile_end

    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;

    int turn = 0;

    // The residual element that this thread's epilogue adds (O-projection: the hidden stack; down: the stream after
    // attention) is requested when the tile starts, so that the epilogue of a CTA's last tile does not begin with a
    // round trip to L2.  One element per thread; the 8-column variant only (the 16-column one does not gain, the wider
    // ones have no register to spare).
    constexpr bool RES_PRE = (EPI == EPI_OPROJ || EPI == EPI_DOWN) && NT == 1;
    float h_pre = 0.f;
    bf16 ga_pre = __float2bfloat16_rn(0.f), gb_pre = __float2bfloat16_rn(0.f);      // the norm gains of that output feature
    // QKV: the rotation's cos / sin of this thread's pair and the cache page of its row
    constexpr bool ROPE_PRE = EPI == EPI_QKV && NT == 1;
    float cs_pre = 0.f, sn_pre = 0.f;
    int pg_pre = 0;
    if (ROPE_PRE) {
        const int cl = tid >> 4, c = row0 + cl;
        if (cl < NR && c < m) pg_pre = a.B.PT[plan->rows[c].seq * a.D.pages_per_seq + (plan->rows[c].pos >> 4)];
    }
    auto prefetch_residual = [&](int item) {
        if (RES_PRE) {
            const int cl = tid >> 4, c = row0 + cl;
            if (cl < NR && c < m) {
                const int o = 16 * item + (tid & 15);
                if (EPI == EPI_OPROJ) h_pre = ldg_cg_f32(a.B.H + stack_row(a.D, a.layer - 1, plan->rows[c].seq, plan->rows[c].slot) * a.D.d + o);
                else h_pre = ldg_cg_f32(a.B.HM + (size_t)c * a.D.d + o);
                if (a.gain_a) ga_pre = a.gain_a[o];
                if (EPI == EPI_DOWN && a.gain_b) gb_pre = a.gain_b[o];
            }
        }
        if (ROPE_PRE) {
            const int cl = tid >> 4, c = row0 + cl, i = tid & 15;
            const int hd = a.D.hd, half = hd >> 1, h8 = hd >> 4;
            const int nq = a.D.nh * h8, nk = a.D.nkv * h8;
            if (cl < NR && c < m && i < 8 && item < nq + nk) {
                const int it = item < nq ? item : item - nq;
                const int j = (it - (it / h8) * h8) * 8 + i;
                cs_pre = a.B.rope_cos[(size_t)plan->rows[c].pos * half + j];
                sn_pre = a.B.rope_sin[(size_t)plan->rows[c].pos * half + j];
            }
        }
    };
    prefetch_residual(cur_item);

    auto tile_end = [&]() {
        // fixed-order sum of the 8 warps' partials
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            red[(warp * NT + nt) * 32 + lane] = make_float4(acc[nt][0], acc[nt][1], acc[nt][2], acc[nt][3]);
            acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
        }
        __syncthreads();
        for (int e = tid; e < NT * 32; e += NTHREADS) {
            float4 s = red[e];
#pragma unroll
            for (int w = 1; w < NW; ++w) {
                const float4 v = red[w * NT * 32 + e];
                s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
            }
            const int nt = e >> 5, l2 = e & 31, g2 = l2 >> 2, t2 = l2 & 3;
            float *r0 = res + (nt * 8 + 2 * t2) * 16;
            r0[g2] = s.x; r0[16 + g2] = s.y; r0[g2 + 8] = s.z; r0[16 + g2 + 8] = s.w;
        }
        __syncthreads();
        const int item = cur_item;
        const int i = tid & 15;
        for (int cl = tid >> 4; cl < NR; cl += NTHREADS / 16) {
            const int c = row0 + cl;                // row of the pass; cl: its column in this launch
            const bool valid = c < m;
            const RowDesc rd = valid ? plan->rows[c] : RowDesc{0, 0, 0, 0};
            // product with the high parts + product with the low parts
            const float ra = HL ? res[cl * 16 + i] + res[(cl + NR) * 16 + i] : res[cl * 16 + i];
            // rows 8..15 of the tile at the same column (rotary partner / up row), read by threads i < 8 only
            const float rb = HL ? res[cl * 16 + (i | 8)] + res[(cl + NR) * 16 + (i | 8)] : 0.f;
            if (EPI == EPI_QKV) {
                if (!valid) continue;
                const float r = rscale[cl];
                const int hd = a.D.hd, half = hd >> 1, h8 = hd >> 4;
                const int nq = a.D.nh * h8, nk = a.D.nkv * h8;
                const int pg = ROPE_PRE ? pg_pre : a.B.PT[rd.seq * a.D.pages_per_seq + (rd.pos >> 4)];
                const int sl = rd.pos & 15;
                if (item < nq + nk) {
                    if (i >= 8) continue;                         // rows 0..7 and their partners 8..15: one thread per pair
                    const float va = r * ra, vb = r * rb;
                    const bool isq = item < nq;
                    const int it = isq ? item : item - nq;
                    const int head = it / h8, j = (it - head * h8) * 8 + i;
                    const float cs = ROPE_PRE ? cs_pre : a.B.rope_cos[(size_t)rd.pos * half + j];
                    const float sn = ROPE_PRE ? sn_pre : a.B.rope_sin[(size_t)rd.pos * half + j];
                    const float oa = va * cs - vb * sn, ob = vb * cs + va * sn;
                    if (isq) {
                        bf16 *q = a.B.Q + (size_t)c * (a.D.nh * hd) + head * hd + j;
                        q[0] = __float2bfloat16_rn(oa);
                        q[half] = __float2bfloat16_rn(ob);
                    } else {
                        bf16 *kp = a.B.KP + ((((size_t)pg * a.D.L + (a.layer - 1)) * a.D.nkv + head) * 16 + sl) * hd + j;
                        kp[0] = __float2bfloat16_rn(oa);
                        kp[half] = __float2bfloat16_rn(ob);
                    }
                } else {
                    const int n0 = 16 * (item - nq - nk) + i;      // value feature
                    const int kvh = n0 / hd, dim = n0 - kvh * hd;
                    a.B.VP[((((size_t)pg * a.D.L + (a.layer - 1)) * a.D.nkv + kvh) * hd + dim) * 16 + sl] = __float2bfloat16_rn(r * ra);
                }
            } else if (EPI == EPI_GATEUP) {
                if (!valid) continue;
                const float r = rscale[cl];
                if (i >= 8) continue;                             // rows 0..7 gate, rows 8..15 the matching up rows
                const float gate = r * ra, up = r * rb;
                const float act = gate / (1.f + __expf(-gate)) * up;
                split_bf16(act, a.B.ACT[(size_t)c * a.D.F + 8 * item + i], a.B.ACTL[(size_t)c * a.D.F + 8 * item + i]);
            } else if (EPI == EPI_OPROJ || EPI == EPI_DOWN) {
                const int o = 16 * item + i;
                float h = 0.f;
                if (valid) {
                    if (EPI == EPI_OPROJ) {
                        h = (RES_PRE ? h_pre : ldg_cg_f32(a.B.H + stack_row(a.D, a.layer - 1, rd.seq, rd.slot) * a.D.d + o)) + ra;
                        a.B.HM[(size_t)c * a.D.d + o] = h;
                        split_bf16(h * bf16_to_f(RES_PRE ? ga_pre : a.gain_a[o]), a.B.XM[(size_t)c * a.D.d + o], a.B.XML[(size_t)c * a.D.d + o]);
                    } else {
                        h = (RES_PRE ? h_pre : ldg_cg_f32(a.B.HM + (size_t)c * a.D.d + o)) + ra;
                        const size_t sr = stack_row(a.D, a.layer, rd.seq, rd.slot);
                        a.B.H[sr * a.D.d + o] = h;
                        if (a.gain_a) split_bf16(h * bf16_to_f(RES_PRE ? ga_pre : a.gain_a[o]), a.B.XS[sr * a.D.d + o], a.B.XSL[sr * a.D.d + o]);
                        if (a.gain_b)
                            a.B.XE[((size_t)rd.seq * a.D.S + rd.slot) * a.D.d + o] = __float2bfloat16_rn(h * bf16_to_f(RES_PRE ? gb_pre : a.gain_b[o]));
                    }
                }
                float ss = h * h;
                ss += __shfl_xor_sync(0xffffffffu, ss, 8);
                ss += __shfl_xor_sync(0xffffffffu, ss, 4);
                ss += __shfl_xor_sync(0xffffffffu, ss, 2);
                ss += __shfl_xor_sync(0xffffffffu, ss, 1);
                if (valid && i == 0) {
                    if (EPI == EPI_OPROJ) a.B.SSM[(size_t)c * a.D.n_sst + item] = ss;
                    else {
                        a.B.SS[stack_row(a.D, a.layer, rd.seq, rd.slot) * a.D.n_sst + item] = ss;
                        if (a.gain_b) a.B.SSE[((size_t)rd.seq * a.D.S + rd.slot) * a.D.n_sst + item] = ss;
                    }
                }
            } else if (EPI == EPI_LMHEAD) {
                float v = valid ? ra : -INFINITY;      // the row's 1/rms is positive: it cannot change the arg-max
                int idx = 16 * item + i;
                if (a.logits_out != nullptr && valid) {
                    // speculative sampling needs the whole row: normalised logit = raw / rms
                    const size_t lr = a.x_by_row ? (size_t)c : (size_t)rd.seq * DEL_SAMPLE_ROWS + rd.slot;
                    a.logits_out[lr * a.D.V + idx] = ra * (rscale[c] * 0.6931471805599453f);
                }
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) {
                    const float v2 = __shfl_xor_sync(0xffffffffu, v, o);
                    const int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
                    if (v2 > v || (v2 == v && i2 < idx)) { v = v2; idx = i2; }
                }
                // running sum of exp over the vocabulary for the confidence score (top-1 probability): the
                // normalised logit is raw / rms, kept as exp2(k * (raw - running maximum)) with k = log2(e) / rms
                const float k = rscale[c];
                float es = valid ? exp2f(k * (ra - v)) : 0.f;
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) es += __shfl_xor_sync(0xffffffffu, es, o);
                if (valid && i == 0) {
                    const float bv = best_v[c];
                    if (v > bv) {
                        best_s[c] = best_s[c] * exp2f(k * (bv - v)) + es;
                        best_v[c] = v;
                        best_i[c] = idx;
                    } else {
                        best_s[c] += es * exp2f(k * (v - bv));
                        if (v == bv && idx < best_i[c]) best_i[c] = idx;
                    }
                }
            }
        }
        // `res` and `best_*` are next written after the following tile's first barrier
    };

    auto mma_burst = [&]() {
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                mma_bf16_16816(acc[nt], wa[u].x, wb[u].x, wa[u].y, wb[u].y, xv[u][nt].x, xv[u][nt].y);
                mma_bf16_16816(acc[nt], wa[u].z, wb[u].z, wa[u].w, wb[u].w, xv[u][nt].z, xv[u][nt].w);
            }
    };

    mma_burst();
    if (EPI == EPI_QKV || EPI == EPI_GATEUP) {
        for (int cl = warp; cl < NR; cl += NW) {
            const int c = row0 + cl;
            float s = 0.f;
            if (cl == warp) {
#pragma unroll
                for (int q = 0; q < SSN; ++q) s += ssv[q];
                if (c < m)
                    for (int i = lane + 32 * SSN; i < a.D.n_sst; i += 32) s += ldg_cg_f32(ss_ptr(c) + i);
            } else if (c < m) {
                const float *ss = ss_ptr(c);
                for (int i = lane; i < a.D.n_sst; i += 32) s += ldg_cg_f32(ss + i);
            }
            s = warp_sum(s);
            if (lane == 0) rscale[cl] = rsqrtf(s / (float)a.D.d + a.D.eps);
        }
    }
    if (EPI == EPI_LMHEAD) {
        for (int c = warp; c < NC; c += NW) {
            float k = 0.f;
            if (c < m) {
                if (a.row_scale) {
                    k = a.row_scale[c];
                } else if (a.B.SSE != nullptr) {    // (callers that want no confidences pass neither: k = 0)
                    const float *ss = a.B.SSE + ((size_t)plan->rows[c].seq * a.D.S + plan->rows[c].slot) * a.D.n_sst;
                    float sq = 0.f;
                    for (int i = lane; i < a.D.n_sst; i += 32) sq += ldg_cg_f32(ss + i);
                    sq = warp_sum(sq);
                    k = rsqrtf(sq / (float)a.D.d + a.D.eps) * 1.4426950408889634f;
                }
            }
            if (lane == 0) {
                rscale[c] = k;
                if (blockIdx.x == 0 && c < m && a.B.RK != nullptr) a.B.RK[c] = k;
            }
        }
    }
    int u0 = U;
    for (;;) {
        for (; u0 < nkw; u0 += U) {
            load_w(u0, true);
            load_x(u0, true);
            mma_burst();
        }
        // the next tile's first burst is in flight while this tile is reduced and written out
        const bool more = nxt_item >= 0;
        if (more) tile_base(nxt_item);
        load_w(0, more);
        load_x(0, more);
        if (tid == 0) s_claim[turn & 1] = claimed;
        tile_end();
        if (!more) break;
        int after;
        if (a.tile_ctr != nullptr) after = s_claim[turn & 1];
        else after = nxt_item + grid;
        cur_item = nxt_item;
        nxt_item = (after >= 0 && after < a.n_items) ? after : -1;
        ++turn;
        claim();
        prefetch_residual(cur_item);
        mma_burst();
        u0 = U;
    }

    if (EPI == EPI_LMHEAD) {
        __syncthreads();
        for (int c = tid; c < m; c += NTHREADS) {
            a.B.LPV[(size_t)blockIdx.x * DEL_ROWS_MAX + c] = best_v[c];
            a.B.LPI[(size_t)blockIdx.x * DEL_ROWS_MAX + c] = best_i[c];
            if (a.B.LPS) a.B.LPS[(size_t)blockIdx.x * DEL_ROWS_MAX + c] = best_s[c];
        }
    }
}

template <int NT> constexpr int depth_for() { return NT == 1 ? 8 : (NT <= 4 ? 4 : 3); }

template <int NT, int EPI, int NW = DEL_GEMM_WARPS>
cudaError_t launch_nt(const GemmArgs &a, int grid, cudaStream_t st, bool pdl) {
    constexpr int D = depth_for<NT>();
    constexpr int NC = NT * 8;
    const size_t smem = small_smem_bytes(NT, NW);
    auto kern = rowgemm_kernel<NT, D, EPI, NW>;
    static SmemAttrOnce attr;
    {
        cudaError_t e = attr.set(kern, (int)((int)smem));
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(NW * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, a);
}

// m: rows this launch handles (layer GEMMs: two columns per row)
template <int EPI>
cudaError_t launch_epi(const GemmArgs &a, int m, int n_sms, cudaStream_t st, bool pdl) {
    const int nt = EPI == EPI_LMHEAD ? (m + 7) / 8 : (m + 3) / 4;
    const int per_sm = a.ctas_per_sm == 1 ? 1 : 2;
    if (nt <= 1) {
        // no more tiles than SMs and at least two bursts per warp even with 16 warps: one CTA of 16 warps per tile
        if constexpr (EPI == EPI_DOWN) {
            if (a.n_items <= n_sms && a.K >= 2 * 16 * 32 * depth_for<1>()) return launch_nt<1, EPI, 16>(a, a.n_items, st, pdl);
        }
        return launch_nt<1, EPI>(a, min(a.n_items, per_sm * n_sms), st, pdl);
    }
    if (nt <= 2) return launch_nt<2, EPI>(a, min(a.n_items, per_sm * n_sms), st, pdl);
    if (nt <= 4) return launch_nt<4, EPI>(a, min(a.n_items, per_sm * n_sms), st, pdl);
    return launch_nt<8, EPI>(a, min(a.n_items, n_sms), st, pdl);
}

}  // namespace

cudaError_t launch_rowgemm(int epi, const GemmArgs &a, int m, int n_sms, cudaStream_t st, bool pdl) {
    if (epi != EPI_LMHEAD) m = min(m - a.row0, DEL_GEMM_ROWS);
    switch (epi) {
        case EPI_QKV: return launch_epi<EPI_QKV>(a, m, n_sms, st, pdl);
        case EPI_OPROJ: return launch_epi<EPI_OPROJ>(a, m, n_sms, st, pdl);
        case EPI_GATEUP: return launch_epi<EPI_GATEUP>(a, m, n_sms, st, pdl);
        case EPI_DOWN: return launch_epi<EPI_DOWN>(a, m, n_sms, st, pdl);
        case EPI_LMHEAD: return launch_epi<EPI_LMHEAD>(a, m, n_sms, st, pdl);
    }
    return cudaErrorInvalidValue;
}

int rowgemm_lmhead_grid(int n_items, int m, int n_sms, int ctas_per_sm) {
    const int nt = (m + 7) / 8;
    const int cap = nt <= 4 ? (ctas_per_sm == 1 ? 1 : 2) * n_sms : n_sms;
    return n_items < cap ? n_items : cap;
}
