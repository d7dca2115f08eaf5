// Multi-query decode attention over the paged bf16 KV cache.
//
// One CTA = (key-range split, kv head, sequence segment), 8 warps.  The query rows of the segment (its
// 1..32 consecutive positions times the query heads sharing this kv head) form 16-row tiles; the warps
// are divided among up to 4 query tiles, and the warps of one tile walk the key pages (16 tokens each)
// of the CTA's key range in a strided fashion.  Scores and the P*V product run on bf16 tensor-core
// MMAs with fp32 accumulation; the softmax is the online (running max / running sum) form, its row
// reductions done with warp shuffles inside the 4-lane groups that own a row.
//
// Fragment loading without shared memory: the MMA sums over its k index, so any permutation of k used
// for both operands is allowed.  For Q*K^T a thread loads 16 contiguous bytes of a key row (and the
// same bytes of the query row) and feeds them to two MMAs.  For P*V the page stores V transposed
// ([head_dim][16 tokens]); the score tile's columns are assigned to tokens such that a thread's four
// probabilities belong to tokens 4t..4t+3, which are 8 contiguous bytes of a V^T row.  The page ids of
// a warp are fetched up front, and all loads of a page (keys and values) are issued before their
// first use.
//
// The warps of a query tile merge their (max, sum, output) states through shared memory, every warp
// of the CTA merging a slice of the output columns.  With one split the result is final; otherwise
// splits write partials and the last CTA to arrive for a (segment, kv head) merges them in split
// order, so the result does not depend on scheduling.
#include "kernels.h"

namespace {

constexpr float LOG2E = 1.4426950408889634f;
constexpr int NW = 8;                 // warps per CTA
constexpr int PG = 4;                 // page ids fetched ahead per warp

template <int HD>
__global__ void __launch_bounds__(NW * 32) attention_kernel(const __grid_constant__ AttnArgs a) {
    constexpr int KS = HD / 32;       // 16-byte chunks per thread along head_dim
    constexpr int NJ = HD / 8;        // output n-tiles
    extern __shared__ __align__(16) float sm[];
    float *sm_o = sm;                               // [NW][32][NJ*4]
    float *sm_ml = sm + NW * 32 * NJ * 4;           // [NW][32][4]
    __shared__ int s_last;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    pdl_launch();
    pdl_wait();

    const PassPlan *plan = &a.plan;
    const Segment seg = plan->seg[blockIdx.z];
    const int kvh = blockIdx.y, split = blockIdx.x, n_splits = a.n_splits;
    const int ms = seg.nrows, group = a.D.nh / a.D.nkv;
    const int R = ms * group, n_mt = (R + 15) >> 4;
    const int kv_len = seg.pos0 + ms;
    const int n_pages = (kv_len + 15) >> 4;
    const int pps = (n_pages + n_splits - 1) / n_splits;
    const int p_begin = split * pps, p_end = min(n_pages, p_begin + pps);
    const int P = n_mt >= 3 ? 4 : n_mt;             // query tiles handled concurrently: 1, 2 or 4
    const int n_kl = NW / P, kl = warp / P;
    const float sc = rsqrtf((float)HD) * LOG2E;
    const int32_t *pt = a.B.PT + seg.seq * a.D.pages_per_seq;
    const size_t page_stride = (size_t)a.D.L * a.D.nkv * 16 * HD;
    const size_t head_off = ((size_t)(a.layer - 1) * a.D.nkv + kvh) * 16 * HD;
    const int qdim = a.D.nh * HD;
    const int n_iter = (n_mt + P - 1) / P;
    const int key0 = 4 * (g >> 1) + (g & 1);        // token of score-tile 0 column g; tile 1: +2

    for (int it = 0; it < n_iter; ++it) {
        const int mt = it * P + warp % P;
        // rows of this thread: rr0 = mt*16+g, rr1 = rr0+8, ordered head-major: rr = hq*ms + i
        const int rr[2] = {mt * 16 + g, mt * 16 + g + 8};
        int ri[2], rh[2];
        bool rv[2];
        uint4 qf[2][KS];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            rv[h] = mt < n_mt && rr[h] < R;
            rh[h] = rv[h] ? rr[h] / ms : 0;
            ri[h] = rv[h] ? rr[h] - rh[h] * ms : 0;
            const bf16 *qp = a.B.Q + (size_t)(seg.row0 + ri[h]) * qdim + (kvh * group + rh[h]) * HD + 8 * t;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) qf[h][ks] = ldg_act16_pred(qp + 32 * ks, rv[h]);
        }
        const int rpos[2] = {seg.pos0 + ri[0], seg.pos0 + ri[1]};
        float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
        float O[NJ][4];
#pragma unroll
        for (int j = 0; j < NJ; ++j) O[j][0] = O[j][1] = O[j][2] = O[j][3] = 0.f;

        if (mt < n_mt) {
            for (int pb = p_begin + kl; pb < p_end; pb += n_kl * PG) {
                int pgs[PG];
#pragma unroll
                for (int q = 0; q < PG; ++q) {
                    const int p = pb + q * n_kl;
                    pgs[q] = p < p_end ? pt[p] : 0;
                }
#pragma unroll
                for (int q = 0; q < PG; ++q) {
                    const int p = pb + q * n_kl;
                    if (p >= p_end) break;
                    const bf16 *kpage = a.B.KP + (size_t)pgs[q] * page_stride + head_off;
                    const bf16 *vpage = a.B.VP + (size_t)pgs[q] * page_stride + head_off;
                    uint4 kf[2][KS];
                    uint2 vf[NJ];
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        kf[0][ks] = ldg_act16(kpage + key0 * HD + 32 * ks + 8 * t);
                        kf[1][ks] = ldg_act16(kpage + (key0 + 2) * HD + 32 * ks + 8 * t);
                    }
#pragma unroll
                    for (int j = 0; j < NJ; ++j) vf[j] = ldg_act8(vpage + (8 * j + g) * 16 + 4 * t);
                    float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        mma_bf16_16816(s0, qf[0][ks].x, qf[1][ks].x, qf[0][ks].y, qf[1][ks].y, kf[0][ks].x, kf[0][ks].y);
                        mma_bf16_16816(s0, qf[0][ks].z, qf[1][ks].z, qf[0][ks].w, qf[1][ks].w, kf[0][ks].z, kf[0][ks].w);
                        mma_bf16_16816(s1, qf[0][ks].x, qf[1][ks].x, qf[0][ks].y, qf[1][ks].y, kf[1][ks].x, kf[1][ks].y);
                        mma_bf16_16816(s1, qf[0][ks].z, qf[1][ks].z, qf[0][ks].w, qf[1][ks].w, kf[1][ks].z, kf[1][ks].w);
                    }
                    // this thread's scores: tokens 4t, 4t+1 (s0) and 4t+2, 4t+3 (s1) of the page, rows g / g+8
                    const int tok0 = p * 16 + 4 * t;
                    float pr[2][4];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        float v[4] = {s0[2 * h] * sc, s0[2 * h + 1] * sc, s1[2 * h] * sc, s1[2 * h + 1] * sc};
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (!rv[h] || tok0 + e > rpos[h]) v[e] = -INFINITY;
                        float mx = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3]));
                        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                        const float m_new = fmaxf(m_run[h], mx);
                        const float base = (m_new == -INFINITY) ? 0.f : m_new;
                        const float alpha = exp2f(m_run[h] - base);
                        m_run[h] = m_new;
                        float psum = 0.f;
#pragma unroll
                        for (int e = 0; e < 4; ++e) { pr[h][e] = exp2f(v[e] - base); psum += pr[h][e]; }
                        l_run[h] = l_run[h] * alpha + psum;
#pragma unroll
                        for (int j = 0; j < NJ; ++j) { O[j][2 * h] *= alpha; O[j][2 * h + 1] *= alpha; }
                    }
                    const uint32_t pa0 = pack_bf16(pr[0][0], pr[0][1]), pa1 = pack_bf16(pr[1][0], pr[1][1]);
                    const uint32_t pa2 = pack_bf16(pr[0][2], pr[0][3]), pa3 = pack_bf16(pr[1][2], pr[1][3]);
#pragma unroll
                    for (int j = 0; j < NJ; ++j) mma_bf16_16816(O[j], pa0, pa1, pa2, pa3, vf[j].x, vf[j].y);
                }
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
            l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
        }

        // ---- merge the warps of each query tile; every warp merges some output column tiles
        {
            // layout [column tile][warp][lane]: consecutive lanes write consecutive 16-byte words
#pragma unroll
            for (int j = 0; j < NJ; ++j)
                *reinterpret_cast<float4 *>(sm_o + (size_t)((j * NW + warp) * 32 + lane) * 4) = make_float4(O[j][0], O[j][1], O[j][2], O[j][3]);
            *reinterpret_cast<float4 *>(sm_ml + (warp * 32 + lane) * 4) = make_float4(m_run[0], l_run[0], m_run[1], l_run[1]);
        }
        __syncthreads();
        for (int task = warp; task < P * NJ; task += NW) {
            const int mp = task / NJ, j = task - mp * NJ;      // query-tile slot of this iteration, column tile
            const int mt2 = it * P + mp;
            if (mt2 >= n_mt) continue;
            float M0 = -INFINITY, M1 = -INFINITY;
            for (int k2 = 0; k2 < n_kl; ++k2) {
                const float4 ml = *reinterpret_cast<const float4 *>(sm_ml + ((mp + k2 * P) * 32 + lane) * 4);
                M0 = fmaxf(M0, ml.x);
                M1 = fmaxf(M1, ml.z);
            }
            const float b0 = M0 == -INFINITY ? 0.f : M0, b1 = M1 == -INFINITY ? 0.f : M1;
            float L0 = 0.f, L1 = 0.f, o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
            for (int k2 = 0; k2 < n_kl; ++k2) {
                const int w2 = mp + k2 * P;
                const float4 ml = *reinterpret_cast<const float4 *>(sm_ml + (w2 * 32 + lane) * 4);
                const float f0 = exp2f(ml.x - b0), f1 = exp2f(ml.z - b1);
                L0 += ml.y * f0;
                L1 += ml.w * f1;
                const float4 ov = *reinterpret_cast<const float4 *>(sm_o + (size_t)((j * NW + w2) * 32 + lane) * 4);
                o0 += ov.x * f0; o1 += ov.y * f0; o2 += ov.z * f1; o3 += ov.w * f1;
            }
            const float Mv[2] = {M0, M1}, Lv[2] = {L0, L1}, ov2[2][2] = {{o0, o1}, {o2, o3}};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int r2 = mt2 * 16 + g + 8 * h;
                if (r2 >= R) continue;
                const int hq = r2 / ms, i = r2 - hq * ms;
                const int c = seg.row0 + i, qh = kvh * group + hq;
                if (n_splits == 1) {
                    const float inv = 1.f / Lv[h];
                    *reinterpret_cast<uint32_t *>(a.B.ATT + (size_t)c * qdim + qh * HD + 8 * j + 2 * t) =
                        pack_bf16(ov2[h][0] * inv, ov2[h][1] * inv);
                } else {
                    const size_t pi = ((size_t)c * a.D.nh + qh) * n_splits + split;
                    *reinterpret_cast<float2 *>(a.B.APO + pi * HD + 8 * j + 2 * t) = make_float2(ov2[h][0], ov2[h][1]);
                    if (j == 0 && t == 0) *reinterpret_cast<float2 *>(a.B.APML + pi * 2) = make_float2(Mv[h], Lv[h]);
                }
            }
        }
        __syncthreads();
    }

    if (n_splits > 1) {
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int ticket = atomicAdd(a.B.ACNT + blockIdx.z * a.D.nkv + kvh, 1);
            s_last = (ticket == n_splits - 1);
            if (s_last) a.B.ACNT[blockIdx.z * a.D.nkv + kvh] = 0;     // ready for the next launch
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            // merge the splits of every (row, head) of this kv head in split order
            for (int e = tid; e < R * (HD / 4); e += NW * 32) {
                const int row = e / (HD / 4), d4 = (e - row * (HD / 4)) * 4;
                const int hq = row / ms, i = row - hq * ms;
                const int c = seg.row0 + i, qh = kvh * group + hq;
                const size_t pi = ((size_t)c * a.D.nh + qh) * n_splits;
                // all loads first (n_splits <= 16), then the arithmetic: two memory latencies in total
                uint2 mlv[16];
                uint4 ovv[16];
#pragma unroll
                for (int s = 0; s < 16; ++s) {
                    const int se = s < n_splits ? s : n_splits - 1;        // clamped: unused slots are masked below
                    mlv[s] = ldg_act8(a.B.APML + (pi + se) * 2);
                    ovv[s] = ldg_act16(a.B.APO + (pi + se) * HD + d4);
                }
                float M = -INFINITY;
#pragma unroll
                for (int s = 0; s < 16; ++s) {
                    if (s >= n_splits) mlv[s].x = 0xff800000u;              // -inf: weight 0
                    M = fmaxf(M, __uint_as_float(mlv[s].x));
                }
                float l = 0.f, o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
#pragma unroll
                for (int s = 0; s < 16; ++s) {
                    const float f = exp2f(__uint_as_float(mlv[s].x) - M);
                    l += f * __uint_as_float(mlv[s].y);
                    o0 += f * __uint_as_float(ovv[s].x); o1 += f * __uint_as_float(ovv[s].y);
                    o2 += f * __uint_as_float(ovv[s].z); o3 += f * __uint_as_float(ovv[s].w);
                }
                const float inv = 1.f / l;
                uint2 pk;
                pk.x = pack_bf16(o0 * inv, o1 * inv);
                pk.y = pack_bf16(o2 * inv, o3 * inv);
                *reinterpret_cast<uint2 *>(a.B.ATT + (size_t)c * qdim + qh * HD + d4) = pk;
            }
        }
    }
}

template <int HD>
cudaError_t launch_one(const AttnArgs &a, int n_seg, cudaStream_t st, bool pdl) {
    const size_t smem = sizeof(float) * ((size_t)NW * 32 * (HD / 8) * 4 + (size_t)NW * 32 * 4);
    auto kern = attention_kernel<HD>;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.n_splits, a.D.nkv, n_seg);
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

}  // namespace

// Key-range splits for a pass whose longest sequence holds `pages` pages, with `n_units` (segment, kv
// head) pairs and query tiles processed `tiles_par` at a time (so 8 / tiles_par warps walk the pages).
int attention_splits(int pages, int n_units, int tiles_par, int n_sms) {
    const int lanes = NW / tiles_par;
    const int per_warp = (pages + lanes - 1) / lanes;   // pages a warp walks if the key range is not split
    if (per_warp <= 2) return 1;                        // one or two page latencies, no cross-CTA merge
    // the kernel keeps one CTA per SM resident: stay within one wave, aim at two pages per warp
    int ns = (per_warp + 1) / 2;
    const int one_wave = n_sms / n_units;
    if (ns > one_wave) ns = one_wave;
    return ns > 16 ? 16 : (ns < 1 ? 1 : ns);
}

cudaError_t launch_attention(const AttnArgs &a, int n_seg, cudaStream_t st, bool pdl) {
    if (a.D.hd == 128) return launch_one<128>(a, n_seg, st, pdl);
    if (a.D.hd == 64) return launch_one<64>(a, n_seg, st, pdl);
    return cudaErrorInvalidValue;
}
