// Multi-query decode attention over the paged bf16 KV cache.
//
// One CTA = (key-range split, kv head, sequence segment).  The query rows of the segment (its 1..32
// consecutive positions times the query heads sharing this kv head) form 16-row tiles; keys are walked
// one 16-token page at a time.  Scores and the P*V product run on bf16 tensor-core MMAs with fp32
// accumulation; the softmax is the online (running max / running sum) form, its row reductions done
// with warp shuffles inside the 4-lane groups that own a row.
//
// Fragment loading without shared memory: the MMA sums over its k index, so any permutation of k used
// for both operands is allowed.  For Q*K^T a thread loads 16 contiguous bytes of a key row (and the
// same bytes of the query row) and feeds them to two MMAs.  For P*V the page stores V transposed
// ([head_dim][16 tokens]); the score tile's columns are assigned to tokens such that a thread's four
// probabilities belong to tokens 4t..4t+3, which are 8 contiguous bytes of a V^T row.
//
// Splits write (max, sum, unnormalised output) partials; the last CTA to arrive for a (segment, kv
// head) merges them in split order, so the result does not depend on scheduling.
#include "kernels.h"

namespace {

constexpr int ATT_THREADS = 128;
constexpr float LOG2E = 1.4426950408889634f;

template <int HD>
__global__ void __launch_bounds__(ATT_THREADS) attention_kernel(const AttnArgs a) {
    constexpr int KS = HD / 32;       // 16-byte chunks per thread along head_dim
    constexpr int NJ = HD / 8;        // output n-tiles
    extern __shared__ __align__(16) float sm[];
    float *sm_o = sm;                               // [4][32][NJ*4]
    float *sm_ml = sm + 4 * 32 * NJ * 4;            // [4][32][4]
    __shared__ int s_last;

    pdl_launch();
    pdl_wait();

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const PassPlan *plan = a.plan;
    const Segment seg = plan->seg[blockIdx.z];
    const int kvh = blockIdx.y, split = blockIdx.x, n_splits = a.n_splits;
    const int ms = seg.nrows, group = a.D.nh / a.D.nkv;
    const int R = ms * group, n_mt = (R + 15) >> 4;
    const int kv_len = seg.pos0 + ms;
    const int n_pages = (kv_len + 15) >> 4;
    const int pps = (n_pages + n_splits - 1) / n_splits;
    const int p_begin = split * pps, p_end = min(n_pages, p_begin + pps);
    const int P = n_mt >= 4 ? 4 : (n_mt >= 2 ? (n_mt == 2 ? 2 : 4) : 1);
    const int n_kl = 4 / P, kl = warp / P;
    const float sc = rsqrtf((float)HD) * LOG2E;
    const int32_t *pt = a.B.PT + seg.seq * a.D.pages_per_seq;
    const size_t page_stride = (size_t)a.D.L * a.D.nkv * 16 * HD;
    const size_t head_off = ((size_t)(a.layer - 1) * a.D.nkv + kvh) * 16 * HD;
    const int qdim = a.D.nh * HD;

    for (int mt = warp % P; mt < n_mt; mt += P) {
        // rows of this thread: rr0 = mt*16+g, rr1 = rr0+8, ordered head-major: rr = hq*ms + i
        int rr[2] = {mt * 16 + g, mt * 16 + g + 8};
        int ri[2], rh[2];
        bool rv[2];
        uint4 qf[2][KS];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            rv[h] = rr[h] < R;
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

        for (int p = p_begin + kl; p < p_end; p += n_kl) {
            const int pg = pt[p];
            const bf16 *kpage = a.B.KP + (size_t)pg * page_stride + head_off;
            const bf16 *vpage = a.B.VP + (size_t)pg * page_stride + head_off;
            const int key0 = 4 * (g >> 1) + (g & 1);       // token of score-tile 0 column g; tile 1: +2
            uint4 kf[2][KS];
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                kf[0][ks] = ldg_act16(kpage + key0 * HD + 32 * ks + 8 * t);
                kf[1][ks] = ldg_act16(kpage + (key0 + 2) * HD + 32 * ks + 8 * t);
            }
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
            for (int j = 0; j < NJ; ++j) {
                const uint2 vf = ldg_act8(vpage + (8 * j + g) * 16 + 4 * t);
                mma_bf16_16816(O[j], pa0, pa1, pa2, pa3, vf.x, vf.y);
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
            l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
        }

        if (n_kl > 1) {          // warps that share this query tile merge through shared memory
            float *so = sm_o + (size_t)(warp * 32 + lane) * NJ * 4;
#pragma unroll
            for (int j = 0; j < NJ; ++j) *reinterpret_cast<float4 *>(so + 4 * j) = make_float4(O[j][0], O[j][1], O[j][2], O[j][3]);
            *reinterpret_cast<float4 *>(sm_ml + (warp * 32 + lane) * 4) = make_float4(m_run[0], l_run[0], m_run[1], l_run[1]);
            __syncthreads();
            if (kl == 0) {
                float M[2] = {m_run[0], m_run[1]};
                for (int k2 = 1; k2 < n_kl; ++k2) {
                    const float4 ml = *reinterpret_cast<float4 *>(sm_ml + ((warp + k2 * P) * 32 + lane) * 4);
                    M[0] = fmaxf(M[0], ml.x);
                    M[1] = fmaxf(M[1], ml.z);
                }
                const float b0 = M[0] == -INFINITY ? 0.f : M[0], b1 = M[1] == -INFINITY ? 0.f : M[1];
                float f0 = exp2f(m_run[0] - b0), f1 = exp2f(m_run[1] - b1);
                l_run[0] *= f0; l_run[1] *= f1;
#pragma unroll
                for (int j = 0; j < NJ; ++j) { O[j][0] *= f0; O[j][1] *= f0; O[j][2] *= f1; O[j][3] *= f1; }
                for (int k2 = 1; k2 < n_kl; ++k2) {
                    const int w2 = warp + k2 * P;
                    const float4 ml = *reinterpret_cast<float4 *>(sm_ml + (w2 * 32 + lane) * 4);
                    f0 = exp2f(ml.x - b0); f1 = exp2f(ml.z - b1);
                    l_run[0] += ml.y * f0; l_run[1] += ml.w * f1;
                    const float *so2 = sm_o + (size_t)(w2 * 32 + lane) * NJ * 4;
#pragma unroll
                    for (int j = 0; j < NJ; ++j) {
                        const float4 o2 = *reinterpret_cast<const float4 *>(so2 + 4 * j);
                        O[j][0] += o2.x * f0; O[j][1] += o2.y * f0; O[j][2] += o2.z * f1; O[j][3] += o2.w * f1;
                    }
                }
                m_run[0] = M[0]; m_run[1] = M[1];
            }
        }
        if (kl == 0) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (!rv[h]) continue;
                const int c = seg.row0 + ri[h], qh = kvh * group + rh[h];
                if (n_splits == 1) {
                    const float inv = 1.f / l_run[h];
                    bf16 *op = a.B.ATT + (size_t)c * qdim + qh * HD + 2 * t;
#pragma unroll
                    for (int j = 0; j < NJ; ++j)
                        *reinterpret_cast<uint32_t *>(op + 8 * j) = pack_bf16(O[j][2 * h] * inv, O[j][2 * h + 1] * inv);
                } else {
                    const size_t pi = ((size_t)c * a.D.nh + qh) * n_splits + split;
                    float *op = a.B.APO + pi * HD + 2 * t;
#pragma unroll
                    for (int j = 0; j < NJ; ++j) *reinterpret_cast<float2 *>(op + 8 * j) = make_float2(O[j][2 * h], O[j][2 * h + 1]);
                    if (t == 0) *reinterpret_cast<float2 *>(a.B.APML + pi * 2) = make_float2(m_run[h], l_run[h]);
                }
            }
        }
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
            for (int e = tid; e < R * (HD / 4); e += ATT_THREADS) {
                const int row = e / (HD / 4), d4 = (e - row * (HD / 4)) * 4;
                const int hq = row / ms, i = row - hq * ms;
                const int c = seg.row0 + i, qh = kvh * group + hq;
                const size_t pi = ((size_t)c * a.D.nh + qh) * n_splits;
                float M = -INFINITY;
                for (int s = 0; s < n_splits; ++s) M = fmaxf(M, ldg_cg_f32(a.B.APML + (pi + s) * 2));
                float l = 0.f, o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
                for (int s = 0; s < n_splits; ++s) {
                    const float f = exp2f(ldg_cg_f32(a.B.APML + (pi + s) * 2) - M);
                    l += f * ldg_cg_f32(a.B.APML + (pi + s) * 2 + 1);
                    const float *op = a.B.APO + (pi + s) * HD + d4;
                    o0 += f * ldg_cg_f32(op); o1 += f * ldg_cg_f32(op + 1);
                    o2 += f * ldg_cg_f32(op + 2); o3 += f * ldg_cg_f32(op + 3);
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

}  // namespace

cudaError_t launch_attention(const AttnArgs &a, int n_seg, cudaStream_t st, bool pdl) {
    const int HD = a.D.hd;
    const size_t smem = sizeof(float) * (4 * 32 * (HD / 8) * 4 + 4 * 32 * 4);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.n_splits, a.D.nkv, n_seg);
    cfg.blockDim = dim3(ATT_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    if (HD == 128) return cudaLaunchKernelEx(&cfg, attention_kernel<128>, a);
    if (HD == 64) return cudaLaunchKernelEx(&cfg, attention_kernel<64>, a);
    return cudaErrorInvalidValue;
}
