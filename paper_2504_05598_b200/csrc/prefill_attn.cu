// Causal attention over a chunk of prompt positions during the bulk prefill (flash style: one pass over the
// keys with an online softmax, nothing of size rows x keys ever stored).
//
// One CTA = 64 query rows of one query head (4 warps x 16 rows).  Keys come in blocks of 64 (four 16-token pages
// of the paged cache): K rows [key][hd] and the per-page transposed V [hd][16] are copied as they lie into
// shared memory with cp.async (two stages), padded so that ldmatrix reads are free of bank conflicts; both are
// then already in the "column" operand layout of mma.sync m16n8k16 (scores: n = key, k = feature; output:
// n = feature, k = key), so no transposition is needed anywhere.  Scores and the output accumulate in fp32, the
// probabilities enter the second product as bf16, like in the decode attention kernel.
#include "kernels.h"

namespace {

constexpr int PA_THREADS = 128;
constexpr int BQ = 64, BKEY = 64;

template <int HD> struct Lay {
    static constexpr int KROW = HD + 8;                    // padded K row (elements)
    static constexpr int VROW = 16 + 8;                    // padded V^T row: 16 keys of one feature (elements)
    static constexpr int K_ELEMS = BKEY * KROW;
    static constexpr int V_ELEMS = (BKEY / 16) * HD * VROW;
    static constexpr int STAGE_ELEMS = K_ELEMS + V_ELEMS;
    static constexpr int SMEM_BYTES = 2 * STAGE_ELEMS * 2;
};

__device__ __forceinline__ void ldsm4(uint32_t (&r)[4], const void *p) {
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}

template <int HD>
__global__ void __launch_bounds__(PA_THREADS) prefill_attention_kernel(const __grid_constant__ PfAttnArgs a) {
    using L = Lay<HD>;
    extern __shared__ __align__(16) unsigned char raw[];
    bf16 *sm = reinterpret_cast<bf16 *>(raw);
    pdl_launch();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int qb = (int)gridDim.x - 1 - (int)blockIdx.x;         // the blocks with the most keys start first
    const int head = blockIdx.y, kvh = head / (a.D.nh / a.D.nkv);
    const int q0 = qb * BQ, qdim = a.D.nh * HD;
    const int kv_len = a.pos0 + a.M;                             // keys that exist
    const int last_row = min(q0 + BQ, a.M) - 1;
    const int n_kb = (a.pos0 + last_row) / BKEY + 1;
    const int32_t *pt = a.PT + (size_t)a.seq * a.D.pages_per_seq;
    pdl_wait();

    // copies key block kb into stage st
    auto load_block = [&](int kb, int st) {
        bf16 *ks = sm + st * L::STAGE_ELEMS, *vs = ks + L::K_ELEMS;
        constexpr int KCH = HD / 8;                              // 16-byte chunks per K row
#pragma unroll
        for (int c = tid; c < BKEY * KCH; c += PA_THREADS) {
            const int key = c / KCH, ch = c - key * KCH, page = kb * 4 + (key >> 4);
            const bool ok = page * 16 < kv_len;
            const int pg = ok ? pt[page] : 0;
            const bf16 *src = a.KP + ((((size_t)pg * a.D.L + (a.layer - 1)) * a.D.nkv + kvh) * 16 + (key & 15)) * HD + ch * 8;
            cp_async16(ks + key * L::KROW + ch * 8, src, ok);
        }
#pragma unroll
        for (int c = tid; c < 4 * HD * 2; c += PA_THREADS) {
            const int p = c / (HD * 2), r = c - p * HD * 2, dim = r >> 1, half = r & 1, page = kb * 4 + p;
            const bool ok = page * 16 < kv_len;
            const int pg = ok ? pt[page] : 0;
            const bf16 *src = a.VP + ((((size_t)pg * a.D.L + (a.layer - 1)) * a.D.nkv + kvh) * HD + dim) * 16 + half * 8;
            cp_async16(vs + (p * HD + dim) * L::VROW + half * 8, src, ok);
        }
        cp_async_commit();
    };

    load_block(0, 0);

    // this warp's query rows as A fragments: rows g and g + 8 of its 16
    constexpr int KS = HD / 16;
    // (queries and probabilities enter their products as bf16 high + low pairs: two MMAs each)
    uint32_t qf[KS][4], ql[KS][4];
    const int r0 = q0 + warp * 16 + g, r1 = r0 + 8;
    {
        const size_t o0 = (size_t)r0 * qdim + head * HD + 2 * t, o1 = (size_t)r1 * qdim + head * HD + 2 * t;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            qf[ks][0] = r0 < a.M ? *reinterpret_cast<const uint32_t *>(a.Q + o0 + 16 * ks) : 0u;
            qf[ks][1] = r1 < a.M ? *reinterpret_cast<const uint32_t *>(a.Q + o1 + 16 * ks) : 0u;
            qf[ks][2] = r0 < a.M ? *reinterpret_cast<const uint32_t *>(a.Q + o0 + 16 * ks + 8) : 0u;
            qf[ks][3] = r1 < a.M ? *reinterpret_cast<const uint32_t *>(a.Q + o1 + 16 * ks + 8) : 0u;
            ql[ks][0] = r0 < a.M ? *reinterpret_cast<const uint32_t *>(a.QL + o0 + 16 * ks) : 0u;
            ql[ks][1] = r1 < a.M ? *reinterpret_cast<const uint32_t *>(a.QL + o1 + 16 * ks) : 0u;
            ql[ks][2] = r0 < a.M ? *reinterpret_cast<const uint32_t *>(a.QL + o0 + 16 * ks + 8) : 0u;
            ql[ks][3] = r1 < a.M ? *reinterpret_cast<const uint32_t *>(a.QL + o1 + 16 * ks + 8) : 0u;
        }
    }
    const int qp0 = a.pos0 + r0, qp1 = a.pos0 + r1;              // positions of the two rows
    const float sc = rsqrtf((float)HD) * 1.4426950408889634f;    // scores in units of log2
    float O[HD / 8][4];
#pragma unroll
    for (int j = 0; j < HD / 8; ++j) O[j][0] = O[j][1] = O[j][2] = O[j][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

    for (int kb = 0; kb < n_kb; ++kb) {
        const int st = kb & 1;
        if (kb + 1 < n_kb) {
            load_block(kb + 1, st ^ 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const bf16 *ks_ = sm + st * L::STAGE_ELEMS, *vs_ = ks_ + L::K_ELEMS;
        // a warp whose rows all lie before this block's first key has nothing to add (causal)
        const bool live = kb * BKEY <= a.pos0 + q0 + warp * 16 + 15;
        if (live) {
            float S[BKEY / 8][4];
#pragma unroll
            for (int j = 0; j < BKEY / 8; ++j) S[j][0] = S[j][1] = S[j][2] = S[j][3] = 0.f;
            // scores: ldmatrix.x4 = B fragments (k-step ks) of key tiles j and j + 1
            const int mi = lane >> 3, mr = lane & 7;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks)
#pragma unroll
                for (int j = 0; j < BKEY / 8; j += 2) {
                    uint32_t b[4];
                    ldsm4(b, ks_ + (8 * (j + (mi >> 1)) + mr) * L::KROW + 16 * ks + 8 * (mi & 1));
                    mma_bf16_16816(S[j], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b[0], b[1]);
                    mma_bf16_16816(S[j + 1], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b[2], b[3]);
                    mma_bf16_16816(S[j], ql[ks][0], ql[ks][1], ql[ks][2], ql[ks][3], b[0], b[1]);
                    mma_bf16_16816(S[j + 1], ql[ks][0], ql[ks][1], ql[ks][2], ql[ks][3], b[2], b[3]);
                }
            // scale, causal mask (only blocks that reach past a row's position need it), running maximum
            const bool diag = kb * BKEY + BKEY - 1 > a.pos0 + q0 + warp * 16;
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int j = 0; j < BKEY / 8; ++j) {
                const int kp = kb * BKEY + 8 * j + 2 * t;
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    S[j][e] = (diag && kp + e > qp0) ? -INFINITY : S[j][e] * sc;
                    S[j][2 + e] = (diag && kp + e > qp1) ? -INFINITY : S[j][2 + e] * sc;
                }
                mx0 = fmaxf(mx0, fmaxf(S[j][0], S[j][1]));
                mx1 = fmaxf(mx1, fmaxf(S[j][2], S[j][3]));
            }
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
            const float n0 = fmaxf(m0, mx0), n1 = fmaxf(m1, mx1);
            const float base0 = n0 == -INFINITY ? 0.f : n0, base1 = n1 == -INFINITY ? 0.f : n1;
            const float al0 = exp2f(m0 - base0), al1 = exp2f(m1 - base1);
            m0 = n0; m1 = n1;
            float ps0 = 0.f, ps1 = 0.f;
            uint32_t pf[BKEY / 8][2], pl[BKEY / 8][2];             // probabilities as bf16 pairs (high, low): rows g, g + 8
#pragma unroll
            for (int j = 0; j < BKEY / 8; ++j) {
                const float p00 = exp2f(S[j][0] - base0), p01 = exp2f(S[j][1] - base0);
                const float p10 = exp2f(S[j][2] - base1), p11 = exp2f(S[j][3] - base1);
                ps0 += p00 + p01;
                ps1 += p10 + p11;
                split_bf16x2(p00, p01, pf[j][0], pl[j][0]);
                split_bf16x2(p10, p11, pf[j][1], pl[j][1]);
            }
            l0 = l0 * al0 + ps0;
            l1 = l1 * al1 + ps1;
#pragma unroll
            for (int j = 0; j < HD / 8; ++j) { O[j][0] *= al0; O[j][1] *= al0; O[j][2] *= al1; O[j][3] *= al1; }
            // output: k-step kk = page kk of the block; ldmatrix.x4 = B fragments of feature tiles jd and jd + 1
#pragma unroll
            for (int kk = 0; kk < BKEY / 16; ++kk)
#pragma unroll
                for (int jd = 0; jd < HD / 8; jd += 2) {
                    uint32_t b[4];
                    ldsm4(b, vs_ + (kk * HD + 8 * (jd + (mi >> 1)) + mr) * L::VROW + 8 * (mi & 1));
                    mma_bf16_16816(O[jd], pf[2 * kk][0], pf[2 * kk][1], pf[2 * kk + 1][0], pf[2 * kk + 1][1], b[0], b[1]);
                    mma_bf16_16816(O[jd + 1], pf[2 * kk][0], pf[2 * kk][1], pf[2 * kk + 1][0], pf[2 * kk + 1][1], b[2], b[3]);
                    mma_bf16_16816(O[jd], pl[2 * kk][0], pl[2 * kk][1], pl[2 * kk + 1][0], pl[2 * kk + 1][1], b[0], b[1]);
                    mma_bf16_16816(O[jd + 1], pl[2 * kk][0], pl[2 * kk][1], pl[2 * kk + 1][0], pl[2 * kk + 1][1], b[2], b[3]);
                }
        }
        __syncthreads();                                           // the stage is free for the block after next
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const float i0 = 1.f / l0, i1 = 1.f / l1;
#pragma unroll
    for (int j = 0; j < HD / 8; ++j) {
        // stored as high + low bf16 parts: the O-projection takes its input as such a pair
        uint32_t hi, lo;
        if (r0 < a.M) {
            split_bf16x2(O[j][0] * i0, O[j][1] * i0, hi, lo);
            *reinterpret_cast<uint32_t *>(a.ATT + (size_t)r0 * qdim + head * HD + 8 * j + 2 * t) = hi;
            *reinterpret_cast<uint32_t *>(a.ATTL + (size_t)r0 * qdim + head * HD + 8 * j + 2 * t) = lo;
        }
        if (r1 < a.M) {
            split_bf16x2(O[j][2] * i1, O[j][3] * i1, hi, lo);
            *reinterpret_cast<uint32_t *>(a.ATT + (size_t)r1 * qdim + head * HD + 8 * j + 2 * t) = hi;
            *reinterpret_cast<uint32_t *>(a.ATTL + (size_t)r1 * qdim + head * HD + 8 * j + 2 * t) = lo;
        }
    }
}

template <int HD>
cudaError_t launch_hd(const PfAttnArgs &a, cudaStream_t st, bool pdl) {
    static SmemAttrOnce attr;
    {
        cudaError_t e = attr.set(prefill_attention_kernel<HD>, (int)(Lay<HD>::SMEM_BYTES));
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((a.M + BQ - 1) / BQ, a.D.nh);
    cfg.blockDim = dim3(PA_THREADS);
    cfg.dynamicSmemBytes = Lay<HD>::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, prefill_attention_kernel<HD>, a);
}

}  // namespace

cudaError_t launch_prefill_attention(const PfAttnArgs &a, cudaStream_t st, bool pdl) {
    return a.D.hd == 128 ? launch_hd<128>(a, st, pdl) : launch_hd<64>(a, st, pdl);
}
