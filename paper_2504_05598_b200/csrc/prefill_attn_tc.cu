// Causal attention of a prefill chunk on the 5th-generation tensor cores (head dimension 128).
//
// One CTA = 128 query rows of one query head.  Keys and values come from the paged cache in blocks of 64
// keys (four pages): the key pages [16 tokens][128 dims] and the value pages, which the cache stores transposed
// ([128 dims][16 tokens]), are exactly the K-major operand tiles tcgen05.mma wants, so TMA copies them as they lie
// (cp.async.bulk.tensor over 5-d maps of the cache, 128-byte swizzle for keys, 32-byte swizzle for values, every
// CTA loading its own tiles) and nothing is transposed.  Per key block:
//   S = Q K^T        16 MMAs (M 128, N 64, K 16) into one of two 64-column accumulators in tensor memory;
//   softmax          four warps, one thread per query row: tcgen05.ld of the row's 64 scores, scale, causal mask,
//                    p = 2^(s - m) against a lazily raised reference maximum m (the running output in tensor
//                    memory is rescaled only when the row maximum has grown by more than 2^8), probabilities
//                    written to shared memory in the swizzled K-major layout;
//   O += P V         8 MMAs (M 128, N 128, K 16: one page each) into a 128-column accumulator.
// Queries and probabilities enter their products as bf16 high + low pairs (two MMAs each), like every other
// matrix input of the layer.  Roles: warp 0 issues the TMA copies (three key/value stages), warp 1 the MMAs (the
// scores of block j + 1 are issued before the probabilities of block j are waited for), warps 2-5 the softmax and
// the final normalisation, which stores the output as a high + low pair for the O-projection.
// Every mbarrier wait is bounded and also gives up as soon as another role has recorded an error; the error word
// is reported by the host as DEL_ETIMEOUT.  Tensor memory is always released.
#include <cuda.h>

#include <cstring>

#include "kernels.h"
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int HD = 128, BQ = 128, BKEY = 64, KV_STAGES = 3;
constexpr int Q_PART = BQ * 128;                 // one 64-dim k-block of the query tile, [128 rows][128 B]: 16 KB
constexpr int Q_BYTES = 4 * Q_PART;              // high part k-blocks 0 / 1, low part k-blocks 0 / 1
constexpr int K_BYTES = 2 * BKEY * 128;          // two k-blocks of [64 keys][128 B]
constexpr int V_BYTES = 4 * HD * 32;             // four pages of [128 dims][32 B]
constexpr int KV_STAGE = K_BYTES + V_BYTES;      // 32 KB
constexpr int P_PART = BQ * 128;                 // [128 rows][64 keys] bf16
constexpr int P_BYTES = 2 * P_PART;              // high and low part
constexpr int SMEM_BYTES = Q_BYTES + KV_STAGES * KV_STAGE + P_BYTES + 1024;
constexpr int THREADS = 192;
constexpr uint32_t TMEM_COLS = 256;              // S buffers at columns 0 and 64, O at 128..255
constexpr float RESCALE_STEP = 8.f;              // log2 units

struct Maps {
    CUtensorMap qh, ql;        // queries [rows][nh * 128], high / low part, box 64 x 128
    CUtensorMap k, v;          // key / value pages of the cache (5-d), boxes 64 x 16 and 16 x 128
};

struct Params {
    Dims D;
    bf16 *ATT, *ATTL;
    const int32_t *PT;
    int32_t M, layer, seq, pos0;
    int32_t *err;
};

__device__ __forceinline__ bool wait_or_err(uint64_t *b, uint32_t parity, volatile int *err) {
    for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
        if (mbar_try(b, parity)) return true;
        if ((i & 255u) == 255u && *err) return false;
    }
    return false;
}
__device__ __forceinline__ void tma_load_5d(void *dst, const CUtensorMap *map, int c0, int c1, int c2, int c3, int c4, uint64_t *bar) {
    asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(smem_u32(bar)) : "memory");
}
// K-major operand tile with 32-byte swizzle: rows of 32 bytes, 8-row groups 256 bytes apart
__device__ __forceinline__ uint64_t umma_desc_sw32(uint32_t smem_addr) {
    uint64_t lo = ((smem_addr & 0x3FFFFu) >> 4) | (1u << 16);
    uint64_t hi = (256u >> 4) | (1u << 14) | (6u << 29);
    return lo | (hi << 32);
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
                 "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
                   "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
                   "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
                 : "memory");
}
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(THREADS, 1) prefill_attention_tc_kernel(const __grid_constant__ Maps maps, const Params p) {
    extern __shared__ unsigned char smem_dyn[];
    __shared__ __align__(8) uint64_t q_full, kv_full[KV_STAGES], kv_empty[KV_STAGES], s_full[2], s_empty[2], p_full, o_done;
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile int s_err;
    unsigned char *base = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    unsigned char *q_sm = base, *kv_sm = base + Q_BYTES, *p_sm = kv_sm + KV_STAGES * KV_STAGE;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(&q_full, 1);
        for (int s = 0; s < KV_STAGES; ++s) { mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&s_full[b], 1); mbar_init(&s_empty[b], 4); }
        mbar_init(&p_full, 4);
        mbar_init(&o_done, 1);
        s_err = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_s;

    pdl_launch();
    pdl_wait();

    const int q0 = blockIdx.x * BQ, head = blockIdx.y, kvh = head / (p.D.nh / p.D.nkv);
    const int last_row = min(q0 + BQ, p.M) - 1;                 // last query row of the tile that exists
    const int n_kb = (p.pos0 + last_row) / BKEY + 1;            // key blocks up to that row's own position

    if (warp == 0) {
        if (lane == 0) {
            mbar_expect_tx(&q_full, Q_BYTES);
            for (int part = 0; part < 2; ++part)
                for (int kb = 0; kb < 2; ++kb)
                    tma_load_2d(q_sm + (part * 2 + kb) * Q_PART, part ? &maps.ql : &maps.qh, head * HD + kb * 64, q0, &q_full);
            const int32_t *pt = p.PT + p.seq * p.D.pages_per_seq;
            for (int j = 0; j < n_kb; ++j) {
                const int s = j % KV_STAGES;
                if (j >= KV_STAGES && !wait_or_err(&kv_empty[s], ((j / KV_STAGES) & 1) ^ 1, &s_err)) { if (!s_err) s_err = 1; break; }
                mbar_expect_tx(&kv_full[s], KV_STAGE);
                unsigned char *kst = kv_sm + (size_t)s * KV_STAGE, *vst = kst + K_BYTES;
                for (int pg = 0; pg < 4; ++pg) {
                    const int pi = j * 4 + pg;
                    const int page = pi < p.D.pages_per_seq ? pt[pi] : 0;      // (pages past the sequence: any page, masked)
                    tma_load_5d(kst + pg * 2048, &maps.k, 0, 0, kvh, p.layer - 1, page, &kv_full[s]);
                    tma_load_5d(kst + 8192 + pg * 2048, &maps.k, 64, 0, kvh, p.layer - 1, page, &kv_full[s]);
                    tma_load_5d(vst + pg * 4096, &maps.v, 0, 0, kvh, p.layer - 1, page, &kv_full[s]);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // instruction descriptors: fp32 accumulate, bf16 x bf16, both operands K-major, M = 128, N = 64 / 128
            const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BKEY >> 3) << 17) | ((uint32_t)(BQ >> 4) << 24);
            const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(HD >> 3) << 17) | ((uint32_t)(BQ >> 4) << 24);
            const uint32_t q_addr = smem_u32(q_sm), p_addr = smem_u32(p_sm);
            bool ok = wait_or_err(&q_full, 0, &s_err);
            if (!ok && !s_err) s_err = 2;
            auto issue_scores = [&](int j) -> bool {
                const int s = j % KV_STAGES, buf = j & 1;
                if (!wait_or_err(&kv_full[s], (j / KV_STAGES) & 1, &s_err)) { if (!s_err) s_err = 3; return false; }
                if (j >= 2 && !wait_or_err(&s_empty[buf], ((j >> 1) & 1) ^ 1, &s_err)) { if (!s_err) s_err = 4; return false; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t k_addr = smem_u32(kv_sm + (size_t)s * KV_STAGE);
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BKEY);
#pragma unroll
                for (int part = 0; part < 2; ++part)
#pragma unroll
                    for (int kb = 0; kb < 2; ++kb) {
                        const uint64_t da = umma_desc(q_addr + (part * 2 + kb) * Q_PART), db = umma_desc(k_addr + kb * 8192);
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc_s, (part | kb | k) != 0);
                    }
                umma_commit(&s_full[buf]);
                return true;
            };
            if (ok) ok = issue_scores(0);
            for (int j = 0; ok && j < n_kb; ++j) {
                if (j + 1 < n_kb) ok = issue_scores(j + 1);
                if (!ok) break;
                if (!wait_or_err(&p_full, j & 1, &s_err)) { if (!s_err) s_err = 5; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const int s = j % KV_STAGES;
                const uint32_t v_addr = smem_u32(kv_sm + (size_t)s * KV_STAGE + K_BYTES);
#pragma unroll
                for (int part = 0; part < 2; ++part) {
                    const uint64_t da = umma_desc(p_addr + part * P_PART);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_bf16(tmem_base + 128u, da + 2 * kk, umma_desc_sw32(v_addr + kk * 4096), idesc_o, (j | part | kk) != 0);
                }
                umma_commit(&kv_empty[s]);       // the stage's keys and values have been read
                umma_commit(&o_done);            // the output holds blocks 0..j; the probabilities may be overwritten
            }
        }
    } else {
        const int q = warp & 3;                  // TMEM lane quarter this warp may access
        const int row = q * 32 + lane, qrow = q0 + row;
        const int qpos = p.pos0 + qrow;          // keys up to this position are visible
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const float sc = rsqrtf((float)HD) * 1.4426950408889634f;
        unsigned char *prow_hi = p_sm + row * 128, *prow_lo = prow_hi + P_PART;
        float m_ref = -INFINITY, l = 0.f;
        bool ok = true;
        for (int j = 0; j < n_kb; ++j) {
            const int buf = j & 1;
            if (!wait_or_err(&s_full[buf], (j >> 1) & 1, &s_err)) { if (!s_err) s_err = 6; ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            uint32_t r0[32], r1[32];
            tmem_ld32(lane_addr + (uint32_t)(buf * BKEY), r0);
            tmem_ld32(lane_addr + (uint32_t)(buf * BKEY + 32), r1);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_empty[buf]);
            // scores in units of log2, causal mask, block maximum
            const int key0 = j * BKEY;
            float sv[64], mx = -INFINITY;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                sv[e] = key0 + e <= qpos ? __uint_as_float(r0[e]) * sc : -INFINITY;
                sv[32 + e] = key0 + 32 + e <= qpos ? __uint_as_float(r1[e]) * sc : -INFINITY;
                mx = fmaxf(mx, fmaxf(sv[e], sv[32 + e]));
            }
            // reference maximum: raised only when the row maximum has outgrown it by RESCALE_STEP
            float alpha = 1.f;
            if (m_ref == -INFINITY) {
                m_ref = mx;                                   // (block 0 always holds key 0, visible to every row)
            } else if (mx > m_ref + RESCALE_STEP) {
                alpha = ex2f(m_ref - mx);
                m_ref = mx;
                l *= alpha;
            }
            float psum = 0.f;
#pragma unroll
            for (int e = 0; e < 64; ++e) { sv[e] = ex2f(sv[e] - m_ref); psum += sv[e]; }
            l += psum;
            // the previous block's P*V has read the probabilities and updated the output
            if (j > 0 && !wait_or_err(&o_done, (j - 1) & 1, &s_err)) { if (!s_err) s_err = 7; ok = false; break; }
            if (__any_sync(0xffffffffu, alpha != 1.f)) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                for (int c0 = 0; c0 < HD; c0 += 32) {
                    uint32_t o[32];
                    tmem_ld32(lane_addr + 128u + (uint32_t)c0, o);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                    tmem_st32(lane_addr + 128u + (uint32_t)c0, o);
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            }
            // probabilities as bf16 high + low parts, K-major rows of 128 bytes with the 128-byte swizzle
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                uint4 hi, lo;
                split_bf16x2(sv[8 * c + 0], sv[8 * c + 1], hi.x, lo.x);
                split_bf16x2(sv[8 * c + 2], sv[8 * c + 3], hi.y, lo.y);
                split_bf16x2(sv[8 * c + 4], sv[8 * c + 5], hi.z, lo.z);
                split_bf16x2(sv[8 * c + 6], sv[8 * c + 7], hi.w, lo.w);
                const int off = (c ^ (row & 7)) << 4;
                *reinterpret_cast<uint4 *>(prow_hi + off) = hi;
                *reinterpret_cast<uint4 *>(prow_lo + off) = lo;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // visible to the tensor core's reads
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&p_full);
        }
        if (ok && !wait_or_err(&o_done, (n_kb - 1) & 1, &s_err)) { if (!s_err) s_err = 8; ok = false; }
        if (ok) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const float inv = 1.f / l;
            const size_t out = (size_t)qrow * (p.D.nh * HD) + head * HD;
            for (int c0 = 0; c0 < HD; c0 += 32) {
                uint32_t o[32];
                tmem_ld32(lane_addr + 128u + (uint32_t)c0, o);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (qrow < p.M) {
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 hi, lo;
                        split_bf16x2(__uint_as_float(o[e + 0]) * inv, __uint_as_float(o[e + 1]) * inv, hi.x, lo.x);
                        split_bf16x2(__uint_as_float(o[e + 2]) * inv, __uint_as_float(o[e + 3]) * inv, hi.y, lo.y);
                        split_bf16x2(__uint_as_float(o[e + 4]) * inv, __uint_as_float(o[e + 5]) * inv, hi.z, lo.z);
                        split_bf16x2(__uint_as_float(o[e + 6]) * inv, __uint_as_float(o[e + 7]) * inv, hi.w, lo.w);
                        *reinterpret_cast<uint4 *>(p.ATT + out + c0 + e) = hi;
                        *reinterpret_cast<uint4 *>(p.ATTL + out + c0 + e) = lo;
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && s_err) atomicMax(p.err, (int)s_err);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *q = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &q, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(q);
    }
    return fn;
}

}  // namespace

bool prefill_attention_tc_supported(const Dims &D) { return D.hd == HD; }

// 5-d maps of the paged cache: keys [page][layer][kv head][16 tokens][128 dims] in boxes of 16 tokens x 64 dims
// (128-byte swizzle), values [page][layer][kv head][128 dims][16 tokens] in boxes of 128 dims x 16 tokens (32-byte
// swizzle).  Both 128-byte blobs (CUtensorMap).
int prefill_attention_tc_make_maps(void *map_k, void *map_v, const void *k_pages, const void *v_pages, const Dims &D, int n_pages) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || D.hd != HD) return -1;
    const cuuint64_t L = (cuuint64_t)D.L, nkv = (cuuint64_t)D.nkv;
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    {
        cuuint64_t dims[5] = {HD, 16, nkv, L, (cuuint64_t)n_pages};
        cuuint64_t strides[4] = {HD * 2, 16 * HD * 2, nkv * 16 * HD * 2, L * nkv * 16 * HD * 2};
        cuuint32_t box[5] = {64, 16, 1, 1, 1};
        if (fn(reinterpret_cast<CUtensorMap *>(map_k), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(k_pages), dims, strides, box,
               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return -2;
    }
    {
        cuuint64_t dims[5] = {16, HD, nkv, L, (cuuint64_t)n_pages};
        cuuint64_t strides[4] = {32, HD * 32, nkv * HD * 32, L * nkv * HD * 32};
        cuuint32_t box[5] = {16, HD, 1, 1, 1};
        if (fn(reinterpret_cast<CUtensorMap *>(map_v), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(v_pages), dims, strides, box,
               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return -3;
    }
    return 0;
}

// map_qh / map_ql: maps of the chunk's query buffers made by lmhead_tc_make_map (boxes of 128 rows x 64 elements)
cudaError_t launch_prefill_attention_tc(const void *map_qh, const void *map_ql, const void *map_k, const void *map_v,
                                        const PfAttnArgs &a, int32_t *err, cudaStream_t st, bool pdl) {
    Maps maps;
    maps.qh = *reinterpret_cast<const CUtensorMap *>(map_qh);
    maps.ql = *reinterpret_cast<const CUtensorMap *>(map_ql);
    maps.k = *reinterpret_cast<const CUtensorMap *>(map_k);
    maps.v = *reinterpret_cast<const CUtensorMap *>(map_v);
    Params p;
    memset(&p, 0, sizeof(p));
    p.D = a.D; p.ATT = a.ATT; p.ATTL = a.ATTL; p.PT = a.PT; p.M = a.M; p.layer = a.layer; p.seq = a.seq; p.pos0 = a.pos0;
    p.err = err;
    static SmemAttrOnce attr;
    {
        cudaError_t e = attr.set(prefill_attention_tc_kernel, SMEM_BYTES);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((a.M + BQ - 1) / BQ, a.D.nh);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, prefill_attention_tc_kernel, maps, p);
}
