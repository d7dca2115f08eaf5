// Prompt prefill on the 5th-generation tensor cores.
//
// The decode kernels stream every weight once per pass of at most 64 rows, which is the right trade for a
// round (1..13 rows) and the wrong one for a prompt: hundreds of positions can share one pass over the
// weights.  Here the four projections of a layer run as tiled GEMMs over up to PF_ROWS prompt positions
// at a time,  Y[M, N] = X[M, K] * W[N, K]^T,  with the layer's element-wise work fused into the epilogue:
//   QKV     1/rms of the row, rotary embedding on q and k, q -> Q buffer, k and v -> paged cache
//   OPROJ   + residual (in place), ffn-norm input, per-tile sums of squares
//   GATEUP  1/rms, SiLU(gate) * up -> activation buffer (the tile holds 128 gate and the same 128 up rows)
//   DOWN    + residual (in place), next layer's attention-norm input, per-tile sums of squares
// Of most prompt positions only the KV cache is needed later.  The last window of positions also seeds
// the acceptance statistics: the hidden state of those rows after every layer (and their embedding) is
// copied into the hidden stack, where the stacked LM head finds it.
//
// The activations enter every GEMM as a pair of bf16 values (high + low part, see common.cuh): each k-block is
// two MMAs on the same weight tile, one per part, into the same accumulator, so that the prompt's keys, values
// and hidden states carry the same accuracy as those the decode kernels make.
//
// CTA tile 128 rows x 256 output features (128 for the two d-wide projections, whose 256-wide tiles would
// fill less than half of the SMs), K blocks of 64 (one 128-byte swizzle span), same roles as
// the stacked LM head: warp 0 issues TMA loads into a 3-stage shared-memory ring, warp 1 issues
// tcgen05.mma into one of two 256-column accumulators in tensor memory, warps 2-5 read their own row
// with tcgen05.ld and run the epilogue while the next tile's MMAs proceed.  Ragged shapes (rows, N, K)
// rely on TMA zero fill plus store masks.  Every mbarrier wait is bounded.
#include <cuda.h>

#include "kernels.h"
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 3;
// a stage: high parts of the activation tile, their low parts, the weight tile
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = 2 * A_BYTES + B_BYTES;
constexpr int PF_THREADS = 192;
// O-proj and down (N = d_model) use a narrower tile, p.bn_narrow, chosen per model shape (prefill_tc_narrow)
template <int EPI> __device__ __forceinline__ int tile_n(const PfArgs &p) {
    return (EPI == PF_OPROJ || EPI == PF_DOWN) ? p.bn_narrow : BN;
}

struct PfMaps {
    CUtensorMap a, a_lo;       // activations [PF_ROWS, K], high and low parts, box 64 x 128
    CUtensorMap b0, b1, b2;    // weights [N, K]: QKV Wq / Wk / Wv (box 64 x 256); GATEUP gate / up (box 64 x 128); else b0
};

// 1/rms of a row from the producer's per-tile sums of squares
__device__ __forceinline__ float row_rscale(const float *ssp, int n_part, int d, float eps) {
    float s = 0.f;
    for (int i = 0; i < n_part; ++i) s += ldg_cg_f32(ssp + i);
    return rsqrtf(s / (float)d + eps);
}

__device__ __forceinline__ void store_bf16x32(bf16 *dst, const float (&v)[32]) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint4 w;
        w.x = pack_bf16(v[8 * q + 0], v[8 * q + 1]);
        w.y = pack_bf16(v[8 * q + 2], v[8 * q + 3]);
        w.z = pack_bf16(v[8 * q + 4], v[8 * q + 5]);
        w.w = pack_bf16(v[8 * q + 6], v[8 * q + 7]);
        *reinterpret_cast<uint4 *>(dst + 8 * q) = w;
    }
}
// the same values as high parts to `hi` and low parts to `lo`
__device__ __forceinline__ void store_split_x32(bf16 *hi, bf16 *lo, const float (&v)[32]) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint4 wh, wl;
        split_bf16x2(v[8 * q + 0], v[8 * q + 1], wh.x, wl.x);
        split_bf16x2(v[8 * q + 2], v[8 * q + 3], wh.y, wl.y);
        split_bf16x2(v[8 * q + 4], v[8 * q + 5], wh.z, wl.z);
        split_bf16x2(v[8 * q + 6], v[8 * q + 7], wh.w, wl.w);
        *reinterpret_cast<uint4 *>(hi + 8 * q) = wh;
        *reinterpret_cast<uint4 *>(lo + 8 * q) = wl;
    }
}

// ---- epilogues: one thread owns one row of the tile; taddr = this warp's lane quarter, accumulator column 0
template <int EPI>
__device__ __forceinline__ void epilogue(const PfArgs &p, uint32_t taddr, int row, int nt) {
    const bool live = row < p.M;
    const Dims &D = p.D;
    uint32_t r0[32], r1[32];
    if (EPI == PF_QKV) {
        const int hd = D.hd, half = hd >> 1;
        const int n_qt = (D.nh * hd + BN - 1) / BN, n_kt = (D.nkv * hd + BN - 1) / BN;
        const int which = nt < n_qt ? 0 : (nt < n_qt + n_kt ? 1 : 2);
        const int n0 = (nt - (which == 0 ? 0 : (which == 1 ? n_qt : n_qt + n_kt))) * BN;   // feature offset in its matrix
        const int n_out = which == 0 ? D.nh * hd : D.nkv * hd;
        const float rs = live ? row_rscale(p.SSP + (size_t)row * p.n_ssp, p.n_ssp, D.d, D.eps) : 0.f;
        const int pos = p.pos0 + (live ? row : 0);
        const int pg = p.PT[p.seq * D.pages_per_seq + (pos >> 4)], sl = pos & 15;
        if (which < 2) {
            const float *cs = p.rope_cos + (size_t)pos * half, *sn = p.rope_sin + (size_t)pos * half;
            for (int h0 = 0; h0 < BN; h0 += hd) {                // heads inside the tile
                for (int jj = 0; jj < half; jj += 32) {
                    __syncwarp();
                    tmem_ld32(taddr + (uint32_t)(h0 + jj), r0);
                    tmem_ld32(taddr + (uint32_t)(h0 + half + jj), r1);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    const int n = n0 + h0;                       // first feature of the head
                    if (!live || n >= n_out) continue;
                    float lo[32], hi[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const float a = rs * __uint_as_float(r0[e]), b = rs * __uint_as_float(r1[e]);
                        const float c = __ldg(cs + jj + e), s = __ldg(sn + jj + e);
                        lo[e] = a * c - b * s;
                        hi[e] = b * c + a * s;
                    }
                    if (which == 0) {
                        const size_t qo = (size_t)row * (D.nh * hd) + n + jj;
                        store_split_x32(p.Q + qo, p.QL + qo, lo);
                        store_split_x32(p.Q + qo + half, p.QL + qo + half, hi);
                    } else {
                        bf16 *dst = p.KP + ((((size_t)pg * D.L + (p.layer - 1)) * D.nkv + n / hd) * 16 + sl) * hd + jj;
                        store_bf16x32(dst, lo);
                        store_bf16x32(dst + half, hi);
                    }
                }
            }
        } else {
            for (int c0 = 0; c0 < BN; c0 += 32) {
                __syncwarp();
                tmem_ld32(taddr + (uint32_t)c0, r0);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (!live) continue;
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const int n = n0 + c0 + e;
                    if (n < n_out) {
                        const int kvh = n / hd, dim = n - kvh * hd;
                        p.VP[((((size_t)pg * D.L + (p.layer - 1)) * D.nkv + kvh) * hd + dim) * 16 + sl] =
                            __float2bfloat16_rn(rs * __uint_as_float(r0[e]));
                    }
                }
            }
        }
    } else if (EPI == PF_GATEUP) {
        const float rs = live ? row_rscale(p.SSPM + (size_t)row * p.n_ssp, p.n_ssp, D.d, D.eps) : 0.f;
        for (int c0 = 0; c0 < BN / 2; c0 += 32) {
            __syncwarp();
            tmem_ld32(taddr + (uint32_t)c0, r0);
            tmem_ld32(taddr + (uint32_t)(BN / 2 + c0), r1);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            const int f0 = nt * (BN / 2) + c0;
            if (!live || f0 >= D.F) continue;
            float act[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                const float g = rs * __uint_as_float(r0[e]), u = rs * __uint_as_float(r1[e]);
                act[e] = g / (1.f + __expf(-g)) * u;
            }
            bf16 *dst = p.ACT + (size_t)row * D.F + f0, *dlo = p.ACTL + (size_t)row * D.F + f0;
            if (f0 + 32 <= D.F) {
                store_split_x32(dst, dlo, act);
            } else {
                for (int e = 0; e < 32 && f0 + e < D.F; ++e) split_bf16(act[e], dst[e], dlo[e]);
            }
        }
    } else {   // PF_OPROJ, PF_DOWN: residual update in place, next norm input, sums of squares of the new h
        float ss = 0.f;
        bf16 *xo = EPI == PF_OPROJ ? p.XM : p.XS, *xl = EPI == PF_OPROJ ? p.XML : p.XSL;
        for (int c0 = 0; c0 < p.bn_narrow; c0 += 32) {
            __syncwarp();
            tmem_ld32(taddr + (uint32_t)c0, r0);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            const int n = nt * p.bn_narrow + c0;
            if (!live || n >= D.d) continue;                     // d is a multiple of 32
            float *hp = p.H + (size_t)row * D.d + n;
            float h[32];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const float4 v = *reinterpret_cast<const float4 *>(hp + 4 * q);
                h[4 * q + 0] = v.x + __uint_as_float(r0[4 * q + 0]);
                h[4 * q + 1] = v.y + __uint_as_float(r0[4 * q + 1]);
                h[4 * q + 2] = v.z + __uint_as_float(r0[4 * q + 2]);
                h[4 * q + 3] = v.w + __uint_as_float(r0[4 * q + 3]);
                *reinterpret_cast<float4 *>(hp + 4 * q) = make_float4(h[4 * q], h[4 * q + 1], h[4 * q + 2], h[4 * q + 3]);
            }
            if (EPI == PF_DOWN && p.pos0 + row >= p.win0) {
                float *sp = p.stackH + stack_row(D, p.layer, p.seq, p.pos0 + row - p.win0) * D.d + n;
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    *reinterpret_cast<float4 *>(sp + 4 * q) = make_float4(h[4 * q], h[4 * q + 1], h[4 * q + 2], h[4 * q + 3]);
            }
            float x[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                ss += h[e] * h[e];
                x[e] = p.gain ? h[e] * bf16_to_f(p.gain[n + e]) : 0.f;
            }
            if (p.gain) store_split_x32(xo + (size_t)row * D.d + n, xl + (size_t)row * D.d + n, x);
            // one partial sum of squares per 128 columns, whatever the tile width: results do not depend on it
            if ((c0 & 127) == 96 || n + 32 >= D.d) {
                (EPI == PF_OPROJ ? p.SSPM : p.SSP)[(size_t)row * p.n_ssp + (n >> 7)] = ss;
                ss = 0.f;
            }
        }
    }
}

template <int EPI>
__global__ void __launch_bounds__(PF_THREADS, 1) prefill_gemm_kernel(const __grid_constant__ PfMaps maps, const PfArgs p) {
    extern __shared__ unsigned char smem_dyn[];
    __shared__ __align__(8) uint64_t full_bar[STAGES], empty_bar[STAGES], tfull_bar[2], tempty_bar[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile int s_err;
    // 1024-byte alignment for the 128-byte swizzle atoms
    unsigned char *tiles = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&tfull_bar[b], 1); mbar_init(&tempty_bar[b], 4); }
        s_err = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_s;

    pdl_launch();
    pdl_wait();

    const int n_kb = (p.K + BK - 1) / BK;
    const int n_mt = (p.M + BM - 1) / BM;
    const int n_tiles = n_mt * p.n_ntiles;
    const int my_tiles = (n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    if (warp == 0) {
        if (lane == 0) {
            const int n_qt = (p.D.nh * p.D.hd + BN - 1) / BN, n_kt = (p.D.nkv * p.D.hd + BN - 1) / BN;
            int it = 0;
            for (int i = 0; i < my_tiles && !s_err; ++i) {
                const int tile = blockIdx.x + i * gridDim.x;
                const int nt = tile / n_mt, mt = tile - nt * n_mt;      // row tiles of one weight tile run together
                for (int kb = 0; kb < n_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    if (!mbar_wait(&empty_bar[s], ((it / STAGES) & 1) ^ 1)) { s_err = 1; break; }
                    mbar_expect_tx(&full_bar[s], 2 * A_BYTES + tile_n<EPI>(p) * BK * 2);
                    unsigned char *sa = tiles + (size_t)s * STAGE_BYTES;
                    tma_load_2d(sa, &maps.a, kb * BK, mt * BM, &full_bar[s]);
                    tma_load_2d(sa + A_BYTES, &maps.a_lo, kb * BK, mt * BM, &full_bar[s]);
                    sa += A_BYTES;               // the weight tile follows the two activation tiles
                    if (EPI == PF_QKV) {
                        if (nt < n_qt) tma_load_2d(sa + A_BYTES, &maps.b0, kb * BK, nt * BN, &full_bar[s]);
                        else if (nt < n_qt + n_kt) tma_load_2d(sa + A_BYTES, &maps.b1, kb * BK, (nt - n_qt) * BN, &full_bar[s]);
                        else tma_load_2d(sa + A_BYTES, &maps.b2, kb * BK, (nt - n_qt - n_kt) * BN, &full_bar[s]);
                    } else if (EPI == PF_GATEUP) {
                        // accumulator columns 0..127: gate rows of this tile, 128..255: the same rows of W_up
                        tma_load_2d(sa + A_BYTES, &maps.b0, kb * BK, nt * (BN / 2), &full_bar[s]);
                        tma_load_2d(sa + A_BYTES + B_BYTES / 2, &maps.b1, kb * BK, nt * (BN / 2), &full_bar[s]);
                    } else {
                        tma_load_2d(sa + A_BYTES, &maps.b0, kb * BK, nt * tile_n<EPI>(p), &full_bar[s]);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // instruction descriptor: fp32 accumulate, bf16 x bf16, both operands K-major, N = tile width, M = 128
            const uint32_t idesc =
                (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(tile_n<EPI>(p) >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            int it = 0;
            for (int i = 0; i < my_tiles && !s_err; ++i) {
                const int buf = i & 1;
                if (!mbar_wait(&tempty_bar[buf], ((i >> 1) & 1) ^ 1)) { s_err = 2; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * BN;
                bool ok = true;
                for (int kb = 0; kb < n_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    if (!mbar_wait(&full_bar[s], (it / STAGES) & 1)) { s_err = 3; ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t sa = smem_u32(tiles + (size_t)s * STAGE_BYTES);
                    const uint64_t da = umma_desc(sa), dl = umma_desc(sa + A_BYTES), db = umma_desc(sa + 2 * A_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
                        umma_bf16(d_tmem, dl + 2 * k, db + 2 * k, idesc, 1u);
                    }
                    umma_commit(&empty_bar[s]);      // the stage may be refilled once these MMAs have read it
                }
                if (!ok) break;
                umma_commit(&tfull_bar[buf]);        // accumulator complete
            }
        }
    } else {
        const int q = warp & 3;                      // TMEM lane quarter this warp may read
        for (int i = 0; i < my_tiles; ++i) {
            const int tile = blockIdx.x + i * gridDim.x;
            const int nt = tile / n_mt, mt = tile - nt * n_mt;
            const int buf = i & 1;
            if (s_err || !mbar_wait(&tfull_bar[buf], (i >> 1) & 1)) { if (!s_err) s_err = 4; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            epilogue<EPI>(p, tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN), mt * BM + q * 32 + lane, nt);
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&tempty_bar[buf]);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
    if (threadIdx.x == 0 && s_err) atomicMax(p.err, (int)s_err);
}

// h^0 of the chunk's rows: embedding as fp32, layer 1's attention-norm input, sum of squares in partial 0
__global__ void __launch_bounds__(256) prefill_embed_kernel(const PfArgs p, const bf16 *tok_emb, const int32_t *prompt, const bf16 *gain0) {
    __shared__ float s_red[8];
    pdl_launch();
    pdl_wait();
    const int row = blockIdx.x, d = p.D.d;
    const bf16 *e = tok_emb + (size_t)prompt[p.pos0 + row] * d;
    float *sp = p.pos0 + row >= p.win0 ? p.stackH + stack_row(p.D, 0, p.seq, p.pos0 + row - p.win0) * d : nullptr;
    float ss = 0.f;
    for (int o = threadIdx.x; o < d; o += 256) {
        const float h = bf16_to_f(e[o]);
        p.H[(size_t)row * d + o] = h;
        if (sp) sp[o] = h;
        split_bf16(h * bf16_to_f(gain0[o]), p.XS[(size_t)row * d + o], p.XSL[(size_t)row * d + o]);
        ss += h * h;
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x < p.n_ssp) {
        float t = 0.f;
        if (threadIdx.x == 0)
            for (int w = 0; w < 8; ++w) t += s_red[w];
        p.SSP[(size_t)row * p.n_ssp + threadIdx.x] = t;
    }
}

template <int EPI>
cudaError_t launch_epi(const PfMaps &maps, const PfArgs &p, int n_sms, cudaStream_t st, bool pdl) {
    const size_t smem = (size_t)STAGES * STAGE_BYTES + 1024;
    auto kern = prefill_gemm_kernel<EPI>;
    static SmemAttrOnce attr;
    {
        cudaError_t e = attr.set(kern, (int)((int)smem));
        if (e != cudaSuccess) return e;
    }
    const int n_tiles = ((p.M + BM - 1) / BM) * p.n_ntiles;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_tiles < n_sms ? n_tiles : n_sms);
    cfg.blockDim = dim3(PF_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, maps, p);
}

}  // namespace

int prefill_tc_ntiles(int epi, const Dims &D) {
    switch (epi) {
        case PF_QKV: return (D.nh * D.hd + BN - 1) / BN + 2 * ((D.nkv * D.hd + BN - 1) / BN);
        case PF_GATEUP: return (D.F + BN / 2 - 1) / (BN / 2);
        default: { const int bn = prefill_tc_narrow(D); return (D.d + bn - 1) / bn; }
    }
}
int prefill_tc_nssp(const Dims &D) { return (D.d + 127) / 128; }

// Tile width of the two GEMMs whose N is d_model: 128 or 256 (whole 128-column groups of the per-row sums of
// squares, so that no result depends on the choice).  A k-block of a 128 x bn tile costs its operand loads,
// (128 + bn) rows of 128 bytes at what one SM can pull from L2, more than its MMAs (measured: tensor pipe 40-68 %
// active), so a tile takes about (128 + bn) units; the width that minimises waves x (128 + bn) for a full chunk
// of PF_ROWS rows on 148 SMs wins: 128 at d = 4096 (128 tiles, one wave), 256 at d = 5120 (80 tiles in one wave
// instead of 160 in two: the 3072-position prefill of that shape 138 -> 127 ms).
int prefill_tc_narrow(const Dims &D) {
    int best = 128;
    long best_cost = -1;
    for (int bn = 128; bn <= 256; bn += 128) {
        const long tiles = (long)(PF_ROWS / BM) * ((D.d + bn - 1) / bn);
        const long cost = ((tiles + 147) / 148) * (128 + bn);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = bn; }
    }
    return best;
}

// map_a / map_b*: 128-byte CUtensorMap blobs made by lmhead_tc_make_map (boxes of 256 rows for Wq / Wk / Wv, of
// 128 rows for the activations and for W_gate / W_up / W_o / W_down)
cudaError_t launch_prefill_gemm(int epi, const void *map_a, const void *map_a_lo, const void *map_b0, const void *map_b1,
                                const void *map_b2, const PfArgs &p, int n_sms, cudaStream_t st, bool pdl) {
    PfMaps maps;
    maps.a = *reinterpret_cast<const CUtensorMap *>(map_a);
    maps.a_lo = *reinterpret_cast<const CUtensorMap *>(map_a_lo);
    maps.b0 = *reinterpret_cast<const CUtensorMap *>(map_b0);
    maps.b1 = *reinterpret_cast<const CUtensorMap *>(map_b1 ? map_b1 : map_b0);
    maps.b2 = *reinterpret_cast<const CUtensorMap *>(map_b2 ? map_b2 : map_b0);
    switch (epi) {
        case PF_QKV: return launch_epi<PF_QKV>(maps, p, n_sms, st, pdl);
        case PF_OPROJ: return launch_epi<PF_OPROJ>(maps, p, n_sms, st, pdl);
        case PF_GATEUP: return launch_epi<PF_GATEUP>(maps, p, n_sms, st, pdl);
        case PF_DOWN: return launch_epi<PF_DOWN>(maps, p, n_sms, st, pdl);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_prefill_embed(const PfArgs &p, const bf16 *tok_emb, const int32_t *prompt, const bf16 *gain0, cudaStream_t st) {
    prefill_embed_kernel<<<p.M, 256, 0, st>>>(p, tok_emb, prompt, gain0);
    return cudaGetLastError();
}
