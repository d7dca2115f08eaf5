// Stacked LM head on the 5th-generation tensor cores: logits[R, V] = Xn[R, d] * W_lm[V, d]^T with the
// per-row arg-max over the vocabulary fused into the epilogue, so the logits never reach memory and
// W_lm is streamed from HBM once for all R = L * (gamma + 1) rows of the round.
//
// CTA tile: 128 rows x 256 vocabulary entries, K blocks of 64 (one 128-byte swizzle span).  Roles:
//   warp 0     one lane issues the TMA loads (cp.async.bulk.tensor, every CTA loads its own tiles) of the Xn tile
//              [128 x 64] and the W_lm tile [256 x 64] into a 4-stage shared-memory ring;
//   warp 1     allocates tensor memory; one lane issues tcgen05.mma (M 128, N 256, K 16, bf16 inputs,
//              fp32 accumulators in TMEM) and commits each stage back to the producer;
//   warps 2-5  epilogue: tcgen05.ld of the thread's own row, running (max, index) over the 256
//              columns in ascending order (lowest index wins ties), one partial per (row, tile).
// Two accumulator buffers (2 x 256 TMEM columns) let the epilogue of tile i overlap the MMAs of tile
// i+1.  Tiles are ordered vocabulary-major so CTAs that run together share the same W_lm tile in L2.
// Every mbarrier wait is bounded: on expiry the kernel records an error code and winds down (TMEM is
// always released).
#include <cuda.h>
#include <cstring>

#include "kernels.h"
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int TC_THREADS = 192;

struct TcParams {
    float *part_v;
    int32_t *part_i;
    float *part_s;               // exp sums relative to part_v (for the confidence score)
    const float *row_scale;      // [rows] log2(e) / rms: the logit behind accumulator v is v / rms
    int32_t n_rows, V, d, n_mtiles, n_vtiles, n_tiles;
    int32_t *err;
    // speculative sampling: rows whose whole logit row is also stored (the target's rows of each sampling sequence)
    int32_t n_sel, pad;
    LogitSel sel[DEL_SEQ_MAX];
};

// 2^x on the special-function unit (one instruction; the confidence score tolerates its 2-ulp error)
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(TC_THREADS, 1)
lmhead_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const TcParams p) {
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

    const int n_kb = p.d / BK;
    const int my_tiles = (p.n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;
            for (int i = 0; i < my_tiles && !s_err; ++i) {
                const int tile = blockIdx.x + i * gridDim.x;
                const int vt = tile / p.n_mtiles, mt = tile - vt * p.n_mtiles;
                for (int kb = 0; kb < n_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    if (!mbar_wait(&empty_bar[s], ((it / STAGES) & 1) ^ 1)) { s_err = 1; break; }
                    mbar_expect_tx(&full_bar[s], STAGE_BYTES);
                    unsigned char *sa = tiles + (size_t)s * STAGE_BYTES;
                    tma_load_2d(sa, &map_x, kb * BK, mt * BM, &full_bar[s]);
                    tma_load_2d(sa + A_BYTES, &map_w, kb * BK, vt * BN, &full_bar[s]);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // instruction descriptor: fp32 accumulate, bf16 x bf16, both operands K-major, N = 256, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
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
                    const uint64_t da = umma_desc(sa), db = umma_desc(sa + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
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
            const int vt = tile / p.n_mtiles, mt = tile - vt * p.n_mtiles;
            const int buf = i & 1;
            if (s_err || !mbar_wait(&tfull_bar[buf], (i >> 1) & 1)) { if (!s_err) s_err = 4; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int row = mt * BM + q * 32 + lane;
            const int v0 = vt * BN;
            const float k = row < p.n_rows ? p.row_scale[row] : 0.f;
            float best = -INFINITY, esum = 0.f;
            int bidx = 0x7fffffff;
            float *ldst = nullptr;                           // this thread's row is one whose logits are kept
            for (int s = 0; s < p.n_sel; ++s) {
                const int rr = row - p.sel[s].row_lo;
                if (rr >= 0 && rr < p.sel[s].n) ldst = p.sel[s].dst + (size_t)rr * p.V;
            }
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c0), r);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const float before = best;
                const int nv = min(32, p.V - (v0 + c0));     // columns of this chunk inside the vocabulary (whole chunk: 32)
                if (ldst != nullptr && nv > 0) {
                    const float ks = k * 0.6931471805599453f;                  // normalised logit = raw / rms
                    float *o = ldst + v0 + c0;
                    if (nv >= 32) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<float4 *>(o + j) =
                                make_float4(__uint_as_float(r[j]) * ks, __uint_as_float(r[j + 1]) * ks,
                                            __uint_as_float(r[j + 2]) * ks, __uint_as_float(r[j + 3]) * ks);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (j < nv) o[j] = __uint_as_float(r[j]) * ks;
                    }
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float v = __uint_as_float(r[j]);
                    if (j < nv && v > best) { best = v; bidx = v0 + c0 + j; }
                }
                // exp sum relative to the running maximum (rescaled when this chunk raised it)
                if (best > before) esum *= ex2(k * (before - best));
                float part[4] = {0.f, 0.f, 0.f, 0.f};          // four chains instead of one 32-long dependent sum
                const float kb = k * best;
                if (nv >= 32) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) part[j & 3] += ex2(fmaf(k, __uint_as_float(r[j]), -kb));
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j < nv) part[j & 3] += ex2(fmaf(k, __uint_as_float(r[j]), -kb));
                }
                esum += (part[0] + part[1]) + (part[2] + part[3]);
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&tempty_bar[buf]);
            if (row < p.n_rows) {
                p.part_v[(size_t)row * p.n_vtiles + vt] = best;
                p.part_i[(size_t)row * p.n_vtiles + vt] = bidx;
                p.part_s[(size_t)row * p.n_vtiles + vt] = esum;
            }
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

}  // namespace

// [rows, d] bf16 row-major tensor, boxes of box_rows x 64 elements, 128-byte swizzle, zero fill outside
int lmhead_tc_make_map(void *map_out, const void *base, uint64_t rows, uint64_t d, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return -1;
    cuuint64_t dims[2] = {d, rows};
    cuuint64_t strides[1] = {d * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(reinterpret_cast<CUtensorMap *>(map_out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims,
                    strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : -2;
}

int lmhead_tc_vtiles(int V) { return (V + BN - 1) / BN; }

cudaError_t launch_lmhead_tc(const void *map_x, const void *map_w, float *part_v, int32_t *part_i, float *part_s,
                             const float *row_scale, int n_rows, int V, int d, int32_t *err, const LogitSel *sel, int n_sel,
                             int n_sms, cudaStream_t st, bool pdl) {
    TcParams p;
    memset(&p, 0, sizeof(p));
    if (n_sel > DEL_SEQ_MAX) return cudaErrorInvalidValue;
    p.n_sel = sel ? n_sel : 0;
    for (int s = 0; s < p.n_sel; ++s) p.sel[s] = sel[s];
    p.part_v = part_v; p.part_i = part_i; p.part_s = part_s; p.row_scale = row_scale; p.n_rows = n_rows; p.V = V; p.d = d;
    p.n_mtiles = (n_rows + BM - 1) / BM;
    p.n_vtiles = (V + BN - 1) / BN;
    p.n_tiles = p.n_mtiles * p.n_vtiles;
    p.err = err;
    const size_t smem = (size_t)STAGES * STAGE_BYTES + 1024;
    static SmemAttrOnce attr;
    {
        cudaError_t e = attr.set(lmhead_tc_kernel, (int)((int)smem));
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.n_tiles < n_sms ? p.n_tiles : n_sms);
    cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, lmhead_tc_kernel, *reinterpret_cast<const CUtensorMap *>(map_x),
                              *reinterpret_cast<const CUtensorMap *>(map_w), p);
}
