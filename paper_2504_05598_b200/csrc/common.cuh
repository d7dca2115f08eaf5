// Shared device-side definitions of libdel: plan structures that describe the rows of a layer pass,
// the device-resident model / workspace description, and small PTX wrappers (streaming 16-byte loads,
// bf16 tensor-core MMA, programmatic-dependent-launch control).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#define DEL_ROWS_MAX 64        // rows of one layer pass
#define DEL_GEMM_ROWS 32       // rows one launch of a layer GEMM serves (each row takes two MMA columns)
#define DEL_SEQ_MAX 16         // sequences per context
#define DEL_GEMM_THREADS 256
#define DEL_GEMM_WARPS 8

typedef __nv_bfloat16 bf16;

// One row of a layer pass: which sequence, which slot of the hidden stack, which position of the
// sequence, and where its input token sits in the token buffer (embedding passes only).
struct RowDesc {
    int32_t seq, slot, pos, tok;
};

// Rows of one sequence inside a pass: consecutive rows, consecutive slots, consecutive positions.
struct Segment {
    int32_t seq, row0, nrows, pos0;
};

struct PassPlan {
    int32_t m, n_seg, pad0, pad1;
    RowDesc rows[DEL_ROWS_MAX];
    Segment seg[DEL_SEQ_MAX];
};

// Per-sequence state that lives on the device.
struct SeqState {
    double Sn;
    int32_t E, gamma;            // choice for the next round
    int32_t fixed_E, fixed_gamma;
    int32_t fs_mode;             // 1: fixed E, gamma moved by the +-1 controller
    int32_t pad;
};

// ---- speculative sampling (Sec. 2): per-row description of the filtered distribution and per-sequence results
#define DEL_SAMPLE_ROWS 32     // logit rows kept per sequence and kind: g_max + 1 <= 32

// Weights are integers W = round(exp((z - m) / T) * 2^40), so that sums do not depend on the order of addition.
// The nucleus keeps every token whose weight key (the fp32 bit pattern of the weight) is above kstar and the
// first tie_keep tokens, in token-id order, whose key equals kstar.
struct RowStat {
    float m;                     // largest logit of the row
    uint32_t kstar;
    int32_t tie_keep, cnt_eq;
    unsigned long long K;        // mass of the kept tokens
    unsigned long long Z;        // mass of all tokens
};

struct SampleOut {
    int32_t n_accept, last_token, n_tests, from_residual;
    float q_x[DEL_SAMPLE_ROWS], p_x[DEL_SAMPLE_ROWS];     // filtered draft / target probability of draft i
};

// Device view of the model shape and of the workspace carve-up (passed by value to kernels).
struct Dims {
    int32_t L, d, nh, nkv, hd, F, V;
    int32_t B, S;                // sequences, hidden-stack slots per sequence
    int32_t max_seq, page_size, pages_per_seq;
    int32_t n_sst;               // sum-of-squares partials per row (= d / 16)
    float eps;
};

struct Buffers {
    float *H;                    // [L+1][B][S][d]    hidden stack (layer 0 = embedding)
    bf16 *XS;                    // [L+1][B][S][d]    h * gain of the next layer's attention norm (high part)
    // Every GEMM input is kept as a pair of bf16 arrays: x ~ hi + lo with hi = bf16(x), lo = bf16(x - hi), i.e.
    // 16 bits of mantissa.  The low parts have the layout of their high parts.
    bf16 *XSL;                   // low part of XS
    float *SS;                   // [L+1][B][S][n_sst] partial sums of squares of h
    bf16 *XE;                    // [B][S][d]         h * gain of the final norm at the exit layer
    bf16 *Q;                     // [ROWS][nh*hd]     queries after the rotary embedding
    bf16 *ATT, *ATTL;            // [ROWS][nh*hd]     attention output, high and low part
    float *HM;                   // [ROWS][d]         residual after attention
    bf16 *XM, *XML;              // [ROWS][d]         HM * gain of the ffn norm, high and low part
    float *SSM;                  // [ROWS][n_sst]
    bf16 *ACT, *ACTL;            // [ROWS][F]         silu(gate) * up, high and low part
    float *APO;                  // attention partial outputs [ROWS][nh][splits][hd]
    float *APML;                 // attention partial (max, sum) [ROWS][nh][splits][2]
    int32_t *ACNT;               // [DEL_SEQ_MAX][nkv] arrival counters of the split combine
    float *LPV;                  // streaming LM head: arg-max partial values [ctas][ROWS]
    int32_t *LPI;                // ... and indices
    float *LPS;                  // ... and sums of exp(scaled logit - scaled partial maximum)
    float *RK;                   // [ROWS] log2(e) / rms of the rows of the last streaming LM-head launch
    float *TPV;                  // tensor-core LM head: partial values [R_max][vocab tiles]
    int32_t *TPI;
    float *TPS;                  // ... and partial exp sums
    float *RS;                   // [R_max] log2(e) / rms of the stacked rows
    float *SSE;                  // [B][S][n_sst] partial sums of squares of h at the exit layer (beside XE)
    float *DCONF;                // [B][S+1] confidence of draft i at [1 + i] (indexed like TOK)
    float *SCONF;                // [B][L][S] confidence (top-1 probability) of the shadow tokens
    double *STCS, *SFCS, *TAU;   // [B][L] decayed confidence sums over matched / mismatched shadow tokens, thresholds
    float *QLOG, *PLOG;          // [B][DEL_SAMPLE_ROWS][V] sampling: logits of the exit head per draft / of the target per row
    RowStat *QSTAT, *PSTAT;      // [B][DEL_SAMPLE_ROWS]
    SampleOut *SMP;              // [B]
    int32_t *PROMPT_ALL;         // [max_seq] prompt tokens of the sequence being prefilled
    bf16 *XN;                    // [R_max][d] normalised rows for the batched LM head
    int32_t *SHADOW;             // [B][L][S] shadow tokens
    int32_t *COUNTS;             // [B][L]
    int32_t *TOK;                // [B][S+1] token buffer: [0] next input, [1+i] draft i
    double *SC;                  // [B][L] decayed match counts
    SeqState *ST;                // [B]
    int32_t *ERR;                // device error word
    int32_t *TCNT;               // ring of per-launch tile-claim counters
    bf16 *KP, *VP;               // KV pages
    int32_t *PT;                 // page table [B][pages_per_seq]
    const float *rope_cos, *rope_sin;
};

// Regions of global memory that a kernel requests into L2 for its successors: up to 3, 16-byte aligned; n = 0: none.
struct AttnPrefetch {
    const void *ptr[3];
    uint32_t bytes[3];
    int32_t n, pad;
};

__device__ __forceinline__ size_t stack_row(const Dims &D, int layer, int seq, int slot) {
    return ((size_t)layer * D.B + seq) * D.S + slot;
}

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// 16-byte streaming load of immutable data (weights): read-only path, no L1 allocation.
__device__ __forceinline__ uint4 ldg_stream16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// 16-byte load of activations written by an earlier kernel (coherent at L2).
__device__ __forceinline__ uint4 ldg_act16(const void *p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// Predicated forms: zero when `pred` is false.  The destination is cleared first and the load itself is
// predicated, so no select instruction has to wait for the loaded value (which would serialise the
// software pipeline on the load latency).
__device__ __forceinline__ uint4 ldg_stream16_pred(const void *p, bool pred) {
    uint4 v;
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %5, 0;\n\tmov.u32 %0, 0;\n\tmov.u32 %1, 0;\n\tmov.u32 %2, 0;\n\tmov.u32 %3, 0;\n\t"
                 "@q ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n\t}"
                 : "=&r"(v.x), "=&r"(v.y), "=&r"(v.z), "=&r"(v.w) : "l"(p), "r"((uint32_t)pred));
    return v;
}
__device__ __forceinline__ uint4 ldg_act16_pred(const void *p, bool pred) {
    uint4 v;
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %5, 0;\n\tmov.u32 %0, 0;\n\tmov.u32 %1, 0;\n\tmov.u32 %2, 0;\n\tmov.u32 %3, 0;\n\t"
                 "@q ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];\n\t}"
                 : "=&r"(v.x), "=&r"(v.y), "=&r"(v.z), "=&r"(v.w) : "l"(p), "r"((uint32_t)pred));
    return v;
}
// request `bytes` (a multiple of 16, 16-byte aligned start) of global memory into L2; nothing waits for it
__device__ __forceinline__ void l2_prefetch_bulk(const void *p, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}
// 16-byte asynchronous global -> shared copy (zero fill when `pred` is false)
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src, bool pred) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    const uint32_t n = pred ? 16u : 0u;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(gmem_src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// waits until at most N of this thread's most recent copy groups are still in flight
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint2 ldg_act8(const void *p) {
    uint2 v;
    asm volatile("ld.global.cg.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ldg_act8_pred(const void *p, bool pred) {
    uint2 v;
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %3, 0;\n\tmov.u32 %0, 0;\n\tmov.u32 %1, 0;\n\t"
                 "@q ld.global.cg.v2.u32 {%0,%1}, [%2];\n\t}"
                 : "=&r"(v.x), "=&r"(v.y) : "l"(p), "r"((uint32_t)pred));
    return v;
}
__device__ __forceinline__ float ldg_cg_f32(const float *p) {
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}

// D += A(16x16, row) * B(16x8, col), bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
// x as a pair of bf16 values: hi = bf16(x), lo = bf16(x - hi); hi + lo carries 16 bits of x's mantissa
__device__ __forceinline__ void split_bf16(float x, bf16 &hi, bf16 &lo) {
    hi = __float2bfloat16_rn(x);
    lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}
// two values: packed high parts (element 0 in the low half-word) and packed low parts
__device__ __forceinline__ void split_bf16x2(float x0, float x1, uint32_t &hi, uint32_t &lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
    const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - __low2float(h), x1 - __high2float(h));
    hi = *reinterpret_cast<const uint32_t *>(&h);
    lo = *reinterpret_cast<const uint32_t *>(&l);
}
__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }
__device__ __forceinline__ float bf16_to_f(bf16 v) { return __bfloat162float(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
