// Multi-query attention over the paged bf16 KV cache (decode rounds and the passes of the prefill).
//
// One CTA = (key-range split, kv head, sequence segment), 8 warps; the device code lives in
// attention_body.cuh.  A segment with a single 16-row query tile (one sequence drafting or verifying a
// few tokens with few query heads per kv head) loads its key / value fragments straight from global
// memory: the shortest dependent chain.  A segment with several query tiles (many rows, grouped-query
// attention, prefill passes of 64 rows) stages the pages in shared memory once for all tiles.
//
// With one split the result is final; otherwise splits write partial online-softmax states and the last
// CTA to arrive for a (segment, kv head) merges them in split order, so the result does not depend on
// scheduling.
#include "attention_body.cuh"
#include "kernels.h"

namespace {

using attn::NW;

template <int HD>
__global__ void __launch_bounds__(NW * 32) attention_kernel(const __grid_constant__ AttnArgs a) {
    extern __shared__ __align__(16) float sm[];
    __shared__ int s_last;
    pdl_launch();                  // (the wait for the producer kernel sits inside partial / partial_staged)

    const AttnView v{a.D, a.B, a.layer, a.early_pos[blockIdx.z], &a.pf};
    const Segment seg = a.plan.seg[blockIdx.z];
    const int kvh = blockIdx.y, split = blockIdx.x, n_splits = a.n_splits;
    const int n_pages = (seg.pos0 + seg.nrows + 15) >> 4;
    const int pps = (n_pages + n_splits - 1) / n_splits;
    const int p_begin = split * pps, p_end = min(n_pages, p_begin + pps);
    // several query tiles share the pages through shared memory; a single tile loads its fragments directly
    const int n_mt = (seg.nrows * (a.D.nh / a.D.nkv) + 15) >> 4;
    if (n_mt >= 2) attn::partial_staged<HD>(v, reinterpret_cast<unsigned char *>(sm), seg, kvh, p_begin, p_end, 0, 0x7fffffff, split, n_splits);
    else attn::partial<HD>(v, sm, seg, kvh, p_begin, p_end, 0, 0x7fffffff, split, n_splits);

    if (n_splits > 1) {
        // The CTA's partial states are published by one release-acquire ticket: the barrier orders every thread's
        // stores before thread 0's release, and the last CTA's acquire, followed by its barrier, orders all splits'
        // stores before the merge's loads (which go to L2, not to L1).
        __syncthreads();
        if (threadIdx.x == 0) {
            int ticket;
            asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(ticket) : "l"(a.B.ACNT + blockIdx.z * a.D.nkv + kvh) : "memory");
            s_last = (ticket == n_splits - 1);
            if (s_last) a.B.ACNT[blockIdx.z * a.D.nkv + kvh] = 0;     // ready for the next launch
        }
        __syncthreads();
        if (s_last) attn::merge_slots<HD>(v, seg, kvh, n_splits);
    }
}

template <int HD>
cudaError_t launch_one(const AttnArgs &a, int n_seg, cudaStream_t st, bool pdl) {
    const size_t smem = attn::staged_smem_bytes(HD);
    auto kern = attention_kernel<HD>;
    static SmemAttrOnce attr;
    {
        cudaError_t e = attr.set(kern, (int)((int)smem));
        if (e != cudaSuccess) return e;
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
    // the kernel keeps one CTA per SM resident: stay within one wave, aim at one page per warp (measured: 0.4 %
    // faster rounds than two pages per warp, 1.1 % faster than three)
    int ns = per_warp;
    const int one_wave = n_sms / n_units;
    if (ns > one_wave) ns = one_wave;
    return ns > 16 ? 16 : (ns < 1 ? 1 : ns);
}

cudaError_t launch_attention(const AttnArgs &a, int n_seg, cudaStream_t st, bool pdl) {
    if (a.D.hd == 128) return launch_one<128>(a, n_seg, st, pdl);
    if (a.D.hd == 64) return launch_one<64>(a, n_seg, st, pdl);
    return cudaErrorInvalidValue;
}
