// Device-side building blocks of the paged multi-query attention kernel (attention.cu).
//
// partial / partial_staged contain the kernel's wait for its producer (programmatic dependent launch): what they
// read before it does not depend on the producer.
//   attn::partial         one CTA walks a range of key pages for one (segment, kv head) and leaves, per
//                         query row and head, an online-softmax state (max, sum, unnormalised output):
//                         either as the final normalised result (one slot) or in one of several slots;
//                         fragments are loaded straight from global memory (best for a single query tile)
//   attn::partial_staged  the same, with the pages staged in shared memory and shared by all query tiles
//   attn::merge_slots     combines the slots of every (row, head) of a (segment, kv head) in slot order
//
// The query rows of the segment (its consecutive positions times the query heads sharing the kv head)
// form 16-row tiles; the 8 warps are divided among up to 4 query tiles, and the warps of one tile walk
// the key pages (16 tokens each) of the range in a strided fashion.  Scores and the P*V product run on
// bf16 tensor-core MMAs with fp32 accumulation; row reductions use shuffles inside the 4-lane groups
// that own a row.  The output is stored as a pair of bf16 values (high + low part) for the O-projection.
//
// Fragment layout: the MMA sums over its k index, so any permutation of k used for both operands is
// allowed.  For Q*K^T a thread loads 16 contiguous bytes of a key row (and the same bytes of the query
// row) and feeds them to two MMAs.  For P*V the page stores V transposed ([head_dim][16 tokens]); the
// score tile's columns are assigned to tokens such that a thread's four probabilities belong to tokens
// 4t..4t+3, which are 8 contiguous bytes of a V^T row.
#pragma once

#include "common.cuh"

struct AttnView {
    const Dims &D;
    const Buffers &B;
    int32_t layer;
    int32_t early_pos;         // of this CTA's segment, see AttnArgs
    const AttnPrefetch *pf;    // weights to request into L2 for the following launches
};

namespace attn {

// head-major row index -> (query head within the group, row of the segment); ms = rows of the segment.
// One-row segments (plain drafting, the common case on the critical path) skip the integer division.
__device__ __forceinline__ void split_row(int rr, int ms, int &hq, int &i) {
    if (ms == 1) { hq = rr; i = 0; return; }
    hq = rr / ms;
    i = rr - hq * ms;
}

constexpr float LOG2E = 1.4426950408889634f;

// Every CTA of the launch requests its share of the regions in pieces of 32 KB, one piece per lane of its last warp
// (called once the warps' own early cache reads have been issued, before the wait for the producer kernel).
__device__ __forceinline__ void prefetch_weights(const AttnPrefetch &pf) {
    constexpr uint32_t PIECE = 32768;
    if ((threadIdx.x >> 5) != 7) return;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t n_cta = gridDim.x * gridDim.y * gridDim.z;
    const uint32_t cta = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
    for (int r = 0; r < pf.n; ++r) {
        const uint32_t n_piece = (pf.bytes[r] + PIECE - 1) / PIECE;
        for (uint32_t i = cta + n_cta * lane; i < n_piece; i += n_cta * 32) {
            const uint32_t off = i * PIECE, len = min(PIECE, pf.bytes[r] - off) & ~15u;
            if (len) l2_prefetch_bulk(reinterpret_cast<const unsigned char *>(pf.ptr[r]) + off, len);
        }
    }
}
constexpr int NW = 8;                 // warps per CTA
constexpr int PG = 4;                 // page ids fetched ahead per warp
constexpr int MAX_SLOTS = 16;

__host__ __device__ constexpr size_t smem_bytes(int hd) {
    return sizeof(float) * ((size_t)NW * 32 * (hd / 8) * 4 + (size_t)NW * 32 * 4);
}

// Per-thread view of one 16-row query tile: which rows of the segment the thread's two MMA rows are,
// their query fragments, and the running softmax state.
template <int HD>
struct TileState {
    static constexpr int KS = HD / 32;    // 16-byte chunks per thread along head_dim
    static constexpr int NJ = HD / 8;     // output n-tiles
    uint4 qf[2][KS];
    bool rv[2];
    int rmax[2];                          // last key a row may see
    float m_run[2], l_run[2];
    float O[NJ][4];
};

// rows of this thread in query tile mt: rr0 = mt*16+g, rr1 = rr0+8, ordered head-major: rr = hq*ms + i
template <int HD>
__device__ __forceinline__ void tile_begin(TileState<HD> &ts, const AttnView &a, const Segment seg, int kvh, int mt, int n_mt,
                                           int k_hi) {
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int ms = seg.nrows, group = a.D.nh / a.D.nkv, R = ms * group, qdim = a.D.nh * HD;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int rr = mt * 16 + g + 8 * h;
        ts.rv[h] = mt < n_mt && rr < R;
        int rh = 0, ri = 0;
        if (ts.rv[h]) split_row(rr, ms, rh, ri);
        const bf16 *qp = a.B.Q + (size_t)(seg.row0 + ri) * qdim + (kvh * group + rh) * HD + 8 * t;
#pragma unroll
        for (int ks = 0; ks < TileState<HD>::KS; ++ks) ts.qf[h][ks] = ldg_act16_pred(qp + 32 * ks, ts.rv[h]);
        ts.rmax[h] = min(seg.pos0 + ri, k_hi);
        ts.m_run[h] = -INFINITY;
        ts.l_run[h] = 0.f;
    }
#pragma unroll
    for (int j = 0; j < TileState<HD>::NJ; ++j) ts.O[j][0] = ts.O[j][1] = ts.O[j][2] = ts.O[j][3] = 0.f;
}

// One key page against the tile: scores, online-softmax update, P*V.  kf[0] / kf[1]: the thread's key
// fragments of score tiles 0 / 1, vf: its V^T fragments; p = page number within the sequence.
template <int HD>
__device__ __forceinline__ void page_update(TileState<HD> &ts, const uint4 (&kf)[2][HD / 32], const uint2 (&vf)[HD / 8], int p,
                                            int k_lo, float sc) {
    constexpr int KS = HD / 32, NJ = HD / 8;
    const int t = threadIdx.x & 3;
    float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
        mma_bf16_16816(s0, ts.qf[0][ks].x, ts.qf[1][ks].x, ts.qf[0][ks].y, ts.qf[1][ks].y, kf[0][ks].x, kf[0][ks].y);
        mma_bf16_16816(s0, ts.qf[0][ks].z, ts.qf[1][ks].z, ts.qf[0][ks].w, ts.qf[1][ks].w, kf[0][ks].z, kf[0][ks].w);
        mma_bf16_16816(s1, ts.qf[0][ks].x, ts.qf[1][ks].x, ts.qf[0][ks].y, ts.qf[1][ks].y, kf[1][ks].x, kf[1][ks].y);
        mma_bf16_16816(s1, ts.qf[0][ks].z, ts.qf[1][ks].z, ts.qf[0][ks].w, ts.qf[1][ks].w, kf[1][ks].z, kf[1][ks].w);
    }
    // this thread's scores: tokens 4t, 4t+1 (s0) and 4t+2, 4t+3 (s1) of the page, rows g / g+8
    const int tok0 = p * 16 + 4 * t;
    float pr[2][4];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        float v[4] = {s0[2 * h] * sc, s0[2 * h + 1] * sc, s1[2 * h] * sc, s1[2 * h + 1] * sc};
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (!ts.rv[h] || tok0 + e > ts.rmax[h] || tok0 + e < k_lo) v[e] = -INFINITY;
        float mx = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(ts.m_run[h], mx);
        const float base = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = exp2f(ts.m_run[h] - base);
        ts.m_run[h] = m_new;
        float psum = 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) { pr[h][e] = exp2f(v[e] - base); psum += pr[h][e]; }
        ts.l_run[h] = ts.l_run[h] * alpha + psum;
#pragma unroll
        for (int j = 0; j < NJ; ++j) { ts.O[j][2 * h] *= alpha; ts.O[j][2 * h + 1] *= alpha; }
    }
    const uint32_t pa0 = pack_bf16(pr[0][0], pr[0][1]), pa1 = pack_bf16(pr[1][0], pr[1][1]);
    const uint32_t pa2 = pack_bf16(pr[0][2], pr[0][3]), pa3 = pack_bf16(pr[1][2], pr[1][3]);
#pragma unroll
    for (int j = 0; j < NJ; ++j) mma_bf16_16816(ts.O[j], pa0, pa1, pa2, pa3, vf[j].x, vf[j].y);
}

// The warps of each query tile merge their states through shared memory (every warp of the CTA merges
// some output column tiles) and write the result: normalised to ATT when n_slots == 1, otherwise as a
// partial state to slot `slot`.  it = iteration over groups of P concurrent query tiles.
template <int HD>
__device__ __forceinline__ void tile_end(TileState<HD> &ts, const AttnView &a, float *sm, const Segment seg, int kvh, int it,
                                         int P, int n_mt, int slot, int n_slots) {
    constexpr int NJ = HD / 8;
    float *sm_o = sm;                               // [NJ][NW][32] float4
    float *sm_ml = sm + NW * 32 * NJ * 4;           // [NW][32] float4
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int ms = seg.nrows, group = a.D.nh / a.D.nkv, R = ms * group, qdim = a.D.nh * HD;
    const int n_kl = NW / P;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        ts.l_run[h] += __shfl_xor_sync(0xffffffffu, ts.l_run[h], 1);
        ts.l_run[h] += __shfl_xor_sync(0xffffffffu, ts.l_run[h], 2);
    }
    if (R <= 8) {
        // Few query rows (one sequence drafting or verifying a handful of tokens): only rows 0..R-1 of the tile
        // carry data, i.e. MMA rows g < R and none of the rows g + 8.  Merge just those: [warp][row][HD] floats.
        float *so = sm;                             // [NW][R][HD]
        float *sml = sm + NW * 8 * HD;              // [NW][8] (max, sum)
        if (g < R) {
            float *dst = so + ((size_t)warp * R + g) * HD + 2 * t;
#pragma unroll
            for (int j = 0; j < NJ; ++j) *reinterpret_cast<float2 *>(dst + 8 * j) = make_float2(ts.O[j][0], ts.O[j][1]);
            if (t == 0) *reinterpret_cast<float2 *>(sml + (warp * 8 + g) * 2) = make_float2(ts.m_run[0], ts.l_run[0]);
        }
        __syncthreads();
        for (int e = tid; e < R * (HD / 2); e += NW * 32) {
            const int row = e / (HD / 2), col = (e - row * (HD / 2)) * 2;
            float M = -INFINITY;
#pragma unroll
            for (int w2 = 0; w2 < NW; ++w2) M = fmaxf(M, sml[(w2 * 8 + row) * 2]);
            const float b = M == -INFINITY ? 0.f : M;
            float L = 0.f, o0 = 0.f, o1 = 0.f;
#pragma unroll
            for (int w2 = 0; w2 < NW; ++w2) {
                const float2 ml = *reinterpret_cast<const float2 *>(sml + (w2 * 8 + row) * 2);
                const float f = exp2f(ml.x - b);
                const float2 ov = *reinterpret_cast<const float2 *>(so + ((size_t)w2 * R + row) * HD + col);
                L += ml.y * f;
                o0 += ov.x * f;
                o1 += ov.y * f;
            }
            int hq, i;
            split_row(row, ms, hq, i);
            const int c = seg.row0 + i, qh = kvh * group + hq;
            if (n_slots == 1) {
                const float inv = 1.f / L;
                uint32_t hi, lo;
                split_bf16x2(o0 * inv, o1 * inv, hi, lo);
                *reinterpret_cast<uint32_t *>(a.B.ATT + (size_t)c * qdim + qh * HD + col) = hi;
                *reinterpret_cast<uint32_t *>(a.B.ATTL + (size_t)c * qdim + qh * HD + col) = lo;
            } else {
                const size_t pi = ((size_t)c * a.D.nh + qh) * n_slots + slot;
                *reinterpret_cast<float2 *>(a.B.APO + pi * HD + col) = make_float2(o0, o1);
                if (col == 0) *reinterpret_cast<float2 *>(a.B.APML + pi * 2) = make_float2(M, L);
            }
        }
        __syncthreads();
        return;
    }
    // layout [column tile][warp][lane]: consecutive lanes write consecutive 16-byte words
#pragma unroll
    for (int j = 0; j < NJ; ++j)
        *reinterpret_cast<float4 *>(sm_o + (size_t)((j * NW + warp) * 32 + lane) * 4) =
            make_float4(ts.O[j][0], ts.O[j][1], ts.O[j][2], ts.O[j][3]);
    *reinterpret_cast<float4 *>(sm_ml + (warp * 32 + lane) * 4) = make_float4(ts.m_run[0], ts.l_run[0], ts.m_run[1], ts.l_run[1]);
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
            int hq, i;
            split_row(r2, ms, hq, i);
            const int c = seg.row0 + i, qh = kvh * group + hq;
            if (n_slots == 1) {
                const float inv = 1.f / Lv[h];
                uint32_t hi, lo;
                split_bf16x2(ov2[h][0] * inv, ov2[h][1] * inv, hi, lo);
                *reinterpret_cast<uint32_t *>(a.B.ATT + (size_t)c * qdim + qh * HD + 8 * j + 2 * t) = hi;
                *reinterpret_cast<uint32_t *>(a.B.ATTL + (size_t)c * qdim + qh * HD + 8 * j + 2 * t) = lo;
            } else {
                const size_t pi = ((size_t)c * a.D.nh + qh) * n_slots + slot;
                *reinterpret_cast<float2 *>(a.B.APO + pi * HD + 8 * j + 2 * t) = make_float2(ov2[h][0], ov2[h][1]);
                if (j == 0 && t == 0) *reinterpret_cast<float2 *>(a.B.APML + pi * 2) = make_float2(Mv[h], Lv[h]);
            }
        }
    }
    __syncthreads();
}

// Keys of pages [p_begin, p_end) that lie in [k_lo, k_hi] and are not in the future of the query row,
// fragments loaded straight from global memory.  `sm` is the CTA's dynamic shared memory
// (smem_bytes(HD)); all 256 threads call.
template <int HD>
__device__ __forceinline__ void partial(const AttnView &a, float *sm, const Segment seg, int kvh, int p_begin, int p_end,
                                        int k_lo, int k_hi, int slot, int n_slots) {
    constexpr int KS = HD / 32, NJ = HD / 8;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int R = seg.nrows * (a.D.nh / a.D.nkv), n_mt = (R + 15) >> 4;
    const int P = n_mt >= 3 ? 4 : n_mt;             // query tiles handled concurrently: 1, 2 or 4
    const int n_kl = NW / P, kl = warp / P;
    const float sc = rsqrtf((float)HD) * LOG2E;
    const int32_t *pt = a.B.PT + seg.seq * a.D.pages_per_seq;
    const size_t page_stride = (size_t)a.D.L * a.D.nkv * 16 * HD;
    const size_t head_off = ((size_t)(a.layer - 1) * a.D.nkv + kvh) * 16 * HD;
    const int n_iter = (n_mt + P - 1) / P;
    const int key0 = 4 * (g >> 1) + (g & 1);        // token of score-tile 0 column g; tile 1: +2

    // Keys and values of positions committed in earlier rounds (below a.early_pos) cannot change any more: every
    // warp requests its first such page before it waits for the producer kernel, so that the cache's round trip to
    // memory runs during the producer's tail.
    const int p_first = p_begin + kl;
    const bool pre = n_iter == 1 && p_first < p_end && p_first < (a.early_pos >> 4);
    uint4 kf0[2][KS];
    uint2 vf0[NJ];
    if (pre) {
        const int pg0 = pt[p_first];
        const bf16 *kpage = a.B.KP + (size_t)pg0 * page_stride + head_off;
        const bf16 *vpage = a.B.VP + (size_t)pg0 * page_stride + head_off;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            kf0[0][ks] = ldg_act16(kpage + key0 * HD + 32 * ks + 8 * t);
            kf0[1][ks] = ldg_act16(kpage + (key0 + 2) * HD + 32 * ks + 8 * t);
        }
#pragma unroll
        for (int j = 0; j < NJ; ++j) vf0[j] = ldg_act8(vpage + (8 * j + g) * 16 + 4 * t);
        // when weights are requested below: the warp's further committed pages first, into L2 (one page per lane, two
        // bulk requests per page), so that none of attention's own reads queues behind the weights
        for (int p2 = p_first + n_kl * (1 + lane); a.pf->n > 0 && p2 < p_end && p2 < (a.early_pos >> 4); p2 += n_kl * 32) {
            const size_t off = (size_t)pt[p2] * page_stride + head_off;
            l2_prefetch_bulk(a.B.KP + off, 16 * HD * 2);
            l2_prefetch_bulk(a.B.VP + off, 16 * HD * 2);
        }
    }
    prefetch_weights(*a.pf);
    pdl_wait();

    for (int it = 0; it < n_iter; ++it) {
        const int mt = it * P + warp % P;
        TileState<HD> ts;
        tile_begin<HD>(ts, a, seg, kvh, mt, n_mt, k_hi);
        if (mt < n_mt) {
            if (pre) page_update<HD>(ts, kf0, vf0, p_first, k_lo, sc);
            for (int pb = p_first + (pre ? n_kl : 0); pb < p_end; pb += n_kl * PG) {
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
                    page_update<HD>(ts, kf, vf, p, k_lo, sc);
                }
            }
        }
        tile_end<HD>(ts, a, sm, seg, kvh, it, P, n_mt, slot, n_slots);
    }
}

// ---- staged variant: the key/value pages travel to shared memory with asynchronous copies
//
// When a CTA serves several query tiles (many rows, or grouped-query attention), every tile needs every
// page of the key range.  Loading the fragments per tile straight from global memory multiplies the L2
// traffic by the number of tiles and pays one dependent load latency per page and warp.  Here all 256
// threads copy whole pages into shared memory (two chunks of pages resident, later chunks requested two
// chunks ahead of their use) and the warps of all tiles read their fragments from there.
//
// Shared-memory layout of a page slot: 16 key rows of HD bf16 whose 64-byte groups are swapped pairwise
// in odd rows (a quarter-warp's fragment loads touch an even and an odd row at the same column, which
// would otherwise share banks), followed by the V^T block [HD][16] as stored in the cache.
template <int HD>
struct Stage {
    static constexpr int KROW = HD * 2;                 // bytes per key row
    static constexpr int KBYTES = 16 * KROW;
    static constexpr int PAGE = KBYTES + HD * 32;       // bytes per page slot
    static constexpr int CH = HD == 128 ? 6 : 12;       // pages per chunk; two chunks are resident
    static constexpr size_t BYTES = 2 * (size_t)CH * PAGE;
};

__host__ __device__ constexpr size_t staged_smem_bytes(int hd) {
    return hd == 128 ? (Stage<128>::BYTES > smem_bytes(128) ? Stage<128>::BYTES : smem_bytes(128))
                     : (Stage<64>::BYTES > smem_bytes(64) ? Stage<64>::BYTES : smem_bytes(64));
}

// Same contract as partial().  `smem`: staged_smem_bytes(HD), 16-byte aligned.
template <int HD>
__device__ __forceinline__ void partial_staged(const AttnView &a, unsigned char *smem, const Segment seg, int kvh, int p_begin,
                                               int p_end, int k_lo, int k_hi, int slot, int n_slots) {
    using S = Stage<HD>;
    constexpr int KS = HD / 32, NJ = HD / 8, CH = S::CH;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int R = seg.nrows * (a.D.nh / a.D.nkv), n_mt = (R + 15) >> 4;
    const int P = n_mt >= 3 ? 4 : n_mt;
    const int n_kl = NW / P, kl = warp / P;
    const float sc = rsqrtf((float)HD) * LOG2E;
    const int32_t *pt = a.B.PT + seg.seq * a.D.pages_per_seq;
    const size_t page_stride = (size_t)a.D.L * a.D.nkv * 16 * HD;
    const size_t head_off = ((size_t)(a.layer - 1) * a.D.nkv + kvh) * 16 * HD;
    const int key0 = 4 * (g >> 1) + (g & 1);
    const int n_pages = max(p_end - p_begin, 0), n_chunks = (n_pages + CH - 1) / CH;
    const int n_iter = (n_mt + P - 1) / P;          // groups of P concurrent query tiles; each group stages the pages again

    prefetch_weights(*a.pf);
    pdl_wait();
    // every thread copies the same pieces of every page: 2*HD 16-byte pieces of keys, 2*HD of values
    auto issue = [&](int c) {
        if (c < n_chunks) {
            unsigned char *buf = smem + (size_t)(c & 1) * CH * S::PAGE;
            const int p0 = p_begin + c * CH;
            int pg[CH];
#pragma unroll
            for (int q = 0; q < CH; ++q) pg[q] = p0 + q < p_end ? pt[p0 + q] : 0;
#pragma unroll
            for (int q = 0; q < CH; ++q) {
                const int p = p0 + q;
                if (p < p_end) {
                    const size_t off = (size_t)pg[q] * page_stride + head_off;
                    const unsigned char *kp = reinterpret_cast<const unsigned char *>(a.B.KP + off);
                    const unsigned char *vp = reinterpret_cast<const unsigned char *>(a.B.VP + off);
                    unsigned char *dst = buf + (size_t)q * S::PAGE;
#pragma unroll
                    for (int pc = tid; pc < 4 * HD; pc += NW * 32) {
                        if (pc < 2 * HD) {
                            const int row = pc / (HD / 8), col = pc - row * (HD / 8);
                            cp_async16(dst + row * S::KROW + (col ^ ((row & 1) << 2)) * 16, kp + (size_t)pc * 16, true);
                        } else {
                            cp_async16(dst + S::KBYTES + (pc - 2 * HD) * 16, vp + (size_t)(pc - 2 * HD) * 16, true);
                        }
                    }
                }
            }
        }
        cp_async_commit();
    };
    for (int it = 0; it < n_iter; ++it) {
    issue(0);
    issue(1);
    const int mt = it * P + warp % P;
    TileState<HD> ts;
    tile_begin<HD>(ts, a, seg, kvh, mt, n_mt, k_hi);
    for (int c = 0; c < n_chunks; ++c) {
        cp_async_wait<1>();                          // chunk c has landed (chunk c + 1 may be in flight)
        __syncthreads();
        const unsigned char *buf = smem + (size_t)(c & 1) * CH * S::PAGE;
        if (mt < n_mt) {
            for (int q = kl; q < CH; q += n_kl) {
                const int p = p_begin + c * CH + q;
                if (p >= p_end) break;
                const unsigned char *kb = buf + (size_t)q * S::PAGE, *vb = kb + S::KBYTES;
                uint4 kf[2][KS];
                uint2 vf[NJ];
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    kf[0][ks] = *reinterpret_cast<const uint4 *>(kb + key0 * S::KROW + 64 * (ks ^ (g & 1)) + 16 * t);
                    kf[1][ks] = *reinterpret_cast<const uint4 *>(kb + (key0 + 2) * S::KROW + 64 * (ks ^ (g & 1)) + 16 * t);
                }
#pragma unroll
                for (int j = 0; j < NJ; ++j) vf[j] = *reinterpret_cast<const uint2 *>(vb + (8 * j + g) * 32 + 8 * t);
                page_update<HD>(ts, kf, vf, p, k_lo, sc);
            }
        }
        __syncthreads();                             // the buffer is free again
        issue(c + 2);
    }
    cp_async_wait<0>();
    __syncthreads();                                 // the merge below reuses the staging memory
    tile_end<HD>(ts, a, reinterpret_cast<float *>(smem), seg, kvh, it, P, n_mt, slot, n_slots);   // ends with a barrier
    }
}

// Combines slots 0..n_slots-1 of every (row, head) of a (segment, kv head) in slot order and writes the
// normalised bf16 result.  The caller has made the slots visible (fence + barrier / arrival counter).
// NS = compile-time bound on the slots, UE = elements a thread works on at once: the loads of an iteration
// (UE * NS partial states) are all in flight together.
template <int HD, int NS, int UE>
__device__ __forceinline__ void merge_slots_n(const AttnView &a, const Segment seg, int kvh, int n_slots) {
    const int ms = seg.nrows, group = a.D.nh / a.D.nkv, R = ms * group, qdim = a.D.nh * HD;
    const int n_el = R * (HD / 4);
    for (int e0 = threadIdx.x; e0 < n_el; e0 += NW * 32 * UE) {
        uint2 mlv[UE][NS];
        uint4 ovv[UE][NS];
        size_t out_off[UE];
        bool live[UE];
        // all loads first, then the arithmetic: two memory latencies per iteration in total
#pragma unroll
        for (int u = 0; u < UE; ++u) {
            const int e = e0 + u * NW * 32;
            live[u] = e < n_el;
            const int ee = live[u] ? e : 0;
            const int row = ee / (HD / 4), d4 = (ee - row * (HD / 4)) * 4;
            int hq, i;
            split_row(row, ms, hq, i);
            const int c = seg.row0 + i, qh = kvh * group + hq;
            const size_t pi = ((size_t)c * a.D.nh + qh) * n_slots;
            out_off[u] = (size_t)c * qdim + qh * HD + d4;
#pragma unroll
            for (int s = 0; s < NS; ++s) {
                const int se = s < n_slots ? s : n_slots - 1;       // clamped: unused slots are masked below
                mlv[u][s] = ldg_act8(a.B.APML + (pi + se) * 2);
                ovv[u][s] = ldg_act16(a.B.APO + (pi + se) * HD + d4);
            }
        }
#pragma unroll
        for (int u = 0; u < UE; ++u) {
            float M = -INFINITY;
#pragma unroll
            for (int s = 0; s < NS; ++s) {
                if (s >= n_slots) mlv[u][s].x = 0xff800000u;        // -inf: weight 0
                M = fmaxf(M, __uint_as_float(mlv[u][s].x));
            }
            float l = 0.f, o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
#pragma unroll
            for (int s = 0; s < NS; ++s) {
                const float f = exp2f(__uint_as_float(mlv[u][s].x) - M);
                l += f * __uint_as_float(mlv[u][s].y);
                o0 += f * __uint_as_float(ovv[u][s].x); o1 += f * __uint_as_float(ovv[u][s].y);
                o2 += f * __uint_as_float(ovv[u][s].z); o3 += f * __uint_as_float(ovv[u][s].w);
            }
            const float inv = 1.f / l;
            uint2 pk, pl;
            split_bf16x2(o0 * inv, o1 * inv, pk.x, pl.x);
            split_bf16x2(o2 * inv, o3 * inv, pk.y, pl.y);
            if (live[u]) {
                *reinterpret_cast<uint2 *>(a.B.ATT + out_off[u]) = pk;
                *reinterpret_cast<uint2 *>(a.B.ATTL + out_off[u]) = pl;
            }
        }
    }
}

template <int HD>
__device__ __forceinline__ void merge_slots(const AttnView &a, const Segment seg, int kvh, int n_slots) {
    // a decode-sized segment has at most one element per thread: one element per thread (least index arithmetic in
    // front of the loads) and no more loads than the split count needs (1 % of a round against always loading
    // 16 clamped slots); large segments (prefill passes) batch several elements per thread
    const int n_el = seg.nrows * (a.D.nh / a.D.nkv) * (HD / 4);
    if (n_el <= NW * 32) {
        if (n_slots <= 2) merge_slots_n<HD, 2, 1>(a, seg, kvh, n_slots);
        else if (n_slots <= 4) merge_slots_n<HD, 4, 1>(a, seg, kvh, n_slots);
        else if (n_slots <= 8) merge_slots_n<HD, 8, 1>(a, seg, kvh, n_slots);
        else merge_slots_n<HD, 16, 1>(a, seg, kvh, n_slots);
    } else if (n_slots > 8) merge_slots_n<HD, 16, 1>(a, seg, kvh, n_slots);
    else if (n_slots <= 4) merge_slots_n<HD, 4, 4>(a, seg, kvh, n_slots);
    else merge_slots_n<HD, 8, 2>(a, seg, kvh, n_slots);
}

}  // namespace attn
