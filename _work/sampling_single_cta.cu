// Speculative sampling (Sec. 2) on rows of logits: temperature, nucleus (top-p) filtering, inverse-CDF draws,
// the acceptance test min(1, p/q) and the residual distribution max(0, p - q).
//
// One CTA works on one row.  Token weights are integers W = round(exp((z - max) / T) * 2^40): sums of integers
// do not depend on the order of addition, so every decision below is reproducible whatever the reduction
// tree looks like.  The nucleus is found without sorting: a token is kept iff the mass of the tokens with a
// larger weight is below top_p * (total mass); the smallest kept weight (as the fp32 bit pattern of the
// weight, `kstar`) is located by a radix descent over the 32 key bits, four bits per pass, each pass summing
// the mass per bucket.  Tokens whose key equals kstar enter in token-id order (`tie_keep` of them).
#include "../../include/del.h"
#include "kernels.h"

namespace {

constexpr int SNT = 512;                   // threads per CTA
constexpr int NBK = 16;                    // buckets per radix pass
constexpr int KEY_CACHE_MAX = 36864;       // rows up to this many tokens keep their keys in shared memory
typedef unsigned long long u64;

// finaliser of the splitmix64 generator; the uniform number of (seed, position, purpose) has 53 bits
__device__ __forceinline__ u64 mix64(u64 x) {
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27; x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}
__device__ __forceinline__ double uniform01(u64 seed, long long pos, int purpose) {
    const u64 ctr = (u64)pos * 4ull + (u64)purpose + 1ull;
    const u64 x = mix64(seed ^ mix64(ctr * 0x9E3779B97F4A7C15ull));
    return (double)(x >> 11) * (1.0 / 9007199254740992.0);
}

__device__ __forceinline__ uint32_t weight_key(float z, float m, double inv_T) {
    // the argument in double (one rounding to fp32), the exponential in fp32
    return __float_as_uint(expf((float)(((double)z - (double)m) * inv_T)));
}
// W = round-to-nearest-even(w * 2^40) for the weight w in [0, 1] whose fp32 bit pattern is `key`, with integer
// shifts only (a float -> integer conversion per token and pass would keep the conversion unit busy)
__device__ __forceinline__ u64 key_weight(uint32_t key) {
    const int sh = (int)(key >> 23) - 127 + 17;              // w = mant * 2^(e - 23), W = mant * 2^(e + 17)
    const uint32_t mant = (key & 0x7fffffu) | 0x800000u;
    if (sh >= 0) return (u64)mant << sh;                     // (w <= 1: sh <= 17)
    const int s = -sh;
    if (s > 24 || key < 0x00800000u) return 0ull;            // below half a unit (or denormal / zero)
    const uint32_t q = mant >> s, rem = mant & ((1u << s) - 1u), half = 1u << (s - 1);
    return (u64)(q + ((rem > half) || (rem == half && (q & 1u))));
}

struct Smem {
    u64 *hist;            // [NBK][SNT]
    u64 *part;            // [NBK][2] / scan scratch
    uint32_t *keys;       // [V] or nullptr
};

__device__ __forceinline__ float block_max(float v, float *scratch) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = scratch[0];
    for (int w = 1; w < SNT / 32; ++w) r = fmaxf(r, scratch[w]);
    return r;
}
__device__ __forceinline__ u64 warp_sum_u64(u64 v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
// sum over the block, the same value in every thread
__device__ __forceinline__ u64 block_sum_u64(u64 v, u64 *scratch) {
    v = warp_sum_u64(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    u64 r = 0;
    for (int w = 0; w < SNT / 32; ++w) r += scratch[w];
    return r;
}
// exclusive prefix over the threads of the block (thread order), plus the total
template <typename T>
__device__ __forceinline__ T block_excl_scan(T v, T *scratch, T &total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    T inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const T t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();
    if (lane == 31) scratch[warp] = inc;
    __syncthreads();
    T base = 0, tot = 0;
    for (int w = 0; w < SNT / 32; ++w) {
        if (w < warp) base += scratch[w];
        tot += scratch[w];
    }
    total = tot;
    return base + inc - v;
}

// Index of token i in the shared-memory key cache: one pad word per 32 tokens, so that both the strided
// passes (consecutive lanes, consecutive tokens) and the chunked passes (lane t at token t * c) spread over
// the banks.
__device__ __forceinline__ int kidx(int i) { return i + (i >> 5); }

// Statistics of the filtered distribution of one logit row; every thread returns the same values.
__device__ RowStat row_stats(const float *z, int V, double inv_T, double top_p, const Smem &sm) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    float mx = -INFINITY;
#pragma unroll 8
    for (int i = tid; i < V; i += SNT) mx = fmaxf(mx, __ldcg(z + i));
    const float m = block_max(mx, reinterpret_cast<float *>(sm.part));
    u64 zsum = 0;
#pragma unroll 8
    for (int i = tid; i < V; i += SNT) {
        const uint32_t key = weight_key(__ldcg(z + i), m, inv_T);
        if (sm.keys) sm.keys[kidx(i)] = key;
        zsum += key_weight(key);
    }
    RowStat r;
    r.m = m;
    r.Z = block_sum_u64(zsum, sm.part);
    if (top_p >= 1.0) {                      // everything stays
        r.kstar = 0; r.tie_keep = 0x7fffffff; r.cnt_eq = 0; r.K = r.Z;
        return r;
    }
    const double tgt = top_p * (double)r.Z;
    // radix descent to kstar = the smallest key k with (mass of the keys above k) < tgt; A = that mass
    uint32_t prefix = 0;
    u64 A = 0;
    for (int s = 28; s >= 0; s -= 4) {
#pragma unroll
        for (int b = 0; b < NBK; ++b) sm.hist[b * SNT + tid] = 0;
        const uint32_t hi_shift = s == 28 ? 0 : s + 4;       // (a shift by 32 is not defined: the top pass takes all keys)
        const uint32_t want = s == 28 ? 0 : prefix;
        // runs of tokens that fall into the same bucket are summed in a register first (in the upper passes
        // nearly all candidates share one bucket, and a read-modify-write chain through shared memory is slow)
        int cb = -1;
        u64 run = 0;
#pragma unroll 4
        for (int i = tid; i < V; i += SNT) {
            const uint32_t key = sm.keys ? sm.keys[kidx(i)] : weight_key(__ldcg(z + i), m, inv_T);
            const bool in = s == 28 || (key >> hi_shift) == want;
            if (in) {
                const int b = (int)((key >> s) & 15u);
                if (b != cb) {
                    if (cb >= 0) sm.hist[cb * SNT + tid] += run;
                    cb = b;
                    run = 0;
                }
                run += key_weight(key);
            }
        }
        if (cb >= 0) sm.hist[cb * SNT + tid] += run;
        __syncthreads();
        u64 acc = 0;                         // warp w sums bucket w (SNT / 32 == NBK warps)
#pragma unroll
        for (int k = 0; k < SNT / 32; ++k) acc += sm.hist[warp * SNT + lane + 32 * k];
        acc = warp_sum_u64(acc);
        if (lane == 0) sm.part[warp] = acc;
        __syncthreads();
        // S_t = mass above bucket t; it grows as t falls; the bucket of kstar is the lowest t with S_t < tgt
        u64 St = A, chosen = A;
        int tstar = 15;
        for (int t = 15; t >= 0; --t) {
            if (!((double)St < tgt)) break;
            tstar = t;
            chosen = St;
            St += sm.part[t];
        }
        prefix = (prefix << 4) | (uint32_t)tstar;
        A = chosen;
        __syncthreads();
    }
    u64 eq = 0;
#pragma unroll 4
    for (int i = tid; i < V; i += SNT) {
        const uint32_t key = sm.keys ? sm.keys[kidx(i)] : weight_key(__ldcg(z + i), m, inv_T);
        eq += key == prefix;
    }
    const int cnt_eq = (int)block_sum_u64(eq, sm.part);
    const u64 wstar = key_weight(prefix);
    int tie_keep = cnt_eq;
    if (cnt_eq > 0 && wstar > 0) {
        // tied token number j (1-based) has A + (j - 1) * wstar ahead of it: kept while that is below tgt
        const double x = ceil((tgt - (double)A) / (double)wstar);
        tie_keep = x >= (double)cnt_eq ? cnt_eq : (x < 1.0 ? 1 : (int)x);
    }
    r.kstar = prefix;
    r.cnt_eq = cnt_eq;
    r.tie_keep = tie_keep;
    r.K = A + (u64)tie_keep * wstar;
    return r;
}

// contiguous chunk of the row owned by a thread in the order-dependent passes (multiple of 4 tokens)
__device__ __forceinline__ void chunk_of(int V, int &i0, int &i1) {
    const int c = (((V + SNT - 1) / SNT) + 3) & ~3;
    i0 = min(V, (int)threadIdx.x * c);
    i1 = min(V, i0 + c);
}

// f(i, key of token i) over the thread's chunk in token-id order: keys from the shared-memory cache when the
// row has one (`keys` belongs to this row), else recomputed from 16-byte loads of the logits
template <typename F>
__device__ __forceinline__ void for_chunk(const float *z, const uint32_t *keys, int V, float m, double inv_T, F f) {
    int i0, i1;
    chunk_of(V, i0, i1);
    if (keys != nullptr) {
#pragma unroll 4
        for (int i = i0; i < i1; ++i) f(i, keys[kidx(i)]);
        return;
    }
    int i = i0;
#pragma unroll 2
    for (; i + 4 <= i1; i += 4) {
        const float4 v = __ldcg(reinterpret_cast<const float4 *>(z + i));
        const uint32_t k0 = weight_key(v.x, m, inv_T), k1 = weight_key(v.y, m, inv_T), k2 = weight_key(v.z, m, inv_T),
                       k3 = weight_key(v.w, m, inv_T);
        f(i, k0); f(i + 1, k1); f(i + 2, k2); f(i + 3, k3);
    }
    for (; i < i1; ++i) f(i, weight_key(__ldcg(z + i), m, inv_T));
}

// kept weight of a token met in token-id order (eq_seen counts the tokens with key == kstar met so far)
__device__ __forceinline__ u64 kept_weight(uint32_t key, const RowStat &st, int &eq_seen) {
    if (key > st.kstar) return key_weight(key);
    if (key == st.kstar) return eq_seen++ < st.tie_keep ? key_weight(key) : 0ull;
    return 0ull;
}

// tokens with key == kstar in the chunks of the threads before this one (only needed when some ties are dropped)
__device__ __forceinline__ int ties_before(const float *z, const uint32_t *keys, int V, const RowStat &st, double inv_T,
                                           int *scratch) {
    if (st.tie_keep >= st.cnt_eq) return 0;                 // every tie is kept: the rank does not matter
    int n = 0, total;
    for_chunk(z, keys, V, st.m, inv_T, [&](int, uint32_t key) { n += key == st.kstar; });
    return block_excl_scan<int>(n, scratch, total);
}

__device__ __forceinline__ int block_min_int(int v, int *scratch) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    int r = scratch[0];
    for (int w = 1; w < SNT / 32; ++w) r = min(r, scratch[w]);
    return r;
}

// Inverse CDF in token-id order over the filtered distribution: the first token whose cumulative kept mass
// exceeds u * K (the last kept token if rounding leaves none).  Same result in every thread.  `keys`: the
// row's key cache in shared memory, or nullptr.
__device__ int pick_token(const float *z, const uint32_t *keys, int V, const RowStat &st, double inv_T, double u, const Smem &sm) {
    const int eq0 = ties_before(z, keys, V, st, inv_T, reinterpret_cast<int *>(sm.part));
    int eq = eq0;
    u64 mine = 0;
    for_chunk(z, keys, V, st.m, inv_T, [&](int, uint32_t key) { mine += kept_weight(key, st, eq); });
    u64 total;
    u64 cum = block_excl_scan<u64>(mine, sm.part, total);
    const double tu = u * (double)st.K;
    int cand = 0x7fffffff, last = -1;
    // only the thread whose chunk holds the crossing walks it again (integers: the test is exact); if rounding
    // of u * K leaves no crossing at all, every thread with mass reports its last kept token instead
    const bool crossing = (double)(cum + mine) > tu && !((double)cum > tu);
    const bool none = !((double)total > tu);
    if (crossing || (none && mine > 0)) {
        eq = eq0;
        for_chunk(z, keys, V, st.m, inv_T, [&](int i, uint32_t key) {
            const u64 w = kept_weight(key, st, eq);
            cum += w;
            if (w > 0) last = i;
            if (w > 0 && cand == 0x7fffffff && (double)cum > tu) cand = i;
        });
    }
    const int first = block_min_int(cand, reinterpret_cast<int *>(sm.part));
    if (first != 0x7fffffff) return first;
    return -block_min_int(-last, reinterpret_cast<int *>(sm.part));
}

// filtered probability of token x; same value in every thread
__device__ double token_prob(const float *z, int V, int x, const RowStat &st, double inv_T, const Smem &sm) {
    const uint32_t key = weight_key(__ldcg(z + x), st.m, inv_T);
    if (key < st.kstar) return 0.0;
    if (key == st.kstar && st.tie_keep < st.cnt_eq) {
        u64 n = 0;                           // rank of x among the tied tokens
#pragma unroll 4
        for (int i = threadIdx.x; i < x; i += SNT) n += weight_key(__ldcg(z + i), st.m, inv_T) == st.kstar;
        if ((int)block_sum_u64(n, sm.part) >= st.tie_keep) return 0.0;
    }
    return (double)key_weight(key) / (double)st.K;
}

// Token from the normalised max(0, p - q) of two filtered rows (from p itself if nothing is left).
__device__ int pick_residual(const float *zp, const float *zq, int V, const RowStat &sp, const RowStat &sq, double inv_T, double u,
                             const Smem &sm) {
    int i0, i1;
    chunk_of(V, i0, i1);
    const int ep0 = ties_before(zp, nullptr, V, sp, inv_T, reinterpret_cast<int *>(sm.part));
    const int eq0 = ties_before(zq, nullptr, V, sq, inv_T, reinterpret_cast<int *>(sm.part));
    const double ikp = 1.0 / (double)sp.K, ikq = 1.0 / (double)sq.K;
    // residual mass of tokens i .. i+3 of the two rows (16-byte loads; the chunks are multiples of 4 tokens, V too)
    auto quad = [&](int i, int &ep, int &eq, double (&r)[4]) {
        const float4 a = __ldcg(reinterpret_cast<const float4 *>(zp + i)), b = __ldcg(reinterpret_cast<const float4 *>(zq + i));
        const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const double p = (double)kept_weight(weight_key(av[j], sp.m, inv_T), sp, ep) * ikp;
            const double q = (double)kept_weight(weight_key(bv[j], sq.m, inv_T), sq, eq) * ikq;
            r[j] = p > q ? p - q : 0.0;
        }
    };
    int ep = ep0, eq = eq0;
    double mine = 0.0;
#pragma unroll 2
    for (int i = i0; i < i1; i += 4) {
        double r[4];
        quad(i, ep, eq, r);
        mine += r[0]; mine += r[1]; mine += r[2]; mine += r[3];
    }
    double R;
    double cum = block_excl_scan<double>(mine, reinterpret_cast<double *>(sm.part), R);
    if (!(R > 0.0)) return pick_token(zp, nullptr, V, sp, inv_T, u, sm);
    const double tu = u * R;
    int cand = 0x7fffffff, last = -1;
    // the threads whose chunk may hold the crossing walk it again; the band is a little wide because a chunk's
    // mass added at once and added term by term can differ in the last bits
    const bool near = cum + mine >= tu * (1.0 - 1e-12) && cum <= tu * (1.0 + 1e-12);
    const bool none = !(R > tu * (1.0 + 1e-9));
    if (mine > 0.0 && (near || none)) {
        ep = ep0; eq = eq0;
        for (int i = i0; i < i1; i += 4) {
            double r[4];
            quad(i, ep, eq, r);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                cum += r[j];
                if (r[j] > 0.0) last = i + j;
                if (r[j] > 0.0 && cand == 0x7fffffff && cum > tu) cand = i + j;
            }
        }
    }
    const int first = block_min_int(cand, reinterpret_cast<int *>(sm.part));
    if (first != 0x7fffffff) return first;
    return -block_min_int(-last, reinterpret_cast<int *>(sm.part));
}

__device__ __forceinline__ Smem carve_smem(unsigned char *raw, int V, bool with_hist) {
    Smem sm;
    sm.part = reinterpret_cast<u64 *>(raw);                       // 64 words of scratch
    sm.hist = with_hist ? sm.part + 64 : nullptr;
    sm.keys = with_hist && V <= KEY_CACHE_MAX ? reinterpret_cast<uint32_t *>(sm.hist + NBK * SNT) : nullptr;   // [V + V / 32]
    return sm;
}

__device__ __forceinline__ const float *logit_row(const float *base, int seq, int row, int V) {
    return base + ((size_t)seq * DEL_SAMPLE_ROWS + row) * V;
}

// Draft i of a sequence: the exit head's row is filtered, the token drawn (purpose 0 at position T + 1 + i) and
// stored as draft i; the row's statistics stay for the acceptance tests.
__global__ void __launch_bounds__(SNT) sample_draft_kernel(const __grid_constant__ SampleArgs a) {
    extern __shared__ __align__(16) unsigned char raw[];
    pdl_launch();
    pdl_wait();
    const SampleSeq s = a.s[blockIdx.x];
    const int V = a.D.V;
    const Smem sm = carve_smem(raw, V, true);
    const float *z = logit_row(a.B.QLOG, s.seq, s.slot, V);
    const RowStat st = row_stats(z, V, s.inv_T, s.top_p, sm);
    const double u = uniform01(s.seed, s.pos0 + 1 + s.slot, 0);
    const int x = pick_token(z, sm.keys, V, st, s.inv_T, u, sm);
    if (threadIdx.x == 0) {
        a.B.QSTAT[s.seq * DEL_SAMPLE_ROWS + s.slot] = st;
        a.B.TOK[s.seq * (a.D.S + 1) + s.slot + 1] = x;
        a.B.SMP[s.seq].q_x[s.slot] =
            (float)((double)key_weight(weight_key(z[x], st.m, s.inv_T)) / (double)st.K);
    }
}

// Statistics of the target's rows 0..g: grid (rows, sequences)
__global__ void __launch_bounds__(SNT) sample_stats_kernel(const __grid_constant__ SampleArgs a) {
    extern __shared__ __align__(16) unsigned char raw[];
    pdl_launch();
    pdl_wait();
    const SampleSeq s = a.s[blockIdx.y];
    const int row = blockIdx.x, V = a.D.V;
    if (row > s.g) return;
    const Smem sm = carve_smem(raw, V, true);
    const RowStat st = row_stats(logit_row(a.B.PLOG, s.seq, row, V), V, s.inv_T, s.top_p, sm);
    if (threadIdx.x == 0) a.B.PSTAT[s.seq * DEL_SAMPLE_ROWS + row] = st;
}

// Acceptance tests of the drafts in order (purpose 1), then the token that ends the round (purpose 2): from the
// residual of the first rejected position, or from the target's row g when every draft was accepted.
__global__ void __launch_bounds__(SNT) sample_verify_kernel(const __grid_constant__ SampleArgs a) {
    extern __shared__ __align__(16) unsigned char raw[];
    pdl_launch();
    pdl_wait();
    const SampleSeq s = a.s[blockIdx.x];
    const int V = a.D.V;
    const Smem sm = carve_smem(raw, V, false);
    const int32_t *tok = a.B.TOK + s.seq * (a.D.S + 1);
    SampleOut *out = a.B.SMP + s.seq;
    int n = 0, rejected = 0;
    while (n < s.g) {
        const int x = tok[1 + n];
        const RowStat sp = a.B.PSTAT[s.seq * DEL_SAMPLE_ROWS + n], sq = a.B.QSTAT[s.seq * DEL_SAMPLE_ROWS + n];
        const double px = token_prob(logit_row(a.B.PLOG, s.seq, n, V), V, x, sp, s.inv_T, sm);
        const double qx = token_prob(logit_row(a.B.QLOG, s.seq, n, V), V, x, sq, s.inv_T, sm);
        const double u = uniform01(s.seed, s.pos0 + 1 + n, 1);
        if (threadIdx.x == 0) out->p_x[n] = (float)px;
        const double ratio = px / qx;
        if (u < (ratio < 1.0 ? ratio : 1.0)) ++n;
        else { rejected = 1; break; }
    }
    const int n_tests = rejected ? n + 1 : n;
    const double u = uniform01(s.seed, s.pos0 + 1 + n, 2);
    const RowStat sp = a.B.PSTAT[s.seq * DEL_SAMPLE_ROWS + n];
    int last;
    if (rejected) {
        const RowStat sq = a.B.QSTAT[s.seq * DEL_SAMPLE_ROWS + n];
        last = pick_residual(logit_row(a.B.PLOG, s.seq, n, V), logit_row(a.B.QLOG, s.seq, n, V), V, sp, sq, s.inv_T, u, sm);
    } else {
        last = pick_token(logit_row(a.B.PLOG, s.seq, n, V), nullptr, V, sp, s.inv_T, u, sm);
    }
    if (threadIdx.x == 0) {
        out->n_accept = n;
        out->last_token = last;
        out->n_tests = n_tests;
        out->from_residual = rejected;
    }
}

// Test hook: the same device functions on one caller-supplied pair of rows.
__global__ void __launch_bounds__(SNT) sample_probe_kernel(const float *zp, const float *zq, int V, double inv_T, double top_p,
                                                           double u_draft, double u_accept, double u_final, int32_t *out,
                                                           double *prob, RowStat *stat) {
    extern __shared__ __align__(16) unsigned char raw[];
    const Smem sm = carve_smem(raw, V, true);
    const RowStat sq = row_stats(zq, V, inv_T, top_p, sm);
    const RowStat sp = row_stats(zp, V, inv_T, top_p, sm);
    const int x = pick_token(zq, nullptr, V, sq, inv_T, u_draft, sm);
    const double qx = token_prob(zq, V, x, sq, inv_T, sm), px = token_prob(zp, V, x, sp, inv_T, sm);
    const double ratio = px / qx;
    const int accepted = u_accept < (ratio < 1.0 ? ratio : 1.0);
    // both endings are reported: the residual draw (as if rejected) and the draw from p (as if all were accepted)
    const int res = pick_residual(zp, zq, V, sp, sq, inv_T, u_final, sm);
    const int bonus = pick_token(zp, sm.keys, V, sp, inv_T, u_final, sm);
    if (threadIdx.x == 0) {
        out[0] = x; out[1] = accepted; out[2] = res; out[3] = bonus;
        prob[0] = qx; prob[1] = px;
        stat[0] = sq; stat[1] = sp;
    }
}

template <typename... KArgs, typename... Args>
cudaError_t launch(void (*kern)(KArgs...), dim3 grid, int smem, cudaStream_t st, bool pdl, Args... args) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(SNT);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

}  // namespace

int sample_smem_bytes(int V) {
    return 64 * 8 + NBK * SNT * 8 + (V <= KEY_CACHE_MAX ? (V + V / 32 + 1) * 4 : 0);
}
cudaError_t launch_sample_draft(const SampleArgs &a, cudaStream_t st, bool pdl) {
    return launch(sample_draft_kernel, dim3(a.n), sample_smem_bytes(a.D.V), st, pdl, a);
}
cudaError_t launch_sample_stats(const SampleArgs &a, int max_rows, cudaStream_t st, bool pdl) {
    return launch(sample_stats_kernel, dim3(max_rows, a.n), sample_smem_bytes(a.D.V), st, pdl, a);
}
cudaError_t launch_sample_verify(const SampleArgs &a, cudaStream_t st, bool pdl) {
    return launch(sample_verify_kernel, dim3(a.n), 64 * 8, st, pdl, a);
}
cudaError_t launch_sample_probe(const float *p_logits, const float *q_logits, int V, double inv_T, double top_p, double u_draft,
                                double u_accept, double u_final, int32_t *out, double *prob, RowStat *stat, cudaStream_t st) {
    return launch(sample_probe_kernel, dim3(1), sample_smem_bytes(V), st, false, p_logits, q_logits, V, inv_T, top_p, u_draft,
                  u_accept, u_final, out, prob, stat);
}
