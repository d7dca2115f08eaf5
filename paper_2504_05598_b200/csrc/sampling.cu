// Speculative sampling (Sec. 2) on rows of logits: temperature, nucleus (top-p) filtering, inverse-CDF draws,
// the acceptance test min(1, p/q) and the residual distribution max(0, p - q).
//
// A thread-block cluster of CL CTAs works on one row: thread t of CTA r owns the EPT consecutive tokens
// starting at (r * SNT + t) * EPT, whose weight keys stay in registers; partial results cross the cluster
// through distributed shared memory (each CTA posts its words in its own shared memory, one cluster barrier,
// every CTA reads all posts and combines them in rank order, so all CTAs hold identical values and take
// identical branches).  The cluster barrier is the hardware one between co-scheduled CTAs: nothing spins.
//
// Token weights are integers W = round(exp((z - max) / T) * 2^40): sums of integers do not depend on the
// order of addition, so every decision is reproducible whatever the reduction tree looks like.  The nucleus
// is found without sorting: a token is kept iff the mass of the tokens with a larger weight is below
// top_p * (total mass); the smallest kept weight (as the fp32 bit pattern of the weight, `kstar`) is located
// by a radix descent over the 32 key bits, four bits per pass, each pass summing the mass per bucket.
// Tokens whose key equals kstar enter in token-id order (`tie_keep` of them).
#include "../../include/del.h"
#include "kernels.h"

#include <cooperative_groups.h>

namespace cg = cooperative_groups;

namespace {

constexpr int SNT = 512;                   // threads per CTA
constexpr int CL = 8;                      // CTAs per cluster (one cluster per row)
constexpr int NBK = 16;                    // buckets per radix pass
constexpr int XW = 32;                     // words of one exchange slot
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

// per-CTA view of the cluster and of this CTA's shared memory
struct Ctx {
    unsigned rank;
    u64 *hist;            // [NBK][SNT] per-thread bucket masses of a radix pass
    u64 *scr;             // [64] scratch of the block-level reductions
    u64 *mine;            // [XW] this CTA's words of the next exchange
    u64 *xch;             // [2][XW] posted words, read by the other CTAs
    u64 *all;             // [XW] result of an exchange
    int par;
};

__device__ __forceinline__ Ctx make_ctx(unsigned char *raw) {
    Ctx c;
    c.rank = cg::this_cluster().block_rank();
    c.scr = reinterpret_cast<u64 *>(raw);
    c.mine = c.scr + 64;
    c.xch = c.mine + XW;
    c.all = c.xch + 2 * XW;
    c.hist = c.all + XW;
    c.par = 0;
    return c;
}
constexpr int SMEM_BYTES = (64 + XW + 2 * XW + XW + NBK * SNT) * 8;

// Posts c.mine[0..n) (written by any threads of this CTA before the call) and waits for every CTA's post.
// Two slots alternate, so one cluster barrier per exchange suffices: a slot is written again only after a
// later barrier, which every CTA reaches after it has read the earlier post.
__device__ __forceinline__ void post_and_wait(Ctx &c, int n) {
    __syncthreads();
    if ((int)threadIdx.x < n) c.xch[c.par * XW + threadIdx.x] = c.mine[threadIdx.x];
    cg::this_cluster().sync();
}
__device__ __forceinline__ const u64 *peer(const Ctx &c, unsigned r) {
    return cg::this_cluster().map_shared_rank(c.xch, r) + c.par * XW;
}
// c.all[j] = sum over the CTAs of their c.mine[j], j < n <= XW; valid in every thread after the call
__device__ __forceinline__ void cluster_sum(Ctx &c, int n) {
    post_and_wait(c, n);
    if ((int)threadIdx.x < n) {
        u64 acc = 0;
        for (unsigned r = 0; r < CL; ++r) acc += peer(c, r)[threadIdx.x];
        c.all[threadIdx.x] = acc;
    }
    c.par ^= 1;
    __syncthreads();
}
// c.all[r * n + j] = CTA r's c.mine[j], j < n, n * CL <= XW
__device__ __forceinline__ void cluster_gather(Ctx &c, int n) {
    post_and_wait(c, n);
    if ((int)threadIdx.x < n * CL) c.all[threadIdx.x] = peer(c, threadIdx.x / n)[threadIdx.x % n];
    c.par ^= 1;
    __syncthreads();
}

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
// exclusive prefix over the threads of the block (thread order), plus the block's total
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
// exclusive prefix over all threads of the cluster in (rank, thread) order = token order; `total` over the cluster
__device__ __forceinline__ u64 cluster_excl_scan_u64(Ctx &c, u64 v, u64 &total) {
    u64 btot;
    const u64 pre = block_excl_scan<u64>(v, c.scr, btot);
    if (threadIdx.x == 0) c.mine[0] = btot;
    cluster_gather(c, 1);
    u64 base = 0, tot = 0;
    for (unsigned r = 0; r < CL; ++r) {
        if (r < c.rank) base += c.all[r];
        tot += c.all[r];
    }
    total = tot;
    return base + pre;
}
__device__ __forceinline__ double cluster_excl_scan_f64(Ctx &c, double v, double &total) {
    double btot;
    const double pre = block_excl_scan<double>(v, reinterpret_cast<double *>(c.scr), btot);
    if (threadIdx.x == 0) c.mine[0] = (u64)__double_as_longlong(btot);
    cluster_gather(c, 1);
    double base = 0.0, tot = 0.0;
    for (unsigned r = 0; r < CL; ++r) {               // rank order: the same sum in every CTA
        const double t = __longlong_as_double((long long)c.all[r]);
        if (r < c.rank) base += t;
        tot += t;
    }
    total = tot;
    return base + pre;
}
// smallest `cand` and largest `last` over the cluster
__device__ __forceinline__ void cluster_min_max(Ctx &c, int cand, int last, int &first, int &final_last) {
    const int bmin = block_min_int(cand, reinterpret_cast<int *>(c.scr));
    const int bmax = -block_min_int(-last, reinterpret_cast<int *>(c.scr));
    if (threadIdx.x == 0) { c.mine[0] = (u64)(uint32_t)bmin; c.mine[1] = (u64)(uint32_t)bmax; }
    cluster_gather(c, 2);
    int f = 0x7fffffff, l = -1;
    for (unsigned r = 0; r < CL; ++r) {
        f = min(f, (int)(uint32_t)c.all[2 * r]);
        l = max(l, (int)(uint32_t)c.all[2 * r + 1]);
    }
    first = f;
    final_last = l;
}

// ---------------------------------------------------------------- a thread's tokens
// first token of this thread
template <int EPT>
__device__ __forceinline__ int my_base(const Ctx &c) { return ((int)c.rank * SNT + (int)threadIdx.x) * EPT; }

// logits of the thread's tokens (-inf beyond the row); V is a multiple of 4, so a group of four is all in or all out
template <int EPT>
__device__ __forceinline__ void load_logits(const float *z, int V, int base, float (&v)[EPT]) {
    if constexpr (EPT % 4 == 0) {
#pragma unroll
        for (int j = 0; j < EPT; j += 4) {
            float4 t = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            if (base + j + 4 <= V) t = __ldcg(reinterpret_cast<const float4 *>(z + base + j));
            v[j] = t.x; v[j + 1] = t.y; v[j + 2] = t.z; v[j + 3] = t.w;
        }
    } else {
#pragma unroll
        for (int j = 0; j < EPT; ++j) v[j] = base + j < V ? __ldcg(z + base + j) : -INFINITY;
    }
}
// weight keys of the thread's tokens for a row whose maximum is known (tokens beyond the row: key 0, weight 0)
template <int EPT>
__device__ __forceinline__ void load_keys(const float *z, int V, int base, float m, double inv_T, uint32_t (&key)[EPT]) {
    float v[EPT];
    load_logits<EPT>(z, V, base, v);
#pragma unroll
    for (int j = 0; j < EPT; ++j) key[j] = base + j < V ? weight_key(v[j], m, inv_T) : 0u;
}

// Statistics of the filtered distribution of one logit row; identical in every thread of the cluster.  The
// thread's keys are left in `key`.
template <int EPT>
__device__ RowStat row_stats(const float *z, int V, double inv_T, double top_p, Ctx &c, uint32_t (&key)[EPT]) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, base = my_base<EPT>(c);
    float m;
    {
        float v[EPT], mx = -INFINITY;
        load_logits<EPT>(z, V, base, v);
#pragma unroll
        for (int j = 0; j < EPT; ++j) mx = fmaxf(mx, v[j]);
        mx = block_max(mx, reinterpret_cast<float *>(c.scr));
        if (tid == 0) c.mine[0] = (u64)__float_as_uint(mx);
        cluster_gather(c, 1);
        m = -INFINITY;
        for (unsigned r = 0; r < CL; ++r) m = fmaxf(m, __uint_as_float((uint32_t)c.all[r]));
        u64 zsum = 0;
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            key[j] = base + j < V ? weight_key(v[j], m, inv_T) : 0u;
            zsum += key_weight(key[j]);
        }
        zsum = block_sum_u64(zsum, c.scr);
        if (tid == 0) c.mine[0] = zsum;
        cluster_sum(c, 1);
    }
    RowStat r;
    r.m = m;
    r.Z = c.all[0];
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
        for (int b = 0; b < NBK; ++b) c.hist[b * SNT + tid] = 0;
        const uint32_t hi_shift = s == 28 ? 0 : s + 4;       // (a shift by 32 is not defined: the top pass takes all keys)
        const uint32_t want = s == 28 ? 0 : prefix;
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            const bool in = s == 28 || (key[j] >> hi_shift) == want;
            if (in) c.hist[((key[j] >> s) & 15u) * SNT + tid] += key_weight(key[j]);
        }
        __syncthreads();
        u64 acc = 0;                         // warp w sums bucket w (SNT / 32 == NBK warps)
#pragma unroll
        for (int k = 0; k < SNT / 32; ++k) acc += c.hist[warp * SNT + lane + 32 * k];
        acc = warp_sum_u64(acc);
        if (lane == 0) c.mine[warp] = acc;
        cluster_sum(c, NBK);
        // S_t = mass above bucket t; it grows as t falls; the bucket of kstar is the lowest t with S_t < tgt
        u64 St = A, chosen = A;
        int tstar = 15;
        for (int t = 15; t >= 0; --t) {
            if (!((double)St < tgt)) break;
            tstar = t;
            chosen = St;
            St += c.all[t];
        }
        prefix = (prefix << 4) | (uint32_t)tstar;
        A = chosen;
    }
    u64 eq = 0;
#pragma unroll
    for (int j = 0; j < EPT; ++j) eq += (base + j < V) && key[j] == prefix;
    eq = block_sum_u64(eq, c.scr);
    if (tid == 0) c.mine[0] = eq;
    cluster_sum(c, 1);
    const int cnt_eq = (int)c.all[0];
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

// kept weight of a token met in token-id order (eq_seen counts the tokens with key == kstar met so far)
__device__ __forceinline__ u64 kept_weight(uint32_t key, bool valid, const RowStat &st, int &eq_seen) {
    if (!valid) return 0ull;
    if (key > st.kstar) return key_weight(key);
    if (key == st.kstar) return eq_seen++ < st.tie_keep ? key_weight(key) : 0ull;
    return 0ull;
}

// tokens with key == kstar before this thread's first token (only needed when some ties are dropped)
template <int EPT>
__device__ __forceinline__ int ties_before(const uint32_t (&key)[EPT], int V, int base, const RowStat &st, Ctx &c) {
    if (st.tie_keep >= st.cnt_eq) return 0;                 // every tie is kept: the rank does not matter
    u64 n = 0, total;
#pragma unroll
    for (int j = 0; j < EPT; ++j) n += (base + j < V) && key[j] == st.kstar;
    return (int)cluster_excl_scan_u64(c, n, total);
}

// Inverse CDF in token-id order over the filtered distribution: the first token whose cumulative kept mass
// exceeds u * K (the last kept token if rounding leaves none).  `key`: the thread's keys of this row.
// Identical in every thread of the cluster.
template <int EPT>
__device__ int pick_token(const uint32_t (&key)[EPT], int V, const RowStat &st, double u, Ctx &c) {
    const int base = my_base<EPT>(c);
    const int eq0 = ties_before<EPT>(key, V, base, st, c);
    int eq = eq0;
    u64 mine = 0;
#pragma unroll
    for (int j = 0; j < EPT; ++j) mine += kept_weight(key[j], base + j < V, st, eq);
    u64 total;
    u64 cum = cluster_excl_scan_u64(c, mine, total);
    const double tu = u * (double)st.K;
    int cand = 0x7fffffff, last = -1;
    // the thread whose tokens hold the crossing walks them again (integers: the test is exact); if rounding of
    // u * K leaves no crossing at all, every thread with mass reports its last kept token instead
    const bool crossing = (double)(cum + mine) > tu && !((double)cum > tu);
    const bool none = !((double)total > tu);
    if (crossing || (none && mine > 0)) {
        eq = eq0;
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            const u64 w = kept_weight(key[j], base + j < V, st, eq);
            cum += w;
            if (w > 0) last = base + j;
            if (w > 0 && cand == 0x7fffffff && (double)cum > tu) cand = base + j;
        }
    }
    int first, final_last;
    cluster_min_max(c, cand, last, first, final_last);
    return first != 0x7fffffff ? first : final_last;
}

// filtered probability of token x of a row with known statistics; identical in every thread of the cluster
template <int EPT>
__device__ double token_prob(const float *z, int V, int x, const RowStat &st, double inv_T, Ctx &c) {
    const uint32_t kx = weight_key(__ldcg(z + x), st.m, inv_T);
    if (kx < st.kstar) return 0.0;
    if (kx == st.kstar && st.tie_keep < st.cnt_eq) {
        // rank of x among the tied tokens
        const int base = my_base<EPT>(c);
        uint32_t key[EPT];
        load_keys<EPT>(z, V, base, st.m, inv_T, key);
        u64 n = 0;
#pragma unroll
        for (int j = 0; j < EPT; ++j) n += (base + j < x) && key[j] == st.kstar;
        n = block_sum_u64(n, c.scr);
        if (threadIdx.x == 0) c.mine[0] = n;
        cluster_sum(c, 1);
        if ((int)c.all[0] >= st.tie_keep) return 0.0;
    }
    return (double)key_weight(kx) / (double)st.K;
}

// Token from the normalised max(0, p - q) of two filtered rows with known statistics; -1 if nothing is left
// (the caller then draws from p itself).  Identical in every thread of the cluster.
template <int EPT>
__device__ int pick_residual(const float *zp, const float *zq, int V, const RowStat &sp, const RowStat &sq, double inv_T, double u,
                             Ctx &c) {
    const int base = my_base<EPT>(c);
    uint32_t kp[EPT], kq[EPT];
    load_keys<EPT>(zp, V, base, sp.m, inv_T, kp);
    load_keys<EPT>(zq, V, base, sq.m, inv_T, kq);
    const int ep0 = ties_before<EPT>(kp, V, base, sp, c);
    const int eq0 = ties_before<EPT>(kq, V, base, sq, c);
    const double ikp = 1.0 / (double)sp.K, ikq = 1.0 / (double)sq.K;
    int ep = ep0, eq = eq0;
    double mine = 0.0;
#pragma unroll
    for (int j = 0; j < EPT; ++j) {
        const double p = (double)kept_weight(kp[j], base + j < V, sp, ep) * ikp;
        const double q = (double)kept_weight(kq[j], base + j < V, sq, eq) * ikq;
        mine += p > q ? p - q : 0.0;
    }
    double R;
    double cum = cluster_excl_scan_f64(c, mine, R);
    if (!(R > 0.0)) return -1;
    const double tu = u * R;
    int cand = 0x7fffffff, last = -1;
    // the threads whose tokens may hold the crossing walk them again; the band is a little wide because a
    // thread's mass added at once and added term by term can differ in the last bits
    const bool near = cum + mine >= tu * (1.0 - 1e-12) && cum <= tu * (1.0 + 1e-12);
    const bool none = !(R > tu * (1.0 + 1e-9));
    if (mine > 0.0 && (near || none)) {
        ep = ep0; eq = eq0;
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            const double p = (double)kept_weight(kp[j], base + j < V, sp, ep) * ikp;
            const double q = (double)kept_weight(kq[j], base + j < V, sq, eq) * ikq;
            const double r = p > q ? p - q : 0.0;
            cum += r;
            if (r > 0.0) last = base + j;
            if (r > 0.0 && cand == 0x7fffffff && cum > tu) cand = base + j;
        }
    }
    int first, final_last;
    cluster_min_max(c, cand, last, first, final_last);
    return first != 0x7fffffff ? first : final_last;
}

// ---------------------------------------------------------------- kernels (one cluster per row / sequence)
__device__ __forceinline__ const float *logit_row(const float *base, int seq, int row, int V) {
    return base + ((size_t)seq * DEL_SAMPLE_ROWS + row) * V;
}
__device__ __forceinline__ void leave_cluster() { cg::this_cluster().sync(); }    // no CTA exits while its posts may be read

// Draft i of a sequence: the exit head's row is filtered, the token drawn (purpose 0 at position T + 1 + i) and
// stored as draft i; the row's statistics stay for the acceptance tests.
template <int EPT>
__global__ void __launch_bounds__(SNT) sample_draft_kernel(const __grid_constant__ SampleArgs a) {
    extern __shared__ __align__(16) unsigned char raw[];
    pdl_launch();
    pdl_wait();
    Ctx c = make_ctx(raw);
    const SampleSeq s = a.s[blockIdx.x / CL];
    const int V = a.D.V;
    const float *z = logit_row(a.B.QLOG, s.seq, s.slot, V);
    uint32_t key[EPT];
    const RowStat st = row_stats<EPT>(z, V, s.inv_T, s.top_p, c, key);
    const double u = uniform01(s.seed, s.pos0 + 1 + s.slot, 0);
    const int x = pick_token<EPT>(key, V, st, u, c);
    if (c.rank == 0 && threadIdx.x == 0) {
        a.B.QSTAT[s.seq * DEL_SAMPLE_ROWS + s.slot] = st;
        a.B.TOK[s.seq * (a.D.S + 1) + s.slot + 1] = x;
        a.B.SMP[s.seq].q_x[s.slot] = (float)((double)key_weight(weight_key(__ldcg(z + x), st.m, s.inv_T)) / (double)st.K);
    }
    leave_cluster();
}

// Statistics of the target's rows 0..g: grid (rows * CL, sequences)
template <int EPT>
__global__ void __launch_bounds__(SNT) sample_stats_kernel(const __grid_constant__ SampleArgs a) {
    extern __shared__ __align__(16) unsigned char raw[];
    pdl_launch();
    pdl_wait();
    const SampleSeq s = a.s[blockIdx.y];
    const int row = blockIdx.x / CL, V = a.D.V;
    if (row > s.g) return;                   // (the whole cluster returns)
    Ctx c = make_ctx(raw);
    uint32_t key[EPT];
    const RowStat st = row_stats<EPT>(logit_row(a.B.PLOG, s.seq, row, V), V, s.inv_T, s.top_p, c, key);
    if (c.rank == 0 && threadIdx.x == 0) a.B.PSTAT[s.seq * DEL_SAMPLE_ROWS + row] = st;
    leave_cluster();
}

// Acceptance tests of the drafts in order (purpose 1), then the token that ends the round (purpose 2): from the
// residual of the first rejected position, or from the target's row g when every draft was accepted.
template <int EPT>
__global__ void __launch_bounds__(SNT) sample_verify_kernel(const __grid_constant__ SampleArgs a) {
    extern __shared__ __align__(16) unsigned char raw[];
    pdl_launch();
    pdl_wait();
    Ctx c = make_ctx(raw);
    const SampleSeq s = a.s[blockIdx.x / CL];
    const int V = a.D.V;
    const bool writer = c.rank == 0 && threadIdx.x == 0;
    const int32_t *tok = a.B.TOK + s.seq * (a.D.S + 1);
    SampleOut *out = a.B.SMP + s.seq;
    int n = 0, rejected = 0;
    while (n < s.g) {
        const int x = tok[1 + n];
        const RowStat sp = a.B.PSTAT[s.seq * DEL_SAMPLE_ROWS + n], sq = a.B.QSTAT[s.seq * DEL_SAMPLE_ROWS + n];
        const double px = token_prob<EPT>(logit_row(a.B.PLOG, s.seq, n, V), V, x, sp, s.inv_T, c);
        const double qx = token_prob<EPT>(logit_row(a.B.QLOG, s.seq, n, V), V, x, sq, s.inv_T, c);
        const double u = uniform01(s.seed, s.pos0 + 1 + n, 1);
        if (writer) out->p_x[n] = (float)px;
        const double ratio = px / qx;
        if (u < (ratio < 1.0 ? ratio : 1.0)) ++n;
        else { rejected = 1; break; }
    }
    const int n_tests = rejected ? n + 1 : n;
    const double u = uniform01(s.seed, s.pos0 + 1 + n, 2);
    const RowStat sp = a.B.PSTAT[s.seq * DEL_SAMPLE_ROWS + n];
    const float *zp = logit_row(a.B.PLOG, s.seq, n, V);
    int last = -1;
    if (rejected) {
        const RowStat sq = a.B.QSTAT[s.seq * DEL_SAMPLE_ROWS + n];
        last = pick_residual<EPT>(zp, logit_row(a.B.QLOG, s.seq, n, V), V, sp, sq, s.inv_T, u, c);
    }
    if (last < 0) {                          // every draft accepted (or an empty residual): from the target's row
        uint32_t key[EPT];
        load_keys<EPT>(zp, V, my_base<EPT>(c), sp.m, s.inv_T, key);
        last = pick_token<EPT>(key, V, sp, u, c);
    }
    if (writer) {
        out->n_accept = n;
        out->last_token = last;
        out->n_tests = n_tests;
        out->from_residual = rejected;
    }
    leave_cluster();
}

// Test hook: the same device functions on one caller-supplied pair of rows.
template <int EPT>
__global__ void __launch_bounds__(SNT) sample_probe_kernel(const float *zp, const float *zq, int V, double inv_T, double top_p,
                                                           double u_draft, double u_accept, double u_final, int32_t *out,
                                                           double *prob, RowStat *stat) {
    extern __shared__ __align__(16) unsigned char raw[];
    Ctx c = make_ctx(raw);
    uint32_t key[EPT];
    const RowStat sq = row_stats<EPT>(zq, V, inv_T, top_p, c, key);
    const int x = pick_token<EPT>(key, V, sq, u_draft, c);
    const RowStat sp = row_stats<EPT>(zp, V, inv_T, top_p, c, key);
    // both endings are reported: the draw from p (as if all were accepted) and the residual draw (as if rejected)
    const int bonus = pick_token<EPT>(key, V, sp, u_final, c);
    const double qx = token_prob<EPT>(zq, V, x, sq, inv_T, c), px = token_prob<EPT>(zp, V, x, sp, inv_T, c);
    const double ratio = px / qx;
    const int accepted = u_accept < (ratio < 1.0 ? ratio : 1.0);
    int res = pick_residual<EPT>(zp, zq, V, sp, sq, inv_T, u_final, c);
    if (res < 0) res = bonus;
    if (c.rank == 0 && threadIdx.x == 0) {
        out[0] = x; out[1] = accepted; out[2] = res; out[3] = bonus;
        prob[0] = qx; prob[1] = px;
        stat[0] = sq; stat[1] = sp;
    }
    leave_cluster();
}

template <typename... KArgs, typename... Args>
cudaError_t launch_cluster(void (*kern)(KArgs...), dim3 grid, cudaStream_t st, bool pdl, Args... args) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(SNT);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = CL;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    // measured: a cluster launch that is also a programmatic dependent launch starts later than one in plain
    // stream order (0.5 % of a round with two drafts), so the second attribute is left out
    (void)pdl;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

// tokens per thread for a vocabulary: the smallest power of two with CL * SNT * EPT >= V (0: too large)
int ept_for(int V) {
    for (int e = 1; e <= 64; e *= 2)
        if ((long long)CL * SNT * e >= V) return e;
    return 0;
}

#define DISPATCH_EPT(V, CALL)                                  \
    switch (ept_for(V)) {                                      \
        case 1: { constexpr int E = 1; return CALL; }          \
        case 2: { constexpr int E = 2; return CALL; }          \
        case 4: { constexpr int E = 4; return CALL; }          \
        case 8: { constexpr int E = 8; return CALL; }          \
        case 16: { constexpr int E = 16; return CALL; }        \
        case 32: { constexpr int E = 32; return CALL; }        \
        case 64: { constexpr int E = 64; return CALL; }        \
        default: return cudaErrorInvalidValue;                 \
    }

}  // namespace

int sample_max_vocab() { return CL * SNT * 64; }
cudaError_t launch_sample_draft(const SampleArgs &a, cudaStream_t st, bool pdl) {
    DISPATCH_EPT(a.D.V, launch_cluster(sample_draft_kernel<E>, dim3(a.n * CL), st, pdl, a))
}
cudaError_t launch_sample_stats(const SampleArgs &a, int max_rows, cudaStream_t st, bool pdl) {
    DISPATCH_EPT(a.D.V, launch_cluster(sample_stats_kernel<E>, dim3(max_rows * CL, a.n), st, pdl, a))
}
cudaError_t launch_sample_verify(const SampleArgs &a, cudaStream_t st, bool pdl) {
    DISPATCH_EPT(a.D.V, launch_cluster(sample_verify_kernel<E>, dim3(a.n * CL), st, pdl, a))
}
cudaError_t launch_sample_probe(const float *p_logits, const float *q_logits, int V, double inv_T, double top_p, double u_draft,
                                double u_accept, double u_final, int32_t *out, double *prob, RowStat *stat, cudaStream_t st) {
    DISPATCH_EPT(V, launch_cluster(sample_probe_kernel<E>, dim3(CL), st, false, p_logits, q_logits, V, inv_T, top_p, u_draft,
                                   u_accept, u_final, out, prob, stat))
}
