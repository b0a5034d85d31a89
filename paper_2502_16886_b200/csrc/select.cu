// Steps S4-S6: ranking, the threshold-free stopping rule and the kept set.
//
// For one unit with squares sq_i = a'_i^2 and ranked order pi, the rule is the
// cumulative form of Eq. 1 (Eq. 3; Algorithm 1 Square, Reorder, Cumsum, Sqrt,
// ratio, Where):
//     C_j = sum_{t<=j} sq[pi_t],  j* = leftmost j with 1 - sqrt(C_j / C_n) < T.
// The budget is b = max(j*, floor); the kept set is the first b ranked positions,
// emitted in ascending position order.
//
// Arithmetic.  fp64 is a slow pipe on this GPU, so the sums are integers: the
// square of an fp32 score is the exact 48-bit product of its mantissa with
// itself, shifted to a per-unit fixed point in which C_n lies in [2^60, 2^61)
// (bits below the unit are dropped: at most n * 2^-60 of C_n in total).  Integer
// sums do not depend on the order of addition, so budgets are deterministic.
// The rule itself is applied as C_j >= C_min, where
//     1 - sqrt(C/C_n) < T  <=>  C_n - C < C_n * T * (2 - T)
// and C_min is placed once per unit with a handful of fp64 operations.
//
// Position ranking (Section 3.2) needs no sort: the order is the m leading
// positions, then the rest from the end backwards, so C_j is a block-wide prefix
// scan over a closed-form order.  Score ranking (Section 4.4) needs the order by
// decreasing score; instead of sorting, a radix descent over the keys (8 bits per
// level) finds the key at which the cumulative sum crosses, using per-digit
// histograms of counts and of sums of squares.
#include <algorithm>

#include <cooperative_groups.h>

#include <mutex>

#include "refree_internal.cuh"
#include "select_groups.cuh"

namespace refree {
namespace {

namespace cg = cooperative_groups;

constexpr int kThreads = 1024;
constexpr int kMaxCluster = 8;     // blocks of a thread-block cluster that share one unit in score ranking
constexpr int kWarps = kThreads / 32;
typedef unsigned long long u64;

struct UnitView {
    const float *sc;        // scores of head 0 (layer scope) or of the unit's head, at the sequence start
    int64_t head_stride;    // distance between heads in the score array
    int heads;              // heads whose squares add up (1 in head scope)
    int n, lead, w_eff;
    int sbias;              // fixed point: a^2 * 2^S = mantissa^2 * 2^(2 * exponent_field + sbias)
};

__device__ inline u64 sq_at(const UnitView &v, int i)
{
    u64 acc = 0;
    for (int h = 0; h < v.heads; ++h) acc += sq_fixed(mag_bits(v.sc[(int64_t)h * v.head_stride + i]), v.sbias);
    return acc;
}

// sort key of an unprotected position: larger key = ranked earlier
__device__ inline u64 key_at(const UnitView &v, int i)
{
    if (v.heads == 1) return (u64)mag_bits(v.sc[i]) << 32;       // a' >= 0: its bits order like its square
    return sq_at(v, i);
}

struct PosRank {     // position ranking: leading positions, then from the end backwards
    __device__ int operator()(const UnitView &v, int j) const { return j < v.lead ? j : v.n - 1 - (j - v.lead); }
};
struct ProtRank {    // protected prefix of the score ranking: leading positions, then the window
    __device__ int operator()(const UnitView &v, int j) const { return j < v.lead ? j : v.n - v.w_eff + (j - v.lead); }
};

// Block-wide exclusive scan; `total` receives the sum.  `buf` holds kWarps + 1 items.
template <typename Tv> __device__ inline Tv block_excl_scan(Tv x, Tv *buf, Tv &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const Tv inc = warp_incl_scan(x);
    __syncthreads();
    if (lane == 31) buf[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const Tv w = buf[lane];
        const Tv wi = warp_incl_scan(w);
        buf[lane] = wi - w;
        if (lane == 31) buf[kWarps] = wi;
    }
    __syncthreads();
    total = buf[kWarps];
    return buf[warp] + inc - x;
}

template <typename Tv, typename Op> __device__ inline Tv block_reduce(Tv x, Tv *buf, Op op)
{
    for (int o = 16; o; o >>= 1) x = op(x, __shfl_xor_sync(0xffffffffu, x, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) buf[threadIdx.x >> 5] = x;
    __syncthreads();
    Tv r = buf[0];
    for (int wv = 1; wv < kWarps; ++wv) r = op(r, buf[wv]);
    return r;
}
// Values combined over the blocks of a cluster through distributed shared memory: every block
// publishes its share, all read all shares in rank order (so all get the same result), and a
// second barrier keeps the slot from being rewritten early.  With one block these are no-ops.
template <typename Tv, typename Op>
__device__ inline Tv cluster_combine(cg::cluster_group &cl, Tv *slot, Tv mine, Op op)
{
    const unsigned int nb = cl.num_blocks();
    if (nb == 1) return mine;
    if (threadIdx.x == 0) *slot = mine;
    cl.sync();
    Tv r = *cl.map_shared_rank(slot, 0);
    for (unsigned int b = 1; b < nb; ++b) r = op(r, *cl.map_shared_rank(slot, b));
    cl.sync();
    return r;
}
struct AddOpU64 { __device__ unsigned long long operator()(unsigned long long a, unsigned long long b) const { return a + b; } };

struct MinOp { __device__ int operator()(int a, int b) const { return min(a, b); } };
struct MaxOpU { __device__ uint32_t operator()(uint32_t a, uint32_t b) const { return max(a, b); } };
struct AddOpF { __device__ float operator()(float a, float b) const { return a + b; } };

// Ranks [lo, lo + len) in the order given by `pos_of` are split into one
// contiguous segment per warp; inside a segment the lanes interleave, so every
// load is a coalesced 128-byte line, and eight loads are in flight per thread.
// range_totals leaves the exclusive prefix of the warp sums in wpre[0..kWarps)
// and the total in wpre[kWarps].
__device__ inline int seg_len(int len) { return ceil_div(ceil_div(len, kWarps), 32) * 32; }

template <typename PosOf>
__device__ inline u64 range_totals(const UnitView &v, int lo, int len, PosOf pos_of, u64 *wpre)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int seg = seg_len(len);
    const int w0 = lo + min(len, warp * seg), w1 = lo + min(len, (warp + 1) * seg);
    u64 local = 0;
    for (int j = w0 + lane; j < w1; j += 32 * 8) {
        u64 x[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) x[q] = (j + 32 * q < w1) ? sq_at(v, pos_of(v, j + 32 * q)) : 0ull;
#pragma unroll
        for (int q = 0; q < 8; ++q) local += x[q];
    }
    for (int o = 16; o; o >>= 1) local += __shfl_xor_sync(0xffffffffu, local, o);
    __syncthreads();
    if (lane == 0) wpre[warp] = local;
    __syncthreads();
    if (warp == 0) {
        const u64 x = wpre[lane];
        const u64 inc = warp_incl_scan(x);
        wpre[lane] = inc - x;
        if (lane == 31) wpre[kWarps] = inc;
    }
    __syncthreads();
    return wpre[kWarps];
}

// First rank count j (1-based) with C_j >= c_min, or INT_MAX, given the warp
// prefixes that range_totals left for ranks [0, count).  The segment whose end
// first reaches c_min holds the crossing; it is split over the warps again until
// it is 32 ranks long, which one warp resolves with a scan and a ballot.
template <typename PosOf>
__device__ inline int range_find(const UnitView &v, int count, PosOf pos_of, u64 c_min, u64 *wpre, int *ibuf)
{
    const int lane = threadIdx.x & 31;
    int lo = 0, len = count;
    u64 base = 0;
    for (;;) {
        // every thread reads the same prefixes and finds the same segment
        const int seg = seg_len(len);
        int hit = -1;
        for (int wv = 0; wv < kWarps; ++wv) {
            const u64 end = base + wpre[wv + 1 < kWarps ? wv + 1 : kWarps];
            if (min(len, wv * seg) < min(len, (wv + 1) * seg) && end >= c_min) { hit = wv; break; }
        }
        if (hit < 0) return INT_MAX;
        const int nlo = lo + min(len, hit * seg), nlen = lo + min(len, (hit + 1) * seg) - nlo;
        base += wpre[hit];
        lo = nlo;
        len = nlen;
        if (len <= 32) break;
        range_totals(v, lo, len, pos_of, wpre);
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        const int j = lo + lane;
        u64 x = lane < len ? sq_at(v, pos_of(v, j)) : 0ull;
        x = warp_incl_scan(x);
        const unsigned m = __ballot_sync(0xffffffffu, lane < len && base + x >= c_min);
        if (lane == 0) ibuf[0] = m ? lo + __ffs(m) : lo + len;
    }
    __syncthreads();
    const int found = ibuf[0];
    __syncthreads();
    return found;
}

// x += v for a 64-bit counter in shared memory, as two 32-bit atomic adds with the carry passed on (the halves
// are only read together after a barrier).  Shared memory has 32-bit atomic adds in hardware; a 64-bit one is a
// compare-and-swap loop, which crawls when most of a warp meets at one counter.
__device__ inline void add_u64_shared(u64 *x, u64 v)
{
    uint32_t *h = reinterpret_cast<uint32_t *>(x);
    const uint32_t lo = (uint32_t)v;
    const uint32_t old = atomicAdd(h, lo);
    const uint32_t hi = (uint32_t)(v >> 32) + (old + lo < old ? 1u : 0u);
    if (hi) atomicAdd(h + 1, hi);
}

struct SelectSmem {
    u64 wpre[kWarps + 1];
    u64 ubuf[kWarps + 1];
    int ibuf[kWarps + 1];
    float fbuf[kWarps + 1];
    unsigned int hcnt[256];
    u64 hsum[256];
    unsigned int hcnt2[2][256];       // register-resident score ranking: the block's histogram of a level, read by
    u64 hsum2[2][256];                // the cluster; two copies taken in turn, so that one exchange needs one barrier
    u64 dsum[8];                      // ... and its digit search: totals of the eight warps that own the digits
    unsigned int dcnt[8];
    int dcand[8];                     // first digit of each of those warps at which the sum crosses, with what is
    u64 dabv_s[8];                    // above it and how many share it
    unsigned int dabv_c[8], ddig[8];
    uint32_t y_mx;                    // fixed point, exchanged once: a block's largest key and its sum of squares
    float y_acc;                      // at that key's scale
    uint32_t z_key;                   // the crossing key, told by the block that holds it when one position has it
    unsigned int wcnt[kWarps][257];   // per-warp private histograms (padded: one bank per warp for a digit)
    u64 wsum[kWarps][257];
    int pack;
    u64 c_min;
    // cluster exchange: what this block contributes, read by every block of the cluster
    u64 x_u64;
    float x_f32;
    uint32_t x_u32;
    // radix state
    u64 prefix, above_sum;
    unsigned int above_cnt;
    int digit;
};

// Fixed point of a unit: returns false when every score is zero (C_n = 0).
__device__ inline bool choose_fixed_point(UnitView &v, SelectSmem &sm, int32_t *dev_status, cg::cluster_group &cl)
{
    // the blocks of a cluster take the positions in interleaved runs of 8 * kThreads
    const int first = (int)cl.block_rank() * kThreads * 8 + threadIdx.x, step = (int)cl.num_blocks() * kThreads * 8;
    uint32_t mx = 0;
    bool bad = false;
    for (int h = 0; h < v.heads; ++h)
        for (int i = first; i < v.n; i += step) {
            uint32_t b[8];
#pragma unroll
            for (int q = 0; q < 8; ++q)
                b[q] = (i + q * kThreads < v.n) ? mag_bits(v.sc[(int64_t)h * v.head_stride + i + q * kThreads]) : 0u;
#pragma unroll
            for (int q = 0; q < 8; ++q) { if ((b[q] >> 23) == 255u) bad = true; else mx = max(mx, b[q]); }
        }
    if (bad && dev_status) atomicOr(dev_status, REFREE_DEV_NONFINITE);
    mx = block_reduce<uint32_t>(mx, reinterpret_cast<uint32_t *>(sm.ibuf), MaxOpU());
    mx = cluster_combine<uint32_t>(cl, &sm.x_u32, mx, MaxOpU());
    if (mx == 0u) return false;
    const int emax = max(1, (int)(mx >> 23));
    // approximate sum of squares of the scores scaled into [0, 2): only its binary order of magnitude is used
    const float f = ldexpf(1.0f, 127 - emax);
    float acc = 0.f;
    for (int h = 0; h < v.heads; ++h)
        for (int i = first; i < v.n; i += step) {
            uint32_t b[8];
#pragma unroll
            for (int q = 0; q < 8; ++q)
                b[q] = (i + q * kThreads < v.n) ? mag_bits(v.sc[(int64_t)h * v.head_stride + i + q * kThreads]) : 0u;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const float a = ((b[q] >> 23) == 255u) ? 0.f : __uint_as_float(b[q]) * f;
                acc = fmaf(a, a, acc);
            }
        }
    acc = block_reduce<float>(acc, sm.fbuf, AddOpF());
    acc = cluster_combine<float>(cl, &sm.x_f32, acc, AddOpF());
    // C_n = acc * 2^(2 (emax - 127)); put C_n * 2^S in [2^60, 2^61)
    const int S = 60 - ilogbf(fmaxf(acc, 0.25f)) - 2 * (emax - 127);
    v.sbias = S - 300;
    return true;
}

__global__ void __launch_bounds__(kThreads)
select_budget_kernel(refree_params p, const float *scores, const int32_t *seq_len,
                     int64_t total_tokens, int32_t *lengths, Cut *cuts, int32_t *dev_status, int skip_upto)
{
    extern __shared__ __align__(16) unsigned char select_smem_raw[];
    SelectSmem &sm = *reinterpret_cast<SelectSmem *>(select_smem_raw);
    cg::cluster_group cl = cg::this_cluster();
    const int nblk = (int)cl.num_blocks(), rank = (int)cl.block_rank();    // > 1 only with score ranking
    const int unit = blockIdx.x / nblk;
    const int Hkv = p.num_kv_heads;
    const bool layer = p.scope == REFREE_SCOPE_LAYER;
    const int s = layer ? unit : unit / Hkv;
    const int g = layer ? 0 : unit % Hkv;
    if (skip_upto > 0 && max(seq_len[s], 0) <= skip_upto) return;      // the register-resident kernel takes these (the whole cluster leaves)
    if (threadIdx.x == 0) {
        int a = 0;
        for (int t = 0; t < s; ++t) a += max(seq_len[t], 0);
        sm.pack = a;
    }
    __syncthreads();
    const int n = max(seq_len[s], 0);
    UnitView v;
    v.sc = scores + (int64_t)g * total_tokens + sm.pack;
    v.head_stride = total_tokens;
    v.heads = layer ? Hkv : 1;
    v.n = n;
    v.w_eff = min(p.window, n);
    v.lead = min(p.sink, n);
    v.sbias = 0;
    const int floor_b = p.keep_window ? min(n, v.lead + v.w_eff) : min(n, 1);

    Cut cut;
    cut.b = n; cut.ties = 0; cut.tau = 0; cut.prot_kept = 0; cut.sbias = 0;

    if (n > 0 && !p.force_full && choose_fixed_point(v, sm, dev_status, cl)) {
        cut.sbias = v.sbias;
        if (p.rank_mode == REFREE_RANK_POSITION) {
            // one pass in rank order gives C_n and the warp prefixes the search needs
            const u64 Cn = range_totals(v, 0, n, PosRank(), sm.wpre);
            if (threadIdx.x == 0) sm.c_min = crossing_level(Cn, (double)p.threshold);
            __syncthreads();
            const int j = range_find(v, n, PosRank(), sm.c_min, sm.wpre, sm.ibuf);
            cut.b = max(j == INT_MAX ? n : j, floor_b);
        } else {
            // score ranking: when the protected prefix covers the sequence the order is 0..n-1
            if (v.lead + v.w_eff >= n) { v.lead = n; v.w_eff = 0; }
            const int prot = v.lead + v.w_eff;
            u64 Cn;
            {   // C_n over every position (the order does not matter for an integer sum): this block's share
                u64 local = 0;
                for (int i = rank * kThreads * 8 + threadIdx.x; i < n; i += nblk * kThreads * 8) {
                    u64 x[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) x[q] = (i + q * kThreads < n) ? sq_at(v, i + q * kThreads) : 0ull;
#pragma unroll
                    for (int q = 0; q < 8; ++q) local += x[q];
                }
                u64 tot;
                block_excl_scan<u64>(local, sm.ubuf, tot);
                Cn = cluster_combine<u64>(cl, &sm.x_u64, tot, AddOpU64());
            }
            if (threadIdx.x == 0) sm.c_min = crossing_level(Cn, (double)p.threshold);
            __syncthreads();
            const u64 c_min = sm.c_min;
            const u64 Sprot = range_totals(v, 0, prot, ProtRank(), sm.wpre);
            const int jp = range_find(v, prot, ProtRank(), c_min, sm.wpre, sm.ibuf);
            int jstar = n;
            cut.prot_kept = prot;
            cut.tau = 0ull;                       // keep every unprotected position ...
            cut.ties = INT_MAX;                   // ... unless a crossing is found below
            if (jp != INT_MAX) {
                jstar = jp;
            } else if (prot < n && c_min != ~0ull) {
                const u64 need = c_min - Sprot;   // mass still missing after the protected prefix (> 0)
                if (threadIdx.x == 0) { sm.prefix = 0ull; sm.above_sum = 0ull; sm.above_cnt = 0u; }
                const int levels = v.heads == 1 ? 4 : 8;
                bool any = true;
                for (int level = 0; level < levels && any; ++level) {
                    const int shift = 56 - 8 * level;
                    // each warp fills a histogram of its own (no contention between warps on a
                    // popular digit); thread t then adds up digit t over the warps
                    const int warp = threadIdx.x >> 5;
                    for (int t = threadIdx.x; t < kWarps * 257; t += kThreads) {
                        (&sm.wcnt[0][0])[t] = 0u;
                        (&sm.wsum[0][0])[t] = 0ull;
                    }
                    __syncthreads();
                    const u64 prefix = sm.prefix;
                    for (int i0 = v.lead + rank * kThreads * 4 + threadIdx.x; i0 < n - v.w_eff; i0 += nblk * kThreads * 4) {
                        u64 key[4], val[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const int i = i0 + q * kThreads;
                            const bool in = i < n - v.w_eff;
                            key[q] = in ? key_at(v, i) : 0ull;
                            val[q] = !in ? 0ull : (v.heads == 1 ? sq_fixed((uint32_t)(key[q] >> 32), v.sbias) : key[q]);
                        }
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            if (i0 + q * kThreads < n - v.w_eff && (level == 0 || (key[q] >> (shift + 8)) == prefix)) {
                                const int dgt = (int)((key[q] >> shift) & 255ull);
                                atomicAdd(&sm.wcnt[warp][dgt], 1u);
                                add_u64_shared(&sm.wsum[warp][dgt], val[q]);
                            }
                        }
                    }
                    __syncthreads();
                    if (threadIdx.x < 256) {
                        unsigned int c = 0u;
                        u64 sumv = 0ull;
                        for (int wv = 0; wv < kWarps; ++wv) { c += sm.wcnt[wv][threadIdx.x]; sumv += sm.wsum[wv][threadIdx.x]; }
                        sm.hcnt[threadIdx.x] = c;
                        sm.hsum[threadIdx.x] = sumv;
                    }
                    __syncthreads();
                    if (nblk > 1) {
                        // the digit histograms of the cluster's blocks add up (integers: any order); every
                        // block then takes the same decision from the same totals
                        cl.sync();
                        unsigned int c = 0u;
                        u64 sumv = 0ull;
                        if (threadIdx.x < 256)
                            for (int b = 0; b < nblk; ++b) {
                                c += cl.map_shared_rank(sm.hcnt, b)[threadIdx.x];
                                sumv += cl.map_shared_rank(sm.hsum, b)[threadIdx.x];
                            }
                        cl.sync();
                        if (threadIdx.x < 256) { sm.hcnt[threadIdx.x] = c; sm.hsum[threadIdx.x] = sumv; }
                        __syncthreads();
                    }
                    // inclusive sums from the top digit down; thread t owns digit 255 - t
                    u64 mysum = 0ull, tot_s;
                    unsigned int mycnt = 0u, tot_c;
                    if (threadIdx.x < 256) { mysum = sm.hsum[255 - threadIdx.x]; mycnt = sm.hcnt[255 - threadIdx.x]; }
                    const u64 abv_s = block_excl_scan<u64>(mysum, sm.ubuf, tot_s);
                    const unsigned int abv_c = block_excl_scan<unsigned int>(mycnt, (unsigned int *)sm.ibuf, tot_c);
                    int cand = INT_MAX;
                    if (threadIdx.x < 256 && mycnt > 0u && sm.above_sum + abv_s + mysum >= need) cand = threadIdx.x;
                    cand = block_reduce<int>(cand, sm.ibuf, MinOp());
                    if (cand == INT_MAX) {
                        any = false;              // the rule is never met: keep all
                    } else if ((int)threadIdx.x == cand) {
                        sm.prefix = (prefix << 8) | (u64)(255 - cand);
                        sm.above_sum += abv_s;
                        sm.above_cnt += abv_c;
                        sm.digit = (int)mycnt;
                    }
                    __syncthreads();
                }
                if (any) {
                    // sm.prefix is the key at which the sum crosses; sm.digit positions share it
                    const u64 tau = v.heads == 1 ? sm.prefix << 32 : sm.prefix;
                    const u64 f = v.heads == 1 ? sq_fixed((uint32_t)sm.prefix, v.sbias) : tau;
                    const u64 miss = need - sm.above_sum;           // > 0: the digits above did not reach it
                    u64 t = f ? (miss + f - 1) / f : 1ull;
                    t = max(1ull, min(t, (u64)sm.digit));
                    jstar = prot + (int)sm.above_cnt + (int)t;
                    cut.tau = tau;
                    cut.ties = (int)t;
                }
            }
            cut.b = max(jstar, floor_b);
            if (cut.b <= prot) {                 // nothing beyond the protected prefix
                cut.prot_kept = cut.b;
                cut.tau = ~0ull;
                cut.ties = 0;
            }
        }
    }
    if (nblk > 1) cl.sync();               // no block exits while another may still read its shared memory
    if (threadIdx.x == 0 && rank == 0) {
        const int g_hi = layer ? Hkv : g + 1;
        for (int gg = g; gg < g_hi; ++gg) {
            lengths[s * Hkv + gg] = cut.b;
            cuts[s * Hkv + gg] = cut;
        }
    }
}

// Score ranking per head (Section 4.4) for sequences short enough that a cluster holds every key in registers:
// position (e * blocks + rank) * kThreads + thread is element e of a thread, E elements each.  Same rule, fixed
// point and radix descent as select_budget_kernel; the scores are read once, and a level of the descent costs a
// handful of block barriers and one cluster barrier.
template <int E>
__global__ void __launch_bounds__(kThreads)
select_score_resident_kernel(refree_params p, const float *scores, const int32_t *seq_len,
                             int64_t total_tokens, int32_t *lengths, Cut *cuts, int32_t *dev_status,
                             int2 *chunk_counts, int chunk_stride)
{
    extern __shared__ __align__(16) unsigned char select_smem_raw[];
    SelectSmem &sm = *reinterpret_cast<SelectSmem *>(select_smem_raw);
    cg::cluster_group cl = cg::this_cluster();
    const int nblk = (int)cl.num_blocks(), rank = (int)cl.block_rank();
    const int unit = blockIdx.x / nblk;
    const int Hkv = p.num_kv_heads;
    const int s = unit / Hkv, g = unit % Hkv;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        int a = 0;
        for (int t = 0; t < s; ++t) a += max(seq_len[t], 0);
        sm.pack = a;
        sm.z_key = 0u;
    }
    __syncthreads();
    const int n = max(seq_len[s], 0);
    if (n > nblk * kThreads * E) return;             // too long to hold: select_budget_kernel takes it
    // elements of this block that lie inside the sequence: a batch sized for its longest sequence leaves most of
    // a short one's element slots empty, and the loops below skip them (the same for every thread of the block)
    const int e_lim = min(E, ceil_div(max(n - rank * kThreads, 0), nblk * kThreads));
    UnitView v;
    v.sc = scores + (int64_t)g * total_tokens + sm.pack;
    v.head_stride = total_tokens;
    v.heads = 1;
    v.n = n;
    v.w_eff = min(p.window, n);
    v.lead = min(p.sink, n);
    v.sbias = 0;
    const int floor_b = p.keep_window ? min(n, v.lead + v.w_eff) : min(n, 1);
    Cut cut;
    cut.b = n; cut.ties = 0; cut.tau = 0; cut.prot_kept = 0; cut.sbias = 0;

    uint32_t kb[E];                              // |score| bits; 0 past the sequence
    uint32_t mx = 0;
    bool bad = false;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const int i = (e * nblk + rank) * kThreads + threadIdx.x;
        kb[e] = (e < e_lim && i < n) ? mag_bits(v.sc[i]) : 0u;
        if ((kb[e] >> 23) == 255u) bad = true; else mx = max(mx, kb[e]);
    }
    if (bad && dev_status) atomicOr(dev_status, REFREE_DEV_NONFINITE);
    // Fixed point of the unit: C_n * 2^S in [2^60, 2^61), from the binary order of magnitude of the sum of squares.
    // A block sums its squares at the scale of its own largest key; the blocks exchange (largest key, sum) once and
    // bring the sums to the scale of the unit's largest key, a power of two apart, in rank order.
    const uint32_t mx_b = block_reduce<uint32_t>(mx, reinterpret_cast<uint32_t *>(sm.ibuf), MaxOpU());
    float acc_b = 0.f;
    {
        const float fb = ldexpf(1.0f, 127 - max(1, (int)(mx_b >> 23)));
#pragma unroll
        for (int e = 0; e < E; ++e) {
            if (e >= e_lim) continue;
            const float a = ((kb[e] >> 23) == 255u) ? 0.f : __uint_as_float(kb[e]) * fb;
            acc_b = fmaf(a, a, acc_b);
        }
        acc_b = block_reduce<float>(acc_b, sm.fbuf, AddOpF());
    }
    float acc = acc_b;
    mx = mx_b;
    if (nblk > 1) {
        if (threadIdx.x == 0) { sm.y_mx = mx_b; sm.y_acc = acc_b; }
        cl.sync();                                  // the slots are written once: no second barrier
        uint32_t rm[kMaxCluster];
        float ra[kMaxCluster];
#pragma unroll
        for (int b = 0; b < kMaxCluster; ++b) {
            rm[b] = b < nblk ? *cl.map_shared_rank(&sm.y_mx, b) : 0u;
            ra[b] = b < nblk ? *cl.map_shared_rank(&sm.y_acc, b) : 0.f;
        }
        mx = 0u;
#pragma unroll
        for (int b = 0; b < kMaxCluster; ++b) mx = max(mx, rm[b]);
        acc = 0.f;
#pragma unroll
        for (int b = 0; b < kMaxCluster; ++b)
            if (b < nblk) acc += ldexpf(ra[b], 2 * (max(1, (int)(rm[b] >> 23)) - max(1, (int)(mx >> 23))));
    }
    if (n > 0 && mx != 0u) {
        const int emax = max(1, (int)(mx >> 23));
        v.sbias = 60 - ilogbf(fmaxf(acc, 0.25f)) - 2 * (emax - 127) - 300;
        cut.sbias = v.sbias;
        if (v.lead + v.w_eff >= n) { v.lead = n; v.w_eff = 0; }      // the protected prefix covers the sequence
        const int prot = v.lead + v.w_eff;
        u64 Cn;
        {
            u64 local = 0;
#pragma unroll
            for (int e = 0; e < E; ++e)
                if (e < e_lim) local += sq_fixed(kb[e], v.sbias);
            u64 tot;
            block_excl_scan<u64>(local, sm.ubuf, tot);
            Cn = tot;
            if (nblk > 1) {
                if (threadIdx.x == 0) sm.x_u64 = tot;
                cl.sync();                              // written once: no second barrier
                u64 rt[kMaxCluster];
#pragma unroll
                for (int b = 0; b < kMaxCluster; ++b) rt[b] = b < nblk ? *cl.map_shared_rank(&sm.x_u64, b) : 0ull;
                Cn = 0ull;
#pragma unroll
                for (int b = 0; b < kMaxCluster; ++b) Cn += rt[b];
            }
        }
        const u64 c_min = crossing_level(Cn, (double)p.threshold);      // every thread: a handful of fp64 operations
        const u64 Sprot = range_totals(v, 0, prot, ProtRank(), sm.wpre);
        const int jp = range_find(v, prot, ProtRank(), c_min, sm.wpre, sm.ibuf);
        int jstar = n;
        cut.prot_kept = prot;
        cut.tau = 0ull;                       // keep every unprotected position ...
        cut.ties = INT_MAX;                   // ... unless a crossing is found below
        if (jp != INT_MAX) {
            jstar = jp;
        } else if (prot < n && c_min != ~0ull) {
            const u64 need = c_min - Sprot;   // mass still missing after the protected prefix (> 0)
            uint32_t prefix = 0u, above_cnt = 0u;     // the same in every thread of the cluster
            u64 above_sum = 0ull;
            int digit_cnt = 0;
            bool any = true;
            auto clear_hist = [&]() {
                for (int t = threadIdx.x; t < kWarps * 257; t += kThreads) {
                    (&sm.wcnt[0][0])[t] = 0u;
                    (&sm.wsum[0][0])[t] = 0ull;
                }
            };
            clear_hist();
            __syncthreads();
            bool spelled = false;             // the crossing key is known in full before the last level
            for (int level = 0; level < 4 && any && !spelled; ++level) {
                const int shift = 24 - 8 * level;
                const int hb = level & 1;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const int i = (e * nblk + rank) * kThreads + threadIdx.x;
                    if (e < e_lim && i >= v.lead && i < n - v.w_eff && (level == 0 || (kb[e] >> (shift + 8)) == prefix)) {
                        const int dgt = (int)((kb[e] >> shift) & 255u);
                        atomicAdd(&sm.wcnt[warp][dgt], 1u);
                        add_u64_shared(&sm.wsum[warp][dgt], sq_fixed(kb[e], v.sbias));
                    }
                }
                __syncthreads();
                if (threadIdx.x < 256) {
                    unsigned int c = 0u;
                    u64 sumv = 0ull;
                    for (int wv = 0; wv < kWarps; ++wv) { c += sm.wcnt[wv][threadIdx.x]; sumv += sm.wsum[wv][threadIdx.x]; }
                    sm.hcnt2[hb][threadIdx.x] = c;
                    sm.hsum2[hb][threadIdx.x] = sumv;
                }
                // thread t < 256 owns digit 255 - t: the cluster's totals of it (integers: any order)
                unsigned int mycnt = 0u;
                u64 mysum = 0ull;
                if (nblk > 1) {
                    cl.sync();
                    if (threadIdx.x < 256) {
                        unsigned int rc[kMaxCluster];
                        u64 rs[kMaxCluster];
#pragma unroll
                        for (int b = 0; b < kMaxCluster; ++b) {          // all remote reads in flight together
                            rc[b] = b < nblk ? cl.map_shared_rank(sm.hcnt2[hb], b)[255 - threadIdx.x] : 0u;
                            rs[b] = b < nblk ? cl.map_shared_rank(sm.hsum2[hb], b)[255 - threadIdx.x] : 0ull;
                        }
#pragma unroll
                        for (int b = 0; b < kMaxCluster; ++b) { mycnt += rc[b]; mysum += rs[b]; }
                    }
                } else {
                    __syncthreads();
                    if (threadIdx.x < 256) { mycnt = sm.hcnt2[hb][255 - threadIdx.x]; mysum = sm.hsum2[hb][255 - threadIdx.x]; }
                }
                clear_hist();                 // for the next level: the per-warp histograms were read before the barrier above
                // sums from the top digit down; the first digit at which they reach what is missing
                const u64 inc_s = warp_incl_scan(mysum);
                const unsigned int inc_c = warp_incl_scan(mycnt);
                if (warp < 8 && lane == 31) { sm.dsum[warp] = inc_s; sm.dcnt[warp] = inc_c; }
                __syncthreads();
                u64 abv_s = inc_s - mysum;
                unsigned int abv_c = inc_c - mycnt;
                if (warp < 8)
                    for (int wv = 0; wv < warp; ++wv) { abv_s += sm.dsum[wv]; abv_c += sm.dcnt[wv]; }
                const bool hit = warp < 8 && mycnt > 0u && above_sum + abv_s + mysum >= need;
                const unsigned int hm = __ballot_sync(0xffffffffu, hit);
                if (warp < 8) {
                    const int first = hm ? __ffs(hm) - 1 : 0;
                    if (lane == first) {          // the warp's first crossing digit leaves its record (none: lane 0 says so)
                        sm.dcand[warp] = hm ? warp * 32 + first : INT_MAX;
                        sm.dabv_s[warp] = abv_s;
                        sm.dabv_c[warp] = abv_c;
                        sm.ddig[warp] = mycnt;
                    }
                }
                __syncthreads();
                int cand = INT_MAX, cw = 0;
#pragma unroll
                for (int wv = 7; wv >= 0; --wv)
                    if (sm.dcand[wv] != INT_MAX) { cand = sm.dcand[wv]; cw = wv; }
                if (cand == INT_MAX) {
                    any = false;              // the rule is never met: keep all
                } else {
                    prefix = (prefix << 8) | (uint32_t)(255 - cand);
                    above_sum += sm.dabv_s[cw];
                    above_cnt += sm.dabv_c[cw];
                    digit_cnt = (int)sm.ddig[cw];
                    if (digit_cnt == 1 && level < 3) {
                        // One position has the crossing digits: the remaining levels would only spell out its key.
                        // The thread that holds it says it; every block reads it after one barrier.
#pragma unroll
                        for (int e = 0; e < E; ++e) {
                            const int i = (e * nblk + rank) * kThreads + threadIdx.x;
                            if (e < e_lim && i >= v.lead && i < n - v.w_eff && (kb[e] >> shift) == prefix) sm.z_key = kb[e];
                        }
                        uint32_t key = 0u;
                        if (nblk > 1) {
                            cl.sync();
#pragma unroll
                            for (int b = 0; b < kMaxCluster; ++b)
                                if (b < nblk) key = max(key, *cl.map_shared_rank(&sm.z_key, b));
                        } else {
                            __syncthreads();
                            key = sm.z_key;
                        }
                        prefix = key;
                        spelled = true;
                    }
                }
            }
            if (any) {
                // `prefix` is the key at which the sum crosses; digit_cnt positions share it
                const u64 tau = (u64)prefix << 32;
                const u64 fq = sq_fixed(prefix, v.sbias);
                const u64 miss = need - above_sum;            // > 0: the digits above did not reach it
                u64 t = fq ? (miss + fq - 1) / fq : 1ull;
                t = max(1ull, min(t, (u64)digit_cnt));
                jstar = prot + (int)above_cnt + (int)t;
                cut.tau = tau;
                cut.ties = (int)t;
            }
        }
        cut.b = max(jstar, floor_b);
        if (cut.b <= prot) {                 // nothing beyond the protected prefix
            cut.prot_kept = cut.b;
            cut.tau = ~0ull;
            cut.ties = 0;
        }
    }
    if (chunk_counts) {
        // For the kernel that writes the index list: per run of kThreads positions, how many are kept for sure
        // and how many sit at the crossing key (element e of this block is run e * blocks + rank).
        const int lead = v.lead, w_eff = v.w_eff;
        int *wc = reinterpret_cast<int *>(&sm.wcnt[0][0]);              // [E][kWarps][2], free after the descent
        __syncthreads();
#pragma unroll
        for (int e = 0; e < E; ++e) {
            if (e >= e_lim) continue;                                  // no run of this block there
            const int i = (e * nblk + rank) * kThreads + threadIdx.x;
            bool sure = false, tie = false;
            if (i < n) {
                if (i < lead) sure = i < cut.prot_kept;
                else if (i >= n - w_eff) sure = lead + (i - (n - w_eff)) < cut.prot_kept;
                else { const u64 key = (u64)kb[e] << 32; sure = key > cut.tau; tie = key == cut.tau; }
            }
            const unsigned int smask = __ballot_sync(0xffffffffu, sure), tmask = __ballot_sync(0xffffffffu, tie);
            if (lane == 0) { wc[(e * kWarps + warp) * 2] = __popc(smask); wc[(e * kWarps + warp) * 2 + 1] = __popc(tmask); }
        }
        __syncthreads();
        if (threadIdx.x < E) {
            const int e = threadIdx.x, c = e * nblk + rank;
            if ((int64_t)c * kThreads < n) {
                int sure = 0, ties = 0;
                for (int wv = 0; wv < kWarps; ++wv) { sure += wc[(e * kWarps + wv) * 2]; ties += wc[(e * kWarps + wv) * 2 + 1]; }
                chunk_counts[(int64_t)(s * Hkv + g) * chunk_stride + c] = make_int2(sure, ties);
            }
        }
    }
    if (nblk > 1) cl.sync();               // no block exits while another may still read its shared memory
    if (threadIdx.x == 0 && rank == 0) {
        lengths[s * Hkv + g] = cut.b;
        cuts[s * Hkv + g] = cut;
    }
}

// Position ranking, one budget per (sequence, KV head), from the per-32-position
// partials that the scoring kernel left (GroupPartial): the stopping rule then
// touches one record per 32 scores plus the 32 scores of the group in which the
// cumulative sum crosses.  Same rule and fixed point as select_budget_kernel, with
// each group's sum first brought to the unit's common scale (a right shift).
__global__ void __launch_bounds__(kThreads)
select_groups_kernel(refree_params p, const float *scores, const int32_t *seq_len, int64_t total_tokens,
                     const GroupPartial *groups, int32_t *lengths, Cut *cuts)
{
    __shared__ u64 ubuf[kWarps + 1];
    __shared__ int ibuf[kWarps + 1];
    __shared__ int s_pack, s_tiles;
    __shared__ u64 s_cmin, s_sink;
    __shared__ int s_found;
    const int Hkv = p.num_kv_heads;
    const int s = blockIdx.x / Hkv, g = blockIdx.x % Hkv;
    if (threadIdx.x == 0) {
        int a = 0, b = 0;
        for (int t = 0; t < s; ++t) { const int nn = max(seq_len[t], 0); a += nn; b += ceil_div(nn, kTile); }
        s_pack = a;
        s_tiles = b;
    }
    __syncthreads();
    const int n = max(seq_len[s], 0);
    const float *sc = scores + (int64_t)g * total_tokens + s_pack;
    const int lead = min(p.sink, n), w_eff = min(p.window, n);
    const int floor_b = p.keep_window ? min(n, lead + w_eff) : min(n, 1);
    const int ng = ceil_div(n, 32);
    const GroupPartial *gp = groups + ((int64_t)s_tiles * Hkv + (int64_t)g * ceil_div(n, kTile)) * 4;
    Cut cut;
    cut.b = n; cut.ties = 0; cut.tau = 0; cut.prot_kept = 0; cut.sbias = 0;
    if (n > 0) {
        // common scale: the largest score's squared mantissa below 2^(56 - L), L = log2 of the group count
        uint32_t mx = 0;
        for (int k = threadIdx.x; k < ng; k += kThreads) mx = max(mx, gp[k].max_bits);
        mx = block_reduce<uint32_t>(mx, reinterpret_cast<uint32_t *>(ibuf), MaxOpU());
        if (mx != 0u) {
            const int emax = max(1, (int)(mx >> 23));
            int L = 0;
            while ((1 << L) < ng) ++L;
            const int sbias = kGroupShift - 2 * emax - L;
            cut.sbias = sbias;
            // mass of the leading positions (ranked first), and of every group without them
            u64 sink = 0;
            for (int i = threadIdx.x; i < lead; i += kThreads) sink += sq_fixed(mag_bits(sc[i]), sbias);
            {
                u64 tot;
                block_excl_scan<u64>(sink, ubuf, tot);
                sink = tot;
            }
            auto group_rest = [&](int k) -> u64 {
                const GroupPartial r = gp[k];
                const int shift = 2 * (emax - max(1, (int)(r.max_bits >> 23))) + L;
                u64 v = shift < 64 ? r.sum >> shift : 0ull;
                if (32 * k < lead) {                   // take the leading positions out of their group
                    u64 in = 0;
                    for (int i = 32 * k; i < min(lead, 32 * k + 32); ++i) in += sq_fixed(mag_bits(sc[i]), sbias);
                    v = v > in ? v - in : 0ull;
                }
                return v;
            };
            // groups in ranked order: from the last one backwards; thread t owns a contiguous run of them
            const int per = ceil_div(ng, kThreads);
            const int r0 = min(ng, (int)threadIdx.x * per), r1 = min(ng, r0 + per);
            u64 local = 0;
            for (int r = r0; r < r1; ++r) local += group_rest(ng - 1 - r);
            u64 rest_total;
            const u64 before = block_excl_scan<u64>(local, ubuf, rest_total);
            const u64 Cn = sink + rest_total;
            if (threadIdx.x == 0) { s_cmin = crossing_level(Cn, (double)p.threshold); s_found = INT_MAX; s_sink = sink; }
            __syncthreads();
            const u64 c_min = s_cmin;
            int jstar = INT_MAX;
            if (threadIdx.x == 0) {                    // crossing among the leading positions
                u64 c = 0;
                for (int i = 0; i < lead; ++i) {
                    c += sq_fixed(mag_bits(sc[i]), sbias);
                    if (c >= c_min) { s_found = i + 1; break; }
                }
            }
            __syncthreads();
            jstar = s_found;
            __syncthreads();
            if (jstar == INT_MAX && c_min != ~0ull) {
                // first group (in ranked order) at whose end the cumulative sum reaches c_min
                int hit = INT_MAX;
                u64 run = sink + before, hit_before = 0;
                for (int r = r0; r < r1; ++r) {
                    const u64 v = per == 1 ? local : group_rest(ng - 1 - r);   // one group per thread: already in a register
                    if (run + v >= c_min) { hit = r; hit_before = run; break; }
                    run += v;
                }
                const int first = block_reduce<int>(hit, ibuf, MinOp());
                if (first != INT_MAX) {
                    if (hit == first) { ubuf[0] = hit_before; }
                    __syncthreads();
                    if (threadIdx.x < 32) {
                        const int k = ng - 1 - first;
                        const int hi = min(n, 32 * k + 32) - 1, lo = max(lead, 32 * k);
                        const int pos = hi - (int)threadIdx.x;
                        u64 x = pos >= lo ? sq_fixed(mag_bits(sc[pos]), sbias) : 0ull;
                        x = warp_incl_scan(x);
                        const unsigned m = __ballot_sync(0xffffffffu, pos >= lo && ubuf[0] + x >= c_min);
                        // rank count of position pos: the leading ones, then n-1 down to pos
                        const int last = m ? hi - (__ffs(m) - 1) : lo;
                        if (threadIdx.x == 0) s_found = lead + (n - last);
                    }
                    __syncthreads();
                    jstar = s_found;
                }
            }
            cut.b = max(jstar == INT_MAX ? n : jstar, floor_b);
        }
    }
    if (threadIdx.x == 0) {
        lengths[blockIdx.x] = cut.b;
        cuts[blockIdx.x] = cut;
    }
}

// Offsets (running sum of lengths) and the kept positions of each unit, ascending.
__global__ void __launch_bounds__(kThreads)
emit_kernel(refree_params p, const float *scores, const int32_t *seq_len, int64_t total_tokens,
            const int32_t *lengths, const Cut *cuts, int64_t *offsets, int32_t *kept_idx,
            int64_t capacity_rows, int32_t *dev_status, const int2 *chunk_counts, int chunk_stride, int counted_upto)
{
    __shared__ long long lbuf[kWarps + 1];
    __shared__ int ibuf[kWarps + 1];
    __shared__ int s_pack;
    const int Hkv = p.num_kv_heads, U = p.num_seqs * Hkv;
    const int u = blockIdx.y, s = u / Hkv, g = u % Hkv;
    // score ranking: a block beyond the end of its sequence has nothing to do (the grid is sized for the longest
    // sequence a call can hold)
    if (blockIdx.x > 0 && p.rank_mode != REFREE_RANK_POSITION && !p.force_full &&
        (int64_t)blockIdx.x * kThreads >= max(seq_len[s], 0))
        return;
    // offsets[u] = sum of lengths before u
    long long part = 0, off;
    for (int t = threadIdx.x; t < u; t += kThreads) part += lengths[t];
    {
        long long tot;
        block_excl_scan<long long>(part, lbuf, tot);
        off = tot;
    }
    const Cut cut = cuts[u];
    const int b = cut.b;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        offsets[u] = off;
        if (u == U - 1) offsets[U] = off + b;
    }
    if (off + b > capacity_rows) {
        if (threadIdx.x == 0 && dev_status) atomicOr(dev_status, REFREE_DEV_CAPACITY);
        return;
    }
    if (kept_idx == nullptr) return;
    const int n = max(seq_len[s], 0);
    int lead = min(p.sink, n), w_eff = min(p.window, n);
    int32_t *dst = kept_idx + off;
    if (p.rank_mode == REFREE_RANK_POSITION || p.force_full) {
        const int head = min(b, lead);
        for (int t = blockIdx.x * kThreads + threadIdx.x; t < b; t += gridDim.x * kThreads)
            dst[t] = t < head ? t : n - b + t;
        return;
    }
    // Score ranking: block c of the unit owns positions [c * kThreads, (c + 1) * kThreads), one per thread.
    const int chunk = blockIdx.x * kThreads;
    if (chunk >= n) return;
    if (threadIdx.x == 0) {
        int a = 0;
        for (int t = 0; t < s; ++t) a += max(seq_len[t], 0);
        s_pack = a;
    }
    __syncthreads();
    if (lead + w_eff >= n) { lead = n; w_eff = 0; }
    UnitView v;
    const bool layer = p.scope == REFREE_SCOPE_LAYER;
    v.sc = scores + (int64_t)(layer ? 0 : g) * total_tokens + s_pack;
    v.head_stride = total_tokens;
    v.heads = layer ? Hkv : 1;
    v.n = n; v.lead = lead; v.w_eff = w_eff;
    v.sbias = cut.sbias;
    // kept for sure (above the crossing key, or protected and inside the budget) / at the crossing key, of
    // which the cut.ties lowest positions are kept
    // the key is loaded first, without a branch around it, so that a thread's loads are in flight together
    const bool one_head = v.heads == 1;
    auto key_of = [&](int i) {
        if (one_head) {                           // a plain predicated load, so the loads of an unrolled loop overlap
            const int ic = min(max(i, 0), n - 1);
            const uint32_t bits = mag_bits(v.sc[ic]);
            return (i >= lead && i < n - w_eff) ? (u64)bits << 32 : 0ull;
        }
        return (i >= lead && i < n - w_eff) ? key_at(v, i) : 0ull;
    };
    auto classify = [&](int i, u64 key, bool &sure, bool &tie) {
        sure = false; tie = false;
        if (i >= n) return;
        if (i < lead) {
            sure = i < cut.prot_kept;
        } else if (i >= n - w_eff) {
            sure = lead + (i - (n - w_eff)) < cut.prot_kept;
        } else {
            sure = key > cut.tau;
            tie = key == cut.tau;
        }
    };
    // What the positions before the chunk contribute: left per run of kThreads positions by the kernel that chose
    // the budget when it held the unit in registers; otherwise every block counts them itself (the scores are in L2).
    long long before = 0;                                   // (sure << 32) + ties
    if (chunk_counts && n <= counted_upto) {
        for (int c = threadIdx.x; c < (int)blockIdx.x; c += kThreads) {
            const int2 cc = chunk_counts[(int64_t)u * chunk_stride + c];
            before += ((long long)cc.x << 32) + (long long)cc.y;
        }
    } else
    for (int i0 = threadIdx.x; i0 < chunk; i0 += 8 * kThreads) {
        u64 key[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) key[q] = key_of(i0 + q * kThreads < chunk ? i0 + q * kThreads : n);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            bool sure, tie;
            classify(i0 + q * kThreads < chunk ? i0 + q * kThreads : n, key[q], sure, tie);
            before += ((long long)sure << 32) + (long long)tie;
        }
    }
    {
        long long tot;
        block_excl_scan<long long>(before, lbuf, tot);
        before = tot;
    }
    const int ties_before = (int)(before & 0xffffffffll), sure_before = (int)(before >> 32);
    const int lane = threadIdx.x & 31;
    bool sure, tie;
    classify(chunk + threadIdx.x, key_of(chunk + threadIdx.x), sure, tie);
    const unsigned int tm = __ballot_sync(0xffffffffu, tie);
    int tie_tot;
    const int tie_base = block_excl_scan<int>(lane == 0 ? __popc(tm) : 0, ibuf, tie_tot);   // lane 0 carries the warp's count
    const int tie_rank = ties_before + __shfl_sync(0xffffffffu, tie_base, 0) + __popc(tm & ((1u << lane) - 1u));
    if (tie && tie_rank < cut.ties) sure = true;
    const unsigned int km = __ballot_sync(0xffffffffu, sure);
    int keep_tot;
    const int keep_base = block_excl_scan<int>(lane == 0 ? __popc(km) : 0, ibuf, keep_tot);
    const int mine = sure_before + min(ties_before, cut.ties) + __shfl_sync(0xffffffffu, keep_base, 0) +
                     __popc(km & ((1u << lane) - 1u));
    if (sure && mine < b) dst[mine] = chunk + threadIdx.x;
}

}  // namespace

cudaError_t launch_select(const refree_params &p, const float *scores, const int32_t *seq_len,
                          int64_t total_tokens, int32_t *lengths, int64_t *offsets,
                          int32_t *kept_idx, int64_t capacity_rows, char *ws, const Workspace &lay,
                          int32_t *dev_status, cudaStream_t st, bool emit, const GroupPartial *groups)
{
    Cut *cuts = reinterpret_cast<Cut *>(ws + lay.cut_off);
    const int U = p.num_seqs * p.num_kv_heads;
    const int sel_units = p.scope == REFREE_SCOPE_LAYER ? p.num_seqs : U;
    {
        // the kernels' shared memory is above the default limit: raised once per device, under a lock
        static std::mutex attr_mutex;
        static bool attr_set[64] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> hold(attr_mutex);
        if (!attr_set[dev]) {
            const int bytes = (int)sizeof(SelectSmem);
            cudaError_t e = cudaFuncSetAttribute(select_budget_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(select_score_resident_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(select_score_resident_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(select_score_resident_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
            if (e != cudaSuccess) return e;
            attr_set[dev] = true;
        }
    }
    int skip_upto = 0;                       // units up to this length went to the register-resident kernel
    int2 *chunk_counts = nullptr;
    const int chunk_stride = (int)((total_tokens + kThreads - 1) / kThreads) + 1;
    if (groups && p.rank_mode == REFREE_RANK_POSITION && p.scope == REFREE_SCOPE_HEAD && !p.force_full) {
        select_groups_kernel<<<U, kThreads, 0, st>>>(p, scores, seq_len, total_tokens, groups, lengths, cuts);
        count_launches(1);
    } else {
        // score ranking walks every score several times: a cluster of blocks shares a unit (distributed
        // shared memory for the few totals they exchange); position ranking keeps one block per unit
        int nblk = 1;
        if (p.rank_mode == REFREE_RANK_SCORE && !p.force_full) {
            const int64_t avg = total_tokens / std::max(1, p.num_seqs);
            while (nblk < kMaxCluster && avg >= (int64_t)nblk * 4096) nblk *= 2;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(sel_units * nblk);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = sizeof(SelectSmem);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = nblk;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (nblk > 1) {
            int clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&clusters, select_budget_kernel, &cfg) != cudaSuccess || clusters < 1) {
                (void)cudaGetLastError();
                nblk = 1;
                cfg.gridDim = dim3(sel_units);
                attr[0].val.clusterDim.x = 1;
            }
        }
        // Score ranking per head: units short enough for a cluster to hold in registers go to the kernel that
        // reads the scores once; the general kernel takes the rest (all of them when none is short enough).
        if (p.rank_mode == REFREE_RANK_SCORE && !p.force_full && p.scope == REFREE_SCOPE_HEAD) {
            // blocks per unit by the mean length, like the general kernel; elements per thread so that the longest
            // sequence the call can hold fits if 16 allow it (longer units go to the general kernel)
            const int rb = nblk;
            const int64_t want = std::min<int64_t>(total_tokens, (int64_t)rb * kThreads * 16);
            int E = 4;
            while (E < 16 && (int64_t)rb * kThreads * E < want) E *= 2;
            cudaLaunchConfig_t rc = cfg;
            cudaLaunchAttribute rattr[1];
            rattr[0] = attr[0];
            rattr[0].val.clusterDim.x = rb;
            rc.attrs = rattr;
            rc.gridDim = dim3(sel_units * rb);
            cudaError_t re = cudaErrorInvalidValue;
            int clusters = 0;
            auto fits = [&](auto kern) {
                return rb == 1 || (cudaOccupancyMaxActiveClusters(&clusters, kern, &rc) == cudaSuccess && clusters >= 1);
            };
            // counts per run of kThreads positions for the index list, where the caller's workspace has room for them
            if (emit && kept_idx && lay.part_bytes >= (size_t)U * (size_t)chunk_stride * sizeof(int2))
                chunk_counts = reinterpret_cast<int2 *>(ws + lay.part_off);
            if (E == 4 && fits(select_score_resident_kernel<4>))
                re = cudaLaunchKernelEx(&rc, select_score_resident_kernel<4>, p, scores, seq_len, total_tokens, lengths, cuts, dev_status, chunk_counts, chunk_stride);
            else if (E == 8 && fits(select_score_resident_kernel<8>))
                re = cudaLaunchKernelEx(&rc, select_score_resident_kernel<8>, p, scores, seq_len, total_tokens, lengths, cuts, dev_status, chunk_counts, chunk_stride);
            else if (E == 16 && fits(select_score_resident_kernel<16>))
                re = cudaLaunchKernelEx(&rc, select_score_resident_kernel<16>, p, scores, seq_len, total_tokens, lengths, cuts, dev_status, chunk_counts, chunk_stride);
            if (re == cudaSuccess) {
                skip_upto = rb * kThreads * E;
                count_launches(1);
            } else {
                (void)cudaGetLastError();
                chunk_counts = nullptr;
            }
        }
        if (skip_upto == 0 || (int64_t)skip_upto < total_tokens) {
            const cudaError_t le = cudaLaunchKernelEx(&cfg, select_budget_kernel, p, scores, seq_len, total_tokens, lengths,
                                                      cuts, dev_status, skip_upto);
            if (le != cudaSuccess) return le;
            count_launches(1);
        }
    }
    if (!emit) return cudaGetLastError();               // the caller forms the offsets itself and needs no index list
    const bool ranges = p.rank_mode == REFREE_RANK_POSITION || p.force_full;
    int gx = 1;
    if (ranges && kept_idx) {
        const int64_t per_unit = std::max<int64_t>(1, total_tokens / std::max(1, p.num_seqs));
        gx = (int)std::min<int64_t>(16, (per_unit + 4 * kThreads - 1) / (4 * kThreads));
    } else if (kept_idx) {
        // score ranking: a block per kThreads positions of the longest sequence there can be
        gx = (int)std::max<int64_t>(1, (total_tokens + kThreads - 1) / kThreads);
    }
    emit_kernel<<<dim3(gx, U), kThreads, 0, st>>>(p, scores, seq_len, total_tokens, lengths, cuts, offsets,
                                                  kept_idx, capacity_rows, dev_status, chunk_counts, chunk_stride, skip_upto);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace refree
