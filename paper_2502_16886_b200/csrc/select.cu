// Steps S4-S6: ranking, the threshold-free stopping rule and the kept set.
//
// For one unit with squares sq_i = (double)a'_i^2 (exact: a' is fp32) and ranked
// order pi, the rule is the cumulative form of Eq. 1 (Eq. 3; Algorithm 1 Square,
// Reorder, Cumsum, Sqrt, ratio, Where):
//     C_j = sum_{t<=j} sq[pi_t],  j* = leftmost j with 1 - sqrt(C_j / C_n) < T,
// all of it in fp64.  The budget is b = max(j*, floor); the kept set is the first
// b ranked positions, emitted in ascending position order.
//
// Position ranking (Section 3.2) needs no sort: the order is the m leading
// positions, then the rest from the end backwards, so C_j is a block-wide prefix
// scan over a closed-form order.  Score ranking (Section 4.4) needs the order by
// decreasing score; instead of sorting, a radix descent over the 64-bit keys
// (8 bits per level) finds the key at which the cumulative sum crosses, using
// per-digit histograms of counts and of fixed-point sums of squares.  Integer
// sums make the result independent of the order in which threads add.
#include <algorithm>

#include "refree_internal.cuh"

namespace refree {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;

__device__ inline bool crossed(double C, double Cn, double T)
{
    return Cn > 0.0 && (1.0 - __dsqrt_rn(__ddiv_rn(C, Cn))) < T;
}

struct UnitView {
    const float *sc;        // scores of head 0 (layer scope) or of the unit's head, at the sequence start
    int64_t head_stride;    // distance between heads in the score array
    int heads;              // heads whose squares add up (1 in head scope)
    int n, lead, w_eff;
};

__device__ inline double sq_at(const UnitView &v, int i)
{
    double acc = 0.0;
    for (int h = 0; h < v.heads; ++h) {
        const double a = (double)v.sc[(int64_t)h * v.head_stride + i];
        acc += a * a;
    }
    return acc;
}

// position of protected rank j: leading positions, then (score ranking) the window
__device__ inline int pos_of_rank_position_mode(const UnitView &v, int j)
{
    return j < v.lead ? j : v.n - 1 - (j - v.lead);
}
__device__ inline int pos_of_protected_rank(const UnitView &v, int j)
{
    return j < v.lead ? j : v.n - v.w_eff + (j - v.lead);
}

template <typename Tv> __device__ inline Tv warp_incl_scan(Tv x)
{
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const Tv y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += y;
    }
    return x;
}

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

__device__ inline int block_min(int x, int *buf)
{
    for (int o = 16; o; o >>= 1) x = min(x, __shfl_xor_sync(0xffffffffu, x, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) buf[threadIdx.x >> 5] = x;
    __syncthreads();
    int r = buf[0];
    for (int wv = 1; wv < kWarps; ++wv) r = min(r, buf[wv]);
    return r;
}

// Prefix scan over ranks [0, count) in the order given by `pos_of`, starting from
// C = 0: returns the first rank count j (1-based) at which the rule is met, or
// INT_MAX, and the sum over all `count` ranks.  Each thread owns a contiguous run
// of ranks.  The rule (an fp64 divide and square root) is evaluated once per
// thread at the end of its run; the leftmost run whose end meets it holds the
// crossing, and warp 0 resolves it inside that run, 32 ranks at a time.
template <typename PosOf>
__device__ inline int scan_find(const UnitView &v, int count, PosOf pos_of, double Cn, double T,
                                bool search, double *dbuf, int *ibuf, double &sum)
{
    const int per = ceil_div(count, kThreads);
    const int j0 = min(count, (int)threadIdx.x * per), j1 = min(count, j0 + per);
    double local = 0.0;
    for (int j = j0; j < j1; ++j) local += sq_at(v, pos_of(v, j));
    const double before = block_excl_scan<double>(local, dbuf, sum);
    if (!search) return INT_MAX;
    int hit = (j1 > j0 && crossed(before + local, Cn, T)) ? (int)threadIdx.x : INT_MAX;
    hit = block_min(hit, ibuf);
    if (hit == INT_MAX) return INT_MAX;
    __syncthreads();
    if ((int)threadIdx.x == hit) dbuf[0] = before;
    __syncthreads();
    const int h0 = min(count, hit * per), h1 = min(count, h0 + per);
    int found = h1;                                   // the run's end meets the rule by construction
    if (threadIdx.x < 32) {
        double run = dbuf[0];
        const int lane = threadIdx.x;
        for (int base = h0; base < h1; base += 32) {
            const int j = base + lane;
            double x = j < h1 ? sq_at(v, pos_of(v, j)) : 0.0;
            x = warp_incl_scan(x);
            const unsigned m = __ballot_sync(0xffffffffu, j < h1 && crossed(run + x, Cn, T));
            if (m) { found = base + __ffs(m); break; }
            run += __shfl_sync(0xffffffffu, x, 31);
        }
        if (lane == 0) ibuf[0] = found;
    }
    __syncthreads();
    found = ibuf[0];
    __syncthreads();
    return found;
}

struct SelectSmem {
    double dbuf[kWarps + 1];
    int ibuf[kWarps + 1];
    unsigned int hcnt[256];
    unsigned long long hsum[256];
    int pack;
    // radix state
    unsigned long long prefix, above_sum;
    unsigned int above_cnt;
    int digit;
};

__global__ void __launch_bounds__(kThreads)
select_budget_kernel(refree_params p, const float *scores, const int32_t *seq_len,
                     int64_t total_tokens, int32_t *lengths, Cut *cuts)
{
    __shared__ SelectSmem sm;
    const int Hkv = p.num_kv_heads;
    const bool layer = p.scope == REFREE_SCOPE_LAYER;
    const int s = layer ? blockIdx.x : blockIdx.x / Hkv;
    const int g = layer ? 0 : blockIdx.x % Hkv;
    if (threadIdx.x == 0) {
        int a = 0;
        for (int t = 0; t < s; ++t) a += max(seq_len[t], 0);
        sm.pack = a;
    }
    __syncthreads();
    const int n = max(seq_len[s], 0);
    const double T = (double)p.threshold;
    UnitView v;
    v.sc = scores + (int64_t)g * total_tokens + sm.pack;
    v.head_stride = total_tokens;
    v.heads = layer ? Hkv : 1;
    v.n = n;
    v.w_eff = min(p.window, n);
    v.lead = min(p.sink, n);
    const int floor_b = p.keep_window ? min(n, v.lead + v.w_eff) : min(n, 1);

    Cut cut;
    cut.b = n; cut.ties = 0; cut.tau = 0; cut.prot_kept = 0; cut.pad = 0;

    if (n > 0 && !p.force_full) {
        if (p.rank_mode == REFREE_RANK_POSITION) {
            double Cn, dummy;
            scan_find(v, n, pos_of_rank_position_mode, 0.0, T, false, sm.dbuf, sm.ibuf, Cn);
            const int j = scan_find(v, n, pos_of_rank_position_mode, Cn, T, true, sm.dbuf, sm.ibuf, dummy);
            const int jstar = (j == INT_MAX) ? n : j;
            cut.b = max(jstar, floor_b);
        } else {
            // score ranking: when the protected prefix covers the sequence the order is 0..n-1
            if (v.lead + v.w_eff >= n) { v.lead = n; v.w_eff = 0; }
            const int prot = v.lead + v.w_eff;
            double Cn, Sprot;
            // C_n over every position (position order is as good as any for the total)
            {
                UnitView all = v; all.lead = n; all.w_eff = 0;
                scan_find(all, n, pos_of_protected_rank, 0.0, T, false, sm.dbuf, sm.ibuf, Cn);
            }
            const int jp = scan_find(v, prot, pos_of_protected_rank, Cn, T, true, sm.dbuf, sm.ibuf, Sprot);
            int jstar = n;
            cut.prot_kept = prot;
            cut.tau = 0ull;                       // keep every unprotected position ...
            cut.ties = INT_MAX;                   // ... unless a crossing is found below
            if (jp != INT_MAX) {
                jstar = jp;
            } else if (Cn > 0.0 && prot < n) {
                // fixed point with C_n * 2^e in [2^61, 2^62)
                const int e = 61 - ilogb(Cn);
                if (threadIdx.x == 0) { sm.prefix = 0ull; sm.above_sum = 0ull; sm.above_cnt = 0u; }
                bool any = true;
                for (int level = 0; level < 8 && any; ++level) {
                    const int shift = 56 - 8 * level;
                    for (int t = threadIdx.x; t < 256; t += kThreads) { sm.hcnt[t] = 0u; sm.hsum[t] = 0ull; }
                    __syncthreads();
                    const unsigned long long prefix = sm.prefix;
                    for (int i = v.lead + threadIdx.x; i < n - v.w_eff; i += kThreads) {
                        const double x = sq_at(v, i);
                        const unsigned long long key = (unsigned long long)__double_as_longlong(x);
                        if (level == 0 || (key >> (shift + 8)) == prefix) {
                            const int dgt = (int)((key >> shift) & 255ull);
                            atomicAdd(&sm.hcnt[dgt], 1u);
                            atomicAdd(&sm.hsum[dgt], __double2ull_rd(ldexp(x, e)));
                        }
                    }
                    __syncthreads();
                    // inclusive sums from the top digit down; thread t owns digit 255 - t
                    unsigned long long mysum = 0ull, tot_s;
                    unsigned int mycnt = 0u, tot_c;
                    if (threadIdx.x < 256) { mysum = sm.hsum[255 - threadIdx.x]; mycnt = sm.hcnt[255 - threadIdx.x]; }
                    const unsigned long long abv_s = block_excl_scan<unsigned long long>(mysum, (unsigned long long *)sm.dbuf, tot_s);
                    const unsigned int abv_c = block_excl_scan<unsigned int>(mycnt, (unsigned int *)sm.ibuf, tot_c);
                    int cand = INT_MAX;
                    if (threadIdx.x < 256 && mycnt > 0u) {
                        const double C = Sprot + ldexp((double)(sm.above_sum + abv_s + mysum), -e);
                        if (crossed(C, Cn, T)) cand = threadIdx.x;
                    }
                    cand = block_min(cand, sm.ibuf);
                    if (cand == INT_MAX) {
                        any = false;              // the rule is never met: keep all
                    } else {
                        if ((int)threadIdx.x == cand) {
                            sm.prefix = (prefix << 8) | (unsigned long long)(255 - cand);
                            sm.above_sum += abv_s;
                            sm.above_cnt += abv_c;
                            sm.digit = (int)mycnt;
                        }
                    }
                    __syncthreads();
                }
                if (any) {
                    // sm.prefix is the full key at which the sum crosses; sm.digit of them tie
                    const unsigned long long tau = sm.prefix;
                    const int ties_total = sm.digit;
                    const unsigned long long f = __double2ull_rd(ldexp(__longlong_as_double((long long)tau), e));
                    int lo = 1, hi = ties_total;   // smallest t with the rule met; t = hi is known to meet it
                    while (lo < hi) {
                        const int mid = (lo + hi) >> 1;
                        const double C = Sprot + ldexp((double)(sm.above_sum + (unsigned long long)mid * f), -e);
                        if (crossed(C, Cn, T)) hi = mid; else lo = mid + 1;
                    }
                    jstar = prot + (int)sm.above_cnt + lo;
                    cut.tau = tau;
                    cut.ties = lo;
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
    if (threadIdx.x == 0) {
        const int g_hi = layer ? Hkv : g + 1;
        for (int gg = g; gg < g_hi; ++gg) {
            lengths[s * Hkv + gg] = cut.b;
            cuts[s * Hkv + gg] = cut;
        }
    }
}

// Offsets (running sum of lengths) and the kept positions of each unit, ascending.
__global__ void __launch_bounds__(kThreads)
emit_kernel(refree_params p, const float *scores, const int32_t *seq_len, int64_t total_tokens,
            const int32_t *lengths, const Cut *cuts, int64_t *offsets, int32_t *kept_idx,
            int64_t capacity_rows, int32_t *dev_status)
{
    __shared__ long long lbuf[kWarps + 1];
    __shared__ int ibuf[kWarps + 1];
    __shared__ int s_pack;
    const int Hkv = p.num_kv_heads, U = p.num_seqs * Hkv;
    const int u = blockIdx.y, s = u / Hkv, g = u % Hkv;
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
    if (blockIdx.x != 0) return;
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
    int base = 0, tie_base = 0;
    for (int i0 = 0; i0 < n; i0 += kThreads) {
        const int i = i0 + threadIdx.x;
        int tie = 0, keep = 0;
        if (i < n) {
            if (i < lead) {
                keep = i < cut.prot_kept;
            } else if (i >= n - w_eff) {
                keep = lead + (i - (n - w_eff)) < cut.prot_kept;
            } else {
                const unsigned long long key = (unsigned long long)__double_as_longlong(sq_at(v, i));
                keep = key > cut.tau;
                tie = key == cut.tau;
            }
        }
        int tie_tot, keep_tot;
        const int tie_rank = tie_base + block_excl_scan<int>(tie, ibuf, tie_tot);
        if (tie && tie_rank < cut.ties) keep = 1;
        const int slot = base + block_excl_scan<int>(keep, ibuf, keep_tot);
        if (keep && slot < b) dst[slot] = i;
        base += keep_tot;
        tie_base += tie_tot;
    }
}

}  // namespace

cudaError_t launch_select(const refree_params &p, const float *scores, const int32_t *seq_len,
                          int64_t total_tokens, int32_t *lengths, int64_t *offsets,
                          int32_t *kept_idx, int64_t capacity_rows, char *ws, const Workspace &lay,
                          int32_t *dev_status, cudaStream_t st, bool emit)
{
    Cut *cuts = reinterpret_cast<Cut *>(ws + lay.cut_off);
    const int U = p.num_seqs * p.num_kv_heads;
    const int sel_units = p.scope == REFREE_SCOPE_LAYER ? p.num_seqs : U;
    select_budget_kernel<<<sel_units, kThreads, 0, st>>>(p, scores, seq_len, total_tokens, lengths, cuts);
    if (!emit) {               // the caller forms the offsets itself and needs no index list
        count_launches(1);
        return cudaGetLastError();
    }
    const bool ranges = p.rank_mode == REFREE_RANK_POSITION || p.force_full;
    int gx = 1;
    if (ranges && kept_idx) {
        const int64_t per_unit = std::max<int64_t>(1, total_tokens / max(1, p.num_seqs));
        gx = (int)std::min<int64_t>(16, (per_unit + 4 * kThreads - 1) / (4 * kThreads));
    }
    emit_kernel<<<dim3(gx, U), kThreads, 0, st>>>(p, scores, seq_len, total_tokens, lengths, cuts, offsets,
                                                  kept_idx, capacity_rows, dev_status);
    count_launches(2);
    return cudaGetLastError();
}

}  // namespace refree
