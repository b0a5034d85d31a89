// Position ranking, one budget per (sequence, KV head), from the per-32-position records (GroupPartial) that a
// scoring kernel leaves: the arithmetic of the stopping rule shared by the selection kernel (a block per unit)
// and by the scoring kernel's finishing warp (a warp per unit, for the unit whose last tile it has just scored).
// Integer sums throughout, so the two agree bit for bit whatever the order of their additions.
#pragma once

#include <limits.h>

#include "refree_internal.cuh"

namespace refree {

// Smallest fixed-point C with 1 - sqrt(C / Cn) < T, i.e. Cn - C < Cn * T * (2 - T); ~0 when there is none.
__device__ inline unsigned long long crossing_level(unsigned long long Cn, double T)
{
    const double lim = (double)Cn * (T * (2.0 - T));
    const double c = ceil(lim);
    if (!(c >= 1.0)) return ~0ull;                 // T = 0: never met
    const unsigned long long dmax = (unsigned long long)c - 1ull;     // largest dropped mass that still meets the rule
    return dmax >= Cn ? 0ull : Cn - dmax;
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

// Common scale of a unit's groups: the largest score's squared mantissa below 2^(56 - L), L = log2 of the group count.
__device__ inline int groups_sbias(uint32_t max_bits, int ng, int &emax, int &L)
{
    emax = max(1, (int)(max_bits >> 23));
    L = 0;
    while ((1 << L) < ng) ++L;
    return kGroupShift - 2 * emax - L;
}

// The whole rule for one unit by one warp (all 32 lanes call it).  `sc` = the unit's scores, `gp` = its records.
// Reads go around L1 (the data may have been written by other SMs a moment ago).
// `mx` = bit pattern of the unit's largest score when the caller has it already (else kNoMax: found here).
constexpr uint32_t kNoMax = 0xffffffffu;
__device__ inline Cut select_unit_from_groups_warp(const refree_params &p, const float *sc, int n, const GroupPartial *gp,
                                                   uint32_t mx = kNoMax)
{
    const int lane = threadIdx.x & 31;
    const int lead = min(p.sink, n), w_eff = min(p.window, n);
    const int floor_b = p.keep_window ? min(n, lead + w_eff) : min(n, 1);
    const int ng = ceil_div(n, 32);
    Cut cut;
    cut.b = n; cut.ties = 0; cut.tau = 0; cut.prot_kept = 0; cut.sbias = 0;
    if (n <= 0) return cut;
    if (mx == kNoMax) {
        mx = 0;
        for (int k = lane; k < ng; k += 32) mx = max(mx, __ldcg(&gp[k].max_bits));
        mx = __reduce_max_sync(0xffffffffu, mx);
    }
    if (mx == 0u) return cut;
    int emax, L;
    const int sbias = groups_sbias(mx, ng, emax, L);
    cut.sbias = sbias;
    auto score_at = [&](int i) { return __ldcg(sc + i); };
    // sum of group k at the unit's scale, without the leading positions (ranked first, apart)
    auto rest_of = [&](const uint4 &raw, int k) -> unsigned long long {
        const uint32_t bits = raw.x;
        const unsigned long long sum = ((unsigned long long)raw.w << 32) | raw.z;
        const int shift = 2 * (emax - max(1, (int)(bits >> 23))) + L;
        unsigned long long v = shift < 64 ? sum >> shift : 0ull;
        if (32 * k < lead) {
            unsigned long long in = 0;
            for (int i = 32 * k; i < min(lead, 32 * k + 32); ++i) in += sq_fixed(mag_bits(score_at(i)), sbias);
            v = v > in ? v - in : 0ull;
        }
        return v;
    };
    const uint4 *raw = reinterpret_cast<const uint4 *>(gp);
    // mass of the leading positions (ranked first)
    unsigned long long sink = 0;
    for (int i = lane; i < lead; i += 32) sink += sq_fixed(mag_bits(score_at(i)), sbias);
    for (int o = 16; o; o >>= 1) sink += __shfl_xor_sync(0xffffffffu, sink, o);
    // groups in ranked order (from the last one backwards): lane t owns a contiguous run of ranks and sums it,
    // eight records in flight at a time
    const int per = ceil_div(ng, 32);
    const int r0 = min(ng, lane * per), r1 = min(ng, r0 + per);
    unsigned long long local = 0;
    for (int r = r0; r < r1; r += 8) {
        uint4 rec[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) rec[q] = r + q < r1 ? __ldcg(raw + (ng - 1 - (r + q))) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int q = 0; q < 8; ++q) if (r + q < r1) local += rest_of(rec[q], ng - 1 - (r + q));
    }
    const unsigned long long inc = warp_incl_scan(local);
    const unsigned long long Cn = sink + __shfl_sync(0xffffffffu, inc, 31);
    const unsigned long long c_min = crossing_level(Cn, (double)p.threshold);
    // crossing among the leading positions, 32 at a time
    int jstar = INT_MAX;
    {
        unsigned long long c = 0;
        for (int i0 = 0; i0 < lead && jstar == INT_MAX; i0 += 32) {
            const int i = i0 + lane;
            const unsigned long long x = i < lead ? sq_fixed(mag_bits(score_at(i)), sbias) : 0ull;
            const unsigned long long xi = warp_incl_scan(x);
            const unsigned m = __ballot_sync(0xffffffffu, i < lead && c + xi >= c_min);
            if (m) jstar = i0 + __ffs(m);
            c += __shfl_sync(0xffffffffu, xi, 31);
        }
    }
    if (jstar == INT_MAX && c_min != ~0ull) {
        // the lane in whose run the cumulative sum reaches c_min, then that run 32 groups at a time by the whole warp
        const unsigned mrun = __ballot_sync(0xffffffffu, r0 < r1 && sink + inc >= c_min);
        if (mrun) {
            const int owner = __ffs(mrun) - 1;
            unsigned long long run = sink + __shfl_sync(0xffffffffu, inc - local, owner);
            const int q0 = min(ng, owner * per), q1 = min(ng, q0 + per);
            int first = INT_MAX;
            unsigned long long base = 0;
            for (int rb = q0; rb < q1 && first == INT_MAX; rb += 32) {
                const int r = rb + lane;
                const unsigned long long v = r < q1 ? rest_of(__ldcg(raw + (ng - 1 - r)), ng - 1 - r) : 0ull;
                const unsigned long long vi = warp_incl_scan(v);
                const unsigned m = __ballot_sync(0xffffffffu, r < q1 && run + vi >= c_min);
                if (m) {
                    const int src = __ffs(m) - 1;
                    first = rb + src;
                    base = run + __shfl_sync(0xffffffffu, vi - v, src);
                }
                run += __shfl_sync(0xffffffffu, vi, 31);
            }
            if (first != INT_MAX) {
                const int k = ng - 1 - first;
                const int hi = min(n, 32 * k + 32) - 1, lo = max(lead, 32 * k);
                const int pos = hi - lane;
                unsigned long long x = pos >= lo ? sq_fixed(mag_bits(score_at(pos)), sbias) : 0ull;
                x = warp_incl_scan(x);
                const unsigned m = __ballot_sync(0xffffffffu, pos >= lo && base + x >= c_min);
                // rank count of position pos: the leading ones, then n-1 down to pos
                const int last = m ? hi - (__ffs(m) - 1) : lo;
                jstar = lead + (n - last);
            }
        }
    }
    cut.b = max(jstar == INT_MAX ? n : jstar, floor_b);
    return cut;
}

}  // namespace refree
