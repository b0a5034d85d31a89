// Scoring for the paper's default reduced attention, w = 1 (Section 3.2 "Reducing
// Overhead", k = 1; Algorithm 1 uses Q[..., -1, :]): one query per head, so the
// logits are G numbers per position and the step is a pure stream over K.
//
//   logits  y[h][i] = (q_h . k_i / sqrt(d)) * log2(e) for the G heads of the KV head.
//           bf16: a warp owns a span of positions of one unit; 16 rows x d of K go from
//           global memory straight into the A fragments of mma.m16n8k16 (16 bytes per lane,
//           the four lanes of a row 64 contiguous bytes per instruction), the queries
//           sit in the B fragments, loaded the same way so the element order inside a
//           k-step cancels.  The tensor-core instruction is used as a dot-product unit
//           (it replaces ~50 fp32 instructions per row); the kernel is bound by the K stream.
//           fp32 (or unaligned queries): lane groups per row on the fp32 pipes, shuffle-reduced.
//           y goes to the workspace (4 G bytes per position against 256 for the K row),
//           with one (max, sum 2^(y - max)) record per head and span
//   scores  L_h = log2 sum_i 2^(y_h[i]) from the span records, then
//           a'[i] = (1/G) sum_h 2^(y_h[i] - L_h)   (Eq. 2 with one row: cnt = 1)
//
// K is read once (intensity G flop/B, far below the ridge).
#include <algorithm>

#include "refree_internal.cuh"

namespace refree {
namespace {

constexpr int kThreadsW1 = 256;
constexpr int kChunk = 256;          // positions per block iteration
constexpr int kMaxG = 16;
constexpr int kMinSpan = 32;         // positions per (max, sum) record of the mma path: a multiple of 16
constexpr int kMaxSpan = 512;
constexpr float kLog2eW1 = 1.4426950408889634f;

struct W1Tables {
    int32_t pack[kMaxSeqs + 1];
    int32_t chunks[kMaxSeqs + 1];    // 256-position chunks before sequence s
    int32_t spans[kMaxSeqs + 1];     // spans (the unit of the (max, sum) records) before sequence s
    int32_t tiles[kMaxSeqs + 1];     // 128-position tiles before sequence s (index of the GroupPartial records)
    int32_t len[kMaxSeqs];
};

__device__ inline void build_w1_tables(W1Tables &t, const int32_t *seq_len, int B, int span)
{
    if (threadIdx.x == 0) {
        int a = 0, b = 0, c = 0, e = 0;
        for (int s = 0; s < B; ++s) {
            t.pack[s] = a; t.chunks[s] = b; t.tiles[s] = c; t.spans[s] = e;
            const int n = max(seq_len[s], 0);
            t.len[s] = n;
            a += n; b += ceil_div(n, kChunk); c += ceil_div(n, kTile); e += ceil_div(n, span);
        }
        t.pack[B] = a; t.chunks[B] = b; t.tiles[B] = c; t.spans[B] = e;
    }
    __syncthreads();
}

struct W1Item { int s, g, chunk, n, pos0; };

// items ordered (sequence, head, piece); `before` counts the pieces (chunks or spans) ahead of a sequence
__device__ inline W1Item decode_w1(const W1Tables &t, const int32_t *before, int piece_len, int B, int Hkv, int item)
{
    int lo = 0, hi = B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((int64_t)before[mid] * Hkv <= item) lo = mid; else hi = mid;
    }
    W1Item it;
    it.s = lo;
    const int cs = before[lo + 1] - before[lo];
    const int rem = item - before[lo] * Hkv;
    it.g = rem / cs;
    it.chunk = rem % cs;
    it.n = t.len[lo];
    it.pos0 = it.chunk * piece_len;
    return it;
}

__device__ inline float ex2(float x)
{
    float y;
    asm("ex2.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// (max, sum) records combine as m = max, z = z1 2^(m1 - m) + z2 2^(m2 - m)
__device__ inline void merge_stats(float &m, float &z, float mo, float zo)
{
    const float mn = fmaxf(m, mo);
    z = mn == -INFINITY ? 0.f : z * ex2(m - mn) + zo * ex2(mo - mn);
    m = mn;
}

template <typename T> struct Row16;                       // 16 bytes of a K row as floats
template <> struct Row16<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static void load(const void *p, float (&f)[8])
    {
        const uint4 r = *reinterpret_cast<const uint4 *>(p);
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};
template <> struct Row16<float> {
    static constexpr int kElems = 4;
    __device__ static void load(const void *p, float (&f)[8])
    {
        const float4 r = *reinterpret_cast<const float4 *>(p);
        f[0] = r.x; f[1] = r.y; f[2] = r.z; f[3] = r.w;
    }
};

struct W1Args {
    refree_params p;
    const int32_t *seq_start, *seq_len;
    float *logits;          // [Hq][total_tokens]
    float2 *stats;          // [spans_total * Hkv][G]: (max, sum) per span and head
    int span;               // positions per record
    GroupPartial *groups;   // nullable
    float *scores;
    int64_t total_tokens;
    int32_t *dev_status;
};

// A K row is covered by LPR = row_bytes / 16 lanes, 16 bytes each, so a warp reads
// 32 / LPR whole rows per load instruction (fully coalesced).  Each lane keeps its
// slice of the G queries in registers; the partial dot products meet by shuffles.
template <typename T, int D, int GMAX>
__global__ void __launch_bounds__(kThreadsW1)
w1_logits_kernel(W1Args a, const T *q_win, const T *k)
{
    constexpr int E = Row16<T>::kElems;              // elements per lane and row
    constexpr int LPR = D / E;                       // lanes per row: 8, 16 or 32
    constexpr int RPW = 32 / LPR;                    // rows per warp and load
    constexpr int kWarpsW1 = kThreadsW1 / 32;
    constexpr int kRowsPerWarp = kChunk / kWarpsW1;  // 32 positions of the chunk per warp
    __shared__ W1Tables tb;
    __shared__ float2 red[kWarpsW1 * RPW][GMAX];
    const refree_params &p = a.p;
    const int B = p.num_seqs, Hkv = p.num_kv_heads, G = p.num_q_heads / Hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane / LPR, part = lane % LPR;   // row of the load this lane helps with, its 16-byte slice
    const float scale = kLog2eW1 * rsqrtf((float)D);
    build_w1_tables(tb, a.seq_len, B, kChunk);      // one record per block chunk: span == kChunk
    const int items = tb.chunks[B] * Hkv;
    int cur_u = -1;
    float qreg[GMAX][E];
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const W1Item it = decode_w1(tb, tb.chunks, kChunk, B, Hkv, item);
        const int u = it.s * Hkv + it.g;
        if (u != cur_u) {                            // this lane's slice of the unit's G queries, pre-scaled
#pragma unroll
            for (int h = 0; h < GMAX; ++h)
#pragma unroll
                for (int e = 0; e < E; ++e)
                    qreg[h][e] = h < G ? to_float(q_win[((int64_t)it.s * p.num_q_heads + it.g * G + h) * D + part * E + e]) * scale
                                       : 0.f;
            cur_u = u;
        }
        const char *base = reinterpret_cast<const char *>(
            k + (int64_t)it.s * p.k_stride_seq + (int64_t)a.seq_start[it.s] * p.k_stride_tok + (int64_t)it.g * p.k_stride_head);
        const int64_t tok_bytes = p.k_stride_tok * (int64_t)sizeof(T);
        // after the butterfly every lane of a row group holds all G logits of the row: lane l of the
        // group takes heads l, l + LPR, ... (one store and one running (max, sum) update per head)
        constexpr int HPL = (GMAX + LPR - 1) / LPR;
        float m[HPL], z[HPL];
#pragma unroll
        for (int j = 0; j < HPL; ++j) { m[j] = -INFINITY; z[j] = 0.f; }
        float *unit_logits = a.logits + (int64_t)(it.g * G) * a.total_tokens + tb.pack[it.s];
        const int wpos0 = it.pos0 + warp * kRowsPerWarp;
#pragma unroll 4
        for (int r = 0; r < kRowsPerWarp; r += RPW) {
            const int i = wpos0 + r + sub;
            const bool valid = i < it.n;
            float kf[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) kf[e] = 0.f;
            if (valid) Row16<T>::load(base + (int64_t)i * tok_bytes + part * 16, kf);
            float y[GMAX];
#pragma unroll
            for (int h = 0; h < GMAX; ++h) {
                float acc = 0.f;
#pragma unroll
                for (int e = 0; e < E; ++e) acc = fmaf(kf[e], qreg[h][e], acc);
                y[h] = acc;
            }
#pragma unroll
            for (int o = LPR / 2; o; o >>= 1)
#pragma unroll
                for (int h = 0; h < GMAX; ++h)
                    if (h < G) y[h] += __shfl_xor_sync(0xffffffffu, y[h], o);
#pragma unroll
            for (int j = 0; j < HPL; ++j) {
                float mine = 0.f;
#pragma unroll
                for (int h = j * LPR; h < GMAX && h < (j + 1) * LPR; ++h) mine = (part == h - j * LPR) ? y[h] : mine;
                const int head = part + j * LPR;
                if (head < G && valid) {
                    unit_logits[(int64_t)head * a.total_tokens + i] = mine;
                    merge_stats(m[j], z[j], mine, 1.f);
                }
            }
        }
        // block (max, sum) per head: the RPW row groups of every warp, in a fixed order
#pragma unroll
        for (int j = 0; j < HPL; ++j)
            if (part + j * LPR < GMAX) red[warp * RPW + sub][part + j * LPR] = make_float2(m[j], z[j]);
        __syncthreads();
        if (threadIdx.x < G) {
            float mm = -INFINITY, zz = 0.f;
            for (int wv = 0; wv < kWarpsW1 * RPW; ++wv) merge_stats(mm, zz, red[wv][threadIdx.x].x, red[wv][threadIdx.x].y);
            a.stats[((int64_t)(tb.chunks[it.s] * Hkv) + (int64_t)it.g * (tb.chunks[it.s + 1] - tb.chunks[it.s]) +
                     it.chunk) * G + threadIdx.x] = make_float2(mm, zz);
        }
        __syncthreads();
    }
}

__device__ inline void mma_bf16_16x8x16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ inline uint4 ld_row16(const char *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// bf16 logits on mma.m16n8k16.  Lane (r, c) = (lane / 4, lane % 4) of a warp loads, for rows r and
// r + 8 of a 16-row block, the 16-byte pieces at byte 64 j + 16 c of the row (the four lanes of a
// row read two whole 32-byte sectors per instruction); the four 32-bit words of a piece feed two
// k-steps as (a0, a2) resp. (a1, a3).  The B operand
// is the query of head r (and r + 8 for the second column tile) cut the same way, so every product
// pairs the same element of k_i and q_h whatever slot of the k-step it occupies.  The accumulator
// of lane (r, c) holds heads 2c, 2c + 1 for rows r and r + 8.  NT column tiles cover G <= 8 NT heads.
template <int D, int NT>
__global__ void __launch_bounds__(kThreadsW1)
w1_logits_mma_kernel(W1Args a, const __nv_bfloat16 *q_win, const __nv_bfloat16 *k)
{
    constexpr int CH = D / 32;                       // 16-byte pieces per lane and row
    constexpr int kWarpsW1 = kThreadsW1 / 32;
    __shared__ W1Tables tb;
    const refree_params &p = a.p;
    const int B = p.num_seqs, Hkv = p.num_kv_heads, G = p.num_q_heads / Hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = lane >> 2, c = lane & 3;
    const float scale = kLog2eW1 * rsqrtf((float)D);
    build_w1_tables(tb, a.seq_len, B, a.span);
    const int items = tb.spans[B] * Hkv;
    const int64_t tok_bytes = p.k_stride_tok * (int64_t)sizeof(__nv_bfloat16);
    int cur_u = -1;
    uint4 qf[NT][CH];
    for (int item = blockIdx.x * kWarpsW1 + warp; item < items; item += gridDim.x * kWarpsW1) {
        const W1Item it = decode_w1(tb, tb.spans, a.span, B, Hkv, item);
        const int u = it.s * Hkv + it.g;
        if (u != cur_u) {
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                const int head = t * 8 + r;
                const char *qrow = reinterpret_cast<const char *>(
                    q_win + ((int64_t)it.s * p.num_q_heads + it.g * G + min(head, G - 1)) * D);
#pragma unroll
                for (int j = 0; j < CH; ++j) {
                    qf[t][j] = *reinterpret_cast<const uint4 *>(qrow + j * 64 + c * 16);
                    if (head >= G) qf[t][j] = make_uint4(0u, 0u, 0u, 0u);
                }
            }
            cur_u = u;
        }
        const char *base = reinterpret_cast<const char *>(
            k + (int64_t)it.s * p.k_stride_seq + (int64_t)a.seq_start[it.s] * p.k_stride_tok + (int64_t)it.g * p.k_stride_head);
        float *unit_logits = a.logits + (int64_t)(it.g * G) * a.total_tokens + tb.pack[it.s];
        const int end = min(it.n, it.pos0 + a.span);
        float m[NT][2], z[NT][2];
#pragma unroll
        for (int t = 0; t < NT; ++t) { m[t][0] = m[t][1] = -INFINITY; z[t][0] = z[t][1] = 0.f; }
#pragma unroll 2
        for (int row0 = it.pos0; row0 < end; row0 += 16) {
            const int i0 = row0 + r, i1 = i0 + 8;
            const bool v0 = i0 < end, v1 = i1 < end;
            uint4 ka[CH], kb[CH];
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                const int off = j * 64 + c * 16;
                ka[j] = v0 ? ld_row16(base + (int64_t)i0 * tok_bytes + off) : make_uint4(0u, 0u, 0u, 0u);
                kb[j] = v1 ? ld_row16(base + (int64_t)i1 * tok_bytes + off) : make_uint4(0u, 0u, 0u, 0u);
            }
            float acc[NT][4];
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f;
#pragma unroll
                for (int j = 0; j < CH; ++j) {
                    mma_bf16_16x8x16(acc[t], ka[j].x, kb[j].x, ka[j].y, kb[j].y, qf[t][j].x, qf[t][j].y);
                    mma_bf16_16x8x16(acc[t], ka[j].z, kb[j].z, ka[j].w, kb[j].w, qf[t][j].z, qf[t][j].w);
                }
            }
#pragma unroll
            for (int t = 0; t < NT; ++t)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int head = t * 8 + 2 * c + e;
                    if (head < G) {
                        const float y0 = acc[t][e] * scale, y1 = acc[t][2 + e] * scale;
                        float *dst = unit_logits + (int64_t)head * a.total_tokens;
                        if (v0) dst[i0] = y0;
                        if (v1) dst[i1] = y1;
                        const float ym = fmaxf(v0 ? y0 : -INFINITY, v1 ? y1 : -INFINITY);
                        if (ym > -INFINITY) {
                            const float mn = fmaxf(m[t][e], ym);
                            z[t][e] = z[t][e] * ex2(m[t][e] - mn) + (v0 ? ex2(y0 - mn) : 0.f) + (v1 ? ex2(y1 - mn) : 0.f);
                            m[t][e] = mn;
                        }
                    }
                }
        }
        // one record per head and span: the eight row lanes of a column pair combine in a fixed order
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) {
                    const float mo = __shfl_xor_sync(0xffffffffu, m[t][e], o);
                    const float zo = __shfl_xor_sync(0xffffffffu, z[t][e], o);
                    merge_stats(m[t][e], z[t][e], mo, zo);
                }
                const int head = t * 8 + 2 * c + e;
                if (r == 0 && head < G)
                    a.stats[((int64_t)tb.spans[it.s] * Hkv + (int64_t)it.g * (tb.spans[it.s + 1] - tb.spans[it.s]) +
                             it.chunk) * G + head] = make_float2(m[t][e], z[t][e]);
            }
    }
}

template <int GMAX>
__global__ void __launch_bounds__(kThreadsW1)
w1_scores_kernel(W1Args a)
{
    constexpr int kWarpsW1 = kThreadsW1 / 32;
    __shared__ W1Tables tb;
    __shared__ float2 red[kWarpsW1][GMAX];
    __shared__ float lse[GMAX];
    const refree_params &p = a.p;
    const int B = p.num_seqs, Hkv = p.num_kv_heads, G = p.num_q_heads / Hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    build_w1_tables(tb, a.seq_len, B, a.span);
    const int items = tb.chunks[B] * Hkv;
    // a block takes consecutive chunks, so it stays inside one unit as long as it can
    const int per = ceil_div(items, (int)gridDim.x);
    const int first = blockIdx.x * per, last = min(items, first + per);
    int cur_u = -1;
    for (int item = first; item < last; ++item) {
        const W1Item it = decode_w1(tb, tb.chunks, kChunk, B, Hkv, item);
        const int u = it.s * Hkv + it.g;
        if (u != cur_u) {
            // L_h = log2 sum_i 2^(y_h[i]) from the unit's span records, combined in a fixed order
            const int cs = tb.spans[it.s + 1] - tb.spans[it.s];
            const float2 *st = a.stats + ((int64_t)tb.spans[it.s] * Hkv + (int64_t)it.g * cs) * G;
            float m[GMAX], z[GMAX];
#pragma unroll
            for (int h = 0; h < GMAX; ++h) { m[h] = -INFINITY; z[h] = 0.f; }
            for (int c = threadIdx.x; c < cs; c += kThreadsW1)
#pragma unroll
                for (int h = 0; h < GMAX; ++h)
                    if (h < G) { const float2 pr = st[(int64_t)c * G + h]; merge_stats(m[h], z[h], pr.x, pr.y); }
#pragma unroll
            for (int h = 0; h < GMAX; ++h)
                if (h < G) {
#pragma unroll
                    for (int o = 16; o; o >>= 1) {
                        const float mo = __shfl_xor_sync(0xffffffffu, m[h], o);
                        const float zo = __shfl_xor_sync(0xffffffffu, z[h], o);
                        merge_stats(m[h], z[h], mo, zo);
                    }
                    if (lane == 0) red[warp][h] = make_float2(m[h], z[h]);
                }
            __syncthreads();
            if (threadIdx.x < G) {
                float mm = -INFINITY, zz = 0.f;
                for (int wv = 0; wv < kWarpsW1; ++wv) merge_stats(mm, zz, red[wv][threadIdx.x].x, red[wv][threadIdx.x].y);
                lse[threadIdx.x] = mm + log2f(zz);
            }
            cur_u = u;
            __syncthreads();
        }
        const int i = it.pos0 + threadIdx.x;
        const bool valid = i < it.n;
        float sc = 0.f;
        if (valid) {
            float tot = 0.f;
            for (int h = 0; h < G; ++h)
                tot += ex2(a.logits[(int64_t)(it.g * G + h) * a.total_tokens + tb.pack[it.s] + i] - lse[h]);
            sc = tot / (float)G;
            if (!isfinite(sc) && a.dev_status) atomicOr(a.dev_status, REFREE_DEV_NONFINITE);
            a.scores[(int64_t)it.g * a.total_tokens + tb.pack[it.s] + i] = sc;
        }
        if (a.groups) {                         // exact sum of squares of this warp's 32 positions
            const uint32_t bits = (valid && isfinite(sc)) ? mag_bits(sc) : 0u;
            const uint32_t mx = __reduce_max_sync(0xffffffffu, bits);
            unsigned long long sq = sq_fixed(bits, kGroupShift - 2 * max(1, (int)(mx >> 23)));
            for (int o = 16; o; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
            const int grp = (it.pos0 >> 5) + warp;
            if (lane == 0 && grp * 32 < ceil_div(it.n, kTile) * kTile) {
                GroupPartial gp; gp.max_bits = mx; gp.pad = 0u; gp.sum = sq;
                a.groups[((int64_t)tb.tiles[it.s] * Hkv + (int64_t)it.g * ceil_div(it.n, kTile)) * 4 + grp] = gp;
            }
        }
    }
}


template <int GMAX>
cudaError_t run_w1_scores(W1Args &a, int64_t chunk_items, cudaStream_t st)
{
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>(chunk_items, sm_count() * 4));
    w1_scores_kernel<GMAX><<<grid, kThreadsW1, 0, st>>>(a);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t run_w1_scores_g(W1Args &a, int64_t chunk_items, cudaStream_t st, int G)
{
    if (G <= 4) return run_w1_scores<4>(a, chunk_items, st);
    if (G <= 8) return run_w1_scores<8>(a, chunk_items, st);
    return run_w1_scores<16>(a, chunk_items, st);
}

template <typename T, int D>
cudaError_t run_w1_lanes(W1Args &a, const void *q_win, const void *k, int grid, cudaStream_t st, int G)
{
    if (G <= 4) w1_logits_kernel<T, D, 4><<<grid, kThreadsW1, 0, st>>>(a, (const T *)q_win, (const T *)k);
    else if (G <= 8) w1_logits_kernel<T, D, 8><<<grid, kThreadsW1, 0, st>>>(a, (const T *)q_win, (const T *)k);
    else w1_logits_kernel<T, D, 16><<<grid, kThreadsW1, 0, st>>>(a, (const T *)q_win, (const T *)k);
    count_launches(1);
    return cudaGetLastError();
}

template <int D>
cudaError_t run_w1_mma(W1Args &a, const void *q_win, const void *k, int grid, cudaStream_t st, int G)
{
    if (G <= 8) w1_logits_mma_kernel<D, 1><<<grid, kThreadsW1, 0, st>>>(a, (const __nv_bfloat16 *)q_win, (const __nv_bfloat16 *)k);
    else w1_logits_mma_kernel<D, 2><<<grid, kThreadsW1, 0, st>>>(a, (const __nv_bfloat16 *)q_win, (const __nv_bfloat16 *)k);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace

bool score_w1_supported(const refree_params &p)
{
    return p.window == 1 && p.num_q_heads / p.num_kv_heads <= kMaxG && (p.head_dim == 64 || p.head_dim == 128);
}

size_t score_w1_scratch_bytes(const refree_params &p, int64_t total_tokens)
{
    const int64_t spans = total_tokens / kMinSpan + p.num_seqs;          // the shortest span bounds the record count
    return (size_t)p.num_q_heads * total_tokens * sizeof(float) + 256 +
           (size_t)spans * p.num_q_heads * sizeof(float2);
}

cudaError_t launch_score_w1(const refree_params &p, const void *q_win, const void *k,
                            const int32_t *seq_start, const int32_t *seq_len,
                            int64_t total_tokens, float *scores, char *ws, const Workspace &lay,
                            int32_t *dev_status, cudaStream_t st, GroupPartial *groups)
{
    W1Args a;
    a.p = p;
    a.seq_start = seq_start;
    a.seq_len = seq_len;
    a.logits = reinterpret_cast<float *>(ws + lay.part_off);
    const size_t logits_bytes = ((size_t)p.num_q_heads * total_tokens * sizeof(float) + 255) & ~(size_t)255;
    a.stats = reinterpret_cast<float2 *>(ws + lay.part_off + logits_bytes);
    a.groups = groups;
    a.scores = scores;
    a.total_tokens = total_tokens;
    a.dev_status = dev_status;
    const int G = p.num_q_heads / p.num_kv_heads;
    const bool f32 = p.dtype == REFREE_DTYPE_F32;
    const int64_t chunk_items = (total_tokens / kChunk + p.num_seqs) * p.num_kv_heads;
    cudaError_t e;
    if (!f32 && !(reinterpret_cast<uintptr_t>(q_win) & 15)) {
        // one span per warp when the pass fits a single wave of 2 blocks per SM; capped so that
        // short sequences still spread over the machine
        const int64_t warps = (int64_t)sm_count() * 2 * (kThreadsW1 / 32);
        const int64_t rows = total_tokens * p.num_kv_heads;
        int64_t span = (rows + warps - 1) / warps;
        span = std::min<int64_t>(kMaxSpan, std::max<int64_t>(kMinSpan, (span + 15) / 16 * 16));
        a.span = (int)span;
        const int64_t span_items = (total_tokens / span + p.num_seqs) * p.num_kv_heads;
        const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((span_items + 7) / 8, sm_count() * 2));
        e = p.head_dim == 64 ? run_w1_mma<64>(a, q_win, k, grid, st, G) : run_w1_mma<128>(a, q_win, k, grid, st, G);
    } else {
        a.span = kChunk;
        const int grid = (int)std::max<int64_t>(1, std::min<int64_t>(chunk_items, sm_count() * 8));
        if (p.head_dim == 64)
            e = f32 ? run_w1_lanes<float, 64>(a, q_win, k, grid, st, G) : run_w1_lanes<__nv_bfloat16, 64>(a, q_win, k, grid, st, G);
        else
            e = f32 ? run_w1_lanes<float, 128>(a, q_win, k, grid, st, G) : run_w1_lanes<__nv_bfloat16, 128>(a, q_win, k, grid, st, G);
    }
    if (e != cudaSuccess) return e;
    return run_w1_scores_g(a, chunk_items, st, G);
}

}  // namespace refree
