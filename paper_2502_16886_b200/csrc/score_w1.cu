// Scoring for the paper's default reduced attention, w = 1 (Section 3.2 "Reducing
// Overhead", k = 1; Algorithm 1 uses Q[..., -1, :]): one query per head, so the
// logits are G numbers per position and the step is a pure stream over K.
//
//   logits  thread = position: y[h][i] = (q_h . k_i / sqrt(d)) * log2(e) for the G heads of
//           the KV head, K row read with 16-byte loads, q broadcast from shared memory;
//           y goes to the workspace (4 G bytes per position against 256 for the K row),
//           with the block's (max, sum 2^(y - max)) per head
//   scores  L_h = log2 sum_i 2^(y_h[i]) from the block partials, then
//           a'[i] = (1/G) sum_h 2^(y_h[i] - L_h)   (Eq. 2 with one row: cnt = 1)
//
// K is read once; no tensor cores (G x 1 x d per position is a matrix-vector
// product: intensity G flop/B, far below the ridge).
#include <algorithm>

#include "refree_internal.cuh"

namespace refree {
namespace {

constexpr int kThreadsW1 = 256;
constexpr int kChunk = 256;          // positions per block iteration
constexpr int kMaxG = 16;
constexpr float kLog2eW1 = 1.4426950408889634f;

struct W1Tables {
    int32_t pack[kMaxSeqs + 1];
    int32_t chunks[kMaxSeqs + 1];    // 256-position chunks before sequence s
    int32_t tiles[kMaxSeqs + 1];     // 128-position tiles before sequence s (index of the GroupPartial records)
    int32_t len[kMaxSeqs];
};

__device__ inline void build_w1_tables(W1Tables &t, const int32_t *seq_len, int B)
{
    if (threadIdx.x == 0) {
        int a = 0, b = 0, c = 0;
        for (int s = 0; s < B; ++s) {
            t.pack[s] = a; t.chunks[s] = b; t.tiles[s] = c;
            const int n = max(seq_len[s], 0);
            t.len[s] = n;
            a += n; b += ceil_div(n, kChunk); c += ceil_div(n, kTile);
        }
        t.pack[B] = a; t.chunks[B] = b; t.tiles[B] = c;
    }
    __syncthreads();
}

struct W1Item { int s, g, chunk, n, pos0; };

// items ordered (sequence, head, chunk)
__device__ inline W1Item decode_w1(const W1Tables &t, int B, int Hkv, int item)
{
    int lo = 0, hi = B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((int64_t)t.chunks[mid] * Hkv <= item) lo = mid; else hi = mid;
    }
    W1Item it;
    it.s = lo;
    const int cs = t.chunks[lo + 1] - t.chunks[lo];
    const int rem = item - t.chunks[lo] * Hkv;
    it.g = rem / cs;
    it.chunk = rem % cs;
    it.n = t.len[lo];
    it.pos0 = it.chunk * kChunk;
    return it;
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
    float2 *stats;          // [chunks_total * Hkv][G]: per block (max, sum)
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
    __shared__ float2 red[kWarpsW1][GMAX];
    const refree_params &p = a.p;
    const int B = p.num_seqs, Hkv = p.num_kv_heads, G = p.num_q_heads / Hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane / LPR, part = lane % LPR;   // row of the load this lane helps with, its 16-byte slice
    const float scale = kLog2eW1 * rsqrtf((float)D);
    build_w1_tables(tb, a.seq_len, B);
    const int items = tb.chunks[B] * Hkv;
    int cur_u = -1;
    float qreg[GMAX][E];
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const W1Item it = decode_w1(tb, B, Hkv, item);
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
        // running (max, sum) per head over the rows this lane leads
        float m[GMAX], z[GMAX];
#pragma unroll
        for (int h = 0; h < GMAX; ++h) { m[h] = -INFINITY; z[h] = 0.f; }
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
            if (part == 0 && valid) {
#pragma unroll
                for (int h = 0; h < GMAX; ++h) {
                    if (h < G) {
                        a.logits[(int64_t)(it.g * G + h) * a.total_tokens + tb.pack[it.s] + i] = y[h];
                        if (y[h] > m[h]) { z[h] = z[h] * exp2f(m[h] - y[h]) + 1.f; m[h] = y[h]; }
                        else z[h] += exp2f(y[h] - m[h]);
                    }
                }
            }
        }
        // block (max, sum) per head: lanes -> warp -> block, in a fixed order
#pragma unroll
        for (int h = 0; h < GMAX; ++h) {
            if (h < G) {
                float mm = m[h];
                for (int o = 16; o; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, o));
                float zz = (z[h] > 0.f) ? z[h] * exp2f(m[h] - mm) : 0.f;
                for (int o = 16; o; o >>= 1) zz += __shfl_xor_sync(0xffffffffu, zz, o);
                if (lane == 0) red[warp][h] = make_float2(mm, zz);
            }
        }
        __syncthreads();
        if (threadIdx.x < G) {
            float mm = -INFINITY, zz = 0.f;
            for (int wv = 0; wv < kWarpsW1; ++wv) mm = fmaxf(mm, red[wv][threadIdx.x].x);
            for (int wv = 0; wv < kWarpsW1; ++wv) {
                const float2 pr = red[wv][threadIdx.x];
                if (pr.y > 0.f) zz += pr.y * exp2f(pr.x - mm);
            }
            a.stats[((int64_t)(tb.chunks[it.s] * Hkv) + (int64_t)it.g * (tb.chunks[it.s + 1] - tb.chunks[it.s]) +
                     it.chunk) * G + threadIdx.x] = make_float2(mm, zz);
        }
        __syncthreads();
    }
}

template <int GMAX>
__global__ void __launch_bounds__(kThreadsW1)
w1_scores_kernel(W1Args a)
{
    __shared__ W1Tables tb;
    __shared__ float lse[GMAX];
    const refree_params &p = a.p;
    const int B = p.num_seqs, Hkv = p.num_kv_heads, G = p.num_q_heads / Hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    build_w1_tables(tb, a.seq_len, B);
    const int items = tb.chunks[B] * Hkv;
    int cur_u = -1;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const W1Item it = decode_w1(tb, B, Hkv, item);
        const int u = it.s * Hkv + it.g;
        __syncthreads();
        if (u != cur_u) {
            // L_h = log2 sum_i 2^(y_h[i]): one warp per head over the unit's block partials, in a fixed order
            const int cs = tb.chunks[it.s + 1] - tb.chunks[it.s];
            const float2 *st = a.stats + ((int64_t)(tb.chunks[it.s] * Hkv) + (int64_t)it.g * cs) * G;
            for (int h = warp; h < G; h += kThreadsW1 / 32) {
                float m = -INFINITY;
                for (int c = lane; c < cs; c += 32) m = fmaxf(m, st[(int64_t)c * G + h].x);
                for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
                float z = 0.f;
                for (int c = lane; c < cs; c += 32) {
                    const float2 pr = st[(int64_t)c * G + h];
                    if (pr.y > 0.f) z += pr.y * exp2f(pr.x - m);
                }
                for (int o = 16; o; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
                if (lane == 0) lse[h] = m + log2f(z);
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
                tot += exp2f(a.logits[(int64_t)(it.g * G + h) * a.total_tokens + tb.pack[it.s] + i] - lse[h]);
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

template <typename T, int D, int GMAX>
cudaError_t run_w1(W1Args &a, const void *q_win, const void *k, int grid, cudaStream_t st)
{
    w1_logits_kernel<T, D, GMAX><<<grid, kThreadsW1, 0, st>>>(a, (const T *)q_win, (const T *)k);
    w1_scores_kernel<GMAX><<<grid, kThreadsW1, 0, st>>>(a);
    count_launches(2);
    return cudaGetLastError();
}

template <typename T, int D>
cudaError_t run_w1_g(W1Args &a, const void *q_win, const void *k, int grid, cudaStream_t st, int G)
{
    if (G <= 4) return run_w1<T, D, 4>(a, q_win, k, grid, st);
    if (G <= 8) return run_w1<T, D, 8>(a, q_win, k, grid, st);
    return run_w1<T, D, 16>(a, q_win, k, grid, st);
}

}  // namespace

bool score_w1_supported(const refree_params &p)
{
    return p.window == 1 && p.num_q_heads / p.num_kv_heads <= kMaxG && (p.head_dim == 64 || p.head_dim == 128);
}

size_t score_w1_scratch_bytes(const refree_params &p, int64_t total_tokens)
{
    const int64_t chunks = total_tokens / kChunk + p.num_seqs;
    return (size_t)p.num_q_heads * total_tokens * sizeof(float) + 256 +
           (size_t)chunks * p.num_q_heads * sizeof(float2);
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
    const int64_t max_items = (total_tokens / kChunk + p.num_seqs) * p.num_kv_heads;
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>(max_items, 148 * 8));
    const int G = p.num_q_heads / p.num_kv_heads;
    const bool f32 = p.dtype == REFREE_DTYPE_F32;
    if (p.head_dim == 64)
        return f32 ? run_w1_g<float, 64>(a, q_win, k, grid, st, G) : run_w1_g<__nv_bfloat16, 64>(a, q_win, k, grid, st, G);
    return f32 ? run_w1_g<float, 128>(a, q_win, k, grid, st, G) : run_w1_g<__nv_bfloat16, 128>(a, q_win, k, grid, st, G);
}

}  // namespace refree
