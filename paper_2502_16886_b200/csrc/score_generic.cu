// Generic scoring path (steps S1-S3) on the plain fp32 pipes: any supported dtype,
// head_dim 64 or 128, any window and query-group size.  It serves the fp32 cache,
// shapes the tensor-core path does not take, and is the simple statement of the
// three-kernel structure the fast path follows:
//   stats   per (tile, KV head, window row): max and sum of 2^(y - max) over the
//           visible positions of the tile, y = (q.k / sqrt(d)) * log2(e)
//   combine per (unit, row): L = log2 sum_i 2^(y_i) over the whole row
//   colsum  per (tile, KV head): a'[i] = (1/G) sum_rows 2^(y - L) / cnt(i)   (Eq. 2)
#include <algorithm>

#include "refree_internal.cuh"

namespace refree {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr float kLog2e = 1.4426950408889634f;

template <int D> struct GenericSmem {
    SeqTables seq;
    float k[kTile][D + 1];
    float q[kWarps][D];
    float red[kWarps][kTile];
};

struct Item {
    int s, g, tile_global, pos0, npos, n, w_eff, pack;
};

__device__ inline Item decode_item(const SeqTables &t, const int32_t *seq_len, int B, int Hkv, int w,
                                   int item)
{
    Item it;
    it.tile_global = item / Hkv;
    it.g = item % Hkv;
    it.s = find_seq(t.tiles, B, it.tile_global);
    it.n = seq_len[it.s];
    it.pos0 = (it.tile_global - t.tiles[it.s]) * kTile;
    it.npos = min(kTile, it.n - it.pos0);
    it.w_eff = min(w, it.n);
    it.pack = t.pack[it.s];
    return it;
}

template <typename T, int D>
__device__ inline void load_k_tile(GenericSmem<D> &sm, const refree_params &p, const T *k,
                                   const int32_t *seq_start, const Item &it)
{
    const T *base = k + (int64_t)it.s * p.k_stride_seq +
                    ((int64_t)seq_start[it.s] + it.pos0) * p.k_stride_tok +
                    (int64_t)it.g * p.k_stride_head;
    for (int e = threadIdx.x; e < it.npos * D; e += kThreads) {
        const int j = e / D, c = e % D;
        sm.k[j][c] = to_float(base[(int64_t)j * p.k_stride_tok + c]);
    }
}

// logit (log2 domain) of query row rr against the 4 positions this lane owns
template <typename T, int D>
__device__ inline void row_logits(GenericSmem<D> &sm, const refree_params &p, const T *q_win,
                                  const Item &it, int rr, float scale, float (&y)[4])
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.num_q_heads / p.num_kv_heads;
    const int hh = rr / it.w_eff, rloc = rr % it.w_eff;
    const int qpos = it.n - it.w_eff + rloc;
    const T *q = q_win + ((((int64_t)it.s * p.num_q_heads + it.g * G + hh) * p.window) +
                          (p.window - it.w_eff + rloc)) * D;
    __syncwarp();
    for (int c = lane; c < D; c += 32) sm.q[warp][c] = to_float(q[c]);
    __syncwarp();
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int j = lane + 32 * u;
        float acc = 0.f;
        if (j < it.npos && it.pos0 + j <= qpos) {
#pragma unroll 8
            for (int c = 0; c < D; ++c) acc = fmaf(sm.q[warp][c], sm.k[j][c], acc);
            y[u] = acc * scale;
        } else {
            y[u] = -INFINITY;
        }
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
score_stats_generic(refree_params p, const T *q_win, const T *k, const int32_t *seq_start,
                    const int32_t *seq_len, float2 *part)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    GenericSmem<D> &sm = *reinterpret_cast<GenericSmem<D> *>(smem_raw);
    const int B = p.num_seqs, Hkv = p.num_kv_heads;
    const int G = p.num_q_heads / Hkv, Rmax = G * p.window;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float scale = kLog2e / sqrtf((float)D);
    build_seq_tables(sm.seq, seq_len, B);
    const int items = sm.seq.tiles[B] * Hkv;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const Item it = decode_item(sm.seq, seq_len, B, Hkv, p.window, item);
        __syncthreads();
        load_k_tile<T, D>(sm, p, k, seq_start, it);
        __syncthreads();
        const int R = G * it.w_eff;
        for (int rr = warp; rr < R; rr += kWarps) {
            float y[4];
            row_logits<T, D>(sm, p, q_win, it, rr, scale, y);
            float m = fmaxf(fmaxf(y[0], y[1]), fmaxf(y[2], y[3]));
            for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            float z = 0.f;
            if (m > -INFINITY) {
#pragma unroll
                for (int u = 0; u < 4; ++u) z += exp2f(y[u] - m);
            }
            for (int o = 16; o; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
            if (lane == 0) part[((int64_t)it.tile_global * Hkv + it.g) * Rmax + rr] = make_float2(m, z);
        }
    }
}

__global__ void score_combine_generic(refree_params p, const int32_t *seq_len, const float2 *part,
                                      float *lse)
{
    __shared__ SeqTables seq;
    const int B = p.num_seqs, Hkv = p.num_kv_heads;
    const int Rmax = (p.num_q_heads / Hkv) * p.window;
    build_seq_tables(seq, seq_len, B);
    const int64_t total = (int64_t)B * Hkv * Rmax;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int rr = (int)(e % Rmax), u = (int)(e / Rmax);
        const int s = u / Hkv, g = u % Hkv;
        const int n = seq_len[s];
        const int R = (p.num_q_heads / Hkv) * min(p.window, n);
        if (rr >= R) continue;
        const int t0 = seq.tiles[s], t1 = seq.tiles[s + 1];
        float m = -INFINITY;
        for (int t = t0; t < t1; ++t) m = fmaxf(m, part[((int64_t)t * Hkv + g) * Rmax + rr].x);
        float z = 0.f;
        for (int t = t0; t < t1; ++t) {
            const float2 pr = part[((int64_t)t * Hkv + g) * Rmax + rr];
            if (pr.y > 0.f) z += pr.y * exp2f(pr.x - m);
        }
        lse[e] = m + log2f(z);
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
score_colsum_generic(refree_params p, const T *q_win, const T *k, const int32_t *seq_start,
                     const int32_t *seq_len, const float *lse, int64_t total_tokens, float *scores,
                     int32_t *dev_status)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    GenericSmem<D> &sm = *reinterpret_cast<GenericSmem<D> *>(smem_raw);
    const int B = p.num_seqs, Hkv = p.num_kv_heads;
    const int G = p.num_q_heads / Hkv, Rmax = G * p.window;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float scale = kLog2e / sqrtf((float)D);
    build_seq_tables(sm.seq, seq_len, B);
    const int items = sm.seq.tiles[B] * Hkv;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const Item it = decode_item(sm.seq, seq_len, B, Hkv, p.window, item);
        __syncthreads();
        load_k_tile<T, D>(sm, p, k, seq_start, it);
        __syncthreads();
        const int R = G * it.w_eff;
        const int u = it.s * Hkv + it.g;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int rr = warp; rr < R; rr += kWarps) {
            float y[4];
            row_logits<T, D>(sm, p, q_win, it, rr, scale, y);
            const float L = lse[(int64_t)u * Rmax + rr];
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[v] += exp2f(y[v] - L);   // 2^(-inf) = 0 for hidden positions
        }
#pragma unroll
        for (int v = 0; v < 4; ++v) sm.red[warp][lane + 32 * v] = acc[v];
        __syncthreads();
        if (threadIdx.x < it.npos) {
            const int j = threadIdx.x;
            float tot = 0.f;
#pragma unroll
            for (int wv = 0; wv < kWarps; ++wv) tot += sm.red[wv][j];
            const int cnt = min(it.w_eff, it.n - (it.pos0 + j));
            const float a = tot / (float)cnt / (float)G;
            if (!isfinite(a) && dev_status) atomicOr(dev_status, REFREE_DEV_NONFINITE);
            scores[(int64_t)it.g * total_tokens + it.pack + it.pos0 + j] = a;
        }
    }
}

template <typename T, int D>
cudaError_t run(const refree_params &p, const void *q_win, const void *k, const int32_t *seq_start,
                const int32_t *seq_len, int64_t total_tokens, float *scores, char *ws,
                const Workspace &lay, int32_t *dev_status, cudaStream_t st)
{
    const size_t smem = sizeof(GenericSmem<D>);
    cudaError_t e;
    e = cudaFuncSetAttribute(score_stats_generic<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(score_colsum_generic<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int64_t max_items = (total_tokens / kTile + p.num_seqs) * p.num_kv_heads;
    const int grid = (int)std::min<int64_t>(std::max<int64_t>(max_items, 1), sm_count() * 16);
    float2 *part = reinterpret_cast<float2 *>(ws + lay.part_off);
    float *lse = reinterpret_cast<float *>(ws + lay.lse_off);
    score_stats_generic<T, D><<<grid, kThreads, smem, st>>>(p, (const T *)q_win, (const T *)k, seq_start, seq_len, part);
    const int64_t rows = (int64_t)p.num_seqs * p.num_q_heads * p.window;
    score_combine_generic<<<(int)std::min<int64_t>((rows + 255) / 256, 1024), 256, 0, st>>>(p, seq_len, part, lse);
    score_colsum_generic<T, D><<<grid, kThreads, smem, st>>>(p, (const T *)q_win, (const T *)k, seq_start, seq_len,
                                                            lse, total_tokens, scores, dev_status);
    count_launches(3);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_score_generic(const refree_params &p, const void *q_win, const void *k,
                                 const int32_t *seq_start, const int32_t *seq_len,
                                 int64_t total_tokens, float *scores, char *ws, const Workspace &lay,
                                 int32_t *dev_status, cudaStream_t st)
{
    const bool f32 = p.dtype == REFREE_DTYPE_F32;
    if (p.head_dim == 64)
        return f32 ? run<float, 64>(p, q_win, k, seq_start, seq_len, total_tokens, scores, ws, lay, dev_status, st)
                   : run<__nv_bfloat16, 64>(p, q_win, k, seq_start, seq_len, total_tokens, scores, ws, lay, dev_status, st);
    return f32 ? run<float, 128>(p, q_win, k, seq_start, seq_len, total_tokens, scores, ws, lay, dev_status, st)
               : run<__nv_bfloat16, 128>(p, q_win, k, seq_start, seq_len, total_tokens, scores, ws, lay, dev_status, st);
}

}  // namespace refree
