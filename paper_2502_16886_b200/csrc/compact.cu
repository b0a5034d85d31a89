// Step S7: gather the kept K and V rows of every unit into the dense ragged
// output (Algorithm 1, "Compress" steps).  Pure data movement: 16-byte vector
// loads and stores, several rows in flight per thread.  Rows are copied bit for
// bit.  With position ranking the kept set is two contiguous ranges, so the
// source row follows from (b, m, n) and no index list is read.
#include <mutex>
#include <cooperative_groups.h>

#include <algorithm>

#include "refree_internal.cuh"

namespace refree {
namespace {

constexpr int kThreads = 256;
constexpr int kThreadsSlim = 128;   // block that fits beside a resident scoring CTA (see launch_compact)
constexpr int kUnroll = 4;

__device__ inline int4 ld_stream(const int4 *p)
{
    int4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ inline void st_stream(int4 *p, const int4 &v)
{
    asm volatile("st.global.cs.v4.s32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

template <int kThreads>
__global__ void __launch_bounds__(kThreads)
compact_kernel(refree_params p, const char *k, const char *v, const int32_t *seq_start,
               const int32_t *seq_len, const int32_t *lengths, const int64_t *offsets,
               const int32_t *kept_idx, int position_ranges, int64_t *offsets_out, char *k_out, char *v_out,
               int64_t capacity_rows, int32_t *dev_status)
{
    __shared__ long long s_part[kThreads / 32];
    const int Hkv = p.num_kv_heads;
    const int u = blockIdx.y, s = u / Hkv, g = u % Hkv;
    const int esz = p.dtype == REFREE_DTYPE_F32 ? 4 : 2;
    const int row_bytes = p.head_dim * esz;
    const int vec_per_row = row_bytes >> 4;
    const int vshift = 31 - __clz(vec_per_row);
    const int n = max(seq_len[s], 0);
    const int b = lengths[u];
    int64_t off;
    if (offsets_out) {
        // fused pass: the running sum of the budgets is formed here instead of in a launch of its own
        long long part = 0;
        for (int t = threadIdx.x; t < u; t += kThreads) part += lengths[t];
        for (int o = 16; o; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
        if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = part;
        __syncthreads();
        off = 0;
        for (int wv = 0; wv < kThreads / 32; ++wv) off += s_part[wv];
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            offsets_out[u] = off;
            if (u == (int)gridDim.y - 1) offsets_out[u + 1] = off + b;
        }
    } else {
        off = offsets[u];
    }
    if (b < 0 || b > n || off < 0 || off + b > capacity_rows) {
        if (threadIdx.x == 0 && blockIdx.x == 0 && dev_status) atomicOr(dev_status, REFREE_DEV_CAPACITY);
        return;
    }
    const int head = min(b, min(p.sink, n));
    const int64_t tok0 = seq_start[s];
    const char *kb = k + ((int64_t)s * p.k_stride_seq + tok0 * p.k_stride_tok + (int64_t)g * p.k_stride_head) * esz;
    const char *vb = v + ((int64_t)s * p.v_stride_seq + tok0 * p.v_stride_tok + (int64_t)g * p.v_stride_head) * esz;
    const int64_t k_tok = p.k_stride_tok * esz, v_tok = p.v_stride_tok * esz;
    char *ko = k_out + off * row_bytes, *vo = v_out + off * row_bytes;
    const int32_t *idx = kept_idx ? kept_idx + off : nullptr;
    const int64_t nvec = (int64_t)b << vshift;
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    for (int64_t e0 = (int64_t)blockIdx.x * kThreads + threadIdx.x; e0 < nvec; e0 += stride * kUnroll) {
        int4 kv[kUnroll], vv[kUnroll];
        bool good[kUnroll];
#pragma unroll
        for (int r = 0; r < kUnroll; ++r) {
            const int64_t e = e0 + r * stride;
            good[r] = false;
            if (e < nvec) {
                const int t = (int)(e >> vshift), c = (int)(e & (vec_per_row - 1));
                const int src = position_ranges ? (t < head ? t : n - b + t) : idx[t];
                // an index list is the caller's: a row outside the sequence is reported, never read
                good[r] = src >= 0 && src < n;
                if (good[r]) {
                    kv[r] = *reinterpret_cast<const int4 *>(kb + (int64_t)src * k_tok + c * 16);
                    vv[r] = ld_stream(reinterpret_cast<const int4 *>(vb + (int64_t)src * v_tok + c * 16));
                } else if (dev_status) {
                    atomicOr(dev_status, REFREE_DEV_CAPACITY);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < kUnroll; ++r) {
            const int64_t e = e0 + r * stride;
            if (e < nvec && good[r]) {
                st_stream(reinterpret_cast<int4 *>(ko + e * 16), kv[r]);
                st_stream(reinterpret_cast<int4 *>(vo + e * 16), vv[r]);
            }
        }
    }
}


// In-place form of the same step.  Every kept row moves towards the front of its own unit
// (destination index t <= source index), so rows can be overwritten as soon as whoever
// needs their old contents has read them.  The kept rows of all units, in order, are cut
// into rounds of as many 16-byte pieces as the grid holds in registers; in a round every
// thread loads its pieces, the grid synchronises, and every thread stores them.  A round
// reads only rows at or beyond its own destinations, which lie beyond every destination of
// the rounds before it, so one grid barrier per round is all the ordering needed.
constexpr int kUnrollInplace = 4;
constexpr int kInplaceTable = 1024;   // running sums held in shared memory (8 KB)

__global__ void __launch_bounds__(kThreads, 4)
compact_inplace_kernel(refree_params p, char *k, char *v, const int32_t *seq_start, const int32_t *seq_len,
                       const int64_t *offsets, const int32_t *kept_idx, int position_ranges, int32_t *dev_status)
{
    namespace cg = cooperative_groups;
    cg::grid_group grid = cg::this_grid();
    const int Hkv = p.num_kv_heads, U = p.num_seqs * Hkv;
    const int esz = p.dtype == REFREE_DTYPE_F32 ? 4 : 2;
    const int vec_per_row = (p.head_dim * esz) >> 4;
    const int vshift = 31 - __clz(vec_per_row);
    // the running sums are searched once per piece: keep them in shared memory when they fit
    __shared__ int64_t s_off[kInplaceTable];
    const int64_t *tab = offsets;
    if (U + 1 <= kInplaceTable) {
        for (int i = threadIdx.x; i <= U; i += kThreads) s_off[i] = __ldg(offsets + i);
        __syncthreads();
        tab = s_off;
    }
    const int64_t total_vec = max((long long)tab[U], 0ll) << vshift;
    const int64_t lanes = (int64_t)gridDim.x * kThreads;
    const int64_t per_round = lanes * kUnrollInplace;
    const int64_t k_tok = p.k_stride_tok * esz, v_tok = p.v_stride_tok * esz;
    bool bad = false;
    for (int64_t base = 0; base < total_vec; base += per_round) {     // the same trip count in every thread
        int4 kv[kUnrollInplace], vv[kUnrollInplace];
        char *kd[kUnrollInplace], *vd[kUnrollInplace];
#pragma unroll
        for (int r = 0; r < kUnrollInplace; ++r) {
            kd[r] = vd[r] = nullptr;
            const int64_t e = base + r * lanes + (int64_t)blockIdx.x * kThreads + threadIdx.x;
            if (e >= total_vec) continue;
            const int64_t row = e >> vshift;
            const int c = (int)(e & (vec_per_row - 1));
            int lo = 0, hi = U;                                       // unit whose rows contain `row`
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (tab[mid] <= row) lo = mid; else hi = mid;
            }
            const int u = lo, s = u / Hkv, g = u % Hkv;
            const int64_t off = tab[u];
            const int n = max(__ldg(seq_len + s), 0);
            const int64_t b64 = tab[u + 1] - off;
            const int t = (int)(row - off);
            if (off < 0 || b64 < 0 || b64 > n) { bad = true; continue; }
            const int b = (int)b64;
            const int head = min(b, min(p.sink, n));
            const int src = position_ranges ? (t < head ? t : n - b + t) : __ldg(kept_idx + row);
            if (src < t || src >= n) { bad = true; continue; }
            if (src == t) continue;                                   // already in place
            const int64_t tok0 = __ldg(seq_start + s);
            char *kb = k + ((int64_t)s * p.k_stride_seq + tok0 * p.k_stride_tok + (int64_t)g * p.k_stride_head) * esz + c * 16;
            char *vb = v + ((int64_t)s * p.v_stride_seq + tok0 * p.v_stride_tok + (int64_t)g * p.v_stride_head) * esz + c * 16;
            kv[r] = __ldcg(reinterpret_cast<const int4 *>(kb + (int64_t)src * k_tok));
            vv[r] = __ldcg(reinterpret_cast<const int4 *>(vb + (int64_t)src * v_tok));
            kd[r] = kb + (int64_t)t * k_tok;
            vd[r] = vb + (int64_t)t * v_tok;
        }
        grid.sync();
#pragma unroll
        for (int r = 0; r < kUnrollInplace; ++r) {
            if (kd[r]) {
                *reinterpret_cast<int4 *>(kd[r]) = kv[r];
                *reinterpret_cast<int4 *>(vd[r]) = vv[r];
            }
        }
    }
    if (bad && dev_status) atomicOr(dev_status, REFREE_DEV_CAPACITY);
}

// In place, anchored at the END of every unit's region (position ranking only): the kept set is
// the `head` leading rows plus the suffix [n - (b - head), n), so it is enough to lift the leading
// rows to just below the suffix; the compacted cache of the unit is then rows [n - b, n) of its
// own region.  At most `sink` rows move per unit.  The move is upwards and may overlap itself
// (n - b < head), so the rows go in blocks of 256 pieces from the top down, each block loaded by
// all threads before any of it is stored; a block's destinations lie above everything that the
// blocks after it still have to read.
__global__ void __launch_bounds__(kThreads)
compact_inplace_back_kernel(refree_params p, char *k, char *v, const int32_t *seq_start, const int32_t *seq_len,
                            const int64_t *offsets, const int32_t *lengths, int64_t *offsets_out, int32_t *dev_status)
{
    __shared__ long long s_part[kThreads / 32];
    const int Hkv = p.num_kv_heads;
    const int u = blockIdx.x, s = u / Hkv, g = u % Hkv;
    const int esz = p.dtype == REFREE_DTYPE_F32 ? 4 : 2;
    const int vec_per_row = (p.head_dim * esz) >> 4;
    const int vshift = 31 - __clz(vec_per_row);
    const int n = max(seq_len[s], 0);
    int64_t off, b64;
    if (lengths) {
        // fused pass: budgets come straight from the selection, and the running sum is formed here
        long long part = 0;
        for (int t = threadIdx.x; t < u; t += kThreads) part += lengths[t];
        for (int o = 16; o; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
        if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = part;
        __syncthreads();
        off = 0;
        for (int wv = 0; wv < kThreads / 32; ++wv) off += s_part[wv];
        b64 = lengths[u];
        if (threadIdx.x == 0) {
            offsets_out[u] = off;
            if (u == (int)gridDim.x - 1) offsets_out[u + 1] = off + b64;
        }
    } else {
        off = offsets[u];
        b64 = offsets[u + 1] - off;
    }
    if (off < 0 || b64 < 0 || b64 > n) {
        if (threadIdx.x == 0 && dev_status) atomicOr(dev_status, REFREE_DEV_CAPACITY);
        return;
    }
    const int b = (int)b64, head = min(b, min(p.sink, n)), shift = n - b;
    if (shift == 0 || head == 0) return;
    const int64_t tok0 = seq_start[s];
    char *kb = k + ((int64_t)s * p.k_stride_seq + tok0 * p.k_stride_tok + (int64_t)g * p.k_stride_head) * esz;
    char *vb = v + ((int64_t)s * p.v_stride_seq + tok0 * p.v_stride_tok + (int64_t)g * p.v_stride_head) * esz;
    const int64_t k_tok = p.k_stride_tok * esz, v_tok = p.v_stride_tok * esz;
    const int total_vec = head << vshift;
    for (int c0 = (total_vec - 1) / kThreads * kThreads; c0 >= 0; c0 -= kThreads) {
        const int e = c0 + threadIdx.x;
        const bool on = e < total_vec;
        const int row = e >> vshift, c = e & (vec_per_row - 1);
        int4 kv = {}, vv = {};
        if (on) {
            kv = __ldcg(reinterpret_cast<const int4 *>(kb + (int64_t)row * k_tok + c * 16));
            vv = __ldcg(reinterpret_cast<const int4 *>(vb + (int64_t)row * v_tok + c * 16));
        }
        __syncthreads();
        if (on) {
            *reinterpret_cast<int4 *>(kb + (int64_t)(row + shift) * k_tok + c * 16) = kv;
            *reinterpret_cast<int4 *>(vb + (int64_t)(row + shift) * v_tok + c * 16) = vv;
        }
    }
}

// Paged form of the same step: row t of unit u goes to row t % block_rows of the block
// block_table[u][t / block_rows] of a pool of fixed-size blocks (the layout of a paged
// serving cache).  Same gather as compact_kernel; only the destination address differs.
__global__ void __launch_bounds__(kThreads)
compact_paged_kernel(refree_params p, const char *k, const char *v, const int32_t *seq_start,
                     const int32_t *seq_len, const int32_t *lengths, const int64_t *offsets,
                     const int32_t *kept_idx, int position_ranges, const int32_t *block_table,
                     int max_blocks_per_unit, int block_rows, char *k_pool, char *v_pool, int64_t num_blocks,
                     int32_t *dev_status)
{
    const int Hkv = p.num_kv_heads;
    const int u = blockIdx.y, s = u / Hkv, g = u % Hkv;
    const int esz = p.dtype == REFREE_DTYPE_F32 ? 4 : 2;
    const int row_bytes = p.head_dim * esz;
    const int vec_per_row = row_bytes >> 4;
    const int vshift = 31 - __clz(vec_per_row);
    const int n = max(seq_len[s], 0);
    const int b = lengths[u];
    if (b < 0 || b > n || (int64_t)b > (int64_t)max_blocks_per_unit * block_rows || (kept_idx && offsets[u] < 0)) {
        if (threadIdx.x == 0 && blockIdx.x == 0 && dev_status) atomicOr(dev_status, REFREE_DEV_CAPACITY);
        return;
    }
    const int head = min(b, min(p.sink, n));
    const int64_t tok0 = seq_start[s];
    const char *kb = k + ((int64_t)s * p.k_stride_seq + tok0 * p.k_stride_tok + (int64_t)g * p.k_stride_head) * esz;
    const char *vb = v + ((int64_t)s * p.v_stride_seq + tok0 * p.v_stride_tok + (int64_t)g * p.v_stride_head) * esz;
    const int64_t k_tok = p.k_stride_tok * esz, v_tok = p.v_stride_tok * esz;
    const int32_t *idx = kept_idx ? kept_idx + offsets[u] : nullptr;
    const int32_t *table = block_table + (int64_t)u * max_blocks_per_unit;
    const int64_t nvec = (int64_t)b << vshift;
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    bool bad = false;
    for (int64_t e0 = (int64_t)blockIdx.x * kThreads + threadIdx.x; e0 < nvec; e0 += stride * kUnroll) {
        int4 kv[kUnroll], vv[kUnroll];
        int64_t dst[kUnroll];
#pragma unroll
        for (int r = 0; r < kUnroll; ++r) {
            const int64_t e = e0 + r * stride;
            dst[r] = -1;
            if (e < nvec) {
                const int t = (int)(e >> vshift), c = (int)(e & (vec_per_row - 1));
                const int src = position_ranges ? (t < head ? t : n - b + t) : idx[t];
                const int blk = __ldg(table + t / block_rows);
                if (blk < 0 || blk >= num_blocks || src < 0 || src >= n) { bad = true; continue; }
                kv[r] = *reinterpret_cast<const int4 *>(kb + (int64_t)src * k_tok + c * 16);
                vv[r] = ld_stream(reinterpret_cast<const int4 *>(vb + (int64_t)src * v_tok + c * 16));
                dst[r] = ((int64_t)blk * block_rows + t % block_rows) * row_bytes + c * 16;
            }
        }
#pragma unroll
        for (int r = 0; r < kUnroll; ++r) {
            if (dst[r] >= 0) {
                st_stream(reinterpret_cast<int4 *>(k_pool + dst[r]), kv[r]);
                st_stream(reinterpret_cast<int4 *>(v_pool + dst[r]), vv[r]);
            }
        }
    }
    if (bad && dev_status) atomicOr(dev_status, REFREE_DEV_CAPACITY);
}

}  // namespace

cudaError_t launch_compact(const refree_params &p, const void *k, const void *v,
                           const int32_t *seq_start, const int32_t *seq_len,
                           const int32_t *lengths, const int64_t *offsets, const int32_t *kept_idx,
                           bool position_ranges, int64_t *offsets_out, void *k_out, void *v_out,
                           int64_t capacity_rows, int32_t *dev_status, cudaStream_t st, bool beside_scoring)
{
    const int U = p.num_seqs * p.num_kv_heads;
    if (beside_scoring) {
        // The launch shares the SMs with a persistent scoring CTA of the next layer (576 threads, 96
        // registers each): 10 240 registers are left per SM, so the block is 128 threads (8 192
        // registers), and the grid is many short-lived blocks, so that a scoring CTA that becomes
        // runnable finds room as soon as a few of them retire.
        const int gx = max(1, (sm_count() * 32) / U);
        compact_kernel<kThreadsSlim><<<dim3(gx, U), kThreadsSlim, 0, st>>>(
            p, (const char *)k, (const char *)v, seq_start, seq_len, lengths, offsets, kept_idx,
            position_ranges ? 1 : 0, offsets_out, (char *)k_out, (char *)v_out, capacity_rows, dev_status);
        count_launches(1);
        return cudaGetLastError();
    }
    const int gx = max(1, (sm_count() * 8) / U);
    compact_kernel<kThreads><<<dim3(gx, U), kThreads, 0, st>>>(p, (const char *)k, (const char *)v, seq_start, seq_len,
                                                     lengths, offsets, kept_idx, position_ranges ? 1 : 0, offsets_out,
                                                     (char *)k_out, (char *)v_out, capacity_rows, dev_status);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_compact_inplace(const refree_params &p, void *k, void *v, const int32_t *seq_start,
                                   const int32_t *seq_len, const int64_t *offsets, const int32_t *kept_idx,
                                   bool position_ranges, bool anchor_back, int32_t *dev_status, cudaStream_t st,
                                   const int32_t *lengths, int64_t *offsets_out)
{
    if (anchor_back) {
        compact_inplace_back_kernel<<<p.num_seqs * p.num_kv_heads, kThreads, 0, st>>>(
            p, (char *)k, (char *)v, seq_start, seq_len, offsets, lengths, offsets_out, dev_status);
        count_launches(1);
        return cudaGetLastError();
    }
    static std::mutex grid_mutex;                 // the per-device grid size is looked up once, under a lock
    static int grid_blocks[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::unique_lock<std::mutex> hold(grid_mutex);
    if (grid_blocks[dev] == 0) {
        // every block of the grid must be resident at once: the rounds end in a grid-wide barrier
        int sms = 0, per_sm = 0, coop = 0;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev)) != cudaSuccess) return e;
        if (!coop) return cudaErrorNotSupported;
        if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, compact_inplace_kernel, kThreads, 0)) != cudaSuccess)
            return e;
        if (per_sm < 1) return cudaErrorLaunchOutOfResources;
        grid_blocks[dev] = sms * std::min(per_sm, 4);
    }
    const int grid = grid_blocks[dev];
    hold.unlock();
    refree_params pv = p;
    char *kc = (char *)k, *vc = (char *)v;
    int ranges = position_ranges ? 1 : 0;
    void *args[9] = {&pv, &kc, &vc, &seq_start, &seq_len, &offsets, &kept_idx, &ranges, &dev_status};
    e = cudaLaunchCooperativeKernel((const void *)compact_inplace_kernel, dim3(grid), dim3(kThreads), args, 0, st);
    if (e != cudaSuccess) return e;
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_compact_paged(const refree_params &p, const void *k, const void *v, const int32_t *seq_start,
                                 const int32_t *seq_len, const int32_t *lengths, const int64_t *offsets,
                                 const int32_t *kept_idx, bool position_ranges, const int32_t *block_table,
                                 int max_blocks_per_unit, int block_rows, void *k_pool, void *v_pool,
                                 int64_t num_blocks, int32_t *dev_status, cudaStream_t st)
{
    const int U = p.num_seqs * p.num_kv_heads;
    const int gx = max(1, (sm_count() * 8) / U);
    compact_paged_kernel<<<dim3(gx, U), kThreads, 0, st>>>(p, (const char *)k, (const char *)v, seq_start, seq_len,
                                                           lengths, offsets, kept_idx, position_ranges ? 1 : 0,
                                                           block_table, max_blocks_per_unit, block_rows,
                                                           (char *)k_pool, (char *)v_pool, num_blocks, dev_status);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace refree
