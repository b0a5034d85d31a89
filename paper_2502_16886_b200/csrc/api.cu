// C-ABI entry points: argument checks, workspace layout, launch sequences.
#include <string.h>

#include <algorithm>
#include <atomic>
#include <mutex>

#include "refree_internal.cuh"

namespace refree {

static std::atomic<long long> g_launches{0};
void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int sm_count()
{
    static std::mutex m;
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    std::lock_guard<std::mutex> lock(m);
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// Window rows scored at once: the whole window when a scoring path takes it, else a chunk that one does
// (512 query rows on the tensor-core path, 1024 on the generic one).
static int chunk_window(const refree_params &p)
{
    const int G = p.num_q_heads / p.num_kv_heads;
    if ((int64_t)G * p.window <= kMaxRows) return p.window;
    const int cap = (p.dtype == REFREE_DTYPE_BF16 && p.head_dim == 128) ? 512 : kMaxRows;
    return std::max(1, cap / G);
}

Workspace workspace_layout(const refree_params &p, int64_t total_tokens)
{
    Workspace w;
    const int64_t U = (int64_t)p.num_seqs * p.num_kv_heads;
    const int64_t G = p.num_q_heads / p.num_kv_heads;
    const int wc = chunk_window(p);
    const int64_t rows = G * wc;
    const int64_t tiles = total_tokens / kTile + p.num_seqs;
    size_t off = 0;
    // partials: per (tile, head, row) for the generic path, per (CTA + unit, column half, padded row) for the tensor-core path
    const int64_t rows_pad = (rows + kTile - 1) / kTile * kTile;
    const int64_t part_items = std::max<int64_t>(tiles * p.num_kv_heads * rows, 2 * (256 + U) * rows_pad);
    size_t part_bytes = (size_t)part_items * sizeof(float2);
    if (score_w1_supported(p)) part_bytes = std::max(part_bytes, score_w1_scratch_bytes(p, total_tokens));
    w.part_off = off;   w.part_bytes = align256(part_bytes);                                               off += w.part_bytes;
    w.lse_off = off;    w.lse_bytes = align256((size_t)(U * rows_pad) * sizeof(float));                    off += w.lse_bytes;
    w.grp_off = off;    w.grp_bytes = align256((size_t)(tiles * p.num_kv_heads * 4) * sizeof(GroupPartial));  off += w.grp_bytes;
    w.cnt_off = off;    w.cnt_bytes = align256((size_t)(2 * U + 256 + 8) * sizeof(int32_t));                         off += w.cnt_bytes;
    w.cut_off = off;    w.cut_bytes = align256((size_t)U * sizeof(Cut));                                   off += w.cut_bytes;
    w.scores_off = off; w.scores_bytes = align256((size_t)(p.num_kv_heads * total_tokens) * sizeof(float)); off += w.scores_bytes;
    w.kept_off = off;   w.kept_bytes = align256((size_t)(p.num_kv_heads * total_tokens) * sizeof(int32_t)); off += w.kept_bytes;
    w.chk_off = off;    w.chk_bytes = 0;
    if (wc < p.window) {
        const size_t esz = p.dtype == REFREE_DTYPE_F32 ? 4 : 2;
        w.chk_bytes = align256((size_t)p.num_seqs * p.num_q_heads * wc * p.head_dim * esz) +
                      align256((size_t)(p.num_kv_heads * total_tokens) * sizeof(float)) +
                      align256((size_t)p.num_seqs * sizeof(int32_t));
    }
    off += w.chk_bytes;
    w.total = off;
    return w;
}

static refree_status check_params(const refree_params *p, int64_t total_tokens)
{
    if (!p) return REFREE_ERR_INVALID_ARG;
    if (p->num_seqs < 1 || p->num_q_heads < 1 || p->num_kv_heads < 1) return REFREE_ERR_INVALID_ARG;
    if (p->num_q_heads % p->num_kv_heads != 0) return REFREE_ERR_INVALID_ARG;
    if (p->window < 1 || p->sink < 0) return REFREE_ERR_INVALID_ARG;
    if (!(p->threshold >= 0.0f && p->threshold < 1.0f)) return REFREE_ERR_INVALID_ARG;
    if (p->rank_mode != REFREE_RANK_POSITION && p->rank_mode != REFREE_RANK_SCORE) return REFREE_ERR_INVALID_ARG;
    if (p->scope != REFREE_SCOPE_HEAD && p->scope != REFREE_SCOPE_LAYER) return REFREE_ERR_INVALID_ARG;
    if (p->dtype != REFREE_DTYPE_F32 && p->dtype != REFREE_DTYPE_BF16) return REFREE_ERR_INVALID_ARG;
    if (total_tokens < 0 || total_tokens > 0x7fffffffLL - kTile) return REFREE_ERR_INVALID_ARG;
    if (p->head_dim != 64 && p->head_dim != 128) return REFREE_ERR_UNSUPPORTED;
    if (p->num_seqs > kMaxSeqs) return REFREE_ERR_UNSUPPORTED;
    if ((int64_t)p->num_seqs * p->num_kv_heads > 65535) return REFREE_ERR_UNSUPPORTED;
    if ((int64_t)(p->num_q_heads / p->num_kv_heads) * p->window > kMaxRows &&
        ((int64_t)(p->num_q_heads / p->num_kv_heads) * p->window > kMaxRowsChunked ||
         p->num_q_heads / p->num_kv_heads > kMaxGroupChunked))
        return REFREE_ERR_UNSUPPORTED;
    return REFREE_OK;
}

static refree_status check_kv_layout(const refree_params *p, const void *k, const void *v, bool need_v)
{
    const int esz = p->dtype == REFREE_DTYPE_F32 ? 4 : 2;
    if (p->kv_tokens < 0) return REFREE_ERR_INVALID_ARG;
    if (p->k_stride_tok < p->head_dim || p->k_stride_seq < 0 || p->k_stride_head < 0) return REFREE_ERR_INVALID_ARG;
    // 16-byte vector access to every row
    if ((reinterpret_cast<uintptr_t>(k) & 15) || (p->k_stride_tok * esz) % 16 || (p->k_stride_head * esz) % 16 ||
        (p->k_stride_seq * esz) % 16)
        return REFREE_ERR_UNSUPPORTED;
    if (need_v) {
        if (p->v_stride_tok < p->head_dim || p->v_stride_seq < 0 || p->v_stride_head < 0) return REFREE_ERR_INVALID_ARG;
        if ((reinterpret_cast<uintptr_t>(v) & 15) || (p->v_stride_tok * esz) % 16 || (p->v_stride_head * esz) % 16 ||
            (p->v_stride_seq * esz) % 16)
            return REFREE_ERR_UNSUPPORTED;
    }
    return REFREE_OK;
}

static refree_status from_cuda(cudaError_t e) { return e == cudaSuccess ? REFREE_OK : REFREE_ERR_CUDA; }

static bool use_tc(const refree_params &p, const void *q_win)
{
    return score_tc_supported(p) && !(reinterpret_cast<uintptr_t>(q_win) & 15);
}

namespace {
// Lengths of the sequences as a chunk of window rows sees them: cut after the chunk's last row.
__global__ void chunk_lens_kernel(const int32_t *seq_len, int32_t *len_c, int num_seqs, int rows_after)
{
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s < num_seqs) len_c[s] = max(0, max(seq_len[s], 0) - rows_after);
}

// scores += chunk scores * (chunk rows that see the position), i.e. the chunk's column sums over G; the last
// chunk divides by the rows of the whole window that see the position (Eq. 2).
__global__ void chunk_accumulate_kernel(refree_params p, const int32_t *seq_len, const int32_t *len_c, const float *sc,
                                        float *scores, int64_t total_tokens, int wc, int last)
{
    __shared__ int s_pack, s_pack_c;
    const int Hkv = p.num_kv_heads, s = blockIdx.y / Hkv, g = blockIdx.y % Hkv;
    if (threadIdx.x == 0) {
        int a = 0, b = 0;
        for (int t = 0; t < s; ++t) { a += max(seq_len[t], 0); b += len_c[t]; }
        s_pack = a;
        s_pack_c = b;
    }
    __syncthreads();
    const int n = max(seq_len[s], 0), nc = len_c[s];
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        float acc = scores[(int64_t)g * total_tokens + s_pack + i];
        if (i < nc) {
            const int cnt_c = max(1, min(min(wc, nc), nc - i));
            acc += sc[(int64_t)g * total_tokens + s_pack_c + i] * (float)cnt_c;
        }
        if (last) acc /= (float)max(1, min(min(p.window, n), n - i));
        scores[(int64_t)g * total_tokens + s_pack + i] = acc;
    }
}
}  // namespace

static cudaError_t run_score(const refree_params &p, const void *q_win, const void *k,
                             const int32_t *seq_start, const int32_t *seq_len, int64_t total_tokens,
                             float *scores, char *ws, const Workspace &lay, int32_t *dev_status,
                             cudaStream_t st, GroupPartial *groups = nullptr)
{
    const int wc = chunk_window(p);
    if (wc < p.window) {
        // Window too long for one pass: chunks of window rows from the last backwards, each scored as a window of
        // its own over the sequences cut at its last row (K is read again per chunk), then weighted back to column
        // sums and added up.  The chunks' scores are exact column sums up to one rounding each.
        const size_t esz = p.dtype == REFREE_DTYPE_F32 ? 4 : 2;
        const size_t row_bytes = (size_t)p.head_dim * esz;
        char *qc = ws + lay.chk_off;
        float *sc = reinterpret_cast<float *>(qc + align256((size_t)p.num_seqs * p.num_q_heads * wc * row_bytes));
        int32_t *len_c = reinterpret_cast<int32_t *>(reinterpret_cast<char *>(sc) +
                                                    align256((size_t)(p.num_kv_heads * total_tokens) * sizeof(float)));
        cudaError_t e = cudaMemsetAsync(scores, 0, (size_t)(p.num_kv_heads * total_tokens) * sizeof(float), st);
        if (e != cudaSuccess) return e;
        const int gx = (int)std::min<int64_t>(1024, (total_tokens + 255) / 256);
        for (int t1 = p.window; t1 > 0; t1 -= wc) {
            const int t0 = std::max(0, t1 - wc), wcur = t1 - t0;
            refree_params pc = p;
            pc.window = wcur;
            e = cudaMemcpy2DAsync(qc, (size_t)wcur * row_bytes, (const char *)q_win + (size_t)t0 * row_bytes,
                                  (size_t)p.window * row_bytes, (size_t)wcur * row_bytes,
                                  (size_t)p.num_seqs * p.num_q_heads, cudaMemcpyDeviceToDevice, st);
            if (e != cudaSuccess) return e;
            chunk_lens_kernel<<<(p.num_seqs + 255) / 256, 256, 0, st>>>(seq_len, len_c, p.num_seqs, p.window - t1);
            count_launches(1);
            e = run_score(pc, qc, k, seq_start, len_c, total_tokens, sc, ws, lay, dev_status, st, nullptr);
            if (e != cudaSuccess) return e;
            chunk_accumulate_kernel<<<dim3(gx, p.num_seqs * p.num_kv_heads), 256, 0, st>>>(p, seq_len, len_c, sc, scores,
                                                                                         total_tokens, wcur, t0 == 0);
            count_launches(1);
        }
        return cudaGetLastError();
    }
    if (use_tc(p, q_win))
        return launch_score_tc(p, q_win, k, seq_start, seq_len, total_tokens, scores, ws, lay, dev_status, st, groups);
    if (score_w1_supported(p))
        return launch_score_w1(p, q_win, k, seq_start, seq_len, total_tokens, scores, ws, lay, dev_status, st, groups);
    return launch_score_generic(p, q_win, k, seq_start, seq_len, total_tokens, scores, ws, lay, dev_status, st);
}

}  // namespace refree

using namespace refree;

extern "C" {

void refree_default_params(refree_params *p)
{
    if (!p) return;
    memset(p, 0, sizeof(*p));
    p->window = 1;
    p->sink = 4;
    p->threshold = 0.01f;
    p->rank_mode = REFREE_RANK_POSITION;
    p->scope = REFREE_SCOPE_HEAD;
    p->keep_window = 1;
    p->force_full = 0;
    p->dtype = REFREE_DTYPE_BF16;
}

int64_t refree_kernel_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

const char *refree_status_string(refree_status s)
{
    switch (s) {
    case REFREE_OK: return "ok";
    case REFREE_ERR_INVALID_ARG: return "invalid argument";
    case REFREE_ERR_UNSUPPORTED: return "unsupported shape, type or alignment";
    case REFREE_ERR_WORKSPACE: return "workspace missing or too small";
    case REFREE_ERR_CAPACITY: return "output capacity too small";
    case REFREE_ERR_CUDA: return "CUDA runtime error";
    case REFREE_ERR_TIMEOUT: return "a bounded on-device wait gave up";
    case REFREE_ERR_NONFINITE: return "non-finite score";
    case REFREE_ERR_STATIC_LIMIT: return "problem exceeds the built-in scratch of the no-allocation entry point";
    }
    return "unknown status";
}

refree_status refree_workspace_size(const refree_params *p, int64_t total_tokens, size_t *bytes)
{
    if (!bytes) return REFREE_ERR_INVALID_ARG;
    const refree_status st = check_params(p, total_tokens);
    if (st != REFREE_OK) return st;
    *bytes = workspace_layout(*p, total_tokens).total;
    return REFREE_OK;
}

refree_status refree_score(const refree_params *p, const void *q_win, const void *k,
                           const int32_t *seq_start, const int32_t *seq_len, int64_t total_tokens,
                           float *scores, void *workspace, size_t workspace_bytes,
                           int32_t *device_status, void *stream)
{
    refree_status st = check_params(p, total_tokens);
    if (st != REFREE_OK) return st;
    if (!q_win || !k || !seq_start || !seq_len || !scores) return REFREE_ERR_INVALID_ARG;
    st = check_kv_layout(p, k, nullptr, false);
    if (st != REFREE_OK) return st;
    const Workspace lay = workspace_layout(*p, total_tokens);
    if (!workspace || workspace_bytes < lay.total || (reinterpret_cast<uintptr_t>(workspace) & 255))
        return REFREE_ERR_WORKSPACE;
    if (total_tokens == 0) return REFREE_OK;
    return from_cuda(run_score(*p, q_win, k, seq_start, seq_len, total_tokens, scores, (char *)workspace, lay,
                               device_status, (cudaStream_t)stream));
}

refree_status refree_select_budget(const refree_params *p, const float *scores,
                                   const int32_t *seq_len, int64_t total_tokens,
                                   int32_t *lengths, int64_t *offsets,
                                   int32_t *kept_idx, int64_t capacity_rows,
                                   void *workspace, size_t workspace_bytes,
                                   int32_t *device_status, void *stream)
{
    const refree_status st = check_params(p, total_tokens);
    if (st != REFREE_OK) return st;
    if (!scores || !seq_len || !lengths || !offsets || capacity_rows < 0) return REFREE_ERR_INVALID_ARG;
    const Workspace lay = workspace_layout(*p, total_tokens);
    if (!workspace || workspace_bytes < lay.total || (reinterpret_cast<uintptr_t>(workspace) & 255))
        return REFREE_ERR_WORKSPACE;
    return from_cuda(launch_select(*p, scores, seq_len, total_tokens, lengths, offsets, kept_idx, capacity_rows,
                                   (char *)workspace, lay, device_status, (cudaStream_t)stream));
}

refree_status refree_compact(const refree_params *p, const void *k, const void *v,
                             const int32_t *seq_start, const int32_t *seq_len,
                             const int32_t *lengths, const int64_t *offsets,
                             const int32_t *kept_idx, void *k_out, void *v_out,
                             int64_t capacity_rows, int32_t *device_status, void *stream)
{
    refree_status st = check_params(p, 0);
    if (st != REFREE_OK) return st;
    if (!k || !v || !seq_start || !seq_len || !lengths || !offsets || !kept_idx || !k_out || !v_out ||
        capacity_rows < 0)
        return REFREE_ERR_INVALID_ARG;
    st = check_kv_layout(p, k, v, true);
    if (st != REFREE_OK) return st;
    if ((reinterpret_cast<uintptr_t>(k_out) & 15) || (reinterpret_cast<uintptr_t>(v_out) & 15))
        return REFREE_ERR_UNSUPPORTED;
    return from_cuda(launch_compact(*p, k, v, seq_start, seq_len, lengths, offsets, kept_idx, false, nullptr, k_out,
                                    v_out, capacity_rows, device_status, (cudaStream_t)stream));
}

refree_status refree_compact_paged(const refree_params *p, const void *k, const void *v,
                                   const int32_t *seq_start, const int32_t *seq_len,
                                   const int32_t *lengths, const int64_t *offsets, const int32_t *kept_idx,
                                   const int32_t *block_table, int32_t max_blocks_per_unit, int32_t block_rows,
                                   void *k_pool, void *v_pool, int64_t num_blocks,
                                   int32_t *device_status, void *stream)
{
    refree_status st = check_params(p, 0);
    if (st != REFREE_OK) return st;
    if (!k || !v || !seq_start || !seq_len || !lengths || !block_table || !k_pool || !v_pool ||
        max_blocks_per_unit < 1 || block_rows < 1 || num_blocks < 0)
        return REFREE_ERR_INVALID_ARG;
    const bool ranges = p->rank_mode == REFREE_RANK_POSITION || p->force_full;
    if (!ranges && (!kept_idx || !offsets)) return REFREE_ERR_INVALID_ARG;
    st = check_kv_layout(p, k, v, true);
    if (st != REFREE_OK) return st;
    if ((reinterpret_cast<uintptr_t>(k_pool) & 15) || (reinterpret_cast<uintptr_t>(v_pool) & 15))
        return REFREE_ERR_UNSUPPORTED;
    return from_cuda(launch_compact_paged(*p, k, v, seq_start, seq_len, lengths, offsets, ranges ? nullptr : kept_idx,
                                          ranges, block_table, max_blocks_per_unit, block_rows, k_pool, v_pool,
                                          num_blocks, device_status, (cudaStream_t)stream));
}

refree_status refree_compact_inplace(const refree_params *p, void *k, void *v,
                                     const int32_t *seq_start, const int32_t *seq_len,
                                     const int64_t *offsets, const int32_t *kept_idx, int32_t anchor,
                                     int32_t *device_status, void *stream)
{
    refree_status st = check_params(p, 0);
    if (st != REFREE_OK) return st;
    if (!k || !v || !seq_start || !seq_len || !offsets) return REFREE_ERR_INVALID_ARG;
    if (anchor != REFREE_ANCHOR_FRONT && anchor != REFREE_ANCHOR_BACK) return REFREE_ERR_INVALID_ARG;
    const bool ranges = p->rank_mode == REFREE_RANK_POSITION || p->force_full;
    if (!ranges && !kept_idx) return REFREE_ERR_INVALID_ARG;
    if (!ranges && anchor == REFREE_ANCHOR_BACK) return REFREE_ERR_UNSUPPORTED;
    st = check_kv_layout(p, k, v, true);
    if (st != REFREE_OK) return st;
    return from_cuda(launch_compact_inplace(*p, k, v, seq_start, seq_len, offsets, ranges ? nullptr : kept_idx, ranges,
                                            anchor == REFREE_ANCHOR_BACK, device_status, (cudaStream_t)stream));
}

static refree_status check_decode(const refree_params *p, int64_t max_rows)
{
    if (!p) return REFREE_ERR_INVALID_ARG;
    if (p->num_seqs < 1 || p->num_q_heads < 1 || p->num_kv_heads < 1) return REFREE_ERR_INVALID_ARG;
    if (p->num_q_heads % p->num_kv_heads != 0) return REFREE_ERR_INVALID_ARG;
    if (p->dtype != REFREE_DTYPE_F32 && p->dtype != REFREE_DTYPE_BF16) return REFREE_ERR_INVALID_ARG;
    if (max_rows < 0 || max_rows > 0x7fffffffLL - 4096) return REFREE_ERR_INVALID_ARG;
    if (p->head_dim != 64 && p->head_dim != 128) return REFREE_ERR_UNSUPPORTED;
    if ((int64_t)p->num_seqs * p->num_kv_heads > 65535) return REFREE_ERR_UNSUPPORTED;
    if (p->num_q_heads / p->num_kv_heads > 16) return REFREE_ERR_UNSUPPORTED;
    return REFREE_OK;
}

refree_status refree_decode_workspace_size(const refree_params *p, int64_t max_rows_per_unit, size_t *bytes)
{
    const refree_status st = check_decode(p, max_rows_per_unit);
    if (st != REFREE_OK) return st;
    if (!bytes) return REFREE_ERR_INVALID_ARG;
    *bytes = decode_workspace_bytes(*p, max_rows_per_unit);
    return REFREE_OK;
}

refree_status refree_decode_attention(const refree_params *p, const void *q_new,
                                      const void *k_c, const void *v_c, const int64_t *offsets,
                                      int64_t max_rows_per_unit, float *out,
                                      void *workspace, size_t workspace_bytes,
                                      int32_t *device_status, void *stream)
{
    const refree_status st = check_decode(p, max_rows_per_unit);
    if (st != REFREE_OK) return st;
    if (!q_new || !k_c || !v_c || !offsets || !out) return REFREE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(k_c) & 15) || (reinterpret_cast<uintptr_t>(v_c) & 15)) return REFREE_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < decode_workspace_bytes(*p, max_rows_per_unit) ||
        (reinterpret_cast<uintptr_t>(workspace) & 255))
        return REFREE_ERR_WORKSPACE;
    return from_cuda(launch_decode_attention(*p, q_new, k_c, v_c, offsets, max_rows_per_unit, out, workspace,
                                             device_status, (cudaStream_t)stream));
}

refree_status refree_decode_attention_inplace(const refree_params *p, const void *q_new,
                                              const void *k, const void *v,
                                              const int32_t *seq_start, const int32_t *seq_len,
                                              const int32_t *lengths, int32_t anchor,
                                              int64_t max_rows_per_unit, float *out,
                                              void *workspace, size_t workspace_bytes,
                                              int32_t *device_status, void *stream)
{
    refree_status st = check_decode(p, max_rows_per_unit);
    if (st != REFREE_OK) return st;
    if (!q_new || !k || !v || !seq_start || !seq_len || !lengths || !out) return REFREE_ERR_INVALID_ARG;
    if (anchor != REFREE_ANCHOR_FRONT && anchor != REFREE_ANCHOR_BACK) return REFREE_ERR_INVALID_ARG;
    st = check_kv_layout(p, k, v, true);
    if (st != REFREE_OK) return st;
    // the rows of a unit must be back to back, and every unit must start on a whole row
    const int64_t d = p->head_dim;
    if (p->k_stride_tok != d || p->v_stride_tok != d || p->k_stride_seq % d || p->k_stride_head % d ||
        p->v_stride_seq % d || p->v_stride_head % d)
        return REFREE_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < decode_workspace_bytes(*p, max_rows_per_unit) ||
        (reinterpret_cast<uintptr_t>(workspace) & 255))
        return REFREE_ERR_WORKSPACE;
    return from_cuda(launch_decode_attention(*p, q_new, k, v, nullptr, max_rows_per_unit, out, workspace, device_status,
                                             (cudaStream_t)stream, seq_start, seq_len, lengths,
                                             anchor == REFREE_ANCHOR_BACK));
}

// The launch sequence of one layer.  `cs` takes scoring and selection; compaction goes to `cc`
// (after `scored`, recorded on `cs`, when the two differ).
static refree_status enqueue_layer(const refree_params *p, const void *q_win, const void *k, const void *v,
                                   const int32_t *seq_start, const int32_t *seq_len, int64_t total_tokens,
                                   void *k_out, void *v_out, int64_t capacity_rows, int32_t *lengths,
                                   int64_t *offsets, int32_t *kept_idx, float *scores, char *ws,
                                   const Workspace &lay, int32_t *device_status, cudaStream_t cs,
                                   cudaStream_t cc, cudaEvent_t scored)
{
    float *sc = scores ? scores : reinterpret_cast<float *>(ws + lay.scores_off);
    const bool ranges = p->rank_mode == REFREE_RANK_POSITION || p->force_full;
    int32_t *kept = kept_idx ? kept_idx : (ranges ? nullptr : reinterpret_cast<int32_t *>(ws + lay.kept_off));
    cudaError_t e = cudaSuccess;
    // a frozen layer needs no scores unless the caller asked for them
    // position ranking per head on the tensor-core path: the scoring kernel also leaves the per-32-position
    // sums of squares, and the stopping rule reads those instead of every score
    GroupPartial *groups = nullptr;
    if ((use_tc(*p, q_win) || score_w1_supported(*p)) && p->rank_mode == REFREE_RANK_POSITION &&
        p->scope == REFREE_SCOPE_HEAD && !p->force_full && total_tokens > 0 && total_tokens <= kGroupSelectMaxTokens)
        groups = reinterpret_cast<GroupPartial *>(ws + lay.grp_off);
    if (total_tokens > 0 && (!p->force_full || scores))
        e = run_score(*p, q_win, k, seq_start, seq_len, total_tokens, sc, ws, lay, device_status, cs, groups);
    if (e != cudaSuccess) return REFREE_ERR_CUDA;
    // with two-range kept sets and no index list wanted, the compaction kernel forms the offsets itself
    const bool lean = ranges && !kept;
    e = launch_select(*p, sc, seq_len, total_tokens, lengths, offsets, kept, capacity_rows, ws, lay, device_status, cs,
                      !lean, groups);
    if (e != cudaSuccess) return REFREE_ERR_CUDA;
    const bool split = cc != cs;
    if (split) {
        if (cudaEventRecord(scored, cs) != cudaSuccess || cudaStreamWaitEvent(cc, scored, 0) != cudaSuccess)
            return REFREE_ERR_CUDA;
    }
    e = launch_compact(*p, k, v, seq_start, seq_len, lengths, offsets, kept, ranges, lean ? offsets : nullptr, k_out,
                       v_out, capacity_rows, device_status, cc, split && use_tc(*p, q_win));
    return from_cuda(e);
}

refree_status refree_compress_layer(const refree_params *p, const void *q_win,
                                    const void *k, const void *v,
                                    const int32_t *seq_start, const int32_t *seq_len,
                                    int64_t total_tokens,
                                    void *k_out, void *v_out, int64_t capacity_rows,
                                    int32_t *lengths, int64_t *offsets,
                                    int32_t *kept_idx, float *scores,
                                    void *workspace, size_t workspace_bytes,
                                    int32_t *device_status, void *stream)
{
    refree_status st = check_params(p, total_tokens);
    if (st != REFREE_OK) return st;
    if (!q_win || !k || !v || !seq_start || !seq_len || !k_out || !v_out || !lengths || !offsets ||
        capacity_rows < 0)
        return REFREE_ERR_INVALID_ARG;
    st = check_kv_layout(p, k, v, true);
    if (st != REFREE_OK) return st;
    if ((reinterpret_cast<uintptr_t>(k_out) & 15) || (reinterpret_cast<uintptr_t>(v_out) & 15))
        return REFREE_ERR_UNSUPPORTED;
    const Workspace lay = workspace_layout(*p, total_tokens);
    if (!workspace || workspace_bytes < lay.total || (reinterpret_cast<uintptr_t>(workspace) & 255))
        return REFREE_ERR_WORKSPACE;
    cudaStream_t cs = (cudaStream_t)stream;
    return enqueue_layer(p, q_win, k, v, seq_start, seq_len, total_tokens, k_out, v_out, capacity_rows, lengths,
                         offsets, kept_idx, scores, (char *)workspace, lay, device_status, cs, cs, nullptr);
}

refree_status refree_compress_layer_inplace(const refree_params *p, const void *q_win, void *k, void *v,
                                            const int32_t *seq_start, const int32_t *seq_len,
                                            int64_t total_tokens, int32_t *lengths, int64_t *offsets,
                                            int32_t anchor, void *workspace, size_t workspace_bytes,
                                            int32_t *device_status, void *stream)
{
    refree_status st = check_params(p, total_tokens);
    if (st != REFREE_OK) return st;
    if (!q_win || !k || !v || !seq_start || !seq_len || !lengths || !offsets) return REFREE_ERR_INVALID_ARG;
    if (anchor != REFREE_ANCHOR_FRONT && anchor != REFREE_ANCHOR_BACK) return REFREE_ERR_INVALID_ARG;
    const bool ranges = p->rank_mode == REFREE_RANK_POSITION || p->force_full;
    if (!ranges && anchor == REFREE_ANCHOR_BACK) return REFREE_ERR_UNSUPPORTED;
    st = check_kv_layout(p, k, v, true);
    if (st != REFREE_OK) return st;
    const Workspace lay = workspace_layout(*p, total_tokens);
    if (!workspace || workspace_bytes < lay.total || (reinterpret_cast<uintptr_t>(workspace) & 255))
        return REFREE_ERR_WORKSPACE;
    char *ws = (char *)workspace;
    cudaStream_t cs = (cudaStream_t)stream;
    float *sc = reinterpret_cast<float *>(ws + lay.scores_off);
    int32_t *kept = ranges ? nullptr : reinterpret_cast<int32_t *>(ws + lay.kept_off);
    GroupPartial *groups = nullptr;
    if ((use_tc(*p, q_win) || score_w1_supported(*p)) && p->rank_mode == REFREE_RANK_POSITION &&
        p->scope == REFREE_SCOPE_HEAD && !p->force_full && total_tokens > 0 && total_tokens <= kGroupSelectMaxTokens)
        groups = reinterpret_cast<GroupPartial *>(ws + lay.grp_off);
    cudaError_t e = cudaSuccess;
    if (total_tokens > 0 && !p->force_full)
        e = run_score(*p, q_win, k, seq_start, seq_len, total_tokens, sc, ws, lay, device_status, cs, groups);
    if (e != cudaSuccess) return REFREE_ERR_CUDA;
    // the end-anchored kernel forms the offsets itself: no emit launch
    const bool lean = anchor == REFREE_ANCHOR_BACK;
    e = launch_select(*p, sc, seq_len, total_tokens, lengths, offsets, kept, (int64_t)p->num_kv_heads * total_tokens, ws,
                      lay, device_status, cs, !lean, groups);
    if (e != cudaSuccess) return REFREE_ERR_CUDA;
    return from_cuda(launch_compact_inplace(*p, k, v, seq_start, seq_len, offsets, kept, ranges, lean, device_status, cs,
                                            lean ? lengths : nullptr, lean ? offsets : nullptr));
}

// ---- a run of device-resident layers, compaction of layer l under the scoring of layer l + 1 ----
namespace {
struct LayerPipe {
    bool ready = false;
    cudaStream_t hi = nullptr, lo = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr, scored[2] = {nullptr, nullptr}, compacted[2] = {nullptr, nullptr};
};
std::mutex g_pipe_mutex;
LayerPipe g_pipe[64];

// Streams and events of the current device, made on first use and kept until the process exits.
LayerPipe *layer_pipe()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    LayerPipe &lp = g_pipe[dev];
    if (lp.ready) return &lp;
    int least = 0, greatest = 0;
    if (cudaDeviceGetStreamPriorityRange(&least, &greatest) != cudaSuccess) return nullptr;
    bool ok = cudaStreamCreateWithPriority(&lp.hi, cudaStreamNonBlocking, greatest) == cudaSuccess &&
              cudaStreamCreateWithPriority(&lp.lo, cudaStreamNonBlocking, least) == cudaSuccess &&
              cudaEventCreateWithFlags(&lp.fork, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&lp.join, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i)
        ok = cudaEventCreateWithFlags(&lp.scored[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&lp.compacted[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return nullptr;
    lp.ready = true;
    return &lp;
}
}  // namespace

refree_status refree_layers_workspace_size(const refree_params *p, int64_t total_tokens, size_t *bytes)
{
    const refree_status st = refree_workspace_size(p, total_tokens, bytes);
    if (st == REFREE_OK) *bytes *= 2;
    return st;
}

refree_status refree_compress_layers(const refree_params *p, int32_t num_layers,
                                     const void *const *q_win, const void *const *k, const void *const *v,
                                     const int32_t *seq_start, const int32_t *seq_len, int64_t total_tokens,
                                     void *const *k_out, void *const *v_out, int64_t capacity_rows,
                                     int32_t *const *lengths, int64_t *const *offsets,
                                     void *workspace, size_t workspace_bytes,
                                     int32_t *device_status, void *stream)
{
    refree_status st = check_params(p, total_tokens);
    if (st != REFREE_OK) return st;
    if (num_layers < 0 || !q_win || !k || !v || !seq_start || !seq_len || !k_out || !v_out || !lengths || !offsets ||
        capacity_rows < 0)
        return REFREE_ERR_INVALID_ARG;
    for (int l = 0; l < num_layers; ++l) {
        if (!q_win[l] || !k[l] || !v[l] || !k_out[l] || !v_out[l] || !lengths[l] || !offsets[l])
            return REFREE_ERR_INVALID_ARG;
        st = check_kv_layout(p, k[l], v[l], true);
        if (st != REFREE_OK) return st;
        if ((reinterpret_cast<uintptr_t>(k_out[l]) & 15) || (reinterpret_cast<uintptr_t>(v_out[l]) & 15))
            return REFREE_ERR_UNSUPPORTED;
    }
    const Workspace lay = workspace_layout(*p, total_tokens);
    if (!workspace || workspace_bytes < 2 * lay.total || (reinterpret_cast<uintptr_t>(workspace) & 255))
        return REFREE_ERR_WORKSPACE;
    if (num_layers == 0) return REFREE_OK;
    // Position ranking on the tensor-core path with rows of a unit contiguous: one stream, the scoring kernel
    // of layer l moves the kept rows of layer l - 1 with a warp of its own, the last layer is compacted by a
    // launch of its own.  No internal streams or events.
    bool fused = num_layers >= 2 && total_tokens > 0 && !p->force_full && p->rank_mode == REFREE_RANK_POSITION &&
                 score_tc_can_copy(*p, total_tokens);
    for (int l = 0; l < num_layers && fused; ++l) fused = use_tc(*p, q_win[l]);
    if (fused) {
        // launch j (0 <= j <= L): column pass and stopping rule of layer j - 1, row pass of layer j, rows of
        // layer j - 2; then the last two layers' rows
        cudaStream_t cs = (cudaStream_t)stream;
        auto layer_of = [&](int l) {
            TcLayer t;
            char *ws = (char *)workspace + (size_t)(l & 1) * lay.total;
            t.q_win = q_win[l];
            t.k = k[l];
            t.ws = ws;
            t.scores = reinterpret_cast<float *>(ws + lay.scores_off);
            t.groups = p->scope == REFREE_SCOPE_HEAD && total_tokens <= kGroupSelectMaxTokens
                           ? reinterpret_cast<GroupPartial *>(ws + lay.grp_off) : nullptr;
            t.sel_lengths = t.groups ? lengths[l] : nullptr;      // the rule runs inside the launch that finishes the layer
            return t;
        };
        auto job_of = [&](int l) {
            TcCopyJob job;
            job.k = (const unsigned char *)k[l];
            job.v = (const unsigned char *)v[l];
            job.k_out = (unsigned char *)k_out[l];
            job.v_out = (unsigned char *)v_out[l];
            job.lengths = lengths[l];
            job.offsets_out = offsets[l];
            job.capacity_rows = capacity_rows;
            job.nslots = 0;
            return job;
        };
        for (int j = 0; j <= num_layers; ++j) {
            TcLayer beg, fin;
            TcCopyJob job;
            if (j < num_layers) beg = layer_of(j);
            if (j >= 1) fin = layer_of(j - 1);
            if (j >= 2) job = job_of(j - 2);
            if (launch_score_tc_pipe(*p, j < num_layers ? &beg : nullptr, j >= 1 ? &fin : nullptr, seq_start, seq_len,
                                     total_tokens, lay, device_status, cs, j >= 2 ? &job : nullptr, true) != cudaSuccess)
                return REFREE_ERR_CUDA;
            if (j >= 1 && !fin.sel_lengths &&
                launch_select(*p, fin.scores, seq_len, total_tokens, lengths[j - 1], offsets[j - 1], nullptr, capacity_rows,
                              fin.ws, lay, device_status, cs, false, fin.groups) != cudaSuccess)
                return REFREE_ERR_CUDA;
        }
        // the rows of the last layer; those of the one before it went with the last scoring launch
        const int l = num_layers - 1;
        return from_cuda(launch_compact(*p, k[l], v[l], seq_start, seq_len, lengths[l], offsets[l], nullptr, true,
                                        offsets[l], k_out[l], v_out[l], capacity_rows, device_status, cs));
    }
    LayerPipe *lp = layer_pipe();
    if (!lp) return REFREE_ERR_CUDA;
    cudaStream_t cs = (cudaStream_t)stream;
    bool ok = cudaEventRecord(lp->fork, cs) == cudaSuccess && cudaStreamWaitEvent(lp->hi, lp->fork, 0) == cudaSuccess &&
              cudaStreamWaitEvent(lp->lo, lp->fork, 0) == cudaSuccess;
    refree_status result = ok ? REFREE_OK : REFREE_ERR_CUDA;
    for (int l = 0; l < num_layers && result == REFREE_OK; ++l) {
        const int slot = l & 1;
        // the half of the workspace is free once the compaction of layer l - 2 has read its budgets
        if (l >= 2 && cudaStreamWaitEvent(lp->hi, lp->compacted[slot], 0) != cudaSuccess) { result = REFREE_ERR_CUDA; break; }
        result = enqueue_layer(p, q_win[l], k[l], v[l], seq_start, seq_len, total_tokens, k_out[l], v_out[l],
                               capacity_rows, lengths[l], offsets[l], nullptr, nullptr,
                               (char *)workspace + (size_t)slot * lay.total, lay, device_status, lp->hi, lp->lo,
                               lp->scored[slot]);
        if (result != REFREE_OK) break;
        if (cudaEventRecord(lp->compacted[slot], lp->lo) != cudaSuccess) { result = REFREE_ERR_CUDA; break; }
    }
    // the caller's stream continues after everything that was enqueued, whatever happened
    if (ok) {
        if (cudaEventRecord(lp->join, lp->hi) != cudaSuccess || cudaStreamWaitEvent(cs, lp->join, 0) != cudaSuccess ||
            cudaEventRecord(lp->join, lp->lo) != cudaSuccess || cudaStreamWaitEvent(cs, lp->join, 0) != cudaSuccess)
            if (result == REFREE_OK) result = REFREE_ERR_CUDA;
    }
    return result;
}

refree_status refree_host_arena_size(const refree_params *p, int64_t total_tokens,
                                     int64_t kv_elems, int64_t capacity_rows, size_t *bytes)
{
    if (!bytes || kv_elems < 0 || capacity_rows < 0) return REFREE_ERR_INVALID_ARG;
    const refree_status st = check_params(p, total_tokens);
    if (st != REFREE_OK) return st;
    const size_t esz = p->dtype == REFREE_DTYPE_F32 ? 4 : 2;
    const size_t U = (size_t)p->num_seqs * p->num_kv_heads;
    size_t tot = 0;
    tot += align256((size_t)p->num_seqs * p->num_q_heads * p->window * p->head_dim * esz);  // q_win
    tot += 2 * align256((size_t)kv_elems * esz);                                            // k, v
    tot += 2 * align256((size_t)p->num_seqs * sizeof(int32_t));                             // seq_start, seq_len
    tot += 2 * align256((size_t)capacity_rows * p->head_dim * esz);                         // k_out, v_out
    tot += align256(U * sizeof(int32_t)) + align256((U + 1) * sizeof(int64_t));             // lengths, offsets
    tot += align256((size_t)capacity_rows * sizeof(int32_t));                               // kept_idx
    tot += align256((size_t)p->num_kv_heads * total_tokens * sizeof(float));                // scores
    tot += align256(sizeof(int32_t));                                                       // device status
    tot += workspace_layout(*p, total_tokens).total;
    *bytes = tot;
    return REFREE_OK;
}

refree_status refree_compress_layer_host(const refree_params *p, const void *q_win,
                                         const void *k, const void *v, int64_t kv_elems,
                                         const int32_t *seq_start, const int32_t *seq_len,
                                         int64_t total_tokens,
                                         void *k_out, void *v_out, int64_t capacity_rows,
                                         int32_t *lengths, int64_t *offsets,
                                         int32_t *kept_idx, float *scores,
                                         void *arena, size_t arena_bytes, void *stream)
{
    size_t need = 0;
    refree_status st = refree_host_arena_size(p, total_tokens, kv_elems, capacity_rows, &need);
    if (st != REFREE_OK) return st;
    if (!q_win || !k || !v || !seq_start || !seq_len || !k_out || !v_out || !lengths || !offsets)
        return REFREE_ERR_INVALID_ARG;
    if (!arena || arena_bytes < need || (reinterpret_cast<uintptr_t>(arena) & 255)) return REFREE_ERR_WORKSPACE;
    cudaStream_t cs = (cudaStream_t)stream;
    const size_t esz = p->dtype == REFREE_DTYPE_F32 ? 4 : 2;
    const size_t U = (size_t)p->num_seqs * p->num_kv_heads;
    char *a = (char *)arena;
    auto take = [&](size_t bytes) { char *r = a; a += align256(bytes); return r; };
    const size_t q_bytes = (size_t)p->num_seqs * p->num_q_heads * p->window * p->head_dim * esz;
    const size_t kv_bytes = (size_t)kv_elems * esz;
    const size_t row_bytes = (size_t)p->head_dim * esz;
    char *d_q = take(q_bytes), *d_k = take(kv_bytes), *d_v = take(kv_bytes);
    int32_t *d_start = (int32_t *)take(p->num_seqs * sizeof(int32_t));
    int32_t *d_len = (int32_t *)take(p->num_seqs * sizeof(int32_t));
    char *d_ko = take(capacity_rows * row_bytes), *d_vo = take(capacity_rows * row_bytes);
    int32_t *d_lengths = (int32_t *)take(U * sizeof(int32_t));
    int64_t *d_offsets = (int64_t *)take((U + 1) * sizeof(int64_t));
    int32_t *d_kept = (int32_t *)take((size_t)capacity_rows * sizeof(int32_t));
    float *d_scores = (float *)take((size_t)p->num_kv_heads * total_tokens * sizeof(float));
    int32_t *d_status = (int32_t *)take(sizeof(int32_t));
    char *d_ws = a;
    const size_t ws_bytes = workspace_layout(*p, total_tokens).total;

    cudaError_t e;
    if ((e = cudaMemcpyAsync(d_q, q_win, q_bytes, cudaMemcpyHostToDevice, cs)) != cudaSuccess) return REFREE_ERR_CUDA;
    if ((e = cudaMemcpyAsync(d_k, k, kv_bytes, cudaMemcpyHostToDevice, cs)) != cudaSuccess) return REFREE_ERR_CUDA;
    if ((e = cudaMemcpyAsync(d_v, v, kv_bytes, cudaMemcpyHostToDevice, cs)) != cudaSuccess) return REFREE_ERR_CUDA;
    if ((e = cudaMemcpyAsync(d_start, seq_start, p->num_seqs * sizeof(int32_t), cudaMemcpyHostToDevice, cs)) != cudaSuccess) return REFREE_ERR_CUDA;
    if ((e = cudaMemcpyAsync(d_len, seq_len, p->num_seqs * sizeof(int32_t), cudaMemcpyHostToDevice, cs)) != cudaSuccess) return REFREE_ERR_CUDA;
    if ((e = cudaMemsetAsync(d_status, 0, sizeof(int32_t), cs)) != cudaSuccess) return REFREE_ERR_CUDA;
    st = refree_compress_layer(p, d_q, d_k, d_v, d_start, d_len, total_tokens, d_ko, d_vo, capacity_rows,
                               d_lengths, d_offsets, kept_idx ? d_kept : nullptr, scores ? d_scores : nullptr,
                               d_ws, ws_bytes, d_status, stream);
    if (st != REFREE_OK) return st;
    int32_t h_status = 0;
    cudaMemcpyAsync(lengths, d_lengths, U * sizeof(int32_t), cudaMemcpyDeviceToHost, cs);
    cudaMemcpyAsync(offsets, d_offsets, (U + 1) * sizeof(int64_t), cudaMemcpyDeviceToHost, cs);
    cudaMemcpyAsync(&h_status, d_status, sizeof(int32_t), cudaMemcpyDeviceToHost, cs);
    if ((e = cudaStreamSynchronize(cs)) != cudaSuccess) return REFREE_ERR_CUDA;
    if (h_status & REFREE_DEV_TIMEOUT) return REFREE_ERR_TIMEOUT;
    if (h_status & REFREE_DEV_CAPACITY) return REFREE_ERR_CAPACITY;
    if (h_status & REFREE_DEV_NONFINITE) return REFREE_ERR_NONFINITE;
    const int64_t rows = offsets[U];
    cudaMemcpyAsync(k_out, d_ko, (size_t)rows * row_bytes, cudaMemcpyDeviceToHost, cs);
    cudaMemcpyAsync(v_out, d_vo, (size_t)rows * row_bytes, cudaMemcpyDeviceToHost, cs);
    if (kept_idx) cudaMemcpyAsync(kept_idx, d_kept, (size_t)rows * sizeof(int32_t), cudaMemcpyDeviceToHost, cs);
    if (scores)
        cudaMemcpyAsync(scores, d_scores, (size_t)p->num_kv_heads * total_tokens * sizeof(float), cudaMemcpyDeviceToHost, cs);
    return from_cuda(cudaStreamSynchronize(cs));
}

}  // extern "C"
