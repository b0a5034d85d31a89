// Internal declarations shared by the kernels of the compression-pass library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "refreekv.h"

namespace refree {

constexpr int kMaxSeqs = 1024;   // sequences per call (prefix tables live in shared memory)
constexpr int kTile = 128;       // positions per scoring tile
constexpr int kMaxRows = 1024;   // G * window handled by the generic scoring path
// Longer windows (Section 4.4 studies windows of up to a tenth of the sequence) are scored in chunks of query rows
// that the scoring paths take, each chunk a window of its own over a sequence cut at its last row.
constexpr int kMaxRowsChunked = 32768;
constexpr int kMaxGroupChunked = 256;   // query heads per KV head when the window is chunked

// Bounded spin: polls before a wait gives up and reports REFREE_DEV_TIMEOUT.
constexpr uint32_t kSpinLimit = 1u << 22;
// The stopping rule fed by per-32-position records sums each group at a scale set by the group's own largest
// score and shifts the sums to the unit's scale, so it drops up to one unit of the fixed point per element and per
// group: about n * 2^(L - 54) of C_n with L = log2(groups), against n * 2^-60 for the rule that reads every score.
// That is 2^-29 at 32K positions and still 2^-25 at 128K, far inside the near-tie band; longer sequences take the
// rule that reads every score.
constexpr int64_t kGroupSelectMaxTokens = 131072;

// Layout of the caller-provided workspace.  All offsets are multiples of 256.
struct Workspace {
    size_t part_off, part_bytes;       // per (tile, head, row) softmax partials (float2: max, sum)
    size_t lse_off, lse_bytes;         // generic path: per (unit, row) log2-sum-exp of the row's logits
    size_t grp_off, grp_bytes;         // per 32 positions: exact partial sum of squared scores (GroupPartial)
    size_t cnt_off, cnt_bytes;         // per unit arrival counters (zeroed by each call)
    size_t cut_off, cut_bytes;         // per unit selection result (struct Cut)
    size_t scores_off, scores_bytes;   // scratch scores when the caller passes none
    size_t kept_off, kept_bytes;       // scratch kept_idx when the caller passes none
    size_t chk_off, chk_bytes;         // chunked windows: one chunk's query rows, its scores, its sequence lengths
    size_t total;
};

// Result of the stopping rule for one unit, enough to enumerate its kept set.
//   position ranking: kept = [0, min(b, lead)) U [n - (b - lead), n)
//   score ranking:    kept = the first min(b, lead + w_eff) protected positions in
//                     order (leading then window), plus unprotected positions whose
//                     key is above `tau`, plus the first `ties` (by position) whose
//                     key equals `tau`.
struct Cut {
    int32_t b;          // budget (kept count)
    int32_t ties;       // score ranking: number of positions with key == tau to keep
    uint64_t tau;       // score ranking: key threshold (score bits << 32, or the fixed-point layer key)
    int32_t prot_kept;  // score ranking: protected positions kept
    int32_t sbias;      // fixed-point exponent bias of the unit's squares (see select.cu)
};

// Sum of squared scores of 32 consecutive positions of one unit, written by the
// scoring kernel so that the stopping rule need not re-read every score.
//   max_bits  bit pattern of the largest score of the group (0 when all are zero)
//   sum       sum over the group of floor(a^2 * 2^(308 - 2E)), E = exponent field of
//             max_bits (at least 1): exact integer squares, at most 2^61 in total
// Records of unit (s, g) are contiguous: index (tiles[s] * Hkv + g * tiles_of(s)) * 4 + i / 32.
struct GroupPartial {
    uint32_t max_bits;
    uint32_t pad;
    unsigned long long sum;
};
constexpr int kGroupShift = 8;   // the squared mantissa (below 2^48) of the group's largest score lands below 2^56

Workspace workspace_layout(const refree_params &p, int64_t total_tokens);

// Bookkeeping for refree_kernel_launch_count(): every launcher adds the kernels it enqueued.
void count_launches(int n);

// Multiprocessors of the current device (looked up once per device; launch geometry is sized by it).
int sm_count();

inline __host__ __device__ int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Per-CTA tables: running sums of sequence lengths and of tiles per sequence.
struct SeqTables {
    int32_t pack[kMaxSeqs + 1];   // positions before sequence s in the packed score array
    int32_t tiles[kMaxSeqs + 1];  // scoring tiles before sequence s
    int32_t len[kMaxSeqs];        // copy of seq_len (clamped at 0)
};

__device__ inline void build_seq_tables(SeqTables &t, const int32_t *seq_len, int B)
{
    if (threadIdx.x == 0) {
        int32_t a = 0, b = 0;
        for (int s = 0; s < B; ++s) {
            t.pack[s] = a;
            t.tiles[s] = b;
            const int n = max(seq_len[s], 0);
            t.len[s] = n;
            a += n;
            b += ceil_div(n, kTile);
        }
        t.pack[B] = a;
        t.tiles[B] = b;
    }
    __syncthreads();
}

// Largest s with table[s] <= x (table ascending, table[0] == 0).
__device__ inline int find_seq(const int32_t *table, int B, int x)
{
    int lo = 0, hi = B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (table[mid] <= x) lo = mid; else hi = mid;
    }
    return lo;
}

// |a| as an integer: non-negative floats order like their bit patterns
__device__ inline uint32_t mag_bits(float a) { return __float_as_uint(a) & 0x7fffffffu; }

// floor(a^2 * 2^S) from the bits of |a|, where 2 * exponent_field + sbias is the left
// shift of the exact 48-bit squared mantissa (S = sbias + 300); non-finite values count as zero
__device__ inline unsigned long long sq_fixed(uint32_t bits, int sbias)
{
    const uint32_t e = bits >> 23;
    if (e == 255u) return 0ull;
    const uint32_t m = (bits & 0x7fffffu) | (e ? 0x800000u : 0u);
    const unsigned long long mm = (unsigned long long)m * m;     // exact, below 2^48
    const int sh = 2 * (int)(e ? e : 1u) + sbias;
    if (sh >= 0) return sh < 16 ? mm << sh : ~0ull >> 2;
    return -sh < 48 ? mm >> -sh : 0ull;
}

template <typename T> __device__ inline float to_float(T v);
template <> __device__ inline float to_float<float>(float v) { return v; }
template <> __device__ inline float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// ---- launchers (defined in the .cu files) ----------------------------------
cudaError_t launch_score_generic(const refree_params &p, const void *q_win, const void *k,
                                 const int32_t *seq_start, const int32_t *seq_len,
                                 int64_t total_tokens, float *scores, char *ws, const Workspace &lay,
                                 int32_t *dev_status, cudaStream_t st);

// Rows of another layer (position ranking: a prefix and a suffix per unit) that the tensor-core scoring
// kernel moves with a warp of its own while it scores, HBM being nearly idle then.  The budgets are read
// on the device; the kernel forms their running sum itself.
struct TcCopyJob {
    const unsigned char *k, *v;     // source cache (same strides and sequences as the scored layer)
    unsigned char *k_out, *v_out;   // dense outputs [capacity_rows, d]
    const int32_t *lengths;         // [num_seqs * num_kv_heads] budgets
    int64_t *offsets_out;           // nullable: [units + 1] running sum of the budgets
    int64_t capacity_rows;
    int nslots;                     // pieces in flight (0: nothing to move); set by the launcher
};

// Returns false when the shape is outside what the tensor-core path handles.
bool score_tc_supported(const refree_params &p);
// True when launch_score_tc can also carry a TcCopyJob for these parameters (rows of a unit contiguous in
// K and V, few enough units, shared memory left for the pieces in flight).
bool score_tc_can_copy(const refree_params &p, int64_t total_tokens);
// Both passes of one layer in one cooperative launch (two plain launches where that is not available).
cudaError_t launch_score_tc(const refree_params &p, const void *q_win, const void *k,
                            const int32_t *seq_start, const int32_t *seq_len,
                            int64_t total_tokens, float *scores, char *ws, const Workspace &lay,
                            int32_t *dev_status, cudaStream_t st, GroupPartial *groups = nullptr);

// One layer of a run of layers, as the scoring launches of the run see it.
struct TcLayer {
    const void *q_win, *k;
    float *scores;          // [Hkv, total_tokens]
    char *ws;               // the layer's workspace (partials between its two passes)
    GroupPartial *groups;   // nullable
    int32_t *sel_lengths;   // nullable: with `groups`, the launch that finishes the layer also evaluates the stopping
                            // rule (position ranking per head) and leaves the budgets here
};
// One launch of a run: the column pass of `finish`, then the row pass of `begin` (either may be null), and the
// rows of `copy` (nullable) moved beside them.  A launch clears the per-unit tile counts that the launch finishing
// its `begin` layer will use; `finish_tickets_clean` says an earlier launch of the run did that for this one.
cudaError_t launch_score_tc_pipe(const refree_params &p, const TcLayer *begin, const TcLayer *finish,
                                 const int32_t *seq_start, const int32_t *seq_len, int64_t total_tokens,
                                 const Workspace &lay, int32_t *dev_status, cudaStream_t st,
                                 const TcCopyJob *copy = nullptr, bool finish_tickets_clean = false);

// Single query row per head (the paper's default reduced attention): a stream over K on the fp32 pipes.
bool score_w1_supported(const refree_params &p);
size_t score_w1_scratch_bytes(const refree_params &p, int64_t total_tokens);
cudaError_t launch_score_w1(const refree_params &p, const void *q_win, const void *k,
                            const int32_t *seq_start, const int32_t *seq_len,
                            int64_t total_tokens, float *scores, char *ws, const Workspace &lay,
                            int32_t *dev_status, cudaStream_t st, GroupPartial *groups = nullptr);

cudaError_t launch_select(const refree_params &p, const float *scores, const int32_t *seq_len,
                          int64_t total_tokens, int32_t *lengths, int64_t *offsets,
                          int32_t *kept_idx, int64_t capacity_rows, char *ws, const Workspace &lay,
                          int32_t *dev_status, cudaStream_t st, bool emit = true,
                          const GroupPartial *groups = nullptr);

cudaError_t launch_compact(const refree_params &p, const void *k, const void *v,
                           const int32_t *seq_start, const int32_t *seq_len,
                           const int32_t *lengths, const int64_t *offsets, const int32_t *kept_idx,
                           bool position_ranges, int64_t *offsets_out, void *k_out, void *v_out,
                           int64_t capacity_rows, int32_t *dev_status, cudaStream_t st,
                           bool beside_scoring = false);

// With `lengths` and `offsets_out` (end-anchored form only) the kernel takes the budgets from `lengths` and
// writes their running sum itself, so the selection need not emit offsets first.
cudaError_t launch_compact_inplace(const refree_params &p, void *k, void *v, const int32_t *seq_start,
                                   const int32_t *seq_len, const int64_t *offsets, const int32_t *kept_idx,
                                   bool position_ranges, bool anchor_back, int32_t *dev_status, cudaStream_t st,
                                   const int32_t *lengths = nullptr, int64_t *offsets_out = nullptr);

cudaError_t launch_compact_paged(const refree_params &p, const void *k, const void *v, const int32_t *seq_start,
                                 const int32_t *seq_len, const int32_t *lengths, const int64_t *offsets,
                                 const int32_t *kept_idx, bool position_ranges, const int32_t *block_table,
                                 int max_blocks_per_unit, int block_rows, void *k_pool, void *v_pool,
                                 int64_t num_blocks, int32_t *dev_status, cudaStream_t st);

size_t decode_workspace_bytes(const refree_params &p, int64_t max_rows);
cudaError_t launch_decode_attention(const refree_params &p, const void *q_new, const void *k_c, const void *v_c,
                                    const int64_t *offsets, int64_t max_rows, float *out, void *workspace,
                                    int32_t *dev_status, cudaStream_t st, const int32_t *seq_start = nullptr,
                                    const int32_t *seq_len = nullptr, const int32_t *lengths = nullptr,
                                    bool anchor_back = false);

}  // namespace refree
