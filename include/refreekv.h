/*
 * refreekv.h - C ABI of the B200 (sm_100a) post-prefill KV-cache compression
 * pass of ReFreeKV (arXiv 2502.16886).
 *
 * For every (sequence s, KV head g) of one Transformer layer the pass
 *   (a) scores each cached position by the softmax attention it receives from
 *       the last `window` queries of the prompt (the reduced attention vector
 *       A' of Section 3.2, Eq. 2, averaged over the query heads of the KV head),
 *   (b) ranks the positions (Section 3.2 "Initial Ranking", or by score as in
 *       Section 4.4) and applies the threshold-free stopping rule (Eq. 1, in
 *       its cumulative form Eq. 3) to choose a budget b,
 *   (c) copies the kept K and V rows, in their original order, into a dense
 *       ragged cache (the "Compress" steps of Algorithm 1).
 *
 * Conventions common to every entry point
 *   - All array arguments are DEVICE pointers owned by the caller unless the
 *     function name ends in `_host`.  The library allocates no device memory
 *     and never synchronises the device (except the `_host` variants, which
 *     also create and destroy streams and events per call), and enqueues its
 *     work on the caller's stream (`stream` is a cudaStream_t passed as void*).
 *     refree_compress_layers may, for shapes outside its one-stream path, use
 *     two internal streams and a few events that are made once per device and
 *     kept until the process exits; they fork from and join the caller's stream.
 *   - The first call of an entry point on a device sets kernel attributes and
 *     reads device properties; make it outside any stream capture.
 *   - Limits, all reported as REFREE_ERR_UNSUPPORTED: num_seqs <= 1024;
 *     num_seqs * num_kv_heads <= 65535; (num_q_heads / num_kv_heads) * window
 *     <= 32768 with at most 256 query heads per KV head (beyond 1024 query rows
 *     per unit the window is scored in chunks of rows, K read once per chunk,
 *     and the workspace holds one chunk's rows and scores more); head_dim 64 or
 *     128; 16-byte aligned K/V base pointers and strides.
 *   - Element (s, g, i, :) of K lives at
 *       k + s*k_stride_seq + (seq_start[s] + i)*k_stride_tok + g*k_stride_head
 *     (strides in elements, head_dim contiguous); V likewise.  Rows
 *     [0, kv_tokens) of the token axis must be readable for every (s, g).
 *   - q_win is [num_seqs, num_q_heads, window, head_dim] contiguous;
 *     q_win[s, h, r, :] is the query at position seq_len[s] - window + r; rows
 *     with a negative position are ignored.
 *   - Per-position arrays (scores) are [num_kv_heads, total_tokens], sequences
 *     packed along the token axis by the running sum of seq_len;
 *     total_tokens = sum of seq_len.
 *   - Unit u = s*num_kv_heads + g owns rows [offsets[u], offsets[u+1]) of
 *     k_out / v_out / kept_idx; lengths[u] = offsets[u+1] - offsets[u].
 *   - The return value reports errors the host can see (bad arguments,
 *     unsupported shapes, workspace too small, CUDA launch failures); nothing
 *     is launched when it is not REFREE_OK.  Conditions only the device can
 *     see are OR-ed into *device_status (nullable, int32, caller zeroes it):
 *       REFREE_DEV_CAPACITY  output rows would exceed capacity_rows (nothing is
 *                            written past capacity)
 *       REFREE_DEV_TIMEOUT   a bounded on-device wait gave up
 *       REFREE_DEV_NONFINITE a score was NaN or infinite
 */
#ifndef REFREEKV_H
#define REFREEKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    REFREE_OK = 0,
    REFREE_ERR_INVALID_ARG = 1,
    REFREE_ERR_UNSUPPORTED = 2,
    REFREE_ERR_WORKSPACE = 3,
    REFREE_ERR_CAPACITY = 4,
    REFREE_ERR_CUDA = 5,
    REFREE_ERR_TIMEOUT = 6,
    REFREE_ERR_NONFINITE = 7,
    REFREE_ERR_STATIC_LIMIT = 8  /* problem too large for the built-in scratch of a *_static entry point */
} refree_status;

enum { REFREE_DEV_CAPACITY = 1, REFREE_DEV_TIMEOUT = 2, REFREE_DEV_NONFINITE = 4 };

enum { REFREE_RANK_POSITION = 0, REFREE_RANK_SCORE = 1 };
enum { REFREE_SCOPE_HEAD = 0, REFREE_SCOPE_LAYER = 1 };
enum { REFREE_DTYPE_F32 = 0, REFREE_DTYPE_BF16 = 1 };

typedef struct {
    int32_t num_seqs, num_q_heads, num_kv_heads, head_dim; /* Hq % Hkv == 0; head_dim 64 or 128 */
    int32_t window;      /* w >= 1: trailing query rows, the paper's k (default 1, Section 4.1)   */
    int32_t sink;        /* m >= 0: leading positions ranked first (default 4, Section 4.1)       */
    float   threshold;   /* T in [0, 1): universal threshold of Eq. 1 (default 0.01, Section 3.2) */
    int32_t rank_mode;   /* REFREE_RANK_POSITION (Section 3.2) or REFREE_RANK_SCORE (Section 4.4) */
    int32_t scope;       /* one budget per (sequence, KV head), or one per sequence for the layer */
    int32_t keep_window; /* 1: budget never below min(n, m + min(w, n))                          */
    int32_t force_full;  /* 1: keep everything (the frozen bottom layers of Section 3.3)          */
    int32_t dtype;       /* REFREE_DTYPE_*: type of q_win, K, V and of k_out, v_out               */
    int64_t kv_tokens;   /* readable extent of the token axis of K and V                          */
    int64_t k_stride_seq, k_stride_tok, k_stride_head;
    int64_t v_stride_seq, v_stride_tok, v_stride_head;
} refree_params;

/* Defaults of the paper (Section 3.2, Section 4.1): w = 1, m = 4, T = 1 %,
 * position ranking, per-head budgets, window floor on, bf16.  Shapes and
 * strides are left zero for the caller to fill. */
void refree_default_params(refree_params *p);

/* Bytes of device scratch that score / select / compress_layer need for this
 * shape.  `bytes` (host pointer) receives the size; pass a buffer at least
 * that large, 256-byte aligned, as `workspace`.  Contents need no
 * initialisation and are not preserved between calls. */
refree_status refree_workspace_size(const refree_params *p, int64_t total_tokens, size_t *bytes);

/* Steps S1-S3: reduced attention A' (Eq. 2) of every position, for every KV
 * head, from the causal softmax of the window queries (Algorithm 1,
 * "Attention" step; Section 3.2 "Reducing Overhead").
 *   scores [num_kv_heads, total_tokens] fp32, written in full. */
refree_status refree_score(const refree_params *p, const void *q_win, const void *k,
                           const int32_t *seq_start, const int32_t *seq_len, int64_t total_tokens,
                           float *scores, void *workspace, size_t workspace_bytes,
                           int32_t *device_status, void *stream);

/* Steps S4-S6: rank the positions, evaluate the stopping rule (Eq. 1 / Eq. 3;
 * Algorithm 1 Square .. Where) over the exact squares of the fp32 scores: the
 * 48-bit squared mantissas are summed as integers in a per-unit fixed point
 * (order-independent, so budgets are deterministic) and the crossing level
 * (1 - T)^2 C_n is evaluated once in fp64; then apply the window floor and emit
 * the kept set in ascending position order.
 *   lengths  [num_seqs * num_kv_heads] int32
 *   offsets  [num_seqs * num_kv_heads + 1] int64, running sum of lengths
 *   kept_idx [capacity_rows] int32 positions within their sequence (nullable:
 *            then only lengths and offsets are produced) */
refree_status refree_select_budget(const refree_params *p, const float *scores,
                                   const int32_t *seq_len, int64_t total_tokens,
                                   int32_t *lengths, int64_t *offsets,
                                   int32_t *kept_idx, int64_t capacity_rows,
                                   void *workspace, size_t workspace_bytes,
                                   int32_t *device_status, void *stream);

/* Step S7: K_c[offsets[u] + t, :] = K[s, kept_idx[offsets[u] + t], g, :], the
 * same for V; rows are copied bit for bit (Algorithm 1 "Compress" steps).
 *   k_out, v_out [capacity_rows, head_dim], must not overlap K or V. */
refree_status refree_compact(const refree_params *p, const void *k, const void *v,
                             const int32_t *seq_start, const int32_t *seq_len,
                             const int32_t *lengths, const int64_t *offsets,
                             const int32_t *kept_idx, void *k_out, void *v_out,
                             int64_t capacity_rows, int32_t *device_status, void *stream);

/* Step S7 into a paged cache (Section 3.3 batches sequences whose budgets
 * differ; a paged serving cache holds such ragged lengths in fixed-size blocks).
 * Row t of unit u = s*num_kv_heads + g, i.e. the row refree_compact would write
 * to k_out[offsets[u] + t], goes to
 *     k_pool[block_table[u * max_blocks_per_unit + t / block_rows], t % block_rows, :]
 * and the same for V; rows are copied bit for bit.
 *   lengths      [num_seqs*num_kv_heads] int32 budgets (device, in)
 *   offsets, kept_idx  as produced by refree_select_budget; both ignored (may be
 *                null) with position ranking or force_full, required with score ranking
 *   block_table  [num_seqs*num_kv_heads, max_blocks_per_unit] int32 block numbers
 *                (device, in); the caller assigns ceil(n / block_rows) blocks per
 *                unit before the call (the budgets are only known on the device)
 *                and can release those beyond ceil(lengths[u] / block_rows) later
 *   k_pool, v_pool  [num_blocks, block_rows, head_dim], params->dtype, 16-byte
 *                aligned (device, out); must not overlap K or V
 * A budget above max_blocks_per_unit * block_rows or the sequence length, or a
 * block number outside [0, num_blocks), sets REFREE_DEV_CAPACITY in
 * *device_status; the rows concerned are not written. */
refree_status refree_compact_paged(const refree_params *p, const void *k, const void *v,
                                   const int32_t *seq_start, const int32_t *seq_len,
                                   const int32_t *lengths, const int64_t *offsets, const int32_t *kept_idx,
                                   const int32_t *block_table, int32_t max_blocks_per_unit, int32_t block_rows,
                                   void *k_pool, void *v_pool, int64_t num_blocks,
                                   int32_t *device_status, void *stream);

/* Step S7 in place, for callers with no room for a second copy of the cache.
 * The kept rows of every unit end up contiguous inside the unit's OWN region of
 * K and V (same strides as the input), bit for bit the rows refree_compact would
 * have written to k_out / v_out, in the same order.  With b = offsets[u+1] -
 * offsets[u] and n the sequence length:
 *   REFREE_ANCHOR_FRONT  rows [0, b) of the unit hold its compacted cache:
 *       K[s, t, g, :] <- K[s, kept(u, t), g, :] for t < b.  Position ranking
 *       (Section 3.2 "Initial Ranking") keeps the leading positions and a suffix,
 *       so the leading rows stay and the suffix slides down behind them; with
 *       score ranking the kept rows (ascending kept_idx) slide down the same way.
 *       Every kept row is read and written once.
 *   REFREE_ANCHOR_BACK   rows [n - b, n) of the unit hold its compacted cache.
 *       Position ranking (or force_full) only: the suffix is already in place, so
 *       only the leading rows (at most `sink` per unit) are lifted to just below
 *       it - a few KB per unit instead of the whole kept cache - and rows that
 *       decoding appends at n, n + 1, .. stay contiguous with it.  Score ranking
 *       returns REFREE_ERR_UNSUPPORTED.
 * Rows outside the stated range keep stale contents.  The cache stays a strided
 * ragged array addressed by (seq_start, strides, per-unit length); it is not the
 * dense [sum b, head_dim] array that refree_decode_attention reads.
 *   k, v      device, read and written
 *   offsets   [num_seqs*num_kv_heads + 1] int64, as produced by refree_select_budget
 *   kept_idx  as produced by refree_select_budget; ignored (may be null) with
 *             position ranking or force_full, required with score ranking
 * Uses no scratch memory.  The FRONT kernel ends each round of copies with a
 * grid-wide barrier and is therefore launched cooperatively (all its blocks
 * resident); REFREE_ERR_CUDA is returned where the device cannot do that.
 * Budgets outside [0, n] or sources outside [t, n) set REFREE_DEV_CAPACITY in
 * *device_status and those pieces are skipped. */
#define REFREE_ANCHOR_FRONT 0
#define REFREE_ANCHOR_BACK 1
refree_status refree_compact_inplace(const refree_params *p, void *k, void *v,
                                     const int32_t *seq_start, const int32_t *seq_len,
                                     const int64_t *offsets, const int32_t *kept_idx, int32_t anchor,
                                     int32_t *device_status, void *stream);

/* The whole per-layer pass of Algorithm 1 (everything after the prefill of the
 * layer): score -> select -> compact, enqueued back to back with no host
 * synchronisation.  kept_idx and scores are nullable (scratch is used then).
 * Worst-case capacity_rows is num_kv_heads * total_tokens. */
refree_status refree_compress_layer(const refree_params *p, const void *q_win,
                                    const void *k, const void *v,
                                    const int32_t *seq_start, const int32_t *seq_len,
                                    int64_t total_tokens,
                                    void *k_out, void *v_out, int64_t capacity_rows,
                                    int32_t *lengths, int64_t *offsets,
                                    int32_t *kept_idx, float *scores,
                                    void *workspace, size_t workspace_bytes,
                                    int32_t *device_status, void *stream);

/* The whole per-layer pass with the compaction done in place: score -> select
 * -> refree_compact_inplace, enqueued back to back on `stream`.  k and v are
 * read by the scoring and then rewritten; lengths and offsets are outputs as in
 * refree_compress_layer; `anchor` and the resulting layout are those of
 * refree_compact_inplace (REFREE_ANCHOR_BACK needs position ranking or
 * force_full).  With position ranking and REFREE_ANCHOR_BACK the pass costs
 * little more than its scoring stage.  workspace as for refree_compress_layer. */
refree_status refree_compress_layer_inplace(const refree_params *p, const void *q_win, void *k, void *v,
                                            const int32_t *seq_start, const int32_t *seq_len,
                                            int64_t total_tokens, int32_t *lengths, int64_t *offsets,
                                            int32_t anchor, void *workspace, size_t workspace_bytes,
                                            int32_t *device_status, void *stream);

/* The pass of Algorithm 1 for a run of `num_layers` device-resident layers that
 * share one shape (Section 3.3: the cache of every layer is compressed once,
 * after prefill).  Scoring is bound by the tensor pipes and compaction by HBM,
 * so the run is software-pipelined over two internal streams: layer l + 1 is
 * scored and its budgets chosen while the kept rows of layer l are copied.
 * Results are bit-identical to num_layers calls of refree_compress_layer.
 *   q_win, k, v, k_out, v_out, lengths, offsets  HOST arrays of `num_layers`
 *            DEVICE pointers, one per layer, each as in refree_compress_layer;
 *            the arrays themselves are read before the call returns
 *   seq_start, seq_len, total_tokens, capacity_rows  common to all layers (device
 *            pointers as in refree_compress_layer)
 *   workspace  refree_layers_workspace_size() bytes (two per-layer workspaces),
 *            256-byte aligned, device
 * Index lists and scores are not returned (use the per-layer call for them).
 * Nothing is allocated in device memory and the host is not synchronised: the
 * work is ordered after what `stream` holds at the call, and `stream` continues
 * only when every layer is done.  The first call on a device creates the two
 * internal streams (highest priority for scoring, lowest for compaction) and
 * their events, which live until the process exits; the device that owns
 * `stream` must be the current device of the calling thread.  Calls from
 * several host threads on one device share the internal streams and are
 * serialised by stream order. */
refree_status refree_layers_workspace_size(const refree_params *p, int64_t total_tokens, size_t *bytes);
refree_status refree_compress_layers(const refree_params *p, int32_t num_layers,
                                     const void *const *q_win, const void *const *k, const void *const *v,
                                     const int32_t *seq_start, const int32_t *seq_len, int64_t total_tokens,
                                     void *const *k_out, void *const *v_out, int64_t capacity_rows,
                                     int32_t *const *lengths, int64_t *const *offsets,
                                     void *workspace, size_t workspace_bytes,
                                     int32_t *device_status, void *stream);

/* The same pass of Algorithm 1 for callers whose cache lives in HOST memory
 * (pinned or pageable): q_win, k, v, seq_start, seq_len are host pointers, and
 * so are the outputs k_out, v_out (capacity_rows rows), lengths, offsets,
 * kept_idx (nullable) and scores (nullable).  k and v are read over `kv_elems`
 * elements each (the size of the caller's arrays).  `arena` is a DEVICE buffer
 * of at least refree_host_arena_size() bytes that stages inputs, outputs and
 * scratch; the call copies in, runs the pass, copies the kept rows back and
 * synchronises `stream` before returning.  Device-side conditions are
 * returned as REFREE_ERR_CAPACITY / _TIMEOUT / _NONFINITE. */
refree_status refree_host_arena_size(const refree_params *p, int64_t total_tokens,
                                     int64_t kv_elems, int64_t capacity_rows, size_t *bytes);
refree_status refree_compress_layer_host(const refree_params *p, const void *q_win,
                                         const void *k, const void *v, int64_t kv_elems,
                                         const int32_t *seq_start, const int32_t *seq_len,
                                         int64_t total_tokens,
                                         void *k_out, void *v_out, int64_t capacity_rows,
                                         int32_t *lengths, int64_t *offsets,
                                         int32_t *kept_idx, float *scores,
                                         void *arena, size_t arena_bytes, void *stream);

/* The same host-memory pass for a run of `num_layers` layers that share one
 * shape (Algorithm 1 is applied layer by layer after prefill, Section 3.3),
 * pipelined over three internal streams: the inputs of layer l + 1 travel to the
 * device and the kept rows of layer l - 1 travel back while layer l is compressed,
 * so the run costs about one direction's copy time per layer.
 *   q_win, k, v, k_out, v_out, lengths, offsets  arrays of `num_layers` HOST
 *            pointers, one per layer, each as in refree_compress_layer_host
 *            (pinned memory lets the copies overlap; pageable memory works but
 *            serialises them)
 *   seq_start, seq_len, total_tokens, kv_elems, capacity_rows  common to all layers
 *   arena    DEVICE buffer of refree_host_pipeline_arena_size() bytes, 256-byte
 *            aligned: two sets of staging buffers and one workspace
 * Index lists and scores are not returned (use the per-layer call for them).
 * The call creates and destroys its streams and events, blocks until every layer
 * is back in host memory, and returns the first error met (device-side
 * conditions as REFREE_ERR_CAPACITY / _TIMEOUT / _NONFINITE). */
refree_status refree_host_pipeline_arena_size(const refree_params *p, int64_t total_tokens, int64_t kv_elems,
                                              int64_t capacity_rows, size_t *bytes);
refree_status refree_compress_layers_host(const refree_params *p, int32_t num_layers,
                                          const void *const *q_win, const void *const *k, const void *const *v,
                                          int64_t kv_elems, const int32_t *seq_start, const int32_t *seq_len,
                                          int64_t total_tokens, void *const *k_out, void *const *v_out,
                                          int64_t capacity_rows, int32_t *const *lengths, int64_t *const *offsets,
                                          void *arena, size_t arena_bytes);

/* Selection without any device allocation (no counterpart in the paper; the
 * arithmetic and the outputs are exactly those of refree_select_budget).
 *
 * Who needs it: code that may not create device memory at the point where it
 * compresses a cache - a serving engine whose memory pool was carved up at
 * start-up and has no slack left for a workspace, a plug-in running inside a
 * host that forbids cudaMalloc after initialisation, a process whose allocator
 * would synchronise the device in the middle of a latency-critical step.  Such
 * callers own scores, lengths, offsets and kept_idx already (they are the
 * stage's inputs and outputs) but cannot obtain the scratch that
 * refree_select_budget takes as `workspace`.
 *
 * Here the scratch is a fixed array of REFREE_STATIC_SCRATCH_BYTES compiled into
 * the library; every GPU that loads the library holds that many bytes until the
 * process exits.  The call performs no cudaMalloc / cudaFree and uses no
 * allocating routine.  A problem whose scratch need exceeds the array (roughly
 * num_seqs * num_kv_heads > REFREE_STATIC_SCRATCH_BYTES / 24) is refused with
 * REFREE_ERR_STATIC_LIMIT and nothing is launched.
 *
 * The first call on each device looks up the device address of the array
 * (cudaGetSymbolAddress, with that device current); make that first call
 * outside any stream capture.  All calls on a device share the one array: it
 * keeps the previous call's contents, which is harmless because each call
 * writes every record before reading it, but two calls whose kernels overlap
 * on the GPU (different streams, no ordering between them) race on it. */
#define REFREE_STATIC_SCRATCH_BYTES (256 * 1024)
refree_status refree_select_budget_static(const refree_params *p, const float *scores,
                                          const int32_t *seq_len, int64_t total_tokens,
                                          int32_t *lengths, int64_t *offsets,
                                          int32_t *kept_idx, int64_t capacity_rows,
                                          int32_t *device_status, void *stream);

/* Decode-step attention over the compacted ragged cache, the consumer of the
 * pass (Algorithm 1 hands K_c, V_c to generation; Section 3.3 batches sequences
 * whose budgets differ).  For every sequence s and query head h, with
 * u = s*num_kv_heads + h / (num_q_heads / num_kv_heads):
 *     out[s, h, :] = softmax(q_new[s, h, :] . K_c[rows of u]^T / sqrt(head_dim)) V_c[rows of u]
 * over rows [offsets[u], offsets[u+1]) of k_c / v_c.
 *   q_new    [num_seqs, num_q_heads, head_dim], params->dtype           (device, in)
 *   k_c, v_c [rows, head_dim] contiguous, params->dtype, 16-byte aligned (device, in):
 *            the k_out / v_out of refree_compact or refree_compress_layer
 *   offsets  [num_seqs*num_kv_heads + 1] int64                          (device, in)
 *   max_rows_per_unit  host-side upper bound of offsets[u+1] - offsets[u] (the longest
 *            sequence length always is one); it sizes the launch.  A longer segment sets
 *            REFREE_DEV_CAPACITY in *device_status and only its first rows are used.
 *   out      [num_seqs, num_q_heads, head_dim] fp32                     (device, out);
 *            an empty segment gives a zero row
 *   workspace  refree_decode_workspace_size(params, max_rows_per_unit) bytes, 256-byte
 *            aligned (device, scratch).
 * Only num_seqs, num_q_heads, num_kv_heads, head_dim and dtype of params are read.
 * Products are exact (bf16) or fp32, sums and the softmax are fp32. */
refree_status refree_decode_workspace_size(const refree_params *params, int64_t max_rows_per_unit, size_t *bytes);
refree_status refree_decode_attention(const refree_params *params, const void *q_new,
                                      const void *k_c, const void *v_c, const int64_t *offsets,
                                      int64_t max_rows_per_unit, float *out,
                                      void *workspace, size_t workspace_bytes,
                                      int32_t *device_status, void *stream);

/* The same decode step over the strided ragged cache that refree_compact_inplace
 * (or refree_compress_layer_inplace) leaves: the rows of unit u = (s, g) are
 * rows [0, lengths[u]) (REFREE_ANCHOR_FRONT) or [n_s - lengths[u], n_s)
 * (REFREE_ANCHOR_BACK) of the unit's own region of k and v, addressed with
 * seq_start and the strides of params as in refree_score.
 *   k, v     the compacted-in-place cache arrays (device, in); head-major
 *            layouts only: k_stride_tok = v_stride_tok = head_dim and the other
 *            strides multiples of head_dim, else REFREE_ERR_UNSUPPORTED
 *   lengths  [num_seqs*num_kv_heads] int32 budgets (device, in)
 * Everything else as in refree_decode_attention. */
refree_status refree_decode_attention_inplace(const refree_params *params, const void *q_new,
                                              const void *k, const void *v,
                                              const int32_t *seq_start, const int32_t *seq_len,
                                              const int32_t *lengths, int32_t anchor,
                                              int64_t max_rows_per_unit, float *out,
                                              void *workspace, size_t workspace_bytes,
                                              int32_t *device_status, void *stream);

/* Diagnostic with no counterpart in the paper: the number of CUDA kernels this
 * library has enqueued in this process so far (all entry points, all streams). */
int64_t refree_kernel_launch_count(void);

/* Measurement aids with no counterpart in the paper: two memory-system probes with the
 * access shape of the pass (Section 3.2's O(n) claim is a statement about exactly this
 * traffic), used by the benchmark to report what such traffic can reach on the device.
 *   refree_sol_read_stream  reads `bytes` (a multiple of 16) from src (device, 16-byte
 *                           aligned) once: the K stream of scoring.
 *   refree_sol_row_mix      reads rows [0, rows) of k, and copies the last kept_rows rows
 *                           of k and of v to k_out and v_out: (rows + kept_rows) rows
 *                           read, 2 * kept_rows written, the mix of the whole pass.
 * `sink` (device int32, nullable) only keeps the loads alive; nothing meaningful is
 * written to it.  Passing REFREE_SOL_BULK as `sink` selects the variant that moves the same
 * bytes with the bulk-copy engine (global -> shared -> global in 16 KB pieces) instead of
 * vector loads and stores in registers; its first call on a device sets a kernel attribute
 * and should come before any stream capture.  Errors: REFREE_ERR_INVALID_ARG for null, misaligned or negative
 * arguments; nothing is launched then. */
#define REFREE_SOL_BULK ((int32_t *)(uintptr_t)1)
refree_status refree_sol_read_stream(const void *src, int64_t bytes, int32_t *sink, void *stream);
refree_status refree_sol_row_mix(const void *k, const void *v, void *k_out, void *v_out,
                                 int64_t rows, int64_t kept_rows, int32_t row_bytes,
                                 int32_t *sink, void *stream);

/* Static string for a status code. */
const char *refree_status_string(refree_status s);

#ifdef __cplusplus
}
#endif
#endif /* REFREEKV_H */
