/*
 * CPU oracle for the post-prefill KV-compression pass of ReFreeKV.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * pass computes, written from the paper, and exists so that the CUDA library
 * can be checked against it.  It shares no code, header, table or helper with
 * the CUDA path, and the CUDA path never calls it.  Only the tests, the smoke
 * check and the benchmark's CPU-baseline leg load it.
 *
 * Everything is computed in fp64 from the stored input bits (fp32 or bf16,
 * widened exactly).  Loops are serial inside one (sequence, KV head) unit;
 * OpenMP only spreads independent units over cores.
 *
 * What pins each function (see tests/test_oracle_pins.py):
 *   oracle_score   - full n x n causal softmax written with numpy (Section 3.2,
 *                    the definition of A) reduced by the literal Eq. 2, on tiny
 *                    inputs; column-mass identities; w = 1 is a textbook softmax.
 *   oracle_select  - Eq. 1 evaluated by masking the ranked vector for every j
 *                    and taking the norm directly (no prefix sum); closed forms
 *                    for uniform, one-hot and geometric score vectors;
 *                    monotonicity in T; scale invariance; numpy stable argsort
 *                    for the score ranking.
 *   oracle_compact - row-by-row byte comparison against numpy fancy indexing.
 *
 * Readings of the paper taken here, where it is silent, garbled or at odds
 * with itself:
 *   - Eq. 2: column i of the last w rows of A, divided by the number of those
 *     rows that can see i causally, min(w_eff, n - i).
 *   - Eq. 1 / Eq. 3: leftmost j with 1 - sqrt(C_j / C_n) < T, strict; the kept
 *     set is the first j ranked positions.  No such j, or C_n = 0: keep all.
 *   - GQA: the score of a KV head is the mean over its query heads.
 *   - keep_window: the budget is never below min(n, m + w_eff).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t num_seqs, num_q_heads, num_kv_heads, head_dim;
    int32_t window;       /* w: number of trailing query rows (paper k)       */
    int32_t sink;         /* m: leading positions ranked first (paper m)      */
    double  threshold;    /* T of Eq. 1                                       */
    int32_t rank_mode;    /* 0 position ranking, 1 ranking by score           */
    int32_t scope;        /* 0 one budget per (seq, KV head), 1 per seq       */
    int32_t keep_window;  /* 1: budget >= min(n, m + w_eff)                   */
    int32_t force_full;   /* 1: keep everything (frozen bottom layers)        */
    int32_t dtype;        /* 0 fp32, 1 bf16                                   */
    int64_t k_stride_seq, k_stride_tok, k_stride_head;   /* in elements      */
    int64_t v_stride_seq, v_stride_tok, v_stride_head;
} oracle_params;

static double widen(const void *base, int64_t idx, int dtype)
{
    if (dtype == 0)
        return (double)((const float *)base)[idx];
    uint32_t bits = (uint32_t)((const uint16_t *)base)[idx] << 16;
    float f;
    memcpy(&f, &bits, 4);
    return (double)f;
}

static int imin(int a, int b) { return a < b ? a : b; }

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int t)
{
#ifdef _OPENMP
    omp_set_num_threads(t);
#else
    (void)t;
#endif
}

/* Reduced attention vector A' (Section 3.2 "Reducing Overhead", Eq. 2) from the
 * last w rows of the causal softmax attention (definition of A, Section 3.2;
 * Algorithm 1 "Attention" step), averaged over the query heads of each KV head.
 *   q_win  [B, Hq, w, d]: q_win[s,h,r] is the query at position n_s - w + r;
 *          rows with a negative position are ignored.
 *   scores [Hkv, total_tokens] fp64, sequences packed by the running sum of
 *          seq_len. */
int oracle_score(const oracle_params *p, const void *q_win, const void *k,
                 const int32_t *seq_start, const int32_t *seq_len,
                 int64_t total_tokens, double *scores)
{
    const int B = p->num_seqs, Hq = p->num_q_heads, Hkv = p->num_kv_heads;
    const int d = p->head_dim, w = p->window, G = Hq / Hkv;
    int64_t *pack = (int64_t *)malloc(sizeof(int64_t) * (size_t)(B + 1));
    pack[0] = 0;
    for (int s = 0; s < B; ++s) pack[s + 1] = pack[s] + seq_len[s];
    const double inv_sqrt_d = 1.0 / sqrt((double)d);

#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int s = 0; s < B; ++s) {
        for (int g = 0; g < Hkv; ++g) {
            const int n = seq_len[s];
            if (n <= 0) continue;
            const int w_eff = imin(w, n);
            double *out = scores + (int64_t)g * total_tokens + pack[s];
            double *e = (double *)malloc(sizeof(double) * (size_t)n);
            double *col = (double *)malloc(sizeof(double) * (size_t)n);
            double *qd = (double *)malloc(sizeof(double) * (size_t)d);
            for (int i = 0; i < n; ++i) out[i] = 0.0;
            for (int hh = 0; hh < G; ++hh) {
                const int h = g * G + hh;
                for (int i = 0; i < n; ++i) col[i] = 0.0;
                for (int rr = 0; rr < w_eff; ++rr) {
                    const int pos = n - w_eff + rr;           /* query position */
                    const int64_t qoff =
                        (((int64_t)s * Hq + h) * w + (w - w_eff + rr)) * d;
                    for (int c = 0; c < d; ++c) qd[c] = widen(q_win, qoff + c, p->dtype);
                    /* logits of the visible keys i <= pos */
                    double mx = -INFINITY;
                    for (int i = 0; i <= pos; ++i) {
                        const int64_t koff = (int64_t)s * p->k_stride_seq +
                            ((int64_t)seq_start[s] + i) * p->k_stride_tok +
                            (int64_t)g * p->k_stride_head;
                        double dot = 0.0;
                        for (int c = 0; c < d; ++c)
                            dot += qd[c] * widen(k, koff + c, p->dtype);
                        e[i] = dot * inv_sqrt_d;
                        if (e[i] > mx) mx = e[i];
                    }
                    double den = 0.0;
                    for (int i = 0; i <= pos; ++i) {
                        e[i] = exp(e[i] - mx);
                        den += e[i];
                    }
                    for (int i = 0; i <= pos; ++i) col[i] += e[i] / den;
                }
                /* Eq. 2: average over the window rows that see column i */
                for (int i = 0; i < n; ++i)
                    out[i] += col[i] / (double)imin(w_eff, n - i);
            }
            for (int i = 0; i < n; ++i) out[i] /= (double)G;
            free(e); free(col); free(qd);
        }
    }
    free(pack);
    return 0;
}

typedef struct { double key; int32_t idx; } ranked_t;

static int by_key_desc_then_index(const void *a, const void *b)
{
    const ranked_t *x = (const ranked_t *)a, *y = (const ranked_t *)b;
    if (x->key > y->key) return -1;
    if (x->key < y->key) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

static int by_int_asc(const void *a, const void *b)
{
    const int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/* Ranked order of the n positions of one unit (0-based positions).
 *   position ranking (Section 3.2 "Initial Ranking"): the first m positions,
 *     then the remaining ones from the last backwards.
 *   score ranking (Section 4.4 "Initial Ranking Strategies"): the m leading
 *     positions and the window in position order, then the rest by decreasing
 *     squared-score key, equal keys by increasing position. */
static void rank_order(int n, int m, int w_eff, int rank_mode, const double *sq, int32_t *pi)
{
    const int lead = imin(m, n);
    if (rank_mode == 0) {
        for (int j = 0; j < lead; ++j) pi[j] = j;
        for (int j = lead; j < n; ++j) pi[j] = n - 1 - (j - lead);
        return;
    }
    if (lead + w_eff >= n) {
        for (int j = 0; j < n; ++j) pi[j] = j;
        return;
    }
    int j = 0;
    for (int i = 0; i < lead; ++i) pi[j++] = i;
    for (int i = n - w_eff; i < n; ++i) pi[j++] = i;
    const int rest = n - lead - w_eff;
    ranked_t *r = (ranked_t *)malloc(sizeof(ranked_t) * (size_t)rest);
    for (int t = 0; t < rest; ++t) { r[t].idx = lead + t; r[t].key = sq[lead + t]; }
    qsort(r, (size_t)rest, sizeof(ranked_t), by_key_desc_then_index);
    for (int t = 0; t < rest; ++t) pi[j++] = r[t].idx;
    free(r);
}

/* Threshold-free stopping rule (Eq. 1 in its cumulative form, Eq. 3, and the
 * Cumsum / Sqrt / ratio / Where steps of Algorithm 1) on fp32 scores.
 *   scores32 [Hkv, total_tokens]  reduced attention, already rounded to fp32
 *   lengths  [B, Hkv]   kept count b per (sequence, KV head)
 *   offsets  [B*Hkv+1]  running sum of lengths
 *   kept_idx [sum b]    kept positions of each unit, ascending, back to back
 *   pi_out   nullable [Hkv, total_tokens]  ranked order per unit
 *   ratio_out nullable [Hkv, total_tokens] sqrt(C_j / C_n) for j = 1..n at j-1
 *   gap_out  nullable [B, Hkv]  min over j in {j*-1, j*} of
 *            |sqrt(C_j/C_n) - (1 - T)|, the distance of the decision from a tie
 *   jstar_out nullable [B, Hkv] the stop index before the window floor */
int oracle_select(const oracle_params *p, const float *scores32, const int32_t *seq_len,
                  int64_t total_tokens, int32_t *lengths, int64_t *offsets, int32_t *kept_idx,
                  int32_t *pi_out, double *ratio_out, double *gap_out, int32_t *jstar_out)
{
    const int B = p->num_seqs, Hkv = p->num_kv_heads, m = p->sink, w = p->window;
    const double T = p->threshold;
    int64_t *pack = (int64_t *)malloc(sizeof(int64_t) * (size_t)(B + 1));
    pack[0] = 0;
    for (int s = 0; s < B; ++s) pack[s + 1] = pack[s] + seq_len[s];
    int32_t **kept_tmp = (int32_t **)calloc((size_t)B * Hkv, sizeof(int32_t *));

#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < B * Hkv; ++u) {
        const int s = u / Hkv, g = u % Hkv;
        const int n = seq_len[s];
        if (p->scope == 1 && g != 0) continue;      /* one decision per sequence */
        if (n <= 0) { lengths[u] = 0; continue; }
        const int w_eff = imin(w, n);
        double *sq = (double *)malloc(sizeof(double) * (size_t)n);
        int32_t *pi = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
        /* Square step of Algorithm 1; in layer scope the squares of all KV
         * heads of the layer add up (the Frobenius norm runs over heads too) */
        for (int i = 0; i < n; ++i) {
            if (p->scope == 0) {
                const double a = (double)scores32[(int64_t)g * total_tokens + pack[s] + i];
                sq[i] = a * a;
            } else {
                double acc = 0.0;
                for (int gg = 0; gg < Hkv; ++gg) {
                    const double a = (double)scores32[(int64_t)gg * total_tokens + pack[s] + i];
                    acc += a * a;
                }
                sq[i] = acc;
            }
        }
        rank_order(n, m, w_eff, p->rank_mode, sq, pi);
        double Cn = 0.0;
        for (int j = 0; j < n; ++j) Cn += sq[pi[j]];
        int jstar = n;
        double gap = INFINITY, C = 0.0, prev_ratio = 0.0;
        int found = 0;
        for (int j = 1; j <= n; ++j) {
            C += sq[pi[j - 1]];
            const double ratio = (Cn > 0.0) ? sqrt(C / Cn) : 1.0;
            if (ratio_out)
                ratio_out[(int64_t)g * total_tokens + pack[s] + (j - 1)] = ratio;
            if (!found && Cn > 0.0 && 1.0 - ratio < T) {
                found = 1;
                jstar = j;
                gap = fabs(ratio - (1.0 - T));
                if (j > 1 && fabs(prev_ratio - (1.0 - T)) < gap)
                    gap = fabs(prev_ratio - (1.0 - T));
                if (!ratio_out) break;
            }
            prev_ratio = ratio;
        }
        if (!found && Cn > 0.0) gap = fabs(1.0 - (1.0 - T));
        int b = jstar;
        const int floor_b = p->keep_window ? imin(n, m + w_eff) : 1;
        if (b < floor_b) b = floor_b;
        if (p->force_full) b = n;
        int32_t *kept = (int32_t *)malloc(sizeof(int32_t) * (size_t)b);
        memcpy(kept, pi, sizeof(int32_t) * (size_t)b);
        qsort(kept, (size_t)b, sizeof(int32_t), by_int_asc);
        const int g_lo = g, g_hi = (p->scope == 1) ? Hkv : g + 1;
        for (int gg = g_lo; gg < g_hi; ++gg) {
            const int uu = s * Hkv + gg;
            lengths[uu] = b;
            if (gap_out) gap_out[uu] = gap;
            if (jstar_out) jstar_out[uu] = jstar;
            if (pi_out)
                memcpy(pi_out + (int64_t)gg * total_tokens + pack[s], pi, sizeof(int32_t) * (size_t)n);
            if (ratio_out && gg != g)
                memcpy(ratio_out + (int64_t)gg * total_tokens + pack[s],
                       ratio_out + (int64_t)g * total_tokens + pack[s], sizeof(double) * (size_t)n);
            if (gg == g_lo) {
                kept_tmp[uu] = kept;
            } else {
                kept_tmp[uu] = (int32_t *)malloc(sizeof(int32_t) * (size_t)b);
                memcpy(kept_tmp[uu], kept, sizeof(int32_t) * (size_t)b);
            }
        }
        free(sq); free(pi);
    }
    offsets[0] = 0;
    for (int u = 0; u < B * Hkv; ++u) offsets[u + 1] = offsets[u] + lengths[u];
    for (int u = 0; u < B * Hkv; ++u) {
        if (kept_tmp[u]) {
            if (kept_idx)
                memcpy(kept_idx + offsets[u], kept_tmp[u], sizeof(int32_t) * (size_t)lengths[u]);
            free(kept_tmp[u]);
        }
    }
    free(kept_tmp); free(pack);
    return 0;
}

/* Compress step of Algorithm 1: copy the kept K and V rows, in their original
 * order, into one dense array per tensor; unit u = s*Hkv + g owns rows
 * [offsets[u], offsets[u+1]).  Rows are copied byte for byte. */
int oracle_compact(const oracle_params *p, const void *k, const void *v,
                   const int32_t *seq_start, const int32_t *seq_len,
                   const int32_t *lengths, const int64_t *offsets, const int32_t *kept_idx,
                   void *k_out, void *v_out)
{
    (void)seq_len;
    const int B = p->num_seqs, Hkv = p->num_kv_heads, d = p->head_dim;
    const size_t esz = p->dtype == 0 ? 4 : 2, row = (size_t)d * esz;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < B * Hkv; ++u) {
        const int s = u / Hkv, g = u % Hkv;
        for (int t = 0; t < lengths[u]; ++t) {
            const int64_t i = kept_idx[offsets[u] + t];
            const int64_t ko = (int64_t)s * p->k_stride_seq +
                ((int64_t)seq_start[s] + i) * p->k_stride_tok + (int64_t)g * p->k_stride_head;
            const int64_t vo = (int64_t)s * p->v_stride_seq +
                ((int64_t)seq_start[s] + i) * p->v_stride_tok + (int64_t)g * p->v_stride_head;
            memcpy((char *)k_out + (size_t)(offsets[u] + t) * row, (const char *)k + (size_t)ko * esz, row);
            memcpy((char *)v_out + (size_t)(offsets[u] + t) * row, (const char *)v + (size_t)vo * esz, row);
        }
    }
    return 0;
}

/* Decode-step attention over a compacted ragged cache (the consumer of the
 * pass: generation reads K_c, V_c after Algorithm 1 returns them).  One new
 * query per (sequence, query head); plain softmax(q K_c^T / sqrt(d)) V_c over
 * the rows of the head's segment, fp64.  out [B, Hq, d] fp64. */
int oracle_decode_attention(const oracle_params *p, const void *q_new /*[B,Hq,d]*/,
                            const void *k_c, const void *v_c, const int64_t *offsets, double *out)
{
    const int B = p->num_seqs, Hq = p->num_q_heads, Hkv = p->num_kv_heads, d = p->head_dim;
    const int G = Hq / Hkv;
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int s = 0; s < B; ++s) {
        for (int h = 0; h < Hq; ++h) {
            const int u = s * Hkv + h / G;
            const int64_t lo = offsets[u], len = offsets[u + 1] - offsets[u];
            double *o = out + ((int64_t)s * Hq + h) * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            if (len <= 0) continue;
            double *e = (double *)malloc(sizeof(double) * (size_t)len);
            double mx = -INFINITY;
            for (int64_t t = 0; t < len; ++t) {
                double dot = 0.0;
                for (int c = 0; c < d; ++c)
                    dot += widen(q_new, ((int64_t)s * Hq + h) * d + c, p->dtype) *
                           widen(k_c, (lo + t) * d + c, p->dtype);
                e[t] = dot * inv_sqrt_d;
                if (e[t] > mx) mx = e[t];
            }
            double den = 0.0;
            for (int64_t t = 0; t < len; ++t) { e[t] = exp(e[t] - mx); den += e[t]; }
            for (int64_t t = 0; t < len; ++t)
                for (int c = 0; c < d; ++c)
                    o[c] += (e[t] / den) * widen(v_c, (lo + t) * d + c, p->dtype);
            free(e);
        }
    }
    return 0;
}
