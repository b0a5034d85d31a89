// Decode-step attention over the compacted ragged cache: the consumer of the pass
// (Algorithm 1 returns K_c, V_c "for generation"; Section 3.3 batches sequences of
// different budgets).  One new query per (sequence, query head):
//     out[s, h, :] = softmax(q[s, h] . K_c[u]^T / sqrt(d)) V_c[u],   u = s Hkv + g(h),
// over rows [offsets[u], offsets[u + 1]) of the dense ragged cache.
//
// The step streams K_c and V_c once (G query heads share every row): HBM-bound.
//
//   bf16   block = (unit, span of rows), eight warps take 16-row blocks round-robin.  A block
//          of 16 rows is contiguous in the compacted cache: one lane of the warp copies it with
//          cp.async.bulk into the warp's private shared-memory ring (three blocks in flight,
//          mbarrier-signalled).  mma.m16n8k16 serves as the dot-product unit:
//            S^T[head, row] = Q K^T   A = the G (<= 16) queries, B = 8 rows of K; each
//                                     lane reads 16-byte pieces of "its" row and the
//                                     queries are cut the same way, so the order of the
//                                     elements inside a k-step cancels;
//            O[head, col]  += P V     A = the probabilities straight from the S^T
//                                     accumulators (split into two bf16 terms, so the
//                                     product carries 16 mantissa bits), B = V: a lane
//                                     reads 16-byte pieces of four rows and interleaves
//                                     row pairs with byte permutes.  The eight columns of
//                                     an output tile are spread over the row (column
//                                     (t / 8) 64 + 8 n + t % 8 for tile t, slot n); the
//                                     order is undone when the result is stored.
//          Running (max, sum) per head (online softmax), warps merged through shared
//          memory, spans merged by a second small kernel when a unit has several.
//   fp32   (or unaligned bf16 pointers) lanes own columns, dot products by warp shuffles.
#include <algorithm>

#include "refree_internal.cuh"

namespace refree {
namespace {

constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;
constexpr float kLog2eDec = 1.4426950408889634f;
constexpr int kDecStages = 3;       // 16-row blocks of K and V in flight per warp

struct DecArgs {
    refree_params p;
    const void *q, *kc, *vc;
    const int64_t *offsets;
    // strided ragged cache (what refree_compact_inplace leaves): rows of unit (s, g) sit in the unit's own
    // region of the original K / V arrays; `lengths` non-null selects this form and `offsets` is unused
    const int32_t *seq_start, *seq_len, *lengths;
    int anchor_back;
    float *out;      // [B, Hq, d]
    float *part;     // [U, gx, G, d + 2]: un-normalised output (block order), max, sum
    int span;        // rows per block, a multiple of 16
    int gx;          // blocks per unit
    int native;      // 1: partials hold the mma tile order, 0: plain column order
    int32_t *dev_status;
};

// First row (in rows of head_dim elements from the array's start) and row count of unit u in K and in V.
__device__ inline void unit_rows(const DecArgs &a, int u, int64_t &lo_k, int64_t &lo_v, int64_t &len64)
{
    if (!a.lengths) {
        lo_k = lo_v = a.offsets[u];
        len64 = a.offsets[u + 1] - lo_k;
        return;
    }
    const int Hkv = a.p.num_kv_heads, s = u / Hkv, g = u % Hkv;
    const int n = max(a.seq_len[s], 0);
    const int b = max(0, min(a.lengths[u], n));
    const int64_t first = (int64_t)a.seq_start[s] + (a.anchor_back ? n - b : 0);
    lo_k = ((int64_t)s * a.p.k_stride_seq + (int64_t)g * a.p.k_stride_head) / a.p.head_dim + first;
    lo_v = ((int64_t)s * a.p.v_stride_seq + (int64_t)g * a.p.v_stride_head) / a.p.head_dim + first;
    len64 = b;
}

__device__ inline float dec_ex2(float x)
{
    float y;
    asm("ex2.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ inline void dec_mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ inline uint4 dec_ld16(const char *p, bool valid)
{
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (valid)
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// ---- per-warp staging ring: bulk copies (TMA engine, no tensor map) signalled on an mbarrier ----
__device__ inline uint32_t dec_smem(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ inline void dec_bar_init(uint64_t *bar)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(dec_smem(bar)) : "memory");
}
__device__ inline void dec_bar_expect(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(dec_smem(bar)), "r"(bytes) : "memory");
}
// contiguous global -> shared copy; addresses 16-byte aligned, size a multiple of 16
__device__ inline void dec_bulk_copy(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dec_smem(dst)), "l"(src), "r"(bytes), "r"(dec_smem(bar)) : "memory");
}
// bounded wait for the phase with the given parity; false when it gave up
__device__ inline bool dec_bar_wait(uint64_t *bar, uint32_t parity)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(dec_smem(bar)), "r"(parity) : "memory");
        if (ok) return true;
        if (it > 64) __nanosleep(it > 4096 ? 256 : 32);
    }
    return false;
}

// p = hi + lo with hi, lo bf16: packs two probabilities per register for the A operand
__device__ inline void split_pack(float p0, float p1, uint32_t &hi, uint32_t &lo)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
    const float2 hf = __bfloat1622float2(h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(p0 - hf.x, p1 - hf.y);
    hi = *reinterpret_cast<const uint32_t *>(&h);
    lo = *reinterpret_cast<const uint32_t *>(&l);
}

// column of the output that slot `idx` of the block order holds
__device__ __host__ inline int native_col(int idx, int native)
{
    if (!native) return idx;
    const int t = idx >> 3, n = idx & 7;
    return (t >> 3) * 64 + n * 8 + (t & 7);
}

// Merge the warps' (max, sum, O) through shared memory in warp order and store the block's
// result: the final output when the unit has one block, a partial record otherwise.
// sm: [kDecWarps][GP][D + 2] floats.
template <int D>
__device__ inline void merge_and_store(const DecArgs &a, float *sm, int GP, int G, int u, int x, int nblocks)
{
    __syncthreads();
    const int Hkv = a.p.num_kv_heads, s = u / Hkv, g = u % Hkv;
    for (int e = threadIdx.x; e < G * (D + 2); e += kDecThreads) {
        const int h = e / (D + 2), idx = e % (D + 2);
        float M = -INFINITY;
        for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, sm[(w * GP + h) * (D + 2) + D]);
        float val = 0.f, L = 0.f;
        for (int w = 0; w < kDecWarps; ++w) {
            const float *rec = sm + (w * GP + h) * (D + 2);
            const float f = rec[D] == -INFINITY ? 0.f : dec_ex2(rec[D] - M);
            val += rec[idx < D ? idx : 0] * f;
            L += rec[D + 1] * f;
        }
        if (nblocks == 1) {
            if (idx < D)
                a.out[((int64_t)s * a.p.num_q_heads + g * G + h) * D + native_col(idx, a.native)] = L > 0.f ? val / L : 0.f;
        } else {
            float *rec = a.part + (((int64_t)u * a.gx + x) * G + h) * (D + 2);
            rec[idx] = idx < D ? val : (idx == D ? M : L);
        }
    }
}

// bf16 path.  UPPER: the group has more than eight query heads (rows 8..15 of the A operand).
template <int D, bool UPPER>
__global__ void __launch_bounds__(kDecThreads, 1)
decode_mma_kernel(DecArgs a)
{
    constexpr int CH = D / 32;          // 16-byte pieces per lane of a K (or Q) row
    constexpr int HF = D / 64;          // 128-byte halves of a V row
    constexpr int NT = D / 8;           // output tiles of eight columns
    constexpr int GP = UPPER ? 16 : 8;
    extern __shared__ float dec_sm[];
    const refree_params &p = a.p;
    const int Hkv = p.num_kv_heads, G = p.num_q_heads / Hkv;
    const int u = blockIdx.y, x = blockIdx.x, s = u / Hkv, g = u % Hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = lane >> 2, c = lane & 3;
    int64_t lo, lo_v, len64;
    unit_rows(a, u, lo, lo_v, len64);
    const int len = (int)max((int64_t)0, min(len64, (int64_t)a.span * a.gx));
    if (len64 > len && x == 0 && threadIdx.x == 0 && a.dev_status) atomicOr(a.dev_status, REFREE_DEV_CAPACITY);
    const int nblocks = ceil_div(len, a.span);
    if (x >= max(nblocks, 1)) return;
    if (len == 0) {                     // empty segment: the output row is zero
        for (int e = threadIdx.x; e < G * D; e += kDecThreads)
            a.out[((int64_t)s * p.num_q_heads + g * G) * D + e] = 0.f;
        return;
    }
    const int begin = x * a.span, end = min(len, begin + a.span);
    const float scale = kLog2eDec * rsqrtf((float)D);

    // queries of heads r (and r + 8), cut into the 16-byte pieces at byte 64 j + 16 c
    uint4 qa[CH], qb[CH];
    {
        const char *qrow = reinterpret_cast<const char *>(a.q) +
                           ((int64_t)s * p.num_q_heads + g * G) * D * (int64_t)sizeof(__nv_bfloat16);
#pragma unroll
        for (int j = 0; j < CH; ++j) {
            qa[j] = dec_ld16(qrow + (int64_t)r * D * 2 + j * 64 + c * 16, r < G);
            qb[j] = UPPER ? dec_ld16(qrow + (int64_t)(r + 8) * D * 2 + j * 64 + c * 16, r + 8 < G) : make_uint4(0u, 0u, 0u, 0u);
        }
    }
    const char *kbase = reinterpret_cast<const char *>(a.kc) + lo * D * 2;
    const char *vbase = reinterpret_cast<const char *>(a.vc) + lo_v * D * 2;

    float o[NT][4];
#pragma unroll
    for (int t = 0; t < NT; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;
    float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};

    // K: B operand of the two S^T products (rows row0 + r and row0 + 8 + r);
    // V: rows 2c, 2c + 1, 8 + 2c, 9 + 2c of the block, piece r of each 128-byte half.
    // A 16-row block of K (and of V) is contiguous in the compacted cache, so one lane brings it in
    // with a bulk copy into the warp's own ring: kDecStages blocks per warp are in flight at the
    // price of two instructions each (registers could hold one, and per-lane cp.async costs more
    // to issue than the products of the block).  The ring is private to the warp: its lanes wait on
    // the warp's barriers and lane 0 refills a slot after all lanes have read it.
    constexpr int kBlockBytes = 16 * D * 2;          // one 16-row block of K (or V)
    unsigned char *ring = reinterpret_cast<unsigned char *>(dec_sm) + (size_t)warp * kDecStages * 2 * kBlockBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(reinterpret_cast<unsigned char *>(dec_sm) +
                                                  (size_t)kDecWarps * kDecStages * 2 * kBlockBytes) + warp * kDecStages;
    if (lane == 0) {
#pragma unroll
        for (int st = 0; st < kDecStages; ++st) dec_bar_init(bars + st);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    auto issue = [&](int row0, int slot) {           // lane 0 only
        if (row0 < end) {
            const uint32_t bytes = (uint32_t)min(16, end - row0) * D * 2;
            dec_bar_expect(bars + slot, 2 * bytes);
            dec_bulk_copy(ring + (size_t)slot * 2 * kBlockBytes, kbase + (int64_t)row0 * D * 2, bytes, bars + slot);
            dec_bulk_copy(ring + (size_t)slot * 2 * kBlockBytes + kBlockBytes, vbase + (int64_t)row0 * D * 2, bytes, bars + slot);
        }
    };
    const int first = begin + warp * 16, stride = kDecWarps * 16;
    if (lane == 0)
#pragma unroll
        for (int st = 0; st < kDecStages; ++st) issue(first + st * stride, st);
    int slot = 0;
    uint32_t parity = 0;
    bool timed_out = false;
    for (int row0 = first; row0 < end; row0 += stride) {
        const int vr[4] = {row0 + 2 * c, row0 + 2 * c + 1, row0 + 8 + 2 * c, row0 + 9 + 2 * c};
        if (!dec_bar_wait(bars + slot, parity)) { timed_out = true; break; }
        const unsigned char *kblk = ring + (size_t)slot * 2 * kBlockBytes, *vblk = kblk + kBlockBytes;
        uint4 k1[CH], k2[CH];
#pragma unroll
        for (int j = 0; j < CH; ++j) {
            k1[j] = *reinterpret_cast<const uint4 *>(kblk + r * D * 2 + j * 64 + c * 16);
            k2[j] = *reinterpret_cast<const uint4 *>(kblk + (8 + r) * D * 2 + j * 64 + c * 16);
        }
        float s1[4] = {0.f, 0.f, 0.f, 0.f}, s2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int j = 0; j < CH; ++j) {
            dec_mma(s1, qa[j].x, qb[j].x, qa[j].y, qb[j].y, k1[j].x, k1[j].y);
            dec_mma(s1, qa[j].z, qb[j].z, qa[j].w, qb[j].w, k1[j].z, k1[j].w);
            dec_mma(s2, qa[j].x, qb[j].x, qa[j].y, qb[j].y, k2[j].x, k2[j].y);
            dec_mma(s2, qa[j].z, qb[j].z, qa[j].w, qb[j].w, k2[j].z, k2[j].w);
        }
        // lane (r, c): y[hh][0..3] = logits of head r + 8 hh for rows vr[0..3]
        float y[2][4];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            y[hh][0] = vr[0] < end ? s1[2 * hh] * scale : -INFINITY;
            y[hh][1] = vr[1] < end ? s1[2 * hh + 1] * scale : -INFINITY;
            y[hh][2] = vr[2] < end ? s2[2 * hh] * scale : -INFINITY;
            y[hh][3] = vr[3] < end ? s2[2 * hh + 1] * scale : -INFINITY;
        }
        float f[2], pr[2][4];
        bool grew = false;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            float bm = fmaxf(fmaxf(y[hh][0], y[hh][1]), fmaxf(y[hh][2], y[hh][3]));
            bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 1));
            bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 2));      // row0 is valid, so bm is finite
            const float mn = fmaxf(m[hh], bm);
            f[hh] = dec_ex2(m[hh] - mn);                              // 0 on the first block
            grew |= mn != m[hh];
            m[hh] = mn;
            float sum = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) { pr[hh][i] = dec_ex2(y[hh][i] - mn); sum += pr[hh][i]; }
            l[hh] = l[hh] * f[hh] + sum;
        }
        if (__any_sync(0xffffffffu, grew)) {
#pragma unroll
            for (int t = 0; t < NT; ++t) { o[t][0] *= f[0]; o[t][1] *= f[0]; o[t][2] *= f[1]; o[t][3] *= f[1]; }
        }
        uint32_t ah[4], al[4];                        // a0, a1, a2, a3 of the P operand, high and low terms
        split_pack(pr[0][0], pr[0][1], ah[0], al[0]);
        split_pack(pr[1][0], pr[1][1], ah[1], al[1]);
        split_pack(pr[0][2], pr[0][3], ah[2], al[2]);
        split_pack(pr[1][2], pr[1][3], ah[3], al[3]);
        if (!UPPER) ah[1] = ah[3] = al[1] = al[3] = 0u;
        // rows past the end of a short last block hold what the slot held before: their probabilities
        // are zero, and zero times a stale NaN must not reach the sums
        uint4 v[4][HF];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int hf = 0; hf < HF; ++hf)
                v[i][hf] = vr[i] < end ? *reinterpret_cast<const uint4 *>(vblk + (vr[i] - row0) * D * 2 + hf * 128 + r * 16)
                                       : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int hf = 0; hf < HF; ++hf) {
            const uint32_t w0[4] = {v[0][hf].x, v[0][hf].y, v[0][hf].z, v[0][hf].w};
            const uint32_t w1[4] = {v[1][hf].x, v[1][hf].y, v[1][hf].z, v[1][hf].w};
            const uint32_t w2[4] = {v[2][hf].x, v[2][hf].y, v[2][hf].z, v[2][hf].w};
            const uint32_t w3[4] = {v[3][hf].x, v[3][hf].y, v[3][hf].z, v[3][hf].w};
#pragma unroll
            for (int wi = 0; wi < 4; ++wi)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const uint32_t sel = e ? 0x7632u : 0x5410u;
                    const uint32_t b0 = __byte_perm(w0[wi], w1[wi], sel), b1 = __byte_perm(w2[wi], w3[wi], sel);
                    const int t = hf * 8 + 2 * wi + e;
                    dec_mma(o[t], ah[0], ah[1], ah[2], ah[3], b0, b1);
                    dec_mma(o[t], al[0], al[1], al[2], al[3], b0, b1);
                }
        }
        __syncwarp();                                // every lane has read the slot
        if (lane == 0) issue(row0 + kDecStages * stride, slot);
        if (++slot == kDecStages) { slot = 0; parity ^= 1u; }
    }
    if (__any_sync(0xffffffffu, timed_out)) {
        if (lane == 0 && a.dev_status) atomicOr(a.dev_status, REFREE_DEV_TIMEOUT);
        for (int st = 0; st < kDecStages; ++st) dec_bar_wait(bars + st, 0) || dec_bar_wait(bars + st, 1);   // let copies in flight land
    }
    __syncthreads();                                 // the ring's memory now takes the warps' records
    // the four column lanes of a head hold partial sums of l
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        l[hh] += __shfl_xor_sync(0xffffffffu, l[hh], 1);
        l[hh] += __shfl_xor_sync(0xffffffffu, l[hh], 2);
    }
    float *mine = dec_sm + (size_t)warp * GP * (D + 2);
#pragma unroll
    for (int hh = 0; hh < (UPPER ? 2 : 1); ++hh) {
        float *rec = mine + (r + 8 * hh) * (D + 2);
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            rec[t * 8 + 2 * c] = o[t][2 * hh];
            rec[t * 8 + 2 * c + 1] = o[t][2 * hh + 1];
        }
        if (c == 0) { rec[D] = m[hh]; rec[D + 1] = l[hh]; }
    }
    merge_and_store<D>(a, dec_sm, GP, G, u, x, nblocks);
}

// fp32 caches and unaligned bf16 pointers: a warp takes rows round-robin, every lane owns
// E = D / 32 columns; the G dot products of a row meet by shuffles.
template <typename T, int D, int GMAX>
__global__ void __launch_bounds__(kDecThreads)
decode_lanes_kernel(DecArgs a)
{
    constexpr int E = D / 32;
    extern __shared__ float dec_sm[];
    const refree_params &p = a.p;
    const int Hkv = p.num_kv_heads, G = p.num_q_heads / Hkv;
    const int u = blockIdx.y, x = blockIdx.x, s = u / Hkv, g = u % Hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int64_t lo, lo_v, len64;
    unit_rows(a, u, lo, lo_v, len64);
    const int len = (int)max((int64_t)0, min(len64, (int64_t)a.span * a.gx));
    if (len64 > len && x == 0 && threadIdx.x == 0 && a.dev_status) atomicOr(a.dev_status, REFREE_DEV_CAPACITY);
    const int nblocks = ceil_div(len, a.span);
    if (x >= max(nblocks, 1)) return;
    if (len == 0) {
        for (int e = threadIdx.x; e < G * D; e += kDecThreads)
            a.out[((int64_t)s * p.num_q_heads + g * G) * D + e] = 0.f;
        return;
    }
    const int begin = x * a.span, end = min(len, begin + a.span);
    const float scale = kLog2eDec * rsqrtf((float)D);
    const T *q = static_cast<const T *>(a.q) + ((int64_t)s * p.num_q_heads + g * G) * D;
    const T *kc = static_cast<const T *>(a.kc) + lo * D, *vc = static_cast<const T *>(a.vc) + lo_v * D;
    float qr[GMAX][E], o[GMAX][E], m[GMAX], l[GMAX];
#pragma unroll
    for (int h = 0; h < GMAX; ++h) {
        m[h] = -INFINITY; l[h] = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            qr[h][e] = h < G ? to_float(q[(int64_t)h * D + lane * E + e]) * scale : 0.f;
            o[h][e] = 0.f;
        }
    }
    for (int row = begin + warp; row < end; row += kDecWarps) {
        float kf[E], vf[E];
#pragma unroll
        for (int e = 0; e < E; ++e) {
            kf[e] = to_float(kc[(int64_t)row * D + lane * E + e]);
            vf[e] = to_float(vc[(int64_t)row * D + lane * E + e]);
        }
#pragma unroll
        for (int h = 0; h < GMAX; ++h)
            if (h < G) {
                float y = 0.f;
#pragma unroll
                for (int e = 0; e < E; ++e) y = fmaf(kf[e], qr[h][e], y);
#pragma unroll
                for (int ofs = 16; ofs; ofs >>= 1) y += __shfl_xor_sync(0xffffffffu, y, ofs);
                const float mn = fmaxf(m[h], y);
                const float f = dec_ex2(m[h] - mn), pv = dec_ex2(y - mn);
                l[h] = l[h] * f + pv;
#pragma unroll
                for (int e = 0; e < E; ++e) o[h][e] = o[h][e] * f + pv * vf[e];
                m[h] = mn;
            }
    }
    float *mine = dec_sm + (size_t)warp * GMAX * (D + 2);
#pragma unroll
    for (int h = 0; h < GMAX; ++h) {
        float *rec = mine + h * (D + 2);
#pragma unroll
        for (int e = 0; e < E; ++e) rec[lane * E + e] = o[h][e];
        if (lane == 0) { rec[D] = m[h]; rec[D + 1] = l[h]; }
    }
    merge_and_store<D>(a, dec_sm, GMAX, G, u, x, nblocks);
}

// One block per (unit, head), one thread per column: merges the span records in span order and
// normalises.  Sixteen records are loaded at once (their (max, sum) words are the same for every
// thread of the block, so the merge weights are simply recomputed by each), so a unit of up to
// sixteen spans costs one round trip to memory after the offsets.
template <int D>
__global__ void __launch_bounds__(D)
decode_combine_kernel(DecArgs a)
{
    const refree_params &p = a.p;
    const int Hkv = p.num_kv_heads, G = p.num_q_heads / Hkv;
    const int u = blockIdx.x / G, h = blockIdx.x % G, s = u / Hkv, g = u % Hkv;
    int64_t lo_k, lo_v, len64;
    unit_rows(a, u, lo_k, lo_v, len64);
    const int len = (int)max((int64_t)0, min(len64, (int64_t)a.span * a.gx));
    const int nblocks = ceil_div(len, a.span);
    if (nblocks <= 1) return;                       // written by the attention kernel itself
    const float *rec0 = a.part + ((int64_t)u * a.gx * G + h) * (D + 2);
    const int64_t stride = (int64_t)G * (D + 2);
    float M = -INFINITY, L = 0.f, val = 0.f;
    for (int b0 = 0; b0 < nblocks; b0 += 16) {
        float mm[16], ll[16], vv[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            const bool in = b0 + q < nblocks;
            const float *rec = rec0 + (int64_t)(in ? b0 + q : b0) * stride;
            mm[q] = in ? __ldcg(rec + D) : -INFINITY;
            ll[q] = in ? __ldcg(rec + D + 1) : 0.f;
            vv[q] = in ? __ldcg(rec + threadIdx.x) : 0.f;
        }
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            const float mn = fmaxf(M, mm[q]);
            if (mn > -INFINITY) {
                const float f0 = dec_ex2(M - mn), f1 = dec_ex2(mm[q] - mn);
                val = val * f0 + vv[q] * f1;
                L = L * f0 + ll[q] * f1;
                M = mn;
            }
        }
    }
    a.out[((int64_t)s * p.num_q_heads + g * G + h) * D + native_col(threadIdx.x, a.native)] = L > 0.f ? val / L : 0.f;
}

template <typename T, int D>
cudaError_t run_lanes(const DecArgs &a, dim3 grid, int G, cudaStream_t st)
{
    const int gp = G <= 4 ? 4 : (G <= 8 ? 8 : 16);
    const size_t smem = (size_t)kDecWarps * gp * (D + 2) * sizeof(float);
    cudaError_t e = cudaSuccess;
    if (gp == 4) {
        decode_lanes_kernel<T, D, 4><<<grid, kDecThreads, smem, st>>>(a);
    } else if (gp == 8) {
        decode_lanes_kernel<T, D, 8><<<grid, kDecThreads, smem, st>>>(a);
    } else {
        e = cudaFuncSetAttribute(decode_lanes_kernel<T, D, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        decode_lanes_kernel<T, D, 16><<<grid, kDecThreads, smem, st>>>(a);
    }
    return cudaGetLastError();
}

template <int D>
cudaError_t run_mma(const DecArgs &a, dim3 grid, int G, cudaStream_t st)
{
    // the staging ring and its barriers; the warps' records reuse the ring's space after the loop
    const size_t ring = (size_t)kDecWarps * kDecStages * 2 * 16 * D * 2 + (size_t)kDecWarps * kDecStages * sizeof(uint64_t);
    if (G <= 8) {
        const size_t smem = std::max(ring, (size_t)kDecWarps * 8 * (D + 2) * sizeof(float));
        cudaError_t e = cudaFuncSetAttribute(decode_mma_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        decode_mma_kernel<D, false><<<grid, kDecThreads, smem, st>>>(a);
    } else {
        const size_t smem = std::max(ring, (size_t)kDecWarps * 16 * (D + 2) * sizeof(float));
        cudaError_t e = cudaFuncSetAttribute(decode_mma_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        decode_mma_kernel<D, true><<<grid, kDecThreads, smem, st>>>(a);
    }
    return cudaGetLastError();
}

// blocks per unit and rows per block for a cache of at most max_rows rows per unit
void decode_shape(const refree_params &p, int64_t max_rows, int &gx, int &span)
{
    const int64_t U = (int64_t)p.num_seqs * p.num_kv_heads;
    const int64_t want = std::max<int64_t>(1, sm_count() / U);   // about one block per SM (one wave: prologue and merge are paid once)
    const int64_t by_rows = std::max<int64_t>(1, (max_rows + 127) / 128);      // at least one 16-row block per warp
    gx = (int)std::min<int64_t>(want, by_rows);
    span = (int)(((max_rows + gx - 1) / gx + 15) / 16 * 16);
    span = std::max(span, 16);
}

}  // namespace

size_t decode_workspace_bytes(const refree_params &p, int64_t max_rows)
{
    int gx, span;
    decode_shape(p, max_rows, gx, span);
    return (size_t)p.num_seqs * p.num_q_heads * gx * (p.head_dim + 2) * sizeof(float) + 256;
}

cudaError_t launch_decode_attention(const refree_params &p, const void *q_new, const void *k_c, const void *v_c,
                                    const int64_t *offsets, int64_t max_rows, float *out, void *workspace,
                                    int32_t *dev_status, cudaStream_t st, const int32_t *seq_start,
                                    const int32_t *seq_len, const int32_t *lengths, bool anchor_back)
{
    DecArgs a;
    a.p = p;
    a.q = q_new; a.kc = k_c; a.vc = v_c;
    a.offsets = offsets;
    a.seq_start = seq_start; a.seq_len = seq_len; a.lengths = lengths;
    a.anchor_back = anchor_back ? 1 : 0;
    a.out = out;
    a.part = static_cast<float *>(workspace);
    a.dev_status = dev_status;
    decode_shape(p, max_rows, a.gx, a.span);
    const int U = p.num_seqs * p.num_kv_heads, G = p.num_q_heads / p.num_kv_heads;
    const dim3 grid(a.gx, U);
    const bool f32 = p.dtype == REFREE_DTYPE_F32;
    const bool aligned = !((reinterpret_cast<uintptr_t>(q_new) | reinterpret_cast<uintptr_t>(k_c) |
                            reinterpret_cast<uintptr_t>(v_c)) & 15);
    cudaError_t e;
    if (!f32 && aligned) {
        a.native = 1;
        e = p.head_dim == 64 ? run_mma<64>(a, grid, G, st) : run_mma<128>(a, grid, G, st);
    } else {
        a.native = 0;
        if (p.head_dim == 64) e = f32 ? run_lanes<float, 64>(a, grid, G, st) : run_lanes<__nv_bfloat16, 64>(a, grid, G, st);
        else e = f32 ? run_lanes<float, 128>(a, grid, G, st) : run_lanes<__nv_bfloat16, 128>(a, grid, G, st);
    }
    count_launches(1);
    if (e != cudaSuccess || a.gx == 1) return e;
    if (p.head_dim == 64) decode_combine_kernel<64><<<U * G, 64, 0, st>>>(a);
    else decode_combine_kernel<128><<<U * G, 128, 0, st>>>(a);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace refree
