// Tensor-core scoring path (steps S1-S3) for bf16 caches with head_dim 128.
//
// The window logits S = Q K^T are the one dense contraction of the pass; they run
// on tcgen05.mma with the accumulator in tensor memory, operands staged in shared
// memory by TMA (128-byte swizzle).  A row's softmax normaliser needs all of the
// row, and the column sums need every row's normaliser, so the logits are formed
// twice (storing them would cost more HBM traffic than K itself):
//
//   pass 1  D[row, position] = Q_blk K_tile^T : one thread per query row sums
//           2^(y - c) over the positions it may see (no cross-thread traffic);
//           partial (c, Z) per (CTA, unit) go to the workspace
//   pass 2  on entering a unit, L[row] = log2 sum_i 2^(y_i) is merged from those
//           partials; then D[position, row] = K_tile Q^T : one thread per position
//           sums 2^(y - L[row]) over the rows that see it -> a'[i]  (Eq. 2)
//
// Both passes use the same shared-memory images of Q and K (K-major, so either
// can be the A or the B operand); only the roles swap, which puts each pass's
// reduction inside a thread.  Persistent CTAs (one per SM) take contiguous ranges
// of (unit, tile) items; warp 16 issues TMA, warp 17 issues MMA, warps 0-15 are the
// epilogue: four warpgroups = (accumulator pair) x (64-column half of a 128-column
// accumulator), two accumulators per pair in flight.  The exponentials bind, and with
// four warps per scheduler instead of two their latencies overlap.  In pass 1 the two
// halves of a row keep separate (c, Z) records; in pass 2 warpgroup 0 adds the other
// warpgroups' column sums from shared memory.  Every wait is bounded: on a timeout the CTA records
// REFREE_DEV_TIMEOUT, stops issuing work, and falls through to the common exit
// where tensor memory is released.
#include <cuda.h>

#include <algorithm>
#include <atomic>
#include <mutex>

#include "refree_internal.cuh"

namespace refree {
namespace {

constexpr int kEpiWarps = 16;                 // four warpgroups: (accumulator pair) x (column half)
constexpr int kHalfCols = 64;                 // tensor-memory columns of an accumulator per warpgroup
constexpr int kThreadsTc = (kEpiWarps + 2) * 32;
constexpr int kD = 128;
constexpr int kHalfBytes = kTile * 128;          // one 64-column half of a 128-row tile: 16 KB
constexpr int kTileBytes = 2 * kHalfBytes;       // 32 KB
constexpr int kMaxRowsTc = 512;
constexpr int kMaxCtas = 256;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kZLimit = 1.2676506e30f;         // 2^100: a tile sum above this is redone with a fresh reference

// ------------------------------------------------------------------ PTX ------
__device__ inline uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ inline void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ inline void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ inline void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ inline bool mbar_try(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and raises the CTA's abort flag) when it gives up.
__device__ inline bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try(bar, parity)) return true;
        if (it > 64) {
            if (*abort_flag) return false;
            __nanosleep(it > 4096 ? 256 : 32);
        }
    }
    *abort_flag = 1;
    return false;
}
__device__ inline void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ inline void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ inline void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ inline void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ inline void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}
__device__ inline void tma_load_3d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ inline void tma_load_4d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2, int c3)
{
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

__device__ inline void tmem_alloc(uint32_t *dst_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ inline void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate; issued by one thread.
// The two shared-memory descriptors are passed as their low words (start address
// and leading offset, see desc_lo) plus the common high word: one thread issues
// every MMA of the CTA, so the issue path is kept to a few instructions.
__device__ inline void umma_bf16(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                 uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
                 "setp.ne.b32 p, %5, 0;\n\t"
                 "mov.b64 da, {%1, %3};\n\t"
                 "mov.b64 db, {%2, %3};\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
}
// The mbarrier receives one arrival once every MMA issued so far by this thread has completed.
__device__ inline void umma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Tensor-memory loads are split into issue and wait so that the next chunk can be
// in flight while the current one is consumed.  The wait names the destination
// registers as in/out operands: the compiler must not read them before it.
#define RF_OUT16(r, o) "=r"(r[o+0]), "=r"(r[o+1]), "=r"(r[o+2]), "=r"(r[o+3]), "=r"(r[o+4]), "=r"(r[o+5]), "=r"(r[o+6]), "=r"(r[o+7]), \
                       "=r"(r[o+8]), "=r"(r[o+9]), "=r"(r[o+10]), "=r"(r[o+11]), "=r"(r[o+12]), "=r"(r[o+13]), "=r"(r[o+14]), "=r"(r[o+15])
#define RF_IO16(r, o) "+r"(r[o+0]), "+r"(r[o+1]), "+r"(r[o+2]), "+r"(r[o+3]), "+r"(r[o+4]), "+r"(r[o+5]), "+r"(r[o+6]), "+r"(r[o+7]), \
                      "+r"(r[o+8]), "+r"(r[o+9]), "+r"(r[o+10]), "+r"(r[o+11]), "+r"(r[o+12]), "+r"(r[o+13]), "+r"(r[o+14]), "+r"(r[o+15])
__device__ inline void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : RF_OUT16(r, 0), RF_OUT16(r, 16) : "r"(taddr) : "memory");
}
__device__ inline void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : RF_OUT16(r, 0) : "r"(taddr) : "memory");
}
__device__ inline void tmem_ld_wait(uint32_t (&r)[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" : RF_IO16(r, 0), RF_IO16(r, 16) :: "memory");
}
__device__ inline float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows 128 B
// apart, groups of 8 rows 1024 B apart (the layout TMA writes with SWIZZLE_128B).
// Low word: start address / 16 in bits 0-13, leading byte offset (unused with
// swizzle) in bits 16-29.  A byte offset o (multiple of 16) inside the operand
// adds o / 16 to the low word.  High word: stride byte offset / 16 in bits 0-13,
// descriptor version 1 in bits 14-15, swizzle mode 2 (128 B) in bits 29-31.
__device__ inline uint32_t desc_lo(uint32_t saddr) { return ((saddr & 0x3FFFFu) >> 4) | (1u << 16); }
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128.
__host__ __device__ inline uint32_t make_idesc(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// ---------------------------------------------------------------- shapes -----
struct TcShape {
    int R;        // query rows per unit: G * window
    int Rpad;     // rows of the shared-memory Q image (multiple of 128)
    int rblocks;  // 128-row blocks: pass-1 accumulators per tile (A operands)
    int cblocks;  // pass-2 accumulators per tile
    int ncol;     // pass-2 columns (rows of Q) per accumulator: R / cblocks, at most 128
    int stages;   // K tile ring depth
    int rank4;    // K tensor map has a sequence axis
};

struct TcSmemTail {
    uint64_t k_full[4], k_empty[4], q_full, q_empty, epi_bar;
    uint64_t acc_full[4], acc_empty[4];       // accumulator (warpgroup * 2 + slot): 128 tensor-memory columns each
    uint64_t half_ready[4];                   // pass 2: the other warpgroups have staged their shares of a tile
    uint32_t tmem_base;
    int abort_flag;
    alignas(16) float stage[4][3][kTile];     // pass 2: partial column sums of warpgroups 1..3, four tiles deep
    alignas(16) float lse[kMaxRowsTc];        // pass 2: log2-sum-exp of the unit's rows
    SeqTables seq;
    int32_t start[kMaxSeqs];                  // copy of seq_start
};

struct ItemTc {
    int u, s, g, n, tile_start, tok0, pack;
    int tile, ntiles;      // tile index inside the sequence, tiles of the sequence
};

__device__ inline void fill_seq_fields(ItemTc &it, const TcSmemTail &tl, int Hkv)
{
    it.u = it.s * Hkv + it.g;
    it.n = tl.seq.len[it.s];
    it.tok0 = tl.start[it.s];
    it.pack = tl.seq.pack[it.s];
    it.tile_start = it.tile * kTile;
}

// Items are ordered (sequence, head, tile): a CTA's consecutive items mostly share a unit.
__device__ inline ItemTc decode_item_tc(const TcSmemTail &tl, int B, int Hkv, int item)
{
    const SeqTables &t = tl.seq;
    int lo = 0, hi = B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((int64_t)t.tiles[mid] * Hkv <= item) lo = mid; else hi = mid;
    }
    ItemTc it;
    it.s = lo;
    it.ntiles = t.tiles[lo + 1] - t.tiles[lo];
    const int rem = item - t.tiles[lo] * Hkv;
    it.g = rem / it.ntiles;
    it.tile = rem % it.ntiles;
    fill_seq_fields(it, tl, Hkv);
    return it;
}

// The item after `it` in the same order, without searching or dividing.
__device__ inline void next_item_tc(ItemTc &it, const TcSmemTail &tl, int B, int Hkv)
{
    if (++it.tile < it.ntiles) {
        it.tile_start += kTile;
        return;
    }
    it.tile = 0;
    if (++it.g == Hkv) {
        it.g = 0;
        do { ++it.s; } while (it.s < B - 1 && tl.seq.tiles[it.s + 1] == tl.seq.tiles[it.s]);
        if (it.s >= B) it.s = B - 1;                 // past the end: never used, kept in range
        it.ntiles = tl.seq.tiles[it.s + 1] - tl.seq.tiles[it.s];
    }
    fill_seq_fields(it, tl, Hkv);
}

// first item of CTA c when `items` are split evenly over `ctas`
__device__ __host__ inline int range_begin(int c, int items, int ctas) { return (int)((int64_t)c * items / ctas); }

struct TcArgs {
    refree_params p;
    TcShape sh;
    const int32_t *seq_start, *seq_len;
    float2 *part;        // [2 (ctas + units)][Rpad]: one record per (CTA, unit, column half)
    GroupPartial *groups; // nullable: per 32 positions, exact sum of squared scores for the stopping rule
    uint32_t *flags;     // fused launch: flags[c] == epoch once CTA c has written its pass-1 partials
    uint32_t epoch;
    float *scores;
    int64_t total_tokens;
    int32_t *dev_status;
};

// Barrier among the epilogue warps, built on an mbarrier so that it is bounded like
// every other wait of the kernel (one arrival per warp).
__device__ inline bool epi_sync(TcSmemTail &tl, uint32_t &phase)
{
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(&tl.epi_bar);
    const bool ok = mbar_wait(&tl.epi_bar, phase, &tl.abort_flag);
    phase ^= 1;
    return ok;
}

// Loop state that survives from pass 1 to pass 2 when both run in one launch.
struct RingState { int stage = 0; uint32_t kphase = 0, qphase = 0; };
struct MmaState : RingState { uint32_t cnt0 = 0, cnt1 = 0; int prev_u = -1; };
struct EpiState { uint32_t cnt = 0, ephase = 0; };

// --------------------------------------------------------- producer / MMA -----
template <int PASS>
__device__ inline void producer_loop(const TcArgs &a, const CUtensorMap *mapq, const CUtensorMap *mapk,
                                     unsigned char *smem_q, unsigned char *smem_k, TcSmemTail &tl,
                                     int item0, int item1, RingState &rs)
{
    const TcShape &sh = a.sh;
    const int G = a.p.num_q_heads / a.p.num_kv_heads;
    int cur_u = -1;
    int &stage = rs.stage;
    uint32_t &kphase = rs.kphase, &qphase = rs.qphase;
    bool ok = true;
    ItemTc it = {};
    if (item0 < item1) it = decode_item_tc(tl, a.p.num_seqs, a.p.num_kv_heads, item0);
    for (int item = item0; item < item1 && ok; ++item, next_item_tc(it, tl, a.p.num_seqs, a.p.num_kv_heads)) {
        if (it.u != cur_u) {
            ok = mbar_wait(&tl.q_empty, qphase ^ 1, &tl.abort_flag);
            if (!ok) break;
            mbar_expect_tx(&tl.q_full, (uint32_t)sh.Rpad * 256u);
            const int row0 = (it.s * a.p.num_q_heads + it.g * G) * a.p.window;
            for (int h = 0; h < 2; ++h)
                for (int rb = 0; rb < sh.rblocks; ++rb)
                    tma_load_2d(smem_q + (size_t)h * sh.Rpad * 128 + (size_t)rb * kHalfBytes, mapq, &tl.q_full,
                                h * 64, row0 + rb * kTile);
            qphase ^= 1;
            cur_u = it.u;
        }
        ok = mbar_wait(&tl.k_empty[stage], kphase ^ 1, &tl.abort_flag);
        if (!ok) break;
        mbar_expect_tx(&tl.k_full[stage], (uint32_t)kTileBytes);
        unsigned char *dst = smem_k + (size_t)stage * kTileBytes;
        for (int h = 0; h < 2; ++h) {
            if (sh.rank4)
                tma_load_4d(dst + h * kHalfBytes, mapk, &tl.k_full[stage], h * 64, it.tok0 + it.tile_start, it.g, it.s);
            else
                tma_load_3d(dst + h * kHalfBytes, mapk, &tl.k_full[stage], h * 64, it.tok0 + it.tile_start, it.g);
        }
        if (++stage == sh.stages) { stage = 0; kphase ^= 1; }
    }
    // Before leaving, let every copy this thread started land (bounded): the ring's
    // full barriers complete only when their bytes have arrived.
    if (!ok) {
        for (int s2 = 0; s2 < sh.stages; ++s2)
            for (uint32_t itw = 0; itw < 4096; ++itw) {
                if (mbar_try(&tl.k_full[s2], 0) || mbar_try(&tl.k_full[s2], 1)) break;
                __nanosleep(64);
            }
    }
}

// Accumulators: four of 128 tensor-memory columns.  Block b of a tile (a 128-row
// block of Q in pass 1, a block of `ncol` rows of Q in pass 2) goes to warpgroup
// b & 1, which owns two accumulators and alternates between them, so the MMA of a
// warpgroup's next block runs while it reads the current one, and the two
// warpgroups (hence the two warps sharing an SM sub-partition) drift out of phase.
template <int PASS>
__device__ inline void mma_loop(const TcArgs &a, unsigned char *smem_q, unsigned char *smem_k, TcSmemTail &tl,
                                uint32_t tmem_base, int item0, int item1, MmaState &ms)
{
    const TcShape &sh = a.sh;
    const uint32_t q_lo = desc_lo(smem_u32(smem_q)), k_lo = desc_lo(smem_u32(smem_k));
    const uint32_t q_half = (uint32_t)(sh.Rpad * 128) >> 4;      // distance between the two 64-column halves of Q
    const uint32_t idesc1 = make_idesc(kTile), idesc2 = make_idesc(sh.ncol);
    const int blocks = PASS == 1 ? sh.rblocks : sh.cblocks;
    int cur_u = -1;
    int &stage = ms.stage, &prev_u = ms.prev_u;
    uint32_t &kphase = ms.kphase, &qphase = ms.qphase, &cnt0 = ms.cnt0, &cnt1 = ms.cnt1;   // blocks issued per warpgroup
    bool ok = true;
    ItemTc it = {};
    if (item0 < item1) it = decode_item_tc(tl, a.p.num_seqs, a.p.num_kv_heads, item0);
    for (int item = item0; item < item1 && ok; ++item, next_item_tc(it, tl, a.p.num_seqs, a.p.num_kv_heads)) {
        if (it.u != cur_u) {
            if (prev_u >= 0) umma_commit(&tl.q_empty);     // every MMA on the previous unit's Q has been issued
            ok = mbar_wait(&tl.q_full, qphase, &tl.abort_flag);
            if (!ok) break;
            qphase ^= 1;
            cur_u = it.u;
            prev_u = it.u;
        }
        ok = mbar_wait(&tl.k_full[stage], kphase, &tl.abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t kt_lo = k_lo + (uint32_t)stage * (kTileBytes >> 4);
        for (int b = 0; b < blocks && ok; ++b) {
            const int wg = b & 1;
            const uint32_t cnt = wg ? cnt1 : cnt0;
            const int acc = wg * 2 + (int)(cnt & 1u);
            ok = mbar_wait(&tl.acc_empty[acc], ((cnt >> 1) & 1u) ^ 1u, &tl.abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d0 = tmem_base + (uint32_t)acc * 128u;
            if (PASS == 1) {
                const uint32_t qa = q_lo + (uint32_t)b * (kHalfBytes >> 4);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t h = kk >> 2, ko = (kk & 3) * 2;          // 32 bytes per K step of 16
                    umma_bf16(d0, qa + h * q_half + ko, kt_lo + h * (kHalfBytes >> 4) + ko, kDescHi, idesc1, kk > 0);
                }
            } else {
                const uint32_t qb = q_lo + (uint32_t)b * (uint32_t)(sh.ncol * 128 >> 4);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t h = kk >> 2, ko = (kk & 3) * 2;
                    umma_bf16(d0, kt_lo + h * (kHalfBytes >> 4) + ko, qb + h * q_half + ko, kDescHi, idesc2, kk > 0);
                }
            }
            umma_commit(&tl.acc_full[acc]);
            if (wg) ++cnt1; else ++cnt0;
        }
        umma_commit(&tl.k_empty[stage]);
        if (++stage == sh.stages) { stage = 0; kphase ^= 1; }
    }
}

// ------------------------------------------------------------- epilogues -----
// Pass 1: thread = query row.  Sum of 2^(y - c) over the positions the row sees.
template <bool MASKED>
__device__ inline float row_sum_tile(uint32_t taddr, float scale, float cref, int limit)
{
    float z0 = 0.f, z1 = 0.f;
    const float nc = -cref;
    uint32_t ra[32], rb[32];
    tmem_ld32_issue(taddr, ra);
    tmem_ld32_issue(taddr + 32, rb);
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        uint32_t (&cur)[32] = c ? rb : ra;
        tmem_ld_wait(cur);
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
            float e0 = ex2(fmaf(__uint_as_float(cur[i]), scale, nc));
            float e1 = ex2(fmaf(__uint_as_float(cur[i + 1]), scale, nc));
            if (MASKED) {
                e0 = (c * 32 + i < limit) ? e0 : 0.f;
                e1 = (c * 32 + i + 1 < limit) ? e1 : 0.f;
            }
            z0 += e0;
            z1 += e1;
        }
    }
    return z0 + z1;
}
__device__ inline float row_max_tile(uint32_t taddr, float scale, int limit)
{
    float m = -INFINITY;
    uint32_t ra[32], rb[32];
    tmem_ld32_issue(taddr, ra);
    tmem_ld32_issue(taddr + 32, rb);
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        uint32_t (&cur)[32] = c ? rb : ra;
        tmem_ld_wait(cur);
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (c * 32 + i < limit) m = fmaxf(m, __uint_as_float(cur[i]) * scale);
    }
    return m;
}

__device__ inline void epilogue_pass1(const TcArgs &a, TcSmemTail &tl, uint32_t tmem_base, int item0, int item1,
                                      EpiState &es)
{
    const TcShape &sh = a.sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wg = (warp >> 2) & 1, half = warp >> 3, lane_base = (warp & 3) * 32;
    const float scale = kLog2e * rsqrtf((float)kD);
    const int w = a.p.window;
    int cur_u = -1;
    uint32_t &cnt = es.cnt;                      // blocks this warpgroup has consumed
    // running reference and sum of this thread's rows (row blocks wg and wg + 2) over its half of the columns
    float cref[2] = {-INFINITY, -INFINITY}, zsum[2] = {0.f, 0.f};
    int rmod[2];
    bool rvalid[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int row = (wg + 2 * j) * kTile + lane_base + lane;
        rmod[j] = row % w;                       // offset of the row's query inside the window
        rvalid[j] = row < sh.R;
    }
    bool ok = true;
    auto flush = [&](int u) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int rb = wg + 2 * j;
            const int row = rb * kTile + lane_base + lane;
            if (rb < sh.rblocks && row < sh.R)
                a.part[((int64_t)(blockIdx.x + u) * 2 + half) * sh.Rpad + row] = make_float2(cref[j], zsum[j]);
            cref[j] = -INFINITY;
            zsum[j] = 0.f;
        }
    };
    ItemTc it = {};
    if (item0 < item1) it = decode_item_tc(tl, a.p.num_seqs, a.p.num_kv_heads, item0);
    for (int item = item0; item < item1 && ok; ++item, next_item_tc(it, tl, a.p.num_seqs, a.p.num_kv_heads)) {
        if (it.u != cur_u) {
            if (cur_u >= 0) flush(cur_u);
            cur_u = it.u;
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int rb = wg + 2 * j;
            if (rb >= sh.rblocks || !ok) continue;
            const int acc = wg * 2 + (int)(cnt & 1u);
            ok = mbar_wait(&tl.acc_full[acc], (cnt >> 1) & 1u, &tl.abort_flag);
            if (!ok) continue;
            ++cnt;
            tc_fence_after();
            int limit = kTile;                                  // visible positions of the tile: [0, limit)
            const bool full = it.tile_start + kTile <= it.n - w + 1;   // tile wholly before the window
            if (!full) {
                limit = it.n - w + rmod[j] - it.tile_start + 1;     // up to this row's own position
                limit = (rvalid[j]) ? max(0, min(kTile, limit)) : 0;
            } else if (!rvalid[j]) {
                limit = 0;
            }
            limit = max(0, min(kHalfCols, limit - half * kHalfCols));   // inside this warpgroup's columns
            const bool uniform = __all_sync(0xffffffffu, limit == kHalfCols);
            const uint32_t taddr = tmem_base + (uint32_t)acc * 128u + (uint32_t)(half * kHalfCols) + ((uint32_t)lane_base << 16);
            bool need_max = (cref[j] == -INFINITY) && limit > 0;
            float zt = 0.f;
            for (int attempt = 0; attempt < 2; ++attempt) {
                if (__any_sync(0xffffffffu, need_max)) {
                    const float m = row_max_tile(taddr, scale, limit);
                    if (need_max && m > cref[j]) {
                        zsum[j] = (cref[j] == -INFINITY) ? 0.f : zsum[j] * ex2(cref[j] - m);
                        cref[j] = m;
                    }
                }
                zt = uniform ? row_sum_tile<false>(taddr, scale, cref[j], limit)
                             : row_sum_tile<true>(taddr, scale, cref[j], limit);
                need_max = !(zt <= kZLimit) && limit > 0;       // overflow against a stale reference
                if (attempt == 1 || !__any_sync(0xffffffffu, need_max)) break;
            }
            if (limit > 0) zsum[j] += zt;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tl.acc_empty[acc]);
        }
    }
    if (cur_u >= 0 && ok) flush(cur_u);
}

// Pass 2: thread = position.  Sum over the rows that see it of 2^(y - L[row]).
// One accumulator's share of a warpgroup: ncol_wg columns (a multiple of 16, at most
// 64) in two chunks of up to 32, both loads in flight.
template <bool MASKED>
__device__ inline float col_sum_job(uint32_t taddr, float scale, const float *lse, int rbase, int ncol_wg,
                                    int w, int pos_gap)
{
    // pos_gap = i - (n - w): row r sees position i iff (r mod w) >= pos_gap
    uint32_t ra[32] = {}, rb[32] = {};
    float s0 = 0.f, s1 = 0.f;
    if (ncol_wg >= 32) tmem_ld32_issue(taddr, ra); else tmem_ld16_issue(taddr, ra);
    if (ncol_wg >= 64) tmem_ld32_issue(taddr + 32, rb); else if (ncol_wg > 32) tmem_ld16_issue(taddr + 32, rb);
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        if (c * 32 < ncol_wg) {
            uint32_t (&cur)[32] = c ? rb : ra;
            tmem_ld_wait(cur);
            const int r0 = rbase + c * 32;
            const int width = min(32, ncol_wg - c * 32);
            int rloc = MASKED ? r0 % w : 0;
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
                if (i < width) {
                    const float4 L = *reinterpret_cast<const float4 *>(lse + r0 + i);
                    float e[4];
                    e[0] = ex2(fmaf(__uint_as_float(cur[i]), scale, -L.x));
                    e[1] = ex2(fmaf(__uint_as_float(cur[i + 1]), scale, -L.y));
                    e[2] = ex2(fmaf(__uint_as_float(cur[i + 2]), scale, -L.z));
                    e[3] = ex2(fmaf(__uint_as_float(cur[i + 3]), scale, -L.w));
                    if (MASKED) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if (rloc < pos_gap) e[j] = 0.f;
                            if (++rloc == w) rloc = 0;
                        }
                    }
                    s0 += e[0] + e[2];
                    s1 += e[1] + e[3];
                }
            }
        }
    }
    return s0 + s1;
}

// CTA that owns item x when `items` are split evenly over `ctas` (ctas <= items).
__device__ inline int cta_of_item(int x, int items, int ctas)
{
    return (int)((((int64_t)x + 1) * ctas - 1) / items);
}

__device__ inline void epilogue_pass2(const TcArgs &a, TcSmemTail &tl, uint32_t tmem_base, int item0, int item1,
                                      int items, int ctas, EpiState &es)
{
    const TcShape &sh = a.sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grp = warp >> 2;                                     // 0 finishes the tile, 1..3 stage their shares
    const int wg = grp & 1, half = grp >> 1, lane_base = (warp & 3) * 32;
    const int tid = threadIdx.x;                                   // 0..511
    const float scale = kLog2e * rsqrtf((float)kD);
    const int w = a.p.window, G = a.p.num_q_heads / a.p.num_kv_heads, Hkv = a.p.num_kv_heads;
    const int pos_in_tile = lane_base + lane;
    const bool two_halves = sh.cblocks > 1;                        // both warpgroups contribute to a tile
    int cur_u = -1;
    uint32_t &cnt = es.cnt, &ephase = es.ephase;                   // blocks consumed, phase of the epilogue barrier
    uint32_t tcount = 0;                                           // tiles seen
    // warpgroup 0 finishes a tile one tile late, when the other warpgroups' shares have long been staged
    float pend_acc = 0.f, pend_norm = 0.f;
    float *pend_dst = nullptr;
    GroupPartial *pend_grp = nullptr;
    uint32_t pend_tile = 0;
    bool pending = false, ok = true;
    auto finish_pending = [&]() -> bool {
        if (!pending) return true;
        float tot = pend_acc;
        if (!mbar_wait(&tl.half_ready[pend_tile & 3u], (pend_tile >> 2) & 1u, &tl.abort_flag)) return false;
        tot += tl.stage[pend_tile & 3u][1][pos_in_tile];                       // same accumulators, other columns
        if (two_halves) tot += tl.stage[pend_tile & 3u][0][pos_in_tile] + tl.stage[pend_tile & 3u][2][pos_in_tile];
        float sc = 0.f;
        if (pend_dst) {
            sc = tot * pend_norm;
            if (!isfinite(sc) && a.dev_status) atomicOr(a.dev_status, REFREE_DEV_NONFINITE);
            *pend_dst = sc;
        }
        if (pend_grp) {
            // this warp's 32 positions: largest score, and the exact squares summed at a scale set by it
            const uint32_t bits = (pend_dst && isfinite(sc)) ? mag_bits(sc) : 0u;
            const uint32_t mx = __reduce_max_sync(0xffffffffu, bits);
            unsigned long long sq = sq_fixed(bits, kGroupShift - 2 * max(1, (int)(mx >> 23)));
            for (int o = 16; o; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
            if (lane == 0) { GroupPartial gp; gp.max_bits = mx; gp.pad = 0u; gp.sum = sq; *pend_grp = gp; }
        }
        pending = false;
        return true;
    };
    ItemTc it = {};
    if (item0 < item1) it = decode_item_tc(tl, a.p.num_seqs, Hkv, item0);
    for (int item = item0; item < item1 && ok; ++item, next_item_tc(it, tl, a.p.num_seqs, Hkv)) {
        if (it.u != cur_u) {
            if (!(ok = epi_sync(tl, ephase))) break;               // nobody still reads the previous unit's L
            // L[row] = log2 sum over the row of 2^y, merged from the (reference, sum) pairs that pass 1
            // left per (CTA, unit), in ascending CTA order (the same order in every CTA that needs it)
            const int ts = tl.seq.tiles[it.s + 1] - tl.seq.tiles[it.s];
            const int ib = tl.seq.tiles[it.s] * Hkv + it.g * ts;
            const int c_lo = cta_of_item(ib, items, ctas), c_hi = cta_of_item(ib + ts - 1, items, ctas);
            if (a.flags) {
                // one launch for both passes: the partials of this unit come from CTAs that may still be in
                // pass 1; wait (bounded) until each of them has published
                for (int c = c_lo + tid; c <= c_hi; c += kEpiWarps * 32) {
                    bool seen = false;
                    for (uint32_t spin = 0; spin < kSpinLimit && !seen; ++spin) {
                        uint32_t v;
                        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(a.flags + c) : "memory");
                        seen = v == a.epoch;
                        if (!seen) { if (tl.abort_flag) break; __nanosleep(spin > 64 ? 256 : 32); }
                    }
                    if (!seen) tl.abort_flag = 1;
                }
                if (!(ok = epi_sync(tl, ephase))) break;
                if (tl.abort_flag) { ok = false; break; }
            }
            for (int r = tid; r < sh.R; r += kEpiWarps * 32) {
                float M = -INFINITY, Z = 0.f;
                const int s_hi = 2 * (c_hi + it.u) + 1;             // records: (CTA, column half)
                for (int s0 = 2 * (c_lo + it.u); s0 <= s_hi; s0 += 8) {
                    float2 pr[8];                                  // eight independent loads in flight
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        pr[q] = (s0 + q <= s_hi) ? __ldcg(&a.part[(int64_t)(s0 + q) * sh.Rpad + r])
                                                 : make_float2(-INFINITY, 0.f);
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        if (pr[q].y > 0.f) {
                            if (pr[q].x > M) { Z = Z * ex2(M - pr[q].x) + pr[q].y; M = pr[q].x; }
                            else Z += pr[q].y * ex2(pr[q].x - M);
                        }
                    }
                }
                tl.lse[r] = Z > 0.f ? M + log2f(Z) : INFINITY;     // a row that sees nothing adds 2^(-inf) = 0
            }
            if (!(ok = epi_sync(tl, ephase))) break;
            cur_u = it.u;
        }
        const int i = it.tile_start + pos_in_tile;
        const int pos_gap = i - (it.n - w);
        // tile wholly before the window and wholly inside the sequence: every row sees every position
        const bool full = it.tile_start + kTile <= it.n - w + 1;
        float accv = 0.f;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int cb = wg + 2 * j;
            if (cb >= sh.cblocks || !ok) continue;
            const int acc = wg * 2 + (int)(cnt & 1u);
            ok = mbar_wait(&tl.acc_full[acc], (cnt >> 1) & 1u, &tl.abort_flag);
            if (!ok) continue;
            ++cnt;
            tc_fence_after();
            const int c_off = half * kHalfCols, ncol_h = max(0, min(kHalfCols, sh.ncol - c_off));
            const uint32_t taddr = tmem_base + (uint32_t)acc * 128u + (uint32_t)c_off + ((uint32_t)lane_base << 16);
            if (ncol_h > 0)
                accv += full ? col_sum_job<false>(taddr, scale, tl.lse, cb * sh.ncol + c_off, ncol_h, w, pos_gap)
                             : col_sum_job<true>(taddr, scale, tl.lse, cb * sh.ncol + c_off, ncol_h, w, pos_gap);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tl.acc_empty[acc]);
        }
        if (!ok) break;
        // Warpgroup 0 completes the previous tile only now, after it has handed this tile's accumulators
        // back, so the MMA of the tile after next overlaps the completion.  The others can then be at most
        // three tiles past the staging slot read here (the accumulators of tile t + 3 need this warpgroup's
        // release of tile t + 1, which comes after this point): four slots.
        if (grp == 0 && !(ok = finish_pending())) break;
        if (grp == 0) {
            const int cnt_i = max(1, min(min(w, it.n), it.n - i));
            pend_acc = accv;
            pend_norm = 1.f / ((float)cnt_i * (float)G);
            pend_dst = i < it.n ? a.scores + (int64_t)it.g * a.total_tokens + it.pack + i : nullptr;
            pend_grp = a.groups ? a.groups + ((int64_t)tl.seq.tiles[it.s] * Hkv + (int64_t)it.g * it.ntiles + it.tile) * 4 +
                                      (warp & 3)
                                : nullptr;
            pend_tile = tcount;
            pending = true;
        } else if (wg == 0 || two_halves) {
            // the second accumulator pair has blocks (and is paced by the MMA warp) only with several column blocks
            tl.stage[tcount & 3u][grp - 1][pos_in_tile] = accv;
            __syncwarp();
            if (lane == 0) mbar_arrive(&tl.half_ready[tcount & 3u]);
        }
        ++tcount;
    }
    if (grp == 0 && ok) finish_pending();
}

// ---------------------------------------------------------------- kernels ----
template <int PASS>
__global__ void __launch_bounds__(kThreadsTc, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap mapq, const __grid_constant__ CUtensorMap mapk, TcArgs a)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const TcShape &sh = a.sh;
    unsigned char *smem_q = smem;
    unsigned char *smem_k = smem + (size_t)sh.Rpad * 256;
    TcSmemTail &tl = *reinterpret_cast<TcSmemTail *>(smem_k + (size_t)sh.stages * kTileBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == kEpiWarps * 32) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapq) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapk) : "memory");
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < 4; ++s) { mbar_init(&tl.k_full[s], 1); mbar_init(&tl.k_empty[s], 1); }
        mbar_init(&tl.q_full, 1);
        mbar_init(&tl.q_empty, 1);
        for (int b = 0; b < 4; ++b) { mbar_init(&tl.acc_full[b], 1); mbar_init(&tl.acc_empty[b], kEpiWarps / 2); }
        // stagers: the other column half of the first accumulator pair, plus both halves of the second pair
        for (int b = 0; b < 4; ++b) mbar_init(&tl.half_ready[b], a.sh.cblocks > 1 ? 12 : 4);
        mbar_init(&tl.epi_bar, kEpiWarps);
        tl.abort_flag = 0;
        fence_barrier_init();
    }
    for (int t = threadIdx.x; t < a.p.num_seqs; t += kThreadsTc) tl.start[t] = a.seq_start[t];
    build_seq_tables(tl.seq, a.seq_len, a.p.num_seqs);       // ends with __syncthreads()
    if (warp == kEpiWarps + 1) tmem_alloc(&tl.tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tl.tmem_base;

    // ranges over min(grid, items) CTAs, so that every CTA that has a range has a non-empty one
    const int items = tl.seq.tiles[a.p.num_seqs] * a.p.num_kv_heads;
    const int ctas = max(1, min((int)gridDim.x, items));
    const bool active = (int)blockIdx.x < ctas;
    const int item0 = active ? range_begin(blockIdx.x, items, ctas) : 0;
    const int item1 = active ? range_begin(blockIdx.x + 1, items, ctas) : 0;

    // PASS 1 or 2: that pass alone; PASS 3: both passes in this launch (all CTAs co-resident)
    if (warp < kEpiWarps) {
        EpiState es;
        if (PASS != 2) epilogue_pass1(a, tl, tmem_base, item0, item1, es);
        if (PASS == 3) {
            // publish: this CTA's partials are in memory
            __threadfence();
            epi_sync(tl, es.ephase);
            if (threadIdx.x == 0)
                asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(a.flags + blockIdx.x), "r"(a.epoch) : "memory");
        }
        if (PASS != 1) epilogue_pass2(a, tl, tmem_base, item0, item1, items, ctas, es);
    } else if (warp == kEpiWarps) {
        if (lane == 0) {
            RingState rs;
            if (PASS != 2) producer_loop<1>(a, &mapq, &mapk, smem_q, smem_k, tl, item0, item1, rs);
            if (PASS != 1) producer_loop<2>(a, &mapq, &mapk, smem_q, smem_k, tl, item0, item1, rs);
        }
    } else {
        if (lane == 0) {
            MmaState ms;
            if (PASS != 2) mma_loop<1>(a, smem_q, smem_k, tl, tmem_base, item0, item1, ms);
            if (PASS != 1) mma_loop<2>(a, smem_q, smem_k, tl, tmem_base, item0, item1, ms);
        }
    }
    __syncwarp();
    // Common exit.  In the normal case the epilogue has consumed every accumulator,
    // which implies every MMA and every copy has completed.
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (threadIdx.x == 0 && tl.abort_flag && a.dev_status) atomicOr(a.dev_status, REFREE_DEV_TIMEOUT);
    if (warp == kEpiWarps + 1) tmem_dealloc(tmem_base, 512);
}

// ------------------------------------------------------------------ host -----
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

bool shape_for(const refree_params &p, TcShape &sh)
{
    if (p.dtype != REFREE_DTYPE_BF16 || p.head_dim != kD) return false;
    const int G = p.num_q_heads / p.num_kv_heads;
    const int64_t R = (int64_t)G * p.window;
    if (R < 32 || R > kMaxRowsTc) return false;
    sh.R = (int)R;
    sh.cblocks = (sh.R + kTile - 1) / kTile;
    if (sh.R % (16 * sh.cblocks) != 0) return false;      // accumulators are read in chunks of 16 columns
    sh.ncol = sh.R / sh.cblocks;
    sh.rblocks = (sh.R + kTile - 1) / kTile;
    sh.Rpad = sh.rblocks * kTile;
    sh.stages = sh.Rpad <= 256 ? 4 : 2;
    sh.rank4 = p.k_stride_seq != 0;
    return true;
}

size_t smem_bytes(const TcShape &sh)
{
    return 1024 + (size_t)sh.Rpad * 256 + (size_t)sh.stages * kTileBytes + sizeof(TcSmemTail);
}

}  // namespace

bool score_tc_supported(const refree_params &p)
{
    TcShape sh;
    if (!shape_for(p, sh)) return false;
    if (p.kv_tokens <= 0 || p.kv_tokens > 0x7fffffffLL) return false;
    return encode_fn() != nullptr;
}

cudaError_t launch_score_tc(const refree_params &p, const void *q_win, const void *k,
                            const int32_t *seq_start, const int32_t *seq_len,
                            int64_t total_tokens, float *scores, char *ws, const Workspace &lay,
                            int32_t *dev_status, cudaStream_t st, GroupPartial *groups)
{
    TcShape sh;
    if (!shape_for(p, sh)) return cudaErrorInvalidValue;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
    CUtensorMap mapq, mapk;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)p.num_seqs * p.num_q_heads * p.window};
        const cuuint64_t strides[1] = {(cuuint64_t)kD * 2};
        const cuuint32_t box[2] = {64, kTile}, estr[2] = {1, 1};
        if (enc(&mapq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(q_win), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        const cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)p.kv_tokens, (cuuint64_t)p.num_kv_heads, (cuuint64_t)p.num_seqs};
        const cuuint64_t strides[3] = {(cuuint64_t)p.k_stride_tok * 2, (cuuint64_t)p.k_stride_head * 2,
                                       (cuuint64_t)p.k_stride_seq * 2};
        const cuuint32_t box[4] = {64, kTile, 1, 1}, estr[4] = {1, 1, 1, 1};
        if (enc(&mapk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, sh.rank4 ? 4 : 3, const_cast<void *>(k), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    static int sm_count[64] = {};
    static bool coop_ok[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (sm_count[dev] == 0) {
        int n = 0;
        e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(score_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(score_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(score_tc_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
        if (e != cudaSuccess) return e;
        int coop = 0;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess) coop = 0;
        coop_ok[dev] = coop != 0;
        sm_count[dev] = std::min(n, kMaxCtas);
    }
    const int64_t max_items = (total_tokens / kTile + p.num_seqs) * p.num_kv_heads;
    const int ctas = (int)std::max<int64_t>(1, std::min<int64_t>(sm_count[dev], max_items));
    TcArgs a;
    a.p = p;
    a.sh = sh;
    a.seq_start = seq_start;
    a.seq_len = seq_len;
    a.part = reinterpret_cast<float2 *>(ws + lay.part_off);
    a.groups = groups;
    a.scores = scores;
    a.total_tokens = total_tokens;
    a.dev_status = dev_status;
    const size_t smem = smem_bytes(sh);
    if (smem > 232448) return cudaErrorInvalidValue;
    a.flags = nullptr;
    a.epoch = 0;
    if (coop_ok[dev]) {
        // Both passes in one cooperative launch (co-residency of all CTAs is what makes the wait of pass 2
        // on other CTAs' pass 1 safe).  The flags hold a per-call token, so a workspace left over from an
        // earlier call needs no clearing.
        static std::atomic<uint32_t> token{0x5eed1234u};
        uint32_t epoch = token.fetch_add(1u, std::memory_order_relaxed) + 1u;
        if (epoch == 0u) epoch = token.fetch_add(1u, std::memory_order_relaxed) + 1u;
        a.flags = reinterpret_cast<uint32_t *>(ws + lay.cnt_off);
        a.epoch = epoch;
        void *args[3] = {(void *)&mapq, (void *)&mapk, (void *)&a};
        const cudaError_t ce = cudaLaunchCooperativeKernel((const void *)score_tc_kernel<3>, dim3(ctas), dim3(kThreadsTc),
                                                           args, smem, st);
        if (ce == cudaSuccess) {
            count_launches(1);
            return cudaGetLastError();
        }
        (void)cudaGetLastError();        // not launchable as one grid here: fall back to one launch per pass
        a.flags = nullptr;
    }
    score_tc_kernel<1><<<ctas, kThreadsTc, smem, st>>>(mapq, mapk, a);
    score_tc_kernel<2><<<ctas, kThreadsTc, smem, st>>>(mapq, mapk, a);
    count_launches(2);
    return cudaGetLastError();
}

}  // namespace refree
