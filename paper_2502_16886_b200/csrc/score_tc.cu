// Tensor-core scoring path (steps S1-S3) for bf16 caches with head_dim 128.
//
// The window logits S = Q K^T are the one dense contraction of the pass; they run
// on tcgen05.mma with the accumulator in tensor memory, operands staged in shared
// memory by TMA (128-byte swizzle, no multicast).  A row's softmax normaliser needs
// all of the row, and the column sums need every row's normaliser, so the logits are
// formed twice (storing them would cost more HBM traffic than K itself):
//
//   pass 1  D[row, position] = Q_blk K_tile^T (M = 128 rows, N = 128 positions): one
//           thread per query row sums 2^(y - c) over the positions it may see;
//           partial (c, Z) per (CTA, unit, column half) go to the workspace
//   pass 2  on entering a unit, L[row] = log2 sum_i 2^(y_i) is merged from those
//           partials; then D[position, row] = K_tile Q^T (M = 128 positions, N = up to
//           256 rows in ONE product per k-step): one thread per position sums
//           2^(y - L[row]) over the rows that see it -> a'[i]  (Eq. 2)
//
// Both passes use the same shared-memory images of Q and K (K-major, so either can be
// the A or the B operand); only the roles swap, which puts each pass's reduction
// inside a thread.  Measured on this part, consecutive products into one accumulator
// cost about 137 cycles at N = 256 (93 % of the nominal rate) but 116-120 cycles at
// N = 128 (55 %), and alternating between accumulators from one product to the next
// is slower still; so pass 2 uses one wide product per k-step, and every accumulator
// is handed back to the MMA warp as soon as its values sit in registers, before any
// exponential is taken.
//
// Persistent CTAs (one per SM) take contiguous ranges of (unit, tile) items; warp 16
// issues TMA, warp 17 issues MMA, warps 0-15 are the epilogue, warp 18 moves rows of
// another layer, warps 19 and 20 finish the column pass.  Pass 1: four accumulators of
// 128 columns, warps = (accumulator pair) x (64-column half).  Pass 2: two accumulators
// of 256 columns, two groups of eight warps take the products in turn, a warp = (lane
// quarter) x (half of the product's columns); the finishing warps add the warps' shares
// of a tile, store the scores and the records of the stopping rule, tile by tile in
// turn (one warp could not keep up with the sixteen: it paced the pass).  Every
// wait is bounded: on a timeout the CTA records REFREE_DEV_TIMEOUT, stops issuing work,
// and falls through to the common exit where tensor memory is released.
#include <cuda.h>

#include <algorithm>
#include <atomic>
#include <mutex>

#include "refree_internal.cuh"
#include "select_groups.cuh"

namespace refree {
namespace {

constexpr int kEpiWarps = 16;
constexpr int kFinishWarps = 1;                      // warps that finish the column pass, taking its tiles in turn
constexpr int kThreadsTc = (kEpiWarps + 3 + kFinishWarps) * 32;    // + TMA warp, MMA warp, copy warp, finishing warps
constexpr int kMaxCopySlots = 10;
constexpr int kMaxCopyUnits = 1024;                 // units whose running budget sum fits the CTA's table
constexpr int kD = 128;
constexpr int kCopyRows = 32;                       // rows of one piece of the in-kernel row copy
constexpr int kCopySlot = kCopyRows * kD * 2;       // 8 KB
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
// K tiles carry an L2 eviction priority: the row pass reads a tile first (keep it: the column pass comes back for
// it), the column pass reads it last (let it go first).
__device__ inline void tma_load_3d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2, uint64_t pol)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "l"(pol) : "memory");
}
__device__ inline void tma_load_4d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2, int c3, uint64_t pol)
{
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(pol) : "memory");
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
__device__ inline void tmem_ld_wait16(uint32_t (&r)[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" : RF_IO16(r, 0) :: "memory");
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
    int cblocks;  // pass-2 products per k-step and tile: 1 up to 256 rows, else 2
    int ncol;     // pass-2 columns (rows of Q) per product: a multiple of 16, cblocks * ncol >= R
    int stages;   // K tile ring depth
    int rank4;    // K tensor map has a sequence axis
};

// What the consumers of an item (one tile of one unit) need to know about it.  The TMA thread walks the
// items and leaves one record per item in a ring in shared memory, written before the item's K tile is
// requested; the MMA thread and the epilogue warps read it after the barriers that order them behind
// that request, instead of each walking the item list in registers.
struct ItemInfo {
    int32_t u;        // unit = sequence * Hkv + head
    int32_t g;        // KV head
    int32_t n;        // length of the sequence
    int32_t tile;     // tile index inside the sequence
    int32_t ntiles;   // tiles of the sequence
    int32_t pack;     // positions before the sequence in the packed score array
    int32_t ib;       // index of the unit's first item
    int32_t new_unit; // the item is the first of its unit in this CTA's pass
};
constexpr int kInfoRing = 16;   // the TMA thread runs at most ring stages + accumulators in flight ahead of the epilogue
// Pass 2: tiles whose column sums wait for the finishing warp.  That warp is slower per tile than the sixteen
// epilogue warps together while rows are being copied beside them, and catches up under the row pass that follows:
// the ring is deep enough to let it fall behind instead of holding the epilogue back.
constexpr int kStageSlots = 8;

struct TcSmemTail {
    uint64_t k_full[4], k_empty[4], q_full, q_empty, epi_bar;
    uint64_t acc_full[4], acc_empty[4];       // pass 1: accumulator (pair * 2 + slot), 128 tensor-memory columns each
    uint64_t p2_full[2], p2_empty[2];         // pass 2: accumulators of 256 columns, one per group of eight warps
    uint64_t chunk_ready[kStageSlots];        // pass 2: every share of a tile has been staged
    uint64_t stage_free[kStageSlots];         // pass 2: the finishing warp has read the slot
    uint64_t c_full[kMaxCopySlots];           // row copy: a piece has landed in its slot
    uint32_t tmem_base;
    int abort_flag;
    alignas(16) ItemInfo info[kInfoRing];
    alignas(16) ItemInfo stage_info[kStageSlots];      // pass 2: the staged tile's record, copied beside its sums
    alignas(16) float stage[kStageSlots][4][kTile];    // pass 2: partial column sums (share = product * 2 + column half)
    alignas(16) float lse[kMaxRowsTc];        // pass 2: log2-sum-exp of the unit's rows
};

// Per-sequence tables of the CTA behind the tail, sized by the number of sequences:
// pack[B + 1], tiles[B + 1] (running sums of lengths and of tiles), len[B], start[B], ne[B + 1] (non-empty
// sequences before each).
struct SeqView {
    const int32_t *pack, *tiles, *len, *start, *ne;
};

struct ItemTc {
    int u, s, g, n, tile_start, tok0, pack;
    int tile, ntiles;      // tile index inside the sequence, tiles of the sequence
};

__device__ inline void fill_seq_fields(ItemTc &it, const SeqView &sv, int Hkv)
{
    it.u = it.s * Hkv + it.g;
    it.n = sv.len[it.s];
    it.tok0 = sv.start[it.s];
    it.pack = sv.pack[it.s];
    it.tile_start = it.tile * kTile;
}

// Items are ordered (sequence, head, tile): a CTA's consecutive items mostly share a unit.
__device__ inline ItemTc decode_item_tc(const SeqView &sv, int B, int Hkv, int item)
{
    int lo = 0, hi = B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((int64_t)sv.tiles[mid] * Hkv <= item) lo = mid; else hi = mid;
    }
    ItemTc it;
    it.s = lo;
    it.ntiles = sv.tiles[lo + 1] - sv.tiles[lo];
    const int rem = item - sv.tiles[lo] * Hkv;
    it.g = rem / it.ntiles;
    it.tile = rem % it.ntiles;
    fill_seq_fields(it, sv, Hkv);
    return it;
}

// The item after `it` in the same order, without searching or dividing.
__device__ inline void next_item_tc(ItemTc &it, const SeqView &sv, int B, int Hkv)
{
    if (++it.tile < it.ntiles) {
        it.tile_start += kTile;
        return;
    }
    it.tile = 0;
    if (++it.g == Hkv) {
        it.g = 0;
        do { ++it.s; } while (it.s < B - 1 && sv.tiles[it.s + 1] == sv.tiles[it.s]);
        if (it.s >= B) it.s = B - 1;                 // past the end: never used, kept in range
        it.ntiles = sv.tiles[it.s + 1] - sv.tiles[it.s];
    }
    fill_seq_fields(it, sv, Hkv);
}

// Split of the items over the CTAs.  A change of unit inside a CTA's range costs about as much as a few tiles (the
// accumulators drain, the new unit's normalisers are merged from the partials, Q is reloaded), so what the CTAs
// get equal shares of is  items + pen * (changes of unit): item i of the o-th non-empty unit sits at
// v = i + pen * o, and CTA c takes the items with v in [c V / ctas, (c + 1) V / ctas).  `pen` stays below the
// share of a CTA, so no CTA's range is empty.
constexpr int kUnitChangeTiles = 3;
struct Split {
    int items, ctas, pen, Hkv;
    int64_t V;
};

__device__ inline Split make_split(const SeqView &sv, int B, int Hkv, int grid)
{
    Split sp;
    sp.Hkv = Hkv;
    sp.items = sv.tiles[B] * Hkv;
    sp.ctas = max(1, min(grid, sp.items));
    sp.pen = max(0, min(kUnitChangeTiles, sp.items / sp.ctas - 1));
    sp.V = (int64_t)sp.items + (int64_t)sp.pen * max(0, sv.ne[B] * Hkv - 1);
    return sp;
}

// first item of CTA c (c == ctas: one past the last item)
__device__ inline int range_begin(const Split &sp, const SeqView &sv, int B, int c)
{
    const int64_t t = ((int64_t)c * sp.V + sp.ctas - 1) / sp.ctas;      // smallest v of the CTA's share
    if (t >= sp.V) return sp.items;
    const int Hkv = sp.Hkv;
    auto key = [&](int q) { return (int64_t)sv.tiles[q] * Hkv + (int64_t)sp.pen * sv.ne[q] * Hkv; };   // v of a sequence's first item
    int lo = 0, hi = B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (key(mid) <= t) lo = mid; else hi = mid;
    }
    const int nt = sv.tiles[lo + 1] - sv.tiles[lo];
    const int64_t rel = t - key(lo);
    const int g = (int)min((int64_t)(Hkv - 1), rel / (nt + sp.pen));
    const int64_t r = rel - (int64_t)g * (nt + sp.pen);
    // a v that falls between two units belongs to the first item of the second
    return sv.tiles[lo] * Hkv + g * nt + (int)min(r, (int64_t)nt);
}

// CTA that owns item x of unit u
__device__ inline int cta_of_item(const Split &sp, const SeqView &sv, int x, int u)
{
    const int ord = sv.ne[u / sp.Hkv] * sp.Hkv + u % sp.Hkv;
    const int64_t v = (int64_t)x + (int64_t)sp.pen * ord;
    return (int)min((int64_t)(sp.ctas - 1), v * sp.ctas / sp.V);
}

struct TcArgs {
    refree_params p;
    TcShape sh;
    const int32_t *seq_start, *seq_len;
    // Pass 1 writes the partials of layer `la`, pass 2 reads those of layer `lb` and writes its scores (the same
    // layer when both passes of one layer run in a launch; consecutive layers of a run otherwise).
    float2 *part_a;      // [2 (ctas + units)][Rpad]: one record per (CTA, unit, column half)
    const float2 *part_b;
    GroupPartial *groups; // nullable: per 32 positions, exact sum of squared scores for the stopping rule
    float *scores;
    uint32_t *flags;     // one layer per launch: flags[c] != 0 once CTA c has written its pass-1 partials (zeroed before the launch)
    int64_t total_tokens;
    int32_t *dev_status;
    // Stopping rule inside the launch (position ranking per head): the finishing warp that completes a unit's
    // last tile (a ticket per unit) evaluates the rule from the unit's records.  All nullable.
    int32_t *sel_lengths;      // [units] budgets out
    Cut *sel_cuts;             // [units]
    uint32_t *tickets;         // [2 units] tiles finished per unit, then the unit's largest score; zero when the launch begins
    uint32_t *tickets_next;    // [2 units] those of the launch that follows, cleared by this one
    int dependent;             // launched with programmatic stream serialization: wait for the launch before
    TcCopyJob cj;          // rows of an earlier layer to move while this layer is scored (nslots == 0: none)
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

// Loop state that survives from pass 1 to pass 2 when both run in one launch.  `icount` numbers the
// items a role has gone through in this launch (both passes): its low bits index the info ring.
struct RingState { int stage = 0; uint32_t kphase = 0, qphase = 0, icount = 0; };
struct MmaState : RingState { uint32_t cnt0 = 0, cnt1 = 0, cnt2 = 0; bool first = true; };
struct EpiState { uint32_t ephase = 0, icount = 0; };

// --------------------------------------------------------- producer / MMA -----
__device__ inline void producer_loop(const TcArgs &a, const CUtensorMap *mapq, const CUtensorMap *mapk,
                                     unsigned char *smem_q, unsigned char *smem_k, TcSmemTail &tl, const SeqView &sv,
                                     int item0, int item1, RingState &rs, bool reverse)
{
    const TcShape &sh = a.sh;
    const int G = a.p.num_q_heads / a.p.num_kv_heads, Hkv = a.p.num_kv_heads;
    int cur_u = -1;
    int &stage = rs.stage;
    uint32_t &kphase = rs.kphase, &qphase = rs.qphase;
    bool ok = true;
    // The column pass walks its items backwards: the row pass before it (of the same layer, in this launch or at
    // the end of the launch before) left its last K tiles in L2, and those are asked for first.
    uint64_t pol;
    if (reverse) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    else asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    ItemTc it = {};
    if (item0 < item1) it = decode_item_tc(sv, a.p.num_seqs, Hkv, reverse ? item1 - 1 : item0);
    for (int x = 0; x < item1 - item0 && ok; ++x) {
        if (x > 0) {
            if (reverse) it = decode_item_tc(sv, a.p.num_seqs, Hkv, item1 - 1 - x);
            else next_item_tc(it, sv, a.p.num_seqs, Hkv);
        }
        const bool new_unit = it.u != cur_u;
        // the ring entry was last used sixteen items ago, which every consumer has long left behind
        ItemInfo &inf = tl.info[rs.icount++ & (kInfoRing - 1)];
        inf.u = it.u; inf.g = it.g; inf.n = it.n; inf.tile = it.tile; inf.ntiles = it.ntiles; inf.pack = it.pack;
        inf.ib = sv.tiles[it.s] * Hkv + it.g * it.ntiles;
        inf.new_unit = new_unit ? 1 : 0;
        // The K tile first: the MMA thread learns of a unit change from the record, which it reads once
        // the tile has landed, and only then gives the Q image back.
        ok = mbar_wait(&tl.k_empty[stage], kphase ^ 1, &tl.abort_flag);
        if (!ok) break;
        mbar_expect_tx(&tl.k_full[stage], (uint32_t)kTileBytes);     // (release) orders the record before the tile
        unsigned char *dst = smem_k + (size_t)stage * kTileBytes;
        for (int h = 0; h < 2; ++h) {
            if (sh.rank4)
                tma_load_4d(dst + h * kHalfBytes, mapk, &tl.k_full[stage], h * 64, it.tok0 + it.tile_start, it.g, it.s, pol);
            else
                tma_load_3d(dst + h * kHalfBytes, mapk, &tl.k_full[stage], h * 64, it.tok0 + it.tile_start, it.g, pol);
        }
        if (new_unit) {
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

// Pass 1.  Block b of a tile (a 128-row block of Q) goes to accumulator pair b & 1, which owns two
// accumulators of 128 columns and alternates between them: the MMA of a pair's next block runs while
// the epilogue reads the current one.
__device__ inline void mma_loop_pass1(const TcArgs &a, unsigned char *smem_q, unsigned char *smem_k, TcSmemTail &tl,
                                      uint32_t tmem_base, int nitems, MmaState &ms)
{
    const TcShape &sh = a.sh;
    const uint32_t q_lo = desc_lo(smem_u32(smem_q)), k_lo = desc_lo(smem_u32(smem_k));
    const uint32_t q_half = (uint32_t)(sh.Rpad * 128) >> 4;      // distance between the two 64-column halves of Q
    const uint32_t idesc = make_idesc(kTile);
    int &stage = ms.stage;
    uint32_t &kphase = ms.kphase, &qphase = ms.qphase, &cnt0 = ms.cnt0, &cnt1 = ms.cnt1;   // blocks issued per pair
    bool ok = true;
    for (int item = 0; item < nitems && ok; ++item) {
        ok = mbar_wait(&tl.k_full[stage], kphase, &tl.abort_flag);
        if (!ok) break;
        tc_fence_after();
        if (tl.info[ms.icount++ & (kInfoRing - 1)].new_unit) {
            if (!ms.first) umma_commit(&tl.q_empty);       // every MMA on the previous unit's Q has been issued
            ms.first = false;
            ok = mbar_wait(&tl.q_full, qphase, &tl.abort_flag);
            if (!ok) break;
            qphase ^= 1;
            tc_fence_after();
        }
        const uint32_t kt_lo = k_lo + (uint32_t)stage * (kTileBytes >> 4);
        for (int b = 0; b < sh.rblocks && ok; ++b) {
            const int pair = b & 1;
            const uint32_t cnt = pair ? cnt1 : cnt0;
            const int acc = pair * 2 + (int)(cnt & 1u);
            ok = mbar_wait(&tl.acc_empty[acc], ((cnt >> 1) & 1u) ^ 1u, &tl.abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d0 = tmem_base + (uint32_t)acc * 128u;
            const uint32_t qa = q_lo + (uint32_t)b * (kHalfBytes >> 4);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t h = kk >> 2, ko = (kk & 3) * 2;          // 32 bytes per K step of 16
                umma_bf16(d0, qa + h * q_half + ko, kt_lo + h * (kHalfBytes >> 4) + ko, kDescHi, idesc, kk > 0);
            }
            umma_commit(&tl.acc_full[acc]);
            if (pair) ++cnt1; else ++cnt0;
        }
        umma_commit(&tl.k_empty[stage]);
        if (++stage == sh.stages) { stage = 0; kphase ^= 1; }
    }
}

// The pass-2 accumulators (two of 256 columns) cover the same tensor-memory columns as the four of
// pass 1: before the first pass-2 product, every pass-1 accumulator must have been handed back.
__device__ inline bool drain_pass1(TcSmemTail &tl, const MmaState &ms)
{
    bool ok = true;
    for (int pair = 0; pair < 2 && ok; ++pair) {
        const uint32_t cnt = pair ? ms.cnt1 : ms.cnt0;
        for (int slot = 0; slot < 2 && ok; ++slot) {
            const uint32_t uses = (cnt + (slot ? 0u : 1u)) >> 1;
            if (uses) ok = mbar_wait(&tl.acc_empty[pair * 2 + slot], (uses - 1u) & 1u, &tl.abort_flag);
        }
    }
    if (ok) tc_fence_after();
    return ok;
}

// The other way round (a launch that finishes one layer and then begins the next).
__device__ inline bool drain_pass2(TcSmemTail &tl, const MmaState &ms)
{
    bool ok = true;
    for (int buf = 0; buf < 2 && ok; ++buf) {
        const uint32_t uses = (ms.cnt2 + (buf ? 0u : 1u)) >> 1;
        if (uses) ok = mbar_wait(&tl.p2_empty[buf], (uses - 1u) & 1u, &tl.abort_flag);
    }
    if (ok) tc_fence_after();
    return ok;
}

// Pass 2: D[position, row] = K_tile Q^T, `ncol` rows of Q per product.
__device__ inline void mma_loop_pass2(const TcArgs &a, unsigned char *smem_q, unsigned char *smem_k, TcSmemTail &tl,
                                      uint32_t tmem_base, int nitems, MmaState &ms)
{
    const TcShape &sh = a.sh;
    const uint32_t q_lo = desc_lo(smem_u32(smem_q)), k_lo = desc_lo(smem_u32(smem_k));
    const uint32_t q_half = (uint32_t)(sh.Rpad * 128) >> 4;
    const uint32_t idesc = make_idesc(sh.ncol);
    int &stage = ms.stage;
    uint32_t &kphase = ms.kphase, &qphase = ms.qphase, &cnt = ms.cnt2;
    bool ok = true;
    for (int item = 0; item < nitems && ok; ++item) {
        ok = mbar_wait(&tl.k_full[stage], kphase, &tl.abort_flag);
        if (!ok) break;
        tc_fence_after();
        if (tl.info[ms.icount++ & (kInfoRing - 1)].new_unit) {
            if (!ms.first) umma_commit(&tl.q_empty);
            ms.first = false;
            ok = mbar_wait(&tl.q_full, qphase, &tl.abort_flag);
            if (!ok) break;
            qphase ^= 1;
            tc_fence_after();
        }
        const uint32_t kt_lo = k_lo + (uint32_t)stage * (kTileBytes >> 4);
        for (int cb = 0; cb < sh.cblocks && ok; ++cb) {
            const int buf = (int)(cnt & 1u);
            ok = mbar_wait(&tl.p2_empty[buf], ((cnt >> 1) & 1u) ^ 1u, &tl.abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d0 = tmem_base + (uint32_t)buf * 256u;
            const uint32_t qb = q_lo + (uint32_t)cb * (uint32_t)(sh.ncol * 128 >> 4);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t h = kk >> 2, ko = (kk & 3) * 2;
                umma_bf16(d0, kt_lo + h * (kHalfBytes >> 4) + ko, qb + h * q_half + ko, kDescHi, idesc, kk > 0);
            }
            umma_commit(&tl.p2_full[buf]);
            ++cnt;
        }
        umma_commit(&tl.k_empty[stage]);
        if (++stage == sh.stages) { stage = 0; kphase ^= 1; }
    }
}

// ------------------------------------------------------------- epilogues -----
// Pass 1: thread = query row, 64 logits of the row in registers.
template <bool MASKED>
__device__ inline float row_sum_regs(const uint32_t (&ra)[32], const uint32_t (&rb)[32], float scale, float cref, int limit)
{
    float z0 = 0.f, z1 = 0.f;
    const float nc = -cref;
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        const uint32_t (&cur)[32] = c ? rb : ra;
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
__device__ inline float row_max_regs(const uint32_t (&ra)[32], const uint32_t (&rb)[32], float scale, int limit)
{
    float m = -INFINITY;
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        const uint32_t (&cur)[32] = c ? rb : ra;
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (c * 32 + i < limit) m = fmaxf(m, __uint_as_float(cur[i]) * scale);
    }
    return m;
}

__device__ inline void epilogue_pass1(const TcArgs &a, TcSmemTail &tl, uint32_t tmem_base, int nitems, EpiState &es)
{
    const TcShape &sh = a.sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pair = (warp >> 2) & 1, half = warp >> 3, lane_base = (warp & 3) * 32;
    const float scale = kLog2e * rsqrtf((float)kD);
    const int w = a.p.window;
    int cur_u = -1;
    uint32_t cnt = 0;                            // blocks this accumulator pair has consumed
    // running reference and sum of this thread's rows (row blocks pair and pair + 2) over its half of the columns
    float cref[2] = {-INFINITY, -INFINITY}, zsum[2] = {0.f, 0.f};
    int rmod[2];
    bool rvalid[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int row = (pair + 2 * j) * kTile + lane_base + lane;
        rmod[j] = row % w;                       // offset of the row's query inside the window
        rvalid[j] = row < sh.R;
    }
    bool ok = true;
    auto flush = [&](int u) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int rb = pair + 2 * j;
            const int row = rb * kTile + lane_base + lane;
            if (rb < sh.rblocks && row < sh.R)
                a.part_a[((int64_t)(blockIdx.x + u) * 2 + half) * sh.Rpad + row] = make_float2(cref[j], zsum[j]);
            cref[j] = -INFINITY;
            zsum[j] = 0.f;
        }
    };
    for (int item = 0; item < nitems && ok; ++item) {
        const ItemInfo *inf = &tl.info[es.icount++ & (kInfoRing - 1)];
        int tile_start = 0, n = 0;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int rb = pair + 2 * j;
            if (rb >= sh.rblocks || !ok) continue;
            const int acc = pair * 2 + (int)(cnt & 1u);
            ok = mbar_wait(&tl.acc_full[acc], (cnt >> 1) & 1u, &tl.abort_flag);
            if (!ok) continue;
            ++cnt;
            tc_fence_after();
            const uint32_t taddr = tmem_base + (uint32_t)acc * 128u + (uint32_t)(half * 64) + ((uint32_t)lane_base << 16);
            uint32_t ra[32], rb2[32];
            tmem_ld32_issue(taddr, ra);
            tmem_ld32_issue(taddr + 32, rb2);
            tmem_ld_wait(ra);
            tmem_ld_wait(rb2);
            // the logits are in registers: the accumulator goes back to the MMA warp before any arithmetic
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tl.acc_empty[acc]);
            if (j == 0 || sh.rblocks <= 2) {
                // the item's record is valid from the first accumulator of the item on
                const int u = inf->u;
                if (u != cur_u) {
                    if (cur_u >= 0) flush(cur_u);
                    cur_u = u;
                }
                tile_start = inf->tile * kTile;
                n = inf->n;
            }
            const bool full = tile_start + kTile <= n - w + 1;      // tile wholly before the window
            int limit = kTile;                                  // visible positions of the tile: [0, limit)
            if (!full) {
                limit = n - w + rmod[j] - tile_start + 1;           // up to this row's own position
                limit = rvalid[j] ? max(0, min(kTile, limit)) : 0;
            } else if (!rvalid[j]) {
                limit = 0;
            }
            limit = max(0, min(64, limit - half * 64));         // inside this warp's columns
            const bool uniform = __all_sync(0xffffffffu, limit == 64);
            bool need_max = (cref[j] == -INFINITY) && limit > 0;
            float zt = 0.f;
            for (int attempt = 0; attempt < 2; ++attempt) {
                if (__any_sync(0xffffffffu, need_max)) {
                    const float m = row_max_regs(ra, rb2, scale, limit);
                    if (need_max && m > cref[j]) {
                        zsum[j] = (cref[j] == -INFINITY) ? 0.f : zsum[j] * ex2(cref[j] - m);
                        cref[j] = m;
                    }
                }
                zt = uniform ? row_sum_regs<false>(ra, rb2, scale, cref[j], limit)
                             : row_sum_regs<true>(ra, rb2, scale, cref[j], limit);
                need_max = !(zt <= kZLimit) && limit > 0;       // overflow against a stale reference
                if (attempt == 1 || !__any_sync(0xffffffffu, need_max)) break;
            }
            if (limit > 0) zsum[j] += zt;
        }
    }
    if (cur_u >= 0 && ok) flush(cur_u);
}

// Pass 2: thread = position.  One product's share of a warp: WIDTH columns (rows of Q; 16, 32, 48 or 64) come
// from tensor memory 16 at a time, the next 16 in flight while 2^(y - L[row]) is summed over the current ones;
// the accumulator is handed back as soon as the last load has landed.
// rbase = row of the first column; pos_gap = i - (n - w): row r sees position i iff (r mod w) >= pos_gap.
template <bool MASKED>
__device__ inline void col_sum16(const uint32_t (&cur)[32], float scale, const float *lse, int r0, int R, int w,
                                 int pos_gap, float &s0, float &s1)
{
    int rloc = MASKED ? r0 % w : 0;
#pragma unroll
    for (int i = 0; i < 16; i += 4) {
        const float4 L = *reinterpret_cast<const float4 *>(lse + r0 + i);
        float e[4];
        e[0] = ex2(fmaf(__uint_as_float(cur[i]), scale, -L.x));
        e[1] = ex2(fmaf(__uint_as_float(cur[i + 1]), scale, -L.y));
        e[2] = ex2(fmaf(__uint_as_float(cur[i + 2]), scale, -L.z));
        e[3] = ex2(fmaf(__uint_as_float(cur[i + 3]), scale, -L.w));
        if (MASKED) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (rloc < pos_gap || r0 + i + j >= R) e[j] = 0.f;     // hidden by causality, or padding
                if (++rloc == w) rloc = 0;
            }
        }
        s0 += e[0] + e[2];
        s1 += e[1] + e[3];
    }
}

// One product's share of a warp: `nch` chunks of 16 columns (rows of Q) come from tensor memory one chunk at a
// time, the next in flight while 2^(y - L[row]) is summed over the current one; the accumulator is handed back
// as soon as the last load has landed.
template <bool MASKED>
__device__ inline float col_job(int nch, uint32_t taddr, uint64_t *empty_bar, int lane, float scale, const float *lse,
                                int rbase, int R, int w, int pos_gap)
{
    uint32_t b0[32], b1[32];               // only the first 16 of each are used
    float s0 = 0.f, s1 = 0.f;
    auto release = [&]() {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar);
    };
    if (nch <= 0) { release(); return 0.f; }
    tmem_ld16_issue(taddr, b0);
    tmem_ld_wait16(b0);
    for (int c = 0; c < nch; c += 2) {
        if (c + 1 < nch) tmem_ld16_issue(taddr + 16 * (c + 1), b1); else release();
        col_sum16<MASKED>(b0, scale, lse, rbase + 16 * c, R, w, pos_gap, s0, s1);
        if (c + 1 < nch) {
            tmem_ld_wait16(b1);
            if (c + 2 < nch) tmem_ld16_issue(taddr + 16 * (c + 2), b0); else release();
            col_sum16<MASKED>(b1, scale, lse, rbase + 16 * (c + 1), R, w, pos_gap, s0, s1);
            if (c + 2 < nch) tmem_ld_wait16(b0);
        }
    }
    return s0 + s1;
}

// L[row] = log2 sum over the row of 2^y for the rows of unit u, merged from the (reference, sum) pairs that pass 1
// left per (CTA, unit, column half), in ascending record order (the same in every CTA that needs the unit).
// Called by all epilogue threads; `ib` = index of the unit's first item, `ts` = its tiles.
__device__ inline bool merge_unit_lse(const TcArgs &a, TcSmemTail &tl, const SeqView &sv, const Split &sp, int u, int ib,
                                      int ts, uint32_t &ephase)
{
    const TcShape &sh = a.sh;
    const int tid = threadIdx.x;
    const int c_lo = cta_of_item(sp, sv, ib, u), c_hi = cta_of_item(sp, sv, ib + ts - 1, u);
    if (a.flags) {
        // one launch for both passes: the partials of this unit come from CTAs that may still be in pass 1;
        // wait (bounded) until each of them has published
        for (int c = c_lo + tid; c <= c_hi; c += kEpiWarps * 32) {
            bool seen = false;
            for (uint32_t spin = 0; spin < kSpinLimit && !seen; ++spin) {
                uint32_t v;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(a.flags + c) : "memory");
                seen = v != 0u;
                if (!seen) { if (tl.abort_flag) break; __nanosleep(spin > 64 ? 256 : 32); }
            }
            if (!seen) tl.abort_flag = 1;
        }
        if (!epi_sync(tl, ephase)) return false;
        if (tl.abort_flag) return false;
    }
    // two threads per row when there are enough threads: even and odd records, then one exchange
    const int per_row = 2 * sh.R <= kEpiWarps * 32 ? 2 : 1;
    const int r = tid / per_row, sub = tid % per_row;
    float M = -INFINITY, Z = 0.f;
    if (r < sh.R) {
        const int s_hi = 2 * (c_hi + u) + 1;               // records: (CTA, column half)
        constexpr int kBatch = 12;                          // independent loads in flight per thread
        for (int s0 = 2 * (c_lo + u) + sub; s0 <= s_hi; s0 += kBatch * per_row) {
            float2 pr[kBatch];
#pragma unroll
            for (int q = 0; q < kBatch; ++q)
                pr[q] = (s0 + q * per_row <= s_hi) ? __ldcg(&a.part_b[(int64_t)(s0 + q * per_row) * sh.Rpad + r])
                                                   : make_float2(-INFINITY, 0.f);
#pragma unroll
            for (int q = 0; q < kBatch; ++q) {
                if (pr[q].y > 0.f) {
                    if (pr[q].x > M) { Z = Z * ex2(M - pr[q].x) + pr[q].y; M = pr[q].x; }
                    else Z += pr[q].y * ex2(pr[q].x - M);
                }
            }
        }
    }
    if (per_row == 2) {
        const float M2 = __shfl_xor_sync(0xffffffffu, M, 1), Z2 = __shfl_xor_sync(0xffffffffu, Z, 1);
        // (even records) then (odd records), in that order on both lanes
        const float Ma = sub ? M2 : M, Za = sub ? Z2 : Z, Mb = sub ? M : M2, Zb = sub ? Z : Z2;
        if (Zb > 0.f) {
            if (Za > 0.f) {
                if (Mb > Ma) { Z = Za * ex2(Ma - Mb) + Zb; M = Mb; }
                else { Z = Za + Zb * ex2(Mb - Ma); M = Ma; }
            } else { Z = Zb; M = Mb; }
        } else { Z = Za; M = Ma; }
    }
    // a row that sees nothing adds 2^(-inf) = 0
    if (r < sh.R && sub == 0) tl.lse[r] = Z > 0.f ? M + log2f(Z) : INFINITY;
    // columns past the unit's rows (padding of the last product) never count
    for (int rr = sh.R + tid; rr < sh.cblocks * sh.ncol; rr += kEpiWarps * 32) tl.lse[rr] = INFINITY;
    return epi_sync(tl, ephase);
}

// Pass 2, the sixteen epilogue warps.  Two groups of eight warps take the products in turn (product j goes to
// group j & 1 and to accumulator j & 1), so the groups run out of step: while one waits for its next accumulator,
// stages a tile or refills its pipeline, the other keeps the exponential units busy.  Inside a group a warp is
// (lane quarter) x (half of the product's columns); it leaves its share of the tile's column sums in a staging
// slot, and the finishing warp adds the shares.
__device__ inline void epilogue_pass2(const TcArgs &a, TcSmemTail &tl, const SeqView &sv, uint32_t tmem_base,
                                      int item0, int nitems, const Split &sp, EpiState &es)
{
    const TcShape &sh = a.sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int group = (warp >> 2) & 1, half = warp >> 3;
    const int lane_base = (warp & 3) * 32;
    const float scale = kLog2e * rsqrtf((float)kD);
    const int w = a.p.window;
    const int pos_in_tile = lane_base + lane;
    const int c_width = sh.ncol >> 1, c_begin = half * c_width;     // this warp's columns of a product
    const bool exact = sh.cblocks * sh.ncol == sh.R;               // no padding columns in the products
    uint32_t &ephase = es.ephase;                                  // phase of the epilogue barrier
    uint32_t gcnt = 0;                                             // products this group has taken
    int next_change = 0;                                           // item (relative) at which the next unit begins
    bool ok = true;
    for (int item = 0; item < nitems && ok; ++item) {
        const ItemInfo *inf = &tl.info[es.icount++ & (kInfoRing - 1)];
        if (item == next_change) {   // `item` counts the pass's items in the order they come: from the CTA's last one backwards
            // A unit begins: all sixteen warps meet (the two groups share L), whichever group takes the item's
            // products.  The unit is looked up in the sequence tables, not in the item's record, which a warp
            // that takes none of the item's products has no barrier to wait for.  The normalisers do not wait
            // for the tile either: the partials come from the row pass, not from anything this pass loads.
            const ItemTc it = decode_item_tc(sv, a.p.num_seqs, a.p.num_kv_heads, item0 + (nitems - 1 - item));
            if (item > 0 && !(ok = epi_sync(tl, ephase))) break;   // nobody still reads the previous unit's L
            ok = merge_unit_lse(a, tl, sv, sp, it.u, sv.tiles[it.s] * a.p.num_kv_heads + it.g * it.ntiles, it.ntiles,
                                ephase);
            if (!ok) break;
            next_change = item + it.tile + 1;                      // the unit's earlier tiles follow
        }
        for (int cb = 0; cb < sh.cblocks && ok; ++cb) {
            const uint32_t j = (uint32_t)item * (uint32_t)sh.cblocks + (uint32_t)cb;      // product index in this pass
            if ((int)(j & 1u) != group) continue;
            ok = mbar_wait(&tl.p2_full[group], gcnt & 1u, &tl.abort_flag);
            if (!ok) break;
            ++gcnt;
            tc_fence_after();
            // the item's record is valid once one of its products is
            const int tile_start = inf->tile * kTile, n = inf->n;
            const int pos_gap = tile_start + pos_in_tile - (n - w);
            // tile wholly before the window and wholly inside the sequence: every row sees every position
            const bool full = tile_start + kTile <= n - w + 1 && exact;
            const uint32_t taddr = tmem_base + (uint32_t)group * 256u + (uint32_t)c_begin + ((uint32_t)lane_base << 16);
            const float part = full ? col_job<false>(c_width >> 4, taddr, &tl.p2_empty[group], lane, scale, tl.lse,
                                                     cb * sh.ncol + c_begin, sh.R, w, pos_gap)
                                    : col_job<true>(c_width >> 4, taddr, &tl.p2_empty[group], lane, scale, tl.lse,
                                                    cb * sh.ncol + c_begin, sh.R, w, pos_gap);
            // the slot's previous tile (four tiles ago) has been read by the finishing warp
            const uint32_t slot = (uint32_t)item % kStageSlots;
            if (!(ok = mbar_wait(&tl.stage_free[slot], (((uint32_t)item / kStageSlots) & 1u) ^ 1u, &tl.abort_flag))) break;
            tl.stage[slot][cb * 2 + half][pos_in_tile] = part;
            // the tile's record travels with its sums (the ring it came from may be reused before the tile is finished)
            if (cb == 0 && half == 0 && lane_base == 0 && lane < 8)
                reinterpret_cast<uint32_t *>(&tl.stage_info[slot])[lane] = reinterpret_cast<const uint32_t *>(inf)[lane];
            __syncwarp();
            if (lane == 0) mbar_arrive(&tl.chunk_ready[slot]);
        }
    }
}

// Pass 2, the finishing warp: a'[i] = (sum of the warps' shares, in a fixed order) / (G * rows that see i)  (Eq. 2), the score
// store, and per 32 positions the record the stopping rule reads.  `icount0` = items the roles have gone through
// before this pass (their ring index).
__device__ inline void finisher_pass2(const TcArgs &a, TcSmemTail &tl, int nitems, uint32_t icount0, int which)
{
    const int lane = threadIdx.x & 31;
    const int w = a.p.window;
    const float g = (float)(a.p.num_q_heads / a.p.num_kv_heads);
    const bool two_products = a.sh.cblocks > 1;
    // This CTA's tiles of a unit are counted once, when its run of them ends: the warp that brings the unit's count
    // to its number of tiles sees every other tile's scores and records (fenced before their counts were added)
    // and evaluates the stopping rule for the unit.
    int run_u = -1, run_n = 0, run_ntiles = 0, run_ib = 0, run_tiles = 0;
    uint32_t run_max = 0;                       // largest score of the run (bit pattern)
    const float *run_dst = nullptr;
    const int U = a.p.num_seqs * a.p.num_kv_heads;
    auto close_run = [&]() {
        if (run_u < 0 || run_tiles == 0) return;
        if (lane == 0) atomicMax(&a.tickets[U + run_u], run_max);      // the unit's largest score, beside its count
        __threadfence();
        __syncwarp();
        uint32_t old = 0;
        if (lane == 0) old = atomicAdd(&a.tickets[run_u], (uint32_t)run_tiles);
        old = __shfl_sync(0xffffffffu, old, 0);
        if ((int)old + run_tiles == run_ntiles) {
            __threadfence();
            uint32_t umax = 0;
            if (lane == 0) umax = atomicMax(&a.tickets[U + run_u], 0u);
            umax = __shfl_sync(0xffffffffu, umax, 0);
            const Cut cut = select_unit_from_groups_warp(a.p, run_dst, run_n, a.groups + (int64_t)run_ib * 4, umax);
            if (lane == 0) {
                a.sel_lengths[run_u] = cut.b;
                if (a.sel_cuts) a.sel_cuts[run_u] = cut;
            }
        }
        run_tiles = 0;
    };
    // tile t of the pass belongs to finishing warp t mod kFinishWarps; a warp counts and closes its own runs of a
    // unit's tiles, and the unit is complete when the warps' counts add up to its tiles
    for (int t = which; t < nitems; t += kFinishWarps) {
        const uint32_t slot = (uint32_t)t % kStageSlots;
        if (!mbar_wait(&tl.chunk_ready[slot], ((uint32_t)t / kStageSlots) & 1u, &tl.abort_flag)) return;
        const ItemInfo *inf = &tl.stage_info[slot];
        const int n = inf->n, tile = inf->tile;
        const int inf_u = inf->u, inf_ntiles = inf->ntiles, inf_ib = inf->ib;     // the record may be reused after the slot is freed
        float *dst = a.scores + (int64_t)inf->g * a.total_tokens + inf->pack;
        GroupPartial *grp = a.groups ? a.groups + ((int64_t)inf->ib + tile) * 4 : nullptr;
        uint32_t tile_max = 0;
        if ((reinterpret_cast<uintptr_t>(dst + (int64_t)tile * kTile) & 15) == 0) {
            // A lane takes four consecutive positions: the shares come as 16-byte loads, the scores leave as one
            // 16-byte store, and the 32 positions of a record are eight neighbouring lanes.  (Few instructions that
            // go through the memory pipe: the sixteen epilogue warps keep it busy, and this warp paces the pass.)
            const int p0 = 4 * lane, i0 = tile * kTile + p0;
            float tot[4];
            {
                const float4 x = *reinterpret_cast<const float4 *>(&tl.stage[slot][0][p0]);
                const float4 y = *reinterpret_cast<const float4 *>(&tl.stage[slot][1][p0]);
                tot[0] = x.x + y.x; tot[1] = x.y + y.y; tot[2] = x.z + y.z; tot[3] = x.w + y.w;
            }
            if (two_products) {
                const float4 x = *reinterpret_cast<const float4 *>(&tl.stage[slot][2][p0]);
                const float4 y = *reinterpret_cast<const float4 *>(&tl.stage[slot][3][p0]);
                tot[0] += x.x; tot[1] += x.y; tot[2] += x.z; tot[3] += x.w;
                tot[0] += y.x; tot[1] += y.y; tot[2] += y.z; tot[3] += y.w;
            }
            float sc[4];
            uint32_t bits[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int i = i0 + k;
                const int cnt_i = max(1, min(min(w, n), n - i));
                sc[k] = i < n ? tot[k] / ((float)cnt_i * g) : 0.f;
                bits[k] = (i < n && isfinite(sc[k])) ? mag_bits(sc[k]) : 0u;
                if (i < n && !isfinite(sc[k]) && a.dev_status) atomicOr(a.dev_status, REFREE_DEV_NONFINITE);
            }
            if (i0 + 3 < n) {
                *reinterpret_cast<float4 *>(dst + i0) = make_float4(sc[0], sc[1], sc[2], sc[3]);
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (i0 + k < n) dst[i0 + k] = sc[k];
            }
            if (grp) {
                // 32 positions = lanes 8q .. 8q + 7: largest score, and the exact squares summed at a scale set by it
                uint32_t mx = max(max(bits[0], bits[1]), max(bits[2], bits[3]));
#pragma unroll
                for (int o = 1; o < 8; o <<= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                const int shift = kGroupShift - 2 * max(1, (int)(mx >> 23));
                unsigned long long sq = sq_fixed(bits[0], shift) + sq_fixed(bits[1], shift) + sq_fixed(bits[2], shift) +
                                        sq_fixed(bits[3], shift);
#pragma unroll
                for (int o = 1; o < 8; o <<= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
                if ((lane & 7) == 0) { GroupPartial gp; gp.max_bits = mx; gp.pad = 0u; gp.sum = sq; grp[lane >> 3] = gp; }
                tile_max = __reduce_max_sync(0xffffffffu, mx);
            }
        } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int pos = q * 32 + lane, i = tile * kTile + pos;
            float tot = tl.stage[slot][0][pos];
            tot += tl.stage[slot][1][pos];
            if (two_products) {
                tot += tl.stage[slot][2][pos];
                tot += tl.stage[slot][3][pos];
            }
            const int cnt_i = max(1, min(min(w, n), n - i));
            float sc = 0.f;
            if (i < n) {
                sc = tot / ((float)cnt_i * g);
                if (!isfinite(sc) && a.dev_status) atomicOr(a.dev_status, REFREE_DEV_NONFINITE);
                dst[i] = sc;
            }
            if (grp) {
                // these 32 positions: largest score, and the exact squares summed at a scale set by it
                const uint32_t bits = (i < n && isfinite(sc)) ? mag_bits(sc) : 0u;
                const uint32_t mx = __reduce_max_sync(0xffffffffu, bits);
                tile_max = max(tile_max, mx);
                unsigned long long sq = sq_fixed(bits, kGroupShift - 2 * max(1, (int)(mx >> 23)));
                for (int o = 16; o; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
                if (lane == 0) { GroupPartial gp; gp.max_bits = mx; gp.pad = 0u; gp.sum = sq; grp[q] = gp; }
            }
        }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&tl.stage_free[slot]);
        if (a.tickets) {
            if (inf_u != run_u) {
                close_run();
                run_u = inf_u; run_n = n; run_ntiles = inf_ntiles; run_ib = inf_ib; run_dst = dst; run_tiles = 0;
                run_max = 0;
            }
            ++run_tiles;
            run_max = max(run_max, tile_max);
        }
    }
    if (a.tickets) close_run();
}

// ------------------------------------------------------------- row copy -----
// Compaction of another layer by one warp of the scoring CTA (position ranking: the kept rows of a unit
// are rows [0, head) and [n - (b - head), n) of its cache, contiguous in memory when a unit's rows are).
// Destination rows are cut into pieces of 32 rows; piece k belongs to CTA k mod grid, and inside the CTA
// to one lane of the warp, which owns a slot of shared memory.  A piece travels global -> shared -> global
// with the bulk-copy engine (no tensor map, no multicast): the load is signalled on the slot's mbarrier,
// the store is a bulk group.  Nothing here touches the registers or pipes of the scoring warps.
__device__ inline void copy_loop(const TcArgs &a, TcSmemTail &tl, const SeqView &sv, unsigned char *smem_c, int32_t *coff)
{
    const TcCopyJob &cj = a.cj;
    const int lane = threadIdx.x & 31;
    const int Hkv = a.p.num_kv_heads, U = a.p.num_seqs * Hkv;
    // running sum of the budgets (clamped to [0, n]); a budget out of range is reported
    int carry = 0;
    bool bad = false;
    for (int base = 0; base < U; base += 32) {
        const int u = base + lane;
        int b = 0;
        if (u < U) {
            b = cj.lengths[u];
            const int n = sv.len[u / Hkv];
            if (b < 0 || b > n) { bad = true; b = max(0, min(b, n)); }
        }
        int x = b;
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if (u < U) coff[u] = carry + x - b;
        carry += __shfl_sync(0xffffffffu, x, 31);
    }
    if (lane == 0) coff[U] = carry;
    __syncwarp();
    bad = __any_sync(0xffffffffu, bad);
    const int64_t rows = min((int64_t)carry, cj.capacity_rows);
    if (blockIdx.x == 0) {
        if (cj.offsets_out)
            for (int u = lane; u <= U; u += 32) cj.offsets_out[u] = coff[u];
        if (lane == 0 && (bad || (int64_t)carry > cj.capacity_rows) && a.dev_status)
            atomicOr(a.dev_status, REFREE_DEV_CAPACITY);
    }
    const int nslots = cj.nslots;
    if (lane >= nslots || rows <= 0) return;

    // Lane j owns slot j and every nslots-th piece of this CTA, and runs its own load -> wait -> store -> wait
    // chain; the lanes drift apart, which spreads the requests in time.
    const int64_t k_tok = a.p.k_stride_tok * 2, v_tok = a.p.v_stride_tok * 2;      // bytes (bf16)
    const int64_t pieces_per_array = (rows + kCopyRows - 1) / kCopyRows, pieces = 2 * pieces_per_array;
    int64_t next = blockIdx.x + (int64_t)lane * gridDim.x;      // next piece of this lane
    const int64_t step = (int64_t)nslots * gridDim.x;
    int r_cur = 0, r_end = 0, u_cur = 0, arr = 0;      // rows [r_cur, r_end) of the current piece still to cut
    unsigned char *slot = smem_c + (size_t)lane * kCopySlot;
    uint64_t *bar = &tl.c_full[lane];
    // the moved rows are used once: they should not push the scored layer's K tiles out of L2
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    uint32_t loads = 0;
    bool ok = true;
    while (ok) {
        // the next run of rows that is contiguous in source and destination
        bool has = true;
        if (r_cur >= r_end) {
            if (next >= pieces) {
                has = false;
            } else {
                arr = next >= pieces_per_array ? 1 : 0;
                const int64_t pk = next - (arr ? pieces_per_array : 0);
                next += step;
                r_cur = (int)(pk * kCopyRows);
                r_end = (int)min((int64_t)r_cur + kCopyRows, rows);
                int lo = 0, hi = U;                             // largest u with coff[u] <= r_cur
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (coff[mid] <= r_cur) lo = mid; else hi = mid;
                }
                u_cur = lo;
            }
        }
        if (!has) break;
        unsigned char *dst = nullptr;
        uint32_t bytes = 0;
        if (has) {
            while (coff[u_cur + 1] <= r_cur) ++u_cur;           // skip units that keep nothing (r_cur < rows <= coff[U])
            const int b = coff[u_cur + 1] - coff[u_cur], t = r_cur - coff[u_cur];
            const int sq = u_cur / Hkv, g = u_cur - sq * Hkv;
            const int n = sv.len[sq], head = min(b, min(a.p.sink, n));
            int src_row, run;
            if (t < head) { src_row = t; run = head - t; }
            else { src_row = n - b + t; run = b - t; }
            run = min(run, r_end - r_cur);
            const int64_t tok = (int64_t)sv.start[sq] + src_row;
            const unsigned char *src =
                arr == 0 ? cj.k + ((int64_t)sq * a.p.k_stride_seq + (int64_t)g * a.p.k_stride_head) * 2 + tok * k_tok
                         : cj.v + ((int64_t)sq * a.p.v_stride_seq + (int64_t)g * a.p.v_stride_head) * 2 + tok * v_tok;
            dst = (arr ? cj.v_out : cj.k_out) + (int64_t)r_cur * (kD * 2);
            bytes = (uint32_t)run * (kD * 2);
            r_cur += run;
            mbar_expect_tx(bar, bytes);
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                         ::"r"(smem_u32(slot)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(pol) : "memory");
            ok = mbar_wait(bar, loads & 1u, &tl.abort_flag);
            ++loads;
            if (ok) {
                asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
                             ::"l"(dst), "r"(smem_u32(slot)), "r"(bytes), "l"(pol) : "memory");
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            }
        }
        ok = ok && !tl.abort_flag;
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// ---------------------------------------------------------------- kernels ----
// MODE 1: pass 1 alone; 2: pass 2 alone; 3: both passes of one layer (cooperative launch: pass 2 waits for the
// pass-1 flags of other CTAs); 4: pass 2 of one layer (maps `_b`), then pass 1 of the next (maps `_a`) - the
// steady state of a run of layers, where the partials pass 2 reads were completed by the launch before.
template <int MODE>
__global__ void __launch_bounds__(kThreadsTc, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap mapq_a, const __grid_constant__ CUtensorMap mapk_a,
                const __grid_constant__ CUtensorMap mapq_b, const __grid_constant__ CUtensorMap mapk_b, TcArgs a)
{
    constexpr bool P1 = MODE != 2, P2 = MODE != 1;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const TcShape &sh = a.sh;
    unsigned char *smem_q = smem;
    unsigned char *smem_k = smem + (size_t)sh.Rpad * 256;
    unsigned char *smem_c = smem_k + (size_t)sh.stages * kTileBytes;        // pieces of the row copy
    TcSmemTail &tl = *reinterpret_cast<TcSmemTail *>(smem_c + (size_t)a.cj.nslots * kCopySlot);
    int32_t *tab = reinterpret_cast<int32_t *>(&tl + 1);
    const int B = a.p.num_seqs;
    int32_t *t_pack = tab, *t_tiles = tab + (B + 1), *t_len = tab + 2 * (B + 1), *t_start = tab + 2 * (B + 1) + B;
    int32_t *t_ne = tab + 4 * B + 2;
    int32_t *coff = tab + 5 * B + 3;             // row copy: running sum of the budgets, units + 1 entries
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == kEpiWarps * 32) {
        if (P1) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapq_a) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapk_a) : "memory");
        }
        if (P2) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapq_b) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&mapk_b) : "memory");
        }
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < 4; ++s) { mbar_init(&tl.k_full[s], 1); mbar_init(&tl.k_empty[s], 1); }
        mbar_init(&tl.q_full, 1);
        mbar_init(&tl.q_empty, 1);
        for (int b = 0; b < 4; ++b) { mbar_init(&tl.acc_full[b], 1); mbar_init(&tl.acc_empty[b], kEpiWarps / 2); }
        for (int b = 0; b < 2; ++b) { mbar_init(&tl.p2_full[b], 1); mbar_init(&tl.p2_empty[b], kEpiWarps / 2); }
        for (int b = 0; b < kStageSlots; ++b) {
            mbar_init(&tl.chunk_ready[b], (kEpiWarps / 2) * a.sh.cblocks);      // eight warps stage a share per product
            mbar_init(&tl.stage_free[b], 1);
        }
        mbar_init(&tl.epi_bar, kEpiWarps);
        for (int b = 0; b < kMaxCopySlots; ++b) mbar_init(&tl.c_full[b], 1);
        tl.abort_flag = 0;
        fence_barrier_init();
    }
    for (int t = threadIdx.x; t < B; t += kThreadsTc) t_start[t] = a.seq_start[t];
    if (threadIdx.x == 32) {
        int32_t pa = 0, ti = 0, ne = 0;
        for (int s = 0; s < B; ++s) {
            t_pack[s] = pa;
            t_tiles[s] = ti;
            t_ne[s] = ne;
            const int n = max(a.seq_len[s], 0);
            t_len[s] = n;
            pa += n;
            ti += ceil_div(n, kTile);
            ne += n > 0 ? 1 : 0;
        }
        t_pack[B] = pa;
        t_tiles[B] = ti;
        t_ne[B] = ne;
    }
    if (warp == kEpiWarps + 1) tmem_alloc(&tl.tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tl.tmem_base;
    // Everything up to here is local to the CTA or reads the caller's inputs.  In a run of layers the launch may have been started while the
    // launch before it was still draining (programmatic dependent launch): from here on its results are needed.
    if (a.dependent) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (a.tickets_next && blockIdx.x == 0)
        for (int t = threadIdx.x; t < 2 * B * a.p.num_kv_heads; t += kThreadsTc) a.tickets_next[t] = 0u;
    if (a.sel_lengths && blockIdx.x == 0)         // an empty sequence has no tile to finish: it keeps nothing
        for (int t = threadIdx.x; t < B * a.p.num_kv_heads; t += kThreadsTc)
            if (a.seq_len[t / a.p.num_kv_heads] <= 0) a.sel_lengths[t] = 0;
    SeqView sv;
    sv.pack = t_pack; sv.tiles = t_tiles; sv.len = t_len; sv.start = t_start; sv.ne = t_ne;

    // ranges over min(grid, items) CTAs, so that every CTA that has a range has a non-empty one
    const Split sp = make_split(sv, B, a.p.num_kv_heads, (int)gridDim.x);
    const bool active = (int)blockIdx.x < sp.ctas && sp.items > 0;
    const int item0 = active ? range_begin(sp, sv, B, blockIdx.x) : 0;
    const int item1 = active ? range_begin(sp, sv, B, blockIdx.x + 1) : 0;

    const int nitems = item1 - item0;
    if (warp < kEpiWarps) {
        EpiState es;
        if (MODE == 4) epilogue_pass2(a, tl, sv, tmem_base, item0, nitems, sp, es);
        if (P1) epilogue_pass1(a, tl, tmem_base, nitems, es);
        if (MODE == 3) {
            // publish: this CTA's partials are in memory
            __threadfence();
            epi_sync(tl, es.ephase);
            if (threadIdx.x == 0)
                asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(a.flags + blockIdx.x), "r"(1u) : "memory");
        }
        if (P2 && MODE != 4) epilogue_pass2(a, tl, sv, tmem_base, item0, nitems, sp, es);
    } else if (warp == kEpiWarps) {
        if (lane == 0) {
            RingState rs;
            if (MODE == 4) producer_loop(a, &mapq_b, &mapk_b, smem_q, smem_k, tl, sv, item0, item1, rs, true);
            if (P1) producer_loop(a, &mapq_a, &mapk_a, smem_q, smem_k, tl, sv, item0, item1, rs, false);
            if (P2 && MODE != 4) producer_loop(a, &mapq_b, &mapk_b, smem_q, smem_k, tl, sv, item0, item1, rs, true);
        }
    } else if (warp == kEpiWarps + 2) {
        if (a.cj.nslots > 0) copy_loop(a, tl, sv, smem_c, coff);
    } else if (warp >= kEpiWarps + 3) {
        if (P2) finisher_pass2(a, tl, nitems, MODE == 3 ? (uint32_t)nitems : 0u, warp - (kEpiWarps + 3));
    } else {
        if (lane == 0) {
            MmaState ms;
            if (MODE == 4) {
                mma_loop_pass2(a, smem_q, smem_k, tl, tmem_base, nitems, ms);
                drain_pass2(tl, ms);
            }
            if (P1 && !tl.abort_flag) mma_loop_pass1(a, smem_q, smem_k, tl, tmem_base, nitems, ms);
            if (MODE == 3) drain_pass1(tl, ms);
            if (P2 && MODE != 4 && !tl.abort_flag) mma_loop_pass2(a, smem_q, smem_k, tl, tmem_base, nitems, ms);
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
    sh.rblocks = (sh.R + kTile - 1) / kTile;
    sh.Rpad = sh.rblocks * kTile;
    sh.cblocks = sh.R > 256 ? 2 : 1;
    sh.ncol = ((sh.R + sh.cblocks - 1) / sh.cblocks + 31) / 32 * 32;   // two warps halve it in groups of 16; rows past R are masked
    sh.stages = sh.Rpad <= 256 ? 4 : 2;
    sh.rank4 = p.k_stride_seq != 0;
    return true;
}

size_t smem_bytes(const TcShape &sh, int num_seqs, int copy_slots = 0, int copy_units = 0)
{
    return 1024 + (size_t)sh.Rpad * 256 + (size_t)sh.stages * kTileBytes + (size_t)copy_slots * kCopySlot +
           sizeof(TcSmemTail) + (size_t)(5 * num_seqs + 3) * sizeof(int32_t) +
           (copy_slots ? (size_t)(copy_units + 1) * sizeof(int32_t) : 0);
}

constexpr size_t kSmemLimit = 232448;

// Per-device facts, looked up once per device under a lock.
struct DevInfo { bool ready = false; int sms = 0; bool coop = false; cudaError_t err = cudaSuccess; };
std::mutex g_dev_mutex;
DevInfo g_dev[64];

cudaError_t device_info(DevInfo &out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    DevInfo &d = g_dev[dev];
    if (!d.ready) {
        int n = 0, coop = 0;
        e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(score_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(score_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(score_tc_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(score_tc_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
        if (e != cudaSuccess) return e;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess) coop = 0;
        d.sms = std::min(n, kMaxCtas);
        d.coop = coop != 0;
        d.ready = true;
    }
    out = d;
    return cudaSuccess;
}

// Ring depth and pieces in flight when the launch also copies rows: the K ring gives up a stage where it
// has four, and the pieces take what is left.  False when fewer than three pieces would fit.
bool copy_shape(const refree_params &p, TcShape &sh, int &nslots)
{
    const int U = p.num_seqs * p.num_kv_heads;
    if (sh.stages > 2) sh.stages = 2;
    for (nslots = kMaxCopySlots; nslots >= 3; --nslots)
        if (smem_bytes(sh, p.num_seqs, nslots, U) <= kSmemLimit) return true;
    return false;
}

}  // namespace

bool score_tc_can_copy(const refree_params &p, int64_t total_tokens)
{
    TcShape sh;
    int nslots = 0;
    if (!shape_for(p, sh)) return false;
    if (p.k_stride_tok != kD || p.v_stride_tok != kD) return false;          // a unit's rows back to back
    if ((int64_t)p.num_seqs * p.num_kv_heads > kMaxCopyUnits) return false;
    if ((int64_t)p.num_kv_heads * total_tokens > 0x7fffffffLL) return false;  // row counts held in 32 bits
    if (p.rank_mode != REFREE_RANK_POSITION && !p.force_full) return false;
    return copy_shape(p, sh, nslots);
}

bool score_tc_supported(const refree_params &p)
{
    TcShape sh;
    if (!shape_for(p, sh)) return false;
    if (p.kv_tokens <= 0 || p.kv_tokens > 0x7fffffffLL) return false;
    if (smem_bytes(sh, p.num_seqs) > kSmemLimit) return false;
    return encode_fn() != nullptr;
}

namespace {

cudaError_t encode_maps(const refree_params &p, const TcShape &sh, const void *q_win, const void *k, CUtensorMap &mapq,
                        CUtensorMap &mapk)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
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
    return cudaSuccess;
}

}  // namespace

// Both passes of one layer.
cudaError_t launch_score_tc(const refree_params &p, const void *q_win, const void *k,
                            const int32_t *seq_start, const int32_t *seq_len,
                            int64_t total_tokens, float *scores, char *ws, const Workspace &lay,
                            int32_t *dev_status, cudaStream_t st, GroupPartial *groups)
{
    TcShape sh;
    if (!shape_for(p, sh)) return cudaErrorInvalidValue;
    CUtensorMap mapq, mapk;
    cudaError_t e = encode_maps(p, sh, q_win, k, mapq, mapk);
    if (e != cudaSuccess) return e;
    DevInfo di;
    e = device_info(di);
    if (e != cudaSuccess) return e;
    const int64_t max_items = (total_tokens / kTile + p.num_seqs) * p.num_kv_heads;
    const int ctas = (int)std::max<int64_t>(1, std::min<int64_t>(di.sms, max_items));
    TcArgs a;
    a.p = p;
    a.sh = sh;
    a.seq_start = seq_start;
    a.seq_len = seq_len;
    a.part_a = reinterpret_cast<float2 *>(ws + lay.part_off);
    a.part_b = a.part_a;
    a.groups = groups;
    a.scores = scores;
    a.total_tokens = total_tokens;
    a.dev_status = dev_status;
    a.sel_lengths = nullptr;
    a.sel_cuts = nullptr;
    a.tickets = a.tickets_next = nullptr;
    a.dependent = 0;
    a.cj = TcCopyJob{};
    const size_t smem = smem_bytes(sh, p.num_seqs);
    if (smem > kSmemLimit) return cudaErrorInvalidValue;
    a.flags = nullptr;
    if (di.coop) {
        // Both passes in one cooperative launch (co-residency of all CTAs is what makes the wait of pass 2
        // on other CTAs' pass 1 safe).  The flags are cleared on the stream before the launch.
        a.flags = reinterpret_cast<uint32_t *>(ws + lay.cnt_off);
        e = cudaMemsetAsync(a.flags, 0, (size_t)kMaxCtas * sizeof(uint32_t), st);
        if (e != cudaSuccess) return e;
        void *args[5] = {(void *)&mapq, (void *)&mapk, (void *)&mapq, (void *)&mapk, (void *)&a};
        const cudaError_t ce = cudaLaunchCooperativeKernel((const void *)score_tc_kernel<3>, dim3(ctas), dim3(kThreadsTc),
                                                           args, smem, st);
        if (ce == cudaSuccess) {
            count_launches(1);
            return cudaGetLastError();
        }
        (void)cudaGetLastError();        // not launchable as one grid here: fall back to one launch per pass
        a.flags = nullptr;
    }
    score_tc_kernel<1><<<ctas, kThreadsTc, smem, st>>>(mapq, mapk, mapq, mapk, a);
    score_tc_kernel<2><<<ctas, kThreadsTc, smem, st>>>(mapq, mapk, mapq, mapk, a);
    count_launches(2);
    return cudaGetLastError();
}

// One launch of a run of layers: pass 2 of `finish` (nullable), then pass 1 of `begin` (nullable), and the rows
// of `copy` (nullable) beside them.  The partials that pass 2 reads were completed by an earlier launch on the
// stream, so no CTA waits for another and the launch is an ordinary one.
cudaError_t launch_score_tc_pipe(const refree_params &p, const TcLayer *begin, const TcLayer *finish,
                                 const int32_t *seq_start, const int32_t *seq_len, int64_t total_tokens,
                                 const Workspace &lay, int32_t *dev_status, cudaStream_t st, const TcCopyJob *copy,
                                 bool finish_tickets_clean)
{
    if (!begin && !finish) return cudaErrorInvalidValue;
    TcShape sh;
    if (!shape_for(p, sh)) return cudaErrorInvalidValue;
    int copy_slots = 0;
    if (copy && !copy_shape(p, sh, copy_slots)) return cudaErrorInvalidValue;
    CUtensorMap mapq_a, mapk_a, mapq_b, mapk_b;
    cudaError_t e = cudaSuccess;
    if (begin && (e = encode_maps(p, sh, begin->q_win, begin->k, mapq_a, mapk_a)) != cudaSuccess) return e;
    if (finish && (e = encode_maps(p, sh, finish->q_win, finish->k, mapq_b, mapk_b)) != cudaSuccess) return e;
    if (!begin) { mapq_a = mapq_b; mapk_a = mapk_b; }
    if (!finish) { mapq_b = mapq_a; mapk_b = mapk_a; }
    DevInfo di;
    e = device_info(di);
    if (e != cudaSuccess) return e;
    const int64_t max_items = (total_tokens / kTile + p.num_seqs) * p.num_kv_heads;
    // with rows to move, every SM takes part whatever the number of scoring items
    const int ctas = copy ? di.sms : (int)std::max<int64_t>(1, std::min<int64_t>(di.sms, max_items));
    TcArgs a;
    a.p = p;
    a.sh = sh;
    a.seq_start = seq_start;
    a.seq_len = seq_len;
    a.part_a = begin ? reinterpret_cast<float2 *>(begin->ws + lay.part_off) : nullptr;
    a.part_b = finish ? reinterpret_cast<const float2 *>(finish->ws + lay.part_off) : nullptr;
    a.groups = finish ? finish->groups : nullptr;
    a.scores = finish ? finish->scores : nullptr;
    a.flags = nullptr;
    a.total_tokens = total_tokens;
    a.dev_status = dev_status;
    // the rule runs inside the launch when the finished layer says where its budgets go
    const bool sel = finish && finish->sel_lengths && finish->groups;
    a.sel_lengths = sel ? finish->sel_lengths : nullptr;
    a.sel_cuts = sel ? reinterpret_cast<Cut *>(finish->ws + lay.cut_off) : nullptr;
    a.tickets = sel ? reinterpret_cast<uint32_t *>(finish->ws + lay.cnt_off) + kMaxCtas : nullptr;
    a.tickets_next = (begin && begin->sel_lengths && begin->groups)
                         ? reinterpret_cast<uint32_t *>(begin->ws + lay.cnt_off) + kMaxCtas : nullptr;
    if (sel && !finish_tickets_clean) {
        e = cudaMemsetAsync(a.tickets, 0, 2 * (size_t)p.num_seqs * p.num_kv_heads * sizeof(uint32_t), st);
        if (e != cudaSuccess) return e;
    }
    if (copy) a.cj = *copy; else a.cj = TcCopyJob{};
    a.cj.nslots = copy ? copy_slots : 0;
    const size_t smem = smem_bytes(sh, p.num_seqs, a.cj.nslots, p.num_seqs * p.num_kv_heads);
    if (smem > kSmemLimit) return cudaErrorInvalidValue;
    // Launches of a run after the first may start while the one before drains: their CTAs set themselves up and
    // then wait (griddepcontrol.wait) until that launch has completed and its results are visible.
    a.dependent = finish_tickets_clean ? 1 : 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctas);
    cfg.blockDim = dim3(kThreadsTc);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.dependent ? 1 : 0;
    if (begin && finish) e = cudaLaunchKernelEx(&cfg, score_tc_kernel<4>, mapq_a, mapk_a, mapq_b, mapk_b, a);
    else if (begin) e = cudaLaunchKernelEx(&cfg, score_tc_kernel<1>, mapq_a, mapk_a, mapq_b, mapk_b, a);
    else e = cudaLaunchKernelEx(&cfg, score_tc_kernel<2>, mapq_a, mapk_a, mapq_b, mapk_b, a);
    if (e != cudaSuccess) return e;
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace refree
