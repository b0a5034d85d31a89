// Two memory-system probes with the access shape of the pass, for the benchmark's ceiling figures: a read-only
// stream (what scoring asks of HBM) and a row copy that reads (1 + rho) and writes 2 rho of the bytes it is given
// (what the whole pass asks: K once, kept V, and the kept K and V rows written).  Plain 16-byte vector loads and
// stores, many in flight per thread; no arithmetic of the method.
#include <mutex>

#include "refree_internal.cuh"

namespace refree {
namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 8;

__device__ inline int4 ld_stream(const int4 *p)
{
    int4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ inline void st_stream(int4 *p, const int4 &v)
{
    asm volatile("st.global.cs.v4.s32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__global__ void __launch_bounds__(kThreads) sol_read_kernel(const int4 *src, int64_t nvec, int *sink)
{
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    int acc = 0;
    for (int64_t e0 = (int64_t)blockIdx.x * kThreads + threadIdx.x; e0 < nvec; e0 += stride * kUnroll) {
        int4 v[kUnroll];
#pragma unroll
        for (int r = 0; r < kUnroll; ++r) v[r] = e0 + r * stride < nvec ? ld_stream(src + e0 + r * stride) : make_int4(0, 0, 0, 0);
#pragma unroll
        for (int r = 0; r < kUnroll; ++r) acc ^= v[r].x ^ v[r].y ^ v[r].z ^ v[r].w;
    }
    if (acc == 0x5a5a5a5b && sink) *sink = acc;      // keeps the loads; practically never true
}

// Rows [0, rows) of k are read; the last `kept` of them are also written to k_out, and the same rows of v are read
// and written to v_out.
__global__ void __launch_bounds__(kThreads)
sol_mix_kernel(const int4 *k, const int4 *v, int4 *k_out, int4 *v_out, int64_t rows, int64_t kept, int vec_per_row, int *sink)
{
    const int64_t nvec = rows * vec_per_row, first = (rows - kept) * vec_per_row;
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    int acc = 0;
    for (int64_t e0 = (int64_t)blockIdx.x * kThreads + threadIdx.x; e0 < nvec; e0 += stride * (kUnroll / 2)) {
        int4 a[kUnroll / 2], b[kUnroll / 2];
#pragma unroll
        for (int r = 0; r < kUnroll / 2; ++r) {
            const int64_t e = e0 + r * stride;
            a[r] = e < nvec ? ld_stream(k + e) : make_int4(0, 0, 0, 0);
            b[r] = e < nvec && e >= first ? ld_stream(v + e) : make_int4(0, 0, 0, 0);
        }
#pragma unroll
        for (int r = 0; r < kUnroll / 2; ++r) {
            const int64_t e = e0 + r * stride;
            if (e < nvec && e >= first) {
                st_stream(k_out + (e - first), a[r]);
                st_stream(v_out + (e - first), b[r]);
            } else {
                acc ^= a[r].x ^ a[r].w;
            }
        }
    }
    if (acc == 0x5a5a5a5b && sink) *sink = acc;
}

// The same two access shapes through the bulk-copy engine (cp.async.bulk, no tensor map, no multicast): 16 KB
// pieces, global -> shared (-> global where a destination is given), a ring of slots per CTA driven by one
// thread.  Up to three segments, each {source, destination or null, bytes}; piece k of the concatenated
// segments belongs to CTA k mod grid.
struct BulkSeg { const unsigned char *src; unsigned char *dst; long long bytes; };
struct BulkJob { BulkSeg seg[3]; int nseg; };
constexpr int kPiece = 16384, kSlots = 8;

__device__ inline unsigned smem_addr(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }

__global__ void __launch_bounds__(32) sol_bulk_kernel(BulkJob job, int *sink)
{
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ unsigned long long full[kSlots];
    __shared__ unsigned long long dsts[kSlots];
    __shared__ unsigned sizes[kSlots];
    if (threadIdx.x != 0) return;
    for (int i = 0; i < kSlots; ++i)
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(&full[i])), "r"(1));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    long long pieces[3], total = 0;
    for (int g = 0; g < 3; ++g) { pieces[g] = g < job.nseg ? (job.seg[g].bytes + kPiece - 1) / kPiece : 0; total += pieces[g]; }
    long long next = blockIdx.x;
    auto issue = [&](unsigned j) -> bool {
        if (next >= total) return false;
        long long k = next;
        next += gridDim.x;
        int g = 0;
        while (k >= pieces[g]) { k -= pieces[g]; ++g; }
        const long long off = k * kPiece;
        const unsigned bytes = (unsigned)min((long long)kPiece, job.seg[g].bytes - off);
        const unsigned slot = j % kSlots;
        dsts[slot] = job.seg[g].dst ? (unsigned long long)(uintptr_t)(job.seg[g].dst + off) : 0ull;
        sizes[slot] = bytes;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(&full[slot])), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_addr(ring + (size_t)slot * kPiece)), "l"(job.seg[g].src + off), "r"(bytes),
                       "r"(smem_addr(&full[slot])) : "memory");
        return true;
    };
    unsigned issued = 0;
    while (issued + 1 < (unsigned)kSlots && issue(issued)) ++issued;
    bool gave_up = false;
    for (unsigned i = 0; i < issued && !gave_up; ++i) {
        const unsigned slot = i % kSlots, parity = (i / kSlots) & 1u;
        bool ok = false;
        for (unsigned spin = 0; spin < (1u << 22) && !ok; ++spin) {
            unsigned done;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(done) : "r"(smem_addr(&full[slot])), "r"(parity) : "memory");
            ok = done != 0;
        }
        if (!ok) { gave_up = true; break; }
        if (dsts[slot]) {
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                         ::"l"(dsts[slot]), "r"(smem_addr(ring + (size_t)slot * kPiece)), "r"(sizes[slot]) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        }
        if (issue(issued)) ++issued;
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (gave_up && sink) *sink = -1;
}

}  // namespace
}  // namespace refree

using namespace refree;

extern "C" {

static refree_status launch_bulk(const BulkJob &job, int32_t *sink, cudaStream_t st)
{
    static std::once_flag once;
    static cudaError_t attr = cudaSuccess;
    std::call_once(once, [] {
        attr = cudaFuncSetAttribute(sol_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSlots * kPiece);
    });
    if (attr != cudaSuccess) return REFREE_ERR_CUDA;
    sol_bulk_kernel<<<sm_count(), 32, kSlots * kPiece, st>>>(job, sink);
    count_launches(1);
    return cudaGetLastError() == cudaSuccess ? REFREE_OK : REFREE_ERR_CUDA;
}

refree_status refree_sol_read_stream(const void *src, int64_t bytes, int32_t *sink, void *stream)
{
    if (!src || bytes < 0 || (bytes & 15) || (reinterpret_cast<uintptr_t>(src) & 15)) return REFREE_ERR_INVALID_ARG;
    if (bytes == 0) return REFREE_OK;
    if (sink == REFREE_SOL_BULK) {
        BulkJob job = {};
        job.seg[0] = BulkSeg{(const unsigned char *)src, nullptr, (long long)bytes};
        job.nseg = 1;
        return launch_bulk(job, nullptr, (cudaStream_t)stream);
    }
    sol_read_kernel<<<sm_count() * 8, kThreads, 0, (cudaStream_t)stream>>>((const int4 *)src, bytes / 16, sink);
    count_launches(1);
    return cudaGetLastError() == cudaSuccess ? REFREE_OK : REFREE_ERR_CUDA;
}

refree_status refree_sol_row_mix(const void *k, const void *v, void *k_out, void *v_out, int64_t rows, int64_t kept_rows,
                                 int32_t row_bytes, int32_t *sink, void *stream)
{
    if (!k || !v || !k_out || !v_out || rows < 0 || kept_rows < 0 || kept_rows > rows || row_bytes < 16 || (row_bytes & 15))
        return REFREE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(k_out) |
         reinterpret_cast<uintptr_t>(v_out)) & 15)
        return REFREE_ERR_INVALID_ARG;
    if (rows == 0) return REFREE_OK;
    if (sink == REFREE_SOL_BULK) {
        const long long rb = row_bytes;
        BulkJob job = {};
        job.seg[0] = BulkSeg{(const unsigned char *)k, nullptr, (long long)(rows - kept_rows) * rb};
        job.seg[1] = BulkSeg{(const unsigned char *)k + (rows - kept_rows) * rb, (unsigned char *)k_out, (long long)kept_rows * rb};
        job.seg[2] = BulkSeg{(const unsigned char *)v + (rows - kept_rows) * rb, (unsigned char *)v_out, (long long)kept_rows * rb};
        job.nseg = 3;
        return launch_bulk(job, nullptr, (cudaStream_t)stream);
    }
    sol_mix_kernel<<<sm_count() * 8, kThreads, 0, (cudaStream_t)stream>>>((const int4 *)k, (const int4 *)v, (int4 *)k_out,
                                                                         (int4 *)v_out, rows, kept_rows, row_bytes / 16, sink);
    count_launches(1);
    return cudaGetLastError() == cudaSuccess ? REFREE_OK : REFREE_ERR_CUDA;
}

}  // extern "C"
