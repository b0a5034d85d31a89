// The pass of Algorithm 1 for a run of layers whose caches live in HOST memory, pipelined
// over three streams: while layer l is compressed, the inputs of layer l + 1 are on their way
// to the device and the kept rows of layer l - 1 on their way back.  With the cache on the
// host the copies dominate (two 64 MB arrays in, ~two out, per 32K layer, against 0.13 ms of
// kernels), and PCIe carries both directions at once, so the pipeline costs about one
// direction's copy time per layer instead of both in sequence.
#include <algorithm>

#include "refree_internal.cuh"

namespace refree {
namespace {

struct Slot {
    char *q, *k, *v, *ko, *vo;
    int32_t *lengths, *status;
    int64_t *offsets;
    cudaEvent_t in_done, comp_done, meta_done, out_done;
    int32_t h_status;
};

inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

struct PipeSizes {
    size_t q, kv, out, lengths, offsets, status, seq, ws;
    size_t total() const { return 2 * (q + 2 * kv + 2 * out + lengths + offsets + status) + 2 * seq + ws; }
};

refree_status pipe_sizes(const refree_params *p, int64_t total_tokens, int64_t kv_elems, int64_t capacity_rows,
                         PipeSizes &z)
{
    if (!p || kv_elems < 0 || capacity_rows < 0 || total_tokens < 0) return REFREE_ERR_INVALID_ARG;
    size_t ws = 0;
    const refree_status st = refree_workspace_size(p, total_tokens, &ws);
    if (st != REFREE_OK) return st;
    const size_t esz = p->dtype == REFREE_DTYPE_F32 ? 4 : 2;
    const size_t U = (size_t)p->num_seqs * p->num_kv_heads;
    z.q = up256((size_t)p->num_seqs * p->num_q_heads * p->window * p->head_dim * esz);
    z.kv = up256((size_t)kv_elems * esz);
    z.out = up256((size_t)capacity_rows * p->head_dim * esz);
    z.lengths = up256(U * sizeof(int32_t));
    z.offsets = up256((U + 1) * sizeof(int64_t));
    z.status = up256(sizeof(int32_t));
    z.seq = up256((size_t)p->num_seqs * sizeof(int32_t));
    z.ws = up256(ws);
    return REFREE_OK;
}

}  // namespace
}  // namespace refree

using namespace refree;

extern "C" {

refree_status refree_host_pipeline_arena_size(const refree_params *p, int64_t total_tokens, int64_t kv_elems,
                                              int64_t capacity_rows, size_t *bytes)
{
    if (!bytes) return REFREE_ERR_INVALID_ARG;
    PipeSizes z;
    const refree_status st = pipe_sizes(p, total_tokens, kv_elems, capacity_rows, z);
    if (st != REFREE_OK) return st;
    *bytes = z.total();
    return REFREE_OK;
}

refree_status refree_compress_layers_host(const refree_params *p, int32_t num_layers,
                                          const void *const *q_win, const void *const *k, const void *const *v,
                                          int64_t kv_elems, const int32_t *seq_start, const int32_t *seq_len,
                                          int64_t total_tokens, void *const *k_out, void *const *v_out,
                                          int64_t capacity_rows, int32_t *const *lengths, int64_t *const *offsets,
                                          void *arena, size_t arena_bytes)
{
    PipeSizes z;
    refree_status st = pipe_sizes(p, total_tokens, kv_elems, capacity_rows, z);
    if (st != REFREE_OK) return st;
    if (num_layers < 0 || !q_win || !k || !v || !seq_start || !seq_len || !k_out || !v_out || !lengths || !offsets)
        return REFREE_ERR_INVALID_ARG;
    for (int l = 0; l < num_layers; ++l)
        if (!q_win[l] || !k[l] || !v[l] || !k_out[l] || !v_out[l] || !lengths[l] || !offsets[l]) return REFREE_ERR_INVALID_ARG;
    if (!arena || arena_bytes < z.total() || (reinterpret_cast<uintptr_t>(arena) & 255)) return REFREE_ERR_WORKSPACE;
    if (num_layers == 0) return REFREE_OK;

    const size_t esz = p->dtype == REFREE_DTYPE_F32 ? 4 : 2;
    const size_t U = (size_t)p->num_seqs * p->num_kv_heads;
    const size_t q_bytes = (size_t)p->num_seqs * p->num_q_heads * p->window * p->head_dim * esz;
    const size_t kv_bytes = (size_t)kv_elems * esz;
    const size_t row_bytes = (size_t)p->head_dim * esz;

    char *a = static_cast<char *>(arena);
    auto take = [&](size_t bytes) { char *r = a; a += bytes; return r; };
    int32_t *d_start = reinterpret_cast<int32_t *>(take(z.seq));
    int32_t *d_len = reinterpret_cast<int32_t *>(take(z.seq));
    char *d_ws = take(z.ws);
    Slot slot[2];
    for (int i = 0; i < 2; ++i) {
        slot[i].q = take(z.q); slot[i].k = take(z.kv); slot[i].v = take(z.kv);
        slot[i].ko = take(z.out); slot[i].vo = take(z.out);
        slot[i].lengths = reinterpret_cast<int32_t *>(take(z.lengths));
        slot[i].offsets = reinterpret_cast<int64_t *>(take(z.offsets));
        slot[i].status = reinterpret_cast<int32_t *>(take(z.status));
        slot[i].in_done = slot[i].comp_done = slot[i].meta_done = slot[i].out_done = nullptr;
        slot[i].h_status = 0;
    }

    cudaStream_t s_in = nullptr, s_comp = nullptr, s_out = nullptr;
    bool ok = cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&s_comp, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i)
        ok = cudaEventCreateWithFlags(&slot[i].in_done, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&slot[i].comp_done, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&slot[i].meta_done, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&slot[i].out_done, cudaEventDisableTiming) == cudaSuccess;

    refree_status result = ok ? REFREE_OK : REFREE_ERR_CUDA;
    auto cu = [&](cudaError_t e) { if (e != cudaSuccess && result == REFREE_OK) result = REFREE_ERR_CUDA; return e == cudaSuccess; };

    // kept rows of layer j come back once its budgets are known on the host
    auto finish = [&](int j) {
        Slot &sl = slot[j & 1];
        if (!cu(cudaEventSynchronize(sl.meta_done))) return;
        if (sl.h_status & REFREE_DEV_TIMEOUT) { result = REFREE_ERR_TIMEOUT; return; }
        if (sl.h_status & REFREE_DEV_CAPACITY) { result = REFREE_ERR_CAPACITY; return; }
        if (sl.h_status & REFREE_DEV_NONFINITE) { result = REFREE_ERR_NONFINITE; return; }
        const int64_t rows = offsets[j][U];
        cu(cudaMemcpyAsync(k_out[j], sl.ko, (size_t)rows * row_bytes, cudaMemcpyDeviceToHost, s_out));
        cu(cudaMemcpyAsync(v_out[j], sl.vo, (size_t)rows * row_bytes, cudaMemcpyDeviceToHost, s_out));
        cu(cudaEventRecord(sl.out_done, s_out));
    };

    if (result == REFREE_OK) {
        cu(cudaMemcpyAsync(d_start, seq_start, p->num_seqs * sizeof(int32_t), cudaMemcpyHostToDevice, s_in));
        cu(cudaMemcpyAsync(d_len, seq_len, p->num_seqs * sizeof(int32_t), cudaMemcpyHostToDevice, s_in));
    }
    int finished = 0;
    for (int l = 0; l < num_layers && result == REFREE_OK; ++l) {
        Slot &sl = slot[l & 1];
        // inputs of the slot are free once layer l - 2 has been compressed
        if (l >= 2) cu(cudaStreamWaitEvent(s_in, sl.comp_done, 0));
        cu(cudaMemcpyAsync(sl.q, q_win[l], q_bytes, cudaMemcpyHostToDevice, s_in));
        cu(cudaMemcpyAsync(sl.k, k[l], kv_bytes, cudaMemcpyHostToDevice, s_in));
        cu(cudaMemcpyAsync(sl.v, v[l], kv_bytes, cudaMemcpyHostToDevice, s_in));
        cu(cudaEventRecord(sl.in_done, s_in));
        // outputs of the slot are free once the rows of layer l - 2 have left
        cu(cudaStreamWaitEvent(s_comp, sl.in_done, 0));
        if (l >= 2) cu(cudaStreamWaitEvent(s_comp, sl.out_done, 0));
        cu(cudaMemsetAsync(sl.status, 0, sizeof(int32_t), s_comp));
        if (result != REFREE_OK) break;
        st = refree_compress_layer(p, sl.q, sl.k, sl.v, d_start, d_len, total_tokens, sl.ko, sl.vo, capacity_rows,
                                   sl.lengths, sl.offsets, nullptr, nullptr, d_ws, z.ws, sl.status, s_comp);
        if (st != REFREE_OK) { result = st; break; }
        cu(cudaEventRecord(sl.comp_done, s_comp));
        cu(cudaStreamWaitEvent(s_out, sl.comp_done, 0));
        cu(cudaMemcpyAsync(lengths[l], sl.lengths, U * sizeof(int32_t), cudaMemcpyDeviceToHost, s_out));
        cu(cudaMemcpyAsync(offsets[l], sl.offsets, (U + 1) * sizeof(int64_t), cudaMemcpyDeviceToHost, s_out));
        cu(cudaMemcpyAsync(&sl.h_status, sl.status, sizeof(int32_t), cudaMemcpyDeviceToHost, s_out));
        cu(cudaEventRecord(sl.meta_done, s_out));
        if (l >= 1 && result == REFREE_OK) { finish(l - 1); finished = l; }
    }
    if (result == REFREE_OK && finished < num_layers) finish(num_layers - 1);

    // leave nothing in flight, whatever happened
    if (s_in) cudaStreamSynchronize(s_in);
    if (s_comp) cudaStreamSynchronize(s_comp);
    if (s_out) { if (cudaStreamSynchronize(s_out) != cudaSuccess && result == REFREE_OK) result = REFREE_ERR_CUDA; }
    for (int i = 0; i < 2; ++i) {
        if (slot[i].in_done) cudaEventDestroy(slot[i].in_done);
        if (slot[i].comp_done) cudaEventDestroy(slot[i].comp_done);
        if (slot[i].meta_done) cudaEventDestroy(slot[i].meta_done);
        if (slot[i].out_done) cudaEventDestroy(slot[i].out_done);
    }
    if (s_in) cudaStreamDestroy(s_in);
    if (s_comp) cudaStreamDestroy(s_comp);
    if (s_out) cudaStreamDestroy(s_out);
    return result;
}

}  // extern "C"
