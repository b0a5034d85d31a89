// refree_select_budget_static: the selection stage for callers that cannot
// allocate device memory.  Its scratch is a fixed array that is part of the
// library image, so nothing is allocated at any point.
#include <mutex>

#include "refree_internal.cuh"

namespace refree {
namespace {

// Scratch of the selection kernels (one Cut record per unit), held by every GPU
// that loads this library until the process exits.
__device__ __align__(256) static unsigned char g_select_scratch[REFREE_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
char *g_scratch_addr[kMaxDevices] = {};   // device address of g_select_scratch, per device ordinal

// The array's name is only a host-side handle here; the kernels need its device
// address, which differs per GPU.  Looked up once per device, with that device
// current (it is: the caller's stream belongs to the current device).
refree_status scratch_for_current_device(char **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return REFREE_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_select_scratch) != cudaSuccess || !ptr) return REFREE_ERR_CUDA;
        g_scratch_addr[dev] = static_cast<char *>(ptr);
    }
    *out = g_scratch_addr[dev];
    return REFREE_OK;
}

}  // namespace
}  // namespace refree

using namespace refree;

extern "C" refree_status refree_select_budget_static(const refree_params *p, const float *scores,
                                                     const int32_t *seq_len, int64_t total_tokens,
                                                     int32_t *lengths, int64_t *offsets,
                                                     int32_t *kept_idx, int64_t capacity_rows,
                                                     int32_t *device_status, void *stream)
{
    if (!p || p->num_seqs < 1 || p->num_kv_heads < 1 || p->num_q_heads < 1 ||
        p->num_q_heads % p->num_kv_heads != 0 || p->window < 1 || p->sink < 0 ||
        !(p->threshold >= 0.0f && p->threshold < 1.0f) ||
        (p->rank_mode != REFREE_RANK_POSITION && p->rank_mode != REFREE_RANK_SCORE) ||
        (p->scope != REFREE_SCOPE_HEAD && p->scope != REFREE_SCOPE_LAYER) ||
        total_tokens < 0 || total_tokens > 0x7fffffffLL - kTile || capacity_rows < 0)
        return REFREE_ERR_INVALID_ARG;
    if (!scores || !seq_len || !lengths || !offsets) return REFREE_ERR_INVALID_ARG;
    if (p->num_seqs > kMaxSeqs) return REFREE_ERR_UNSUPPORTED;
    // the whole scratch need of the selection stage must fit the built-in array
    const Workspace full = workspace_layout(*p, total_tokens);
    if (full.cut_bytes > (size_t)REFREE_STATIC_SCRATCH_BYTES ||
        (int64_t)p->num_seqs * p->num_kv_heads > 65535)
        return REFREE_ERR_STATIC_LIMIT;
    char *scratch = nullptr;
    const refree_status st = scratch_for_current_device(&scratch);
    if (st != REFREE_OK) return st;
    Workspace lay = {};
    lay.cut_off = 0;
    lay.cut_bytes = full.cut_bytes;
    lay.total = full.cut_bytes;
    // Every Cut record read by a call is written earlier in the same call, so the
    // contents left by the previous call need no clearing.
    const cudaError_t e = launch_select(*p, scores, seq_len, total_tokens, lengths, offsets, kept_idx,
                                        capacity_rows, scratch, lay, device_status, (cudaStream_t)stream);
    return e == cudaSuccess ? REFREE_OK : REFREE_ERR_CUDA;
}
