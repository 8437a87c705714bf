// sam_retrieve_noalloc: one-shot draft retrieval that allocates nothing.
//
// Who needs it: code that runs inside a host application which has already taken the device's
// free memory for its own pools (an inference server that hands nearly all of HBM to its KV cache,
// a plugin bound by a "no allocation after start-up" rule).  There cudaMalloc fails or is not
// permitted, so the per-sequence automata cannot live in a workspace the caller allocates.  Here
// they live in a fixed array that is part of the library image itself.
//
// The array below is that scratch: control blocks, token text, root tables and the slab pool of a
// short-lived batch, laid out exactly like a caller-provided workspace.  Every GPU that loads the
// library holds these SAM_NOALLOC_BYTES until the process exits.
#include "common.h"

#include <mutex>

#define SAM_NOALLOC_BYTES (8u << 20)
#define SAM_NOALLOC_MAX_DEVICES 64

static __device__ __align__(256) unsigned char g_noalloc_scratch[SAM_NOALLOC_BYTES];

namespace {

std::mutex g_setup_mutex;
void* g_scratch_addr[SAM_NOALLOC_MAX_DEVICES];      // device address of the array, per device
bool g_scratch_ready[SAM_NOALLOC_MAX_DEVICES];

// The array's name is only a host-side handle: the address kernels may use has to be asked for,
// once per device, with that device current.
int scratch_for_device(int device, void** out) {
    if (device < 0 || device >= SAM_NOALLOC_MAX_DEVICES) return SAM_ERR_ARG;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ready[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) { sam_set_cuda_error(e); cudaGetLastError(); return SAM_ERR_CUDA; }
        g_scratch_addr[device] = p;
        g_scratch_ready[device] = true;
    }
    *out = g_scratch_addr[device];
    return SAM_OK;
}

}  // namespace

extern "C" size_t sam_noalloc_capacity_bytes(void) { return SAM_NOALLOC_BYTES; }

extern "C" int sam_retrieve_noalloc(const sam_static_t* st, int32_t vocab, int32_t batch,
                                    const int32_t* tokens_dev, int32_t stride, const int32_t* counts_dev,
                                    int32_t L, int32_t l_bias, int32_t min_match,
                                    int32_t* draft_tokens_dev, int32_t* draft_len_dev, int32_t* match_len_dev,
                                    int32_t* source_dev, int32_t* state_dev, int32_t* status_dev, void* stream) {
    if (!tokens_dev || !counts_dev || !draft_tokens_dev || !draft_len_dev || !match_len_dev || !source_dev ||
        !status_dev)
        return SAM_ERR_ARG;
    if (batch < 1 || stride < 1 || L < 1 || L > 128 || l_bias < 0 || min_match < 0) return SAM_ERR_ARG;
    if (!st && vocab < 1) return SAM_ERR_ARG;

    int device = 0;
    if (st) device = st->device;
    else SAM_CUDA(cudaGetDevice(&device));
    SamDeviceGuard guard(device);
    if (!guard.ok) return SAM_ERR_CUDA;

    sam_batch_opts_t o;
    o.batch = batch; o.max_seq_len = stride; o.max_draft_len = L; o.l_bias = l_bias; o.min_match = min_match;
    o.vocab = st ? st->info.vocab : vocab; o.max_host_stride = 1; o.slab_bytes = 0; o.pool_slabs = 0;
    o.stop_token_plus_one = 0; o.reserved = 0;
    size_t need = 0;
    int rc = sam_plan_view(&o, o.vocab, nullptr, nullptr, &need, nullptr);
    if (rc) return rc;
    if (need > SAM_NOALLOC_BYTES) return SAM_ERR_LIMIT;       // batch x stride too large for the built-in scratch

    void* base = nullptr;
    rc = scratch_for_device(device, &base);
    if (rc) return rc;

    sam_batch tmp{};                                          // lives for this call only; nothing is allocated
    tmp.device = device; tmp.st = st; tmp.opts = o; tmp.workspace_bytes = need;
    tmp.max_host_stride = 0; tmp.stage_words = 0; tmp.host_stage = nullptr; tmp.host_stage_dev = nullptr; tmp.host_seq = 0;
    rc = sam_plan_view(&o, o.vocab, base, &tmp.view, nullptr, nullptr);
    if (rc) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    rc = sam_launch_init(tmp.view, s);                        // the array keeps the last call's contents: start clean
    if (rc) return rc;
    return sam_launch_step(&tmp, tokens_dev, stride, counts_dev, L, draft_tokens_dev, draft_len_dev,
                           match_len_dev, source_dev, state_dev, status_dev, s);
}
