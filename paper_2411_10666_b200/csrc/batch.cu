// Batch objects: workspace layout, slot initialisation and reset, the slab pool's free stack,
// the host-array step, the step replay loop and the inspection calls.
#include "common.h"

#include <chrono>
#include <cstring>
#include <new>
#include <vector>

namespace {

constexpr size_t SAM_ZERO_COPY_MAX_BYTES = 4u << 20;     // larger host steps go through two DMA copies
constexpr size_t SAM_DIRECT_MIN_BYTES = 64u << 10;       // from this size on, page-locked caller arrays are used in place
constexpr int SAM_POLL_LIMIT_US = 2000;                  // how long a host step polls its completion flag

struct WsLayout {
    size_t off_hdr, off_ctrl, off_free, off_owner, off_reset, off_order, off_text, off_pstate, off_root, off_stage, off_pool, total;
    int32_t text_stride, root_cap, slab_shift, pool_slabs, max_host_stride;
    size_t stage_words;
};

inline uint32_t pow2_ceil(uint64_t x) { uint64_t p = 1; while (p < x) p <<= 1; return (uint32_t)p; }

int plan(const sam_batch_opts_t* o, WsLayout* w) {
    if (!o || o->batch < 1 || o->max_seq_len < 1 || o->max_draft_len < 1 || o->max_draft_len > 128 ||
        o->l_bias < 0 || o->min_match < 0 || o->max_host_stride < 0 || o->pool_slabs < 0 ||
        o->stop_token_plus_one < 0 || o->reserved != 0)
        return SAM_ERR_ARG;
    if (o->max_seq_len > (1 << 28) || o->batch > (1 << 24)) return SAM_ERR_LIMIT;
    const int64_t n = o->max_seq_len;
    uint32_t slab = o->slab_bytes ? (uint32_t)o->slab_bytes : pow2_ceil((uint64_t)8 * n);
    if (!o->slab_bytes && slab < 16384) slab = 16384;
    if (slab < 4096 || (slab & (slab - 1)) || slab > (1u << 30)) return SAM_ERR_ARG;
    // a slot's state records (at most 2n+1 of 32 bytes) must fit SAM_MAX_REC_SLABS slabs
    if ((uint64_t)(2 * n + 2) * 32 > (uint64_t)slab * SAM_MAX_REC_SLABS) return SAM_ERR_ARG;
    int shift = 0;
    while ((1u << shift) < slab) shift++;
    w->slab_shift = shift;
    int64_t per_slot = ((64 + 96) * n + slab - 1) / slab + 2;
    int64_t slabs = o->pool_slabs ? o->pool_slabs : per_slot * o->batch;
    if (slabs < 2 || slabs > (1ll << 31) - 1 || slabs * (int64_t)slab > (1ll << 38)) return SAM_ERR_LIMIT;
    w->pool_slabs = (int32_t)slabs;
    w->text_stride = (int32_t)sam_align_up((size_t)n, 32);
    // the root has at most one transition per text position: twice that many slots
    uint32_t rc = pow2_ceil((uint64_t)2 * n);
    w->root_cap = rc < 64 ? 64 : (int32_t)rc;             // never fewer than two 32-entry probe windows
    w->max_host_stride = o->max_host_stride ? o->max_host_stride : 32;
    w->stage_words = (size_t)o->batch * ((size_t)w->max_host_stride + 1 + (size_t)o->max_draft_len + 7);

    size_t off = 0;
    w->off_hdr = off;   off = sam_align_up(off + 256, 256);
    w->off_ctrl = off;  off = sam_align_up(off + (size_t)o->batch * SAM_CTRL_WORDS * 4, 256);
    w->off_free = off;  off = sam_align_up(off + (size_t)slabs * 4, 256);
    w->off_owner = off; off = sam_align_up(off + (size_t)slabs * 4, 256);
    w->off_reset = off; off = sam_align_up(off + (size_t)o->batch * 4 * 2, 256);   // flags + slot list
    w->off_order = off; off = sam_align_up(off + (size_t)o->batch * 4 * 3 + 64, 256);   // two order buffers, the sort keys, two counts
    w->off_text = off;  off = sam_align_up(off + (size_t)o->batch * w->text_stride * 4, 256);
    w->off_pstate = off; off = sam_align_up(off + (size_t)o->batch * w->text_stride * 4, 256);
    w->off_root = off;  off = sam_align_up(off + (size_t)o->batch * w->root_cap * 8, 256);
    w->off_stage = off; off = sam_align_up(off + w->stage_words * 4, 256);
    w->off_pool = off;  off = sam_align_up(off + (size_t)slabs * slab, 256);
    w->total = off;
    return SAM_OK;
}

// ---- kernels ----------------------------------------------------------------

__global__ void init_pool_kernel(SamBatchView W) {
    size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t s = i; s < (size_t)W.pool_slabs; s += stride) {
        W.free_stack[s] = (int32_t)(W.pool_slabs - 1 - s);      // slab 0 is handed out first
        W.slab_owner[s] = -1;
    }
    for (size_t b = i; b < (size_t)W.batch; b += stride) W.reset_flag[b] = 0;
    if (i == 0) { W.pool_hdr[0] = W.pool_slabs; W.pool_hdr[1] = W.pool_slabs; W.pool_hdr[4] = 0; }
}

// slots == nullptr: every slot.  Clears control blocks and root tables and raises reset flags.
__global__ void reset_slots_kernel(SamBatchView W, const int32_t* slots, int32_t n) {
    const int which = blockIdx.x;
    if (which >= n) return;
    const int b = slots ? slots[which] : which;
    if (b < 0 || b >= W.batch) return;
    uint32_t* cb = W.ctrl + (size_t)b * SAM_CTRL_WORDS;
    for (int i = threadIdx.x; i < SAM_CTRL_WORDS; i += blockDim.x) cb[i] = 0;
    uint2* root = W.root_tab + (size_t)b * W.root_cap;
    for (int i = threadIdx.x; i < W.root_cap; i += blockDim.x) root[i] = make_uint2(SAM_NONE, 0);
    if (threadIdx.x == 0) W.reset_flag[b] = 1;
}

// give the slabs of flagged slots back to the pool
__global__ void release_slabs_kernel(SamBatchView W) {
    size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t s = i; s < (size_t)W.pool_slabs; s += stride) {
        int owner = W.slab_owner[s];
        if (owner >= 0 && W.reset_flag[owner]) {
            W.slab_owner[s] = -1;
            int pos = atomicAdd(W.pool_hdr, 1);
            W.free_stack[pos] = (int32_t)s;
        }
    }
}

__global__ void clear_flags_kernel(SamBatchView W) {
    size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    if (i < (size_t)W.batch) W.reset_flag[i] = 0;
}

// one warp copies a slot's automaton into flat arrays
__global__ void dump_kernel(SamBatchView W, int32_t slot, int32_t* hdr, int32_t* length, int32_t* link,
                            int32_t* min_endpos, int32_t* deg, int32_t max_states,
                            int32_t* e_src, int32_t* e_tok, int32_t* e_tgt, int32_t max_edges) {
    const int lane = threadIdx.x;
    const uint32_t* cb = W.ctrl + (size_t)slot * SAM_CTRL_WORDS;
    const uint32_t n_states = cb[CB_NSTATES] ? cb[CB_NSTATES] : 1;
    const int rps_shift = W.slab_shift - 5;
    int n_edges = 0;
    // root: state 0
    if (lane == 0 && max_states > 0) { length[0] = 0; link[0] = -1; min_endpos[0] = 0; deg[0] = (int32_t)cb[CB_ROOTDEG]; }
    const uint2* root = W.root_tab + (size_t)slot * W.root_cap;
    for (int base = 0; base < W.root_cap; base += 32) {
        uint2 e = root[base + lane];
        unsigned has = __ballot_sync(0xFFFFFFFFu, e.x != SAM_NONE);
        if (e.x != SAM_NONE) {
            int k = n_edges + __popc(has & ((1u << lane) - 1));
            if (k < max_edges) { e_src[k] = 0; e_tok[k] = (int32_t)e.x; e_tgt[k] = (int32_t)(e.y & SAM_IDMASK); }
        }
        n_edges += __popc(has);
    }
    for (uint32_t s = 1; s < n_states; s++) {
        uint32_t slab = cb[CB_SLABTAB + (s >> rps_shift)];
        const uint4* rp = reinterpret_cast<const uint4*>(W.pool + ((size_t)slab << W.slab_shift) +
                                                         ((size_t)(s & ((1u << rps_shift) - 1)) << 5));
        const uint4 a = rp[0], b = rp[1];
        if (lane == 0 && s < (uint32_t)max_states) {
            length[s] = (int32_t)a.x; link[s] = (int32_t)a.y; min_endpos[s] = (int32_t)a.z; deg[s] = (int32_t)a.w;
        }
        if (a.w <= 2) {
            if (lane == 0) {
                if (a.w >= 1 && n_edges < max_edges) { e_src[n_edges] = (int32_t)s; e_tok[n_edges] = (int32_t)b.x; e_tgt[n_edges] = (int32_t)(b.y & SAM_IDMASK); }
                if (a.w == 2 && n_edges + 1 < max_edges) { e_src[n_edges + 1] = (int32_t)s; e_tok[n_edges + 1] = (int32_t)b.z; e_tgt[n_edges + 1] = (int32_t)(b.w & SAM_IDMASK); }
            }
            n_edges += (int)a.w;
        } else {
            const uint2* blk = reinterpret_cast<const uint2*>(W.pool + (size_t)b.x * 128);
            for (uint32_t i = lane; i < a.w; i += 32) {
                uint2 e = blk[i];
                int k = n_edges + (int)i;
                if (k < max_edges) { e_src[k] = (int32_t)s; e_tok[k] = (int32_t)e.x; e_tgt[k] = (int32_t)(e.y & SAM_IDMASK); }
            }
            n_edges += (int)a.w;
        }
    }
    if (lane == 0) { hdr[0] = (int32_t)cb[CB_NTOK]; hdr[1] = (int32_t)n_states; hdr[2] = n_edges; }
}

}  // namespace

// ---- helpers for callers that bring their own memory for a short-lived batch ----------------

// Lay a batch with these options out over `base` (device memory of at least *total bytes).
int sam_plan_view(const sam_batch_opts_t* opts, int32_t vocab, void* base, SamBatchView* view,
                  size_t* total, size_t* stage_words) {
    WsLayout w;
    int rc = plan(opts, &w);
    if (rc) return rc;
    if (total) *total = w.total;
    if (stage_words) *stage_words = w.stage_words;
    if (base && view) {
        char* b = (char*)base;
        view->pool_hdr = (int32_t*)(b + w.off_hdr);
        view->ctrl = (uint32_t*)(b + w.off_ctrl);
        view->free_stack = (int32_t*)(b + w.off_free);
        view->slab_owner = (int32_t*)(b + w.off_owner);
        view->reset_flag = (int32_t*)(b + w.off_reset);
        view->order = (int32_t*)(b + w.off_order);
        view->text = (int32_t*)(b + w.off_text);
        view->pstate = (uint32_t*)(b + w.off_pstate);
        view->root_tab = (uint2*)(b + w.off_root);
        view->stage = (int32_t*)(b + w.off_stage);
        view->pool = (unsigned char*)(b + w.off_pool);
        view->batch = opts->batch; view->max_seq_len = opts->max_seq_len; view->text_stride = w.text_stride;
        view->root_cap = w.root_cap; view->slab_shift = w.slab_shift;
        view->l_bias = opts->l_bias; view->min_match = opts->min_match;
        view->vocab = vocab;
        view->pool_slabs = w.pool_slabs;
        view->stop_token = opts->stop_token_plus_one - 1;
    }
    return SAM_OK;
}

// Put every slot of the view into the empty state and fill the slab pool's free stack.
int sam_launch_init(const SamBatchView& V, cudaStream_t s) {
    init_pool_kernel<<<296, 256, 0, s>>>(V);
    reset_slots_kernel<<<V.batch, 128, 0, s>>>(V, nullptr, V.batch);
    clear_flags_kernel<<<(V.batch + 255) / 256, 256, 0, s>>>(V);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { sam_set_cuda_error(e); return SAM_ERR_CUDA; }
    return SAM_OK;
}

extern "C" int sam_batch_workspace_bytes(const sam_batch_opts_t* opts, size_t* out) {
    if (!opts || !out) return SAM_ERR_ARG;
    WsLayout w;
    int rc = plan(opts, &w);
    if (rc) return rc;
    *out = w.total;
    return SAM_OK;
}

extern "C" int sam_batch_create(const sam_static_t* st, const sam_batch_opts_t* opts,
                                void* workspace_dev, size_t workspace_bytes, void* stream, sam_batch_t** out) {
    if (!out) return SAM_ERR_ARG;
    *out = nullptr;
    if (!opts || !workspace_dev) return SAM_ERR_ARG;
    if (!st && opts->vocab < 1) return SAM_ERR_ARG;
    WsLayout w;
    int rc = plan(opts, &w);
    if (rc) return rc;
    if (((uintptr_t)workspace_dev & 255) != 0 || workspace_bytes < w.total) return SAM_ERR_WORKSPACE;

    cudaPointerAttributes attr;
    cudaError_t e = cudaPointerGetAttributes(&attr, workspace_dev);
    if (e != cudaSuccess) { sam_set_cuda_error(e); cudaGetLastError(); return SAM_ERR_CUDA; }
    if (attr.type != cudaMemoryTypeDevice) return SAM_ERR_ARG;
    if (st && st->device != attr.device) return SAM_ERR_ARG;

    sam_batch* b = new (std::nothrow) sam_batch();
    if (!b) return SAM_ERR_NOMEM;
    memset(b, 0, sizeof(*b));
    b->device = attr.device;
    b->st = st;
    b->opts = *opts;
    b->workspace_bytes = w.total;
    b->max_host_stride = w.max_host_stride;
    b->stage_words = w.stage_words;
    char* base = (char*)workspace_dev;
    SamBatchView& V = b->view;
    V.pool_hdr = (int32_t*)(base + w.off_hdr);
    V.ctrl = (uint32_t*)(base + w.off_ctrl);
    V.free_stack = (int32_t*)(base + w.off_free);
    V.slab_owner = (int32_t*)(base + w.off_owner);
    V.reset_flag = (int32_t*)(base + w.off_reset);
    V.order = (int32_t*)(base + w.off_order);
    V.text = (int32_t*)(base + w.off_text);
    V.pstate = (uint32_t*)(base + w.off_pstate);
    V.root_tab = (uint2*)(base + w.off_root);
    V.stage = (int32_t*)(base + w.off_stage);
    V.pool = (unsigned char*)(base + w.off_pool);
    V.batch = opts->batch; V.max_seq_len = opts->max_seq_len; V.text_stride = w.text_stride;
    V.root_cap = w.root_cap; V.slab_shift = w.slab_shift;
    V.l_bias = opts->l_bias; V.min_match = opts->min_match;
    V.vocab = st ? st->info.vocab : opts->vocab;
    V.pool_slabs = w.pool_slabs;
    V.stop_token = opts->stop_token_plus_one - 1;

    SamDeviceGuard guard(b->device);
    if (!guard.ok) { delete b; return SAM_ERR_CUDA; }
    e = cudaHostAlloc((void**)&b->host_stage, (w.stage_words + 16) * 4, cudaHostAllocMapped);   // + the completion flag
    if (e == cudaSuccess) e = cudaHostGetDevicePointer((void**)&b->host_stage_dev, b->host_stage, 0);
    if (e != cudaSuccess) {
        sam_set_cuda_error(e); cudaGetLastError();
        if (b->host_stage) cudaFreeHost(b->host_stage);
        delete b;
        return SAM_ERR_NOMEM;
    }
    b->host_stage[w.stage_words] = 0;
    cudaStream_t s = (cudaStream_t)stream;
    init_pool_kernel<<<296, 256, 0, s>>>(V);
    reset_slots_kernel<<<V.batch, 128, 0, s>>>(V, nullptr, V.batch);
    clear_flags_kernel<<<(V.batch + 255) / 256, 256, 0, s>>>(V);
    e = cudaGetLastError();
    if (e != cudaSuccess) { sam_set_cuda_error(e); cudaFreeHost(b->host_stage); delete b; return SAM_ERR_CUDA; }
    *out = b;
    return SAM_OK;
}

extern "C" void sam_batch_destroy(sam_batch_t* b) {
    if (!b) return;
    SamDeviceGuard guard(b->device);
    if (b->host_stage) cudaFreeHost(b->host_stage);
    delete b;
}

extern "C" int sam_batch_reset(sam_batch_t* b, const int32_t* slots_host, int32_t n, void* stream) {
    if (!b) return SAM_ERR_ARG;
    if (!slots_host && n >= 0) return n == 0 ? SAM_OK : SAM_ERR_ARG;
    SamDeviceGuard guard(b->device);
    if (!guard.ok) return SAM_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    const SamBatchView& V = b->view;
    if (!slots_host) {
        reset_slots_kernel<<<V.batch, 128, 0, s>>>(V, nullptr, V.batch);
    } else {
        if (n > V.batch) return SAM_ERR_ARG;
        for (int32_t i = 0; i < n; i++) if (slots_host[i] < 0 || slots_host[i] >= V.batch) return SAM_ERR_ARG;
        if (n == 0) return SAM_OK;
        int32_t* list_dev = V.reset_flag + V.batch;           // second half of the reset area
        SAM_CUDA(cudaMemcpyAsync(list_dev, slots_host, (size_t)n * 4, cudaMemcpyHostToDevice, s));
        reset_slots_kernel<<<n, 128, 0, s>>>(V, list_dev, n);
    }
    release_slabs_kernel<<<296, 256, 0, s>>>(V);
    clear_flags_kernel<<<(V.batch + 255) / 256, 256, 0, s>>>(V);
    SAM_CUDA(cudaGetLastError());
    if (slots_host) SAM_CUDA(cudaStreamSynchronize(s));        // the caller's list may be reused at once
    return SAM_OK;
}

static int check_step_args(const sam_batch* b, const void* toks, int32_t stride, const void* counts, int32_t L,
                           const void* dt, const void* dl, const void* ml, const void* src, const void* status) {
    if (!b || !toks || !counts || !dt || !dl || !ml || !src || !status) return SAM_ERR_ARG;
    if (stride < 1 || L < 1 || L > b->opts.max_draft_len) return SAM_ERR_ARG;
    return SAM_OK;
}

extern "C" int sam_step(sam_batch_t* b, const int32_t* new_tokens_dev, int32_t stride,
                        const int32_t* counts_dev, int32_t L,
                        int32_t* draft_tokens_dev, int32_t* draft_len_dev, int32_t* match_len_dev,
                        int32_t* source_dev, int32_t* state_dev, int32_t* status_dev, void* stream) {
    int rc = check_step_args(b, new_tokens_dev, stride, counts_dev, L, draft_tokens_dev, draft_len_dev,
                             match_len_dev, source_dev, status_dev);
    if (rc) return rc;
    return sam_launch_step(b, new_tokens_dev, stride, counts_dev, L, draft_tokens_dev, draft_len_dev,
                           match_len_dev, source_dev, state_dev, status_dev, (cudaStream_t)stream);
}

extern "C" int sam_step_verified(sam_batch_t* b, const int32_t* target_tokens_dev, int32_t prev_L,
                                 const int32_t* prev_draft_tokens_dev, const int32_t* prev_draft_len_dev,
                                 const int32_t* max_new_dev, int32_t L,
                                 int32_t* draft_tokens_dev, int32_t* draft_len_dev, int32_t* match_len_dev,
                                 int32_t* source_dev, int32_t* state_dev, int32_t* status_dev,
                                 int32_t* counts_out_dev, int32_t* accepted_out_dev, void* stream) {
    int rc = check_step_args(b, target_tokens_dev, prev_L + 1, prev_draft_len_dev, L, draft_tokens_dev, draft_len_dev,
                             match_len_dev, source_dev, status_dev);
    if (rc) return rc;
    if (!prev_draft_tokens_dev || prev_L < 1 || prev_L > 128) return SAM_ERR_ARG;
    if (prev_draft_tokens_dev == draft_tokens_dev || prev_draft_len_dev == draft_len_dev) return SAM_ERR_ARG;
    return sam_launch_step_full(b, target_tokens_dev, prev_L + 1, nullptr, L, draft_tokens_dev, draft_len_dev,
                                match_len_dev, source_dev, state_dev, status_dev, (cudaStream_t)stream, nullptr, 0,
                                prev_draft_tokens_dev, prev_draft_len_dev, max_new_dev, counts_out_dev, accepted_out_dev);
}

extern "C" int sam_run_steps(sam_batch_t* b, const int32_t* new_tokens_dev, int32_t stride,
                             const int32_t* counts_dev, int32_t n_steps, int32_t L, int32_t out_per_step,
                             int32_t* draft_tokens_dev, int32_t* draft_len_dev, int32_t* match_len_dev,
                             int32_t* source_dev, int32_t* state_dev, int32_t* status_dev, void* stream) {
    int rc = check_step_args(b, new_tokens_dev, stride, counts_dev, L, draft_tokens_dev, draft_len_dev,
                             match_len_dev, source_dev, status_dev);
    if (rc) return rc;
    if (n_steps < 0) return SAM_ERR_ARG;
    const size_t B = (size_t)b->view.batch;
    for (int32_t s = 0; s < n_steps; s++) {
        const size_t o = out_per_step ? (size_t)s : 0;
        rc = sam_launch_step(b, new_tokens_dev + (size_t)s * B * stride, stride, counts_dev + (size_t)s * B, L,
                             draft_tokens_dev + o * B * L, draft_len_dev + o * B, match_len_dev + o * B * 2,
                             source_dev + o * B, state_dev ? state_dev + o * B * 2 : nullptr,
                             status_dev + o * B, (cudaStream_t)stream);
        if (rc) return rc;
    }
    return SAM_OK;
}

extern "C" int sam_step_host(sam_batch_t* b, const int32_t* new_tokens_host, int32_t stride,
                             const int32_t* counts_host, int32_t L,
                             int32_t* draft_tokens_host, int32_t* draft_len_host, int32_t* match_len_host,
                             int32_t* source_host, int32_t* state_host, int32_t* status_host, void* stream) {
    int rc = check_step_args(b, new_tokens_host, stride, counts_host, L, draft_tokens_host, draft_len_host,
                             match_len_host, source_host, status_host);
    if (rc) return rc;
    if (stride > b->max_host_stride) return SAM_ERR_ARG;
    SamDeviceGuard guard(b->device);
    if (!guard.ok) return SAM_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t B = (size_t)b->view.batch;
    // staging layout (int32 words): inputs [tokens B*stride | counts B], then outputs
    // [draft B*L | draft_len B | match_len 2B | source B | state 2B | status B]
    int32_t* dev = b->view.stage;
    int32_t* hst = b->host_stage;
    const size_t in_words = B * stride + B;
    const size_t out_words = B * L + 7 * B;
    if ((in_words + out_words) * 4 >= SAM_DIRECT_MIN_BYTES) {
        // Large steps: copying the arrays through the staging area on the host costs more than the step.
        // If every array the caller passed is page-locked memory the device can address (cudaHostAlloc /
        // cudaHostRegister: what a pinned torch tensor is), the kernel reads and writes them in place.
        const void* hp[8] = {new_tokens_host, counts_host, draft_tokens_host, draft_len_host, match_len_host,
                             source_host, status_host, state_host};
        void* dp[8] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
        bool direct = true;
        for (int i = 0; i < 8 && direct; i++) {
            if (!hp[i]) continue;                              // state_host may be null
            if (cudaHostGetDevicePointer(&dp[i], const_cast<void*>(hp[i]), 0) != cudaSuccess) { cudaGetLastError(); direct = false; }
        }
        if (direct) {
            volatile int32_t* flag = b->host_stage + b->stage_words;
            const int32_t seq = ++b->host_seq == 0 ? ++b->host_seq : b->host_seq;
            rc = sam_launch_step_signal(b, (const int32_t*)dp[0], stride, (const int32_t*)dp[1], L, (int32_t*)dp[2], (int32_t*)dp[3],
                                        (int32_t*)dp[4], (int32_t*)dp[5], (int32_t*)dp[7], (int32_t*)dp[6], s,
                                        b->host_stage_dev + b->stage_words, seq);
            if (rc) return rc;
            const auto t0 = std::chrono::steady_clock::now();
            bool seen = false;
            for (uint32_t spin = 0;; spin++) {
                if (*flag == seq) { seen = true; break; }
                if ((spin & 1023u) == 1023u &&
                    std::chrono::steady_clock::now() - t0 > std::chrono::microseconds(SAM_POLL_LIMIT_US)) break;
            }
            if (!seen) SAM_CUDA(cudaStreamSynchronize(s));
            return SAM_OK;
        }
    }
    memcpy(hst, new_tokens_host, B * stride * 4);
    memcpy(hst + B * stride, counts_host, B * 4);
    int32_t* ho = hst + in_words;
    if ((in_words + out_words) * 4 <= SAM_ZERO_COPY_MAX_BYTES) {
        // small steps: the kernel reads its inputs from, and writes its outputs to, the mapped host
        // staging area directly; the bytes cross the bus inside the kernel instead of in two copies
        int32_t* zd = b->host_stage_dev;
        int32_t* zo = zd + in_words;
        // completion: the last block writes this step's sequence number into the flag word behind the
        // staging area; polling it costs less than a stream synchronisation.  The poll is bounded;
        // past the bound (other work queued ahead on the stream, or a failed launch) it falls back.
        volatile int32_t* flag = b->host_stage + b->stage_words;
        const int32_t seq = ++b->host_seq == 0 ? ++b->host_seq : b->host_seq;
        rc = sam_launch_step_signal(b, zd, stride, zd + B * stride, L, zo, zo + B * L, zo + B * L + B, zo + B * L + 3 * B,
                                    zo + B * L + 4 * B, zo + B * L + 6 * B, s, b->host_stage_dev + b->stage_words, seq);
        if (rc) return rc;
        const auto t0 = std::chrono::steady_clock::now();
        bool seen = false;
        for (uint32_t spin = 0;; spin++) {
            if (*flag == seq) { seen = true; break; }
            if ((spin & 1023u) == 1023u &&
                std::chrono::steady_clock::now() - t0 > std::chrono::microseconds(SAM_POLL_LIMIT_US)) break;
        }
        if (!seen) SAM_CUDA(cudaStreamSynchronize(s));
    } else {
        SAM_CUDA(cudaMemcpyAsync(dev, hst, in_words * 4, cudaMemcpyHostToDevice, s));
        int32_t* o = dev + in_words;
        rc = sam_launch_step(b, dev, stride, dev + B * stride, L, o, o + B * L, o + B * L + B, o + B * L + 3 * B,
                             o + B * L + 4 * B, o + B * L + 6 * B, s);
        if (rc) return rc;
        SAM_CUDA(cudaMemcpyAsync(ho, o, out_words * 4, cudaMemcpyDeviceToHost, s));
        SAM_CUDA(cudaStreamSynchronize(s));
    }
    memcpy(draft_tokens_host, ho, B * L * 4);
    memcpy(draft_len_host, ho + B * L, B * 4);
    memcpy(match_len_host, ho + B * L + B, 2 * B * 4);
    memcpy(source_host, ho + B * L + 3 * B, B * 4);
    if (state_host) memcpy(state_host, ho + B * L + 4 * B, 2 * B * 4);
    memcpy(status_host, ho + B * L + 6 * B, B * 4);
    return SAM_OK;
}

extern "C" int sam_batch_launches_per_step(const sam_batch_t* b) {
    if (!b) return SAM_ERR_ARG;
    return sam_step_launch_count(b);
}

extern "C" int sam_batch_pool_info(sam_batch_t* b, int64_t* total_slabs, int64_t* free_slabs, void* stream) {
    if (!b || !total_slabs || !free_slabs) return SAM_ERR_ARG;
    SamDeviceGuard guard(b->device);
    if (!guard.ok) return SAM_ERR_CUDA;
    int32_t hdr[2] = {0, 0};
    SAM_CUDA(cudaMemcpyAsync(hdr, b->view.pool_hdr, 8, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    SAM_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    *free_slabs = hdr[0]; *total_slabs = hdr[1];
    return SAM_OK;
}

extern "C" int sam_batch_dump(sam_batch_t* b, int32_t slot, int32_t* n_tokens, int32_t* n_states,
                              int32_t* n_edges, int32_t* length, int32_t* link, int32_t* min_endpos,
                              int32_t* deg, int32_t max_states,
                              int32_t* edge_src, int32_t* edge_tok, int32_t* edge_tgt, int32_t max_edges,
                              void* stream) {
    if (!b || slot < 0 || slot >= b->view.batch || max_states < 0 || max_edges < 0) return SAM_ERR_ARG;
    if (max_states > 0 && (!length || !link || !min_endpos || !deg)) return SAM_ERR_ARG;
    if (max_edges > 0 && (!edge_src || !edge_tok || !edge_tgt)) return SAM_ERR_ARG;
    SamDeviceGuard guard(b->device);
    if (!guard.ok) return SAM_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t words = 4 + 4 * (size_t)max_states + 3 * (size_t)max_edges;
    int32_t* dev = nullptr;
    cudaError_t e = cudaMalloc(&dev, words * 4);
    if (e != cudaSuccess) { sam_set_cuda_error(e); cudaGetLastError(); return SAM_ERR_NOMEM; }
    int32_t* d_len = dev + 4; int32_t* d_link = d_len + max_states; int32_t* d_end = d_link + max_states;
    int32_t* d_deg = d_end + max_states; int32_t* d_es = d_deg + max_states; int32_t* d_et = d_es + max_edges;
    int32_t* d_eg = d_et + max_edges;
    dump_kernel<<<1, 32, 0, s>>>(b->view, slot, dev, d_len, d_link, d_end, d_deg, max_states, d_es, d_et, d_eg, max_edges);
    std::vector<int32_t> host;
    try { host.resize(words); } catch (const std::bad_alloc&) { cudaFree(dev); return SAM_ERR_NOMEM; }
    e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemcpyAsync(host.data(), dev, words * 4, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    cudaFree(dev);
    if (e != cudaSuccess) { sam_set_cuda_error(e); return SAM_ERR_CUDA; }
    if (n_tokens) *n_tokens = host[0];
    if (n_states) *n_states = host[1];
    if (n_edges) *n_edges = host[2];
    const int32_t ns = host[1] < max_states ? host[1] : max_states;
    const int32_t ne = host[2] < max_edges ? host[2] : max_edges;
    if (ns > 0) {
        memcpy(length, host.data() + 4, (size_t)ns * 4);
        memcpy(link, host.data() + 4 + max_states, (size_t)ns * 4);
        memcpy(min_endpos, host.data() + 4 + 2 * (size_t)max_states, (size_t)ns * 4);
        memcpy(deg, host.data() + 4 + 3 * (size_t)max_states, (size_t)ns * 4);
    }
    if (ne > 0) {
        const int32_t* eb = host.data() + 4 + 4 * (size_t)max_states;
        memcpy(edge_src, eb, (size_t)ne * 4);
        memcpy(edge_tok, eb + max_edges, (size_t)ne * 4);
        memcpy(edge_tgt, eb + 2 * (size_t)max_edges, (size_t)ne * 4);
    }
    return SAM_OK;
}
