// Internal definitions shared by the library's translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include "layout.h"
#include "../../include/samdraft.h"

struct sam_static {
    int device;
    void* dev_base;               // one allocation holding every section
    size_t dev_bytes;
    size_t off_rec, off_root, off_hash, off_corpus, off_freq, off_topk, off_pstate;   // section offsets in dev_base
    size_t len_rec, len_root, len_hash, len_corpus, len_freq, len_topk, len_pstate;   // section sizes in bytes
    SamStaticView view;
    sam_static_info_t info;
};

struct sam_batch {
    int device;
    const sam_static* st;
    sam_batch_opts_t opts;
    SamBatchView view;
    size_t workspace_bytes;
    int32_t max_host_stride;
    size_t stage_words;           // int32 words of device staging
    int32_t* host_stage;          // pinned, device-mapped host staging area
    int32_t* host_stage_dev;      // the same memory as the device addresses it
    int32_t host_seq;             // sequence number of the last host-array step (completion flag value)
    mutable int32_t order_phase;  // which of the two slot-order buffers the next large-batch step uses
};

void sam_set_cuda_error(cudaError_t e);

#define SAM_CUDA(call)                                          \
    do {                                                        \
        cudaError_t _e = (call);                                \
        if (_e != cudaSuccess) { sam_set_cuda_error(_e); return SAM_ERR_CUDA; } \
    } while (0)

// RAII device switch
struct SamDeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit SamDeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~SamDeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

static inline size_t sam_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// launchers implemented in step.cu
int sam_launch_step(const sam_batch* b, const int32_t* new_tokens, int32_t stride, const int32_t* counts,
                    int32_t L, int32_t* draft_tokens, int32_t* draft_len, int32_t* match_len,
                    int32_t* source, int32_t* state, int32_t* status, cudaStream_t stream);

int sam_launch_step_signal(const sam_batch* b, const int32_t* new_tokens, int32_t stride, const int32_t* counts,
                           int32_t L, int32_t* draft_tokens, int32_t* draft_len, int32_t* match_len,
                           int32_t* source, int32_t* state, int32_t* status, cudaStream_t stream,
                           int32_t* done_flag_dev, int32_t done_seq);

int sam_launch_step_full(const sam_batch* b, const int32_t* new_tokens, int32_t stride, const int32_t* counts,
                         int32_t L, int32_t* draft_tokens, int32_t* draft_len, int32_t* match_len,
                         int32_t* source, int32_t* state, int32_t* status, cudaStream_t stream,
                         int32_t* done_flag_dev, int32_t done_seq,
                         const int32_t* v_draft, const int32_t* v_draft_len, const int32_t* v_max_new,
                         int32_t* v_counts_out, int32_t* v_accepted_out);

// 1, or 2 when the batch is large enough for the slot-ordering kernel (step.cu)
int sam_step_launch_count(const sam_batch* b);

// helpers implemented in batch.cu
int sam_plan_view(const sam_batch_opts_t* opts, int32_t vocab, void* base, SamBatchView* view,
                  size_t* total, size_t* stage_words);
int sam_launch_init(const SamBatchView& V, cudaStream_t s);
