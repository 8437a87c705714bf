// Closing the decoding loop on the device: greedy verification of a draft against the target
// model's tokens (Section 2.2 of SAM-Decoding) produces the next step's counts / new_tokens without
// a host round trip, and the adaptive choice between the automaton's draft and an auxiliary
// drafter's (Section 3.4) substitutes the auxiliary draft where the automaton's match is too short.
#include "common.h"

namespace {

// one warp per slot
__global__ void accept_greedy_kernel(int32_t batch, const int32_t* __restrict__ draft, const int32_t* __restrict__ draft_len,
                                     int32_t L, const int32_t* __restrict__ target, const int32_t* __restrict__ max_new,
                                     int32_t* __restrict__ new_tokens, int32_t stride, int32_t* __restrict__ counts,
                                     int32_t* __restrict__ accepted) {
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (b >= batch) return;
    int dl = draft_len[b];
    dl = dl < 0 ? 0 : (dl > L ? L : dl);
    const int32_t* d = draft + (size_t)b * L;
    const int32_t* t = target + (size_t)b * (L + 1);
    // a = length of the longest prefix of the draft that the target reproduces
    int a = dl;
    for (int base = 0; base < dl; base += 32) {
        const int j = base + lane;
        const bool differs = j < dl && d[j] != t[j];
        const unsigned bad = __ballot_sync(0xFFFFFFFFu, differs);
        if (bad) { a = base + __ffs(bad) - 1; break; }
    }
    int m = a + 1;                                   // the matching draft tokens and the target's next one
    if (m > stride) m = stride;
    if (max_new) { int cap = max_new[b]; if (cap < 0) cap = 0; if (m > cap) m = cap; }
    for (int j = lane; j < stride; j += 32) new_tokens[(size_t)b * stride + j] = j < m ? t[j] : -1;
    if (lane == 0) { counts[b] = m; if (accepted) accepted[b] = a < m ? a : m; }
}

__global__ void select_auxiliary_kernel(int32_t batch, int32_t L, int32_t* draft, int32_t* draft_len, int32_t* source,
                                        const int32_t* __restrict__ aux, const int32_t* __restrict__ aux_len) {
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (b >= batch) return;
    if (source[b] != SAM_SRC_NONE) return;
    int al = aux_len[b];
    al = al < 0 ? 0 : (al > L ? L : al);
    if (al == 0) return;
    for (int j = lane; j < L; j += 32) draft[(size_t)b * L + j] = j < al ? aux[(size_t)b * L + j] : -1;
    if (lane == 0) { draft_len[b] = al; source[b] = SAM_SRC_AUXILIARY; }
}

}  // namespace

extern "C" int sam_accept_greedy(int32_t batch, const int32_t* draft_tokens_dev, const int32_t* draft_len_dev, int32_t L,
                                 const int32_t* target_tokens_dev, const int32_t* max_new_dev,
                                 int32_t* new_tokens_dev, int32_t stride, int32_t* counts_dev, int32_t* accepted_dev,
                                 void* stream) {
    if (!draft_tokens_dev || !draft_len_dev || !target_tokens_dev || !new_tokens_dev || !counts_dev) return SAM_ERR_ARG;
    if (batch < 1 || L < 1 || stride < 1) return SAM_ERR_ARG;
    const int warps = 4;
    accept_greedy_kernel<<<(batch + warps - 1) / warps, warps * 32, 0, (cudaStream_t)stream>>>(
        batch, draft_tokens_dev, draft_len_dev, L, target_tokens_dev, max_new_dev, new_tokens_dev, stride, counts_dev,
        accepted_dev);
    SAM_CUDA(cudaGetLastError());
    return SAM_OK;
}

extern "C" int sam_select_auxiliary(int32_t batch, int32_t L, int32_t* draft_tokens_dev, int32_t* draft_len_dev,
                                    int32_t* source_dev, const int32_t* aux_tokens_dev, const int32_t* aux_len_dev,
                                    void* stream) {
    if (!draft_tokens_dev || !draft_len_dev || !source_dev || !aux_tokens_dev || !aux_len_dev) return SAM_ERR_ARG;
    if (batch < 1 || L < 1) return SAM_ERR_ARG;
    const int warps = 4;
    select_auxiliary_kernel<<<(batch + warps - 1) / warps, warps * 32, 0, (cudaStream_t)stream>>>(
        batch, L, draft_tokens_dev, draft_len_dev, source_dev, aux_tokens_dev, aux_len_dev);
    SAM_CUDA(cudaGetLastError());
    return SAM_OK;
}
