// Tree drafts from the static automaton: best-first expansion over the top-k successors
// (Algorithm 5 of SAM-Decoding, "Drafting via Prim's Algorithm", with the successor frequencies of
// Appendix A.1/A.2).
//
// One warp per slot.  The queue lives in shared memory as plain arrays; an entry holds its path
// probability, state, token, parent node, the state's freq and the state's successor candidates
// (its two inline transitions, or its precomputed top-k if its transitions are hashed).  Because a
// state's candidates travel with its entry, expanding a popped node needs exactly one round of
// reads: lanes 0..n-1 each fetch one child's freq, record and, if flagged, top-k entry together.
// Popping is a strided scan of the queue with a warp arg-max (larger probability first, then the
// earlier push).  Probabilities are IEEE float32: quotient freq(child) / freq(state) rounded first,
// then the product with the parent's probability.
#include "common.h"

namespace {

constexpr unsigned FULL = 0xFFFFFFFFu;

struct TreeArgs {
    SamStaticView S;
    const int32_t* states; const int32_t* start_tokens;
    int32_t batch, max_size, k;
    int32_t* tokens; int32_t* parents; float* probs; int32_t* sizes;
};

// successor candidates of state u (id without flag) read by ONE lane: from the record when the
// state has at most two transitions, else from the top-k table.  Returns how many; cand[] gets
// (token, target | F) pairs.  hashed states come back in top-k order, inline ones in record order.
__device__ __forceinline__ int load_candidates(const SamStaticView& S, uint32_t u, bool flagged, int k,
                                               uint32_t ctok[SAM_TOPK_MAX], uint32_t ctgt[SAM_TOPK_MAX], bool& ordered) {
    ordered = false;
    if (!flagged) {
        const uint4 a = __ldg(S.rec + 2 * (size_t)u), b = __ldg(S.rec + 2 * (size_t)u + 1);
        int n = (int)(a.w < 2u ? a.w : 2u);
        if (a.w > 2u) n = 0;                      // unflagged reference to a hashed state cannot happen
        ctok[0] = b.x; ctgt[0] = b.y; ctok[1] = b.z; ctgt[1] = b.w;
        return n;
    }
    ordered = true;
    uint32_t at = sam_hash1(u) & S.topk_mask;
    for (uint32_t probe = 0; probe <= S.topk_mask; probe++) {
        // the whole 64-byte entry in one round of reads; the header decides afterwards
        const uint4 h = __ldg(S.topk + (size_t)at * 4), w1 = __ldg(S.topk + (size_t)at * 4 + 1),
                    w2 = __ldg(S.topk + (size_t)at * 4 + 2), w3 = __ldg(S.topk + (size_t)at * 4 + 3);
        if (h.x == u) {
            // layout: {state, n, 0, 0} {tok0..3} {tok4, tok5, tgt0, tgt1} {tgt2..5}
            ctok[0] = w1.x; ctok[1] = w1.y; ctok[2] = w1.z; ctok[3] = w1.w; ctok[4] = w2.x; ctok[5] = w2.y;
            ctgt[0] = w2.z; ctgt[1] = w2.w; ctgt[2] = w3.x; ctgt[3] = w3.y; ctgt[4] = w3.z; ctgt[5] = w3.w;
            int n = (int)h.y;
            return n < k ? n : k;
        }
        if (h.x == SAM_NONE) return 0;
        at = (at + 1) & S.topk_mask;
    }
    return 0;
}

__global__ void __launch_bounds__(32) tree_draft_kernel(const __grid_constant__ TreeArgs A) {
    extern __shared__ uint32_t smem[];
    const int b = blockIdx.x, lane = threadIdx.x;
    const int K = A.k, M = A.max_size;
    const int Q = M * K + 1;
    float* q_p = reinterpret_cast<float*>(smem);            // < 0: popped
    uint32_t* q_state = smem + Q;                           // id | F
    uint32_t* q_tok = smem + 2 * Q;
    int32_t* q_par = reinterpret_cast<int32_t*>(smem + 3 * Q);
    uint32_t* q_freq = smem + 4 * Q;
    uint32_t* q_n = smem + 5 * Q;                           // candidates | ordered << 8
    uint32_t* q_ctok = smem + 6 * Q;                        // [Q][SAM_TOPK_MAX]
    uint32_t* q_ctgt = smem + 6 * Q + (size_t)Q * SAM_TOPK_MAX;

    int32_t* out_tok = A.tokens + (size_t)b * M;
    int32_t* out_par = A.parents + (size_t)b * M;
    float* out_p = A.probs ? A.probs + (size_t)b * M : nullptr;
    for (int j = lane; j < M; j += 32) { out_tok[j] = -1; out_par[j] = -1; if (out_p) out_p[j] = 0.f; }

    const int32_t s0 = A.states[b];
    if (s0 <= 0 || (int64_t)s0 >= A.S.n_states) { if (lane == 0) A.sizes[b] = 0; return; }

    int qn = 0;
    if (lane == 0) {                                         // the start node: probability 1
        uint32_t ctok[SAM_TOPK_MAX], ctgt[SAM_TOPK_MAX];
        bool ordered;
        const bool flagged = __ldg(A.S.rec + 2 * (size_t)s0).w > 2u;
        const int n = load_candidates(A.S, (uint32_t)s0, flagged, K, ctok, ctgt, ordered);
        q_p[0] = 1.0f; q_state[0] = (uint32_t)s0; q_tok[0] = (uint32_t)A.start_tokens[b]; q_par[0] = -1;
        q_freq[0] = __ldg(A.S.freq + s0); q_n[0] = (uint32_t)n | (ordered ? 256u : 0u);
        for (int j = 0; j < SAM_TOPK_MAX; j++) { q_ctok[j] = ctok[j]; q_ctgt[j] = ctgt[j]; }
    }
    qn = 1;
    __syncwarp();

    int n_out = 0;
    while (n_out < M) {
        // pop: largest probability, earliest push among equals
        float bp = -1.0f; int bi = 0x7FFFFFFF;
        for (int i = lane; i < qn; i += 32) { const float p = q_p[i]; if (p > bp) { bp = p; bi = i; } }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float op = __shfl_xor_sync(FULL, bp, off); const int oi = __shfl_xor_sync(FULL, bi, off);
            if (op > bp || (op == bp && oi < bi)) { bp = op; bi = oi; }
        }
        if (bp < 0.0f) break;                                // queue empty
        const int node = n_out++;
        const uint32_t st = q_state[bi] & SAM_IDMASK, fs = q_freq[bi];
        const uint32_t nn = q_n[bi];
        const int n = (int)(nn & 255u); const bool ordered = (nn & 256u) != 0;
        if (lane == 0) {
            out_tok[node] = (int32_t)q_tok[bi]; out_par[node] = q_par[bi]; if (out_p) out_p[node] = bp;
        }
        __syncwarp();
        if (lane == 0) q_p[bi] = -1.0f;
        if (n_out >= M) break;                               // the last node needs no expansion
        (void)st;
        // expand: lane j takes candidate j
        uint32_t ctok = 0, ctgt = 0, cf = 0; int cn = 0; bool cord = false;
        uint32_t gtok[SAM_TOPK_MAX], gtgt[SAM_TOPK_MAX];
        if (lane < n) {
            ctok = q_ctok[(size_t)bi * SAM_TOPK_MAX + lane]; ctgt = q_ctgt[(size_t)bi * SAM_TOPK_MAX + lane];
            const uint32_t u = ctgt & SAM_IDMASK;
            cf = __ldg(A.S.freq + u);
            cn = load_candidates(A.S, u, (ctgt >> 31) != 0, K, gtok, gtgt, cord);
        }
        // order two inline candidates by (freq descending, token ascending); keep the first K
        int pos = lane;
        if (!ordered && n == 2) {
            const uint32_t of = __shfl_xor_sync(FULL, cf, 1), ot = __shfl_xor_sync(FULL, ctok, 1);
            if (lane < 2) {
                const bool other_first = of > cf || (of == cf && ot < ctok);
                pos = other_first ? 1 : 0;
            }
        }
        const int keep = n < K ? n : K;
        if (lane < n && pos < keep) {
            const int e = qn + pos;
            q_p[e] = __fmul_rn(bp, __fdiv_rn(__uint2float_rn(cf), __uint2float_rn(fs)));
            q_state[e] = ctgt; q_tok[e] = ctok; q_par[e] = node; q_freq[e] = cf;
            q_n[e] = (uint32_t)cn | (cord ? 256u : 0u);
            for (int j = 0; j < SAM_TOPK_MAX; j++) { q_ctok[(size_t)e * SAM_TOPK_MAX + j] = gtok[j]; q_ctgt[(size_t)e * SAM_TOPK_MAX + j] = gtgt[j]; }
        }
        qn += keep;
        __syncwarp();
    }
    if (lane == 0) A.sizes[b] = n_out;
}

}  // namespace

extern "C" int sam_tree_draft(const sam_static_t* st, int32_t batch, const int32_t* states_dev,
                              const int32_t* start_tokens_dev, int32_t max_size, int32_t k,
                              int32_t* tree_tokens_dev, int32_t* tree_parents_dev, float* tree_probs_dev,
                              int32_t* tree_size_dev, void* stream) {
    if (!st || !states_dev || !start_tokens_dev || !tree_tokens_dev || !tree_parents_dev || !tree_size_dev) return SAM_ERR_ARG;
    if (batch < 1 || max_size < 1 || max_size > 128 || k < 1) return SAM_ERR_ARG;
    if (st->info.tree_topk < 1 || k > st->info.tree_topk) return SAM_ERR_ARG;   // built without (enough) tree data
    SamDeviceGuard guard(st->device);
    if (!guard.ok) return SAM_ERR_CUDA;
    TreeArgs A;
    A.S = st->view; A.states = states_dev; A.start_tokens = start_tokens_dev;
    A.batch = batch; A.max_size = max_size; A.k = k;
    A.tokens = tree_tokens_dev; A.parents = tree_parents_dev; A.probs = tree_probs_dev; A.sizes = tree_size_dev;
    const size_t Q = (size_t)max_size * k + 1;
    const size_t smem = Q * (6 + 2 * SAM_TOPK_MAX) * sizeof(uint32_t);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(tree_draft_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) { sam_set_cuda_error(e); return SAM_ERR_CUDA; }
    }
    tree_draft_kernel<<<batch, 32, smem, (cudaStream_t)stream>>>(A);
    SAM_CUDA(cudaGetLastError());
    return SAM_OK;
}
