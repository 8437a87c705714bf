/*
 * samdraft.h — C ABI of libsamdraft: batched suffix-automaton draft retrieval on one GPU.
 *
 * The library implements the draft-retrieval path of SAM-Decoding (arXiv 2411.10666) for a batch
 * of decoding sequences:
 *   - a STATIC suffix automaton over a token corpus, built offline on the host (Build-SAM,
 *     Algorithm 3) and stored on the device;
 *   - one DYNAMIC suffix automaton per sequence, extended on the device with every accepted
 *     token (Expand, Algorithm 3) after the sequence's match state has been advanced on the
 *     automaton as it was (Transfer, Algorithm 1; order of Section 3.3);
 *   - the draft d = T[p+1 : p+n] read after the first end position p (min_endpos, Section 3.1)
 *     of the matched state, from the static text iff l1 > l2 + l_bias (Section 3.2).
 *
 * Conventions
 *   - Every function returns 0 on success or a negative sam_err_t; none aborts or throws.
 *   - "host" / "device" in a parameter comment says where the pointed-to memory must live.
 *     Device pointers must belong to the device the object was created on.
 *   - Tokens are int32 in [0, vocab).  Positions reported by the paper's algorithms are 1-based;
 *     nothing 1-based crosses this interface (only tokens, lengths and state ids do).
 *   - State ids are creation-order ids of Algorithm 3: root 0, each new state before its clone.
 *   - All device work is enqueued on the caller's stream (a cudaStream_t passed as void*; NULL
 *     is the legacy default stream) and is asynchronous unless stated otherwise.
 *   - Objects are not thread-safe; calls on one sam_batch_t must be externally ordered.
 */
#ifndef SAMDRAFT_H
#define SAMDRAFT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SAM_OK = 0,
    SAM_ERR_ARG = -1,        /* null pointer, size out of range, inconsistent options        */
    SAM_ERR_CUDA = -2,       /* a CUDA runtime call failed (sam_last_cuda_error has its code)  */
    SAM_ERR_NOMEM = -3,      /* host or device allocation failed                              */
    SAM_ERR_WORKSPACE = -4,  /* caller's workspace too small or misaligned                    */
    SAM_ERR_IO = -5,         /* file could not be read / written                              */
    SAM_ERR_FORMAT = -6,     /* file is not a static-automaton image, or its checksum is bad  */
    SAM_ERR_LIMIT = -7,      /* corpus or option exceeds what the layout can index            */
    SAM_ERR_NO_DEVICE = -8,  /* no usable CUDA device                                         */
    SAM_ERR_UNSUPPORTED = -9 /* this build of the library lacks the feature                   */
} sam_err_t;

/* Per-sequence status written by sam_step (status_dev).  Non-zero is sticky until reset. */
enum {
    SAM_SEQ_OK = 0,
    SAM_SEQ_CAPACITY = 1,    /* seq_len + count > max_seq_len, or the slab pool ran dry       */
    SAM_SEQ_WALK_LIMIT = 2,  /* a bounded probe / link walk hit its limit (corrupt state)     */
    SAM_SEQ_BAD_TOKEN = 3,   /* a token outside [0, vocab)                                    */
    SAM_SEQ_BAD_COUNT = 4    /* count < 0 or count > stride                                   */
};

/* source_dev values */
enum { SAM_SRC_NONE = 0, SAM_SRC_STATIC = 1, SAM_SRC_DYNAMIC = 2, SAM_SRC_AUXILIARY = 3 };

typedef struct sam_static sam_static_t;   /* device-resident static automaton, owned by the library */
typedef struct sam_batch sam_batch_t;     /* batch of sequences; its device memory is the caller's  */

typedef struct {
    double hash_load;        /* target load of the overflow-edge hash table, (0, 0.9]; 0 = 0.5 */
    int32_t keep_host_copy;  /* reserved, must be 0                                            */
    int32_t tree_topk;       /* 0 = no tree-draft data; k in 1..6 = also compute freq and the k most
                                frequent successors of every state (Appendix A.2) for sam_tree_draft */
} sam_build_opts_t;

typedef struct {
    int64_t n_tokens;        /* corpus length                                                  */
    int64_t n_states;        /* states of the automaton (<= 2 n_tokens - 1)                    */
    int64_t n_transitions;   /* transitions (<= 3 n_tokens - 4)                                */
    int64_t n_hash_edges;    /* transitions stored in the overflow hash table                  */
    int64_t hash_buckets;    /* 128-byte buckets of that table                                 */
    int32_t hash_max_probe;  /* longest bucket probe sequence any stored edge needs            */
    int32_t vocab;
    size_t device_bytes;     /* device memory held                                             */
    double build_seconds;    /* host construction time (0 for a loaded image)                  */
    int32_t tree_topk;       /* k the tree-draft data was built with (0: none)                 */
    int32_t reserved;
} sam_static_info_t;

typedef struct {
    int32_t batch;            /* number of sequence slots B, >= 1                              */
    int32_t max_seq_len;      /* most tokens (prompt + accepted) a slot may hold, >= 1         */
    int32_t max_draft_len;    /* largest L any sam_step will ask for, 1..128                   */
    int32_t l_bias;           /* static wins iff l1 > l2 + l_bias (Section 3.2); >= 0          */
    int32_t min_match;        /* a chosen match shorter than max(1, min_match) gives no draft  */
    int32_t vocab;            /* token range when there is no static automaton, else ignored   */
    int32_t max_host_stride;  /* largest stride sam_step_host accepts; 0 = 32                  */
    int32_t slab_bytes;       /* slab size, a power of two >= 4 KiB; 0 = max(16 KiB, pow2 >= 8*max_seq_len) */
    int64_t pool_slabs;       /* slabs in the shared pool; 0 = batch * (ceil(160 * max_seq_len / slab_bytes) + 2) */
    int32_t stop_token_plus_one; /* 0 = none; t + 1 = a draft ends before the first token t (e.g. the EOS
                                  that separates the documents of a concatenated corpus, Section 3.1) */
    int32_t reserved;         /* must be 0 */
} sam_batch_opts_t;

/* ---- static automaton -------------------------------------------------------------------- */

/* Build-SAM (Algorithm 3) over corpus_host[0, n_tokens) on the host, then store the result on
 * `device`: one 32-byte record per state (length, link, min_endpos and up to two transitions
 * inline), a dense row for the root, a bucketed (state, token) hash table for the remaining
 * transitions, and the corpus itself for draft reads.  Synchronous; this is the offline step.
 * corpus_host: host, n_tokens int32, each in [0, vocab); not retained.  opts may be NULL.
 * *out is owned by the library; release it with sam_static_destroy.
 * Errors: ARG (null, n_tokens < 1, vocab < 1, token out of range), LIMIT (n_tokens > 2^30),
 * NOMEM, CUDA. */
int sam_build_static(const int32_t* corpus_host, int64_t n_tokens, int32_t vocab, int device,
                     const sam_build_opts_t* opts, sam_static_t** out);

/* Write / read the device image of a built automaton so large corpora are indexed once.
 * The file holds a header (magic, version, sizes, FNV-1a checksum of the payload) and the raw
 * sections.  Both calls are synchronous.  Errors: ARG, IO, FORMAT, NOMEM, CUDA. */
int sam_static_save(const sam_static_t* st, const char* path);
int sam_static_load(const char* path, int device, sam_static_t** out);

int sam_static_info(const sam_static_t* st, sam_static_info_t* out);

/* Copy one state's record back to the host (synchronous; for inspection and tests).
 * next_tokens / next_targets receive up to max_edges of the state's transitions in no particular
 * order; *n_edges gets the state's out-degree (which may exceed max_edges).
 * For the root only the out-degree is reported through this call's edge arrays when max_edges
 * is smaller than it.  Errors: ARG (state out of range), CUDA. */
int sam_static_state(const sam_static_t* st, int64_t state, int32_t* length, int32_t* link,
                     int32_t* min_endpos, int32_t* n_edges,
                     int32_t* next_tokens, int32_t* next_targets, int32_t max_edges);

/* Copy length, link (root: -1), min_endpos and out-degree of the first max_states states to the
 * host (synchronous; inspection and tests).  Errors: ARG, NOMEM, CUDA. */
int sam_static_tables(const sam_static_t* st, int32_t* length, int32_t* link, int32_t* min_endpos,
                      int32_t* deg, int64_t max_states);

/* HOST ONLY, no device needed: run the same construction as sam_build_static and decode the image
 * it would upload (inline transitions, root row, hash buckets) back into flat tables; also checks
 * the image's internal consistency (hash reachability, has-hashed-transitions bits) and returns
 * FORMAT if that fails.  Arrays may be NULL to get the counts only.  For tests and inspection.
 * Errors: ARG, LIMIT, NOMEM, FORMAT. */
int sam_build_static_tables(const int32_t* corpus_host, int64_t n_tokens, int32_t vocab,
                            int64_t* n_states, int64_t* n_transitions, int32_t* hash_max_probe,
                            int32_t* length, int32_t* link, int32_t* min_endpos, int32_t* deg,
                            int64_t max_states,
                            int32_t* edge_src, int32_t* edge_tok, int32_t* edge_tgt, int64_t max_edges);

void sam_static_destroy(sam_static_t* st);

/* ---- batch of sequences ------------------------------------------------------------------- */

/* Bytes of device workspace a batch with these options needs (256-byte aligned base).
 * Errors: ARG. */
int sam_batch_workspace_bytes(const sam_batch_opts_t* opts, size_t* out);

/* Lay a batch out in workspace_dev (device memory the CALLER owns and must keep alive and
 * untouched until sam_batch_destroy) and initialise every slot to the empty sequence: empty
 * dynamic automaton, both matchers at the root.  st may be NULL (no static source: l1 = 0).
 * The per-sequence dynamic automata take their state records and edge blocks from a pool of
 * slabs shared by all slots, handed out on demand.  Initialisation kernels run on `stream`.
 * Errors: ARG, WORKSPACE (too small / base not 256-byte aligned), NOMEM, CUDA. */
int sam_batch_create(const sam_static_t* st, const sam_batch_opts_t* opts,
                     void* workspace_dev, size_t workspace_bytes, void* stream, sam_batch_t** out);

/* Return slots to the empty sequence and their slabs to the pool (continuous batching).
 * slots_host: host, n slot indices; NULL with n < 0 resets every slot.  Errors: ARG, CUDA. */
int sam_batch_reset(sam_batch_t* b, const int32_t* slots_host, int32_t n, void* stream);

/* One decoding step for all B slots (Sections 3.2, 3.3).  For slot i with m = counts[i]:
 * each of new_tokens[i, 0..m) is fed, in order, to Transfer on the static automaton, and to
 * Transfer-then-Expand on the slot's dynamic automaton; then the source is chosen and up to L
 * draft tokens are read.  m = 0 changes nothing and re-emits the draft of the current state; the
 * prompt is fed the same way (m = prompt length).
 *
 *   new_tokens_dev  device, int32 [B, stride]          counts_dev  device, int32 [B]
 *   L               1..max_draft_len
 *   draft_tokens_dev device, int32 [B, L]   drafted tokens, -1 from draft_len on
 *   draft_len_dev    device, int32 [B]      min(L, tokens that follow the first end position)
 *   match_len_dev    device, int32 [B, 2]   (l1 static, l2 dynamic)
 *   source_dev       device, int32 [B]      SAM_SRC_*
 *   state_dev        device, int32 [B, 2]   (static state, dynamic state); may be NULL
 *   status_dev       device, int32 [B]      SAM_SEQ_*; a failed slot reports zeros and -1 drafts
 *
 * Host-visible argument errors (null, L out of range, stride < 1) return ARG synchronously and
 * launch nothing; data-dependent problems are reported per slot in status_dev and freeze the
 * slot until it is reset.  A slot is validated (count, capacity, token range) before any of its
 * state changes.
 *
 * Stream order is all the call needs: new_tokens_dev and counts_dev may be written by the kernel
 * that precedes this call on `stream` (sam_accept_greedy, sam_step_verified's counts_out_dev, the
 * caller's own kernel).  The step reads them only after everything earlier on the stream has
 * completed.  For batches that take two launches (sam_batch_launches_per_step), the first launch
 * looks at counts_dev early, possibly before they are final, but only to decide in which order
 * the slots are started; no result depends on what it saw. */
int sam_step(sam_batch_t* b, const int32_t* new_tokens_dev, int32_t stride,
             const int32_t* counts_dev, int32_t L,
             int32_t* draft_tokens_dev, int32_t* draft_len_dev, int32_t* match_len_dev,
             int32_t* source_dev, int32_t* state_dev, int32_t* status_dev, void* stream);

/* Replay n_steps consecutive steps from device arrays without returning to the caller in
 * between: new_tokens_dev [n_steps, B, stride], counts_dev [n_steps, B].  If out_per_step is
 * non-zero every output array has a leading n_steps dimension and keeps each step's results,
 * otherwise the arrays are those of sam_step and hold the last step's.  The launches of each
 * step are those sam_step makes (sam_batch_launches_per_step). */
int sam_run_steps(sam_batch_t* b, const int32_t* new_tokens_dev, int32_t stride,
                  const int32_t* counts_dev, int32_t n_steps, int32_t L, int32_t out_per_step,
                  int32_t* draft_tokens_dev, int32_t* draft_len_dev, int32_t* match_len_dev,
                  int32_t* source_dev, int32_t* state_dev, int32_t* status_dev, void* stream);

/* sam_step with HOST arrays: copies new_tokens and counts to the device, runs the step, copies
 * every output back and waits for the stream — the end-to-end call a serving loop that keeps its
 * tokens on the host would make.  stride <= max_host_stride.  Any host memory works.  How the
 * bytes travel depends on the step's size: small steps go through a page-locked staging area that
 * the kernel reads and writes itself; from 64 KiB of arrays on, arrays that are ALL page-locked and
 * device-addressable (cudaHostAlloc, cudaHostRegister, a pinned torch tensor) are read and written
 * in place by the kernel, and any others are copied through the staging area.  state_host may be
 * NULL.  Synchronous: the results are in the arrays when the call returns.  Errors: as sam_step,
 * plus CUDA. */
int sam_step_host(sam_batch_t* b, const int32_t* new_tokens_host, int32_t stride,
                  const int32_t* counts_host, int32_t L,
                  int32_t* draft_tokens_host, int32_t* draft_len_host, int32_t* match_len_host,
                  int32_t* source_host, int32_t* state_host, int32_t* status_host, void* stream);

/* Copy slot's dynamic automaton to the host (synchronous; inspection and tests).
 * length/link/min_endpos/deg: host, max_states int32 each; edge_src/edge_tok/edge_tgt: host,
 * max_edges int32 each.  *n_states / *n_edges receive the true counts; arrays are filled up to
 * their capacity.  Errors: ARG, NOMEM, CUDA. */
int sam_batch_dump(sam_batch_t* b, int32_t slot, int32_t* n_tokens, int32_t* n_states,
                   int32_t* n_edges, int32_t* length, int32_t* link, int32_t* min_endpos,
                   int32_t* deg, int32_t max_states,
                   int32_t* edge_src, int32_t* edge_tok, int32_t* edge_tgt, int32_t max_edges,
                   void* stream);

/* Pool occupancy: slabs in the pool, slabs currently free.  Synchronous. */
int sam_batch_pool_info(sam_batch_t* b, int64_t* total_slabs, int64_t* free_slabs, void* stream);

/* Number of kernels one sam_step launches for this batch: 1, or 2 for a batch larger than the GPU holds
 * at once (a small kernel first orders the slots so that those with the most tokens start first; the
 * step's results do not depend on it).  sam_step_host, being synchronous, gains nothing from the order
 * when its kernel works on the host arrays in place, and then makes one launch whatever the batch.
 * Returns a negative sam_err_t for a null handle. */
int sam_batch_launches_per_step(const sam_batch_t* b);

/* Forget the batch.  The workspace is the caller's and is not freed. */
void sam_batch_destroy(sam_batch_t* b);

/* ---- closing the loop on the device -------------------------------------------------------- */

/* Greedy verification (Section 2.2): the target model has scored the draft; target_tokens_dev[i, j]
 * is its token for the position after the first j draft tokens (j = 0..L, so row i has L + 1
 * entries, of which draft_len[i] + 1 are read).  Slot i accepts a = the length of the longest
 * prefix of its draft that equals target[i, 0..a), and its accepted tokens x_accept are
 * target[i, 0..a] — the a confirmed draft tokens and the target's own next token — so
 * m = a + 1, clipped to `stride` and, if max_new_dev is given, to max_new_dev[i] (0 stops a slot).
 * Writes counts_dev[i] = m and new_tokens_dev[i, 0..m) (-1 beyond), ready to be the next sam_step's
 * input, and accepted_dev[i] = min(a, m) if accepted_dev is not NULL.
 *   draft_tokens_dev device int32 [B, L]; draft_len_dev [B]; target_tokens_dev [B, L+1];
 *   max_new_dev [B] or NULL; new_tokens_dev [B, stride]; counts_dev [B]; accepted_dev [B] or NULL.
 * Asynchronous on `stream`.  Errors: ARG, CUDA. */
int sam_accept_greedy(int32_t batch, const int32_t* draft_tokens_dev, const int32_t* draft_len_dev, int32_t L,
                      const int32_t* target_tokens_dev, const int32_t* max_new_dev,
                      int32_t* new_tokens_dev, int32_t stride, int32_t* counts_dev, int32_t* accepted_dev,
                      void* stream);

/* sam_accept_greedy and sam_step in one launch: slot i's accepted tokens are derived inside the step
 * kernel from its previous draft (prev_draft_tokens_dev [B, prev_L], prev_draft_len_dev [B]) and the
 * target's tokens (target_tokens_dev [B, prev_L + 1]) exactly as sam_accept_greedy derives them
 * (m = confirmed prefix + 1, clipped to max_new_dev[i] if given), and are fed to the automata at once;
 * the new draft and the other outputs are those of sam_step.  counts_out_dev / accepted_out_dev
 * ([B], may be NULL) receive m and the number of confirmed draft tokens.  The previous draft's
 * buffers must not be this call's output buffers (alternate between two sets).
 * Asynchronous on `stream`.  Errors: ARG, CUDA. */
int sam_step_verified(sam_batch_t* b, const int32_t* target_tokens_dev, int32_t prev_L,
                      const int32_t* prev_draft_tokens_dev, const int32_t* prev_draft_len_dev,
                      const int32_t* max_new_dev, int32_t L,
                      int32_t* draft_tokens_dev, int32_t* draft_len_dev, int32_t* match_len_dev,
                      int32_t* source_dev, int32_t* state_dev, int32_t* status_dev,
                      int32_t* counts_out_dev, int32_t* accepted_out_dev, void* stream);

/* Adaptive draft selection (Section 3.4): the auxiliary drafter stands in with a fixed virtual match
 * length l_threshold.  With min_match = l_threshold in sam_batch_opts_t, sam_step reports
 * source = SAM_SRC_NONE exactly where the automaton's chosen match is shorter than that; this call
 * then substitutes the auxiliary draft there, in place: for every slot with source == SAM_SRC_NONE
 * and aux_len > 0, draft_tokens[i, :] = aux_tokens[i, 0..aux_len) (-1 beyond), draft_len = aux_len,
 * source = SAM_SRC_AUXILIARY.  aux_tokens_dev device int32 [B, L]; aux_len_dev [B].
 * Asynchronous on `stream`.  Errors: ARG, CUDA. */
int sam_select_auxiliary(int32_t batch, int32_t L, int32_t* draft_tokens_dev, int32_t* draft_len_dev,
                         int32_t* source_dev, const int32_t* aux_tokens_dev, const int32_t* aux_len_dev,
                         void* stream);

/* ---- tree drafts from the static automaton --------------------------------------------------- */

/* Best-first tree draft over the top-k successors (Algorithm 5, with freq and top-k successors as in
 * Appendix A.1/A.2; the automaton must have been built with tree_topk >= k).  For slot i the queue
 * starts with (probability 1, states_dev[i], start_tokens_dev[i]); the most probable entry is
 * popped and appended until max_size nodes are out or the queue is empty; a popped node pushes its
 * k most frequent successors (freq descending, token ascending) with probability
 * p * (freq(successor) / freq(state)) in IEEE float32 (quotient rounded first).  Among equal
 * probabilities the entry pushed earlier is popped first.
 *   states_dev        device int32 [B]   static state ids (sam_step's state[:, 0]); <= 0 gives an empty tree
 *   start_tokens_dev  device int32 [B]   the token of node 0 (the last accepted token)
 *   max_size 1..128, k 1..tree_topk
 *   tree_tokens_dev   device int32 [B, max_size]  tokens in pop order, -1 beyond tree_size
 *   tree_parents_dev  device int32 [B, max_size]  index of each node's parent, -1 for node 0 and beyond
 *   tree_probs_dev    device float [B, max_size]  path probabilities; may be NULL
 *   tree_size_dev     device int32 [B]
 * Asynchronous on `stream`.  Errors: ARG (no tree data, k too large, sizes), CUDA. */
int sam_tree_draft(const sam_static_t* st, int32_t batch, const int32_t* states_dev,
                   const int32_t* start_tokens_dev, int32_t max_size, int32_t k,
                   int32_t* tree_tokens_dev, int32_t* tree_parents_dev, float* tree_probs_dev,
                   int32_t* tree_size_dev, void* stream);

/* Copy freq (occurrences of each state's substrings in the corpus) of the first max_states states to
 * the host (synchronous; inspection and tests).  Errors: ARG (no tree data), CUDA. */
int sam_static_freq(const sam_static_t* st, uint32_t* freq_host, int64_t max_states);

/* ---- retrieval without any allocation ------------------------------------------------------ */

/* (The paper has no counterpart to this call; it exists for deployment reasons only.)
 *
 * One-shot retrieval for callers that cannot allocate device memory: a drafting hook that runs
 * inside an inference server which has already given the device's free memory to its own KV-cache
 * pool, or any component held to a "no allocation after start-up" rule.  Such a caller cannot
 * provide the workspace sam_batch_create needs, so this call keeps the per-sequence automata in a
 * fixed scratch array that is part of the library image: sam_noalloc_capacity_bytes() bytes
 * (8 MiB), resident on every GPU that loads the library until the process exits.
 *
 * Semantics: exactly sam_batch_create on an empty batch of `batch` slots with max_seq_len = stride,
 * followed by one sam_step — each slot i starts EMPTY, is fed tokens_dev[i, 0..counts_dev[i]) (its
 * whole text so far: prompt plus accepted tokens) and reports the draft, lengths, source, states
 * and status exactly as sam_step does.  Nothing persists between calls.
 *   st may be NULL (then `vocab` gives the token range and l1 = 0); otherwise vocab is ignored.
 *   tokens_dev device int32 [batch, stride]; counts_dev device int32 [batch]; outputs as sam_step
 *   (state_dev may be NULL); l_bias and min_match as in sam_batch_opts_t; L in 1..128.
 * Limits and errors: the layout for (batch, stride) must fit the scratch array, otherwise LIMIT is
 * returned and nothing is launched (for scale: 16 slots of 1024 tokens need about 3.5 MiB); ARG for
 * null pointers or out-of-range sizes; CUDA if the runtime fails.
 * The call makes no cudaMalloc / cudaFree / pinned-host allocation.  The first call on a device
 * looks up the array's device address (cudaGetSymbolAddress with that device current) and caches
 * it; make that first call before any stream capture begins.  Work is enqueued on `stream` and is
 * asynchronous.  All calls on a device share the one array and each call re-initialises it, so two
 * calls whose kernels can overlap on the GPU (different streams, or other threads) race with each
 * other: keep them on one stream or order them yourself. */
int sam_retrieve_noalloc(const sam_static_t* st, int32_t vocab, int32_t batch,
                         const int32_t* tokens_dev, int32_t stride, const int32_t* counts_dev,
                         int32_t L, int32_t l_bias, int32_t min_match,
                         int32_t* draft_tokens_dev, int32_t* draft_len_dev, int32_t* match_len_dev,
                         int32_t* source_dev, int32_t* state_dev, int32_t* status_dev, void* stream);

/* Size of the built-in scratch array in bytes. */
size_t sam_noalloc_capacity_bytes(void);

/* ---- memory-system probes (the denominators of the random-access roofline) ---------------- */

/* Independent uniformly random aligned reads of `granule` bytes (32, 64 or 128) over
 * buf_dev[0, footprint_bytes): every SM full of warps, several loads in flight per thread.
 * Runs `iters` timed launches after one warm-up; *gbps gets bytes read / best time, *mreq_s the
 * matching requests per microsecond.  buf_dev: device, footprint_bytes, caller-owned (contents
 * irrelevant).  Synchronous.  Errors: ARG, CUDA. */
int sam_probe_random_read(void* buf_dev, size_t footprint_bytes, int32_t granule, int32_t iters,
                          void* stream, double* gbps, double* mreq_s);

/* Dependent-load latency: `chains` single-thread chains (one per block, 1..65536) each chase a
 * random cyclic permutation of the 128-byte lines of buf_dev[0, footprint_bytes) for `hops` hops,
 * starting at evenly spaced points of the cycle; *ns_per_hop gets the time per hop of one chain
 * (so chains / ns_per_hop is the rate of dependent reads at that concurrency).  The permutation is
 * written into buf_dev by this call.  Synchronous.  Errors: ARG, NOMEM, CUDA. */
int sam_probe_chase(void* buf_dev, size_t footprint_bytes, int64_t hops, int32_t chains,
                    void* stream, double* ns_per_hop);

/* ---- operation counters (library built with -DSAM_COUNTERS) -------------------------------- */

/* What the step kernels can count per slot: the operations the paper's algorithms are made of — the link and
 * next moves of Transfer on the static automaton (Algorithm 1; their sum is what Appendix A.3 bounds by two per
 * token), and of Expand on the slot's own automaton the transitions added on the suffix-link walk, the clones,
 * the transitions a clone copies and the redirected transitions (Algorithm 3) — plus, per chain, the rounds of
 * dependent reads it waited for (a read whose address came out of the read before it).  The regular build
 * counts nothing and costs nothing; a second build of the same sources with -DSAM_COUNTERS does. */
enum {
    SAM_CNT_STATIC_ROUNDS = 0, SAM_CNT_STATIC_LINK_MOVES, SAM_CNT_STATIC_NEXT_MOVES,
    SAM_CNT_DYNAMIC_ROUNDS, SAM_CNT_WALK_INSERTS, SAM_CNT_CLONES, SAM_CNT_COPIED_EDGES, SAM_CNT_REDIRECTS,
    SAM_CNT_TOKENS, SAM_CNT_SEQ_STEPS,
    SAM_N_COUNTERS = 12
};

/* 1 if this library was built with the counters, else 0. */
int sam_counters_available(void);

/* Make every later step on the current device add its counts to counters_dev, device uint64
 * [slots, SAM_N_COUNTERS] (caller-owned, zeroed by the caller; slot i of ANY batch adds to row i, so attach one
 * batch's array at a time); NULL with slots 0 detaches.  Synchronous with respect to the host; issue it when
 * no step is in flight.  Errors: UNSUPPORTED in the regular build, ARG, CUDA. */
int sam_counters_attach(uint64_t* counters_dev, int32_t slots);

/* ---- diagnostics --------------------------------------------------------------------------- */

const char* sam_strerror(int err);
int sam_last_cuda_error(void);          /* cudaError_t of the last failed runtime call, else 0 */
const char* sam_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SAMDRAFT_H */
