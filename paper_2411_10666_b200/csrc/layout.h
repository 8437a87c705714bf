// Device data layout shared by the host-side static builder and the kernels.
//
// STATIC automaton (read-only while kernels run)
//   rec       : 32 bytes per state, two 16-byte words
//                 a = { len, link | F, min_endpos, deg }
//                 b = { tok0, tgt0 | F, tok1, tgt1 | F }      (first two transitions, inline)
//               F (bit 31) on a state reference says "that state has transitions in the hash
//               table", so a matcher arriving there can issue the bucket read together with the
//               record read instead of after it.  A state with deg <= 2 is one 32-byte sector.
//   root_row  : vocab x uint32, tgt | F or SAM_NONE — the root's transitions, dense.
//   hash      : buckets of 8 x 16-byte entries { state, tok, tgt | F, 0 } = one 128-byte line;
//               holds the third and later transitions of states with deg > 2.  Home bucket =
//               hash(state, tok) & mask, overflow goes to the following buckets.  An empty entry
//               has state == SAM_NONE; a bucket with an empty entry ends a probe sequence.
//   corpus    : the int32 token text, padded so vector reads past the end stay in bounds.
//   pstate    : uint32 per corpus token: id | F of the state Build-SAM created for it (the state of the
//               whole prefix ending there; exactly the states with len == min_endpos).  The transition
//               of such a state on the next corpus token is solid and therefore never redirected: it
//               leads to the next entry of this array.  A match that sits in a prefix state and goes on
//               as the corpus does can take its states from this array instead of one record after the
//               other; a token that differs from the corpus takes the ordinary Transfer (the state may
//               well have other transitions and other occurrences).  Derived on the device after each upload.
//   freq, topk: optional, for tree drafts — the occurrence count of every state, and for states
//               with hashed transitions their k most frequent successors (a state with at most two
//               transitions has them all in its record).
//
// DYNAMIC automata (one per sequence slot, written by the slot's own warp only)
//   rec       : 32 bytes per state, in slabs from the shared pool, addressed through the slot's
//               slab table:  a = { len, link, min_endpos, deg }
//                 deg <= 2 : b = { tok0, tgt0 | S, tok1, tgt1 | S }
//                 deg  > 2 : b = { block offset (128-byte units from the pool base), capacity, 0, 0 }
//               S (bit 31) on a transition marks it solid: len[src] + 1 == len[tgt].  Lengths never
//               change once a state exists, so the bit is fixed when the transition is written and
//               Expand's "p.length + 1 = q.length" test needs no read of q.
//   block     : capacity (16 * 2^k) x 8-byte { tok, tgt | S }, first `deg` used, unordered.
//   root table: per slot, 8-byte { tok, tgt | S } entries, linear probing from the start of the
//               token's home bucket (8 entries = 64 bytes); tok == SAM_NONE is empty.  A warp reads
//               32 consecutive entries per probe; a single lane can settle most lookups from the
//               home bucket alone (found, or absent because the bucket still has an empty entry).
//   text      : per slot, int32[max_seq_len].
//   pstate    : per slot, uint32[max_seq_len]: pstate[i] is the id of the state Expand created for token i
//               (the state of the whole prefix of length i + 1), so the states along an earlier
//               occurrence of a passage can be addressed without following their transitions.
#pragma once
#include <stdint.h>
#include <vector_types.h>

#if defined(__CUDACC__)
#define SAM_HD __host__ __device__ __forceinline__
#else
#define SAM_HD inline
#endif

#define SAM_NONE 0xFFFFFFFFu
#define SAM_FLAG 0x80000000u
#define SAM_IDMASK 0x7FFFFFFFu

#define SAM_HASH_BUCKET 8          // entries per static hash bucket (8 x 16 B = 128 B)
#define SAM_ROOT_BUCKET 8          // entries per dynamic root-table bucket (8 x 8 B = 64 B)
#define SAM_BLOCK_MIN 16           // smallest dynamic edge block (16 x 8 B = 128 B)
#define SAM_MAX_REC_SLABS 32       // entries of a slot's state-slab table (one per lane)
#define SAM_CTRL_WORDS 64          // per-slot control block, 256 bytes

// control-block word indices
enum {
    CB_STATUS = 0, CB_NTOK, CB_NSTATES, CB_LAST, CB_S1, CB_L1, CB_S2, CB_L2,
    CB_S1FLAG, CB_BLK_CUR, CB_BLK_END, CB_NRECSLABS, CB_ROOTDEG,
    CB_ARRIVE,        // split step: how many of the slot's two sides have finished (parity: 2 per step)
    CB_NTOK_S,        // the text length as the static side keeps it (it may not read CB_NTOK while the dynamic side writes it)
    CB_ERR_S,         // split step: error met by the static side (walk limit), 0 otherwise
    CB_SLABTAB = 16,  // .. 47
    CB_REC1 = 48,     // .. 55: copy of the static match state's record (valid when s1 != 0)
    CB_REC2 = 56      // .. 63: copy of the dynamic match state's record (valid when s2 != 0)
};

struct SamStaticRec {   // 32 bytes
    int32_t len; uint32_t link; int32_t min_endpos; uint32_t deg;
    uint32_t tok0, tgt0, tok1, tgt1;
};

struct SamHashEnt { uint32_t state, tok, tgt, pad; };   // 16 bytes

#define SAM_TOPK_MAX 6
// Top-k successors of a state with hashed transitions (freq descending, token ascending): 64 bytes.
// Kept in an open-addressing table keyed by state (linear probing, state == SAM_NONE is empty).
struct SamTopkEnt { uint32_t state, n, pad0, pad1; uint32_t tok[SAM_TOPK_MAX]; uint32_t tgt[SAM_TOPK_MAX]; };

// 64-bit multiplicative mix of (state, token); upper half is the hash.
SAM_HD uint32_t sam_hash2(uint32_t state, uint32_t tok) {
    uint64_t k = ((uint64_t)state << 32) | tok;
    k *= 0x9E3779B97F4A7C15ull;
    k ^= k >> 29;
    k *= 0xBF58476D1CE4E5B9ull;
    return (uint32_t)(k >> 32);
}

SAM_HD uint32_t sam_hash1(uint32_t tok) {
    uint32_t k = tok * 0x9E3779B1u;
    k ^= k >> 15;
    k *= 0x85EBCA77u;
    return k ^ (k >> 13);
}

// Device-side view of a static automaton (plain pointers; lives in the sam_static object).
struct SamStaticView {
    const uint4* rec;
    const uint32_t* root_row;
    const uint4* hash;
    const int32_t* corpus;
    uint32_t hash_mask;       // buckets - 1
    int32_t hash_max_probe;
    int32_t vocab;
    int64_t n_tokens;
    int64_t n_states;
    // tree drafts (present when the automaton was built with tree_topk > 0)
    const uint32_t* freq;     // occurrences of each state's substrings in the corpus
    const uint4* topk;        // SamTopkEnt table, four 16-byte words per entry
    uint32_t topk_mask;       // entries - 1
    int32_t tree_k;           // successors kept per hashed state (0: no tree data)
    const uint32_t* pstate;   // [n_tokens]: id | F of the state of the prefix ending with corpus token i
};

// Device-side view of a batch workspace.
struct SamBatchView {
    uint32_t* ctrl;           // [B][SAM_CTRL_WORDS]
    int32_t* pool_hdr;        // [0] free slabs, [1] total slabs
    int32_t* free_stack;      // [pool_slabs]
    int32_t* slab_owner;      // [pool_slabs], -1 = free
    int32_t* reset_flag;      // [B]
    int32_t* order;           // [3][B] + 16: slots sorted by their step's token count (large batches), two buffers in turn; the sort keys; per buffer, at 3B + 8 x buffer, the number of slots with many tokens
    int32_t* text;            // [B][text_stride]
    uint32_t* pstate;         // [B][text_stride]: id of the state created by each text position
    uint2* root_tab;          // [B][root_cap]
    unsigned char* pool;      // pool_slabs * slab_bytes
    int32_t* stage;           // staging for sam_step_host (inputs then outputs)
    int32_t batch, max_seq_len, text_stride, root_cap;
    int32_t slab_shift;       // log2(slab_bytes)
    int32_t l_bias, min_match, vocab;
    int32_t pool_slabs;
    int32_t stop_token;       // drafts end before the first such token; -1 = none
};
