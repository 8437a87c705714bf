// The hot kernel: one decoding step of SAM-Decoding's draft retrieval for a batch of sequences.
//
// One block of two warps per sequence slot.  Warp 0 advances the slot's match state through the
// STATIC automaton (Transfer, Algorithm 1) for each accepted token; warp 1 extends the slot's own
// DYNAMIC automaton (Expand, Algorithm 3) with the same tokens and keeps its match state, which
// after each Expand is link[last] with length len[link[last]] (the state Transfer would reach on
// the automaton as it was before the token, Section 3.3, made canonical).  Both warps then read
// the first end position of their state, fetch their candidate draft speculatively, and the
// source rule l1 > l2 + l_bias (Section 3.2) picks which one is written out.
//
// Each warp runs one dependent chain of memory reads, so the work is latency-bound, and the code
// is organised around the number of read round trips per step:
//   - everything a step needs to start (64 control words with copies of both match states'
//     records, the count, the first 32 tokens) is read in one round trip;
//   - values are warp-uniform (all lanes read the same 32-byte record: one request); lanes work
//     side by side only where a structure is wide (a 128-byte hash bucket, a window of 32 root-table
//     entries, an edge block, the draft read);
//   - independent reads go out together: a static state's record with its hash bucket, the root-row
//     entries of all tokens of the step, and the dynamic root-table lookups of all tokens of a chunk,
//     one lane per token;
//   - runs of tokens that are new to the sequence while nothing is matched are extended by the lanes
//     in parallel (each such Expand is three independent writes);
//   - runs of tokens that repeat a passage of the sequence and make every Expand clone are extended by
//     the lanes in parallel as well: the states the clones are made from are guessed (position -> state
//     map, or ids two apart), read in one round trip and checked (dyn_repeat_run);
//   - a static match that sits in the state of a whole corpus prefix is advanced by comparing the step's
//     tokens with the corpus, its state read from the corpus' position -> state array (a prefix state's
//     transition on the next corpus token always leads to the next prefix state);
//   - when the batch is larger than the GPU holds at once, the slots with the most tokens are started
//     first (order_slots_kernel);
//   - from 8192 slots on the two sides of a slot run as separate one-warp blocks (the static side of a slot
//     with few tokens on a single lane), neither waiting for the other, and whichever finishes last writes
//     the slot's outputs (sam_step_split_kernel, further down).
#include "common.h"

#include <cstring>

// Operation counters (library built with -DSAM_COUNTERS only): per slot, what its two chains did — the
// moves and insertions Algorithms 1 and 3 count, and the rounds of dependent reads each chain waited for.
// They exist to be compared with the CPU oracle's counters and to put a number on the latency bound;
// the regular build carries none of this.
#ifdef SAM_COUNTERS
__device__ unsigned long long* g_sam_counters = nullptr;     // [slots][SAM_N_COUNTERS]
__device__ int g_sam_counter_slots = 0;
#define SAM_COUNT(x, n) ((x) += (n))
#else
#define SAM_COUNT(x, n) ((void)0)
#endif

namespace {

constexpr unsigned FULL = 0xFFFFFFFFu;

// counts of one chain of one slot in one step (registers; dropped by the compiler in the regular build)
struct ChainCounts { uint32_t rounds, a, b, c, d; };

__device__ __forceinline__ void flush_counts(int slot, int lane, bool is_static, const ChainCounts& k, int m) {
#ifdef SAM_COUNTERS
    if (g_sam_counters && lane == 0 && slot < g_sam_counter_slots) {
        unsigned long long* o = g_sam_counters + (size_t)slot * SAM_N_COUNTERS;
        if (is_static) {
            o[SAM_CNT_STATIC_ROUNDS] += k.rounds; o[SAM_CNT_STATIC_LINK_MOVES] += k.a; o[SAM_CNT_STATIC_NEXT_MOVES] += k.b;
        } else {
            o[SAM_CNT_DYNAMIC_ROUNDS] += k.rounds; o[SAM_CNT_WALK_INSERTS] += k.a; o[SAM_CNT_CLONES] += k.b;
            o[SAM_CNT_COPIED_EDGES] += k.c; o[SAM_CNT_REDIRECTS] += k.d;
            o[SAM_CNT_TOKENS] += (unsigned)m; o[SAM_CNT_SEQ_STEPS] += m > 0 ? 1u : 0u;
        }
    }
#endif
}
constexpr int MAX_DRAFT_REGS = 4;     // 4 x 32 lanes = 128 draft tokens

struct StepArgs {
    SamStaticView S;
    SamBatchView W;
    int32_t has_static;
    const int32_t* new_tokens; int32_t stride; const int32_t* counts; int32_t L;
    int32_t* draft_tokens; int32_t* draft_len; int32_t* match_len; int32_t* source;
    int32_t* state; int32_t* status;
    // optional completion signal for the host-array step: the last block to finish writes done_seq to
    // *done_flag (host-mapped memory) so the host can poll instead of synchronising the stream
    int32_t* done_count; int32_t* done_flag; int32_t done_seq;
    // optional fused greedy verification (Section 2.2): when v_draft is set, new_tokens holds the target
    // model's tokens [B, stride] with stride = previous draft length limit + 1, and each slot's count is
    // derived here: the confirmed prefix of its previous draft plus the target's next token
    const int32_t* v_draft; const int32_t* v_draft_len; const int32_t* v_max_new;
    int32_t* v_counts_out; int32_t* v_accepted_out;
    // optional: block i works on slot order[i] (slots with many tokens first; see order_slots_kernel)
    const int32_t* order;
    // split step (sam_step_split_kernel): blocks [0, n_warp_blocks) run the static side of one slot each (the
    // first *split_count slots of `order`, those with many tokens), the next n_lane_blocks blocks the static
    // side of 32 slots each, the remaining blocks the dynamic side of one slot each
    int32_t n_warp_blocks, n_lane_blocks;
    const int32_t* split_count;
};

// ------------------------------------------------------------------ draft read
// d[r] (lane j of round r) = text[e + 32 r + j] for 32 r + j < dl, else -1.  The window is read as
// aligned 16-byte vectors (nine lanes per 32 tokens) and realigned with shuffles.
// READ: 0 plain loads, 1 read-only path (text that no kernel writes), 2 loads that bypass the L1 (text
// written by another block of the grid that is running).
template <int READ>
__device__ __forceinline__ void gather_draft(const int32_t* text, int64_t e, int dl, int L, int lane,
                                             int32_t d[MAX_DRAFT_REGS]) {
    const int off = (int)(e & 3);
    const int4* v = reinterpret_cast<const int4*>(text + (e - off));
    const int nvec = (off + dl + 3) >> 2;
    const int src = (off + lane) >> 2, comp = (off + lane) & 3;
#pragma unroll
    for (int r = 0; r < MAX_DRAFT_REGS; r++) {
        d[r] = -1;
        if (r * 32 < L) {
            int4 q = make_int4(0, 0, 0, 0);
            const int vi = 8 * r + lane;
            if (lane < 9 && vi < nvec) q = READ == 1 ? __ldg(v + vi) : READ == 2 ? __ldcg(v + vi) : v[vi];
            int x0 = __shfl_sync(FULL, q.x, src), x1 = __shfl_sync(FULL, q.y, src);
            int x2 = __shfl_sync(FULL, q.z, src), x3 = __shfl_sync(FULL, q.w, src);
            int val = comp == 0 ? x0 : comp == 1 ? x1 : comp == 2 ? x2 : x3;
            if (r * 32 + lane < dl) d[r] = val;
        }
    }
}

// A draft ends before the first stop token (the separator between documents of a concatenated
// corpus): returns the shortened length and blanks the lanes from there on.
__device__ __forceinline__ int cut_at_stop(int32_t d[MAX_DRAFT_REGS], int dl, int lane, int32_t stop) {
    if (stop < 0) return dl;
#pragma unroll
    for (int r = 0; r < MAX_DRAFT_REGS; r++) {
        const unsigned hit = __ballot_sync(FULL, r * 32 + lane < dl && d[r] == stop);
        if (hit) { dl = r * 32 + __ffs(hit) - 1; break; }
    }
#pragma unroll
    for (int r = 0; r < MAX_DRAFT_REGS; r++) if (r * 32 + lane >= dl) d[r] = -1;
    return dl;
}

// ------------------------------------------------------------------ static side
// Transfer (Algorithm 1) for one token.  (s, sf, l): state, its F bit, match length.
// root_e is root_row[t], fetched beforehand.  If have_rec, (pa, pb) is the record of s, read earlier;
// if have_ent, pent is this lane's entry of the home bucket of (s, t), read earlier.
__device__ __forceinline__ void static_transfer(const SamStaticView& S, uint32_t& s, uint32_t& sf, int32_t& l,
                                                uint32_t t, uint32_t root_e, int lane, int& err,
                                                bool have_rec, uint4 pa, uint4 pb, bool have_ent, uint4 pent, ChainCounts& kc) {
    int guard = l + 2;                       // at most l link moves
    bool len_from_rec = false;
    for (;;) {
        if (s == 0) {                        // at the root the match length is 0
            if (root_e != SAM_NONE) { s = root_e & SAM_IDMASK; sf = root_e >> 31; l = 1; SAM_COUNT(kc.b, 1); }
            else l = 0;
            return;
        }
        uint32_t home = sam_hash2(s, t) & S.hash_mask;
        uint4 ent = make_uint4(SAM_NONE, 0, 0, 0);
        if (sf) ent = have_ent ? pent : __ldg(S.hash + (size_t)home * SAM_HASH_BUCKET + (lane & 7));
        have_ent = false;
        uint4 a = pa, b = pb;
        if (!have_rec) { a = __ldg(S.rec + 2 * (size_t)s); b = __ldg(S.rec + 2 * (size_t)s + 1); SAM_COUNT(kc.rounds, 1); }
        have_rec = false;
        if (len_from_rec) { l = (int32_t)a.x; len_from_rec = false; }
        uint32_t tgt = SAM_NONE;
        if (a.w >= 1 && b.x == t) tgt = b.y;
        else if (a.w >= 2 && b.z == t) tgt = b.w;
        else if (a.w > 2) {
            if (!sf) { ent = __ldg(S.hash + (size_t)home * SAM_HASH_BUCKET + (lane & 7)); SAM_COUNT(kc.rounds, 1); }
            for (int probe = 1;; probe++) {
                unsigned hit = __ballot_sync(FULL, ent.x == s && ent.y == t);
                if (hit) { tgt = __shfl_sync(FULL, ent.z, __ffs(hit) - 1); break; }
                unsigned empty = __ballot_sync(FULL, ent.x == SAM_NONE);
                if (empty || probe >= S.hash_max_probe) break;
                home = (home + 1) & S.hash_mask;
                ent = __ldg(S.hash + (size_t)home * SAM_HASH_BUCKET + (lane & 7));
                SAM_COUNT(kc.rounds, 1);
            }
        }
        if (tgt != SAM_NONE) { s = tgt & SAM_IDMASK; sf = tgt >> 31; l += 1; SAM_COUNT(kc.b, 1); return; }
        SAM_COUNT(kc.a, 1);
        s = a.y & SAM_IDMASK; sf = a.y >> 31;            // s <- link(s), l <- len(link(s))
        if (s == 0) l = 0; else len_from_rec = true;
        if (--guard < 0) { err = SAM_SEQ_WALK_LIMIT; return; }
    }
}

// ------------------------------------------------------------------ dynamic side
struct Dyn {
    unsigned char* pool;
    uint2* root;                 // this slot's root table
    int32_t* text;               // this slot's token text
    uint32_t* pstate;            // this slot's position -> state map (the state each token created)
    int32_t* pool_hdr; int32_t* free_stack; int32_t* slab_owner;
    uint32_t* cb;                // this slot's control block
    uint32_t tab;                // lane i: slab index of state slab i
    uint32_t n_rec_slabs, n_states, blk_cur, blk_end, root_deg, root_bmask;
    int slab_shift, rps_shift, seq, lane, err;
    // Root-table lookups settled ahead of time, one lane per token of the current chunk of 32
    // (root_precompute): pr_state 0 = not known (or stale), 1 = present, 2 = absent.
    uint32_t pr_state, pr_tgt, pr_slot, pr_bucket;
    int cur;                     // lane that holds the answer for the token being processed
    mutable ChainCounts kc;      // rounds, walk-inserts, clones, copied transitions, redirects
};

struct Pre {                     // records read ahead for the clone branch of Expand, kept in shared memory
    bool valid;
    uint32_t q;                  // rec[0..1] is the record of q, rec[2..3] that of link[s2] (if it is not the root)
    const uint4* rec;
};

struct Look {                    // result of looking a token up in a non-root state
    uint32_t len, link, deg, b0, b1, b2, b3;
    uint32_t tgt;                // transition target with its S bit, valid if found
    uint32_t idx;                // 0 / 1 inline slot, or index in the edge block
    bool found;
};

__device__ __forceinline__ uint4* rec_ptr(const Dyn& D, uint32_t s) {
    uint32_t slab = __shfl_sync(FULL, D.tab, (int)(s >> D.rps_shift));
    return reinterpret_cast<uint4*>(D.pool + ((size_t)slab << D.slab_shift) +
                                    ((size_t)(s & ((1u << D.rps_shift) - 1)) << 5));
}
__device__ __forceinline__ uint2* blk_ptr(const Dyn& D, uint32_t off) {
    return reinterpret_cast<uint2*>(D.pool + (size_t)off * 128);
}

__device__ __forceinline__ int alloc_slab(Dyn& D) {
    int idx = -1;
    if (D.lane == 0) {
        int old = atomicSub(D.pool_hdr, 1);
        if (old <= 0) atomicAdd(D.pool_hdr, 1);
        else { idx = D.free_stack[old - 1]; D.slab_owner[idx] = D.seq; }
    }
    return __shfl_sync(FULL, idx, 0);
}

// make sure state id s has a record to live in
__device__ __forceinline__ void ensure_rec(Dyn& D, uint32_t s) {
    uint32_t si = s >> D.rps_shift;
    if (si < D.n_rec_slabs) return;
    if (si >= SAM_MAX_REC_SLABS) { D.err = SAM_SEQ_CAPACITY; return; }
    int slab = alloc_slab(D);
    if (slab < 0) { D.err = SAM_SEQ_CAPACITY; return; }
    if (D.lane == (int)si) D.tab = (uint32_t)slab;
    if (D.lane == 0) D.cb[CB_SLABTAB + si] = (uint32_t)slab;
    D.n_rec_slabs = si + 1;
}

// edge block of `cap` entries; returns its offset in 128-byte units from the pool base
__device__ __forceinline__ uint32_t alloc_block(Dyn& D, uint32_t cap) {
    uint32_t need = cap >> 4, slab_units = 1u << (D.slab_shift - 7);
    if (need > slab_units) { D.err = SAM_SEQ_CAPACITY; return 0; }
    if (D.blk_cur + need > D.blk_end) {
        int slab = alloc_slab(D);
        if (slab < 0) { D.err = SAM_SEQ_CAPACITY; return 0; }
        D.blk_cur = (uint32_t)slab << (D.slab_shift - 7);
        D.blk_end = D.blk_cur + slab_units;
    }
    uint32_t off = D.blk_cur;
    D.blk_cur += need;
    return off;
}

__device__ __forceinline__ Look lookup_state(const Dyn& D, uint32_t p, uint32_t t,
                                             bool have_rec = false, uint4 pa = make_uint4(0, 0, 0, 0),
                                             uint4 pb = make_uint4(0, 0, 0, 0)) {
    uint4 a = pa, b = pb;
    if (!have_rec) { const uint4* rp = rec_ptr(D, p); a = rp[0]; b = rp[1]; SAM_COUNT(D.kc.rounds, 1); }
    Look r;
    r.len = a.x; r.link = a.y; r.deg = a.w; r.b0 = b.x; r.b1 = b.y; r.b2 = b.z; r.b3 = b.w;
    r.found = false; r.tgt = 0; r.idx = 0;
    if (a.w <= 2) {
        if (a.w >= 1 && b.x == t) { r.found = true; r.tgt = b.y; r.idx = 0; }
        else if (a.w == 2 && b.z == t) { r.found = true; r.tgt = b.w; r.idx = 1; }
        return r;
    }
    // 128 entries per round trip: the four reads of a lane are independent and go out together
    const uint2* blk = blk_ptr(D, b.x);
    for (uint32_t base = 0; base < a.w; base += 128) {
        SAM_COUNT(D.kc.rounds, 1);
        uint2 e[4];
#pragma unroll
        for (int u = 0; u < 4; u++) {
            const uint32_t i = base + 32 * u + D.lane;
            e[u] = make_uint2(SAM_NONE, 0);
            if (i < a.w) e[u] = blk[i];
        }
#pragma unroll
        for (int u = 0; u < 4; u++) {
            const unsigned hit = __ballot_sync(FULL, e[u].x == t);
            if (hit && !r.found) {
                const int src = __ffs(hit) - 1;
                r.found = true; r.tgt = __shfl_sync(FULL, e[u].y, src); r.idx = base + 32 * u + src;
            }
        }
        if (r.found) break;
    }
    return r;
}

// add the transition (p, t) -> tgt to a non-root state whose record is in lk
__device__ __forceinline__ void insert_edge(Dyn& D, uint32_t p, const Look& lk, uint32_t t, uint32_t tgt) {
    uint4* rp = rec_ptr(D, p);
    uint32_t* rw = reinterpret_cast<uint32_t*>(rp);
    if (lk.deg < 2) {
        if (D.lane == 0) {
            reinterpret_cast<uint2*>(rp)[2 + lk.deg] = make_uint2(t, tgt);
            rw[3] = lk.deg + 1;
        }
    } else if (lk.deg == 2) {
        uint32_t off = alloc_block(D, SAM_BLOCK_MIN);
        if (D.err) return;
        if (D.lane == 0) {
            uint2* blk = blk_ptr(D, off);
            blk[0] = make_uint2(lk.b0, lk.b1); blk[1] = make_uint2(lk.b2, lk.b3); blk[2] = make_uint2(t, tgt);
            rp[1] = make_uint4(off, SAM_BLOCK_MIN, 0, 0);
            rw[3] = 3;
        }
    } else {
        uint32_t off = lk.b0, cap = lk.b1;
        if (lk.deg < cap) {
            if (D.lane == 0) { blk_ptr(D, off)[lk.deg] = make_uint2(t, tgt); rw[3] = lk.deg + 1; }
        } else {
            uint32_t noff = alloc_block(D, cap * 2);
            if (D.err) return;
            const uint2* ob = blk_ptr(D, off);
            uint2* nb = blk_ptr(D, noff);
            for (uint32_t i = D.lane; i < lk.deg; i += 32) nb[i] = ob[i];
            if (D.lane == 0) {
                nb[lk.deg] = make_uint2(t, tgt);
                rp[1] = make_uint4(noff, cap * 2, 0, 0);
                rw[3] = lk.deg + 1;
            }
        }
    }
    __syncwarp();
}

struct RootLook { uint32_t tgt, slot; bool found; };

// Each lane looks its own token up in the root table by itself: the home bucket (64 bytes, four
// 16-byte reads) settles it when the token is there, or when the bucket still has an empty entry
// (linear probing never skips one).  All tokens of the chunk are looked up in one round trip,
// before any of them is processed; later changes to the table mark the affected answers stale.
__device__ __forceinline__ void root_precompute(Dyn& D, uint32_t tk, bool valid) {
    D.pr_state = 0; D.pr_tgt = 0; D.pr_slot = 0; D.pr_bucket = SAM_NONE;
    if (!valid) return;
    const uint32_t home = sam_hash1(tk) & D.root_bmask;
    const uint4* bk = reinterpret_cast<const uint4*>(D.root + (size_t)home * SAM_ROOT_BUCKET);
    uint4 v[4];
#pragma unroll
    for (int i = 0; i < 4; i++) v[i] = bk[i];
    D.pr_bucket = home;
    int first_empty = -1;
#pragma unroll
    for (int i = 3; i >= 0; i--) {                       // descending, so the lowest index wins
        if (v[i].z == SAM_NONE) first_empty = 2 * i + 1;
        if (v[i].x == SAM_NONE) first_empty = 2 * i;
    }
#pragma unroll
    for (int i = 0; i < 4; i++) {
        if (v[i].x == tk) { D.pr_state = 1; D.pr_tgt = v[i].y; D.pr_slot = home * SAM_ROOT_BUCKET + 2 * i; }
        if (v[i].z == tk) { D.pr_state = 1; D.pr_tgt = v[i].w; D.pr_slot = home * SAM_ROOT_BUCKET + 2 * i + 1; }
    }
    if (D.pr_state == 0 && first_empty >= 0) { D.pr_state = 2; D.pr_slot = home * SAM_ROOT_BUCKET + first_empty; }
}

__device__ __forceinline__ RootLook root_lookup(Dyn& D, uint32_t t) {
    RootLook r; r.found = false; r.tgt = 0; r.slot = 0;
    const uint32_t st = __shfl_sync(FULL, D.pr_state, D.cur);
    if (st != 0) {                                       // settled ahead of time and still current
        r.found = st == 1;
        r.tgt = __shfl_sync(FULL, D.pr_tgt, D.cur);
        r.slot = __shfl_sync(FULL, D.pr_slot, D.cur);
        return r;
    }
    const uint32_t cap_mask = (D.root_bmask + 1) * SAM_ROOT_BUCKET - 1;
    const uint32_t base = (sam_hash1(t) & D.root_bmask) * SAM_ROOT_BUCKET;
    for (uint32_t off = 0; off <= cap_mask; off += 32) {
        SAM_COUNT(D.kc.rounds, 1);
        uint2 e = D.root[(base + off + D.lane) & cap_mask];
        unsigned hit = __ballot_sync(FULL, e.x == t);
        if (hit) {
            int src = __ffs(hit) - 1;
            r.found = true; r.tgt = __shfl_sync(FULL, e.y, src); r.slot = (base + off + src) & cap_mask;
            return r;
        }
        unsigned empty = __ballot_sync(FULL, e.x == SAM_NONE);
        if (empty) { r.slot = (base + off + (__ffs(empty) - 1)) & cap_mask; return r; }
    }
    D.err = SAM_SEQ_WALK_LIMIT;           // table full: cannot happen with root_cap >= 2 * distinct tokens
    return r;
}

// new root transition; answers settled ahead of time for the bucket it lands in are no longer current
__device__ __forceinline__ void root_insert(Dyn& D, uint32_t slot, uint32_t t, uint32_t tgt) {
    if (D.lane == 0) D.root[slot] = make_uint2(t, tgt);
    if (D.pr_bucket == slot / SAM_ROOT_BUCKET) D.pr_state = 0;
    __syncwarp();
    D.root_deg++;
}
// change the target of an existing root transition
__device__ __forceinline__ void root_retarget(Dyn& D, uint32_t slot, uint32_t tgt) {
    if (D.lane == 0) D.root[slot].y = tgt;
    if (D.pr_state == 1 && D.pr_slot == slot) D.pr_tgt = tgt;
}

// The redirect loop of Expand's clone branch (Algorithm 3): from state pp up the suffix links, every
// t-transition that leads to q is pointed to the clone cl instead; the walk ends at the first state
// whose t-transition leads elsewhere, or past the root.  If first, (na, nb2) is the record of pp.
__device__ __forceinline__ void redirect_walk(Dyn& D, uint32_t pp, uint32_t t, uint32_t q, uint32_t cl, int guard,
                                              bool first, uint4 na, uint4 nb2) {
    for (;;) {
        if (pp == 0) {
            RootLook r2 = root_lookup(D, t);
            if (D.err) return;
            if (r2.found && (r2.tgt & SAM_IDMASK) == q) { root_retarget(D, r2.slot, cl); SAM_COUNT(D.kc.d, 1); }
            return;
        }
        Look l2k = lookup_state(D, pp, t, first, na, nb2);
        first = false;
        if (!l2k.found) { D.err = SAM_SEQ_WALK_LIMIT; return; }   // every state up the chain has t
        if ((l2k.tgt & SAM_IDMASK) != q) return;
        uint32_t* rw2 = reinterpret_cast<uint32_t*>(rec_ptr(D, pp));
        if (D.lane == 0) {
            if (l2k.deg <= 2) rw2[5 + 2 * l2k.idx] = cl;
            else blk_ptr(D, l2k.b0)[l2k.idx].y = cl;
        }
        SAM_COUNT(D.kc.d, 1);
        pp = l2k.link;
        if (--guard < 0) { D.err = SAM_SEQ_WALK_LIMIT; return; }
    }
}

// Expand (Algorithm 3) for token t, fused with the dynamic matcher's Transfer.
// last: state of the whole text; ntok: text length; (s2, l2): match state = link[last], its length.
// On entry, if have_rec, (pa, pb) is the record of s2 as it stands; on exit have_rec says whether
// (pa, pb) is the record of the new s2 (known without a read when s2 is a fresh clone).
__device__ __forceinline__ void dyn_extend(Dyn& D, uint32_t t, uint32_t& last, uint32_t& ntok,
                                           uint32_t& s2, uint32_t& l2, bool& have_rec, uint4& pa, uint4& pb,
                                           const Pre& pre) {
    bool use_rec = have_rec;
    have_rec = false;
    const uint32_t k = ntok + 1;                       // max_length after this token
    const uint32_t c = D.n_states;
    ensure_rec(D, c);
    if (D.err) return;
    D.n_states = c + 1;

    uint32_t p;
    if (last != 0) {
        // `last` has no transition yet; it gets (t -> c), solid, and its record is complete now
        uint4* rl = rec_ptr(D, last);
        if (D.lane == 0) {
            rl[0] = make_uint4(ntok, s2, ntok, 1);
            rl[1] = make_uint4(t, c | SAM_FLAG, 0, 0);
        }
        __syncwarp();
        SAM_COUNT(D.kc.a, 1);
        p = s2;                                        // link[last]
    } else {
        p = 0;                                         // empty automaton: last is the root
    }

    // walk the suffix links from p, adding (t -> c) until a state already has t
    bool found = false, at_root = false;
    uint32_t qt = 0, plen = 0, root_slot = 0;
    Look lk;
    lk.len = lk.link = lk.deg = lk.b0 = lk.b1 = lk.b2 = lk.b3 = lk.tgt = lk.idx = 0; lk.found = false;
    int guard = (int)k + 2;
    for (;;) {
        if (p == 0) {
            RootLook rl = root_lookup(D, t);
            if (D.err) return;
            if (rl.found) { found = true; at_root = true; qt = rl.tgt; plen = 0; root_slot = rl.slot; }
            else {
                root_insert(D, rl.slot, t, c | (k == 1 ? SAM_FLAG : 0u));
                SAM_COUNT(D.kc.a, 1);
            }
            break;
        }
        lk = lookup_state(D, p, t, use_rec, pa, pb);
        use_rec = false;
        if (lk.found) { found = true; qt = lk.tgt; plen = lk.len; break; }
        insert_edge(D, p, lk, t, c);                   // len[p] + 1 < k: not solid
        SAM_COUNT(D.kc.a, 1);
        if (D.err) return;
        p = lk.link;
        if (--guard < 0) { D.err = SAM_SEQ_WALK_LIMIT; return; }
    }

    if (!found) {                                      // walked past the root
        s2 = 0; l2 = 0;
    } else {
        const uint32_t q = qt & SAM_IDMASK;
        if (qt & SAM_FLAG) {                           // len[p] + 1 == len[q]
            s2 = q; l2 = plen + 1;
        } else {
            // clone q as cl with len[p] + 1
            const uint32_t cl = D.n_states;
            ensure_rec(D, cl);
            if (D.err) return;
            D.n_states = cl + 1;
            uint4* rq = rec_ptr(D, q);
            // the redirect walk's first read (the record of link[p]) does not depend on q's record:
            // both go out together.  link[p] is neither p, q nor cl, so nothing below changes it.
            const bool ahead = !at_root && lk.link != 0;
            const uint4* rn = rec_ptr(D, ahead ? lk.link : q);
            uint4 qa, qb, na = make_uint4(0, 0, 0, 0), nb2 = make_uint4(0, 0, 0, 0);
            if (pre.valid && pre.q == q) {              // both were read by a run attempt that did not apply
                qa = pre.rec[0]; qb = pre.rec[1];
                if (ahead) { na = pre.rec[2]; nb2 = pre.rec[3]; }
            } else {
                qa = rq[0]; qb = rq[1];
                if (ahead) { na = rn[0]; nb2 = rn[1]; }
                SAM_COUNT(D.kc.rounds, 1);
            }
            SAM_COUNT(D.kc.b, 1); SAM_COUNT(D.kc.c, qa.w); SAM_COUNT(D.kc.d, 1);   // the clone, its copied transitions, p's own redirect
            uint4 nb;
            if (qa.w <= 2) {
                nb = make_uint4(qb.x, qb.y & SAM_IDMASK, qb.z, qb.w & SAM_IDMASK);   // copies are never solid
            } else {
                uint32_t noff = alloc_block(D, qb.y);
                if (D.err) return;
                const uint2* ob = blk_ptr(D, qb.x);
                uint2* nbk = blk_ptr(D, noff);
                for (uint32_t i = D.lane; i < qa.w; i += 32) { uint2 e = ob[i]; e.y &= SAM_IDMASK; nbk[i] = e; }
                nb = make_uint4(noff, qb.y, 0, 0);
            }
            uint4* rc = rec_ptr(D, cl);
            if (D.lane == 0) {
                rc[0] = make_uint4(plen + 1, qa.y, qa.z, qa.w);      // link[q], min_endpos[q], deg[q]
                rc[1] = nb;
            }
            __syncwarp();
            // redirect p and the states above it whose t-transition is q
            if (at_root) {
                root_retarget(D, root_slot, cl | SAM_FLAG);
            } else {
                uint32_t* rw = reinterpret_cast<uint32_t*>(rec_ptr(D, p));
                if (D.lane == 0) {
                    if (lk.deg <= 2) rw[5 + 2 * lk.idx] = cl | SAM_FLAG;
                    else blk_ptr(D, lk.b0)[lk.idx].y = cl | SAM_FLAG;
                }
                redirect_walk(D, lk.link, t, q, cl, (int)plen + 2, ahead, na, nb2);
                if (D.err) return;
            }
            if (D.lane == 0) reinterpret_cast<uint32_t*>(rq)[1] = cl;        // link[q] = cl
            __syncwarp();
            s2 = cl; l2 = plen + 1;
            have_rec = true;                                                 // cl's record as just written
            pa = make_uint4(plen + 1, qa.y, qa.z, qa.w); pb = nb;
        }
    }
    if (D.lane == 0) { D.text[ntok] = (int32_t)t; D.pstate[ntok] = c; }
    last = c; ntok = k;
}

// A run of tokens that are all new to the sequence, met while nothing is matched (s2 is the root):
// Expand for each of them is the same three writes — the previous state's record with its one
// solid transition, a root transition, the text — and none depends on another, so lanes j..j+r-1
// do one token each at once.  A token qualifies if its root lookup was settled ahead of time as
// "absent" and no earlier token of the run shares its home bucket (so slots and tokens differ).
// Returns r (0 if token j does not qualify).
__device__ __forceinline__ int dyn_fresh_run(Dyn& D, uint32_t tk, int j, int cnt, unsigned bucket_peers,
                                             uint32_t& last, uint32_t& ntok) {
    const unsigned from_j = ~((1u << j) - 1u);
    const unsigned lt = (1u << D.lane) - 1u;
    const bool first_of_bucket = (bucket_peers & from_j & lt) == 0;
    const unsigned elig = __ballot_sync(FULL, D.pr_state == 2 && first_of_bucket && D.lane >= j && D.lane < cnt);
    const unsigned gap = ~(elig >> j);
    int r = gap ? __ffs(gap) - 1 : 32 - j;
    if (r <= 0) return 0;
    const uint32_t c0 = D.n_states;
    ensure_rec(D, c0);
    if (!D.err) ensure_rec(D, c0 + r - 1);
    if (D.err) return 0;
    const int idx = D.lane - j;
    const bool mine = idx >= 0 && idx < r;
    const uint32_t c = c0 + (uint32_t)idx;
    const uint32_t prev = idx == 0 ? last : c - 1;            // the state this token's transition leaves
    const uint32_t plen = ntok + (uint32_t)idx;               // its length = tokens before this one
    uint4* rp = rec_ptr(D, mine ? prev : 1u);
    if (mine) {
        if (prev != 0) {
            rp[0] = make_uint4(plen, 0, plen, 1);             // link is the root: nothing was matched
            rp[1] = make_uint4(tk, c | SAM_FLAG, 0, 0);
        }
        D.root[D.pr_slot] = make_uint2(tk, c | (plen == 0 ? SAM_FLAG : 0u));
        D.text[plen] = (int32_t)tk;
        D.pstate[plen] = c;
    }
    const unsigned run = ((r >= 32 ? 0u : (1u << r)) - 1u) << j;
    if (bucket_peers & run) D.pr_state = 0;                   // those buckets changed
    __syncwarp();
    SAM_COUNT(D.kc.a, 2 * r - (last == 0 ? 1 : 0));            // per token: the previous state's transition (none from the root) and the root's
    D.n_states = c0 + r; D.root_deg += r;
    last = c0 + r - 1; ntok += r;
    return r;
}

// A run of tokens that repeat a passage of the sequence and all make Expand clone (Algorithm 3).
// While the match (state s2, length l0, first end position e) is extended by the tokens that followed
// its earliest occurrence, token k of the run reaches q_k, a state with first end position e + 1 + k,
// through a transition that is not solid: a new state c_k, a clone cl_k of q_k with length l0 + k + 1,
// the transition of the previous clone pointed to cl_k, link[q_k] = cl_k.  One Expand after the other
// finds q_k only from q_{k-1}'s record.  Here the q_k are guessed — the states of the prefixes ending at
// e + 1 + k (position -> state map) when the passage occurred once before, ids two apart when q_0 is a
// clone left by an earlier repeat — their records are read in one round trip, one lane per token, and
// checked (q_{k-1}'s transition on token k must lead to the guessed q_k); the lanes then write their
// new states side by side.  Only the redirect walks above each clone (they start at the old link of
// q_{k-1}) run one after the other.  Writing every link[q_k] before the walks gives what one Expand
// after the other gives: a walk of token k follows states shorter than l0 + k, every q_k' with k' > k
// is longer, and what a walk reads ahead (its first record) is checked not to be a q_k.
// On entry (pa, pb) is the record of s2.  Returns the number of tokens taken (0: not such a run; pre
// then offers the records read on the way to the ordinary Expand of token j).
__device__ __forceinline__ int dyn_repeat_run(Dyn& D, uint32_t tk, int j, int cnt, uint32_t& last, uint32_t& ntok,
                                              uint32_t& s2, uint32_t& l2, uint4& pa, uint4& pb, Pre& pre,
                                              uint32_t (*stage)[12]) {
    pre.valid = false;
    if (pa.w == 0 || pa.w > 2 || cnt - j < 2) return 0;
    const int lane = D.lane;
    const uint32_t t0 = __shfl_sync(FULL, tk, j);
    int idx0; uint32_t qt;
    if (pb.x == t0) { idx0 = 0; qt = pb.y; }
    else if (pa.w == 2 && pb.z == t0) { idx0 = 1; qt = pb.w; }
    else return 0;
    if (qt & SAM_FLAG) return 0;                               // solid: Expand does not clone
    const uint32_t q0 = qt, e = pa.z, l0 = l2, u0 = pa.y;
    const int rmax = min(cnt - j, (int)(ntok - e));            // text[e + k] must exist already
    if (rmax < 2) return 0;
    __syncwarp();

    // first round trip: the text after the earlier occurrence and the states created there; the records of q_0
    // and of link[s2] (what the ordinary Expand of token j would read, should this not be a run)
    const uint32_t tkr = __shfl_sync(FULL, tk, (j + lane) & 31);          // lane k: token k of the run
    const uint32_t tnext = __shfl_sync(FULL, tk, (j + lane + 1) & 31);
    int32_t tx = -1; uint32_t ps = SAM_NONE;
    if (lane < rmax) { tx = D.text[e + lane]; ps = D.pstate[e + lane]; }
    const uint4* rq0 = rec_ptr(D, q0);
    const uint4* ru0 = rec_ptr(D, u0 ? u0 : q0);
    uint4 qa = rq0[0], qb = rq0[1], ua = make_uint4(0, 0, 0, 0), ub = ua;
    if (u0) { ua = ru0[0]; ub = ru0[1]; }
    SAM_COUNT(D.kc.rounds, 1);
    const unsigned same = __ballot_sync(FULL, lane < rmax && (uint32_t)tx == tkr);
    // q_0 may be `last` itself (if token j does not continue the earliest occurrence), whose record is
    // only completed by the Expand of token j: what was read of it is then not used
    if (q0 != last) {
        uint4* keep = reinterpret_cast<uint4*>(&stage[0][0]);
        if (lane == 0) { keep[0] = qa; keep[1] = qb; keep[2] = ua; keep[3] = ub; }
        __syncwarp();
        pre.valid = true; pre.q = q0; pre.rec = keep;
    }
    int r = (~same) ? __ffs(~same) - 1 : 32;
    if (r < 2) return 0;
    // Where the q_k are expected: the states of the prefixes ending there if the passage occurred once
    // before (q_0 is then the prefix state); otherwise q_0 is a clone from an earlier repeat of the
    // passage, and clones made token after token have ids two apart.  Either guess is checked below.
    if (__shfl_sync(FULL, ps, 0) != q0) ps = q0 + 2 * (uint32_t)lane;

    // second round trip: the records of q_1 .. q_{r-1} (states that exist and are complete: not `last`)
    const bool exists = ps < D.n_states && ps != last;
    {
        const bool rd = lane > 0 && lane < r && exists;
        const uint4* rqk = rec_ptr(D, rd ? ps : q0);
        if (rd) { qa = rqk[0]; qb = rqk[1]; }
    }
    // q_k: inline transitions only, first end position e + 1 + k, reached by a transition that is not
    // solid; and, but for the last of the run, its transition on the next token leads to q_{k+1}
    int nidx = -1;
    if (qa.w >= 1 && qa.w <= 2 && qb.x == tnext) nidx = 0;
    else if (qa.w == 2 && qb.z == tnext) nidx = 1;
    const uint32_t ntgt = (nidx == 0 ? qb.y : qb.w) & SAM_IDMASK;
    const uint32_t psn = __shfl_down_sync(FULL, ps, 1);
    const unsigned okm = __ballot_sync(FULL, lane < r && exists && qa.w <= 2 && qa.z == e + 1 + (uint32_t)lane &&
                                                 qa.x > l0 + 1 + (uint32_t)lane);
    const unsigned nxm = __ballot_sync(FULL, nidx >= 0 && ntgt == psn);
    r = min(r, (~okm) ? __ffs(~okm) - 1 : 32);
    r = min(r, ((~nxm) ? __ffs(~nxm) - 1 : 32) + 1);
    if (r < 2) return 0;

    // third round trip: where each redirect walk starts, the old link of q_{k-1} (of s2 for k = 0)
    uint32_t u = __shfl_up_sync(FULL, qa.y, 1);
    if (lane == 0) u = u0;
    {
        const bool rd = lane > 0 && lane < r && u != 0;
        const uint4* ruk = rec_ptr(D, rd ? u : q0);
        if (rd) { ua = ruk[0]; ub = ruk[1]; }
    }
    {   // a walk's first record has been read now, before link[q_k] changes: it must not be one of the
        // q_k (the q_k are told apart by their first end positions e + 1 + k)
        const int kk = (int)ua.z - (int)e - 1;
        const uint32_t cand = __shfl_sync(FULL, ps, kk & 31);
        const unsigned inq = __ballot_sync(FULL, lane < r && u != 0 && kk >= 0 && kk < r && cand == u);
        if (inq) r = min(r, __ffs(inq) - 1);
        if (r < 2) return 0;
    }

    *reinterpret_cast<uint4*>(&stage[lane][0]) = ua;
    *reinterpret_cast<uint4*>(&stage[lane][4]) = ub;
    *reinterpret_cast<uint4*>(&stage[lane][8]) = make_uint4(tkr, ps, u, 0);

    const uint32_t n0 = D.n_states;                            // c_k = n0 + 2k, cl_k = n0 + 2k + 1
    ensure_rec(D, n0);
    if (!D.err) ensure_rec(D, n0 + 2 * (uint32_t)r - 1);
    if (D.err) return 0;

    // the new states, side by side
    const bool mine = lane < r;
    const uint32_t ck = n0 + 2 * (uint32_t)lane, clk = ck + 1;
    uint4* rprev = rec_ptr(D, mine ? (lane == 0 ? last : ck - 2) : 1u);      // the state whose transition t_k leaves
    uint4* rcl = rec_ptr(D, mine ? clk : 1u);
    uint32_t* rqw = reinterpret_cast<uint32_t*>(rec_ptr(D, mine ? ps : 1u));
    uint32_t* rs2 = reinterpret_cast<uint32_t*>(rec_ptr(D, s2));
    uint4 nb = make_uint4(qb.x, qb.y & SAM_IDMASK, qb.z, qb.w & SAM_IDMASK);  // copies are never solid ...
    if (lane < r - 1) {                                                       // ... until redirected to the next clone
        if (nidx == 0) nb.y = (clk + 2) | SAM_FLAG; else nb.w = (clk + 2) | SAM_FLAG;
    }
    if (mine) {
        rprev[0] = make_uint4(ntok + lane, lane == 0 ? s2 : clk - 2, ntok + lane, 1);
        rprev[1] = make_uint4(tkr, ck | SAM_FLAG, 0, 0);
        rcl[0] = make_uint4(l0 + 1 + lane, qa.y, qa.z, qa.w);
        rcl[1] = nb;
        rqw[1] = clk;                                                         // link[q_k] = cl_k
        D.text[ntok + lane] = (int32_t)tkr;
        D.pstate[ntok + lane] = ck;
        if (lane == 0) rs2[5 + 2 * idx0] = clk | SAM_FLAG;                    // s2's transition on t_0
    }
    __syncwarp();

    // the redirect walks, one after the other; what each needs was left in shared memory by its lane
    for (int k = 0; k < r && !D.err; k++) {
        D.cur = j + k;
        const uint4 xa = *reinterpret_cast<const uint4*>(&stage[k][0]);
        const uint4 xb = *reinterpret_cast<const uint4*>(&stage[k][4]);
        const uint4 xc = *reinterpret_cast<const uint4*>(&stage[k][8]);       // token, q_k, start of the walk
        redirect_walk(D, xc.z, xc.x, xc.y, n0 + 2 * (uint32_t)k + 1, (int)(l0 + k) + 2, xc.z != 0, xa, xb);
    }
    if (D.err) return 0;
    SAM_COUNT(D.kc.rounds, 2);
    SAM_COUNT(D.kc.a, r); SAM_COUNT(D.kc.b, r); SAM_COUNT(D.kc.d, r);
    {
        uint32_t copied = mine ? qa.w : 0u;
        for (int o = 16; o; o >>= 1) copied += __shfl_xor_sync(FULL, copied, o);
        SAM_COUNT(D.kc.c, copied);
    }

    const int lr = r - 1;                                      // the last clone is the new match state
    pa = make_uint4(l0 + (uint32_t)r, __shfl_sync(FULL, qa.y, lr), __shfl_sync(FULL, qa.z, lr), __shfl_sync(FULL, qa.w, lr));
    pb = make_uint4(__shfl_sync(FULL, nb.x, lr), __shfl_sync(FULL, nb.y, lr), __shfl_sync(FULL, nb.z, lr), __shfl_sync(FULL, nb.w, lr));
    D.n_states = n0 + 2 * (uint32_t)r;
    last = n0 + 2 * (uint32_t)lr; s2 = last + 1; l2 = l0 + (uint32_t)r; ntok += (uint32_t)r;
    pre.valid = false;
    return r;
}

// The static side of one slot's step, run by one warp: Transfer (Algorithm 1) for each of the slot's m
// tokens, then the static words of the control block.  cw holds control words 0..31 as read at the start
// of the step; on entry (ra, rb) is the copy of the match state's record kept in the control block, ntok0
// the text length before the step.  On exit (s, sf, l) is the match state, and, if l > 0 and no error,
// (ra, rb) its record.  DRAFT: also fetch the draft after the state's first end position into d / my_dl
// (requested early where the address is known early).
template <bool DRAFT>
__device__ __forceinline__ void static_chain(const StepArgs& A, int b, int lane, uint32_t* cb, uint32_t cw, int32_t tok_first,
                                             const int32_t* toks, int m, uint32_t ntok0, uint4& ra, uint4& rb,
                                             uint32_t& s_out, uint32_t& sf_out, int32_t& l_out, int& err,
                                             int32_t d[MAX_DRAFT_REGS], int32_t& my_dl) {
    const int L = A.L;
    ChainCounts kc = {1, 0, 0, 0, 0};                    // one round already: the control words
    uint32_t s = __shfl_sync(FULL, cw, CB_S1), sf = __shfl_sync(FULL, cw, CB_S1FLAG);
    int32_t l = (int32_t)__shfl_sync(FULL, cw, CB_L1);
    bool have = s != 0;
    // The match state is the state Build-SAM created for a whole corpus prefix (len == min_endpos:
    // not a clone), the prefix ending at e.  Its transition on the next corpus token was created
    // solid (len + 1) and a solid transition is never redirected, so it still leads to the state of
    // the prefix one longer, with match length l + 1.  The state may occur more than once and have
    // other transitions too ("ab" in "ababc"): nothing is assumed about those.  The step's tokens
    // are compared with the corpus after e; as long as they agree the state is taken from the
    // position -> state array, and the first token that differs goes through the ordinary Transfer
    // below.  All in one round trip, in which the draft after e + m is requested as well in case
    // every token agrees.
    int j0 = 0;                      // tokens already taken
    bool drafted = false;
    if (have && m >= 1 && m <= 32 && ra.x == ra.z) {
        const int64_t e = (int64_t)ra.z;
        int32_t cx = -2; uint32_t px = 0;
        if (lane < m && e + lane < A.S.n_tokens) { cx = __ldg(A.S.corpus + e + lane); px = __ldg(A.S.pstate + e + lane); }
        const int64_t e2 = e + m;
        const int64_t room = A.S.n_tokens - e2;
        const int dl2 = (int)(room < L ? (room < 0 ? 0 : room) : L);
        if (DRAFT) gather_draft<1>(A.S.corpus, e2, dl2, L, lane, d);
        const unsigned agree = __ballot_sync(FULL, lane < m && cx == tok_first);
        j0 = (~agree) ? __ffs(~agree) - 1 : 32;
        SAM_COUNT(kc.rounds, 1); SAM_COUNT(kc.b, j0);
        if (j0 > 0) {
            const uint32_t ref = __shfl_sync(FULL, px, j0 - 1);
            s = ref & SAM_IDMASK; sf = ref >> 31; l += j0; have = false;
            if (j0 == m) {                                  // the whole step: the draft is in already
                ra = __ldg(A.S.rec + 2 * (size_t)s);        // its record, for the next step
                rb = __ldg(A.S.rec + 2 * (size_t)s + 1);
                if (DRAFT) my_dl = cut_at_stop(d, dl2, lane, A.W.stop_token);
                drafted = true;
            }
        }
    }
    for (int base = 0; base < m && !err && j0 < m; base += 32) {
        const int i = base + lane;
        uint32_t tk = 0, re = SAM_NONE;
        if (i < m) { tk = (uint32_t)(base == 0 ? tok_first : toks[i]); re = __ldg(A.S.root_row + tk); }
        const int cnt = min(32, m - base);
        SAM_COUNT(kc.rounds, 1);
        // Most tokens end a short match: the lookup misses, the link leads to the root, and the
        // root row gives the next state u = root_row[t].  The token after that is then looked up
        // in u — a lookup whose address is known now.  Lookups k = 0..7 (state root_row[t_k],
        // token t_{k+1}) are read ahead here, eight lanes each: the state's record in lanes 0-1
        // of the group, its hash bucket in all eight.  They are used if the matcher really is
        // in that state when the token comes.
        uint4 sp_rec[2], sp_ent[2];
#pragma unroll
        for (int r = 0; r < 2; r++) {
            const int k = 4 * r + (lane >> 3), e = lane & 7;
            const uint32_t uref = __shfl_sync(FULL, re, k);
            const uint32_t tnext = __shfl_sync(FULL, tk, k + 1);
            sp_rec[r] = make_uint4(0, 0, 0, 0);
            sp_ent[r] = make_uint4(SAM_NONE, 0, 0, 0);
            if (k + 1 < cnt && uref != SAM_NONE) {
                const uint32_t u = uref & SAM_IDMASK;
                if (e < 2) sp_rec[r] = __ldg(A.S.rec + 2 * (size_t)u + e);
                if (uref >> 31)
                    sp_ent[r] = __ldg(A.S.hash + (size_t)(sam_hash2(u, tnext) & A.S.hash_mask) * SAM_HASH_BUCKET + e);
            }
        }
        for (int j = j0; j < cnt && !err; j++) {
            bool pre = false;
            uint4 pa = ra, pb = rb, pent = make_uint4(SAM_NONE, 0, 0, 0);
            if (j >= 1 && j <= 8 && s != 0) {
                const uint32_t prev = __shfl_sync(FULL, re, j - 1);
                if (prev != SAM_NONE && (prev & SAM_IDMASK) == s) {        // the state read ahead
                    const int k = j - 1, g8 = 8 * (k & 3);
                    const uint4 xr = (k >> 2) ? sp_rec[1] : sp_rec[0];
                    const uint4 xe = (k >> 2) ? sp_ent[1] : sp_ent[0];
                    pa.x = __shfl_sync(FULL, xr.x, g8); pa.y = __shfl_sync(FULL, xr.y, g8);
                    pa.z = __shfl_sync(FULL, xr.z, g8); pa.w = __shfl_sync(FULL, xr.w, g8);
                    pb.x = __shfl_sync(FULL, xr.x, g8 + 1); pb.y = __shfl_sync(FULL, xr.y, g8 + 1);
                    pb.z = __shfl_sync(FULL, xr.z, g8 + 1); pb.w = __shfl_sync(FULL, xr.w, g8 + 1);
                    const int src = g8 + (lane & 7);
                    pent.x = __shfl_sync(FULL, xe.x, src); pent.y = __shfl_sync(FULL, xe.y, src);
                    pent.z = __shfl_sync(FULL, xe.z, src); pent.w = __shfl_sync(FULL, xe.w, src);
                    pre = true;
                }
            }
            static_transfer(A.S, s, sf, l, __shfl_sync(FULL, tk, j), __shfl_sync(FULL, re, j), lane, err,
                            have || pre, pa, pb, pre, pent, kc);
            have = false;
        }
    }
    l_out = l; s_out = s; sf_out = sf;
    if (l > 0 && !err) SAM_COUNT(kc.rounds, (m > 0 ? 1 : 0) + (DRAFT && !drafted ? 1 : 0));
    flush_counts(b, lane, true, kc, m);
    if (l > 0 && !err && !drafted) {
        if (m > 0) {                                    // the state moved: read its record, keep a copy
            ra = __ldg(A.S.rec + 2 * (size_t)s);
            rb = __ldg(A.S.rec + 2 * (size_t)s + 1);
        }
        if (DRAFT) {
            const int64_t e = (int64_t)ra.z;            // min_endpos
            int64_t room = A.S.n_tokens - e;
            my_dl = (int)(room < L ? (room < 0 ? 0 : room) : L);
            gather_draft<1>(A.S.corpus, e, my_dl, L, lane, d);
            my_dl = cut_at_stop(d, my_dl, lane, A.W.stop_token);
        }
    }
    if (m > 0 && lane == 0 && !err) {
        cb[CB_S1] = s; cb[CB_L1] = (uint32_t)l; cb[CB_S1FLAG] = sf; cb[CB_NTOK_S] = ntok0 + (uint32_t)m;
        if (l > 0) { reinterpret_cast<uint4*>(cb + CB_REC1)[0] = ra; reinterpret_cast<uint4*>(cb + CB_REC1)[1] = rb; }
    }
}

// The dynamic side of one slot's step, run by one warp: Expand (fused with the dynamic matcher's Transfer)
// for each of the slot's m tokens, then the slot's control words.  cw / cw2 are the slot's 64 control
// words as read at the start of the step (lane i holds words i and 32 + i); on entry (ra, rb) is the copy
// of the match state's record kept in the control block.  On exit (s2, l2) is the match state, ntok the
// text length, and, if l2 > 0 and no error, (ra, rb) the record of s2 (also stored in the control block).
__device__ __forceinline__ void dynamic_chain(const StepArgs& A, int b, int lane, uint32_t* cb, uint32_t cw, uint32_t cw2,
                                              int32_t tok_first, const int32_t* toks, int m, uint32_t ntok0,
                                              uint4& ra, uint4& rb, uint32_t (*sh_run)[12],
                                              uint32_t& s2_out, uint32_t& l2_out, uint32_t& ntok_out, int& err) {
    Dyn D;
    D.pool = A.W.pool;
    D.root = A.W.root_tab + (size_t)b * A.W.root_cap;
    D.text = A.W.text + (size_t)b * A.W.text_stride;
    D.pstate = A.W.pstate + (size_t)b * A.W.text_stride;
    D.pool_hdr = A.W.pool_hdr; D.free_stack = A.W.free_stack; D.slab_owner = A.W.slab_owner;
    D.cb = cb;
    {   // slab table entry i is control word 16 + i
        uint32_t lo = __shfl_sync(FULL, cw, (lane + 16) & 31), hi = __shfl_sync(FULL, cw2, (lane + 16) & 31);
        D.tab = lane < 16 ? lo : hi;
    }
    D.n_rec_slabs = __shfl_sync(FULL, cw, CB_NRECSLABS);
    D.n_states = __shfl_sync(FULL, cw, CB_NSTATES);
    D.blk_cur = __shfl_sync(FULL, cw, CB_BLK_CUR);
    D.blk_end = __shfl_sync(FULL, cw, CB_BLK_END);
    D.root_deg = __shfl_sync(FULL, cw, CB_ROOTDEG);
    D.root_bmask = (uint32_t)(A.W.root_cap / SAM_ROOT_BUCKET) - 1;
    D.slab_shift = A.W.slab_shift; D.rps_shift = A.W.slab_shift - 5;
    D.seq = b; D.lane = lane; D.err = 0;
    D.pr_state = 0; D.pr_tgt = 0; D.pr_slot = 0; D.pr_bucket = SAM_NONE; D.cur = 0;
    D.kc = ChainCounts{1, 0, 0, 0, 0};                   // one round already: the control words
    uint32_t last = __shfl_sync(FULL, cw, CB_LAST), ntok = ntok0;
    uint32_t s2 = __shfl_sync(FULL, cw, CB_S2), l2 = __shfl_sync(FULL, cw, CB_L2);
    if (D.n_states == 0) D.n_states = 1;            // the root exists implicitly (no record is read for it)

    bool have = s2 != 0;
    for (int base = 0; base < m && !D.err; base += 32) {
        const int i = base + lane;
        uint32_t tk = 0;
        if (i < m) tk = (uint32_t)(base == 0 ? tok_first : toks[i]);
        root_precompute(D, tk, i < m);              // most walks end in the root table
        SAM_COUNT(D.kc.rounds, 1);
        const unsigned bucket_peers = __match_any_sync(FULL, D.pr_bucket);
        const int cnt = min(32, m - base);
        int j = 0;
        while (j < cnt && !D.err) {
            if (s2 == 0) {
                const int r = dyn_fresh_run(D, tk, j, cnt, bucket_peers, last, ntok);
                if (r > 0) { j += r; have = false; continue; }
                if (D.err) break;
            }
            Pre pre;
            pre.valid = false;
            if (s2 != 0 && have) {
                const int r = dyn_repeat_run(D, tk, j, cnt, last, ntok, s2, l2, ra, rb, pre, sh_run);
                if (r > 0) { j += r; continue; }
                if (D.err) break;
            }
            D.cur = j;
            dyn_extend(D, __shfl_sync(FULL, tk, j), last, ntok, s2, l2, have, ra, rb, pre);
            j++;
        }
    }
    err = D.err;
    if (m > 0 && !err) {
        // the newest state's record, without a transition yet
        uint4* rl = rec_ptr(D, last);
        if (lane == 0) {
            rl[0] = make_uint4(ntok, s2, ntok, 0);
            rl[1] = make_uint4(0, 0, 0, 0);
            cb[CB_NTOK] = ntok; cb[CB_NSTATES] = D.n_states; cb[CB_LAST] = last;
            cb[CB_S2] = s2; cb[CB_L2] = l2; cb[CB_BLK_CUR] = D.blk_cur; cb[CB_BLK_END] = D.blk_end;
            cb[CB_NRECSLABS] = D.n_rec_slabs; cb[CB_ROOTDEG] = D.root_deg;
        }
        __syncwarp();
    }
    if (l2 > 0 && !err) SAM_COUNT(D.kc.rounds, 1);       // the draft
    if (l2 > 0 && !err && m > 0) {                      // the state moved: get its record, keep a copy
        if (!have) { const uint4* rs = rec_ptr(D, s2); ra = rs[0]; rb = rs[1]; SAM_COUNT(D.kc.rounds, 1); }
        if (lane == 0) { reinterpret_cast<uint4*>(cb + CB_REC2)[0] = ra; reinterpret_cast<uint4*>(cb + CB_REC2)[1] = rb; }
    }
    s2_out = s2; l2_out = l2; ntok_out = ntok;
    if (!err) flush_counts(b, lane, false, D.kc, m);
}

// Called by one thread of a block after the block's outputs are written (and made known to that
// thread by a block barrier where another warp wrote some of them).
// A block orders its output stores (to mapped host memory) before its count with a device-scope fence;
// the block that counts last has thereby observed all the others, and its one system-scope fence — fences
// are cumulative — orders every block's stores before the flag the host polls.  (A system-scope fence in
// every block is what the host waited for: 3.5 us more at 64 blocks, 7 us more at 256.)
__device__ __forceinline__ void signal_done(const StepArgs& A) {
    __threadfence();
    const int prev = atomicAdd(A.done_count, 1);
    if (prev == (int)gridDim.x - 1) {
        *A.done_count = 0;
        __threadfence_system();
        *reinterpret_cast<volatile int32_t*>(A.done_flag) = A.done_seq;
    }
}

// ------------------------------------------------------------------ the kernel
// VERIFY: the accepted tokens are derived from the previous draft and the target's tokens (sam_step_verified).
template <bool VERIFY>
__global__ void __launch_bounds__(64) sam_step_kernel(const __grid_constant__ StepArgs A) {
    // Programmatic dependent launch: this grid may be scheduled while the previous kernel of the stream
    // is still finishing.  Nothing is read before that kernel has completed and flushed; the kernel
    // after this one is allowed to get scheduled right away (it waits in the same way).
    if (!A.order) {
        // While the previous kernel of the stream finishes: touch (prefetch, no data is used) the lines this
        // block reads first, so that their address translations and L2 lines are at hand after the wait.
        const int pb_ = blockIdx.x, pl_ = threadIdx.x & 31;
        const char* p0 = reinterpret_cast<const char*>(A.W.ctrl + (size_t)pb_ * SAM_CTRL_WORDS);
        const char* p1 = reinterpret_cast<const char*>(A.new_tokens + (size_t)pb_ * A.stride);
        const char* p2 = reinterpret_cast<const char*>(VERIFY ? A.v_draft_len + pb_ : A.counts + pb_);
        const char* pp_ = pl_ == 0 ? p0 : pl_ == 1 ? p0 + 128 : pl_ == 2 ? p1 : p2;
        if (pl_ < 4) asm volatile("prefetch.global.L2 [%0];" ::"l"(pp_));
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");
    const int b = A.order ? A.order[blockIdx.x] : (int)blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __shared__ int32_t sh_l[2], sh_s[2], sh_dl[2], sh_err[2];
    __shared__ __align__(16) uint32_t sh_run[32][12];   // per-token staging of a repeat run (dynamic warp)

    // Everything the step needs to get going is read in one round trip: the slot's 64 control
    // words (state, slab table, copies of the two match states' records), its count, and the
    // first 32 tokens of its row (read before the count is known; unused lanes are ignored).
    uint32_t* cb = A.W.ctrl + (size_t)b * SAM_CTRL_WORDS;
    const int32_t* toks = A.new_tokens + (size_t)b * A.stride;
    const uint32_t cw = cb[lane];                       // control words 0..31
    const uint32_t cw2 = cb[32 + lane];                 // control words 32..63
    int32_t tok_first = 0;
    if (lane < A.stride) tok_first = toks[lane];
    int m, confirmed = 0;
    if (VERIFY) {
        // x_accept = the draft tokens the target reproduces, then the target's own next token
        const int Lp = A.stride - 1;
        int dl = A.v_draft_len[b];
        dl = dl < 0 ? 0 : (dl > Lp ? Lp : dl);
        const int32_t* dr = A.v_draft + (size_t)b * Lp;
        int a = dl;
        for (int base = 0; base < dl; base += 32) {
            const int j = base + lane;
            const bool differs = j < dl && dr[j] != toks[j];
            const unsigned bad = __ballot_sync(FULL, differs);
            if (bad) { a = base + __ffs(bad) - 1; break; }
        }
        m = a + 1;
        if (A.v_max_new) { int cap = A.v_max_new[b]; cap = cap < 0 ? 0 : cap; m = m < cap ? m : cap; }
        confirmed = a < m ? a : m;
    } else {
        m = A.counts[b];
    }
    int status = (int)__shfl_sync(FULL, cw, CB_STATUS);
    const uint32_t ntok0 = __shfl_sync(FULL, cw, CB_NTOK);
    const int L = A.L;
    __syncthreads();          // both warps hold the slot's state as it was before either writes any of it

    // validate the whole step before any state changes (both warps reach the same verdict)
    bool fresh_fail = false;
    if (status == 0) {
        if (m < 0 || m > A.stride) status = SAM_SEQ_BAD_COUNT;
        else if ((int64_t)ntok0 + m > A.W.max_seq_len) status = SAM_SEQ_CAPACITY;
        else {
            const int vocab = A.has_static ? A.S.vocab : A.W.vocab;
            bool bad = false;
            for (int base = 0; base < m; base += 32) {
                int i = base + lane;
                if (i < m) { int t = base == 0 ? tok_first : toks[i]; bad |= (t < 0 || t >= vocab); }
            }
            if (__any_sync(FULL, bad)) status = SAM_SEQ_BAD_TOKEN;
        }
        fresh_fail = status != 0;
    }
    if (status != 0) {
        if (warp == 0) {
            if (fresh_fail && lane == 0) cb[CB_STATUS] = (uint32_t)status;
            for (int j = lane; j < L; j += 32) A.draft_tokens[(size_t)b * L + j] = -1;
            if (lane == 0) {
                A.draft_len[b] = 0; A.match_len[2 * b] = 0; A.match_len[2 * b + 1] = 0; A.source[b] = 0;
                if (A.state) { A.state[2 * b] = 0; A.state[2 * b + 1] = 0; }
                A.status[b] = status;
                if (VERIFY && A.v_counts_out) A.v_counts_out[b] = m;
                if (VERIFY && A.v_accepted_out) A.v_accepted_out[b] = confirmed;
            }
            __syncwarp();
            if (A.done_flag && lane == 0) signal_done(A);
        }
        return;
    }

    // this warp's copy of its match state's record: words CB_REC1.. (warp 0) or CB_REC2.. (warp 1)
    const int rbase = (warp == 0 ? CB_REC1 : CB_REC2) - 32;
    uint4 ra, rb;
    ra.x = __shfl_sync(FULL, cw2, rbase + 0); ra.y = __shfl_sync(FULL, cw2, rbase + 1);
    ra.z = __shfl_sync(FULL, cw2, rbase + 2); ra.w = __shfl_sync(FULL, cw2, rbase + 3);
    rb.x = __shfl_sync(FULL, cw2, rbase + 4); rb.y = __shfl_sync(FULL, cw2, rbase + 5);
    rb.z = __shfl_sync(FULL, cw2, rbase + 6); rb.w = __shfl_sync(FULL, cw2, rbase + 7);

    int32_t d[MAX_DRAFT_REGS] = {-1, -1, -1, -1};
    int32_t my_l = 0, my_s = 0, my_dl = 0;
    int err = 0;

    if (warp == 0) {
        // ---------------- static automaton: Transfer per token ----------------
        if (A.has_static) {
            uint32_t s, sf; int32_t l;
            static_chain<true>(A, b, lane, cb, cw, tok_first, toks, m, ntok0, ra, rb, s, sf, l, err, d, my_dl);
            my_l = l; my_s = (int32_t)s;
        }
    } else {
        // ---------------- dynamic automaton: Expand per token ----------------
        uint32_t s2, l2, ntok;
        dynamic_chain(A, b, lane, cb, cw, cw2, tok_first, toks, m, ntok0, ra, rb, sh_run, s2, l2, ntok, err);
        my_l = (int32_t)l2; my_s = (int32_t)s2;
        if (l2 > 0 && !err) {
            const int64_t e = (int64_t)ra.z;                    // min_endpos
            int64_t room = (int64_t)ntok - e;
            my_dl = (int)(room < L ? (room < 0 ? 0 : room) : L);
            gather_draft<0>(A.W.text + (size_t)b * A.W.text_stride, e, my_dl, L, lane, d);
            my_dl = cut_at_stop(d, my_dl, lane, A.W.stop_token);
        }
    }

    if (lane == 0) { sh_l[warp] = my_l; sh_s[warp] = my_s; sh_dl[warp] = my_dl; sh_err[warp] = err; }
    __syncthreads();
    const int any_err = sh_err[0] ? sh_err[0] : sh_err[1];
    const int l1 = sh_l[0], l2v = sh_l[1];
    const bool use_static = A.has_static && l1 > l2v + A.W.l_bias;        // Section 3.2
    const int lsel = use_static ? l1 : l2v;
    const int need = A.W.min_match > 1 ? A.W.min_match : 1;
    const int src = (any_err || lsel < need) ? SAM_SRC_NONE : (use_static ? SAM_SRC_STATIC : SAM_SRC_DYNAMIC);
    const int winner = src == SAM_SRC_DYNAMIC ? 1 : 0;

    if (warp == winner) {
#pragma unroll
        for (int r = 0; r < MAX_DRAFT_REGS; r++) {
            int j = r * 32 + lane;
            if (j < L) A.draft_tokens[(size_t)b * L + j] = (src == SAM_SRC_NONE) ? -1 : d[r];
        }
    }
    if (warp == 0 && lane == 0) {
        if (any_err) cb[CB_STATUS] = (uint32_t)any_err;
        A.draft_len[b] = src == SAM_SRC_NONE ? 0 : sh_dl[winner];
        A.match_len[2 * b] = any_err ? 0 : l1;
        A.match_len[2 * b + 1] = any_err ? 0 : l2v;
        A.source[b] = src;
        if (A.state) { A.state[2 * b] = any_err ? 0 : sh_s[0]; A.state[2 * b + 1] = any_err ? 0 : sh_s[1]; }
        A.status[b] = any_err;
        if (VERIFY && A.v_counts_out) A.v_counts_out[b] = m;
        if (VERIFY && A.v_accepted_out) A.v_accepted_out[b] = confirmed;
    }
    if (A.done_flag) {
        __syncthreads();
        if (threadIdx.x == 0) signal_done(A);
    }
}

// ------------------------------------------------------------------ the split step (large batches)
// With more slots than the GPU holds blocks of the kernel above, throughput is set by how many chains are
// resident, and a block of two warps holds two warps' worth of registers for as long as its slower chain
// runs.  The split step gives the two sides of a slot to different blocks (of one warp) of one grid:
//   - the dynamic side keeps its warp per slot (dynamic_chain);
//   - the static side of a slot with few tokens needs no cooperation between lanes (a state is one 32-byte
//     record, a hash bucket eight 16-byte entries), so one LANE carries it: a warp advances 32 slots, each
//     round of reads serving 32 chains (static_lanes);
//   - the static side of a slot with many tokens is what a step waits for, so it keeps a warp of its own
//     and everything that shortens the chain (static_chain: read-ahead lookups, prefix states).
// The slots come sorted by token count (order_slots_kernel), which also says how many of them have "many".
// Neither side waits for the other.  Each writes its result to the slot's control block and then counts
// itself in CB_ARRIVE; the side that finds the other already counted (an odd count) reads both results,
// chooses the source, reads the draft and writes the slot's outputs.  Stores are ordered before the
// count by a device-scope fence, and what the other side wrote is read with loads that bypass the L1.
// A slot that fails its validation, or whose dynamic side runs into an error, is reported by the dynamic
// side alone before it counts itself; the static side validates on its own (it keeps the text length in
// CB_NTOK_S because CB_NTOK may change under it) and never commits a state for a step that is refused.

__device__ __forceinline__ void write_failed_slot(const StepArgs& A, int b, int lane, int status) {
    for (int j = lane; j < A.L; j += 32) A.draft_tokens[(size_t)b * A.L + j] = -1;
    if (lane == 0) {
        A.draft_len[b] = 0; A.match_len[2 * b] = 0; A.match_len[2 * b + 1] = 0; A.source[b] = 0;
        if (A.state) { A.state[2 * b] = 0; A.state[2 * b + 1] = 0; }
        A.status[b] = status;
    }
}

// How many sides of the slot have counted themselves, read with acquire semantics: if the count is odd the
// other side is done and everything it wrote may be read from here on (with loads that bypass the L1).
__device__ __forceinline__ uint32_t arrive_look(const uint32_t* cb) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(cb + CB_ARRIVE) : "memory");
    return v;
}

// Count this warp's side of slot `cb` as finished; true if the other side had finished before.
// A side that finds the other one done already (an acquiring look, one read) has no reader for what it wrote
// in this kernel: it counts itself without waiting for its stores.  Otherwise its stores are ordered before
// the count by a device-scope fence — the wait for them to be acknowledged is what that costs — and the
// count's old value decides.
__device__ __forceinline__ bool arrive_warp(uint32_t* cb, int lane) {
    const uint32_t seen = arrive_look(cb);                 // every lane looks for itself (one request)
    if (__all_sync(FULL, (seen & 1u) != 0)) {
        if (lane == 0) atomicAdd(cb + CB_ARRIVE, 1u);
        return true;
    }
    __threadfence();                                       // every lane's own stores ...
    __syncwarp();
    unsigned old = 0;
    if (lane == 0) { __threadfence(); old = atomicAdd(cb + CB_ARRIVE, 1u); }   // ... and, cumulatively, all of them before the count
    old = __shfl_sync(FULL, old, 0);
    if (old & 1u) __threadfence();                         // the other side's stores before this warp's reads of them
    return (old & 1u) != 0;
}

// Both sides of slot b are done: choose the source (Section 3.2), read the draft, write the outputs.
// Run by a whole warp.
__device__ __forceinline__ void split_epilogue(const StepArgs& A, int b, int lane) {
    uint32_t* cb = A.W.ctrl + (size_t)b * SAM_CTRL_WORDS;
    const uint32_t cw = __ldcg(cb + lane), cw2 = __ldcg(cb + 32 + lane);
    if (__shfl_sync(FULL, cw, CB_STATUS) != 0) return;                  // reported by the dynamic side
    const int err_s = (int)__shfl_sync(FULL, cw, CB_ERR_S);
    if (err_s) {
        write_failed_slot(A, b, lane, err_s);
        if (lane == 0) cb[CB_STATUS] = (uint32_t)err_s;
        return;
    }
    const int l1 = (int)__shfl_sync(FULL, cw, CB_L1), l2 = (int)__shfl_sync(FULL, cw, CB_L2);
    const int s1 = (int)__shfl_sync(FULL, cw, CB_S1), s2 = (int)__shfl_sync(FULL, cw, CB_S2);
    const int64_t ntok = (int64_t)__shfl_sync(FULL, cw, CB_NTOK);
    const int64_t e1 = (int64_t)__shfl_sync(FULL, cw2, CB_REC1 + 2 - 32), e2 = (int64_t)__shfl_sync(FULL, cw2, CB_REC2 + 2 - 32);
    const int L = A.L;
    const bool use_static = l1 > l2 + A.W.l_bias;                       // Section 3.2
    const int lsel = use_static ? l1 : l2;
    const int need = A.W.min_match > 1 ? A.W.min_match : 1;
    const int src = lsel < need ? SAM_SRC_NONE : (use_static ? SAM_SRC_STATIC : SAM_SRC_DYNAMIC);
    int32_t d[MAX_DRAFT_REGS] = {-1, -1, -1, -1};
    int dl = 0;
    if (src == SAM_SRC_STATIC) {
        const int64_t room = A.S.n_tokens - e1;
        dl = (int)(room < L ? (room < 0 ? 0 : room) : L);
        gather_draft<1>(A.S.corpus, e1, dl, L, lane, d);
        dl = cut_at_stop(d, dl, lane, A.W.stop_token);
    } else if (src == SAM_SRC_DYNAMIC) {
        const int64_t room = ntok - e2;
        dl = (int)(room < L ? (room < 0 ? 0 : room) : L);
        gather_draft<2>(A.W.text + (size_t)b * A.W.text_stride, e2, dl, L, lane, d);
        dl = cut_at_stop(d, dl, lane, A.W.stop_token);
    }
#pragma unroll
    for (int r = 0; r < MAX_DRAFT_REGS; r++) {
        const int j = r * 32 + lane;
        if (j < L) A.draft_tokens[(size_t)b * L + j] = d[r];
    }
    if (lane == 0) {
        A.draft_len[b] = dl; A.match_len[2 * b] = l1; A.match_len[2 * b + 1] = l2; A.source[b] = src;
        if (A.state) { A.state[2 * b] = s1; A.state[2 * b + 1] = s2; }
        A.status[b] = 0;
    }
}

// The same for the slots of the lanes of a static_lanes warp that found their dynamic side done (`second`).
// Each such lane knows its own side's result (l1, s1, e1, err_s) and reads the other's from its control block;
// the drafts are then read by the whole warp, row after row — lane k reads token k of every pending row, all
// rows' reads issued together — and written the same way.
__device__ __forceinline__ void split_epilogue_lanes(const StepArgs& A, bool second, int b, int lane,
                                                     int l1, int s1, int64_t e1, int err_s) {
    const unsigned pending0 = __ballot_sync(FULL, second);
    if (!pending0) return;
    uint32_t* cb = A.W.ctrl + (size_t)b * SAM_CTRL_WORDS;
    const int L = A.L;
    int l2 = 0, s2 = 0, src = SAM_SRC_NONE, dl = 0, status = 0;
    int64_t e = 0;
    const int32_t* text = A.S.corpus;
    bool mine = second;
    if (second) {
        const uint32_t st = __ldcg(cb + CB_STATUS);
        l2 = (int)__ldcg(cb + CB_L2); s2 = (int)__ldcg(cb + CB_S2);
        const int64_t ntok = (int64_t)__ldcg(cb + CB_NTOK), e2 = (int64_t)__ldcg(cb + CB_REC2 + 2);
        if (st != 0) mine = false;                                       // reported by the dynamic side
        else if (err_s) { status = err_s; l1 = l2 = 0; s1 = s2 = 0; cb[CB_STATUS] = (uint32_t)err_s; }
        else {
            const bool use_static = l1 > l2 + A.W.l_bias;               // Section 3.2
            const int lsel = use_static ? l1 : l2;
            const int need = A.W.min_match > 1 ? A.W.min_match : 1;
            src = lsel < need ? SAM_SRC_NONE : (use_static ? SAM_SRC_STATIC : SAM_SRC_DYNAMIC);
            if (!use_static) text = A.W.text + (size_t)b * A.W.text_stride;
            e = use_static ? e1 : e2;
            const int64_t room = (use_static ? A.S.n_tokens : ntok) - e;
            dl = src == SAM_SRC_NONE ? 0 : (int)(room < L ? (room < 0 ? 0 : room) : L);
        }
    }
    const unsigned pending = __ballot_sync(FULL, mine);
    const int32_t* src_ptr = text + e;
    int32_t* row = A.draft_tokens + (size_t)b * L;
    const int32_t stop = A.W.stop_token;
    int cut = dl;                                                        // this lane's row ends here
    for (int base = 0; base < L; base += 32) {
        int32_t v[32];
#pragma unroll
        for (int i = 0; i < 32; i++) {                                   // row i, token base + lane
            const int32_t* p_i = reinterpret_cast<const int32_t*>(__shfl_sync(FULL, (unsigned long long)src_ptr, i));
            const int dl_i = __shfl_sync(FULL, dl, i);
            v[i] = -1;
            if (base + lane < dl_i) v[i] = __ldcg(p_i + base + lane);
        }
#pragma unroll
        for (int i = 0; i < 32; i++) {
            int cut_i = __shfl_sync(FULL, cut, i);
            const unsigned hit = __ballot_sync(FULL, stop >= 0 && v[i] == stop && base + lane < cut_i);
            if (hit) cut_i = base + __ffs(hit) - 1;                      // a draft ends before the first stop token
            if (lane == i) cut = cut_i;
            int32_t* row_i = reinterpret_cast<int32_t*>(__shfl_sync(FULL, (unsigned long long)row, i));
            if (((pending >> i) & 1u) && base + lane < L) row_i[base + lane] = base + lane < cut_i ? v[i] : -1;
        }
    }
    if (mine) {
        A.draft_len[b] = cut; A.match_len[2 * b] = l1; A.match_len[2 * b + 1] = l2; A.source[b] = src;
        if (A.state) { A.state[2 * b] = s1; A.state[2 * b + 1] = s2; }
        A.status[b] = status;
    }
}

// The static side of 32 slots, one per lane: Transfer (Algorithm 1) for each of the slot's tokens.
// Every pass of the loop is one round of reads for all lanes that still have tokens: the record of the
// lane's state, the home bucket of (state, token) when the state has hashed transitions, the root-row
// entry of the token (used when the walk reaches the root in this pass) and the slot's next token.
__device__ __forceinline__ void static_lanes(const StepArgs& A, int w, int lane) {
    const SamStaticView& S = A.S;
    const int idx = A.W.batch - 1 - (w * 32 + lane);      // from the end of the sorted order: the fewest tokens first
    const int ob = A.order[idx > 0 ? idx : 0];            // (read together with the count below)
    const int first = min(*A.split_count, A.n_warp_blocks);   // the slots before this one have a warp of their own
    const bool live = idx >= first;
    if (!__any_sync(FULL, live)) return;
    const int b = live ? ob : 0;
    uint32_t* cb = A.W.ctrl + (size_t)b * SAM_CTRL_WORDS;
    const int32_t* toks = A.new_tokens + (size_t)b * A.stride;
    uint32_t status = 0, s = 0, sf = 0, ntok_s = 0;
    int32_t l = 0, t = 0;
    int m = 0;
    uint4 ra = make_uint4(0, 0, 0, 0), rb = ra;
    if (live) {
        status = cb[CB_STATUS]; s = cb[CB_S1]; l = (int32_t)cb[CB_L1]; sf = cb[CB_S1FLAG]; ntok_s = cb[CB_NTOK_S];
        ra = *reinterpret_cast<const uint4*>(cb + CB_REC1); rb = *reinterpret_cast<const uint4*>(cb + CB_REC1 + 4);
        m = A.counts[b];
        t = toks[0];
    }
    // the same checks, in the same order, as the dynamic side makes (bad count, capacity, then the tokens
    // one by one as they come up): a refused step leaves the static state as it was
    bool run = live && status == 0 && m >= 0 && m <= A.stride && (int64_t)ntok_s + m <= A.W.max_seq_len;
    bool active = run && m > 0;
    if (active && (t < 0 || t >= S.vocab)) { active = false; run = false; }
    bool have = s != 0;                                  // (ra, rb) is the record of s
    bool need_len = false;
    int j = 0, err = 0;
    int guard = l + 2 * m + 4;                           // at most l + m link moves in all (Appendix A.3)
    [[maybe_unused]] ChainCounts kc = {2, 0, 0, 0, 0};   // two rounds already: the slot's index, its control words
    while (__any_sync(FULL, active)) {
        if (active) SAM_COUNT(kc.rounds, 1);
        // One round of reads for every lane, none of them under a branch (lanes that took different branches
        // would otherwise wait for their reads one group after the other): a lane that does not need a line
        // reads one that every such lane shares (record 0, bucket 0, its own first token).
        const bool at_root = s == 0;
        const bool want_rec = active && !at_root && !have;
        const bool want_bucket = active && !at_root && sf != 0;
        uint32_t home = want_bucket ? sam_hash2(s, (uint32_t)t) & S.hash_mask : 0u;
        const uint32_t re = __ldg(S.root_row + (active ? t : 0));
        const int32_t tn = toks[(active && j + 1 < m) ? j + 1 : 0];
        const size_t ri = want_rec ? (size_t)s : 0;
        uint4 a = __ldg(S.rec + 2 * ri), bb = __ldg(S.rec + 2 * ri + 1);
        uint4 ent[SAM_HASH_BUCKET];
#pragma unroll
        for (int e = 0; e < SAM_HASH_BUCKET; e++) ent[e] = __ldg(S.hash + (size_t)home * SAM_HASH_BUCKET + e);
        if (have) { a = ra; bb = rb; }
        if (active) {
            have = false;
            bool advance = false;
            if (at_root) {                                // at the root the match length is 0
                if (re != SAM_NONE) { s = re & SAM_IDMASK; sf = re >> 31; l = 1; SAM_COUNT(kc.b, 1); } else l = 0;
                advance = true;
            } else {
                if (need_len) { l = (int32_t)a.x; need_len = false; }
                uint32_t tgt = SAM_NONE;
                if (a.w >= 1 && bb.x == (uint32_t)t) tgt = bb.y;
                else if (a.w >= 2 && bb.z == (uint32_t)t) tgt = bb.w;
                else if (a.w > 2) {
                    if (!sf) {                            // (every reference to a state with hashed transitions carries the flag)
                        home = sam_hash2(s, (uint32_t)t) & S.hash_mask;
#pragma unroll
                        for (int e = 0; e < SAM_HASH_BUCKET; e++) ent[e] = __ldg(S.hash + (size_t)home * SAM_HASH_BUCKET + e);
                    }
                    for (int probe = 1;; probe++) {
                        bool empty = false;
#pragma unroll
                        for (int e = 0; e < SAM_HASH_BUCKET; e++) {
                            if (ent[e].x == s && ent[e].y == (uint32_t)t) tgt = ent[e].z;
                            empty |= ent[e].x == SAM_NONE;
                        }
                        if (tgt != SAM_NONE || empty || probe >= S.hash_max_probe) break;
                        home = (home + 1) & S.hash_mask;
#pragma unroll
                        for (int e = 0; e < SAM_HASH_BUCKET; e++) ent[e] = __ldg(S.hash + (size_t)home * SAM_HASH_BUCKET + e);
                    }
                }
                if (tgt != SAM_NONE) { s = tgt & SAM_IDMASK; sf = tgt >> 31; l += 1; advance = true; SAM_COUNT(kc.b, 1); }
                else {                                    // s <- link(s), l <- len(link(s))
                    SAM_COUNT(kc.a, 1);
                    s = a.y & SAM_IDMASK; sf = a.y >> 31;
                    if (s == 0) {                         // the root either has the token or not: known already
                        if (re != SAM_NONE) { s = re & SAM_IDMASK; sf = re >> 31; l = 1; SAM_COUNT(kc.b, 1); } else l = 0;
                        advance = true;
                    } else need_len = true;
                    if (--guard < 0) { err = SAM_SEQ_WALK_LIMIT; active = false; }
                }
            }
            if (advance && active) {
                if (++j < m) {
                    t = tn;
                    if (t < 0 || t >= S.vocab) { active = false; run = false; }
                } else active = false;
            }
        }
    }
    int64_t e1 = (int64_t)ra.z;
    if (run && m > 0 && !err) {
        if (l > 0) {                                      // the state moved: read its record, keep a copy
            ra = __ldg(S.rec + 2 * (size_t)s); rb = __ldg(S.rec + 2 * (size_t)s + 1);
            *reinterpret_cast<uint4*>(cb + CB_REC1) = ra; *reinterpret_cast<uint4*>(cb + CB_REC1 + 4) = rb;
            e1 = (int64_t)ra.z;
        }
        cb[CB_S1] = s; cb[CB_L1] = (uint32_t)l; cb[CB_S1FLAG] = sf; cb[CB_NTOK_S] = ntok_s + (uint32_t)m;
    }
    if (live && err) cb[CB_ERR_S] = (uint32_t)err;
#ifdef SAM_COUNTERS
    if (g_sam_counters && run && b < g_sam_counter_slots) {
        unsigned long long* o = g_sam_counters + (size_t)b * SAM_N_COUNTERS;
        o[SAM_CNT_STATIC_ROUNDS] += kc.rounds + (l > 0 && m > 0 ? 1u : 0u);
        o[SAM_CNT_STATIC_LINK_MOVES] += kc.a; o[SAM_CNT_STATIC_NEXT_MOVES] += kc.b;
    }
#endif
    bool second = false;
    if (live) {
        if (arrive_look(cb) & 1u) { atomicAdd(cb + CB_ARRIVE, 1u); second = true; }
        else {
            __threadfence();
            second = (atomicAdd(cb + CB_ARRIVE, 1u) & 1u) != 0;
            if (second) __threadfence();
        }
    }
    split_epilogue_lanes(A, second, b, lane, l, (int32_t)s, e1, err);
}

// The dynamic side of one slot (one warp), including everything that reports a slot as failed.
__device__ __forceinline__ void dynamic_slot(const StepArgs& A, int b, int lane, uint32_t (*sh_run)[12]) {
    uint32_t* cb = A.W.ctrl + (size_t)b * SAM_CTRL_WORDS;
    const int32_t* toks = A.new_tokens + (size_t)b * A.stride;
    const uint32_t cw = cb[lane];
    const uint32_t cw2 = cb[32 + lane];
    int32_t tok_first = 0;
    if (lane < A.stride) tok_first = toks[lane];
    const int m = A.counts[b];
    int status = (int)__shfl_sync(FULL, cw, CB_STATUS);
    const uint32_t ntok0 = __shfl_sync(FULL, cw, CB_NTOK);
    bool fresh_fail = false;
    if (status == 0) {                                   // validate the whole step before any state changes
        if (m < 0 || m > A.stride) status = SAM_SEQ_BAD_COUNT;
        else if ((int64_t)ntok0 + m > A.W.max_seq_len) status = SAM_SEQ_CAPACITY;
        else {
            bool bad = false;
            for (int base = 0; base < m; base += 32) {
                const int i = base + lane;
                if (i < m) { const int tt = base == 0 ? tok_first : toks[i]; bad |= (tt < 0 || tt >= A.S.vocab); }
            }
            if (__any_sync(FULL, bad)) status = SAM_SEQ_BAD_TOKEN;
        }
        fresh_fail = status != 0;
    }
    int err = 0;
    if (status == 0) {
        const int rbase = CB_REC2 - 32;
        uint4 ra, rb;
        ra.x = __shfl_sync(FULL, cw2, rbase + 0); ra.y = __shfl_sync(FULL, cw2, rbase + 1);
        ra.z = __shfl_sync(FULL, cw2, rbase + 2); ra.w = __shfl_sync(FULL, cw2, rbase + 3);
        rb.x = __shfl_sync(FULL, cw2, rbase + 4); rb.y = __shfl_sync(FULL, cw2, rbase + 5);
        rb.z = __shfl_sync(FULL, cw2, rbase + 6); rb.w = __shfl_sync(FULL, cw2, rbase + 7);
        uint32_t s2, l2, ntok;
        dynamic_chain(A, b, lane, cb, cw, cw2, tok_first, toks, m, ntok0, ra, rb, sh_run, s2, l2, ntok, err);
        if (err) { status = err; fresh_fail = true; }
    }
    if (status != 0) {
        if (fresh_fail && lane == 0) cb[CB_STATUS] = (uint32_t)status;
        write_failed_slot(A, b, lane, status);
        arrive_warp(cb, lane);
        return;
    }
    if (arrive_warp(cb, lane)) split_epilogue(A, b, lane);
}

// The static side of one slot with a warp of its own.
__device__ __forceinline__ void static_slot(const StepArgs& A, int b, int lane) {
    uint32_t* cb = A.W.ctrl + (size_t)b * SAM_CTRL_WORDS;
    const int32_t* toks = A.new_tokens + (size_t)b * A.stride;
    const uint32_t cw = cb[lane];
    const uint32_t cw2 = cb[32 + lane];
    int32_t tok_first = 0;
    if (lane < A.stride) tok_first = toks[lane];
    const int m = A.counts[b];
    const uint32_t ntok_s = __shfl_sync(FULL, cw, CB_NTOK_S);
    bool run = __shfl_sync(FULL, cw, CB_STATUS) == 0 && m >= 0 && m <= A.stride && (int64_t)ntok_s + m <= A.W.max_seq_len;
    if (run) {                                           // the dynamic side reports a refused step; this side only keeps out
        bool bad = false;
        for (int base = 0; base < m; base += 32) {
            const int i = base + lane;
            if (i < m) { const int tt = base == 0 ? tok_first : toks[i]; bad |= (tt < 0 || tt >= A.S.vocab); }
        }
        run = !__any_sync(FULL, bad);
    }
    if (run) {
        const int rbase = CB_REC1 - 32;
        uint4 ra, rb;
        ra.x = __shfl_sync(FULL, cw2, rbase + 0); ra.y = __shfl_sync(FULL, cw2, rbase + 1);
        ra.z = __shfl_sync(FULL, cw2, rbase + 2); ra.w = __shfl_sync(FULL, cw2, rbase + 3);
        rb.x = __shfl_sync(FULL, cw2, rbase + 4); rb.y = __shfl_sync(FULL, cw2, rbase + 5);
        rb.z = __shfl_sync(FULL, cw2, rbase + 6); rb.w = __shfl_sync(FULL, cw2, rbase + 7);
        uint32_t s, sf; int32_t l, dl = 0;
        int32_t d[MAX_DRAFT_REGS];
        int err = 0;
        static_chain<false>(A, b, lane, cb, cw, tok_first, toks, m, ntok_s, ra, rb, s, sf, l, err, d, dl);
        if (err && lane == 0) cb[CB_ERR_S] = (uint32_t)err;
    }
    if (arrive_warp(cb, lane)) split_epilogue(A, b, lane);
}

__global__ void __launch_bounds__(32) sam_step_split_kernel(const __grid_constant__ StepArgs A) {
    {   // while the previous kernel of the stream finishes: a dynamic-side block touches (prefetch, no data is
        // used) the lines it reads first
        const int pi = (int)blockIdx.x - A.n_warp_blocks - A.n_lane_blocks, pl = (int)threadIdx.x;
        if (pi >= 0 && pl < 4) {
            const char* p0 = reinterpret_cast<const char*>(A.W.ctrl + (size_t)pi * SAM_CTRL_WORDS);
            const char* p1 = reinterpret_cast<const char*>(A.new_tokens + (size_t)pi * A.stride);
            const char* p2 = reinterpret_cast<const char*>(A.counts + pi);
            const char* pp = pl == 0 ? p0 : pl == 1 ? p0 + 128 : pl == 2 ? p1 : p2;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(pp));
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");
    __shared__ __align__(16) uint32_t sh_run[32][12];   // per-token staging of a repeat run (dynamic side)
    const int lane = threadIdx.x;
    int i = (int)blockIdx.x;
    if (i < A.n_warp_blocks + A.n_lane_blocks) {
        // slots whose static side gets a warp: the first n_big of the sorted order (read together with order[])
        if (i < A.n_warp_blocks) {
            const int b = A.order[i];
            if (i < min(*A.split_count, A.n_warp_blocks)) static_slot(A, b, lane);
        } else {
            static_lanes(A, i - A.n_warp_blocks, lane);
        }
    } else {
        // the dynamic side's time hardly depends on the token count: slots in their own order, one read less
        dynamic_slot(A, i - A.n_warp_blocks - A.n_lane_blocks, lane, sh_run);
    }
    if (A.done_flag) {
        __syncwarp();
        if (lane == 0) signal_done(A);
    }
}

// A batch larger than the GPU holds at once runs in waves, and a step is as long as its last block: a
// slot with many tokens that starts in the last wave ends late.  This kernel sorts the slots by their
// token count, largest first (a counting sort in shared memory), so that block i of the step kernel takes
// slot order[i] and the long slots start in the first wave.  It reads only the step's counts, so it runs
// while the step before is still going; it ends with griddepcontrol.wait, so that its own completion —
// all the next step kernel waits for — implies that of the step before.
// The counts may still be changing while this kernel reads them (when the kernel before it on the stream
// is the one that writes them), so each count is read exactly once: the key taken from it is kept in
// `keys` and used for both passes.  order[] is therefore a permutation of the slots whatever was read;
// a count read too early only costs the intended launch order, never a result (the step kernel reads the
// counts itself, after its own dependency wait).
constexpr int SAM_ORDER_KEYS = 64;
constexpr int SAM_ORDER_THREADS = 1024;
// (SPLIT: the instance launched ahead of the split step; it is given that kernel's split between L1 and shared
// memory, because kernels that want different ones do not share an SM.)
template <bool SPLIT>
__global__ void __launch_bounds__(SAM_ORDER_THREADS) order_slots_kernel(const int32_t* counts, int32_t B, int32_t* order,
                                                                        int32_t* keys, int32_t big_m, int32_t* n_big) {
    asm volatile("griddepcontrol.launch_dependents;");
    __shared__ int hist[SAM_ORDER_KEYS];
    const int lane = threadIdx.x & 31;
    const unsigned lt = (1u << lane) - 1u;
    for (int k = threadIdx.x; k < SAM_ORDER_KEYS; k += blockDim.x) hist[k] = 0;
    __syncthreads();
    // Four slots per thread and round, so that four reads are under way at a time; the lanes of a warp that
    // hold the same key count themselves with one addition (the counts cluster on a few small values).
    constexpr int U = 4;
    for (int base = 0; base < B; base += U * SAM_ORDER_THREADS) {
        int key[U];
#pragma unroll
        for (int u = 0; u < U; u++) {
            const int i = base + u * SAM_ORDER_THREADS + (int)threadIdx.x;
            key[u] = -1;
            if (i < B) {
                const int m = *reinterpret_cast<const volatile int32_t*>(counts + i);
                key[u] = m < 0 ? 0 : (m >= SAM_ORDER_KEYS ? SAM_ORDER_KEYS - 1 : m);
            }
        }
#pragma unroll
        for (int u = 0; u < U; u++) {
            const int i = base + u * SAM_ORDER_THREADS + (int)threadIdx.x;
            if (i < B) keys[i] = key[u];                     // read back by this same thread below
            const unsigned peers = __match_any_sync(FULL, key[u]);
            if (key[u] >= 0 && (peers & lt) == 0) atomicAdd(&hist[key[u]], __popc(peers));
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {                                  // hist[k] <- first position of key k, keys descending
        int at = 0;
        for (int k = SAM_ORDER_KEYS - 1; k >= 0; k--) {
            const int n = hist[k]; hist[k] = at; at += n;
            if (k == big_m) *n_big = at;                     // slots with at least big_m tokens: the first `at` of order[]
        }
    }
    __syncthreads();
    for (int base = 0; base < B; base += U * SAM_ORDER_THREADS) {
        int key[U];
#pragma unroll
        for (int u = 0; u < U; u++) {
            const int i = base + u * SAM_ORDER_THREADS + (int)threadIdx.x;
            key[u] = i < B ? keys[i] : -1;
        }
#pragma unroll
        for (int u = 0; u < U; u++) {
            const int i = base + u * SAM_ORDER_THREADS + (int)threadIdx.x;
            const unsigned peers = __match_any_sync(FULL, key[u]);
            const int leader = __ffs(peers) - 1;
            int pos = 0;
            if (key[u] >= 0 && lane == leader) pos = atomicAdd(&hist[key[u]], __popc(peers));
            pos = __shfl_sync(FULL, pos, leader) + __popc(peers & lt);
            if (key[u] >= 0 && pos < B) order[pos] = i;      // always true: the keys are those counted above
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// From how many tokens on a slot's static side gets a warp of its own in the split step.  A lane's chain costs
// about 1.3 us per read round against 0.5 us per token for a warp's; up to a few thousand slots a step is as
// long as its slowest slot, beyond that the number of resident warps counts for more.
constexpr int split_big_m(int batch) { return batch >= 8192 ? 8 : 5; }

// The split kernel's blocks are single warps with 1.5 KB of shared memory each: the default split between L1
// and shared memory would hold only a dozen of them per SM.  Once per device.
int split_kernel_setup(int device);

constexpr int SAM_SPLIT_MIN_BATCH = 8192;                    // the split step is used from this many slots on
constexpr int SAM_ORDER_MIN_BATCH = 1536;                    // more slots than a B200 holds blocks of this kernel (148 x 10)

}  // namespace

namespace {
int split_kernel_setup(int device) {
    static bool done[64];
    if (device < 0 || device >= 64) return SAM_ERR_ARG;
    if (!done[device]) {
        cudaError_t e = cudaFuncSetAttribute(sam_step_split_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 50);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(order_slots_kernel<true>, cudaFuncAttributePreferredSharedMemoryCarveout, 50);
        if (e != cudaSuccess) { sam_set_cuda_error(e); return SAM_ERR_CUDA; }
        done[device] = true;
    }
    return SAM_OK;
}
}  // namespace

int sam_step_launch_count(const sam_batch* b) { return b->view.batch >= SAM_ORDER_MIN_BATCH ? 2 : 1; }

int sam_launch_step(const sam_batch* b, const int32_t* new_tokens, int32_t stride, const int32_t* counts,
                    int32_t L, int32_t* draft_tokens, int32_t* draft_len, int32_t* match_len,
                    int32_t* source, int32_t* state, int32_t* status, cudaStream_t stream) {
    return sam_launch_step_signal(b, new_tokens, stride, counts, L, draft_tokens, draft_len, match_len, source, state,
                                  status, stream, nullptr, 0);
}

int sam_launch_step_signal(const sam_batch* b, const int32_t* new_tokens, int32_t stride, const int32_t* counts,
                           int32_t L, int32_t* draft_tokens, int32_t* draft_len, int32_t* match_len,
                           int32_t* source, int32_t* state, int32_t* status, cudaStream_t stream,
                           int32_t* done_flag_dev, int32_t done_seq) {
    return sam_launch_step_full(b, new_tokens, stride, counts, L, draft_tokens, draft_len, match_len, source, state,
                                status, stream, done_flag_dev, done_seq, nullptr, nullptr, nullptr, nullptr, nullptr);
}

int sam_launch_step_full(const sam_batch* b, const int32_t* new_tokens, int32_t stride, const int32_t* counts,
                         int32_t L, int32_t* draft_tokens, int32_t* draft_len, int32_t* match_len,
                         int32_t* source, int32_t* state, int32_t* status, cudaStream_t stream,
                         int32_t* done_flag_dev, int32_t done_seq,
                         const int32_t* v_draft, const int32_t* v_draft_len, const int32_t* v_max_new,
                         int32_t* v_counts_out, int32_t* v_accepted_out) {
    StepArgs A;
    A.v_draft = v_draft; A.v_draft_len = v_draft_len; A.v_max_new = v_max_new;
    A.v_counts_out = v_counts_out; A.v_accepted_out = v_accepted_out;
    A.done_count = b->view.pool_hdr + 4; A.done_flag = done_flag_dev; A.done_seq = done_seq;
    A.has_static = b->st != nullptr;
    if (b->st) A.S = b->st->view;
    else { A.S = SamStaticView(); A.S.vocab = b->view.vocab; }
    A.W = b->view;
    A.new_tokens = new_tokens; A.stride = stride; A.counts = counts; A.L = L;
    A.draft_tokens = draft_tokens; A.draft_len = draft_len; A.match_len = match_len;
    A.source = source; A.state = state; A.status = status;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    A.order = nullptr; A.split_count = nullptr;
    // (A host-array step is synchronous: nothing runs before it that the ordering kernel could overlap with, so it
    // would cost more than the order saves; such a step is always the one two-warp launch, slots in their own order.)
    if (!v_draft && !done_flag_dev && b->view.batch >= SAM_ORDER_MIN_BATCH) {
        int32_t* order = b->view.order + (size_t)(b->order_phase & 1) * b->view.batch;
        cudaLaunchConfig_t oc;
        memset(&oc, 0, sizeof(oc));
        oc.gridDim = dim3(1); oc.blockDim = dim3(SAM_ORDER_THREADS); oc.stream = stream; oc.attrs = attr; oc.numAttrs = 1;
        int32_t* n_big = b->view.order + 3 * (size_t)b->view.batch + 8 * (b->order_phase & 1);
        const bool split = A.has_static && b->view.batch >= SAM_SPLIT_MIN_BATCH;
        if (split) { int rc = split_kernel_setup(b->device); if (rc) return rc; }
        cudaError_t oe = split
            ? cudaLaunchKernelEx(&oc, order_slots_kernel<true>, counts, (int32_t)b->view.batch, order,
                                 b->view.order + 2 * (size_t)b->view.batch, split_big_m(b->view.batch), n_big)
            : cudaLaunchKernelEx(&oc, order_slots_kernel<false>, counts, (int32_t)b->view.batch, order,
                                 b->view.order + 2 * (size_t)b->view.batch, split_big_m(b->view.batch), n_big);
        A.split_count = n_big;
        b->order_phase ^= 1;
        if (oe != cudaSuccess) { sam_set_cuda_error(oe); return SAM_ERR_CUDA; }
        A.order = order;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)b->view.batch); cfg.blockDim = dim3(64); cfg.dynamicSmemBytes = 0; cfg.stream = stream;
    cfg.attrs = attr; cfg.numAttrs = 1;
    A.n_warp_blocks = A.n_lane_blocks = 0;
    cudaError_t e;
    if (A.order && A.has_static && b->view.batch >= SAM_SPLIT_MIN_BATCH) {   // the two sides of a slot in different blocks
        int rc = split_kernel_setup(b->device);
        if (rc) return rc;
        A.n_warp_blocks = (b->view.batch + 3) / 4;
        A.n_lane_blocks = (b->view.batch + 31) / 32;
        cfg.gridDim = dim3((unsigned)(b->view.batch + A.n_warp_blocks + A.n_lane_blocks)); cfg.blockDim = dim3(32);
        e = cudaLaunchKernelEx(&cfg, sam_step_split_kernel, A);
    } else {
        e = v_draft ? cudaLaunchKernelEx(&cfg, sam_step_kernel<true>, A)
                    : cudaLaunchKernelEx(&cfg, sam_step_kernel<false>, A);
    }
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { sam_set_cuda_error(e); return SAM_ERR_CUDA; }
    return SAM_OK;
}

extern "C" int sam_counters_available(void) {
#ifdef SAM_COUNTERS
    return 1;
#else
    return 0;
#endif
}

extern "C" int sam_counters_attach(uint64_t* counters_dev, int32_t slots) {
#ifdef SAM_COUNTERS
    if (slots < 0 || (!counters_dev && slots > 0)) return SAM_ERR_ARG;
    unsigned long long* p = reinterpret_cast<unsigned long long*>(counters_dev);
    int n = counters_dev ? slots : 0;
    SAM_CUDA(cudaMemcpyToSymbol(g_sam_counters, &p, sizeof(p)));
    SAM_CUDA(cudaMemcpyToSymbol(g_sam_counter_slots, &n, sizeof(n)));
    return SAM_OK;
#else
    (void)counters_dev; (void)slots;
    return SAM_ERR_UNSUPPORTED;
#endif
}
