/*
 * sam_oracle.c — TEST INFRASTRUCTURE.  A plain, slow, obviously-correct CPU suffix automaton
 * and the batched draft-retrieval step built on it.  It exists to check the CUDA library and to
 * be timed beside it as a reported CPU baseline; nothing in the product path may call it, and it
 * shares no code, header, table or helper with the CUDA path.
 *
 * Everything follows the paper's notation (SAM-Decoding, arXiv 2411.10666):
 *   state fields  link, next, length, min_endpos          (Section 3.1, Appendix A.1)
 *   Transfer      longest-suffix-match step               (Algorithm 1)
 *   Expand        Blumer's online extension with clone    (Algorithm 3)
 *   Build-SAM     Expand over every token                 (Algorithm 3)
 *   update order  Transfer on the automaton as it was, then Expand (Section 3.3)
 *   draft         d = T[p+1 : p+n], p = min_endpos of the matched state (Section 3.2)
 *   source choice static iff l1 > l2 + l_bias             (Section 3.2)
 * Positions are 1-based exactly as in Algorithm 3 (max_length is incremented before it is used),
 * so min_endpos = p says "the first occurrence ends at the p-th token" and, in 0-based array
 * terms, the draft starts at index p.
 *
 * Data structure: one growable array of (token, target) pairs per state, kept sorted by token
 * and searched by bisection; `next` of a clone is a plain copy of that array.  No hashing, no
 * inline edges, no renumbering: states are numbered in creation order (root 0, a new state c
 * before its clone cl).
 *
 * Parity pins (tests/test_oracle_*.py): the automaton of "ABCBC" derived by hand from
 * Algorithm 3; brute-force longest-suffix search on thousands of tiny random inputs; size and
 * structure invariants (states <= 2n-1, transitions <= 3n-4, len/link/min_endpos relations,
 * distinct-substring count); closed forms (a^n, all-distinct, periodic, corpus-prefix streams);
 * the 2L bound on Transfer moves (Appendix A.3).  What only an automaton can certify at 10M+
 * tokens (that a reported match is the LONGEST and its end position the EARLIEST) is pinned
 * transitively through those; beyond that it is "parity unpinned".
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct { int32_t tok, tgt; } oedge_t;

typedef struct {
    int32_t* link;
    int32_t* length;
    int32_t* min_endpos;
    oedge_t** next;          /* next[s]: sorted array of deg[s] pairs */
    int32_t* deg;
    int32_t* cap;
    uint8_t* is_clone;       /* 1 for states made by cloning (freq starts at 0), Appendix A.1 */
    int64_t n_states, cap_states;
    int64_t n_transitions;
    int32_t last;
    int32_t max_length;
    int err;                 /* 1 = out of memory, 2 = an asserted property failed */
    /* counters of Expand */
    int64_t c_walk_inserts, c_walk_steps, c_clones, c_copied_edges, c_redirects;
} osam_t;

/* ------------------------------------------------------------------ next map */

static int next_find(const osam_t* S, int32_t s, int32_t t) {       /* index or -1 */
    const oedge_t* e = S->next[s];
    int lo = 0, hi = S->deg[s] - 1;
    while (lo <= hi) {
        int mid = (lo + hi) >> 1;
        if (e[mid].tok == t) return mid;
        if (e[mid].tok < t) lo = mid + 1; else hi = mid - 1;
    }
    return -1;
}

static int32_t next_get(const osam_t* S, int32_t s, int32_t t) {    /* target or -1 */
    int i = next_find(S, s, t);
    return i < 0 ? -1 : S->next[s][i].tgt;
}

static void next_set(osam_t* S, int32_t s, int32_t t, int32_t tgt) {
    int i = next_find(S, s, t);
    if (i >= 0) { S->next[s][i].tgt = tgt; return; }
    if (S->deg[s] == S->cap[s]) {
        int32_t nc = S->cap[s] ? S->cap[s] * 2 : 2;
        oedge_t* ne = (oedge_t*)realloc(S->next[s], sizeof(oedge_t) * (size_t)nc);
        if (!ne) { S->err = 1; return; }
        S->next[s] = ne; S->cap[s] = nc;
    }
    oedge_t* e = S->next[s];
    int k = S->deg[s];
    while (k > 0 && e[k - 1].tok > t) { e[k] = e[k - 1]; k--; }
    e[k].tok = t; e[k].tgt = tgt;
    S->deg[s]++; S->n_transitions++;
}

/* ------------------------------------------------------------------ states */

static int grow_states(osam_t* S, int64_t want) {
    if (want <= S->cap_states) return 0;
    int64_t nc = S->cap_states ? S->cap_states : 16;
    while (nc < want) nc *= 2;
    int32_t* a = (int32_t*)realloc(S->link, sizeof(int32_t) * (size_t)nc);        if (!a) return -1; S->link = a;
    int32_t* b = (int32_t*)realloc(S->length, sizeof(int32_t) * (size_t)nc);      if (!b) return -1; S->length = b;
    int32_t* c = (int32_t*)realloc(S->min_endpos, sizeof(int32_t) * (size_t)nc);  if (!c) return -1; S->min_endpos = c;
    oedge_t** d = (oedge_t**)realloc(S->next, sizeof(oedge_t*) * (size_t)nc);     if (!d) return -1; S->next = d;
    int32_t* e = (int32_t*)realloc(S->deg, sizeof(int32_t) * (size_t)nc);         if (!e) return -1; S->deg = e;
    int32_t* f = (int32_t*)realloc(S->cap, sizeof(int32_t) * (size_t)nc);         if (!f) return -1; S->cap = f;
    uint8_t* g = (uint8_t*)realloc(S->is_clone, (size_t)nc);                      if (!g) return -1; S->is_clone = g;
    S->cap_states = nc;
    return 0;
}

/* Expand-State (Algorithm 3): a new state with the given link, empty next, length and position. */
static int32_t expand_state(osam_t* S, int32_t link, int32_t length, int32_t pos) {
    if (grow_states(S, S->n_states + 1)) { S->err = 1; return -1; }
    int32_t s = (int32_t)S->n_states++;
    S->link[s] = link; S->length[s] = length; S->min_endpos[s] = pos;
    S->next[s] = NULL; S->deg[s] = 0; S->cap[s] = 0; S->is_clone[s] = 0;
    return s;
}

/* INIT_SAM (Appendix A.1): root only, link -1, next empty, length 0, min_endpos 0. */
osam_t* osam_new(int64_t states_hint) {
    osam_t* S = (osam_t*)calloc(1, sizeof(osam_t));
    if (!S) return NULL;
    if (states_hint > 0 && grow_states(S, states_hint)) { free(S); return NULL; }
    expand_state(S, -1, 0, 0);
    S->last = 0; S->max_length = 0;
    return S;
}

void osam_free(osam_t* S) {
    if (!S) return;
    for (int64_t s = 0; s < S->n_states; s++) free(S->next[s]);
    free(S->link); free(S->length); free(S->min_endpos); free(S->next); free(S->deg); free(S->cap); free(S->is_clone);
    free(S);
}

/* Expand (Algorithm 3). */
void osam_expand(osam_t* S, int32_t t) {
    S->max_length += 1;
    int32_t l = S->max_length;
    int32_t c = expand_state(S, -1, l, l);
    if (c < 0) return;
    int32_t p = S->last;
    while (p != -1 && next_get(S, p, t) == -1) {
        next_set(S, p, t, c);
        S->c_walk_inserts++;
        p = S->link[p];
    }
    if (p == -1) {
        S->link[c] = 0;
    } else {
        int32_t q = next_get(S, p, t);
        if (S->length[p] + 1 == S->length[q]) {
            S->link[c] = q;
        } else {
            int32_t cl = expand_state(S, -1, -1, -1);
            if (cl < 0) return;
            S->is_clone[cl] = 1;
            S->link[cl] = S->link[q];
            for (int i = 0; i < S->deg[q]; i++) {               /* cl.next = copy of q.next */
                next_set(S, cl, S->next[q][i].tok, S->next[q][i].tgt);
                S->c_copied_edges++;
            }
            S->length[cl] = S->length[p] + 1;
            S->min_endpos[cl] = S->min_endpos[q];
            S->c_clones++;
            while (p != -1) {
                int32_t u = next_get(S, p, t);
                if (u == -1) { S->err = 2; break; }              /* every state up the chain has t */
                if (u != q) break;
                next_set(S, p, t, cl);
                S->c_redirects++;
                p = S->link[p];
            }
            S->link[q] = cl;
            S->link[c] = cl;
        }
    }
    S->last = c;
}

/* Build-SAM (Algorithm 3). */
osam_t* osam_build(const int32_t* tokens, int64_t n) {
    osam_t* S = osam_new(n + n / 2 + 16);
    if (!S) return NULL;
    for (int64_t i = 0; i < n && !S->err; i++) osam_expand(S, tokens[i]);
    return S;
}

/* Transfer (Algorithm 1).  moves[0] += link moves, moves[1] += next moves (may be NULL). */
void osam_transfer(const osam_t* S, int32_t t, int32_t* s_io, int32_t* l_io, int64_t* moves) {
    int32_t s = *s_io, l = *l_io;
    while (s != 0 && next_get(S, s, t) == -1) {
        s = S->link[s];
        l = S->length[s];
        if (moves) moves[0]++;
    }
    int32_t u = next_get(S, s, t);
    if (u != -1) { s = u; l = l + 1; if (moves) moves[1]++; }
    else l = 0;
    *s_io = s; *l_io = l;
}

/* ------------------------------------------------------------------ inspection */

int64_t osam_n_states(const osam_t* S) { return S->n_states; }
int64_t osam_n_transitions(const osam_t* S) { return S->n_transitions; }
int32_t osam_last(const osam_t* S) { return S->last; }
int osam_err(const osam_t* S) { return S->err; }
int32_t osam_link(const osam_t* S, int32_t s) { return S->link[s]; }
int32_t osam_length(const osam_t* S, int32_t s) { return S->length[s]; }
int32_t osam_min_endpos(const osam_t* S, int32_t s) { return S->min_endpos[s]; }
int32_t osam_deg(const osam_t* S, int32_t s) { return S->deg[s]; }
int32_t osam_next(const osam_t* S, int32_t s, int32_t t) { return next_get(S, s, t); }
void osam_edges(const osam_t* S, int32_t s, int32_t* toks, int32_t* tgts) {
    for (int i = 0; i < S->deg[s]; i++) { toks[i] = S->next[s][i].tok; tgts[i] = S->next[s][i].tgt; }
}
/* whole-table dumps: link, length, min_endpos, deg, each [n_states] */
void osam_tables(const osam_t* S, int32_t* link, int32_t* length, int32_t* min_endpos, int32_t* deg) {
    memcpy(link, S->link, sizeof(int32_t) * (size_t)S->n_states);
    memcpy(length, S->length, sizeof(int32_t) * (size_t)S->n_states);
    memcpy(min_endpos, S->min_endpos, sizeof(int32_t) * (size_t)S->n_states);
    memcpy(deg, S->deg, sizeof(int32_t) * (size_t)S->n_states);
}
/* counters: walk_inserts, clones, copied_edges, redirects */
void osam_counters(const osam_t* S, int64_t* out) {
    out[0] = S->c_walk_inserts; out[1] = S->c_clones; out[2] = S->c_copied_edges; out[3] = S->c_redirects;
}

/* ------------------------------------------------------------------ frequencies and top-k successors
 *
 * Appendix A.1 / A.2: every state carries `freq`, the frequency of occurrence of its substrings in
 * the reference text, initialised to 1 for states made by expansion and 0 for clones; the top-k
 * successors of a state are its transitions with the largest freq, and the transition probability
 * is freq(target) / freq(state).
 * Reading taken for the accumulation: freq(s) = init(s) + sum of freq(u) over the states u whose
 * suffix link is s, i.e. the number of end positions of s's substrings.  (The printed recursion
 * over `next` visits a state once per path that reaches it; the prose fixes the meaning.)
 * Which states are clones is recorded when Expand makes them.
 */
void osam_freq(const osam_t* S, int64_t* freq) {
    int64_t n = S->n_states;
    /* order states by decreasing length with a counting sort */
    int32_t maxlen = S->max_length;
    int64_t* bucket = (int64_t*)calloc((size_t)maxlen + 2, sizeof(int64_t));
    int32_t* order = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    for (int64_t s = 0; s < n; s++) bucket[S->length[s] + 1]++;
    for (int32_t l = 0; l <= maxlen; l++) bucket[l + 1] += bucket[l];
    for (int64_t s = 0; s < n; s++) order[bucket[S->length[s]]++] = (int32_t)s;
    for (int64_t s = 0; s < n; s++) freq[s] = (s != 0 && S->is_clone[s] == 0) ? 1 : 0;
    for (int64_t i = n - 1; i > 0; i--) {
        int32_t s = order[i];
        if (S->link[s] >= 0) freq[S->link[s]] += freq[s];
    }
    free(bucket); free(order);
}

/* top-k successors of state s by (freq descending, token ascending); returns how many */
int32_t osam_topk(const osam_t* S, const int64_t* freq, int32_t s, int32_t k, int32_t* toks, int32_t* tgts) {
    int32_t n = 0;
    for (int i = 0; i < S->deg[s]; i++) {
        int32_t t = S->next[s][i].tok, u = S->next[s][i].tgt;      /* tokens come in ascending order */
        int32_t pos = n;
        while (pos > 0 && freq[tgts[pos - 1]] < freq[u]) pos--;     /* strictly larger moves ahead: ties keep token order */
        if (pos >= k) continue;
        int32_t last = n < k ? n : k - 1;
        for (int32_t j = last; j > pos; j--) { toks[j] = toks[j - 1]; tgts[j] = tgts[j - 1]; }
        toks[pos] = t; tgts[pos] = u;
        if (n < k) n++;
    }
    return n;
}

/* ------------------------------------------------------------------ batched step
 *
 * One decoding step for B sequences (Sections 3.2 and 3.3).  For sequence b with m = counts[b]
 * accepted tokens x_{t+1..t+m}:
 *   static :  (s1, l1) <- Transfer(S_static, x, s1, l1)                       for each token
 *   dynamic:  (s2, l2) <- Transfer(S_dyn, x, s2, l2);  S_dyn <- Expand(S_dyn, x)  for each token
 * then the source is static iff l1 > l2 + l_bias, and the draft is the slice of that source's
 * text after min_endpos of its state, at most L tokens, clipped at the end of the text.
 *
 * Readings where the paper is silent:
 *   - after Expand clones the state the dynamic matcher sits in, the matcher is moved to the
 *     canonical state of its match length: while len[link[s]] >= l, s <- link[s].  It must then
 *     equal link[last] with l = len[s]; this is asserted after every token (err 2 otherwise).
 *   - every token of a sequence, prompt included, goes through both automata.
 *   - a chosen match shorter than max(1, min_match) yields no draft (source 0).
 *   - ties go to the dynamic automaton (strict >).
 *   - a draft is clipped at the end of the text; no wrap-around.
 *   - with a stop token set (the EOS that joins the corpus' documents, Section 3.1) a draft ends
 *     before its first occurrence.
 * Boundary conventions of the library that the oracle mirrors so whole arrays compare equal:
 *   status 1: n + m > max_seq_len; 3: a token outside [0, vocab); 4: m < 0 or m > stride.
 *   A sequence with a non-zero status is frozen from then on and reports zeros / -1 drafts.
 *   m = 0 re-emits the draft for the current state.
 */
typedef struct {
    const osam_t* st;           /* static automaton or NULL */
    const int32_t* corpus; int64_t corpus_len;
    int32_t batch, vocab, max_seq_len, l_bias, min_match;
    int32_t stop_token;         /* a draft ends before the first such token; -1 = none */
    osam_t** dyn;               /* [batch] */
    int32_t** text;             /* [batch][max_seq_len] */
    int32_t *n, *s1, *l1, *s2, *l2, *status;
    int err;
    /* per-sequence counters: static link moves, static next moves, dynamic link moves,
       dynamic next moves, tokens, draft tokens, non-empty steps */
    int64_t (*cnt)[8];
} obatch_t;

obatch_t* obatch_new(const osam_t* st, const int32_t* corpus, int64_t corpus_len,
                     int32_t batch, int32_t vocab, int32_t max_seq_len,
                     int32_t l_bias, int32_t min_match, int32_t stop_token) {
    obatch_t* B = (obatch_t*)calloc(1, sizeof(obatch_t));
    B->st = st; B->corpus = corpus; B->corpus_len = corpus_len;
    B->batch = batch; B->vocab = vocab; B->max_seq_len = max_seq_len;
    B->l_bias = l_bias; B->min_match = min_match; B->stop_token = stop_token;
    B->dyn = (osam_t**)calloc((size_t)batch, sizeof(osam_t*));
    B->text = (int32_t**)calloc((size_t)batch, sizeof(int32_t*));
    B->n = (int32_t*)calloc((size_t)batch, 4); B->s1 = (int32_t*)calloc((size_t)batch, 4);
    B->l1 = (int32_t*)calloc((size_t)batch, 4); B->s2 = (int32_t*)calloc((size_t)batch, 4);
    B->l2 = (int32_t*)calloc((size_t)batch, 4); B->status = (int32_t*)calloc((size_t)batch, 4);
    B->cnt = calloc((size_t)batch, sizeof(int64_t[8]));
    for (int32_t b = 0; b < batch; b++) {
        B->dyn[b] = osam_new(0);
        B->text[b] = (int32_t*)malloc(sizeof(int32_t) * (size_t)(max_seq_len > 0 ? max_seq_len : 1));
    }
    return B;
}

void obatch_free(obatch_t* B) {
    if (!B) return;
    for (int32_t b = 0; b < B->batch; b++) { osam_free(B->dyn[b]); free(B->text[b]); }
    free(B->dyn); free(B->text); free(B->n); free(B->s1); free(B->l1); free(B->s2); free(B->l2);
    free(B->status); free(B->cnt); free(B);
}

/* Forget sequence `slot` (empty dynamic automaton, both matchers at the root). */
void obatch_reset(obatch_t* B, int32_t slot) {
    osam_free(B->dyn[slot]);
    B->dyn[slot] = osam_new(0);
    B->n[slot] = B->s1[slot] = B->l1[slot] = B->s2[slot] = B->l2[slot] = B->status[slot] = 0;
}

static void step_one(obatch_t* B, int32_t b, const int32_t* toks, int32_t stride, int32_t m,
                     int32_t L, int32_t* draft, int32_t* draft_len, int32_t* match_len,
                     int32_t* source, int32_t* state, int32_t* status) {
    for (int32_t i = 0; i < L; i++) draft[i] = -1;
    *draft_len = 0; match_len[0] = match_len[1] = 0; *source = 0; state[0] = state[1] = 0;
    if (B->status[b] == 0) {                                   /* validate before touching anything */
        if (m < 0 || m > stride) B->status[b] = 4;
        else if ((int64_t)B->n[b] + m > B->max_seq_len) B->status[b] = 1;
        else for (int32_t i = 0; i < m; i++) if (toks[i] < 0 || toks[i] >= B->vocab) { B->status[b] = 3; break; }
    }
    *status = B->status[b];
    if (B->status[b] != 0) return;

    osam_t* D = B->dyn[b];
    int64_t* cnt = B->cnt[b];
    for (int32_t i = 0; i < m; i++) {
        int32_t t = toks[i];
        if (B->st) osam_transfer(B->st, t, &B->s1[b], &B->l1[b], &cnt[0]);      /* Section 3.3, static */
        osam_transfer(D, t, &B->s2[b], &B->l2[b], &cnt[2]);                      /* Section 3.3, dynamic: Transfer ... */
        osam_expand(D, t);                                                       /* ... then Expand */
        int32_t s = B->s2[b], l = B->l2[b];
        while (s != 0 && D->length[D->link[s]] >= l) s = D->link[s];             /* canonical state of length l */
        B->s2[b] = s;
        if (s != D->link[D->last] || l != D->length[s]) B->err = 2;
        B->text[b][B->n[b]++] = t;
        cnt[4]++;
    }
    if (D->err) B->err = D->err;
    if (m > 0) cnt[6]++;

    int32_t l1 = B->st ? B->l1[b] : 0, l2 = B->l2[b];
    match_len[0] = l1; match_len[1] = l2;
    state[0] = B->st ? B->s1[b] : 0; state[1] = B->s2[b];
    int use_static = l1 > l2 + B->l_bias;                                        /* Section 3.2 */
    int32_t lsel = use_static ? l1 : l2;
    int32_t need = B->min_match > 1 ? B->min_match : 1;
    if (lsel < need) return;
    *source = use_static ? 1 : 2;
    const int32_t* text = use_static ? B->corpus : B->text[b];
    int64_t n_text = use_static ? B->corpus_len : B->n[b];
    int64_t p = use_static ? B->st->min_endpos[B->s1[b]] : D->min_endpos[B->s2[b]];
    int64_t dl = n_text - p; if (dl > L) dl = L; if (dl < 0) dl = 0;             /* d = T[p+1 : p+n], clipped */
    if (B->stop_token >= 0)                                                      /* stop at a document separator */
        for (int64_t i = 0; i < dl; i++) if (text[p + i] == B->stop_token) { dl = i; break; }
    for (int64_t i = 0; i < dl; i++) draft[i] = text[p + i];
    *draft_len = (int32_t)dl;
    cnt[5] += dl;
}

/* new_tokens [batch, stride], counts [batch]; outputs draft_tokens [batch, L], draft_len [batch],
 * match_len [batch, 2], source [batch], state [batch, 2], status [batch].  threads > 1 splits the
 * sequences over that many OpenMP threads (the static automaton is shared read-only). */
int obatch_step(obatch_t* B, const int32_t* new_tokens, int32_t stride, const int32_t* counts,
                int32_t L, int32_t* draft_tokens, int32_t* draft_len, int32_t* match_len,
                int32_t* source, int32_t* state, int32_t* status, int32_t threads) {
    #pragma omp parallel for schedule(dynamic, 1) num_threads(threads > 0 ? threads : 1)
    for (int32_t b = 0; b < B->batch; b++)
        step_one(B, b, new_tokens + (int64_t)b * stride, stride, counts[b], L,
                 draft_tokens + (int64_t)b * L, draft_len + b, match_len + 2 * (int64_t)b,
                 source + b, state + 2 * (int64_t)b, status + b);
    return B->err;
}

/* Run a whole schedule without returning to the caller between steps (used for timing):
 * new_tokens [n_steps, batch, stride], counts [n_steps, batch]; outputs of the LAST step only. */
int obatch_run(obatch_t* B, const int32_t* new_tokens, int32_t stride, const int32_t* counts,
               int32_t n_steps, int32_t L, int32_t* draft_tokens, int32_t* draft_len,
               int32_t* match_len, int32_t* source, int32_t* state, int32_t* status, int32_t threads) {
    #pragma omp parallel for schedule(dynamic, 1) num_threads(threads > 0 ? threads : 1)
    for (int32_t b = 0; b < B->batch; b++)
        for (int32_t s = 0; s < n_steps; s++)
            step_one(B, b, new_tokens + ((int64_t)s * B->batch + b) * stride, stride,
                     counts[(int64_t)s * B->batch + b], L,
                     draft_tokens + (int64_t)b * L, draft_len + b, match_len + 2 * (int64_t)b,
                     source + b, state + 2 * (int64_t)b, status + b);
    return B->err;
}

osam_t* obatch_dyn(obatch_t* B, int32_t b) { return B->dyn[b]; }
int32_t obatch_len(const obatch_t* B, int32_t b) { return B->n[b]; }
/* summed counters: static link moves, static next moves, dynamic link moves, dynamic next moves,
 * tokens, draft tokens, non-empty sequence-steps, then Expand's walk_inserts, clones,
 * copied_edges, redirects, states, transitions */
void obatch_counters(const obatch_t* B, int64_t* out) {
    for (int k = 0; k < 13; k++) out[k] = 0;
    for (int32_t b = 0; b < B->batch; b++) {
        for (int k = 0; k < 7; k++) out[k] += B->cnt[b][k];
        out[7] += B->dyn[b]->c_walk_inserts; out[8] += B->dyn[b]->c_clones;
        out[9] += B->dyn[b]->c_copied_edges; out[10] += B->dyn[b]->c_redirects;
        out[11] += B->dyn[b]->n_states; out[12] += B->dyn[b]->n_transitions;
    }
}
