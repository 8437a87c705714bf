/*
 * samgen — seeded synthetic token streams for suffix-automaton draft retrieval.
 *
 * This file only DRAWS INPUTS: token corpora, prompts, generated continuations and
 * per-step accepted-token counts.  It holds no suffix-automaton arithmetic and is
 * the one piece of code that both the CPU oracle's tests and the CUDA path's tests
 * consume (each gets the same arrays).
 *
 * Random numbers: a counter-based generator.  Draw number `i` of stream `k` under
 * seed `s` is  splitmix64_finalise(s' + (i+1) * GOLDEN)  with s' = finalise(s ^ finalise(k)),
 * the finaliser being the published splitmix64 output function (Steele, Lea, Flood 2014).
 *
 * Token models
 *   zipf    : rank r in [0,V) with P(r) proportional to (r+1)^-s, inverse-CDF by binary search;
 *             token id = perm[r], perm a seeded permutation so ids are not frequency-sorted.
 *   markov2 : the same ranks, but the rank->id map is rotated by a hash of the two previous
 *             tokens: id = perm[(r + h(t[i-2], t[i-1])) mod V].  Every order-2 context has its
 *             own Zipf-ranked next-token row without any table being stored.
 *   spans   : at each position a verbatim copy of length U[lo,hi] starts with probability
 *             q = f / (f + mean_len * (1 - f)), which makes copies cover a fraction f of all
 *             positions in expectation; the copy source start is uniform over the source text.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

#define GOLDEN 0x9E3779B97F4A7C15ull

static inline uint64_t fin64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

typedef struct { uint64_t key, ctr; } rng_t;

static inline void rng_init(rng_t* r, uint64_t seed, uint64_t stream) {
    r->key = fin64(seed ^ fin64(stream + GOLDEN));
    r->ctr = 0;
}
static inline uint64_t rng_u64(rng_t* r) { r->ctr++; return fin64(r->key + r->ctr * GOLDEN); }
static inline double rng_u01(rng_t* r) { return (double)(rng_u64(r) >> 11) * (1.0 / 9007199254740992.0); }
/* uniform integer in [lo, hi], hi >= lo; modulo bias is below 2^-32 for the ranges used here */
static inline int64_t rng_range(rng_t* r, int64_t lo, int64_t hi) {
    return lo + (int64_t)(rng_u64(r) % (uint64_t)(hi - lo + 1));
}

/* ---------------------------------------------------------------- token model */

typedef struct {
    int32_t vocab;
    int32_t markov;      /* 0: plain zipf, 1: order-2 rotated rows */
    double* cdf;         /* [vocab], cdf[v-1] == 1 */
    int32_t* perm;       /* [vocab] */
} model_t;

void* samgen_model_new(int32_t vocab, double zipf_s, int32_t markov, uint64_t seed) {
    model_t* m = (model_t*)calloc(1, sizeof(model_t));
    m->vocab = vocab; m->markov = markov;
    m->cdf = (double*)malloc(sizeof(double) * (size_t)vocab);
    m->perm = (int32_t*)malloc(sizeof(int32_t) * (size_t)vocab);
    double tot = 0.0;
    for (int32_t r = 0; r < vocab; r++) { tot += pow((double)(r + 1), -zipf_s); m->cdf[r] = tot; }
    for (int32_t r = 0; r < vocab; r++) m->cdf[r] /= tot;
    m->cdf[vocab - 1] = 1.0;
    for (int32_t r = 0; r < vocab; r++) m->perm[r] = r;
    rng_t g; rng_init(&g, seed, 0x7065726Dull /* "perm" */);
    for (int32_t r = vocab - 1; r > 0; r--) {
        int32_t j = (int32_t)rng_range(&g, 0, r);
        int32_t tmp = m->perm[r]; m->perm[r] = m->perm[j]; m->perm[j] = tmp;
    }
    return m;
}

void samgen_model_free(void* mp) {
    model_t* m = (model_t*)mp;
    if (!m) return;
    free(m->cdf); free(m->perm); free(m);
}

static inline int32_t draw_rank(const model_t* m, rng_t* g) {
    double u = rng_u01(g);
    int32_t lo = 0, hi = m->vocab - 1;
    while (lo < hi) { int32_t mid = (lo + hi) >> 1; if (m->cdf[mid] > u) hi = mid; else lo = mid + 1; }
    return lo;
}

static inline int32_t fresh_token(const model_t* m, rng_t* g, const int32_t* text, int64_t i) {
    int32_t r = draw_rank(m, g);
    if (m->markov && i >= 2) {
        uint64_t h = fin64(((uint64_t)(uint32_t)text[i - 2] << 32) | (uint32_t)text[i - 1]);
        r = (int32_t)(((uint64_t)r + h % (uint64_t)m->vocab) % (uint64_t)m->vocab);
    }
    return m->perm[r];
}

/* ---------------------------------------------------------------- span-copy text
 * Fill text[start, end) token by token.  A copy, when it starts, reads from one of two sources:
 *   source A ("other"): other[0, other_len)            (e.g. the corpus), chosen with prob p_other
 *   source B ("own")  : text[own_lo, min(own_hi, i))    (what this text holds so far)
 * own_hi < 0 means "up to the current position".  A copy from the own text may run into the
 * positions it is itself writing (the read index stays behind the write index), which yields a
 * periodic continuation; that is allowed.  If the chosen source is empty the token is fresh.
 */
static void fill_text(const model_t* m, rng_t* g, int32_t* text, int64_t start, int64_t end,
                      double f, int32_t lo, int32_t hi,
                      const int32_t* other, int64_t other_len, double p_other,
                      int64_t own_lo, int64_t own_hi) {
    double mean_len = 0.5 * ((double)lo + (double)hi);
    double q = (f <= 0.0) ? 0.0 : f / (f + mean_len * (1.0 - f));
    int64_t i = start;
    while (i < end) {
        int copied = 0;
        if (q > 0.0 && rng_u01(g) < q) {
            int64_t len = rng_range(g, lo, hi);
            int use_other = (other_len > 0) && (rng_u01(g) < p_other);
            if (use_other) {
                int64_t src = rng_range(g, 0, other_len - 1);
                int64_t n = len;
                if (n > other_len - src) n = other_len - src;
                if (n > end - i) n = end - i;
                for (int64_t k = 0; k < n; k++) text[i + k] = other[src + k];
                i += n; copied = (n > 0);
            } else {
                int64_t lim = (own_hi < 0 || own_hi > i) ? i : own_hi;
                if (lim - own_lo > 0) {
                    int64_t src = rng_range(g, own_lo, lim - 1);
                    int64_t n = len;
                    if (own_hi >= 0 && n > lim - src) n = lim - src;   /* bounded source: stay inside it */
                    if (n > end - i) n = end - i;
                    for (int64_t k = 0; k < n; k++) text[i + k] = text[src + k];
                    i += n; copied = (n > 0);
                }
            }
        }
        if (!copied) { text[i] = fresh_token(m, g, text, i); i++; }
    }
}

/* Corpus: n tokens, copies (fraction f, length U[lo,hi]) come from the corpus' own earlier text. */
void samgen_corpus(void* model, int32_t* out, int64_t n, double f, int32_t lo, int32_t hi,
                   uint64_t seed) {
    rng_t g; rng_init(&g, seed, 0x636F7270ull /* "corp" */);
    fill_text((const model_t*)model, &g, out, 0, n, f, lo, hi, NULL, 0, 0.0, 0, -1);
}

/* Multi-document corpus: the text is cut into documents whose lengths (separator included) are
 * U[lo, hi], and the last token of each document is replaced by the separator id `eos` — a corpus
 * of many documents joined into one string by an end-of-sequence token.  Any `eos` the token model
 * itself drew inside a document is replaced by (eos + 1) mod vocab, so the separator occurs at
 * document ends only.  Returns the number of documents. */
int64_t samgen_join_documents(int32_t* corpus, int64_t n, int32_t vocab, int32_t eos, int32_t lo, int32_t hi,
                              uint64_t seed) {
    rng_t g; rng_init(&g, seed, 0x646F6373ull /* "docs" */);
    int64_t docs = 0, i = 0;
    while (i < n) {
        int64_t len = rng_range(&g, lo, hi);
        int64_t end = i + len < n ? i + len : n;
        for (int64_t k = i; k < end - 1; k++) if (corpus[k] == eos) corpus[k] = (eos + 1) % vocab;
        corpus[end - 1] = eos;
        i = end; docs++;
    }
    return docs;
}

/* Sequences: out is [batch, prompt_len + gen_len] row-major.
 * Prompt tokens use (f_prompt, p_other_prompt); generated tokens use (f_gen, p_other_gen).
 * own_prompt_only != 0 restricts own-text copies in the generated part to the prompt. */
void samgen_sequences(void* model, int32_t* out, int32_t batch, int32_t prompt_len, int32_t gen_len,
                      const int32_t* corpus, int64_t corpus_len,
                      double f_prompt, double p_other_prompt,
                      double f_gen, double p_other_gen, int32_t own_prompt_only,
                      int32_t lo, int32_t hi, uint64_t seed) {
    int64_t n = (int64_t)prompt_len + gen_len;
    for (int32_t b = 0; b < batch; b++) {
        rng_t g; rng_init(&g, seed, 0x73657100000000ull + (uint64_t)b);
        int32_t* row = out + (int64_t)b * n;
        fill_text((const model_t*)model, &g, row, 0, prompt_len, f_prompt, lo, hi,
                  corpus, corpus_len, p_other_prompt, 0, -1);
        fill_text((const model_t*)model, &g, row, prompt_len, n, f_gen, lo, hi,
                  corpus, corpus_len, p_other_gen, 0, own_prompt_only ? prompt_len : -1);
    }
}

/* Accepted-token counts per decoding step.
 *   kind 0: uniform on 1..kmax
 *   kind 1: min(kmax, 1 + G), G = number of failures before the first success of a Bernoulli(p)
 * For each sequence, counts are drawn until gen_len tokens are used up; the last one is cut to
 * what remains.  counts is [max_steps, batch] row-major, zero where a sequence has finished.
 * Returns the number of steps the longest sequence needs (<= max_steps), or -1 if max_steps is
 * too small. */
int32_t samgen_schedule(int32_t* counts, int32_t max_steps, int32_t batch, int32_t gen_len,
                        int32_t kind, int32_t kmax, double p, uint64_t seed) {
    int32_t longest = 0;
    memset(counts, 0, sizeof(int32_t) * (size_t)max_steps * (size_t)batch);
    for (int32_t b = 0; b < batch; b++) {
        rng_t g; rng_init(&g, seed, 0x73636800000000ull + (uint64_t)b);
        int32_t left = gen_len, step = 0;
        while (left > 0) {
            int32_t c;
            if (kind == 0) c = (int32_t)rng_range(&g, 1, kmax);
            else { c = 1; while (c < kmax && rng_u01(&g) >= p) c++; }
            if (c > left) c = left;
            if (step >= max_steps) return -1;
            counts[(int64_t)step * batch + b] = c;
            left -= c; step++;
        }
        if (step > longest) longest = step;
    }
    return longest;
}

/* Pack the generated part of each sequence into per-step rows:
 * new_tokens[step, b, 0..counts[step,b]) = the next counts[step,b] tokens of sequence b;
 * the rest of each row is filled with `fill`.  new_tokens is [n_steps, batch, stride]. */
void samgen_pack_steps(const int32_t* seqs, int32_t batch, int32_t prompt_len, int32_t gen_len,
                       const int32_t* counts, int32_t n_steps, int32_t stride, int32_t fill,
                       int32_t* new_tokens) {
    int64_t n = (int64_t)prompt_len + gen_len;
    for (int32_t b = 0; b < batch; b++) {
        int64_t pos = prompt_len;
        for (int32_t s = 0; s < n_steps; s++) {
            int32_t c = counts[(int64_t)s * batch + b];
            int32_t* row = new_tokens + ((int64_t)s * batch + b) * stride;
            for (int32_t k = 0; k < stride; k++) row[k] = (k < c) ? seqs[(int64_t)b * n + pos + k] : fill;
            pos += c;
        }
    }
}
