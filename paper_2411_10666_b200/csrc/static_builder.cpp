// Offline host construction of the static suffix automaton (Build-SAM / Expand, Algorithm 3 of
// SAM-Decoding), written straight into the 32-byte state records of the device layout.
//
// Working representation while building:
//   - the first two transitions of a state live inline in its record;
//   - further transitions live in one global open-addressing table keyed (state, token); the
//     entries of one state are threaded into a list through `next_tok` so a clone can enumerate
//     them; the list head of state s is the entry (s, HEAD_TOK);
//   - the root's transitions are a dense row indexed by token.
// After the last token the records get their F bits (layout.h), and the overflow transitions are
// re-packed into 128-byte buckets for the device.
#include "static_builder.h"
#include "../../include/samdraft.h"

#include <sys/mman.h>
#include <chrono>
#include <algorithm>
#include <cstring>
#include <new>
#include <utility>

namespace {

constexpr uint32_t HEAD_TOK = 0xFFFFFFFEu;

struct OvfEnt { uint32_t state, tok, tgt, next_tok; };

// (state, tok) -> (tgt, next_tok); linear probing; never deletes.
class OvfTable {
public:
    OvfTable() { resize(1u << 16); }
    OvfEnt* find(uint32_t s, uint32_t t) {
        size_t i = slot(s, t);
        for (;;) {
            OvfEnt& e = tab_[i];
            if (e.state == SAM_NONE) return nullptr;
            if (e.state == s && e.tok == t) return &e;
            i = (i + 1) & mask_;
        }
    }
    // key must not be present
    OvfEnt* insert(uint32_t s, uint32_t t, uint32_t tgt, uint32_t next_tok) {
        if ((count_ + 1) * 10 > (mask_ + 1) * 6) grow();
        OvfEnt* e = place(s, t);
        e->state = s; e->tok = t; e->tgt = tgt; e->next_tok = next_tok;
        count_++;
        return e;
    }
    size_t capacity() const { return mask_ + 1; }
    const OvfEnt& at(size_t i) const { return tab_[i]; }
private:
    std::vector<OvfEnt> tab_;
    size_t mask_ = 0, count_ = 0;
    size_t slot(uint32_t s, uint32_t t) const { return (size_t)sam_hash2(s, t) & mask_; }
    OvfEnt* place(uint32_t s, uint32_t t) {
        size_t i = slot(s, t);
        while (tab_[i].state != SAM_NONE) i = (i + 1) & mask_;
        return &tab_[i];
    }
    void resize(size_t n) {
        tab_.assign(n, OvfEnt{SAM_NONE, 0, 0, 0});
        mask_ = n - 1;
    }
    void grow() {
        std::vector<OvfEnt> old;
        old.swap(tab_);
        resize(old.size() * 2);
        for (const OvfEnt& e : old)
            if (e.state != SAM_NONE) *place(e.state, e.tok) = e;
    }
};

class Builder {
public:
    Builder(SamStaticRec* rec, int64_t cap, int32_t vocab)
        : rec_(rec), cap_(cap), root_(vocab, SAM_NONE), clone_((size_t)(cap / 64 + 1), 0) {
        new_state(0, 0);
        rec_[0].link = SAM_NONE;
    }

    bool extend(uint32_t t) {
        n_text_ += 1;
        if (n_states_ + 2 > cap_) return false;
        uint32_t c = new_state(n_text_, n_text_);
        int64_t p = last_;
        uint32_t q = SAM_NONE;
        while (p >= 0) {
            q = find((uint32_t)p, t);
            if (q != SAM_NONE) break;
            add((uint32_t)p, t, c);
            p = up(p);
        }
        if (p < 0) {
            rec_[c].link = 0;
        } else if (rec_[p].len + 1 == rec_[q].len) {
            rec_[c].link = q;
        } else {
            uint32_t cl = new_state(rec_[p].len + 1, rec_[q].min_endpos);
            clone_[cl >> 6] |= 1ull << (cl & 63);
            copy_edges(q, cl);
            rec_[cl].link = rec_[q].link;
            while (p >= 0 && find((uint32_t)p, t) == q) {
                redirect((uint32_t)p, t, cl);
                p = up(p);
            }
            rec_[q].link = cl;
            rec_[c].link = cl;
        }
        last_ = c;
        return true;
    }

    int64_t n_states() const { return n_states_; }
    int64_t n_transitions() const { return n_trans_; }
    int64_t n_ovf() const { return n_ovf_; }
    std::vector<uint32_t>& root() { return root_; }
    const OvfTable& ovf() const { return ovf_; }
    bool is_clone(int64_t s) const { return (clone_[(size_t)(s >> 6)] >> (s & 63)) & 1; }
    // every transition of a state with hashed transitions: the two inline ones and the threaded list
    void edges_of(uint32_t s, std::vector<std::pair<uint32_t, uint32_t>>& out) {
        out.clear();
        const SamStaticRec& r = rec_[s];
        if (r.deg >= 1) out.emplace_back(r.tok0, r.tgt0 & SAM_IDMASK);
        if (r.deg >= 2) out.emplace_back(r.tok1, r.tgt1 & SAM_IDMASK);
        if (r.deg > 2) {
            OvfEnt* h = ovf_.find(s, HEAD_TOK);
            uint32_t t = h ? h->tgt : SAM_NONE;
            while (t != SAM_NONE) { OvfEnt* e = ovf_.find(s, t); out.emplace_back(t, e->tgt & SAM_IDMASK); t = e->next_tok; }
        }
    }

private:
    SamStaticRec* rec_;
    int64_t cap_;
    int64_t n_states_ = 0, n_trans_ = 0, n_ovf_ = 0;
    int32_t n_text_ = 0;
    int64_t last_ = 0;
    std::vector<uint32_t> root_;
    std::vector<uint64_t> clone_;     // bit s: state s was made by cloning
    OvfTable ovf_;

    uint32_t new_state(int32_t len, int32_t endpos) {
        SamStaticRec& r = rec_[n_states_];
        r.len = len; r.link = 0; r.min_endpos = endpos; r.deg = 0;
        r.tok0 = r.tgt0 = r.tok1 = r.tgt1 = 0;
        return (uint32_t)n_states_++;
    }
    int64_t up(int64_t p) const { return p == 0 ? -1 : (int64_t)rec_[p].link; }

    uint32_t find(uint32_t s, uint32_t t) {
        if (s == 0) return root_[t];
        const SamStaticRec& r = rec_[s];
        if (r.deg >= 1 && r.tok0 == t) return r.tgt0;
        if (r.deg >= 2 && r.tok1 == t) return r.tgt1;
        if (r.deg > 2) { OvfEnt* e = ovf_.find(s, t); if (e) return e->tgt; }
        return SAM_NONE;
    }
    void add(uint32_t s, uint32_t t, uint32_t tgt) {
        n_trans_++;
        if (s == 0) { root_[t] = tgt; rec_[0].deg++; return; }
        SamStaticRec& r = rec_[s];
        if (r.deg == 0) { r.tok0 = t; r.tgt0 = tgt; }
        else if (r.deg == 1) { r.tok1 = t; r.tgt1 = tgt; }
        else {
            uint32_t prev_head = SAM_NONE;
            if (r.deg > 2) prev_head = ovf_.find(s, HEAD_TOK)->tgt;
            ovf_.insert(s, t, tgt, prev_head);                      // may rehash: look the head up again
            if (r.deg > 2) ovf_.find(s, HEAD_TOK)->tgt = t;
            else ovf_.insert(s, HEAD_TOK, t, SAM_NONE);
            n_ovf_++;
        }
        r.deg++;
    }
    void redirect(uint32_t s, uint32_t t, uint32_t tgt) {
        if (s == 0) { root_[t] = tgt; return; }
        SamStaticRec& r = rec_[s];
        if (r.deg >= 1 && r.tok0 == t) { r.tgt0 = tgt; return; }
        if (r.deg >= 2 && r.tok1 == t) { r.tgt1 = tgt; return; }
        OvfEnt* e = ovf_.find(s, t);
        if (e) e->tgt = tgt;
    }
    // cl.next = q.next; q is never the root (its length is at least 1)
    void copy_edges(uint32_t q, uint32_t cl) {
        const SamStaticRec rq = rec_[q];
        SamStaticRec& rc = rec_[cl];
        rc.tok0 = rq.tok0; rc.tgt0 = rq.tgt0; rc.tok1 = rq.tok1; rc.tgt1 = rq.tgt1;
        rc.deg = rq.deg < 2 ? rq.deg : 2;
        n_trans_ += rc.deg;
        if (rq.deg > 2) {
            OvfEnt* h = ovf_.find(q, HEAD_TOK);
            uint32_t t = h ? h->tgt : SAM_NONE;
            while (t != SAM_NONE) {
                OvfEnt e = *ovf_.find(q, t);       // copy: add() may rehash
                add(cl, t, e.tgt);
                t = e.next_tok;
            }
        }
    }
};

}  // namespace

SamHostImage::~SamHostImage() {
    if (rec) munmap(rec, rec_map_bytes);
}

int sam_host_build(const int32_t* corpus, int64_t n, int32_t vocab, double hash_load, int32_t tree_k,
                   SamHostImage* out) {
    if (!corpus || n < 1 || vocab < 1 || !out) return SAM_ERR_ARG;
    if (n > (1ll << 30)) return SAM_ERR_LIMIT;          // state ids must fit 31 bits
    if (tree_k < 0 || tree_k > SAM_TOPK_MAX) return SAM_ERR_ARG;
    if (!(hash_load > 0.0) || hash_load > 0.9) hash_load = 0.5;
    auto t0 = std::chrono::steady_clock::now();

    int64_t cap = 2 * n + 2;
    size_t map_bytes = ((size_t)cap * sizeof(SamStaticRec) + 4095) & ~(size_t)4095;
    void* mem = mmap(nullptr, map_bytes, PROT_READ | PROT_WRITE, MAP_PRIVATE | MAP_ANONYMOUS | MAP_NORESERVE, -1, 0);
    if (mem == MAP_FAILED) return SAM_ERR_NOMEM;
    out->rec = (SamStaticRec*)mem;
    out->rec_map_bytes = map_bytes;
    out->vocab = vocab;
    out->n_tokens = n;

    try {
        Builder b(out->rec, cap, vocab);
        for (int64_t i = 0; i < n; i++) {
            int32_t t = corpus[i];
            if (t < 0 || t >= vocab) return SAM_ERR_ARG;
            if (!b.extend((uint32_t)t)) return SAM_ERR_LIMIT;
        }
        out->n_states = b.n_states();
        out->n_transitions = b.n_transitions();
        out->n_hash_edges = b.n_ovf();
        out->root_row.swap(b.root());

        // F bits: which states keep transitions in the hash table
        SamStaticRec* rec = out->rec;
        const int64_t ns = out->n_states;
        std::vector<uint64_t> big((size_t)(ns / 64 + 1), 0);
        for (int64_t s = 1; s < ns; s++)
            if (rec[s].deg > 2) big[(size_t)(s >> 6)] |= 1ull << (s & 63);
        auto flagged = [&](uint32_t s) -> uint32_t {
            return ((big[s >> 6] >> (s & 63)) & 1) ? (s | SAM_FLAG) : s;
        };
        for (int64_t s = 1; s < ns; s++) {
            SamStaticRec& r = rec[s];
            r.link = flagged(r.link);
            if (r.deg >= 1) r.tgt0 = flagged(r.tgt0);
            if (r.deg >= 2) r.tgt1 = flagged(r.tgt1);
        }
        for (uint32_t& e : out->root_row) if (e != SAM_NONE) e = flagged(e);

        // device hash table: 128-byte buckets, linear probing over buckets
        const OvfTable& ovf = b.ovf();
        uint64_t want = (uint64_t)((double)out->n_hash_edges / (hash_load * SAM_HASH_BUCKET)) + 1;
        uint64_t buckets = 1;
        while (buckets < want) buckets <<= 1;
        for (;;) {
            if (buckets > (1ull << 31)) return SAM_ERR_LIMIT;
            out->hash.assign((size_t)buckets * SAM_HASH_BUCKET, SamHashEnt{SAM_NONE, 0, 0, 0});
            std::vector<uint8_t> fill((size_t)buckets, 0);
            uint32_t mask = (uint32_t)(buckets - 1);
            int32_t max_probe = 1;
            bool ok = true;
            for (size_t i = 0; i < ovf.capacity() && ok; i++) {
                const OvfEnt& e = ovf.at(i);
                if (e.state == SAM_NONE || e.tok == HEAD_TOK) continue;
                uint32_t home = sam_hash2(e.state, e.tok) & mask;
                int32_t probe = 0;
                uint32_t bk = home;
                while (fill[bk] == SAM_HASH_BUCKET) {
                    bk = (bk + 1) & mask;
                    if (++probe >= 16) { ok = false; break; }
                }
                if (!ok) break;
                out->hash[(size_t)bk * SAM_HASH_BUCKET + fill[bk]++] = SamHashEnt{e.state, e.tok, flagged(e.tgt), 0};
                if (probe + 1 > max_probe) max_probe = probe + 1;
            }
            if (ok) { out->hash_mask = mask; out->hash_max_probe = max_probe; break; }
            buckets <<= 1;                                 // pathological clustering: halve the load
        }

        // Tree-draft data (Appendix A.1/A.2): freq = occurrences of a state's substrings, 1 for a
        // state made by expansion and 0 for a clone, summed over the suffix-link tree from the
        // longest states down; then the k most frequent successors of every state whose
        // transitions are hashed (freq descending, token ascending).
        out->tree_k = tree_k;
        if (tree_k > 0) {
            std::vector<uint32_t>& freq = out->freq;
            freq.assign((size_t)ns, 0);
            std::vector<uint32_t> start((size_t)n + 2, 0), order((size_t)ns);
            for (int64_t s = 0; s < ns; s++) start[(size_t)rec[s].len + 1]++;
            for (int64_t l = 0; l <= n; l++) start[(size_t)l + 1] += start[(size_t)l];
            for (int64_t s = 0; s < ns; s++) order[start[(size_t)rec[s].len]++] = (uint32_t)s;
            for (int64_t s = 1; s < ns; s++) freq[(size_t)s] = b.is_clone(s) ? 0u : 1u;
            for (int64_t i = ns - 1; i > 0; i--) {
                uint32_t s = order[(size_t)i];
                freq[rec[s].link & SAM_IDMASK] += freq[s];
            }
            int64_t hashed = 0;
            for (int64_t s = 1; s < ns; s++) hashed += rec[s].deg > 2;
            uint64_t cap_t = 16;
            while (cap_t < (uint64_t)hashed * 2) cap_t <<= 1;
            SamTopkEnt empty;
            memset(&empty, 0, sizeof(empty));
            empty.state = SAM_NONE;
            out->topk.assign((size_t)cap_t, empty);
            out->topk_mask = (uint32_t)(cap_t - 1);
            std::vector<std::pair<uint32_t, uint32_t>> ed;
            for (int64_t s = 1; s < ns; s++) {
                if (rec[s].deg <= 2) continue;
                b.edges_of((uint32_t)s, ed);
                size_t keep = std::min<size_t>((size_t)tree_k, ed.size());
                std::partial_sort(ed.begin(), ed.begin() + keep, ed.end(),
                                  [&](const std::pair<uint32_t, uint32_t>& x, const std::pair<uint32_t, uint32_t>& y) {
                                      if (freq[x.second] != freq[y.second]) return freq[x.second] > freq[y.second];
                                      return x.first < y.first;
                                  });
                SamTopkEnt e = empty;
                e.state = (uint32_t)s; e.n = (uint32_t)keep;
                for (size_t j = 0; j < keep; j++) { e.tok[j] = ed[j].first; e.tgt[j] = flagged(ed[j].second); }
                uint32_t at = sam_hash1((uint32_t)s) & out->topk_mask;
                while (out->topk[at].state != SAM_NONE) at = (at + 1) & out->topk_mask;
                out->topk[at] = e;
            }
        }
    } catch (const std::bad_alloc&) {
        return SAM_ERR_NOMEM;
    }
    out->build_seconds = std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count();
    return SAM_OK;
}
