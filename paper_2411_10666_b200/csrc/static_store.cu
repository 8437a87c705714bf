// Static automaton on the device: upload of a host-built image, file save / load, inspection.
#include "common.h"
#include "static_builder.h"

#include <cstdio>
#include <cstring>
#include <vector>
#include <new>

namespace {

thread_local int g_last_cuda = 0;

constexpr uint64_t FILE_MAGIC = 0x314D41534D415353ull;   // "SSAMSAM1"
constexpr uint32_t FILE_VERSION = 2;
constexpr size_t CORPUS_PAD_TOKENS = 64;                  // vector reads past the end stay in bounds

struct FileHeader {
    uint64_t magic;
    uint32_t version, vocab;
    int64_t n_tokens, n_states, n_transitions, n_hash_edges, hash_buckets;
    int32_t hash_max_probe, pad;
    uint64_t len_rec, len_root, len_hash, len_corpus, len_freq, len_topk;
    int32_t tree_k, pad2;
    uint64_t checksum;
};

// 64-bit FNV-1a taken over 8-byte words (all sections are multiples of 8 bytes)
inline uint64_t fnv_words(uint64_t h, const void* data, size_t bytes) {
    const uint64_t* w = (const uint64_t*)data;
    for (size_t i = 0; i < bytes / 8; i++) { h ^= w[i]; h *= 0x100000001B3ull; }
    return h;
}

void layout_sections(sam_static* st) {
    size_t off = 0;
    st->off_rec = off;    off = sam_align_up(off + st->len_rec, 256);
    st->off_root = off;   off = sam_align_up(off + st->len_root, 256);
    st->off_hash = off;   off = sam_align_up(off + st->len_hash, 256);
    st->off_corpus = off; off = sam_align_up(off + st->len_corpus, 256);
    st->off_freq = off;   off = sam_align_up(off + st->len_freq, 256);
    st->off_topk = off;   off = sam_align_up(off + st->len_topk, 256);
    // derived on the device after every upload, never stored in a file: position -> prefix state
    st->len_pstate = sam_align_up(((size_t)st->info.n_tokens + CORPUS_PAD_TOKENS) * 4, 8);
    st->off_pstate = off; off = sam_align_up(off + st->len_pstate, 256);
    st->dev_bytes = off;
}

void make_view(sam_static* st) {
    char* base = (char*)st->dev_base;
    st->view.rec = (const uint4*)(base + st->off_rec);
    st->view.root_row = (const uint32_t*)(base + st->off_root);
    st->view.hash = (const uint4*)(base + st->off_hash);
    st->view.corpus = (const int32_t*)(base + st->off_corpus);
    st->view.hash_mask = (uint32_t)(st->info.hash_buckets - 1);
    st->view.hash_max_probe = st->info.hash_max_probe;
    st->view.vocab = st->info.vocab;
    st->view.n_tokens = st->info.n_tokens;
    st->view.n_states = st->info.n_states;
    st->view.freq = (const uint32_t*)(base + st->off_freq);
    st->view.topk = (const uint4*)(base + st->off_topk);
    st->view.topk_mask = st->len_topk ? (uint32_t)(st->len_topk / sizeof(SamTopkEnt) - 1) : 0;
    st->view.tree_k = st->info.tree_topk;
    st->view.pstate = (const uint32_t*)(base + st->off_pstate);
}

// pstate[i] = id | F of the state Build-SAM created for corpus token i, the state of the whole prefix
// of length i + 1.  These are the states that are not clones: exactly those with len == min_endpos.
__global__ void derive_pstate_kernel(const uint4* rec, int64_t n_states, uint32_t* pstate, int64_t n_tokens) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t s = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; s < n_states; s += stride) {
        const uint4 a = rec[2 * s];
        if (s > 0 && a.x == a.z && a.x >= 1 && (int64_t)a.x <= n_tokens)
            pstate[a.x - 1] = (uint32_t)s | (a.w > 2 ? SAM_FLAG : 0u);
    }
}

int derive_pstate(sam_static* st) {
    int sms = 0;
    cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, st->device);
    if (e != cudaSuccess || sms < 1) { sam_set_cuda_error(e); return SAM_ERR_CUDA; }
    derive_pstate_kernel<<<sms * 8, 256>>>(st->view.rec, st->info.n_states,
                                           (uint32_t*)((char*)st->dev_base + st->off_pstate), st->info.n_tokens);
    e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { sam_set_cuda_error(e); return SAM_ERR_CUDA; }
    return SAM_OK;
}

// collect the transitions of one state: inline ones, hashed ones, or the root row
__global__ void collect_edges_kernel(SamStaticView S, uint32_t state, int32_t* toks, int32_t* tgts,
                                     int32_t max_edges, int32_t* count) {
    size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    size_t stride = (size_t)gridDim.x * blockDim.x;
    if (state == 0) {
        for (size_t t = i; t < (size_t)S.vocab; t += stride) {
            uint32_t e = S.root_row[t];
            if (e != SAM_NONE) {
                int k = atomicAdd(count, 1);
                if (k < max_edges) { toks[k] = (int32_t)t; tgts[k] = (int32_t)(e & SAM_IDMASK); }
            }
        }
        return;
    }
    size_t n_ent = ((size_t)S.hash_mask + 1) * SAM_HASH_BUCKET;
    for (size_t e = i; e < n_ent; e += stride) {
        uint4 v = S.hash[e];
        if (v.x == state) {
            int k = atomicAdd(count, 1);
            if (k < max_edges) { toks[k] = (int32_t)v.y; tgts[k] = (int32_t)(v.z & SAM_IDMASK); }
        }
    }
}

}  // namespace

void sam_set_cuda_error(cudaError_t e) { g_last_cuda = (int)e; }

extern "C" int sam_last_cuda_error(void) { return g_last_cuda; }

extern "C" const char* sam_version(void) { return "samdraft 0.1 (sm_100a)"; }

extern "C" const char* sam_strerror(int err) {
    switch (err) {
        case SAM_OK: return "ok";
        case SAM_ERR_ARG: return "invalid argument";
        case SAM_ERR_CUDA: return "CUDA runtime call failed";
        case SAM_ERR_NOMEM: return "out of memory";
        case SAM_ERR_WORKSPACE: return "workspace too small or misaligned";
        case SAM_ERR_IO: return "file input/output failed";
        case SAM_ERR_FORMAT: return "not a static-automaton image or checksum mismatch";
        case SAM_ERR_LIMIT: return "size exceeds what the layout can index";
        case SAM_ERR_NO_DEVICE: return "no usable CUDA device";
        case SAM_ERR_UNSUPPORTED: return "this build of the library lacks the feature";
        default: return "unknown error";
    }
}

static int check_device(int device) {
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || n < 1) { cudaGetLastError(); return SAM_ERR_NO_DEVICE; }
    if (device < 0 || device >= n) return SAM_ERR_ARG;
    return SAM_OK;
}

extern "C" int sam_build_static(const int32_t* corpus_host, int64_t n_tokens, int32_t vocab, int device,
                                const sam_build_opts_t* opts, sam_static_t** out) {
    if (!out) return SAM_ERR_ARG;
    *out = nullptr;
    if (!corpus_host || n_tokens < 1 || vocab < 1) return SAM_ERR_ARG;
    if (opts && (opts->keep_host_copy != 0 || opts->tree_topk < 0 || opts->tree_topk > SAM_TOPK_MAX)) return SAM_ERR_ARG;
    if (n_tokens > (1ll << 30)) return SAM_ERR_LIMIT;
    int rc = check_device(device);
    if (rc) return rc;

    SamHostImage img;
    rc = sam_host_build(corpus_host, n_tokens, vocab, opts ? opts->hash_load : 0.0, opts ? opts->tree_topk : 0, &img);
    if (rc) return rc;

    sam_static* st = new (std::nothrow) sam_static();
    if (!st) return SAM_ERR_NOMEM;
    memset(st, 0, sizeof(*st));
    st->device = device;
    st->info.n_tokens = n_tokens;
    st->info.n_states = img.n_states;
    st->info.n_transitions = img.n_transitions;
    st->info.n_hash_edges = img.n_hash_edges;
    st->info.hash_buckets = (int64_t)img.hash_mask + 1;
    st->info.hash_max_probe = img.hash_max_probe;
    st->info.vocab = vocab;
    st->info.build_seconds = img.build_seconds;
    st->len_rec = (size_t)img.n_states * sizeof(SamStaticRec);
    st->len_root = sam_align_up((size_t)vocab * 4, 8);
    st->len_hash = img.hash.size() * sizeof(SamHashEnt);
    st->len_corpus = sam_align_up(((size_t)n_tokens + CORPUS_PAD_TOKENS) * 4, 8);
    st->info.tree_topk = img.tree_k;
    st->len_freq = sam_align_up(img.freq.size() * 4, 8);
    st->len_topk = img.topk.size() * sizeof(SamTopkEnt);
    layout_sections(st);
    st->info.device_bytes = st->dev_bytes;

    SamDeviceGuard guard(device);
    if (!guard.ok) { delete st; return SAM_ERR_CUDA; }
    cudaError_t e = cudaMalloc(&st->dev_base, st->dev_bytes);
    if (e != cudaSuccess) { sam_set_cuda_error(e); cudaGetLastError(); delete st; return SAM_ERR_NOMEM; }
    char* base = (char*)st->dev_base;
    e = cudaMemset(base, 0, st->dev_bytes);
    if (e == cudaSuccess) e = cudaMemcpy(base + st->off_rec, img.rec, st->len_rec, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(base + st->off_root, img.root_row.data(), (size_t)vocab * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(base + st->off_hash, img.hash.data(), st->len_hash, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(base + st->off_corpus, corpus_host, (size_t)n_tokens * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && !img.freq.empty()) e = cudaMemcpy(base + st->off_freq, img.freq.data(), img.freq.size() * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && !img.topk.empty()) e = cudaMemcpy(base + st->off_topk, img.topk.data(), st->len_topk, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { sam_set_cuda_error(e); cudaFree(st->dev_base); delete st; return SAM_ERR_CUDA; }
    make_view(st);
    if (derive_pstate(st) != SAM_OK) { cudaFree(st->dev_base); delete st; return SAM_ERR_CUDA; }
    *out = st;
    return SAM_OK;
}

extern "C" void sam_static_destroy(sam_static_t* st) {
    if (!st) return;
    SamDeviceGuard guard(st->device);
    if (st->dev_base) cudaFree(st->dev_base);
    delete st;
}

extern "C" int sam_static_info(const sam_static_t* st, sam_static_info_t* out) {
    if (!st || !out) return SAM_ERR_ARG;
    *out = st->info;
    return SAM_OK;
}

extern "C" int sam_static_save(const sam_static_t* st, const char* path) {
    if (!st || !path) return SAM_ERR_ARG;
    SamDeviceGuard guard(st->device);
    if (!guard.ok) return SAM_ERR_CUDA;
    FILE* f = fopen(path, "wb");
    if (!f) return SAM_ERR_IO;
    FileHeader h;
    memset(&h, 0, sizeof(h));
    h.magic = FILE_MAGIC; h.version = FILE_VERSION; h.vocab = (uint32_t)st->info.vocab;
    h.n_tokens = st->info.n_tokens; h.n_states = st->info.n_states;
    h.n_transitions = st->info.n_transitions; h.n_hash_edges = st->info.n_hash_edges;
    h.hash_buckets = st->info.hash_buckets; h.hash_max_probe = st->info.hash_max_probe;
    h.len_rec = st->len_rec; h.len_root = st->len_root; h.len_hash = st->len_hash; h.len_corpus = st->len_corpus;
    h.len_freq = st->len_freq; h.len_topk = st->len_topk; h.tree_k = st->info.tree_topk;
    int rc = SAM_OK;
    if (fwrite(&h, sizeof(h), 1, f) != 1) rc = SAM_ERR_IO;
    const size_t CHUNK = 64u << 20;
    std::vector<char> buf;
    try { buf.resize(CHUNK); } catch (const std::bad_alloc&) { fclose(f); return SAM_ERR_NOMEM; }
    uint64_t sum = 0xCBF29CE484222325ull;
    const size_t offs[6] = {st->off_rec, st->off_root, st->off_hash, st->off_corpus, st->off_freq, st->off_topk};
    const size_t lens[6] = {st->len_rec, st->len_root, st->len_hash, st->len_corpus, st->len_freq, st->len_topk};
    for (int s = 0; s < 6 && rc == SAM_OK; s++) {
        for (size_t done = 0; done < lens[s] && rc == SAM_OK; done += CHUNK) {
            size_t n = lens[s] - done < CHUNK ? lens[s] - done : CHUNK;
            cudaError_t e = cudaMemcpy(buf.data(), (char*)st->dev_base + offs[s] + done, n, cudaMemcpyDeviceToHost);
            if (e != cudaSuccess) { sam_set_cuda_error(e); rc = SAM_ERR_CUDA; break; }
            sum = fnv_words(sum, buf.data(), n);
            if (fwrite(buf.data(), 1, n, f) != n) rc = SAM_ERR_IO;
        }
    }
    if (rc == SAM_OK) {
        h.checksum = sum;
        if (fseek(f, 0, SEEK_SET) != 0 || fwrite(&h, sizeof(h), 1, f) != 1) rc = SAM_ERR_IO;
    }
    if (fclose(f) != 0 && rc == SAM_OK) rc = SAM_ERR_IO;
    return rc;
}

extern "C" int sam_static_load(const char* path, int device, sam_static_t** out) {
    if (!out) return SAM_ERR_ARG;
    *out = nullptr;
    if (!path) return SAM_ERR_ARG;
    int rc = check_device(device);
    if (rc) return rc;
    FILE* f = fopen(path, "rb");
    if (!f) return SAM_ERR_IO;
    FileHeader h;
    if (fread(&h, sizeof(h), 1, f) != 1) { fclose(f); return SAM_ERR_FORMAT; }
    bool sane = h.magic == FILE_MAGIC && h.version == FILE_VERSION && h.n_tokens >= 1 && h.n_states >= 1 &&
                h.hash_buckets >= 1 && (h.hash_buckets & (h.hash_buckets - 1)) == 0 &&
                h.len_rec == (uint64_t)h.n_states * sizeof(SamStaticRec) &&
                h.len_root == sam_align_up((size_t)h.vocab * 4, 8) &&
                h.len_hash == (uint64_t)h.hash_buckets * SAM_HASH_BUCKET * sizeof(SamHashEnt) &&
                h.len_corpus == sam_align_up(((size_t)h.n_tokens + CORPUS_PAD_TOKENS) * 4, 8) &&
                h.tree_k >= 0 && h.tree_k <= SAM_TOPK_MAX &&
                (h.tree_k == 0 ? (h.len_freq == 0 && h.len_topk == 0)
                               : (h.len_freq == sam_align_up((size_t)h.n_states * 4, 8) && h.len_topk >= sizeof(SamTopkEnt) &&
                                  h.len_topk % sizeof(SamTopkEnt) == 0 &&
                                  ((h.len_topk / sizeof(SamTopkEnt)) & (h.len_topk / sizeof(SamTopkEnt) - 1)) == 0));
    if (!sane) { fclose(f); return SAM_ERR_FORMAT; }

    sam_static* st = new (std::nothrow) sam_static();
    if (!st) { fclose(f); return SAM_ERR_NOMEM; }
    memset(st, 0, sizeof(*st));
    st->device = device;
    st->info.n_tokens = h.n_tokens; st->info.n_states = h.n_states; st->info.n_transitions = h.n_transitions;
    st->info.n_hash_edges = h.n_hash_edges; st->info.hash_buckets = h.hash_buckets;
    st->info.hash_max_probe = h.hash_max_probe; st->info.vocab = (int32_t)h.vocab;
    st->len_rec = h.len_rec; st->len_root = h.len_root; st->len_hash = h.len_hash; st->len_corpus = h.len_corpus;
    st->len_freq = h.len_freq; st->len_topk = h.len_topk; st->info.tree_topk = h.tree_k;
    layout_sections(st);
    st->info.device_bytes = st->dev_bytes;

    SamDeviceGuard guard(device);
    if (!guard.ok) { delete st; fclose(f); return SAM_ERR_CUDA; }
    cudaError_t e = cudaMalloc(&st->dev_base, st->dev_bytes);
    if (e != cudaSuccess) { sam_set_cuda_error(e); cudaGetLastError(); delete st; fclose(f); return SAM_ERR_NOMEM; }
    cudaMemset(st->dev_base, 0, st->dev_bytes);
    const size_t CHUNK = 64u << 20;
    std::vector<char> buf;
    try { buf.resize(CHUNK); } catch (const std::bad_alloc&) { cudaFree(st->dev_base); delete st; fclose(f); return SAM_ERR_NOMEM; }
    uint64_t sum = 0xCBF29CE484222325ull;
    const size_t offs[6] = {st->off_rec, st->off_root, st->off_hash, st->off_corpus, st->off_freq, st->off_topk};
    const size_t lens[6] = {st->len_rec, st->len_root, st->len_hash, st->len_corpus, st->len_freq, st->len_topk};
    rc = SAM_OK;
    for (int s = 0; s < 6 && rc == SAM_OK; s++) {
        for (size_t done = 0; done < lens[s] && rc == SAM_OK; done += CHUNK) {
            size_t n = lens[s] - done < CHUNK ? lens[s] - done : CHUNK;
            if (fread(buf.data(), 1, n, f) != n) { rc = SAM_ERR_FORMAT; break; }
            sum = fnv_words(sum, buf.data(), n);
            e = cudaMemcpy((char*)st->dev_base + offs[s] + done, buf.data(), n, cudaMemcpyHostToDevice);
            if (e != cudaSuccess) { sam_set_cuda_error(e); rc = SAM_ERR_CUDA; }
        }
    }
    fclose(f);
    if (rc == SAM_OK && sum != h.checksum) rc = SAM_ERR_FORMAT;
    if (rc != SAM_OK) { cudaFree(st->dev_base); delete st; return rc; }
    make_view(st);
    if (derive_pstate(st) != SAM_OK) { cudaFree(st->dev_base); delete st; return SAM_ERR_CUDA; }
    *out = st;
    return SAM_OK;
}

extern "C" int sam_static_state(const sam_static_t* st, int64_t state, int32_t* length, int32_t* link,
                                int32_t* min_endpos, int32_t* n_edges,
                                int32_t* next_tokens, int32_t* next_targets, int32_t max_edges) {
    if (!st || state < 0 || state >= st->info.n_states || max_edges < 0) return SAM_ERR_ARG;
    if (max_edges > 0 && (!next_tokens || !next_targets)) return SAM_ERR_ARG;
    SamDeviceGuard guard(st->device);
    if (!guard.ok) return SAM_ERR_CUDA;
    SamStaticRec r;
    SAM_CUDA(cudaMemcpy(&r, (const char*)st->view.rec + (size_t)state * sizeof(r), sizeof(r), cudaMemcpyDeviceToHost));
    if (length) *length = r.len;
    if (link) *link = state == 0 ? -1 : (int32_t)(r.link & SAM_IDMASK);
    if (min_endpos) *min_endpos = r.min_endpos;
    if (n_edges) *n_edges = (int32_t)r.deg;
    int32_t k = 0;
    if (state != 0) {
        if (r.deg >= 1 && k < max_edges) { next_tokens[k] = (int32_t)r.tok0; next_targets[k] = (int32_t)(r.tgt0 & SAM_IDMASK); k++; }
        if (r.deg >= 2 && k < max_edges) { next_tokens[k] = (int32_t)r.tok1; next_targets[k] = (int32_t)(r.tgt1 & SAM_IDMASK); k++; }
    }
    if ((state == 0 || r.deg > 2) && max_edges > k) {
        int32_t room = max_edges - k;
        int32_t *d_tok = nullptr, *d_tgt = nullptr, *d_cnt = nullptr;
        SAM_CUDA(cudaMalloc(&d_tok, (size_t)room * 4));
        cudaError_t e = cudaMalloc(&d_tgt, (size_t)room * 4);
        if (e == cudaSuccess) e = cudaMalloc(&d_cnt, 4);
        if (e == cudaSuccess) e = cudaMemset(d_cnt, 0, 4);
        if (e == cudaSuccess) {
            collect_edges_kernel<<<592, 256>>>(st->view, (uint32_t)state, d_tok, d_tgt, room, d_cnt);
            e = cudaGetLastError();
        }
        int32_t got = 0;
        if (e == cudaSuccess) e = cudaMemcpy(&got, d_cnt, 4, cudaMemcpyDeviceToHost);
        if (got > room) got = room;
        if (e == cudaSuccess && got > 0) e = cudaMemcpy(next_tokens + k, d_tok, (size_t)got * 4, cudaMemcpyDeviceToHost);
        if (e == cudaSuccess && got > 0) e = cudaMemcpy(next_targets + k, d_tgt, (size_t)got * 4, cudaMemcpyDeviceToHost);
        cudaFree(d_tok); cudaFree(d_tgt); cudaFree(d_cnt);
        if (e != cudaSuccess) { sam_set_cuda_error(e); return SAM_ERR_CUDA; }
    }
    return SAM_OK;
}

extern "C" int sam_static_tables(const sam_static_t* st, int32_t* length, int32_t* link, int32_t* min_endpos,
                                 int32_t* deg, int64_t max_states) {
    if (!st || !length || !link || !min_endpos || !deg || max_states < 0) return SAM_ERR_ARG;
    SamDeviceGuard guard(st->device);
    if (!guard.ok) return SAM_ERR_CUDA;
    int64_t n = st->info.n_states < max_states ? st->info.n_states : max_states;
    const int64_t CH = 1 << 20;
    std::vector<SamStaticRec> buf;
    try { buf.resize((size_t)(n < CH ? n : CH)); } catch (const std::bad_alloc&) { return SAM_ERR_NOMEM; }
    for (int64_t done = 0; done < n; done += CH) {
        int64_t m = n - done < CH ? n - done : CH;
        SAM_CUDA(cudaMemcpy(buf.data(), (const char*)st->view.rec + (size_t)done * sizeof(SamStaticRec),
                            (size_t)m * sizeof(SamStaticRec), cudaMemcpyDeviceToHost));
        for (int64_t i = 0; i < m; i++) {
            length[done + i] = buf[i].len;
            link[done + i] = (done + i == 0) ? -1 : (int32_t)(buf[i].link & SAM_IDMASK);
            min_endpos[done + i] = buf[i].min_endpos;
            deg[done + i] = (int32_t)buf[i].deg;
        }
    }
    return SAM_OK;
}

// Host-only: build the image and decode it back into flat tables, reading the very sections the
// device would get (inline transitions, root row, hash buckets) and checking the F bits.
extern "C" int sam_build_static_tables(const int32_t* corpus_host, int64_t n_tokens, int32_t vocab,
                                       int64_t* n_states, int64_t* n_transitions, int32_t* hash_max_probe,
                                       int32_t* length, int32_t* link, int32_t* min_endpos, int32_t* deg,
                                       int64_t max_states,
                                       int32_t* edge_src, int32_t* edge_tok, int32_t* edge_tgt, int64_t max_edges) {
    if (!n_states || !n_transitions) return SAM_ERR_ARG;
    SamHostImage img;
    int rc = sam_host_build(corpus_host, n_tokens, vocab, 0.0, 0, &img);
    if (rc) return rc;
    *n_states = img.n_states;
    *n_transitions = img.n_transitions;
    if (hash_max_probe) *hash_max_probe = img.hash_max_probe;
    auto flag_ok = [&](uint32_t ref) {
        uint32_t s = ref & SAM_IDMASK;
        return s < (uint64_t)img.n_states && ((ref >> 31) != 0) == (s != 0 && img.rec[s].deg > 2);
    };
    int64_t k = 0;
    auto emit = [&](uint32_t src, uint32_t tok, uint32_t ref) {
        if (!flag_ok(ref)) rc = SAM_ERR_FORMAT;
        if (k < max_edges && edge_src && edge_tok && edge_tgt) {
            edge_src[k] = (int32_t)src; edge_tok[k] = (int32_t)tok; edge_tgt[k] = (int32_t)(ref & SAM_IDMASK);
        }
        k++;
    };
    for (int64_t s = 0; s < img.n_states; s++) {
        const SamStaticRec& r = img.rec[s];
        if (s < max_states && length && link && min_endpos && deg) {
            length[s] = r.len; link[s] = s == 0 ? -1 : (int32_t)(r.link & SAM_IDMASK);
            min_endpos[s] = r.min_endpos; deg[s] = (int32_t)r.deg;
        }
        if (s == 0) continue;
        if (!flag_ok(r.link)) rc = SAM_ERR_FORMAT;
        if (r.deg >= 1) emit((uint32_t)s, r.tok0, r.tgt0);
        if (r.deg >= 2) emit((uint32_t)s, r.tok1, r.tgt1);
    }
    for (int32_t t = 0; t < vocab; t++)
        if (img.root_row[(size_t)t] != SAM_NONE) emit(0, (uint32_t)t, img.root_row[(size_t)t]);
    for (size_t i = 0; i < img.hash.size(); i++) {
        const SamHashEnt& e = img.hash[i];
        if (e.state == SAM_NONE) continue;
        // the entry must be reachable from its home bucket within hash_max_probe buckets
        uint32_t home = sam_hash2(e.state, e.tok) & img.hash_mask;
        uint32_t at = (uint32_t)(i / SAM_HASH_BUCKET);
        uint32_t dist = (at - home) & img.hash_mask;
        if ((int32_t)dist >= img.hash_max_probe) rc = SAM_ERR_FORMAT;
        for (uint32_t d = 0; d < dist; d++) {                 // every bucket before it must be full
            size_t bk = (size_t)((home + d) & img.hash_mask) * SAM_HASH_BUCKET;
            for (int j = 0; j < SAM_HASH_BUCKET; j++) if (img.hash[bk + j].state == SAM_NONE) rc = SAM_ERR_FORMAT;
        }
        emit(e.state, e.tok, e.tgt);
    }
    if (k != img.n_transitions) rc = SAM_ERR_FORMAT;
    return rc;
}

extern "C" int sam_static_freq(const sam_static_t* st, uint32_t* freq_host, int64_t max_states) {
    if (!st || !freq_host || max_states < 0) return SAM_ERR_ARG;
    if (st->info.tree_topk <= 0) return SAM_ERR_ARG;
    SamDeviceGuard guard(st->device);
    if (!guard.ok) return SAM_ERR_CUDA;
    int64_t n = st->info.n_states < max_states ? st->info.n_states : max_states;
    SAM_CUDA(cudaMemcpy(freq_host, st->view.freq, (size_t)n * 4, cudaMemcpyDeviceToHost));
    return SAM_OK;
}
