// Host-side construction of the static suffix automaton in its device layout.
#pragma once
#include <stdint.h>
#include <stddef.h>
#include <vector>
#include "layout.h"

struct SamHostImage {
    SamStaticRec* rec = nullptr;      // mmap'd, n_states used
    size_t rec_map_bytes = 0;
    int64_t n_states = 0;
    int64_t n_transitions = 0;
    int64_t n_hash_edges = 0;
    std::vector<uint32_t> root_row;   // vocab
    std::vector<SamHashEnt> hash;     // buckets * SAM_HASH_BUCKET
    uint32_t hash_mask = 0;
    int32_t hash_max_probe = 0;
    int32_t vocab = 0;
    int64_t n_tokens = 0;
    std::vector<uint32_t> freq;       // n_states, if tree_k > 0
    std::vector<SamTopkEnt> topk;     // open-addressing table, if tree_k > 0
    uint32_t topk_mask = 0;
    int32_t tree_k = 0;
    double build_seconds = 0.0;
    ~SamHostImage();
    SamHostImage() = default;
    SamHostImage(const SamHostImage&) = delete;
    SamHostImage& operator=(const SamHostImage&) = delete;
};

// Build-SAM (Algorithm 3) over corpus[0, n); returns 0 or a negative sam_err_t.
int sam_host_build(const int32_t* corpus, int64_t n, int32_t vocab, double hash_load, int32_t tree_k,
                   SamHostImage* out);
