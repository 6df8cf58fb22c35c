// Host-side context of one TreeKV layer (private to the library's .cu files).
#pragma once

#include "common.cuh"

struct treekv_ctx {
    treekv::CacheView cv;
    treekv::PrefillScratch ps;
    CUtensorMap tmK, tmV;  // 2-D maps over the K and V slabs (rows x head_dim), box 128 rows x 64 channels (bf16, d=128)
    bool has_tma;
    treekv_dtype dt;
    int max_chunk;
    int G;
    size_t elem;
    // staging for the *_host entry points (sized for a chunk)
    void *st_q, *st_k, *st_v, *st_out;
    // options
    int opt_decode_split;
    int opt_prefill_path;
    int opt_decode_path;
    int opt_prefill_append;
    int sm_count;
    int device;  // ordinal of the device that was current at creation: the workspace lives there
    // host-side record
    int64_t n_seen[treekv::kMaxBatch];
    uint64_t evictions;
    uint64_t launches;
    int last_cuda_error;
};
