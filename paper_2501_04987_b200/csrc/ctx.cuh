// Host-side context of one TreeKV layer (private to the library's .cu files).
#pragma once

#include "common.cuh"

struct treekv_ctx {
    treekv::CacheView cv;
    treekv::PrefillScratch ps;
    CUtensorMap tmK, tmV;  // 2-D maps over the K and V slabs (rows x head_dim), box 128 rows x 64 channels (bf16, d=128)
    CUtensorMap tmKrot;    // the same over k_rot, the slab of keys encoded at their cache slots (in-cache positions)
    void* k_rot;
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
    int opt_prefill_key_split;
    // eviction stream (TREEKV_OPT_EVICTION_STREAM): the score update + eviction kernel of a chunk runs on `side`, after
    // the chunk's attention (ev_attn), and everything enqueued later for this context waits for it (ev_state)
    cudaStream_t side;
    cudaEvent_t ev_attn, ev_state;
    bool side_pending;  // a kernel on `side` may still be running that the caller's stream has not been told to wait for
    int sm_count;
    long attn_blocks;  // thread blocks of the last chunk-attention launch (0: a kernel whose grid is not counted)
    int device;  // ordinal of the device that was current at creation: the workspace lives there
    // host-side record
    int64_t n_seen[treekv::kMaxBatch];
    uint64_t evictions;
    uint64_t launches;
    int last_cuda_error;
};

namespace treekv {
// chunk score update + eviction as blocks of 1024 threads, at most max_blocks of them (0 = one per unit): state.cu
cudaError_t launch_chunk_update_evict_beside(const CacheView& cv, treekv_dtype dt, const PrefillScratch& ps,
                                             const ChunkLens& lens, int max_blocks, cudaStream_t stream);
// Orders `stream` behind the context's eviction stream, if a kernel there has not been waited for yet.  Every entry
// point that enqueues work on the cache calls this first.
inline cudaError_t join_eviction_stream(treekv_ctx* ctx, cudaStream_t stream) {
    if (!ctx->side_pending) return cudaSuccess;
    const cudaError_t e = cudaStreamWaitEvent(stream, ctx->ev_state, 0);
    if (e == cudaSuccess) ctx->side_pending = false;
    return e;
}
}  // namespace treekv
