/*
 * treekv.h -- C ABI of the TreeKV cache library for NVIDIA B200 (sm_100a).
 *
 * TreeKV (arXiv 2501.04987) keeps a key/value cache of fixed size c per
 * attention head.  Each step appends the new token, attends over the cache
 * (Section 3.1: a = SoftMax(q K^T / sqrt(d)), o = a V), accumulates for every
 * cached token the attention weight it received (Algorithm 1: S <- S + a,
 * C <- C + 1, importance = S / C), and once the cache is longer than c evicts
 * the lower-scored member of the adjacent pair {idx, idx+1}, where idx cycles
 * 1..c (Section 4.1 "Eviction Scope").  Old context thins out like a binary
 * tree; recent context stays dense.
 *
 * Conventions shared by every entry point
 *   - One treekv_ctx is one attention layer for `batch` sequences.  A layer
 *     stack is an array of contexts driven in layer order.
 *   - "dev" pointers are device memory, "host" pointers are host memory.  The
 *     caller owns every buffer it passes, including the workspace, for the
 *     life of the context.  The library allocates no device memory, never
 *     frees caller memory and never synchronises the stream unless an entry
 *     point says so: a call only enqueues work on `stream` (a cudaStream_t
 *     passed as void*, NULL = the default stream).
 *   - Tensors are contiguous, 16-byte aligned, element type = the context's
 *     dtype (fp32 or bf16).  q and k arrive with any position encoding already
 *     applied; the library is position-agnostic (unless treekv_set_positions
 *     switches in-cache positions on) and records for every cached token its
 *     0-based stream index.
 *   - Grouped-query attention: query head h uses KV head h / (n_heads /
 *     n_kv_heads); the weight a cached token receives in a step is the mean
 *     over the query heads of its group (equal to Algorithm 1 when the group
 *     size is 1).
 *   - Calls on one context execute in the order in which they were made when they are made on one stream;
 *     the kernels of consecutive calls may overlap at their edges (programmatic dependent launch) and order
 *     their own memory accesses.  Calls made on different streams, or from several host threads at once,
 *     for the same context are the caller's to order.
 *   - Errors are returned, never thrown or trapped.  Argument and state errors
 *     are detected before anything is enqueued.  Asynchronous CUDA errors
 *     surface on a later call or in treekv_get_stats.
 */
#ifndef TREEKV_H
#define TREEKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct treekv_ctx treekv_ctx; /* opaque, host-side; owned by the library */

typedef enum {
    TREEKV_OK = 0,
    TREEKV_ERR_INVALID_ARG = 1, /* null pointer, misaligned buffer, length out of range */
    TREEKV_ERR_BAD_STATE = 2,   /* call not valid in the context's current state */
    TREEKV_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small */
    TREEKV_ERR_UNSUPPORTED = 4, /* shape or dtype outside what the kernels cover */
    TREEKV_ERR_CUDA = 5,        /* a CUDA runtime call failed; see treekv_stats.last_cuda_error */
    TREEKV_ERR_TIMEOUT = 6      /* a bounded device-side wait gave up; the context must be reset */
} treekv_status;

typedef enum { TREEKV_F32 = 0, TREEKV_BF16 = 1 } treekv_dtype;

/* Eviction rule.  SCORES is Algorithm 1.  KEEP_LEFT is the ablation of Section 5.4 (always keep the
 * left token of the scope).  EVICT_LEFT is what an exact tie does under Algorithm 1's strict '>'.
 * The two score-free rules make the retained set a function of the schedule alone.  ACCUMULATED is Algorithm 1
 * with the accumulated attention weight S in place of the averaged weight S / C - a criterion Section 4.1
 * ("Importance Score") reports as tried and found worse than the average; in the one-shot prefill a block's
 * importance is then the mean of its tokens' S.  treekv_scores reports S / C under every rule. */
typedef enum {
    TREEKV_RULE_SCORES = 0,
    TREEKV_RULE_KEEP_LEFT = 1,
    TREEKV_RULE_EVICT_LEFT = 2,
    TREEKV_RULE_ACCUMULATED = 3
} treekv_rule;

/* Options for treekv_set_option. */
typedef enum {
    TREEKV_OPT_DECODE_SPLIT = 0, /* thread blocks per (sequence, KV head) in decode: 0 = automatic, else 1,2,4,8 */
    TREEKV_OPT_PREFILL_PATH = 1, /* 0 = automatic, 1 = CUDA-core kernel, 2 / 3 = tcgen05 tensor-core kernel with 128 / 256
                                    query rows per thread block (bf16, head_dim 128) */
    TREEKV_OPT_DECODE_PATH = 2,  /* 0 = automatic, 1 = CUDA-core kernel, 2 = cp.async + mma.sync kernel (bf16 only) */
    TREEKV_OPT_PREFILL_APPEND = 3, /* 0 = automatic: the tensor-core prefill kernels read the chunk's own keys and values
                                    from dev_k / dev_v and append them to the cache themselves whenever every sequence's
                                    chunk length is a multiple of 128 (no separate append kernel); 1 = always append with
                                    a kernel of its own before the attention.  Same result either way. */
    TREEKV_OPT_PREFILL_KEY_SPLIT = 5, /* two-tile tensor-core prefill kernel: which tile pairs (256 query rows) are given to a pair
                                    of thread blocks that halve the pair's key tiles and exchange row statistics and
                                    partial outputs.  0 = automatic:
                                    the pairs of a last, at most half-full wave; 1 = none; 2 = every pair; 3 = the
                                    automatic rule for a machine of four SMs (for tests) */
    TREEKV_OPT_EVICTION_STREAM = 4 /* 0 (default) = every kernel of a call runs on the caller's stream.  1 = the last
                                    kernel of treekv_prefill_chunk (score update + eviction + compaction, which only
                                    touches the workspace) runs on a stream the context owns, behind the chunk's
                                    attention; whatever the caller enqueues next on its own stream - the rest of the
                                    layer, the next layer's chunk - overlaps it, and every later call on this context
                                    first orders its stream behind that kernel.  dev_out, dev_q, dev_k, dev_v are only
                                    touched on the caller's stream.  Setting it creates (0: synchronises and destroys)
                                    the stream and two events; treekv_destroy then waits for the stream; calls made
                                    while the caller's stream is being captured into a graph are not supported. */
} treekv_option;

typedef struct {
    uint64_t evictions;       /* pair evictions performed, summed over sequences (not over heads) */
    uint64_t near_ties;       /* pair decisions whose relative score gap was below 1e-4, summed over heads */
    uint64_t kernel_launches; /* kernels this context has enqueued since creation or reset */
    uint32_t device_error;    /* 0, or the code a kernel left when it refused to continue */
    int32_t last_cuda_error;  /* last cudaError_t seen by the library, 0 if none */
} treekv_stats;

/*
 * Bytes of device workspace a context of this shape needs (0 if the shape is unsupported).
 * The workspace holds, per (sequence, KV head): K and V slabs of 2*budget + max_chunk rows, the score sums
 * S and the stream positions of the cached tokens; plus per-call scratch for chunked prefill (partial
 * column sums), for bf16 / head_dim 128 contexts with chunks a third slab for keys encoded at their cache slots
 * (used when in-cache positions are on), and staging buffers for the *_host entry points.
 * max_chunk = 0 makes a decode-only context.
 */
size_t treekv_workspace_bytes(int budget, int n_heads, int n_kv_heads, int head_dim, treekv_dtype dtype,
                              int batch, int max_chunk);

/*
 * Create a layer context (Algorithm 1, initialisation: empty cache, idx = 1).
 *   budget      cache size c, 2..65536                n_heads / n_kv_heads   query / KV heads, n_heads % n_kv_heads == 0,
 *   head_dim    64 or 128                                                    group size in {1,2,4,8}
 *   batch       1..1024 sequences                     max_chunk              longest prefill chunk, 0..8192
 *   dev_workspace  device memory, 256-byte aligned, at least treekv_workspace_bytes(...) bytes; owned by the caller and
 *                  used by the context until treekv_destroy
 * Enqueues the initialisation of the workspace on `stream`.  On error *out is NULL.
 */
treekv_status treekv_create(treekv_ctx** out, int budget, int n_heads, int n_kv_heads, int head_dim,
                            treekv_dtype dtype, int batch, int max_chunk, void* dev_workspace,
                            size_t workspace_bytes, void* stream);

/*
 * One decode step for every active sequence (Algorithm 1, one iteration of the loop; Section 3.1 for the
 * attention): append k,v; attend over the cache including the new token; add the weights to S; if the cache
 * is longer than c, evict one member of the scope and advance idx.
 *   dev_q, dev_out  [batch][n_heads][head_dim]        dev_k, dev_v  [batch][n_kv_heads][head_dim]
 *   host_active     [batch] bytes, nonzero = take the step; NULL = all sequences.  Read before returning.
 * Inactive sequences are untouched and their rows of dev_out are not written.
 */
treekv_status treekv_decode_step(treekv_ctx* ctx, const void* dev_q, const void* dev_k, const void* dev_v,
                                 void* dev_out, const uint8_t* host_active, void* stream);

/*
 * One chunk of chunked prefill (the paper's prefill is one-shot; this applies Algorithm 1 to a chunk at a
 * time): append chunk_lens[b] tokens to sequence b; chunk row i attends to every cached token and to chunk
 * rows <= i; S gains the column sums of the chunk's probability matrix and C advances by the chunk; then
 * Algorithm 1's eviction branch is repeated with those scores until the cache is back to c.
 *   dev_q, dev_out  [batch][chunk_stride][n_heads][head_dim]
 *   dev_k, dev_v    [batch][chunk_stride][n_kv_heads][head_dim]
 *   host_chunk_lens [batch] int32 in 0..min(chunk_stride, max_chunk) (0 = sequence not in this call); NULL = all
 *                   chunk_stride.  Read before returning.
 * Rows of dev_out beyond a sequence's chunk length are not written.
 */
treekv_status treekv_prefill_chunk(treekv_ctx* ctx, const void* dev_q, const void* dev_k, const void* dev_v,
                                   void* dev_out, const int32_t* host_chunk_lens, int chunk_stride,
                                   void* stream);

/*
 * One-shot, block-level prefill of an empty cache (Section 4.2): the whole prompt of host_lens[b] tokens is attended
 * causally (dev_out = plain attention over the prompt), the last `block` tokens are the observation window whose
 * queries alone score the prompt (Algorithm 1's S and C updates for those rows: a token older than the window gets
 * C = block, window token u gets C = block - u), a block's importance is the mean of its tokens' S / C, and
 * Algorithm 1's eviction branch runs on blocks of `block` tokens - each block standing for one token of Figure 3 - with
 * a cache of budget / block blocks.  Afterwards the cache holds min(prompt, budget) tokens in whole blocks, and decode
 * steps or chunks continue from there (the eviction pointer stands on the first token of the block the block pointer
 * reached; S and C carry on).  The paper fixes neither `block` nor a ragged tail: prompt lengths and the budget must be
 * multiples of `block` (TREEKV_ERR_INVALID_ARG otherwise).
 *   dev_q, dev_out  [batch][stride][n_heads][head_dim]     dev_k, dev_v  [batch][stride][n_kv_heads][head_dim]
 *   host_lens       [batch] int32 in 0..min(stride, max_chunk), 0 = sequence not in this call; NULL = all `stride`
 * Sequences in the call must not have seen a token yet (TREEKV_ERR_BAD_STATE); with protected tokens set the call
 * returns TREEKV_ERR_UNSUPPORTED.  Nothing is enqueued on an error.
 */
treekv_status treekv_prefill_oneshot(treekv_ctx* ctx, const void* dev_q, const void* dev_k, const void* dev_v,
                                     void* dev_out, const int32_t* host_lens, int stride, int block, void* stream);

/*
 * The same two calls with HOST tensors (pageable or page-locked), all enqueued on `stream`: host_out is valid,
 * and the host inputs may be reused, once the stream has been synchronised.  Shapes as above.
 * treekv_decode_step_host: when all four tensors are page-locked memory the GPU can address (cudaHostAlloc /
 * cudaHostRegister, 16-byte aligned), the step's kernel reads q, k, v from them and writes the output to them
 * directly across the bus - one launch, no staging copy; otherwise the inputs are copied to staging buffers
 * inside the workspace, the step runs, and the output is copied back.  host_q, host_k, host_v must hold their
 * final values when the call is made (the CPU filled them): on the direct path the kernel may fetch them
 * before earlier work in `stream` has finished.  The cache and host_out are touched only after it.
 * treekv_prefill_chunk_host always stages through the workspace.
 */
treekv_status treekv_decode_step_host(treekv_ctx* ctx, const void* host_q, const void* host_k, const void* host_v,
                                      void* host_out, const uint8_t* host_active, void* stream);
treekv_status treekv_prefill_chunk_host(treekv_ctx* ctx, const void* host_q, const void* host_k,
                                        const void* host_v, void* host_out, const int32_t* host_chunk_lens,
                                        int chunk_stride, void* stream);

/*
 * treekv_prefill_chunk for callers that cannot allocate device memory.  (The paper has no counterpart: this
 * is a deployment variant of the call above, not a different computation.)
 *
 * Same arguments and the same result as treekv_prefill_chunk within the library's tolerances (it always runs the
 * CUDA-core attention kernel, so against a context that runs the tensor-core kernel outputs and scores agree to
 * rounding, and against one forced to the CUDA-core kernel bit for bit), but none of the call's scratch (partial
 * column sums, rows staged during compaction) is taken from the workspace: it lives in a fixed 16 MiB area that is
 * part of the library image and stays on every GPU that has used this entry point until the process exits.  It is meant for code that may not call cudaMalloc at the point where it
 * runs - a server that has frozen its memory pool, a plug-in inside another framework's allocator, a loop
 * that cannot take cudaMalloc's device-wide synchronisation - and so cannot size scratch per call.  The
 * entry point itself calls no allocating routine.
 *   - Limit: with u = batch * n_kv_heads, m = the longest chunk of this call, g = n_heads / n_kv_heads and
 *     e = element size, it needs  u * (ceil(g*m/128) * (budget + m) * 4  +  2 * m * head_dim * e  +  8 * m)
 *     bytes (each of the five parts rounded up to 256); beyond 16 MiB it returns TREEKV_ERR_UNSUPPORTED and
 *     enqueues nothing.
 *   - The first call on a device looks up the area's device address (once per device, with that device
 *     current).  That lookup is also the moment the CUDA runtime loads the part of the library that holds the
 *     area, i.e. when the GPU commits the 16 MiB; it may synchronise the device and can fail when no memory is
 *     left.  So make one warm-up call per device at start-up - before a memory pool is frozen and outside any
 *     stream capture; every later call only reads the cached address.
 *   - The device that is current at the call must be the one the context was created on (where its workspace
 *     lives); otherwise TREEKV_ERR_BAD_STATE.
 *   - Every context of the process shares the one area of its GPU, and the area keeps whatever the last call
 *     left.  A call never reads a slot it has not itself written first, so nothing needs clearing between
 *     calls; but two calls that overlap on the GPU (issued on different streams, whether for the same context
 *     or for different ones) race on it.  Keep calls to this entry point ordered on one stream, or serialise
 *     them some other way.
 */
treekv_status treekv_prefill_chunk_static_scratch(treekv_ctx* ctx, const void* dev_q, const void* dev_k,
                                                  const void* dev_v, void* dev_out,
                                                  const int32_t* host_chunk_lens, int chunk_stride, void* stream);

/*
 * Stream positions of the retained tokens (what Figures 1 and 3 draw), in cache order, i.e. strictly increasing.
 *   dev_pos    [batch][n_kv_heads][budget] int32, unused tail filled with -1
 *   dev_count  [batch][n_kv_heads] int32, number of retained tokens (= min(tokens seen, budget))
 */
treekv_status treekv_retained_positions(treekv_ctx* ctx, int32_t* dev_pos, int32_t* dev_count, void* stream);

/*
 * Importance score S / C (Algorithm 1, "Importance Scores") of every retained token, in cache order.
 *   dev_sbar   [batch][n_kv_heads][budget] float, unused tail filled with 0
 */
treekv_status treekv_scores(treekv_ctx* ctx, float* dev_sbar, void* stream);

/*
 * State image: everything Algorithm 1 carries from one step to the next, in cache order, so that a context of the
 * same shape can continue the stream elsewhere or later (the paper has no counterpart; idx and the counters C follow
 * from the tokens seen, the stored positions and the scoring start).  Layout of the image, each part starting on a 256-byte boundary:
 *   K   [batch][n_kv_heads][budget][head_dim]  dtype     V    the same
 *   S   [batch][n_kv_heads][budget] float (sums, not averages)      pos  [batch][n_kv_heads][budget] int32
 *   tokens seen [batch] int32                                       scoring start [batch] int32 (0 unless the
 *                                                                   sequence was prefilled in one shot)
 * Slots beyond a sequence's cache length are zero (pos: -1).  The protected-token setting is not part of the image:
 * the importing context must have the same one.
 * treekv_export_state enqueues the copy and writes the host-side token counts to host_tokens_seen[batch] before
 * returning; treekv_import_state replaces the context's state by the image (enqueued on `stream`) and takes the
 * same counts back - they must be the ones exported with the image.
 */
size_t treekv_state_bytes(const treekv_ctx* ctx);
treekv_status treekv_export_state(treekv_ctx* ctx, void* dev_image, int64_t* host_tokens_seen, void* stream);
treekv_status treekv_import_state(treekv_ctx* ctx, const void* dev_image, const int64_t* host_tokens_seen,
                                  void* stream);

/* Counters and error words.  Synchronises `stream` to read the device-side counters.  *host_out is filled
 * whenever the read itself succeeded; the return value is TREEKV_ERR_TIMEOUT when device_error is non-zero, i.e.
 * when a kernel's bounded wait gave up (bits: 4 TMA producer, 8 MMA issuer, 16 softmax / epilogue warps of the
 * tensor-core prefill kernels, 32 misaligned shared memory, 64 the self-test below, 128 the decode kernel's fetch of the step's q, k, v).  treekv_reset clears it. */
treekv_status treekv_get_stats(treekv_ctx* ctx, treekv_stats* host_out, void* stream);

/*
 * Self-test of the give-up path (the paper has no counterpart).  Enqueues a kernel of one thread block that waits,
 * for at most `attempts` polls (1..4096), on a barrier that nothing signals - with the helper every bounded wait of
 * the library uses - and then records the give-up in the context's device error word, as a real kernel would.  The
 * cache is not touched.  Afterwards treekv_get_stats returns TREEKV_ERR_TIMEOUT with device_error = 64 until
 * treekv_reset.  Healthy runs never take this path, so this call is how the status plumbing is exercised.
 */
treekv_status treekv_selftest_wait_giveup(treekv_ctx* ctx, int attempts, void* stream);

/* Tokens seen so far by sequence b according to the host-side record (-1 on bad arguments). */
int64_t treekv_tokens_seen(const treekv_ctx* ctx, int b);

treekv_status treekv_set_rule(treekv_ctx* ctx, treekv_rule rule);

/*
 * Protected tokens (Section 5.2: the language-modelling runs split a cache of 1024 into 4 initial tokens, 508 recent ones
 * and 512 chosen by the method).  The first n_sink tokens of every sequence and its n_recent newest
 * cached tokens are never in an eviction scope; Algorithm 1 runs on the budget - n_sink - n_recent slots between
 * them (idx cycles over that many slots), and a token becomes eligible in the step in which it stops being one of
 * the n_recent newest.  S and C of every cached token advance from its arrival as in Algorithm 1.  The paper gives
 * the split, not these mechanics.  (0, 0) - the default - is Algorithm 1 as printed.
 * Needs n_sink + n_recent <= budget - 2 (TREEKV_ERR_INVALID_ARG) and a context that has not seen a token yet
 * (after creation or treekv_reset; else TREEKV_ERR_BAD_STATE).  Host-side only, nothing is enqueued.
 */
treekv_status treekv_set_protection(treekv_ctx* ctx, int n_sink, int n_recent);
/*
 * In-cache positions (Section 4.1 "Position Encoding": positional encodings are re-assigned after eviction - a cache
 * holding tokens {0,1,2,3,7,8,9} plus the new token is encoded at positions 0..7).  With tables set, q and k must
 * arrive WITHOUT positional encoding; the cache keeps k as given, and every attention encodes the key in cache
 * slot j (0-based, cache order) at position j and each query at its own slot (the last slot in a decode step, the
 * row's slot in a chunk) with rotary embedding, rotate-half pairing (t, t + head_dim/2).
 *   dev_cos, dev_sin  [slots][head_dim/2] float, device memory, 16-byte aligned, owned by the caller and read by
 *                     every later call; slots >= budget + max(1, max_chunk).  Both NULL: back to position-agnostic.
 * Numeric contract: x1' = fma(x1, cos, -(x2 sin)), x2' = fma(x2, cos, x1 sin) in fp32, rounded to the context's dtype
 * before the dot product (the paper's runs are bf16 throughout; an fp32 context does not round).
 * Only on a context that has not seen a token (TREEKV_ERR_BAD_STATE otherwise).  Decode steps of a bf16
 * context keep their fast kernel, which encodes each key tile in shared memory on its way to the tensor cores; prefill
 * chunks of a bf16 / head_dim 128 context keep the tensor-core kernels, which then run on keys and queries that a
 * kernel of the same call has encoded at their slots (into a second key slab of the workspace and the query staging
 * buffer: for such a context chunk_stride must not exceed max_chunk, TREEKV_ERR_UNSUPPORTED otherwise); fp32 contexts
 * and head_dim 64 run on the CUDA-core kernels, which encode while they stream.  Host-side only, nothing is enqueued.
 */
treekv_status treekv_set_positions(treekv_ctx* ctx, const float* dev_cos, const float* dev_sin, int slots);

treekv_status treekv_set_option(treekv_ctx* ctx, treekv_option opt, int value);

/* Back to the empty cache (idx = 1, nothing seen).  Enqueued on `stream`. */
treekv_status treekv_reset(treekv_ctx* ctx, void* stream);

/* Frees the host-side context (with TREEKV_OPT_EVICTION_STREAM on, after waiting for the context's own stream).  The
 * workspace stays the caller's. */
void treekv_destroy(treekv_ctx* ctx);

const char* treekv_status_string(treekv_status s);

/* Library version, "major.minor". */
const char* treekv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TREEKV_H */
