// C ABI of the TreeKV library: context bookkeeping, argument checks, workspace carving, launch sequencing.
// Every step of the path runs in the kernels of decode.cu, prefill_*.cu and state.cu; this file only decides
// what to enqueue.
#include <new>
#include <string.h>

#include "common.cuh"
#include "ctx.cuh"
#include "tma.cuh"

using namespace treekv;

namespace {

constexpr size_t kAlign = 256;
constexpr size_t kSmemLimit = 227 * 1024;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Layout {
    size_t K, V, Krot, S, pos, n_seen, w0, stats, colsum, st_q, st_k, st_v, st_out, total;
    int R, QT, n_max;
};

bool shape_ok(int budget, int n_heads, int n_kv_heads, int head_dim, treekv_dtype dt, int batch, int max_chunk) {
    if (budget < 2 || budget > 65536) return false;
    if (n_heads < 1 || n_kv_heads < 1 || n_heads % n_kv_heads) return false;
    const int G = n_heads / n_kv_heads;
    if (!(G == 1 || G == 2 || G == 4 || G == 8)) return false;
    if (!(head_dim == 64 || head_dim == 128)) return false;
    if (!(dt == TREEKV_F32 || dt == TREEKV_BF16)) return false;
    if (batch < 1 || batch > kMaxBatch) return false;
    if (max_chunk < 0 || max_chunk > 8192) return false;
    if (n_kv_heads > 65535 || (long long)batch * n_kv_heads > 65535) return false;  // grid.y of the per-unit kernels
    if (decode_smem_bytes(G, head_dim, budget, 8) > kSmemLimit) return false;
    if (dt == TREEKV_BF16 && decode_mma_smem_bytes(G, head_dim, budget, 8) > kSmemLimit) return false;
    if (max_chunk > 0 && prefill_simt_smem_bytes(G, head_dim, budget + max_chunk) > kSmemLimit) return false;
    return true;
}

Layout make_layout(int budget, int n_heads, int n_kv_heads, int head_dim, treekv_dtype dt, int batch, int max_chunk) {
    Layout L;
    const size_t e = dt == TREEKV_F32 ? 4 : 2;
    const size_t units = (size_t)batch * n_kv_heads;
    const int G = n_heads / n_kv_heads;
    L.R = 2 * budget + max_chunk;
    L.QT = max_chunk > 0 ? (max_chunk * G + kQTileRows - 1) / kQTileRows : 0;
    L.n_max = budget + max_chunk;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    L.K = take(units * L.R * head_dim * e);
    L.V = take(units * L.R * head_dim * e);
    // keys encoded at their cache slots, rebuilt per call for the tensor-core prefill when in-cache positions are on
    L.Krot = (dt == TREEKV_BF16 && head_dim == 128 && max_chunk > 0) ? take(units * L.R * head_dim * e) : 0;
    L.S = take(units * L.R * 4);
    L.pos = take(units * L.R * 4);
    L.n_seen = take(units * 4);
    L.w0 = take(units * 4);
    L.stats = take(sizeof(DevStats));
    L.colsum = take(units * L.QT * L.n_max * 4);
    const size_t mc = max_chunk > 0 ? max_chunk : 1;
    L.st_q = take((size_t)batch * mc * n_heads * head_dim * e);
    L.st_k = take((size_t)batch * mc * n_kv_heads * head_dim * e);
    L.st_v = take((size_t)batch * mc * n_kv_heads * head_dim * e);
    L.st_out = take((size_t)batch * mc * n_heads * head_dim * e);
    L.total = off;
    return L;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

treekv_status cuda_fail(treekv_ctx* ctx, cudaError_t e) {
    if (ctx) ctx->last_cuda_error = (int)e;
    return TREEKV_ERR_CUDA;
}

// (With in-cache positions the tensor-core kernels run on keys and queries encoded by a kernel of their own first.)
bool use_tc_prefill(const treekv_ctx* ctx) { return ctx->has_tma && ctx->opt_prefill_path != 1; }

bool use_mma_decode(const treekv_ctx* ctx) {
    if (ctx->dt != TREEKV_BF16) return false;
    return ctx->opt_decode_path != 1;
}

size_t decode_smem_for(const treekv_ctx* ctx, int split) {
    return use_mma_decode(ctx) ? decode_mma_smem_bytes(ctx->G, ctx->cv.d, ctx->cv.c, split)
                               : decode_smem_bytes(ctx->G, ctx->cv.d, ctx->cv.c, split);
}

// Thread blocks (cluster size) per unit.  The bf16 kernel keeps one CTA per unit once there are at least as many
// units as SMs (its CTAs are small and several are resident per SM) and otherwise splits until the machine is
// covered about twice - but clusters of eight only while all CTAs fit one per SM: a cluster must be placed inside
// one GPC, and with more CTAs than SMs some clusters of eight waited for a second wave.  The CUDA-core kernel
// splits while a CTA keeps at least 128 rows.
int pick_decode_split(const treekv_ctx* ctx) {
    const int c = ctx->cv.c, units = ctx->cv.B * ctx->cv.Hkv;
    int s = ctx->opt_decode_split;
    if (s == 0) {
        s = 1;
        if (use_mma_decode(ctx)) {
            while (s < 8 && units * (2 * s) <= (2 * s == 8 ? 1 : 2) * ctx->sm_count && (c + 1) / (2 * s) >= 64) s *= 2;
        } else {
            while (s < 8 && units * s < 3 * ctx->sm_count && (c + 1) / (2 * s) >= 128) s *= 2;
        }
    }
    while (s < 8 && decode_smem_for(ctx, s) > kSmemLimit) s *= 2;
    return s;
}

// Device-side alias of a host pointer when the GPU can address it directly (page-locked memory registered with
// the CUDA runtime, or memory allocated by it), else nullptr.
void* device_alias(const void* host_ptr) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host_ptr) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    if (at.type != cudaMemoryTypeHost && at.type != cudaMemoryTypeManaged && at.type != cudaMemoryTypeDevice) return nullptr;
    return at.devicePointer;
}

}  // namespace

extern "C" {

size_t treekv_workspace_bytes(int budget, int n_heads, int n_kv_heads, int head_dim, treekv_dtype dtype, int batch,
                              int max_chunk) {
    if (!shape_ok(budget, n_heads, n_kv_heads, head_dim, dtype, batch, max_chunk)) return 0;
    return make_layout(budget, n_heads, n_kv_heads, head_dim, dtype, batch, max_chunk).total;
}

treekv_status treekv_create(treekv_ctx** out, int budget, int n_heads, int n_kv_heads, int head_dim, treekv_dtype dtype,
                            int batch, int max_chunk, void* dev_workspace, size_t workspace_bytes, void* stream) {
    if (!out) return TREEKV_ERR_INVALID_ARG;
    *out = nullptr;
    if (!shape_ok(budget, n_heads, n_kv_heads, head_dim, dtype, batch, max_chunk)) return TREEKV_ERR_UNSUPPORTED;
    const Layout L = make_layout(budget, n_heads, n_kv_heads, head_dim, dtype, batch, max_chunk);
    if (!dev_workspace || (reinterpret_cast<uintptr_t>(dev_workspace) % kAlign) != 0 || workspace_bytes < L.total)
        return TREEKV_ERR_WORKSPACE;
    treekv_ctx* ctx = new (std::nothrow) treekv_ctx;
    if (!ctx) return TREEKV_ERR_INVALID_ARG;
    memset(ctx, 0, sizeof(*ctx));
    char* base = static_cast<char*>(dev_workspace);
    ctx->cv.K = base + L.K;
    ctx->cv.V = base + L.V;
    ctx->cv.S = reinterpret_cast<float*>(base + L.S);
    ctx->cv.pos = reinterpret_cast<int32_t*>(base + L.pos);
    ctx->cv.n_seen = reinterpret_cast<int32_t*>(base + L.n_seen);
    ctx->cv.w0 = reinterpret_cast<int32_t*>(base + L.w0);
    ctx->cv.stats = reinterpret_cast<DevStats*>(base + L.stats);
    ctx->cv.c = budget; ctx->cv.R = L.R; ctx->cv.Hq = n_heads; ctx->cv.Hkv = n_kv_heads; ctx->cv.B = batch;
    ctx->cv.d = head_dim; ctx->cv.rule = TREEKV_RULE_SCORES;
    ctx->cv.ns = 0; ctx->cv.nr = 0; ctx->cv.cm = budget;
    ctx->cv.rope_cos = nullptr; ctx->cv.rope_sin = nullptr;
    ctx->ps.colsum = reinterpret_cast<float*>(base + L.colsum);
    // (rows in flight during compaction stay in registers: the context has no staging rows; PrefillScratch's
    //  staging pointers are only used by the entry point that brings its own scratch)
    ctx->ps.QT = L.QT; ctx->ps.n_max = L.n_max; ctx->ps.max_chunk = max_chunk; ctx->ps.window = 0;
    ctx->st_q = base + L.st_q; ctx->st_k = base + L.st_k; ctx->st_v = base + L.st_v; ctx->st_out = base + L.st_out;
    ctx->dt = dtype; ctx->max_chunk = max_chunk; ctx->G = n_heads / n_kv_heads;
    ctx->elem = dtype == TREEKV_F32 ? 4 : 2;
    {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
            sms = 148;
        ctx->sm_count = sms;
        ctx->device = dev;
    }
    ctx->has_tma = false;
    if (dtype == TREEKV_BF16 && head_dim == 128 && max_chunk > 0) {
        const uint64_t rows = (uint64_t)batch * n_kv_heads * L.R;
        const uint64_t dims[2] = {(uint64_t)head_dim, rows};
        const uint64_t strides[1] = {(uint64_t)head_dim * 2};
        const uint32_t box[2] = {64u, 128u};
        ctx->k_rot = base + L.Krot;
        ctx->has_tma = make_tensor_map_bf16(&ctx->tmK, ctx->cv.K, 2, dims, strides, box) &&
                       make_tensor_map_bf16(&ctx->tmV, ctx->cv.V, 2, dims, strides, box) &&
                       make_tensor_map_bf16(&ctx->tmKrot, ctx->k_rot, 2, dims, strides, box);
    }
    // The workspace starts as zeros: the tensor-core prefill reads whole 128-row tiles, and rows that hold no token
    // yet must be finite (they are multiplied by a probability of exactly zero).
    cudaError_t e = cudaMemsetAsync(dev_workspace, 0, L.total, static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess) e = launch_init_state(ctx->cv, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { delete ctx; return TREEKV_ERR_CUDA; }
    ctx->launches = 1;
    *out = ctx;
    return TREEKV_OK;
}

treekv_status treekv_reset(treekv_ctx* ctx, void* stream) {
    if (!ctx) return TREEKV_ERR_INVALID_ARG;
    cudaError_t e = join_eviction_stream(ctx, static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess) e = launch_init_state(ctx->cv, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    memset(ctx->n_seen, 0, sizeof(ctx->n_seen));
    ctx->evictions = 0;
    ctx->launches = 1;
    return TREEKV_OK;
}

void treekv_destroy(treekv_ctx* ctx) {
    if (!ctx) return;
    if (ctx->side) {  // the workspace is the caller's to free after this call: nothing of ours may still run on it
        cudaStreamSynchronize(ctx->side);
        cudaEventDestroy(ctx->ev_attn);
        cudaEventDestroy(ctx->ev_state);
        cudaStreamDestroy(ctx->side);
    }
    delete ctx;
}

}  // extern "C"

namespace {
treekv_status decode_step_impl(treekv_ctx* ctx, const void* dev_q, const void* dev_k, const void* dev_v, void* dev_out,
                               const uint8_t* host_active, void* stream, int inputs_final) {
    if (!ctx || !dev_q || !dev_k || !dev_v || !dev_out) return TREEKV_ERR_INVALID_ARG;
    if (!aligned16(dev_q) || !aligned16(dev_k) || !aligned16(dev_v) || !aligned16(dev_out)) return TREEKV_ERR_INVALID_ARG;
    ActiveMask mask;
    memset(&mask, 0, sizeof(mask));
    int n_active = 0;
    for (int b = 0; b < ctx->cv.B; ++b) {
        if (!host_active || host_active[b]) {
            if (ctx->n_seen[b] >= 0x7fffffff - 1) return TREEKV_ERR_BAD_STATE;
            mask.w[b >> 5] |= 1u << (b & 31);
            ++n_active;
        }
    }
    if (n_active == 0) return TREEKV_OK;
    if (ctx->side_pending) {
        const cudaError_t je = join_eviction_stream(ctx, static_cast<cudaStream_t>(stream));
        if (je != cudaSuccess) return cuda_fail(ctx, je);
    }
    const cudaError_t e =
        use_mma_decode(ctx)
            ? launch_decode_mma(ctx->cv, dev_q, dev_k, dev_v, dev_out, mask, pick_decode_split(ctx), inputs_final,
                                static_cast<cudaStream_t>(stream))
            : launch_decode(ctx->cv, ctx->dt, dev_q, dev_k, dev_v, dev_out, mask, pick_decode_split(ctx),
                            static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    for (int b = 0; b < ctx->cv.B; ++b) {
        if (mask.test(b)) {
            ctx->n_seen[b] += 1;
            if (ctx->n_seen[b] > ctx->cv.c) ctx->evictions += 1;
        }
    }
    return TREEKV_OK;
}

// Attention of a chunk over [cache | chunk] with the column sums of its probability matrix (all of the chunk's
// rows, or the last ps.window tokens): tensor-core kernels for bf16 / head_dim 128, CUDA cores otherwise.
// `direct`: the tensor-core kernels take the chunk's key / value tiles from dev_k / dev_v and append the chunk to the
// slabs themselves (see chunk_direct_ok); otherwise the chunk's rows must already be in the slabs.
treekv_status launch_chunk_attention(treekv_ctx* ctx, const PrefillScratch& ps, const void* dev_q, const void* dev_k,
                                     const void* dev_v, bool direct, void* dev_out, const ChunkLens& lens, int chunk_stride,
                                     int max_m, cudaStream_t s) {
    cudaError_t e;
    if (use_tc_prefill(ctx)) {
        const CUtensorMap* tmKeys = &ctx->tmK;
        if (ctx->cv.rope_cos) {
            // in-cache positions: every live key encoded at its slot into the rotated slab, the chunk's queries at their
            // own slots into the staging buffer (in place when the caller's q already is that buffer)
            e = launch_rope_chunk(ctx->cv, lens, chunk_stride, max_m, ctx->k_rot, dev_q, ctx->st_q, s);
            if (e != cudaSuccess) return cuda_fail(ctx, e);
            ctx->launches += 1;
            dev_q = ctx->st_q;
            tmKeys = &ctx->tmKrot;
        }
        ChunkTensors ct;
        ct.k = nullptr; ct.v = nullptr;
        if (direct) {
            const uint64_t kdims[3] = {128ull, (uint64_t)ctx->cv.Hkv, (uint64_t)ctx->cv.B * (uint64_t)chunk_stride};
            const uint64_t kstrides[2] = {256ull, (uint64_t)ctx->cv.Hkv * 256ull};
            const uint32_t kbox[3] = {64u, 1u, 128u};
            if (!make_tensor_map_bf16(&ct.tmK, dev_k, 3, kdims, kstrides, kbox) ||
                !make_tensor_map_bf16(&ct.tmV, dev_v, 3, kdims, kstrides, kbox))
                return TREEKV_ERR_CUDA;
            ct.k = dev_k; ct.v = dev_v;
        }
        // q is [batch*chunk_stride tokens][n_heads][128]; a tile is 64 channels x G heads x 128/G tokens
        CUtensorMap tmQ;
        const uint64_t dims[3] = {128ull, (uint64_t)ctx->cv.Hq, (uint64_t)ctx->cv.B * (uint64_t)chunk_stride};
        const uint64_t strides[2] = {256ull, (uint64_t)ctx->cv.Hq * 256ull};
        const uint32_t box[3] = {64u, (uint32_t)ctx->G, (uint32_t)(128 / ctx->G)};
        if (!make_tensor_map_bf16(&tmQ, dev_q, 3, dims, strides, box)) return TREEKV_ERR_CUDA;
        // Which kernel: two query tiles per CTA (every K / V tile load feeds twice the tensor work) once the one-tile grid
        // would cover the machine at least twice, one tile per CTA for smaller calls.
        const long tiles = (long)ctx->cv.B * ctx->cv.Hkv * ((max_m * ctx->G + kQTileRows - 1) / kQTileRows);
        const bool two = ctx->opt_prefill_path == 3 || (ctx->opt_prefill_path == 0 && tiles >= 2L * ctx->sm_count);
        // Key split of the two-tile kernel.  A grid that is not a whole number of waves ends with a wave of few CTAs; when
        // those last tile pairs are at most half a wave, each of them goes to a cluster of two CTAs that halve its key
        // tiles, so the last wave is full and about half as long (the CTAs of the full waves are launched as clusters
        // too, one whole tile pair each, exchanging nothing).  Splitting every pair costs more in exchanges than it
        // gains, and is on request only.  Option value 3 applies the same rule for a machine of four SMs (small test grids).
        int n_whole = -1;
        if (two) {
            const long pairs = (long)ctx->cv.B * ctx->cv.Hkv * ((max_m * ctx->G + 2 * kQTileRows - 1) / (2 * kQTileRows));
            const int opt = ctx->opt_prefill_key_split;
            if (opt == 2) {
                n_whole = 0;
            } else if (opt == 0 || opt == 3) {
                const long sms = opt == 3 ? 4 : (ctx->sm_count & ~1);
                const long rem = pairs % sms;
                if (rem > 0 && 2 * rem <= sms && pairs > rem) n_whole = (int)((pairs - rem) / 2);
            }
        }
        ctx->attn_blocks = tiles;
        if (two) {  // one block per tile pair; with key splitting two per cluster: whole-pair clusters, then one cluster per pair
            const long pairs = (long)ctx->cv.B * ctx->cv.Hkv * ((max_m * ctx->G + 2 * kQTileRows - 1) / (2 * kQTileRows));
            ctx->attn_blocks = n_whole < 0 ? pairs : 2 * (n_whole + std::max(0L, pairs - 2L * n_whole));
        }
        e = two ? launch_prefill_tc2(ctx->cv, ps, tmQ, *tmKeys, ctx->tmV, ct, dev_out, lens, chunk_stride, max_m, n_whole, s)
                : launch_prefill_tc(ctx->cv, ps, tmQ, *tmKeys, ctx->tmV, ct, dev_out, lens, chunk_stride, max_m, s);
    } else {
        ctx->attn_blocks = 0;
        e = launch_prefill_simt(ctx->cv, ctx->dt, ps, dev_q, dev_out, lens, chunk_stride, max_m, s);
    }
    return e == cudaSuccess ? TREEKV_OK : cuda_fail(ctx, e);
}

// The tensor-core kernels can read the chunk's keys and values from the caller's tensors - and append them - when
// every chunk tile of 128 tokens holds tokens of the call only (rows past a sequence's length are the caller's
// padding and may hold anything, which a value tile must not) and the cached tokens already cover the protected
// initial tokens (so that the chunk's rows lie behind both cached segments).
bool chunk_direct_ok(const treekv_ctx* ctx, const ChunkLens& lens) {
    if (!use_tc_prefill(ctx) || ctx->opt_prefill_append == 1 || ctx->cv.rope_cos) return false;
    for (int b = 0; b < ctx->cv.B; ++b) {
        if (lens.m[b] == 0) continue;
        if (lens.m[b] % 128 || ctx->n_seen[b] < ctx->cv.ns) return false;
    }
    return true;
}

}  // namespace

extern "C" {

treekv_status treekv_decode_step(treekv_ctx* ctx, const void* dev_q, const void* dev_k, const void* dev_v, void* dev_out,
                                 const uint8_t* host_active, void* stream) {
    return decode_step_impl(ctx, dev_q, dev_k, dev_v, dev_out, host_active, stream, 0);
}

treekv_status treekv_prefill_chunk(treekv_ctx* ctx, const void* dev_q, const void* dev_k, const void* dev_v, void* dev_out,
                                   const int32_t* host_chunk_lens, int chunk_stride, void* stream) {
    if (!ctx || !dev_q || !dev_k || !dev_v || !dev_out) return TREEKV_ERR_INVALID_ARG;
    if (!aligned16(dev_q) || !aligned16(dev_k) || !aligned16(dev_v) || !aligned16(dev_out)) return TREEKV_ERR_INVALID_ARG;
    if (ctx->max_chunk == 0) return TREEKV_ERR_BAD_STATE;  // decode-only context
    if (chunk_stride < 1) return TREEKV_ERR_INVALID_ARG;
    // with in-cache positions the tensor-core path keeps the encoded queries in a staging buffer sized for max_chunk
    if (ctx->cv.rope_cos && use_tc_prefill(ctx) && chunk_stride > ctx->max_chunk) return TREEKV_ERR_UNSUPPORTED;
    ChunkLens lens;
    memset(&lens, 0, sizeof(lens));
    int max_m = 0;
    for (int b = 0; b < ctx->cv.B; ++b) {
        const int m = host_chunk_lens ? host_chunk_lens[b] : chunk_stride;
        if (m < 0 || m > chunk_stride || m > ctx->max_chunk) return TREEKV_ERR_INVALID_ARG;
        if (ctx->n_seen[b] + m >= 0x7fffffff - 1) return TREEKV_ERR_BAD_STATE;
        lens.m[b] = (uint16_t)m;
        if (m > max_m) max_m = m;
    }
    if (max_m == 0) return TREEKV_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool direct = chunk_direct_ok(ctx, lens);
    // the previous chunk's eviction must be over before this chunk's attention reads the cache and writes column sums
    cudaError_t e = join_eviction_stream(ctx, s);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    if (!direct) {
        e = launch_chunk_append(ctx->cv, ctx->dt, dev_k, dev_v, lens, chunk_stride, max_m, s);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    }
    const treekv_status ast =
        launch_chunk_attention(ctx, ctx->ps, dev_q, dev_k, dev_v, direct, dev_out, lens, chunk_stride, max_m, s);
    if (ast != TREEKV_OK) return ast;
    // score update, all eviction segments and the token counters in one launch - on the eviction stream when there is
    // one: nothing the caller does next with the chunk's output depends on it
    if (ctx->side) {
        e = cudaEventRecord(ctx->ev_attn, s);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->side, ctx->ev_attn, 0);
        // Beside the next attention kernel (typically the next layer's chunk, with the grid this one had): when that
        // grid leaves SMs free, the eviction takes no more blocks than those SMs - an eviction block and an attention
        // block do not fit on one SM, and blocks that got there first would hold up part of the attention's only wave.
        // With fewer free SMs than a quarter of the units the blocks would run long enough to be in the way for longer
        // than a full launch is: then every unit gets its block.
        int max_blocks = 0;
        if (ctx->attn_blocks > 0 && ctx->attn_blocks < ctx->sm_count) {
            const int units = ctx->cv.B * ctx->cv.Hkv, free_sms = (int)(ctx->sm_count - ctx->attn_blocks);
            if (free_sms < units && 4 * free_sms >= units) max_blocks = free_sms;
        }
        if (e == cudaSuccess) e = launch_chunk_update_evict_beside(ctx->cv, ctx->dt, ctx->ps, lens, max_blocks, ctx->side);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_state, ctx->side);
        ctx->side_pending = true;  // also after a failure half-way: a later call then still orders itself behind `side`
    } else {
        e = launch_chunk_update_evict(ctx->cv, ctx->dt, ctx->ps, lens, false, s);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += direct ? 2 : 3;  // (append,) attention, update + eviction
    for (int b = 0; b < ctx->cv.B; ++b) {
        const int64_t before = ctx->n_seen[b];
        ctx->n_seen[b] += lens.m[b];
        const int64_t ev_before = before > ctx->cv.c ? before - ctx->cv.c : 0;
        const int64_t ev_after = ctx->n_seen[b] > ctx->cv.c ? ctx->n_seen[b] - ctx->cv.c : 0;
        ctx->evictions += (uint64_t)(ev_after - ev_before);
    }
    return TREEKV_OK;
}

treekv_status treekv_prefill_oneshot(treekv_ctx* ctx, const void* dev_q, const void* dev_k, const void* dev_v, void* dev_out,
                                     const int32_t* host_lens, int stride, int block, void* stream) {
    if (!ctx || !dev_q || !dev_k || !dev_v || !dev_out) return TREEKV_ERR_INVALID_ARG;
    if (!aligned16(dev_q) || !aligned16(dev_k) || !aligned16(dev_v) || !aligned16(dev_out)) return TREEKV_ERR_INVALID_ARG;
    if (ctx->max_chunk == 0) return TREEKV_ERR_BAD_STATE;  // decode-only context
    if (stride < 1 || block < 1 || ctx->cv.c % block) return TREEKV_ERR_INVALID_ARG;
    if (ctx->cv.rope_cos && use_tc_prefill(ctx) && stride > ctx->max_chunk) return TREEKV_ERR_UNSUPPORTED;
    if (ctx->cv.ns || ctx->cv.nr) return TREEKV_ERR_UNSUPPORTED;  // block-level eviction with protected tokens is not defined
    ChunkLens lens;
    memset(&lens, 0, sizeof(lens));
    int max_m = 0;
    for (int b = 0; b < ctx->cv.B; ++b) {
        const int m = host_lens ? host_lens[b] : stride;
        if (m < 0 || m > stride || m > ctx->max_chunk || m % block) return TREEKV_ERR_INVALID_ARG;
        if (m > 0 && ctx->n_seen[b] != 0) return TREEKV_ERR_BAD_STATE;  // the prompt enters an empty cache
        lens.m[b] = (uint16_t)m;
        if (m > max_m) max_m = m;
    }
    if (max_m == 0) return TREEKV_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = join_eviction_stream(ctx, s);
    if (e == cudaSuccess) e = launch_chunk_append(ctx->cv, ctx->dt, dev_k, dev_v, lens, stride, max_m, s);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    PrefillScratch ps = ctx->ps;
    ps.window = block;  // only the last block's queries score the prompt
    const treekv_status ast = launch_chunk_attention(ctx, ps, dev_q, dev_k, dev_v, false, dev_out, lens, stride, max_m, s);
    if (ast != TREEKV_OK) return ast;
    e = launch_oneshot_update_evict(ctx->cv, ctx->dt, ps, lens, block, s);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 3;
    for (int b = 0; b < ctx->cv.B; ++b) {
        ctx->n_seen[b] += lens.m[b];
        if (lens.m[b] > ctx->cv.c) ctx->evictions += (uint64_t)(lens.m[b] - ctx->cv.c);
    }
    return TREEKV_OK;
}

treekv_status treekv_decode_step_host(treekv_ctx* ctx, const void* host_q, const void* host_k, const void* host_v,
                                      void* host_out, const uint8_t* host_active, void* stream) {
    if (!ctx || !host_q || !host_k || !host_v || !host_out) return TREEKV_ERR_INVALID_ARG;
    // Page-locked host tensors are read and written by the kernel itself across the bus (q, k, v are each read
    // early in the kernel, under the cache stream; the output is written once): no copy, no staging, one launch.
    {
        void* dq = device_alias(host_q);
        void* dk = dq ? device_alias(host_k) : nullptr;
        void* dv = dk ? device_alias(host_v) : nullptr;
        void* dout = dv ? device_alias(host_out) : nullptr;
        if (dout && aligned16(dq) && aligned16(dk) && aligned16(dv) && aligned16(dout))
            return decode_step_impl(ctx, dq, dk, dv, dout, host_active, stream, 1);
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t qb = (size_t)ctx->cv.B * ctx->cv.Hq * ctx->cv.d * ctx->elem;
    const size_t kb = (size_t)ctx->cv.B * ctx->cv.Hkv * ctx->cv.d * ctx->elem;
    cudaError_t e = cudaMemcpyAsync(ctx->st_q, host_q, qb, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->st_k, host_k, kb, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->st_v, host_v, kb, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    const treekv_status st = treekv_decode_step(ctx, ctx->st_q, ctx->st_k, ctx->st_v, ctx->st_out, host_active, stream);
    if (st != TREEKV_OK) return st;
    e = cudaMemcpyAsync(host_out, ctx->st_out, qb, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return TREEKV_OK;
}

treekv_status treekv_prefill_chunk_host(treekv_ctx* ctx, const void* host_q, const void* host_k, const void* host_v,
                                        void* host_out, const int32_t* host_chunk_lens, int chunk_stride, void* stream) {
    if (!ctx || !host_q || !host_k || !host_v || !host_out) return TREEKV_ERR_INVALID_ARG;
    if (ctx->max_chunk == 0) return TREEKV_ERR_BAD_STATE;
    if (chunk_stride < 1 || chunk_stride > ctx->max_chunk) return TREEKV_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t qb = (size_t)ctx->cv.B * chunk_stride * ctx->cv.Hq * ctx->cv.d * ctx->elem;
    const size_t kb = (size_t)ctx->cv.B * chunk_stride * ctx->cv.Hkv * ctx->cv.d * ctx->elem;
    cudaError_t e = cudaMemcpyAsync(ctx->st_q, host_q, qb, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->st_k, host_k, kb, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->st_v, host_v, kb, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    const treekv_status st =
        treekv_prefill_chunk(ctx, ctx->st_q, ctx->st_k, ctx->st_v, ctx->st_out, host_chunk_lens, chunk_stride, stream);
    if (st != TREEKV_OK) return st;
    e = cudaMemcpyAsync(host_out, ctx->st_out, qb, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return TREEKV_OK;
}

treekv_status treekv_retained_positions(treekv_ctx* ctx, int32_t* dev_pos, int32_t* dev_count, void* stream) {
    if (!ctx || !dev_pos || !dev_count) return TREEKV_ERR_INVALID_ARG;
    cudaError_t e = join_eviction_stream(ctx, static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess) e = launch_retained_positions(ctx->cv, dev_pos, dev_count, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return TREEKV_OK;
}

treekv_status treekv_scores(treekv_ctx* ctx, float* dev_sbar, void* stream) {
    if (!ctx || !dev_sbar) return TREEKV_ERR_INVALID_ARG;
    cudaError_t e = join_eviction_stream(ctx, static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess) e = launch_scores(ctx->cv, dev_sbar, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return TREEKV_OK;
}

static size_t state_image_layout(const treekv_ctx* ctx, void* base, StateImage* img) {
    const size_t units = (size_t)ctx->cv.B * ctx->cv.Hkv, slots = units * ctx->cv.c;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    const size_t oK = take(slots * ctx->cv.d * ctx->elem), oV = take(slots * ctx->cv.d * ctx->elem);
    const size_t oS = take(slots * 4), oP = take(slots * 4), oN = take((size_t)ctx->cv.B * 4);
    const size_t oW = take((size_t)ctx->cv.B * 4);
    if (img) {
        char* p = static_cast<char*>(base);
        img->K = p + oK; img->V = p + oV;
        img->S = reinterpret_cast<float*>(p + oS); img->pos = reinterpret_cast<int32_t*>(p + oP);
        img->seen = reinterpret_cast<int32_t*>(p + oN);
        img->w0 = reinterpret_cast<int32_t*>(p + oW);
    }
    return off;
}

size_t treekv_state_bytes(const treekv_ctx* ctx) { return ctx ? state_image_layout(ctx, nullptr, nullptr) : 0; }

treekv_status treekv_export_state(treekv_ctx* ctx, void* dev_image, int64_t* host_tokens_seen, void* stream) {
    if (!ctx || !dev_image || !host_tokens_seen || !aligned16(dev_image)) return TREEKV_ERR_INVALID_ARG;
    StateImage img;
    state_image_layout(ctx, dev_image, &img);
    cudaError_t e = join_eviction_stream(ctx, static_cast<cudaStream_t>(stream));
    // every part starts on a 256-byte boundary: zero the padding behind each, so that two images of the same state are equal
    // byte for byte (the kernel fills every byte of the parts themselves)
    {
        const size_t slots = (size_t)ctx->cv.B * ctx->cv.Hkv * ctx->cv.c;
        const size_t sizes[6] = {slots * ctx->cv.d * ctx->elem, slots * ctx->cv.d * ctx->elem, slots * 4, slots * 4,
                                 (size_t)ctx->cv.B * 4, (size_t)ctx->cv.B * 4};
        size_t off = 0;
        for (int part = 0; part < 6 && e == cudaSuccess; ++part) {
            const size_t end = off + sizes[part], next = align_up(end);
            if (next > end) e = cudaMemsetAsync(static_cast<char*>(dev_image) + end, 0, next - end, static_cast<cudaStream_t>(stream));
            off = next;
        }
    }
    if (e == cudaSuccess) e = launch_export_state(ctx->cv, ctx->dt, img, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    for (int b = 0; b < ctx->cv.B; ++b) host_tokens_seen[b] = ctx->n_seen[b];
    return TREEKV_OK;
}

treekv_status treekv_import_state(treekv_ctx* ctx, const void* dev_image, const int64_t* host_tokens_seen, void* stream) {
    if (!ctx || !dev_image || !host_tokens_seen || !aligned16(dev_image)) return TREEKV_ERR_INVALID_ARG;
    for (int b = 0; b < ctx->cv.B; ++b)
        if (host_tokens_seen[b] < 0 || host_tokens_seen[b] >= 0x7fffffff - 1) return TREEKV_ERR_INVALID_ARG;
    StateImage img;
    state_image_layout(ctx, const_cast<void*>(dev_image), &img);
    cudaError_t e = join_eviction_stream(ctx, static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess) e = launch_import_state(ctx->cv, ctx->dt, img, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    ctx->evictions = 0;
    for (int b = 0; b < ctx->cv.B; ++b) {
        ctx->n_seen[b] = host_tokens_seen[b];
        if (host_tokens_seen[b] > ctx->cv.c) ctx->evictions += (uint64_t)(host_tokens_seen[b] - ctx->cv.c);
    }
    return TREEKV_OK;
}

treekv_status treekv_get_stats(treekv_ctx* ctx, treekv_stats* host_out, void* stream) {
    if (!ctx || !host_out) return TREEKV_ERR_INVALID_ARG;
    DevStats ds;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = join_eviction_stream(ctx, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(&ds, ctx->cv.stats, sizeof(ds), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    host_out->evictions = ctx->evictions;
    host_out->near_ties = ds.near_ties;
    host_out->kernel_launches = ctx->launches;
    host_out->device_error = ds.error;
    host_out->last_cuda_error = ctx->last_cuda_error;
    return ds.error ? TREEKV_ERR_TIMEOUT : TREEKV_OK;
}

int64_t treekv_tokens_seen(const treekv_ctx* ctx, int b) {
    if (!ctx || b < 0 || b >= ctx->cv.B) return -1;
    return ctx->n_seen[b];
}

treekv_status treekv_set_rule(treekv_ctx* ctx, treekv_rule rule) {
    if (!ctx) return TREEKV_ERR_INVALID_ARG;
    if (rule != TREEKV_RULE_SCORES && rule != TREEKV_RULE_KEEP_LEFT && rule != TREEKV_RULE_EVICT_LEFT &&
        rule != TREEKV_RULE_ACCUMULATED)
        return TREEKV_ERR_INVALID_ARG;
    ctx->cv.rule = (int)rule;
    return TREEKV_OK;
}

treekv_status treekv_set_protection(treekv_ctx* ctx, int n_sink, int n_recent) {
    if (!ctx) return TREEKV_ERR_INVALID_ARG;
    if (n_sink < 0 || n_recent < 0 || (long long)n_sink + n_recent > ctx->cv.c - 2) return TREEKV_ERR_INVALID_ARG;
    for (int b = 0; b < ctx->cv.B; ++b)
        if (ctx->n_seen[b] != 0) return TREEKV_ERR_BAD_STATE;  // the layout of a cache in use cannot change
    ctx->cv.ns = n_sink; ctx->cv.nr = n_recent; ctx->cv.cm = ctx->cv.c - n_sink - n_recent;
    return TREEKV_OK;
}

treekv_status treekv_set_positions(treekv_ctx* ctx, const float* dev_cos, const float* dev_sin, int slots) {
    if (!ctx) return TREEKV_ERR_INVALID_ARG;
    for (int b = 0; b < ctx->cv.B; ++b)
        if (ctx->n_seen[b] != 0) return TREEKV_ERR_BAD_STATE;  // keys already cached were encoded by the caller
    if (!dev_cos && !dev_sin) { ctx->cv.rope_cos = nullptr; ctx->cv.rope_sin = nullptr; return TREEKV_OK; }
    if (!dev_cos || !dev_sin || !aligned16(dev_cos) || !aligned16(dev_sin)) return TREEKV_ERR_INVALID_ARG;
    // slots in use: 0 .. budget during decode (the query sits in slot budget), 0 .. budget + chunk - 1 during prefill
    const int need = ctx->cv.c + (ctx->max_chunk > 1 ? ctx->max_chunk : 1);
    if (slots < need) return TREEKV_ERR_INVALID_ARG;
    ctx->cv.rope_cos = dev_cos; ctx->cv.rope_sin = dev_sin;
    return TREEKV_OK;
}

treekv_status treekv_set_option(treekv_ctx* ctx, treekv_option opt, int value) {
    if (!ctx) return TREEKV_ERR_INVALID_ARG;
    switch (opt) {
        case TREEKV_OPT_DECODE_SPLIT:
            if (!(value == 0 || value == 1 || value == 2 || value == 4 || value == 8)) return TREEKV_ERR_INVALID_ARG;
            if (value && decode_smem_for(ctx, value) > kSmemLimit) return TREEKV_ERR_UNSUPPORTED;
            ctx->opt_decode_split = value;
            return TREEKV_OK;
        case TREEKV_OPT_DECODE_PATH:
            if (value < 0 || value > 2) return TREEKV_ERR_INVALID_ARG;
            if (value == 2 && ctx->dt != TREEKV_BF16) return TREEKV_ERR_UNSUPPORTED;
            ctx->opt_decode_path = value;
            ctx->opt_decode_split = 0;
            return TREEKV_OK;
        case TREEKV_OPT_PREFILL_PATH:
            if (value < 0 || value > 3) return TREEKV_ERR_INVALID_ARG;
            if (value >= 2 && !ctx->has_tma) return TREEKV_ERR_UNSUPPORTED;
            ctx->opt_prefill_path = value;
            return TREEKV_OK;
        case TREEKV_OPT_EVICTION_STREAM: {
            if (value < 0 || value > 1) return TREEKV_ERR_INVALID_ARG;
            if (value == 1 && !ctx->side) {
                // Lowest priority: an attention thread block fills an SM's shared memory, so an eviction block never shares
                // an SM with one; the eviction kernel should take the SMs the attention kernel behind it leaves free (a
                // grid smaller than the machine, or the tail of its last wave), not delay that kernel's blocks.
                int lo = 0, hi = 0;
                cudaError_t e = cudaDeviceGetStreamPriorityRange(&lo, &hi);
                cudaStream_t st = nullptr;
                cudaEvent_t ea = nullptr, es = nullptr;
                if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&st, cudaStreamNonBlocking, lo);
                if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ea, cudaEventDisableTiming);
                if (e == cudaSuccess) e = cudaEventCreateWithFlags(&es, cudaEventDisableTiming);
                if (e != cudaSuccess) {
                    if (es) cudaEventDestroy(es);
                    if (ea) cudaEventDestroy(ea);
                    if (st) cudaStreamDestroy(st);
                    return cuda_fail(ctx, e);
                }
                ctx->side = st; ctx->ev_attn = ea; ctx->ev_state = es;
            } else if (value == 0 && ctx->side) {
                // kernels already on the eviction stream stay ordered through side_pending; later chunks use the caller's
                const cudaError_t e = cudaStreamSynchronize(ctx->side);
                cudaEventDestroy(ctx->ev_attn);
                cudaEventDestroy(ctx->ev_state);
                cudaStreamDestroy(ctx->side);
                ctx->side = nullptr; ctx->ev_attn = nullptr; ctx->ev_state = nullptr; ctx->side_pending = false;
                if (e != cudaSuccess) return cuda_fail(ctx, e);
            }
            return TREEKV_OK;
        }
        case TREEKV_OPT_PREFILL_KEY_SPLIT:
            if (value < 0 || value > 3) return TREEKV_ERR_INVALID_ARG;
            ctx->opt_prefill_key_split = value;
            return TREEKV_OK;
        case TREEKV_OPT_PREFILL_APPEND:
            if (value < 0 || value > 1) return TREEKV_ERR_INVALID_ARG;
            ctx->opt_prefill_append = value;
            return TREEKV_OK;
    }
    return TREEKV_ERR_INVALID_ARG;
}

const char* treekv_status_string(treekv_status s) {
    switch (s) {
        case TREEKV_OK: return "ok";
        case TREEKV_ERR_INVALID_ARG: return "invalid argument";
        case TREEKV_ERR_BAD_STATE: return "call not valid in this state";
        case TREEKV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case TREEKV_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case TREEKV_ERR_CUDA: return "CUDA runtime error";
        case TREEKV_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

const char* treekv_version(void) { return "0.1"; }

}  // extern "C"
