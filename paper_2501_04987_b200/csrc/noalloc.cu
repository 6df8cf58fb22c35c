// treekv_prefill_chunk_static_scratch: the prefill-chunk call for callers that must not allocate.
//
// The regular call keeps its per-call scratch (the partial column sums) in the workspace the caller sized and
// allocated at creation.  This variant runs the kernels that need nothing but global scratch: CUDA-core attention
// and the three-step score update / eviction, whose compaction goes through staging rows.  Some callers can only hand over the
// tensors of the call itself: they run where device allocation is off the table (an inference server that
// froze its memory pool at start-up, a plug-in living inside another framework's allocator, a latency-bound
// loop that cannot afford cudaMalloc's implicit device-wide synchronisation), so whatever scratch a call needs
// has to exist already.  For them this file keeps one fixed scratch area inside the library image itself: a
// file-scope __device__ array, present on every GPU that loads the library from load until exit.
//
// The array's name is only meaningful in device code.  In host code it is a host-side shadow symbol, not a
// device address, so the host asks the runtime for the real address once per device (cudaGetSymbolAddress,
// with that device current) and passes that pointer to the kernels.
#include <string.h>

#include <mutex>

#include "common.cuh"
#include "ctx.cuh"

using namespace treekv;

namespace {

constexpr size_t kStaticScratchBytes = size_t(16) << 20;  // 16 MiB per GPU, the hard limit of this entry point
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices];  // device address of g_static_scratch, per device ordinal; 0 = not looked up yet
std::mutex g_scratch_mutex;         // host threads may make their first calls at the same time

// Device address of the static scratch on the current device.  The first call on a device performs the lookup
// (the runtime loads the module that holds the array at that moment, which is when the device commits its 16 MiB).
cudaError_t static_scratch_address(void** out, int* dev_out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    *dev_out = dev;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" treekv_status treekv_prefill_chunk_static_scratch(treekv_ctx* ctx, const void* dev_q, const void* dev_k,
                                                             const void* dev_v, void* dev_out,
                                                             const int32_t* host_chunk_lens, int chunk_stride,
                                                             void* stream) {
    if (!ctx || !dev_q || !dev_k || !dev_v || !dev_out) return TREEKV_ERR_INVALID_ARG;
    if (!aligned16(dev_q) || !aligned16(dev_k) || !aligned16(dev_v) || !aligned16(dev_out)) return TREEKV_ERR_INVALID_ARG;
    if (ctx->max_chunk == 0) return TREEKV_ERR_BAD_STATE;
    if (chunk_stride < 1) return TREEKV_ERR_INVALID_ARG;
    ChunkLens lens;
    memset(&lens, 0, sizeof(lens));
    int max_m = 0, max_seg = 0;
    for (int b = 0; b < ctx->cv.B; ++b) {
        const int m = host_chunk_lens ? host_chunk_lens[b] : chunk_stride;
        if (m < 0 || m > chunk_stride || m > ctx->max_chunk) return TREEKV_ERR_INVALID_ARG;
        if (ctx->n_seen[b] + m >= 0x7fffffff - 1) return TREEKV_ERR_BAD_STATE;
        lens.m[b] = (uint16_t)m;
        if (m > max_m) max_m = m;
        if (m > 0) {
            const int ns = evict_segment(ctx->n_seen[b], m, ctx->cv, 0).nseg;
            if (ns > max_seg) max_seg = ns;
        }
    }
    if (max_m == 0) return TREEKV_OK;

    // carve this call's scratch out of the static array, sized by the longest chunk of THIS call
    const size_t units = (size_t)ctx->cv.B * ctx->cv.Hkv;
    PrefillScratch ps;
    ps.QT = (max_m * ctx->G + kQTileRows - 1) / kQTileRows;
    ps.n_max = ctx->cv.c + max_m;
    // rows in flight at once: the survivors of a segment, or after a wrap the rows behind the last pair (the
    // protected recent tokens and what is still above budget), which can be more than the chunk itself
    const int stage_rows = max_m + ctx->cv.nr;
    ps.max_chunk = stage_rows;
    ps.window = 0;
    const size_t b_col = up256(units * ps.QT * ps.n_max * sizeof(float));
    const size_t b_row = up256(units * stage_rows * ctx->cv.d * ctx->elem);
    const size_t b_scalar = up256(units * stage_rows * 4);
    if (b_col + 2 * b_row + 2 * b_scalar > kStaticScratchBytes) return TREEKV_ERR_UNSUPPORTED;  // beyond the 16 MiB limit
    if (prefill_simt_smem_bytes(ctx->G, ctx->cv.d, ps.n_max) > 227 * 1024) return TREEKV_ERR_UNSUPPORTED;
    void* base_v = nullptr;
    int dev = -1;
    cudaError_t e = static_scratch_address(&base_v, &dev);
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return TREEKV_ERR_CUDA; }
    // the area is per device: the kernels of this call must run where the context's workspace lives
    if (dev != ctx->device) return TREEKV_ERR_BAD_STATE;
    unsigned char* base = static_cast<unsigned char*>(base_v);
    ps.colsum = reinterpret_cast<float*>(base);
    ps.stage_K = base + b_col;
    ps.stage_V = base + b_col + b_row;
    ps.stage_S = reinterpret_cast<float*>(base + b_col + 2 * b_row);
    ps.stage_pos = reinterpret_cast<int32_t*>(base + b_col + 2 * b_row + b_scalar);
    // Nothing in the scratch has to start at zero: every slot a kernel of this call reads was written earlier in
    // the same call (each query tile writes its whole slice of column sums, each staged row is gathered before it
    // is scattered), so what the previous call left behind is never observed.

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    auto fail = [&](cudaError_t err) { ctx->last_cuda_error = (int)err; return TREEKV_ERR_CUDA; };
    e = join_eviction_stream(ctx, s);
    if (e != cudaSuccess) return fail(e);
    e = launch_chunk_append(ctx->cv, ctx->dt, dev_k, dev_v, lens, chunk_stride, max_m, s);
    if (e != cudaSuccess) return fail(e);
    e = launch_prefill_simt(ctx->cv, ctx->dt, ps, dev_q, dev_out, lens, chunk_stride, max_m, s);
    if (e != cudaSuccess) return fail(e);
    e = launch_chunk_scores(ctx->cv, ps, lens, max_m, s);
    if (e != cudaSuccess) return fail(e);
    ctx->launches += 3;
    for (int seg = 0; seg < max_seg; ++seg) {
        int max_items = 0;
        for (int b = 0; b < ctx->cv.B; ++b) {
            if (!lens.m[b]) continue;
            const EvictSegment sg = evict_segment(ctx->n_seen[b], lens.m[b], ctx->cv, seg);
            if (sg.E + sg.rebase > max_items) max_items = sg.E + sg.rebase;
        }
        e = launch_chunk_evict(ctx->cv, ctx->dt, ps, lens, seg, max_items, s);
        if (e != cudaSuccess) return fail(e);
        ctx->launches += 2;
    }
    e = launch_chunk_finalize(ctx->cv, lens, s);
    if (e != cudaSuccess) return fail(e);
    ctx->launches += 1;
    for (int b = 0; b < ctx->cv.B; ++b) {
        const int64_t before = ctx->n_seen[b];
        ctx->n_seen[b] += lens.m[b];
        const int64_t ev_before = before > ctx->cv.c ? before - ctx->cv.c : 0;
        const int64_t ev_after = ctx->n_seen[b] > ctx->cv.c ? ctx->n_seen[b] - ctx->cv.c : 0;
        ctx->evictions += (uint64_t)(ev_after - ev_before);
    }
    return TREEKV_OK;
}
