// Cache-state kernels of the TreeKV library: initialisation, read-outs in cache order, and the per-chunk
// steps around prefill attention: append, score update (Algorithm 1: S <- S + a, summed over the chunk),
// repeated pair eviction with frozen scores, compaction.
#include <cooperative_groups.h>

#include "common.cuh"
#include "ctx.cuh"

namespace treekv {

// ---------------------------------------------------------------------------------------------------------
__global__ void init_state_kernel(CacheView cv) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t < cv.B * cv.Hkv) { cv.n_seen[t] = 0; cv.w0[t] = 0; }
    if (t == 0) { cv.stats->near_ties = 0ull; cv.stats->error = 0u; cv.stats->pad = 0u; }
}
cudaError_t launch_init_state(const CacheView& cv, cudaStream_t stream) {
    const int units = cv.B * cv.Hkv;
    init_state_kernel<<<(units + 255) / 256, 256, 0, stream>>>(cv);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------
// Retained positions / averaged scores in cache order (live index order).
__global__ void retained_positions_kernel(CacheView cv, int32_t* pos_out, int32_t* count_out) {
    const int unit = blockIdx.x;
    const int N = cv.n_seen[unit];
    const UnitState st = unit_state(N, cv);
    const int32_t* Pc = cv.pos + (size_t)unit * cv.R;
    for (int lam = threadIdx.x; lam < cv.c; lam += blockDim.x)
        pos_out[(size_t)unit * cv.c + lam] = lam < st.L ? Pc[phys_row(lam, st)] : -1;
    if (threadIdx.x == 0) count_out[unit] = st.L;
}
cudaError_t launch_retained_positions(const CacheView& cv, int32_t* pos_out, int32_t* count_out, cudaStream_t stream) {
    retained_positions_kernel<<<cv.B * cv.Hkv, 256, 0, stream>>>(cv, pos_out, count_out);
    return cudaGetLastError();
}

__global__ void scores_kernel(CacheView cv, float* sbar_out) {
    const int unit = blockIdx.x;
    const int N = cv.n_seen[unit];
    const UnitState st = unit_state(N, cv);
    const int32_t* Pc = cv.pos + (size_t)unit * cv.R;
    const float* Sc = cv.S + (size_t)unit * cv.R;
    for (int lam = threadIdx.x; lam < cv.c; lam += blockDim.x) {
        float r = 0.f;
        if (lam < st.L) {
            const int ph = phys_row(lam, st);
            r = __fdiv_rn(Sc[ph], (float)score_count(N, Pc[ph], cv.w0[unit]));  // Algorithm 1: S-bar = S / C
        }
        sbar_out[(size_t)unit * cv.c + lam] = r;
    }
}
cudaError_t launch_scores(const CacheView& cv, float* sbar_out, cudaStream_t stream) {
    scores_kernel<<<cv.B * cv.Hkv, 256, 0, stream>>>(cv, sbar_out);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------
// State image: the live rows of every unit in cache order.  One warp per (unit, slot).
template <typename T, bool kImport>
__global__ void state_image_kernel(CacheView cv, StateImage img) {
    const int unit = blockIdx.y;
    const int b = unit / cv.Hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int lam = blockIdx.x * (blockDim.x >> 5) + warp;
    if (lam >= cv.c) return;
    const int N = kImport ? img.seen[b] : cv.n_seen[unit];
    const UnitState st = unit_state(N, cv);
    const int chunks = cv.d * (int)sizeof(T) / 16;
    const size_t slot = (size_t)unit * cv.c + lam;
    uint4* ki = reinterpret_cast<uint4*>(reinterpret_cast<T*>(img.K) + slot * cv.d);
    uint4* vi = reinterpret_cast<uint4*>(reinterpret_cast<T*>(img.V) + slot * cv.d);
    if (lam < st.L) {
        const size_t row = (size_t)unit * cv.R + phys_row(lam, st);
        uint4* kc = reinterpret_cast<uint4*>(reinterpret_cast<T*>(cv.K) + row * cv.d);
        uint4* vc = reinterpret_cast<uint4*>(reinterpret_cast<T*>(cv.V) + row * cv.d);
        if (kImport) {
            for (int e = lane; e < chunks; e += 32) { kc[e] = ki[e]; vc[e] = vi[e]; }
            if (lane == 0) { cv.S[row] = img.S[slot]; cv.pos[row] = img.pos[slot]; }
        } else {
            for (int e = lane; e < chunks; e += 32) { ki[e] = kc[e]; vi[e] = vc[e]; }
            if (lane == 0) { img.S[slot] = cv.S[row]; img.pos[slot] = cv.pos[row]; }
        }
    } else if (!kImport) {
        for (int e = lane; e < chunks; e += 32) { ki[e] = make_uint4(0, 0, 0, 0); vi[e] = make_uint4(0, 0, 0, 0); }
        if (lane == 0) { img.S[slot] = 0.f; img.pos[slot] = -1; }
    }
    if (lam == 0 && lane == 0) {
        if (kImport) { cv.n_seen[unit] = N; cv.w0[unit] = img.w0[b]; }
        else if (unit % cv.Hkv == 0) { img.seen[b] = N; img.w0[b] = cv.w0[unit]; }
    }
}
template <bool kImport>
static cudaError_t launch_state_image(const CacheView& cv, treekv_dtype dt, const StateImage& img, cudaStream_t stream) {
    dim3 grid((cv.c + 7) / 8, cv.B * cv.Hkv);
    if (dt == TREEKV_F32) state_image_kernel<float, kImport><<<grid, 256, 0, stream>>>(cv, img);
    else state_image_kernel<__nv_bfloat16, kImport><<<grid, 256, 0, stream>>>(cv, img);
    return cudaGetLastError();
}
cudaError_t launch_export_state(const CacheView& cv, treekv_dtype dt, const StateImage& img, cudaStream_t stream) {
    return launch_state_image<false>(cv, dt, img, stream);
}
cudaError_t launch_import_state(const CacheView& cv, treekv_dtype dt, const StateImage& img, cudaStream_t stream) {
    return launch_state_image<true>(cv, dt, img, stream);
}

// ---------------------------------------------------------------------------------------------------------
// Chunk append: chunk token t of sequence b goes to physical row L + i + t of every KV head's slab.
// One warp per (token, unit); k,v are [B][chunk_stride][Hkv][d].
template <typename T>
__global__ void chunk_append_kernel(CacheView cv, const T* __restrict__ k, const T* __restrict__ v, ChunkLens lens,
                                    int chunk_stride) {
    pdl_trigger();
    pdl_wait();
    const int unit = blockIdx.y;
    const int b = unit / cv.Hkv, kh = unit % cv.Hkv;
    const int m = lens.m[b];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + warp;
    if (t >= m) return;
    const int N = cv.n_seen[unit];
    const UnitState st = unit_state(N, cv);
    const int row = st.L + st.i + t;
    const int chunks = cv.d * (int)sizeof(T) / 16;
    const uint4* ks = reinterpret_cast<const uint4*>(k + (((size_t)b * chunk_stride + t) * cv.Hkv + kh) * cv.d);
    const uint4* vs = reinterpret_cast<const uint4*>(v + (((size_t)b * chunk_stride + t) * cv.Hkv + kh) * cv.d);
    uint4* kd = reinterpret_cast<uint4*>(reinterpret_cast<T*>(cv.K) + ((size_t)unit * cv.R + row) * cv.d);
    uint4* vd = reinterpret_cast<uint4*>(reinterpret_cast<T*>(cv.V) + ((size_t)unit * cv.R + row) * cv.d);
    for (int e = lane; e < chunks; e += 32) { kd[e] = ks[e]; vd[e] = vs[e]; }
    if (lane == 0) {
        cv.pos[(size_t)unit * cv.R + row] = N + t;
        cv.S[(size_t)unit * cv.R + row] = 0.f;
    }
}
cudaError_t launch_chunk_append(const CacheView& cv, treekv_dtype dt, const void* k, const void* v, const ChunkLens& lens,
                                int chunk_stride, int max_m, cudaStream_t stream) {
    dim3 grid((max_m + 7) / 8, cv.B * cv.Hkv);
    if (dt == TREEKV_F32)
        return launch_pdl(chunk_append_kernel<float>, grid, dim3(256), 0, stream, cv, (const float*)k, (const float*)v, lens,
                          chunk_stride);
    return launch_pdl(chunk_append_kernel<__nv_bfloat16>, grid, dim3(256), 0, stream, cv, (const __nv_bfloat16*)k,
                      (const __nv_bfloat16*)v, lens, chunk_stride);
}

// ---------------------------------------------------------------------------------------------------------
// In-cache positions (Section 4.1 "Position Encoding") for the tensor-core prefill kernels, whose operands go from
// memory to the tensor cores without passing through registers: after the chunk has been appended, every live row of
// a unit - cache slot lam, physical row phys_row(lam) - is encoded at position lam into the rotated-key slab (same row),
// and every query row of the chunk at its own slot L + t.  Same arithmetic as rope_apply() / the oracle.  The slab is
// rebuilt on every call because evictions move tokens to other slots; it costs one read and one write of the unit's
// keys against two passes of attention over them.  bf16, head_dim 128.  One half-warp per row.
__global__ void rope_chunk_kernel(CacheView cv, ChunkLens lens, int chunk_stride, __nv_bfloat16* __restrict__ k_rot,
                                  const __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ q_rot) {
    constexpr int D = 128, CPR = 16;
    const int unit = blockIdx.y;
    const int b = unit / cv.Hkv, kh = unit % cv.Hkv;
    const int m = lens.m[b];
    if (m == 0) return;
    const int G = cv.Hq / cv.Hkv;
    const int N = cv.n_seen[unit];
    const UnitState st = unit_state(N, cv);
    const int n = st.L + m;
    const int hw = (blockIdx.x * blockDim.x + threadIdx.x) >> 4, cidx = threadIdx.x & 7;  // half-warp index; piece pair (cidx, cidx + 8)
    const bool second = (threadIdx.x >> 3) & 1;  // the half-warp's upper eight lanes take the next row
    const int item = 2 * hw + (second ? 1 : 0);
    if (item < n) {  // a key row
        const int lam = item;
        const size_t row = (size_t)unit * cv.R + phys_row(lam, st);
        const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(cv.K) + row * D);
        uint4* dst = reinterpret_cast<uint4*>(k_rot + row * D);
        uint4 a = src[cidx], c2 = src[cidx + CPR / 2];
        rope_piece_pair(a, c2, cv.rope_cos + (size_t)lam * (D / 2) + cidx * 8, cv.rope_sin + (size_t)lam * (D / 2) + cidx * 8);
        dst[cidx] = a; dst[cidx + CPR / 2] = c2;
    } else if (item < n + m * G) {  // a query row of the chunk: token t, head h of the group
        const int r = item - n, t = r / G, h = r % G;
        const size_t qo = (((size_t)b * chunk_stride + t) * cv.Hq + kh * G + h) * D;
        const uint4* src = reinterpret_cast<const uint4*>(q + qo);
        uint4* dst = reinterpret_cast<uint4*>(q_rot + qo);
        const int slot = st.L + t;
        uint4 a = src[cidx], c2 = src[cidx + CPR / 2];
        rope_piece_pair(a, c2, cv.rope_cos + (size_t)slot * (D / 2) + cidx * 8, cv.rope_sin + (size_t)slot * (D / 2) + cidx * 8);
        dst[cidx] = a; dst[cidx + CPR / 2] = c2;
    }
}
cudaError_t launch_rope_chunk(const CacheView& cv, const ChunkLens& lens, int chunk_stride, int max_m, void* k_rot,
                              const void* q, void* q_rot, cudaStream_t stream) {
    const int G = cv.Hq / cv.Hkv;
    const int items = cv.c + max_m + max_m * G;      // key rows + query rows of a unit, at most
    dim3 grid((items * 8 + 255) / 256, cv.B * cv.Hkv);  // eight lanes per item
    rope_chunk_kernel<<<grid, 256, 0, stream>>>(cv, lens, chunk_stride, reinterpret_cast<__nv_bfloat16*>(k_rot),
                                                reinterpret_cast<const __nv_bfloat16*>(q), reinterpret_cast<__nv_bfloat16*>(q_rot));
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------
// Chunk score update: S[row(lam)] += (sum over query tiles of the partial column sums) / G, tiles added in
// a fixed order so the result does not depend on scheduling.
__global__ void chunk_scores_kernel(CacheView cv, PrefillScratch ps, ChunkLens lens) {
    pdl_trigger();  // launched in plain stream order itself; the eviction kernel behind it may be scheduled early
    const int unit = blockIdx.y;
    const int b = unit / cv.Hkv;
    const int m = lens.m[b];
    if (m == 0) return;
    const int G = cv.Hq / cv.Hkv;
    const int N = cv.n_seen[unit];
    const UnitState st = unit_state(N, cv);
    const int n = st.L + m;
    const int lam = blockIdx.x * blockDim.x + threadIdx.x;
    if (lam >= n) return;
    const int qt = (m * G + kQTileRows - 1) / kQTileRows;
    const float* part = ps.colsum + (size_t)unit * ps.QT * ps.n_max + lam;
    float s = 0.f;
    for (int t = 0; t < qt; ++t) s += part[(size_t)t * ps.n_max];
    float* Sp = cv.S + (size_t)unit * cv.R + phys_row(lam, st);
    *Sp = *Sp + s * (1.0f / (float)G);  // chunk rows were zeroed by the append
}
cudaError_t launch_chunk_scores(const CacheView& cv, const PrefillScratch& ps, const ChunkLens& lens, int max_m,
                                cudaStream_t stream) {
    const int n_up = cv.c + max_m;
    dim3 grid((n_up + 255) / 256, cv.B * cv.Hkv);
    chunk_scores_kernel<<<grid, 256, 0, stream>>>(cv, ps, lens);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------
// Chunk eviction, one segment (see EvictSegment).  Algorithm 1's "length > c" branch repeated with frozen
// averaged scores: between two wraps of idx the scopes are disjoint, so all pairs of a segment are decided
// at once.  The survivor of pair p must land on row ns+i+p, which can be a source row of an earlier pair, so the
// move goes through staging rows: gather (decide + copy out), then scatter (copy in) as a second launch.
template <typename T>
__global__ void chunk_evict_gather_kernel(CacheView cv, PrefillScratch ps, ChunkLens lens, int seg) {
    pdl_trigger();
    pdl_wait();
    const int unit = blockIdx.y;
    const int b = unit / cv.Hkv;
    const int m = lens.m[b];
    if (m == 0) return;
    const int N = cv.n_seen[unit];
    const EvictSegment sg = evict_segment(N, m, cv, seg);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int item = blockIdx.x * (blockDim.x >> 5) + warp;
    if (item >= sg.E + sg.rebase) return;
    const int N1 = N + m;
    T* Kc = reinterpret_cast<T*>(cv.K) + (size_t)unit * cv.R * cv.d;
    T* Vc = reinterpret_cast<T*>(cv.V) + (size_t)unit * cv.R * cv.d;
    const float* Sc = cv.S + (size_t)unit * cv.R;
    const int32_t* Pc = cv.pos + (size_t)unit * cv.R;
    int src;
    if (item < sg.E) {
        const int l = cv.ns + 2 * (sg.i + item), r = l + 1;
        int evict_right = 0;
        if (lane == 0) {
            bool near_tie = false;
            const int w0 = cv.w0[unit];
            evict_right = pair_evicts_right(Sc[l], score_count(N1, Pc[l], w0), Sc[r], score_count(N1, Pc[r], w0), cv.rule,
                                            &near_tie) ? 1 : 0;
            if (near_tie) atomicAdd(&cv.stats->near_ties, 1ull);
        }
        evict_right = __shfl_sync(0xffffffffu, evict_right, 0);
        src = evict_right ? l : r;
    } else {
        src = cv.ns + 2 * cv.cm + (item - sg.E);
    }
    const int chunks = cv.d * (int)sizeof(T) / 16;
    const size_t so = ((size_t)unit * ps.max_chunk + item);
    uint4* kd = reinterpret_cast<uint4*>(reinterpret_cast<T*>(ps.stage_K) + so * cv.d);
    uint4* vd = reinterpret_cast<uint4*>(reinterpret_cast<T*>(ps.stage_V) + so * cv.d);
    const uint4* ks = reinterpret_cast<const uint4*>(Kc + (size_t)src * cv.d);
    const uint4* vs = reinterpret_cast<const uint4*>(Vc + (size_t)src * cv.d);
    for (int e = lane; e < chunks; e += 32) { kd[e] = ks[e]; vd[e] = vs[e]; }
    if (lane == 0) { ps.stage_S[so] = Sc[src]; ps.stage_pos[so] = Pc[src]; }
}

template <typename T>
__global__ void chunk_evict_scatter_kernel(CacheView cv, PrefillScratch ps, ChunkLens lens, int seg) {
    pdl_trigger();
    pdl_wait();
    const int unit = blockIdx.y;
    const int b = unit / cv.Hkv;
    const int m = lens.m[b];
    if (m == 0) return;
    const int N = cv.n_seen[unit];
    const EvictSegment sg = evict_segment(N, m, cv, seg);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int item = blockIdx.x * (blockDim.x >> 5) + warp;
    if (item >= sg.E + sg.rebase) return;
    const int dst = cv.ns + (item < sg.E ? sg.i + item : cv.cm + (item - sg.E));
    const int chunks = cv.d * (int)sizeof(T) / 16;
    const size_t so = ((size_t)unit * ps.max_chunk + item);
    const uint4* ks = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(ps.stage_K) + so * cv.d);
    const uint4* vs = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(ps.stage_V) + so * cv.d);
    uint4* kd = reinterpret_cast<uint4*>(reinterpret_cast<T*>(cv.K) + ((size_t)unit * cv.R + dst) * cv.d);
    uint4* vd = reinterpret_cast<uint4*>(reinterpret_cast<T*>(cv.V) + ((size_t)unit * cv.R + dst) * cv.d);
    for (int e = lane; e < chunks; e += 32) { kd[e] = ks[e]; vd[e] = vs[e]; }
    if (lane == 0) {
        cv.S[(size_t)unit * cv.R + dst] = ps.stage_S[so];
        cv.pos[(size_t)unit * cv.R + dst] = ps.stage_pos[so];
    }
}

cudaError_t launch_chunk_evict(const CacheView& cv, treekv_dtype dt, const PrefillScratch& ps, const ChunkLens& lens,
                               int seg, int max_items, cudaStream_t stream) {
    if (max_items <= 0) return cudaSuccess;
    dim3 grid((max_items + 7) / 8, cv.B * cv.Hkv);
    cudaError_t e;
    if (dt == TREEKV_F32) {
        e = launch_pdl(chunk_evict_gather_kernel<float>, grid, dim3(256), 0, stream, cv, ps, lens, seg);
        if (e == cudaSuccess) e = launch_pdl(chunk_evict_scatter_kernel<float>, grid, dim3(256), 0, stream, cv, ps, lens, seg);
    } else {
        e = launch_pdl(chunk_evict_gather_kernel<__nv_bfloat16>, grid, dim3(256), 0, stream, cv, ps, lens, seg);
        if (e == cudaSuccess)
            e = launch_pdl(chunk_evict_scatter_kernel<__nv_bfloat16>, grid, dim3(256), 0, stream, cv, ps, lens, seg);
    }
    return e;
}

// ---------------------------------------------------------------------------------------------------------
// The three steps above in one launch: score update, every eviction segment of the chunk, n_seen += m.
// A unit is owned by a cluster of CL thread blocks: four blocks of 512 threads when the kernel runs in the caller's
// stream, where its latency counts (the barriers are cluster barriers), or one block of 1024 threads when it runs on
// the context's eviction stream beside the next attention kernel, where a small footprint counts (block barriers).  Inside a segment the pairs are taken in rounds of
// increasing pair index; a round first reads everything it moves into registers (decision, survivor's K and V
// rows, its S and position), the cluster synchronises, then the round writes.  That is enough because the
// destination row i+p of pair p can only be a source row of an earlier pair ((p-i)/2 < p) - read in this round
// or a previous one - and never of a later pair; rows moved down after a wrap follow the same rule.  A new
// segment starts after a further cluster barrier, since its pairs read rows the previous one wrote.
constexpr int evict_threads(int cl) { return cl == 1 ? 1024 : 512; }
constexpr int kEvictItemsPerWarp = 4;

template <typename T, int kEvictCluster>
__global__ void __launch_bounds__(evict_threads(kEvictCluster))
chunk_update_evict_kernel(CacheView cv, PrefillScratch ps, ChunkLens lens) {
    constexpr int kEvictThreads = evict_threads(kEvictCluster);
    pdl_trigger();
    pdl_wait();
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    auto unit_sync = [&]() { if (kEvictCluster == 1) __syncthreads(); else cluster.sync(); };
    // a block (cluster) takes the units blockIdx.y, blockIdx.y + gridDim.y, ...: one each unless the launch asked for
    // fewer blocks than units
    for (int unit = blockIdx.y; unit < cv.B * cv.Hkv; unit += gridDim.y) {
    const int b = unit / cv.Hkv;
    const int m = lens.m[b];
    if (m == 0) continue;  // the whole cluster shares the unit
    const int rank = (int)cluster.block_rank();
    const int G = cv.Hq / cv.Hkv;
    const int N = cv.n_seen[unit];
    const UnitState st = unit_state(N, cv);
    const int n = st.L + m;
    const int N1 = N + m;
    const int w0 = cv.w0[unit];
    T* Kc = reinterpret_cast<T*>(cv.K) + (size_t)unit * cv.R * cv.d;
    T* Vc = reinterpret_cast<T*>(cv.V) + (size_t)unit * cv.R * cv.d;
    float* Sc = cv.S + (size_t)unit * cv.R;
    int32_t* Pc = cv.pos + (size_t)unit * cv.R;

    // ---- score update (Algorithm 1: S <- S + a, summed over the chunk's steps; group mean): tiles added in a
    //      fixed order so the result does not depend on scheduling
    {
        const int qt = (m * G + kQTileRows - 1) / kQTileRows;
        const float inv_g = 1.0f / (float)G;
        for (int lam = rank * kEvictThreads + threadIdx.x; lam < n; lam += kEvictCluster * kEvictThreads) {
            const float* part = ps.colsum + (size_t)unit * ps.QT * ps.n_max + lam;
            float s = 0.f;
            for (int t = 0; t < qt; ++t) s += part[(size_t)t * ps.n_max];
            float* Sp = Sc + phys_row(lam, st);
            *Sp = *Sp + s * inv_g;  // chunk rows were zeroed by the append
        }
    }
    unit_sync();  // every S of the unit is final; every block has read n_seen
    if (rank == 0 && threadIdx.x == 0) cv.n_seen[unit] = N1;

    // ---- eviction segments (Algorithm 1's "length > c" branch repeated with the scores frozen)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gwarp = rank * (kEvictThreads / 32) + warp;
    constexpr int kWarps = kEvictCluster * kEvictThreads / 32;
    constexpr int kRound = kWarps * kEvictItemsPerWarp;
    const int chunks = cv.d * (int)sizeof(T) / 16;  // 16-byte pieces per row: at most 32
    const int nseg = evict_segment(N, m, cv, 0).nseg;
    for (int seg = 0; seg < nseg; ++seg) {
        const EvictSegment sg = evict_segment(N, m, cv, seg);
        const int items = sg.E + sg.rebase;
        for (int r0 = 0; r0 < items; r0 += kRound) {
            uint4 kr[kEvictItemsPerWarp], vr[kEvictItemsPerWarp];
            float sr[kEvictItemsPerWarp];
            int32_t pr[kEvictItemsPerWarp];
#pragma unroll
            for (int u = 0; u < kEvictItemsPerWarp; ++u) {
                const int item = r0 + u * kWarps + gwarp;
                if (item >= items) continue;
                int src;
                if (item < sg.E) {
                    const int l = cv.ns + 2 * (sg.i + item), r = l + 1;
                    int evict_right = 0;
                    if (lane == 0) {
                        bool near_tie = false;
                        evict_right = pair_evicts_right(Sc[l], score_count(N1, Pc[l], w0), Sc[r], score_count(N1, Pc[r], w0),
                                                        cv.rule, &near_tie) ? 1 : 0;
                        if (near_tie) atomicAdd(&cv.stats->near_ties, 1ull);
                    }
                    evict_right = __shfl_sync(0xffffffffu, evict_right, 0);
                    src = evict_right ? l : r;
                } else {
                    src = cv.ns + 2 * cv.cm + (item - sg.E);
                }
                if (lane < chunks) {
                    kr[u] = reinterpret_cast<const uint4*>(Kc + (size_t)src * cv.d)[lane];
                    vr[u] = reinterpret_cast<const uint4*>(Vc + (size_t)src * cv.d)[lane];
                }
                if (lane == 0) { sr[u] = Sc[src]; pr[u] = Pc[src]; }
            }
            unit_sync();  // everything this round moves has been read
#pragma unroll
            for (int u = 0; u < kEvictItemsPerWarp; ++u) {
                const int item = r0 + u * kWarps + gwarp;
                if (item >= items) continue;
                const int dst = cv.ns + (item < sg.E ? sg.i + item : cv.cm + (item - sg.E));
                if (lane < chunks) {
                    reinterpret_cast<uint4*>(Kc + (size_t)dst * cv.d)[lane] = kr[u];
                    reinterpret_cast<uint4*>(Vc + (size_t)dst * cv.d)[lane] = vr[u];
                }
                if (lane == 0) { Sc[dst] = sr[u]; Pc[dst] = pr[u]; }
            }
        }
        if (seg + 1 < nseg) unit_sync();  // the next segment's pairs read rows this one wrote
    }
    }
}

template <typename T, int CL>
static cudaError_t launch_chunk_update_evict_t(const CacheView& cv, const PrefillScratch& ps, const ChunkLens& lens,
                                               int max_blocks, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    const int units = cv.B * cv.Hkv;
    cfg.gridDim = dim3(CL, max_blocks > 0 && max_blocks < units ? max_blocks : units);
    cfg.blockDim = dim3(evict_threads(CL));
    cfg.stream = stream;  // plain stream order behind the attention kernel; the kernel after it may be scheduled early
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CL;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = CL > 1 ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, chunk_update_evict_kernel<T, CL>, cv, ps, lens);
}

cudaError_t launch_chunk_update_evict(const CacheView& cv, treekv_dtype dt, const PrefillScratch& ps, const ChunkLens& lens,
                                      bool small_footprint, cudaStream_t stream) {
    return small_footprint ? launch_chunk_update_evict_beside(cv, dt, ps, lens, 0, stream)
                           : (dt == TREEKV_F32 ? launch_chunk_update_evict_t<float, 4>(cv, ps, lens, 0, stream)
                                               : launch_chunk_update_evict_t<__nv_bfloat16, 4>(cv, ps, lens, 0, stream));
}

// The form that runs beside another kernel (eviction stream): one block of 1024 threads per unit, at most max_blocks
// blocks (0 = one per unit), each then taking several units in turn.
cudaError_t launch_chunk_update_evict_beside(const CacheView& cv, treekv_dtype dt, const PrefillScratch& ps,
                                             const ChunkLens& lens, int max_blocks, cudaStream_t stream) {
    return dt == TREEKV_F32 ? launch_chunk_update_evict_t<float, 1>(cv, ps, lens, max_blocks, stream)
                            : launch_chunk_update_evict_t<__nv_bfloat16, 1>(cv, ps, lens, max_blocks, stream);
}

// ---------------------------------------------------------------------------------------------------------
// One-shot, block-level prefill of an empty cache (Section 4.2 of the paper), the part after the attention: the
// prompt's m tokens sit in rows [0, m); the attention kernel left the column sums of the observation window (the
// last `bs` tokens) per query tile.  This kernel adds them to S (Algorithm 1's S update for the window's rows; the
// counter C of a token is the number of window rows that see it, kept implicitly through w0 = m - bs), then plays
// Algorithm 1's "length > c" branch on blocks of bs tokens, a block standing for one token: a block's score
// is the mean of its tokens' S / C, the cache holds c / bs blocks, and the cycle-coordinate layout applies to
// block rows (block r = token rows [r bs, (r+1) bs)), so that the final token rows are exactly the token-level
// layout at cycle position ((m - c) mod c).  Per segment: one warp per pair decides (decisions go to the unit's
// column-sum scratch, free by then), cluster barrier, then the rows move in rounds as in the kernel above.
template <typename T>
__global__ void __cluster_dims__(4, 1, 1) __launch_bounds__(evict_threads(4))
oneshot_update_evict_kernel(CacheView cv, PrefillScratch ps, ChunkLens lens, int bs) {
    constexpr int kEvictCluster = 4, kEvictThreads = evict_threads(4);
    pdl_trigger();
    pdl_wait();
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    auto unit_sync = [&]() { if (kEvictCluster == 1) __syncthreads(); else cluster.sync(); };
    const int unit = blockIdx.y;
    const int b = unit / cv.Hkv;
    const int m = lens.m[b];
    if (m == 0) return;  // the whole cluster shares the unit
    const int rank = (int)cluster.block_rank();
    const int G = cv.Hq / cv.Hkv;
    const int wstart = m - bs;  // first token of the observation window; also the step at which scoring starts
    T* Kc = reinterpret_cast<T*>(cv.K) + (size_t)unit * cv.R * cv.d;
    T* Vc = reinterpret_cast<T*>(cv.V) + (size_t)unit * cv.R * cv.d;
    float* Sc = cv.S + (size_t)unit * cv.R;
    int32_t* Pc = cv.pos + (size_t)unit * cv.R;
    float* scratch = ps.colsum + (size_t)unit * ps.QT * ps.n_max;

    // ---- S of every prompt token = group mean of the window's column sums; only the query tiles that hold window
    //      rows are added, in tile order
    {
        const int qt = (m * G + kQTileRows - 1) / kQTileRows;
        const int tile0 = (wstart * G) / kQTileRows;
        const float inv_g = 1.0f / (float)G;
        for (int lam = rank * kEvictThreads + threadIdx.x; lam < m; lam += kEvictCluster * kEvictThreads) {
            const float* part = scratch + lam;
            float s = 0.f;
            for (int t = tile0; t < qt; ++t) s += part[(size_t)t * ps.n_max];
            Sc[lam] = Sc[lam] + s * inv_g;  // the append left S = 0
        }
    }
    unit_sync();  // every S of the unit is final, the column sums have been consumed
    if (rank == 0 && threadIdx.x == 0) { cv.n_seen[unit] = m; cv.w0[unit] = wstart; }

    // ---- Algorithm 1 on blocks
    CacheView blk = cv;  // geometry in block units: a cache of c / bs blocks, nothing protected
    blk.c = cv.c / bs; blk.cm = blk.c; blk.ns = 0; blk.nr = 0;
    const int nb = m / bs, cb = blk.c;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gwarp = rank * (kEvictThreads / 32) + warp;
    constexpr int kWarps = kEvictCluster * kEvictThreads / 32;
    constexpr int kRound = kWarps * kEvictItemsPerWarp;
    const int chunks = cv.d * (int)sizeof(T) / 16;
    int* dec = reinterpret_cast<int*>(scratch);  // [pairs of the segment] 1 = the right block goes
    const float inv_bs = 1.0f / (float)bs;
    const bool accumulated = cv.rule == TREEKV_RULE_ACCUMULATED;
    auto block_score = [&](int brow) {  // mean of S / C (of S: accumulated rule) over the block's tokens, in a fixed order
        float a = 0.f;
        for (int t = lane; t < bs; t += 32) {
            const int row = brow * bs + t;
            a += accumulated ? Sc[row] : __fdiv_rn(Sc[row], (float)score_count(m, Pc[row], wstart));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        return a * inv_bs;
    };
    const int nseg = evict_segment(0, nb, blk, 0).nseg;
    for (int seg = 0; seg < nseg; ++seg) {
        const EvictSegment sg = evict_segment(0, nb, blk, seg);
        for (int p = gwarp; p < sg.E; p += kWarps) {
            const int lb = 2 * (sg.i + p), rb = lb + 1;
            const float sl = block_score(lb), sr = block_score(rb);
            if (lane == 0) {
                int evict_right;
                if (cv.rule == TREEKV_RULE_KEEP_LEFT) evict_right = 1;
                else if (cv.rule == TREEKV_RULE_EVICT_LEFT) evict_right = 0;
                else {
                    const float mx = fmaxf(fabsf(sl), fabsf(sr));
                    if (!(fabsf(sl - sr) >= kNearTieRel * mx)) atomicAdd(&cv.stats->near_ties, 1ull);
                    evict_right = sl > sr ? 1 : 0;  // strict: ties evict the left (older) block
                }
                dec[p] = evict_right;
            }
        }
        unit_sync();  // the segment's decisions are visible to the whole cluster
        const int items = (sg.E + sg.rebase) * bs;  // token rows to move
        for (int r0 = 0; r0 < items; r0 += kRound) {
            uint4 kr[kEvictItemsPerWarp], vr[kEvictItemsPerWarp];
            float sr[kEvictItemsPerWarp];
            int32_t pr[kEvictItemsPerWarp];
#pragma unroll
            for (int u = 0; u < kEvictItemsPerWarp; ++u) {
                const int item = r0 + u * kWarps + gwarp;
                if (item >= items) continue;
                const int ib = item / bs, t = item - ib * bs;
                const int sb = ib < sg.E ? 2 * (sg.i + ib) + (dec[ib] ? 0 : 1) : 2 * cb + (ib - sg.E);
                const int src = sb * bs + t;
                if (lane < chunks) {
                    kr[u] = reinterpret_cast<const uint4*>(Kc + (size_t)src * cv.d)[lane];
                    vr[u] = reinterpret_cast<const uint4*>(Vc + (size_t)src * cv.d)[lane];
                }
                if (lane == 0) { sr[u] = Sc[src]; pr[u] = Pc[src]; }
            }
            unit_sync();  // everything this round moves has been read
#pragma unroll
            for (int u = 0; u < kEvictItemsPerWarp; ++u) {
                const int item = r0 + u * kWarps + gwarp;
                if (item >= items) continue;
                const int ib = item / bs, t = item - ib * bs;
                const int db = ib < sg.E ? sg.i + ib : cb + (ib - sg.E);
                const int dst = db * bs + t;
                if (lane < chunks) {
                    reinterpret_cast<uint4*>(Kc + (size_t)dst * cv.d)[lane] = kr[u];
                    reinterpret_cast<uint4*>(Vc + (size_t)dst * cv.d)[lane] = vr[u];
                }
                if (lane == 0) { Sc[dst] = sr[u]; Pc[dst] = pr[u]; }
            }
        }
        if (seg + 1 < nseg) unit_sync();  // the next segment's pairs read rows (and overwrite decisions) of this one
    }
}

cudaError_t launch_oneshot_update_evict(const CacheView& cv, treekv_dtype dt, const PrefillScratch& ps, const ChunkLens& lens,
                                        int block, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(4, cv.B * cv.Hkv);
    cfg.blockDim = dim3(evict_threads(4));
    cfg.stream = stream;
    if (dt == TREEKV_F32) return cudaLaunchKernelEx(&cfg, oneshot_update_evict_kernel<float>, cv, ps, lens, block);
    return cudaLaunchKernelEx(&cfg, oneshot_update_evict_kernel<__nv_bfloat16>, cv, ps, lens, block);
}

__global__ void chunk_finalize_kernel(CacheView cv, ChunkLens lens) {
    pdl_trigger();
    pdl_wait();
    const int unit = blockIdx.x * blockDim.x + threadIdx.x;
    if (unit < cv.B * cv.Hkv) cv.n_seen[unit] += lens.m[unit / cv.Hkv];
}
cudaError_t launch_chunk_finalize(const CacheView& cv, const ChunkLens& lens, cudaStream_t stream) {
    const int units = cv.B * cv.Hkv;
    return launch_pdl(chunk_finalize_kernel, dim3((units + 255) / 256), dim3(256), 0, stream, cv, lens);
}

}  // namespace treekv
