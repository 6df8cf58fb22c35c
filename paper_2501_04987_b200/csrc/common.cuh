// Shared declarations of the TreeKV CUDA library: cache geometry, parameter blocks, small device helpers.
//
// Cache geometry ("cycle coordinates").  Algorithm 1 of the TreeKV paper evicts from the scope {idx, idx+1}
// with idx cycling 1..c.  During one cycle of c evictions the scopes are the disjoint pairs (2p, 2p+1),
// p = 0..c-1 (0-based), of the sequence [cache at cycle start | tokens appended during the cycle].  Each unit
// (sequence, KV head) therefore owns a slab of R = 2c + max_chunk rows whose physical row index is the index
// in that sequence: the survivor of pair p is moved to row p and nothing else ever moves.  With i evictions
// done in the current cycle (i = idx - 1) and L cached tokens the live rows are
//     [0, i)  and  [2i, L + i)            (both in stream order, the first entirely older than the second)
// and the next token is appended at row L + i.  While the cache is still filling, i = 0 and the live rows
// are [0, L).  "Live index" lambda in [0, L) maps to the physical row  lambda < i ? lambda : lambda + i.
//
// Protected tokens (Section 5.2 of the paper keeps 4 initial and 508 recent tokens beside 512 selected ones): the
// first n_sink tokens of the stream and the newest n_recent cached tokens are never in a scope, and Algorithm 1
// runs on the c_mid = c - n_sink - n_recent slots between them.  In the slab the sinks are rows [0, n_sink) and
// the cycle sequence [middle region at cycle start | every later token] starts at row n_sink: pairs are rows
// (n_sink + 2p, n_sink + 2p + 1), p = 0..c_mid-1, the survivor of pair p moves to row n_sink + p, and the live
// rows are
//     [0, a)  and  [a + i, L + i)     with the split point a = n_sink + i
// - again two contiguous segments; without protection a = i and this is the layout above.  When a cycle ends
// (i reaches c_mid) the n_recent rows that follow the last pair, [n_sink + 2 c_mid, ...), are moved down to
// [n_sink + c_mid, ...) so that the next cycle starts from a contiguous cache ("re-base").
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/treekv.h"

namespace treekv {

constexpr int kMaxBatch = 1024;
constexpr float kNearTieRel = 1e-4f;
constexpr float kLog2e = 1.4426950408889634f;

// device counters, one block per context
struct DevStats {
    unsigned long long near_ties;
    unsigned int error;
    unsigned int pad;
};

// geometry + slab pointers, passed by value to every kernel
struct CacheView {
    void* K;          // [units][R][d]
    void* V;          // [units][R][d]
    float* S;         // [units][R]   sum of attention received
    int32_t* pos;     // [units][R]   0-based stream index of the token in the row
    int32_t* n_seen;  // [units]      tokens fed so far (kept per unit so a kernel only reads what it alone writes)
    int32_t* w0;      // [units]      stream step at which scoring started: C_j = tokens seen - max(pos_j, w0); 0 = Algorithm 1
    DevStats* stats;
    int c;            // budget
    int R;            // rows per slab
    int Hq, Hkv, B, d;
    int rule;
    int ns;           // protected initial tokens (sinks)
    int nr;           // protected newest tokens (recent window)
    int cm;           // c - ns - nr: slots Algorithm 1 runs on = evictions per cycle
    const float* rope_cos;  // in-cache positions (Section 4.1 "Position Encoding"): cos / sin by cache slot,
    const float* rope_sin;  // [slots][d/2] fp32, caller-owned; nullptr = the library is position-agnostic
};

struct ActiveMask {
    uint32_t w[kMaxBatch / 32];
    __host__ __device__ bool test(int b) const { return (w[b >> 5] >> (b & 31)) & 1u; }
};

// cache state derived from the number of tokens seen
struct UnitState {
    int L;  // cached tokens
    int i;  // evictions done in the current cycle (idx - 1)
    int a;  // split point n_sink + i: live indices below it sit at row = index, the others at index + i
};
__host__ __device__ inline UnitState unit_state(long long n_seen, int c, int cm, int ns) {
    UnitState s;
    if (n_seen <= c) { s.L = (int)n_seen; s.i = 0; }
    else { s.L = c; s.i = (int)((n_seen - c) % cm); }
    s.a = ns + s.i;
    return s;
}
__host__ __device__ inline UnitState unit_state(long long n_seen, const CacheView& cv) {
    return unit_state(n_seen, cv.c, cv.cm, cv.ns);
}
__host__ __device__ inline int phys_row(int lambda, const UnitState& st) { return lambda < st.a ? lambda : lambda + st.i; }

// One segment of a chunk's eviction: E pairs (ns + 2(i+p), ns + 2(i+p) + 1) -> row ns + i + p, then, if the cycle
// wraps, the `rebase` rows that follow the last pair, [ns + 2 cm, ns + 2 cm + rebase), move down to
// [ns + cm, ns + cm + rebase): the protected recent tokens and whatever is still above budget.
struct EvictSegment {
    int i;       // cycle position at segment start
    int len;     // live rows at segment start
    int E;       // evictions in this segment
    int rebase;  // rows moved down after a wrap
    int nseg;    // total number of segments for this chunk
};
__host__ __device__ inline EvictSegment evict_segment(long long n_seen_before, int m, const CacheView& cv, int seg) {
    const int c = cv.c, cm = cv.cm;
    UnitState st = unit_state(n_seen_before, cv);
    EvictSegment cur;
    cur.i = st.i; cur.len = st.L + m; cur.E = 0; cur.rebase = 0; cur.nseg = 0;
    int i = st.i, len = st.L + m;
    int s = 0;
    while (len > c) {
        const int E = len - c < cm - i ? len - c : cm - i;
        const int len2 = len - E;
        int i2 = i + E, rebase = 0;
        if (i2 == cm) { i2 = 0; rebase = len2 - (cv.ns + cm); }
        if (s == seg) { cur.i = i; cur.len = len; cur.E = E; cur.rebase = rebase; }
        i = i2; len = len2; ++s;
    }
    cur.nseg = s;
    if (seg >= s) { cur.E = 0; cur.rebase = 0; }
    return cur;
}

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kVec = 4;  // elements per 16-byte load
    __device__ static void unpack(const uint4& u, float (&f)[4]) {
        f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y); f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
    }
    __device__ static float to_float(float x) { return x; }
    __device__ static float from_float(float x) { return x; }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kVec = 8;
    __device__ static void unpack(const uint4& u, float (&f)[8]) {
        f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xffff0000u);
        f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xffff0000u);
        f[4] = __uint_as_float(u.z << 16); f[5] = __uint_as_float(u.z & 0xffff0000u);
        f[6] = __uint_as_float(u.w << 16); f[7] = __uint_as_float(u.w & 0xffff0000u);
    }
    __device__ static float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
    __device__ static __nv_bfloat16 from_float(float x) { return __float2bfloat16_rn(x); }
};

// 128-bit streaming load of a cache row: served from L2, no L1 allocation.  Deliberately not the non-coherent
// (.nc) form: the kernel that streams a slab also writes rows of it (the appended token, the survivor's move), and
// .nc is only defined for data nobody writes while the kernel runs.
__device__ inline uint4 ld_stream(const void* p) {
    uint4 r;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ inline uint4 ld_plain(const void* p) { return *reinterpret_cast<const uint4*>(p); }

// Algorithm 1's counter C of the token at stream position `pos` once `n_seen` tokens have been fed: the steps in
// which the token was scored.  That is every step since its arrival, except after a one-shot prefill, where the
// tokens older than the observation window were only scored from the window's first query (w0) on.
__host__ __device__ inline int score_count(int n_seen, int pos, int w0) { return n_seen - (pos > w0 ? pos : w0); }

// Algorithm 1's comparison on the averaged scores (on the accumulated ones under TREEKV_RULE_ACCUMULATED); returns true when the right member of the pair is evicted.
// Also reports whether the decision was a near-tie (relative gap below kNearTieRel).
__device__ inline bool pair_evicts_right(float S_l, int C_l, float S_r, int C_r, int rule, bool* near_tie) {
    *near_tie = false;
    if (rule == TREEKV_RULE_KEEP_LEFT) return true;
    if (rule == TREEKV_RULE_EVICT_LEFT) return false;
    const bool acc = rule == TREEKV_RULE_ACCUMULATED;  // the sums themselves instead of the averages
    const float a = acc ? S_l : __fdiv_rn(S_l, (float)C_l);
    const float b = acc ? S_r : __fdiv_rn(S_r, (float)C_r);
    const float mx = fmaxf(fabsf(a), fabsf(b));
    *near_tie = !(fabsf(a - b) >= kNearTieRel * mx);
    return a > b;  // strict: ties and NaN evict the left (older) slot
}

// In-cache positions: x (this lane's slice of a row spread over LPR lanes, VEC elements each) encoded at `slot`.
// Rotate-half pairing (t, t + d/2): the partner element sits LPR/2 lanes away.  Numeric contract: two fp32
// operations per output, x1' = fma(x1, cos, -(x2 sin)), x2' = fma(x2, cos, x1 sin), then rounding to the cache's
// element type - as a model that keeps rotated keys in the cache dtype would produce them.  Every lane of the warp
// must call this (shuffles); `slot` must be a valid table row for every lane.
#ifdef __CUDACC__
template <typename T, int D>
__device__ inline void rope_apply(float (&f)[Elem<T>::kVec], int slot, int sub, const float* cos_tab, const float* sin_tab) {
    constexpr int VEC = Elem<T>::kVec, LPR = D / VEC, HL = LPR / 2;
    const bool lower = sub < HL;
    const float* cs = cos_tab + (size_t)slot * (D / 2) + (sub % HL) * VEC;
    const float* sn = sin_tab + (size_t)slot * (D / 2) + (sub % HL) * VEC;
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
        const float partner = __shfl_xor_sync(0xffffffffu, f[e], HL);
        const float ps = __fmul_rn(partner, __ldg(sn + e));
        const float y = __fmaf_rn(f[e], __ldg(cs + e), lower ? -ps : ps);
        f[e] = Elem<T>::to_float(Elem<T>::from_float(y));
    }
}
#endif

#ifdef __CUDACC__
__device__ inline uint32_t rope_pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// In-cache positions (Section 4.1 "Position Encoding"): 16-byte piece c (8 channels, c < D/16) of a row and its
// rotate-half partner piece c + D/16, encoded at `slot`, with the numeric contract of rope_apply() in common.cuh:
// x1' = fma(x1, cos, -(x2 sin)), x2' = fma(x2, cos, x1 sin) in fp32, each rounded to bf16.
// cos / sin of eight consecutive channels (two float4 each), as loaded from the tables
struct RopeTab {
    float4 c0, c1, s0, s1;
};
__device__ inline RopeTab rope_tab_load(const float* cos_row, const float* sin_row) {
    RopeTab t;
    t.c0 = __ldg(reinterpret_cast<const float4*>(cos_row));
    t.c1 = __ldg(reinterpret_cast<const float4*>(cos_row) + 1);
    t.s0 = __ldg(reinterpret_cast<const float4*>(sin_row));
    t.s1 = __ldg(reinterpret_cast<const float4*>(sin_row) + 1);
    return t;
}
__device__ inline void rope_piece_pair(uint4& lo, uint4& hi, const RopeTab& t) {
    float a[8], b[8];
    Elem<__nv_bfloat16>::unpack(lo, a);
    Elem<__nv_bfloat16>::unpack(hi, b);
    const float cs[8] = {t.c0.x, t.c0.y, t.c0.z, t.c0.w, t.c1.x, t.c1.y, t.c1.z, t.c1.w};
    const float sn[8] = {t.s0.x, t.s0.y, t.s0.z, t.s0.w, t.s1.x, t.s1.y, t.s1.z, t.s1.w};
    float ya[8], yb[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        ya[e] = __fmaf_rn(a[e], cs[e], -__fmul_rn(b[e], sn[e]));
        yb[e] = __fmaf_rn(b[e], cs[e], __fmul_rn(a[e], sn[e]));
    }
    lo = make_uint4(rope_pack_bf16(ya[0], ya[1]), rope_pack_bf16(ya[2], ya[3]), rope_pack_bf16(ya[4], ya[5]), rope_pack_bf16(ya[6], ya[7]));
    hi = make_uint4(rope_pack_bf16(yb[0], yb[1]), rope_pack_bf16(yb[2], yb[3]), rope_pack_bf16(yb[4], yb[5]), rope_pack_bf16(yb[6], yb[7]));
}
__device__ inline void rope_piece_pair(uint4& lo, uint4& hi, const float* cos_row, const float* sin_row) {
    rope_piece_pair(lo, hi, rope_tab_load(cos_row, sin_row));
}
#endif

// chunk length of every sequence in a prefill call (0 = not in the call), passed by value
struct ChunkLens {
    uint16_t m[kMaxBatch];
};

// per-call scratch of chunked prefill, carved from the context's workspace
struct PrefillScratch {
    float* colsum;    // [units][QT][n_max] partial column sums of the chunk's probability matrix, one slice per
                      // tile of 128 query rows (row = token * G + head), indexed by live index
    void* stage_K;    // [units][max_chunk][d] rows in flight during compaction
    void* stage_V;    // [units][max_chunk][d]
    float* stage_S;   // [units][max_chunk]
    int32_t* stage_pos;  // [units][max_chunk]
    int QT;           // tiles per unit: ceil(G * max_chunk / 128)
    int n_max;        // c + max_chunk
    int max_chunk;
    int window;       // 0: every query row of the chunk adds to the column sums (Algorithm 1 per row); > 0: only the
                      // last `window` tokens of each sequence's chunk do (observation window of the one-shot prefill)
};
constexpr int kQTileRows = 128;  // query rows (token x head-in-group) per prefill tile

// ---- programmatic dependent launch.  A kernel launched with launch_pdl may be scheduled while the kernel before
// it in the stream is still running; it calls pdl_wait() before it reads or writes anything of the cache or the
// scratch, which returns once every earlier kernel in the stream has completed and its writes are visible, and
// pdl_trigger() (first statement) lets the kernel after it be scheduled in turn.  Launch latency and block
// scheduling thereby overlap the predecessor's tail.  Every block waits, also one that then finds nothing to
// do, so that the order of the chain stays transitive.  Launched without the attribute, both are no-ops.
#ifdef __CUDACC__
__device__ inline void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ inline void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
#endif

// ---- launchers implemented in the .cu files (each enqueues on `stream` and returns the launch status)
size_t decode_smem_bytes(int G, int D, int c, int split);
cudaError_t launch_decode(const CacheView& cv, treekv_dtype dt, const void* q, const void* k, const void* v, void* out,
                          const ActiveMask& active, int split, cudaStream_t stream);

size_t decode_mma_smem_bytes(int G, int D, int c, int split);
// inputs_final: q, k, v held their final values before the launch (they may then be read ahead of the stream-order wait)
cudaError_t launch_decode_mma(const CacheView& cv, const void* q, const void* k, const void* v, void* out,
                              const ActiveMask& active, int split, int inputs_final, cudaStream_t stream);

cudaError_t launch_init_state(const CacheView& cv, cudaStream_t stream);
// state image in cache order (see treekv_export_state): pointers into the caller's buffer
struct StateImage {
    void* K;
    void* V;
    float* S;
    int32_t* pos;
    int32_t* seen;  // [B]
    int32_t* w0;    // [B] stream step at which scoring started (0 unless the sequence was prefilled in one shot)
};
cudaError_t launch_export_state(const CacheView& cv, treekv_dtype dt, const StateImage& img, cudaStream_t stream);
cudaError_t launch_import_state(const CacheView& cv, treekv_dtype dt, const StateImage& img, cudaStream_t stream);
cudaError_t launch_retained_positions(const CacheView& cv, int32_t* pos_out, int32_t* count_out, cudaStream_t stream);
cudaError_t launch_scores(const CacheView& cv, float* sbar_out, cudaStream_t stream);
cudaError_t launch_chunk_append(const CacheView& cv, treekv_dtype dt, const void* k, const void* v, const ChunkLens& lens,
                                int chunk_stride, int max_m, cudaStream_t stream);
cudaError_t launch_chunk_scores(const CacheView& cv, const PrefillScratch& ps, const ChunkLens& lens, int max_m,
                                cudaStream_t stream);
cudaError_t launch_chunk_evict(const CacheView& cv, treekv_dtype dt, const PrefillScratch& ps, const ChunkLens& lens,
                               int seg, int max_items, cudaStream_t stream);  // gather + scatter: two launches
cudaError_t launch_chunk_finalize(const CacheView& cv, const ChunkLens& lens, cudaStream_t stream);
// score update + every eviction segment + n_seen update of a chunk in one launch; small_footprint: one large block
// per unit instead of a cluster of four (for running beside another kernel)
cudaError_t launch_chunk_update_evict(const CacheView& cv, treekv_dtype dt, const PrefillScratch& ps, const ChunkLens& lens,
                                      bool small_footprint, cudaStream_t stream);

// In-cache positions for the tensor-core prefill: the unit's live rows (cache and appended chunk) encoded at their slots
// into the rotated-key slab k_rot (same geometry as the K slab), and the chunk's queries, encoded at their own slots,
// into q_rot (may be q itself)
cudaError_t launch_rope_chunk(const CacheView& cv, const ChunkLens& lens, int chunk_stride, int max_m, void* k_rot,
                              const void* q, void* q_rot, cudaStream_t stream);

// one-shot prefill of an empty cache: scores from the observation window, block means, Algorithm 1 on blocks
cudaError_t launch_oneshot_update_evict(const CacheView& cv, treekv_dtype dt, const PrefillScratch& ps, const ChunkLens& lens,
                                        int block, cudaStream_t stream);

size_t prefill_simt_smem_bytes(int G, int D, int n_max);
cudaError_t launch_prefill_simt(const CacheView& cv, treekv_dtype dt, const PrefillScratch& ps, const void* q, void* out,
                                const ChunkLens& lens, int chunk_stride, int max_m, cudaStream_t stream);

// The chunk's k and v tensors with tensor maps over them, when the tensor-core prefill kernels read their chunk tiles
// from there and append the chunk themselves (k == nullptr: an append kernel put the rows into the slab first).
struct ChunkTensors {
    const void* k;
    const void* v;
    CUtensorMap tmK, tmV;  // channels x KV heads x tokens of the call, box 64 x 1 x 128
};

size_t prefill_tc2_smem_bytes();
cudaError_t launch_prefill_tc2(const CacheView& cv, const PrefillScratch& ps, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                               const CUtensorMap& tmV, const ChunkTensors& ct, void* out, const ChunkLens& lens,
                               int chunk_stride, int max_m, int n_whole_clusters, cudaStream_t stream);
// 256 query rows per CTA.  n_whole_clusters < 0: one CTA per tile pair; else two-CTA clusters, the first n_whole_clusters
// with one tile pair per CTA, the others splitting a pair's key tiles

size_t prefill_tc_smem_bytes();
cudaError_t launch_prefill_tc(const CacheView& cv, const PrefillScratch& ps, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                              const CUtensorMap& tmV, const ChunkTensors& ct, void* out, const ChunkLens& lens,
                              int chunk_stride, int max_m, cudaStream_t stream);

}  // namespace treekv
