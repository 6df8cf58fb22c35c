// Decode step of TreeKV for bf16 caches (Algorithm 1, one loop iteration; attention of Section 3.1), one launch.
//
// Same contract as decode.cu, built for bandwidth with grouped queries: a cluster of `split` CTAs owns one
// unit (sequence, KV head); inside a CTA every warp runs a private pipeline
//     cp.async (16-byte, L2-only) of 16 K rows + 16 V rows into its ring of shared-memory stages
//  -> ldmatrix -> mma.sync m16n8k16 for q.K^T of all G heads of the group at once
//  -> online softmax in registers (running max, lazy rescale)
//  -> ldmatrix.trans -> mma.sync for P.V with P taken straight from the logits' accumulator registers.
// K and V are read from HBM exactly once, there is no block-wide barrier inside the streaming loop, and the
// instruction count per byte does not grow with the group size (the G query heads ride in the N=8 / M=16
// dimensions of the MMA tiles).  Logits are kept in shared memory; every CTA pushes its (max, sum) to all CTAs
// of the cluster and its partial output to CTA 0 with remote shared-memory stores, so that after one cluster
// barrier each CTA can write the exact normalised probabilities' group mean into S and CTA 0 can write the
// output.  CTA 0 then plays Algorithm 1's eviction branch.
#include <algorithm>

#include <cooperative_groups.h>

#include "common.cuh"
#include "tma.cuh"

namespace cg = cooperative_groups;

namespace treekv {

namespace {

__device__ inline uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ inline void cp_async_16(uint32_t dst, const void* src, bool valid) {
    const int sz = valid ? 16 : 0;  // src-size 0: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
// the same copy for data that is read once: its L2 lines are the first to be replaced
__device__ inline void cp_async_16_stream(uint32_t dst, const void* src, bool valid, uint64_t policy) {
    const int sz = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2, %3;" ::"r"(dst), "l"(src), "r"(sz), "l"(policy) : "memory");
}
__device__ inline uint64_t l2_evict_first_policy() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ inline void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ inline void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ inline void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ inline void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ inline void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ inline uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// bulk L2 prefetch of a 16-byte aligned range whose size is a multiple of 16
__device__ inline void l2_prefetch(const void* p, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}
// 2^x in one special-function instruction (about 2 ulp; arguments here are <= 0, results below 2^-126 flush to zero)
__device__ inline float ex2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// 2^(a-b) with the convention 2^(-inf - anything) = 0, so empty partials (max = -inf) never produce NaN
__device__ inline float exp2_diff(float a, float b) { return a == -INFINITY ? 0.f : ex2_fast(a - b); }

constexpr int kBlk = 16;      // keys per pipeline stage
constexpr int kPrefetchRows = 256;  // rows of K and of V a CTA asks L2 for before its stream-order wait (0 = none)
constexpr int kMaxSplit = 8;  // largest cluster
constexpr int kMmaWarps = 4;
constexpr int kMmaStages = 2;

int mma_rows_cap(int c, int split) {
    const int nblk_all = (c + 1 + kBlk - 1) / kBlk;
    return ((nblk_all + split - 1) / split) * kBlk;
}

}  // namespace

template <int D, int G, int NW, int NS, bool ROPE>
__global__ void __launch_bounds__(NW * 32)
decode_mma_kernel(CacheView cv, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k_in,
                  const __nv_bfloat16* __restrict__ v_in, __nv_bfloat16* __restrict__ out, ActiveMask active,
                  int rows_cap, int inputs_final) {
    using T = __nv_bfloat16;
    constexpr int NT = NW * 32;
    constexpr int ROWB = D * 2;             // bytes per row
    constexpr int CPR = ROWB / 16;          // 16-byte chunks per row
    constexpr int STAGE = 2 * kBlk * ROWB;  // K block + V block
    constexpr int CHUNKS = D * 2 / 16;

    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int nsplit = (int)cluster.num_blocks();
    const int kh = blockIdx.y, b = blockIdx.z;
    // Programmatic dependent launch: the next kernel in the stream may be scheduled while this one runs (it does
    // the same), and nothing below the wait is read before the previous kernel's writes are complete and visible.
    pdl_trigger();
    const int unit = b * cv.Hkv + kh;
    const T* k_new = k_in + (size_t)unit * D;
    const T* v_new = v_in + (size_t)unit * D;

    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char* ring = smem_raw;                                        // [NW][NS][STAGE]
    float* sl = reinterpret_cast<float*>(ring + (size_t)NW * NS * STAGE);  // [G][rows_cap] logits (log2 units)
    float* wstat = sl + (size_t)G * rows_cap;                              // [NW+1][2][G] per-warp (max, sum); slot NW = new token
    float* gstat = wstat + (NW + 1) * 2 * G;                               // [nsplit][2][G] every CTA's (max, sum), pushed by its owner
    float* o_all = gstat + kMaxSplit * 2 * G;                              // [nsplit][G][D] partial outputs, pushed into CTA 0 only
    float* s_old = o_all + (size_t)nsplit * G * D;                         // [rows_cap] S of this CTA's rows, prefetched
    unsigned char* pair_kv = reinterpret_cast<unsigned char*>(                   // [4][ROWB] K,V of the scope's two rows
        (reinterpret_cast<uintptr_t>(s_old + rows_cap) + 15) & ~uintptr_t(15));
    float* pair_s = reinterpret_cast<float*>(pair_kv + 4 * ROWB);          // [2] updated S of rows 2i, 2i+1 (split == 1)
    unsigned char* tok = pair_kv + 4 * ROWB + 16;                          // [G+2][ROWB] this step's q heads, k, v
    float* o_warp = reinterpret_cast<float*>(ring);                        // [NW][G][D], aliases the ring after the loop

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const float scale = kLog2e * rsqrtf((float)D);

    // ---- this step's inputs go to shared memory once per CTA (warp 0, one commit group of their own): the q rows of
    //      the group's heads and the new key and value rows.  Everything that needs them reads the copy, so q, k, v
    //      are fetched once, early, whether they live in HBM or in page-locked host memory.  When the caller
    //      guarantees that the inputs held their final values before the launch (host tensors filled by the CPU),
    //      the fetch starts before the stream-order wait and its latency hides behind the previous kernel's tail.
    // They come as three bulk copies (the group's q rows are contiguous; one row each of k and v) that signal an
    // mbarrier: across the bus a bulk copy travels as a few large read requests instead of one per 16-byte piece.
    __shared__ __align__(8) uint64_t in_bar;
    if (tid == 0) { mbar_init(smem_addr_u32(&in_bar), 1); mbar_fence_init(); }
    __syncwarp();
    auto stage_inputs = [&]() {  // warp 0
        if (lane == 0) {
            const T* qrow = q + ((size_t)b * cv.Hq + kh * G) * D;
            const uint32_t bar = smem_addr_u32(&in_bar);
            mbar_arrive_expect_tx(bar, (G + 2) * ROWB);
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_u32(tok)), "l"(qrow), "r"(G * ROWB), "r"(bar) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_u32(tok + G * ROWB)), "l"(k_new), "r"(ROWB), "r"(bar) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_u32(tok + (G + 1) * ROWB)), "l"(v_new), "r"(ROWB), "r"(bar) : "memory");
        }
    };
    if (inputs_final && warp == 0 && active.test(b)) stage_inputs();
    // While the previous kernel of the stream drains, ask L2 for the first rows this CTA will stream.  This is a hint
    // and nothing more: the token count is read before the wait and may be one step old (the rows then shift by one),
    // no data reaches a register, and L2 is the point of coherence, so a line that the previous kernel still writes
    // is simply up to date when it is read after the wait.
    if (kPrefetchRows > 0 && threadIdx.x == 0 && active.test(b)) {
        int Ns;
        asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(Ns) : "l"(cv.n_seen + unit));
        if (Ns >= 0) {
            const UnitState ss = unit_state(Ns, cv);
            const int blk_all = (ss.L + 1 + kBlk - 1) / kBlk, per = (blk_all + nsplit - 1) / nsplit;
            const int lo_s = min(rank * per * kBlk, ss.L), hi_s = min(min(lo_s + per * kBlk, ss.L), lo_s + kPrefetchRows);
            const unsigned char* Kb = reinterpret_cast<const unsigned char*>(cv.K) + (size_t)unit * cv.R * ROWB;
            const unsigned char* Vb = reinterpret_cast<const unsigned char*>(cv.V) + (size_t)unit * cv.R * ROWB;
            const int a1 = min(hi_s, max(lo_s, ss.a));  // live indices [lo_s, a1) sit at row = index, [a1, hi_s) at index + i
            if (a1 > lo_s) {
                l2_prefetch(Kb + (size_t)lo_s * ROWB, (uint32_t)(a1 - lo_s) * ROWB);
                l2_prefetch(Vb + (size_t)lo_s * ROWB, (uint32_t)(a1 - lo_s) * ROWB);
            }
            if (hi_s > a1) {
                l2_prefetch(Kb + (size_t)(a1 + ss.i) * ROWB, (uint32_t)(hi_s - a1) * ROWB);
                l2_prefetch(Vb + (size_t)(a1 + ss.i) * ROWB, (uint32_t)(hi_s - a1) * ROWB);
            }
        }
    }
    pdl_wait();  // every block waits, also one of an inactive sequence
    if (!active.test(b)) return;  // the whole cluster shares b
    // Remote shared-memory stores below need every CTA of the cluster to have started.  Arrive here (relaxed: nothing
    // is published yet) and wait just before the first remote store; the whole streaming loop lies between the two,
    // so the barrier costs nothing.  A cluster of one has no remote stores and stays barrier-free.
    if (nsplit > 1) asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");

    const int N = cv.n_seen[unit];
    const UnitState st = unit_state(N, cv);
    const int n = st.L + 1;  // live rows including the token appended by this step
    const int i_cyc = st.i;
    const int a_cyc = st.a;          // live indices below it sit at row = index, the others at index + i_cyc
    const int row_l = a_cyc + i_cyc; // the scope {idx, idx+1} is physical rows (row_l, row_l + 1); the survivor moves to a_cyc
    // rows are dealt to the cluster in whole 16-key blocks
    const int nblk_all = (n + kBlk - 1) / kBlk;
    const int blk_per = (nblk_all + nsplit - 1) / nsplit;
    const int lo = min(rank * blk_per * kBlk, n), hi = min(lo + blk_per * kBlk, n);
    const int nrows = hi - lo;
    const bool owns_new = (hi == n) && nrows > 0;
    const int nblk = (nrows - (owns_new ? 1 : 0) + kBlk - 1) / kBlk;  // tiles of cached rows; the new token is merged separately

    T* Kc = reinterpret_cast<T*>(cv.K) + (size_t)unit * cv.R * D;
    T* Vc = reinterpret_cast<T*>(cv.V) + (size_t)unit * cv.R * D;
    float* Sc = cv.S + (size_t)unit * cv.R;
    int32_t* Pc = cv.pos + (size_t)unit * cv.R;
    const int new_row = st.L + i_cyc;

    if (!inputs_final && warp == 0) stage_inputs();

    const uint32_t ring_w = smem_u32(ring) + warp * NS * STAGE;
    // Copy of one 16-row block: lane (half = lane / CPR... ) moves 16-byte chunk `cidx` of rows rsub*(16/RPI) + it.
    // Shared-memory layout of a tile: row r at r * ROWB, its 16-byte chunk c at position c ^ (r & 7).
    constexpr int RPI = 32 / CPR;          // rows copied per warp-wide cp.async (2 for d=128, 4 for d=64)
    constexpr int ITERS = kBlk / RPI;      // iterations per tile (8 or 4)
    const int c_rsub = lane / CPR, c_cidx = lane % CPR;
    const uint32_t c_lane_off = c_rsub * ITERS * ROWB;  // lane's first row = rsub * ITERS
    const int c_row7 = (c_rsub * ITERS) & 7;            // (row & 7) of iteration `it` is c_row7 + it (no carry)
    const uint64_t stream_policy = l2_evict_first_policy();  // K and V rows are read once per step
    auto issue = [&](int blk, int stage) {
        if (blk < nblk) {
            const uint32_t kst = ring_w + stage * STAGE, vst = kst + kBlk * ROWB;
            const int lam0 = lo + blk * kBlk;
            // fast path: all 16 rows exist, none is the new token, and they are consecutive physical rows
            const bool whole = (lam0 + kBlk <= hi) && (lam0 + kBlk <= n - 1) && (lam0 >= a_cyc || lam0 + kBlk <= a_cyc);
            if (whole) {
                const size_t r0 = (size_t)phys_row(lam0, st) + c_rsub * ITERS;
                const unsigned char* ks = reinterpret_cast<const unsigned char*>(Kc) + r0 * ROWB + c_cidx * 16;
                const unsigned char* vs = reinterpret_cast<const unsigned char*>(Vc) + r0 * ROWB + c_cidx * 16;
#pragma unroll
                for (int it = 0; it < ITERS; ++it) {
                    const uint32_t off = c_lane_off + it * ROWB + ((c_cidx ^ (c_row7 + it)) << 4);
                    cp_async_16_stream(kst + off, ks + it * ROWB, true, stream_policy);
                    cp_async_16_stream(vst + off, vs + it * ROWB, true, stream_policy);
                }
            } else {
#pragma unroll
                for (int it = 0; it < ITERS; ++it) {
                    const int row = c_rsub * ITERS + it;
                    const int lam = lam0 + row;
                    const bool valid = lam < hi && lam != n - 1;  // the new token is merged separately
                    const size_t ro = valid ? (size_t)phys_row(lam, st) * ROWB : 0;
                    const uint32_t off = c_lane_off + it * ROWB + ((c_cidx ^ (c_row7 + it)) << 4);
                    cp_async_16_stream(kst + off, reinterpret_cast<const unsigned char*>(Kc) + ro + c_cidx * 16, valid, stream_policy);
                    cp_async_16_stream(vst + off, reinterpret_cast<const unsigned char*>(Vc) + ro + c_cidx * 16, valid, stream_policy);
                }
            }
        }
        cp_async_commit();
    };
    // ---- prefetch what the epilogue needs, so that after the streaming loop nothing waits on a global load:
    //      S of this CTA's rows (4-byte cp.async; they join the first commit group), and in CTA 0 the K/V rows of
    //      the eviction scope (rows row_l and row_l + 1; the new token's row comes from k_in / v_in)
    const bool will_evict = (N + 1 > cv.c);
    int pos_l = 0, pos_r = 0, w0 = 0;  // stream positions of the scope's two tokens (used by lane 0 of warp 0 in CTA 0)
    if (rank == 0 && will_evict && tid == 0) {
        pos_l = Pc[row_l];
        pos_r = (row_l + 1 == new_row) ? N : Pc[row_l + 1];
        w0 = cv.w0[unit];
    }
    for (int j = tid; j < nrows; j += NT) {
        const int lam = lo + j;
        if (lam != n - 1)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(s_old + j)), "l"(Sc + phys_row(lam, st)) : "memory");
    }
    if (rank == 0 && will_evict && warp == NW - 1) {
        for (int e = lane; e < 4 * CPR; e += 32) {
            const int which = e / CPR, cidx = e % CPR;   // 0: K left, 1: K right, 2: V left, 3: V right
            const int prow = row_l + (which & 1);
            if (prow == new_row) continue;  // the appended row is taken from the staged inputs below
            const T* srcrow = ((which < 2) ? Kc : Vc) + (size_t)prow * D;
            cp_async_16(smem_u32(pair_kv + which * ROWB + cidx * 16), reinterpret_cast<const unsigned char*>(srcrow) + cidx * 16, true);
        }
    }
#pragma unroll
    for (int s = 0; s < NS; ++s) issue(warp + s * NW, s);

    // the staged inputs have landed (bounded wait; a give-up is recorded and the step's result is then meaningless)
    if (warp == 0 && !mbar_wait(smem_addr_u32(&in_bar), 0) && lane == 0) atomicOr(&cv.stats->error, 128u);
    __syncthreads();
    const T* tq = reinterpret_cast<const T*>(tok);
    const T* tk = reinterpret_cast<const T*>(tok + G * ROWB);
    const T* tv = reinterpret_cast<const T*>(tok + (G + 1) * ROWB);
    // in-cache positions: the query sits in the last slot, n - 1; its staged rows are encoded in place.  Keys stay as
    // given in the cache and are encoded at their slot in shared memory, tile by tile, below.
    constexpr bool rope = ROPE;  // in-cache positions: a kernel of its own (it keeps the next tile's cos / sin in registers)
    if (rope) {
        for (int e = tid; e < G * (CPR / 2); e += NT) {
            const int r = e / (CPR / 2), cidx = e % (CPR / 2);
            uint4* plo = reinterpret_cast<uint4*>(tok + r * ROWB) + cidx;
            uint4* phi = plo + CPR / 2;
            uint4 a = *plo, bq = *phi;
            rope_piece_pair(a, bq, cv.rope_cos + (size_t)(n - 1) * (D / 2) + cidx * 8, cv.rope_sin + (size_t)(n - 1) * (D / 2) + cidx * 8);
            *plo = a; *phi = bq;
        }
        __syncthreads();
    }

    // ---- append (Algorithm 1: K <- K u {k}, V <- V u {v}); the step itself uses the staged copy of the new token
    if (warp == NW - 1) {
        if (owns_new) {
            for (int e = lane; e < CHUNKS; e += 32) {
                reinterpret_cast<uint4*>(Kc + (size_t)new_row * D)[e] = reinterpret_cast<const uint4*>(tk)[e];
                reinterpret_cast<uint4*>(Vc + (size_t)new_row * D)[e] = reinterpret_cast<const uint4*>(tv)[e];
            }
        }
        if (rank == 0 && will_evict && new_row == row_l + 1) {  // the scope's right row is the appended one
            for (int e = lane; e < CHUNKS; e += 32) {
                reinterpret_cast<uint4*>(pair_kv + 1 * ROWB)[e] = reinterpret_cast<const uint4*>(tk)[e];
                reinterpret_cast<uint4*>(pair_kv + 3 * ROWB)[e] = reinterpret_cast<const uint4*>(tv)[e];
            }
        }
    }

    // ---- the new token's logit q.k_new (warp 0 of the owning CTA)
    if (warp == 0) {
        float sn[G];
#pragma unroll
        for (int h = 0; h < G; ++h) sn[h] = -INFINITY;
        if (owns_new) {
            // this lane's channels of the new key (lane, lane + 32, ...): with in-cache positions encoded at slot n - 1,
            // channel e < D/2 pairing with e + D/2, which the same lane holds
            float kn[D / 32];
#pragma unroll
            for (int u = 0; u < D / 32; ++u) kn[u] = __bfloat162float(tk[lane + 32 * u]);
            if (rope) {
#pragma unroll
                for (int u = 0; u < D / 64; ++u) {
                    const int e = lane + 32 * u;  // < D/2
                    const float cs = __ldg(cv.rope_cos + (size_t)(n - 1) * (D / 2) + e), sv = __ldg(cv.rope_sin + (size_t)(n - 1) * (D / 2) + e);
                    const float x1 = kn[u], x2 = kn[u + D / 64];
                    kn[u] = __bfloat162float(__float2bfloat16_rn(__fmaf_rn(x1, cs, -__fmul_rn(x2, sv))));
                    kn[u + D / 64] = __bfloat162float(__float2bfloat16_rn(__fmaf_rn(x2, cs, __fmul_rn(x1, sv))));
                }
            }
#pragma unroll
            for (int h = 0; h < G; ++h) {
                float a = 0.f;
#pragma unroll
                for (int u = 0; u < D / 32; ++u) a += __bfloat162float(tq[h * D + lane + 32 * u]) * kn[u];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
                sn[h] = a * scale;
            }
        }
        if (lane == 0) {
#pragma unroll
            for (int h = 0; h < G; ++h) {
                wstat[(NW * 2 + 0) * G + h] = sn[h];
                wstat[(NW * 2 + 1) * G + h] = owns_new ? 1.f : 0.f;
            }
        }
    }

    // ---- A fragments of q: row g = head, k = channel; rows >= G are zero
    uint32_t qa[D / 16][2];
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
        qa[kk][0] = 0u; qa[kk][1] = 0u;
        if (g < G) {
            const T* qh = tq + g * D + 16 * kk + 2 * t;
            qa[kk][0] = *reinterpret_cast<const uint32_t*>(qh);
            qa[kk][1] = *reinterpret_cast<const uint32_t*>(qh + 8);
        }
    }

    // per-lane ldmatrix offsets inside a K tile (4 matrices = 8 keys x 32 channels) and a V tile (4 matrices = 16 keys
    // x 16 channels), swizzle included; the row half hb adds 8 rows
    uint32_t koff[D / 32], voff[D / 16];
#pragma unroll
    for (int u = 0; u < D / 32; ++u) {
        const int row = lane & 7, cidx = 4 * u + (lane >> 3);
        koff[u] = row * ROWB + ((cidx ^ row) << 4);
    }
#pragma unroll
    for (int cc = 0; cc < D / 16; ++cc) {
        const int row = (lane & 7) + ((lane >> 4) << 3), cidx = 2 * cc + ((lane >> 3) & 1);
        voff[cc] = row * ROWB + ((cidx ^ (row & 7)) << 4);
    }

    float m_run = -INFINITY, l_run = 0.f;  // of head g (replicated over the 4 lanes t; l_run is a per-lane partial)
    float acc[D / 16][4];
#pragma unroll
    for (int cc = 0; cc < D / 16; ++cc)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[cc][e] = 0.f;

    // In-cache positions: the cos / sin values a lane needs for a tile (piece pairs (c, c + CPR/2) of rows, eight lanes
    // per row) are fetched into registers one tile ahead, right after the previous tile has been encoded, so their
    // latency hides behind that tile's MMAs.
    constexpr int kRopeItems = kBlk * (CPR / 2) / 32;
    RopeTab tab[ROPE ? kRopeItems : 1];
    auto load_tabs = [&](int blk) {
#pragma unroll
        for (int i2 = 0; i2 < (ROPE ? kRopeItems : 0); ++i2) {
            const int item = lane + 32 * i2, r = item / (CPR / 2), cidx = item % (CPR / 2);
            const int slot = min(lo + blk * kBlk + r, n - 1);
            tab[i2] = rope_tab_load(cv.rope_cos + (size_t)slot * (D / 2) + cidx * 8, cv.rope_sin + (size_t)slot * (D / 2) + cidx * 8);
        }
    };
    if (rope && warp < nblk) load_tabs(warp);

    for (int it = 0;; ++it) {
        const int blk = warp + it * NW;
        if (blk >= nblk) break;
        const int stage = it % NS;
        cp_async_wait<NS - 1>();
        __syncwarp();
        const uint32_t kst = ring_w + stage * STAGE, vst = kst + kBlk * ROWB;
        if (rope) {
            // encode the tile's keys at their cache slots, in place: row r of the tile is slot lo + 16 blk + r; a lane
            // takes piece pairs (c, c + CPR/2) of rows, eight lanes per row (conflict-free 16-byte accesses)
            unsigned char* kt = ring + (size_t)(warp * NS + stage) * STAGE;
#pragma unroll
            for (int i2 = 0; i2 < (ROPE ? kRopeItems : 0); ++i2) {
                const int item = lane + 32 * i2, r = item / (CPR / 2), cidx = item % (CPR / 2);
                uint4* plo = reinterpret_cast<uint4*>(kt + r * ROWB + ((cidx ^ (r & 7)) << 4));
                uint4* phi = reinterpret_cast<uint4*>(kt + r * ROWB + (((cidx + CPR / 2) ^ (r & 7)) << 4));
                uint4 a = *plo, bq = *phi;
                rope_piece_pair(a, bq, tab[i2]);
                *plo = a; *phi = bq;
            }
            if (blk + NW < nblk) load_tabs(blk + NW);
            __syncwarp();
        }

        // ---- logits of 16 keys x G heads
        float c[2][4];
#pragma unroll
        for (int hb = 0; hb < 2; ++hb)
#pragma unroll
            for (int e = 0; e < 4; ++e) c[hb][e] = 0.f;
#pragma unroll
        for (int u = 0; u < D / 32; ++u) {
#pragma unroll
            for (int hb = 0; hb < 2; ++hb) {
                uint32_t r0, r1, r2, r3;
                ldmatrix_x4(kst + hb * 8 * ROWB + koff[u], r0, r1, r2, r3);
                mma_bf16(c[hb], qa[2 * u][0], 0u, qa[2 * u][1], 0u, r0, r1);
                mma_bf16(c[hb], qa[2 * u + 1][0], 0u, qa[2 * u + 1][1], 0u, r2, r3);
            }
        }
        // lane (g,t) holds head g, keys 2t, 2t+1 (c[0]) and 8+2t, 9+2t (c[1]) of the block
        float s4[4] = {c[0][0] * scale, c[0][1] * scale, c[1][0] * scale, c[1][1] * scale};
        const int key0 = blk * kBlk + 2 * t;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int key = key0 + (e & 1) + (e >> 1) * 8;
            const int lam = lo + key;
            if (!(lam < hi && lam != n - 1)) s4[e] = -INFINITY;
            if (g < G && key < nrows) sl[g * rows_cap + key] = s4[e];
        }
        float bm = fmaxf(fmaxf(s4[0], s4[1]), fmaxf(s4[2], s4[3]));
        bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 1));
        bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 2));
        const float m_new = fmaxf(m_run, bm);
        if (__any_sync(0xffffffffu, m_new > m_run)) {
            const float corr = (m_new == -INFINITY) ? 1.f : exp2_diff(m_run, m_new);
            l_run *= corr;
            m_run = m_new;
            const float c0 = __shfl_sync(0xffffffffu, corr, (2 * t) * 4);      // head 2t   (columns of acc)
            const float c1 = __shfl_sync(0xffffffffu, corr, (2 * t + 1) * 4);  // head 2t+1
#pragma unroll
            for (int cc = 0; cc < D / 16; ++cc) { acc[cc][0] *= c0; acc[cc][1] *= c1; acc[cc][2] *= c0; acc[cc][3] *= c1; }
        }
        float p[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) p[e] = (m_run == -INFINITY) ? 0.f : exp2_diff(s4[e], m_run);
        l_run += (p[0] + p[1]) + (p[2] + p[3]);
        const uint32_t pb0 = pack_bf16(p[0], p[1]), pb1 = pack_bf16(p[2], p[3]);

        // ---- o^T[ch][head] += V^T[ch][key] P^T[key][head]
#pragma unroll
        for (int cc = 0; cc < D / 16; ++cc) {
            uint32_t r0, r1, r2, r3;
            ldmatrix_x4_trans(vst + voff[cc], r0, r1, r2, r3);
            mma_bf16(acc[cc], r0, r1, r2, r3, pb0, pb1);
        }
        __syncwarp();
        issue(blk + NS * NW, stage);
    }
    cp_async_wait<0>();

    // ---- per-warp partials (max, sum) of head g
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    if (t == 0 && g < G) { wstat[(warp * 2 + 0) * G + g] = m_run; wstat[(warp * 2 + 1) * G + g] = l_run; }
    __syncthreads();  // every warp is done with its ring: o_warp may overwrite it
#pragma unroll
    for (int cc = 0; cc < D / 16; ++cc) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int head = 2 * t + (e & 1), ch = 16 * cc + g + (e >> 1) * 8;
            if (head < G) o_warp[(warp * G + head) * D + ch] = acc[cc][e];
        }
    }
    if (owns_new && tid < G) sl[tid * rows_cap + (n - 1 - lo)] = wstat[(NW * 2 + 0) * G + tid];  // the new token's logit
    __syncthreads();

    // ---- CTA partial: (max, sum) per head and the output relative to the CTA max, pushed with remote stores
    //      (statistics into every CTA of the cluster, the output into CTA 0): nobody waits on a remote load
    if (nsplit > 1) asm volatile("barrier.cluster.wait.aligned;" ::: "memory");  // every CTA of the cluster is running
    float* o_all0 = cluster.map_shared_rank(o_all, 0);
    for (int idx = tid; idx < G * D; idx += NT) {
        const int h = idx / D, ch = idx % D;
        float M = -INFINITY;
        for (int w = 0; w <= NW; ++w) M = fmaxf(M, wstat[(w * 2) * G + h]);
        float o = 0.f, l = 0.f;
        for (int w = 0; w < NW; ++w) {
            const float f = exp2_diff(wstat[(w * 2) * G + h], M);
            o += o_warp[(w * G + h) * D + ch] * f;
            l += wstat[(w * 2 + 1) * G + h] * f;
        }
        if (owns_new) {
            const float f = exp2_diff(wstat[(NW * 2) * G + h], M);
            o += __bfloat162float(tv[ch]) * f;
            l += f;
        }
        o_all0[(size_t)rank * G * D + idx] = o;
        if (ch < nsplit) {  // thread (h, ch = r) delivers this CTA's statistics to CTA r
            float* gs = cluster.map_shared_rank(gstat, ch);
            gs[(rank * 2 + 0) * G + h] = M;
            gs[(rank * 2 + 1) * G + h] = l;
        }
    }

    // a cluster of one needs no cluster-scope release of its global stores: a block barrier orders shared memory
    auto unit_barrier = [&]() { if (nsplit == 1) __syncthreads(); else cluster.sync(); };
    unit_barrier();  // (A) every CTA's statistics (and, in CTA 0, every partial output) have arrived

    float Mg[G], invL[G];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        float M = -INFINITY;
        for (int r = 0; r < nsplit; ++r) M = fmaxf(M, gstat[(r * 2) * G + h]);
        float L = 0.f;
        for (int r = 0; r < nsplit; ++r) L += gstat[(r * 2 + 1) * G + h] * exp2_diff(gstat[(r * 2) * G + h], M);
        Mg[h] = M; invL[h] = 1.0f / L;
    }
    // ---- in a cluster of several CTAs the scope's two updated scores go to CTA 0 first (remote shared-memory
    //      stores), and the cluster barrier is split around the bulk of the global stores: arrive now - its release
    //      only has these few stores to cover - and wait after the output and the score update have been issued.
    //      Each value is computed with the same expression the bulk loop uses.
    const int ncached = nrows - (owns_new ? 1 : 0);
    auto updated_score = [&](int j) {  // j: index among this CTA's rows; the appended token starts from S = 0
        float ps = 0.f;
#pragma unroll
        for (int h = 0; h < G; ++h) ps += ex2_fast(sl[h * rows_cap + j] - Mg[h]) * invL[h];
        return (j < ncached ? s_old[j] : 0.f) + ps * (1.0f / G);
    };
    if (nsplit > 1) {
        if (will_evict && tid < 2) {
            const int lam = a_cyc + tid;  // live indices of the scope's physical rows
            if (lam >= lo && lam < hi) cluster.map_shared_rank(pair_s, 0)[tid] = updated_score(lam - lo);
        }
        __syncwarp();
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    }

    if (rank == 0) {
#pragma unroll
        for (int h = 0; h < G; ++h) {
            for (int ch = tid; ch < D; ch += NT) {
                float o = 0.f;
                for (int r = 0; r < nsplit; ++r)
                    o += o_all[((size_t)r * G + h) * D + ch] * exp2_diff(gstat[(r * 2) * G + h], Mg[h]);
                out[((size_t)b * cv.Hq + kh * G + h) * D + ch] = __float2bfloat16_rn(o * invL[h]);
            }
        }
    }
    // ---- normalised probabilities; score update (Algorithm 1: S <- (S u {0}) + a, group mean)
    //      (a masked or padded logit is -inf and 2^-inf = 0, so exp2f needs no guard here: Mg is finite).  The two
    //      rows of the scope are left to the eviction below, which writes the survivor's score to its new row.
#pragma unroll 8
    for (int j = tid; j < ncached; j += NT) {
        const int ph = phys_row(lo + j, st);
        const float s_new = updated_score(j);
        if (!(will_evict && (unsigned)(ph - row_l) < 2u)) Sc[ph] = s_new;
        else if (nsplit == 1) pair_s[ph - row_l] = s_new;  // a single CTA takes the scope's scores from its own loop
    }
    if (owns_new && tid == NT - 1) {
        Pc[new_row] = N;
        const float s_new = updated_score(ncached);
        if (!(will_evict && (unsigned)(new_row - row_l) < 2u)) Sc[new_row] = s_new;
        else if (nsplit == 1) pair_s[new_row - row_l] = s_new;
    }

    // (B) the scope's scores have arrived in CTA 0
    if (nsplit > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    else __syncthreads();

    if (rank == 0 && warp == 0 && will_evict) {
        // ---- Algorithm 1, "length > c" branch: scope {idx, idx+1} = physical rows (row_l, row_l + 1)
        const int N1 = N + 1;
        const int l = row_l, r = l + 1;
        int evict_right = 0;
        if (lane == 0) {
            bool near_tie = false;
            const float S_l = pair_s[0], S_r = pair_s[1];
            evict_right = pair_evicts_right(S_l, score_count(N1, pos_l, w0), S_r, score_count(N1, pos_r, w0), cv.rule, &near_tie) ? 1 : 0;
            if (near_tie) atomicAdd(&cv.stats->near_ties, 1ull);
            const int src = evict_right ? l : r;
            Sc[a_cyc] = evict_right ? S_l : S_r;  // also when the survivor stays in place: the score update skipped the scope
            Pc[a_cyc] = evict_right ? pos_l : pos_r;
        }
        evict_right = __shfl_sync(0xffffffffu, evict_right, 0);
        const int src = evict_right ? l : r, dst = a_cyc;
        if (src != dst) {  // survivor's K and V rows were staged in shared memory at kernel start
            const unsigned char* ksrc = pair_kv + (evict_right ? 0 : 1) * ROWB;
            const unsigned char* vsrc = pair_kv + (evict_right ? 2 : 3) * ROWB;
            for (int e = lane; e < CHUNKS; e += 32) {
                reinterpret_cast<uint4*>(Kc + (size_t)dst * D)[e] = reinterpret_cast<const uint4*>(ksrc)[e];
                reinterpret_cast<uint4*>(Vc + (size_t)dst * D)[e] = reinterpret_cast<const uint4*>(vsrc)[e];
            }
        }
    }
    // ---- end of a cycle with a protected recent window: the nr rows behind the last pair move down next to the
    //      middle region, so that the next cycle starts from a contiguous cache.  Once per c_mid steps.  The whole
    //      cluster takes part, in rounds of "read into registers / cluster barrier / write": a destination row can
    //      be a source row of the same round when the window is longer than the middle region, never of a later one.
    if (will_evict && cv.nr > 0 && i_cyc == cv.cm - 1) {
        if (nsplit > 1) cluster.sync(); else __syncthreads();  // every S, pos and appended row of the unit is visible
        constexpr int PER = 4;                 // rows per warp and round
        const int src0 = cv.ns + 2 * cv.cm, dst0 = cv.ns + cv.cm, nmove = cv.nr;
        const int gw = rank * NW + warp, nw_all = nsplit * NW;
        for (int r0 = 0; r0 < nmove; r0 += nw_all * PER) {
            uint4 kr[PER], vr[PER];
            float sr[PER];
            int32_t pr[PER];
#pragma unroll
            for (int u = 0; u < PER; ++u) {
                const int it = r0 + u * nw_all + gw;
                if (it >= nmove) continue;
                if (lane < CHUNKS) {
                    kr[u] = __ldcg(reinterpret_cast<const uint4*>(Kc + (size_t)(src0 + it) * D) + lane);
                    vr[u] = __ldcg(reinterpret_cast<const uint4*>(Vc + (size_t)(src0 + it) * D) + lane);
                }
                if (lane == 0) { sr[u] = __ldcg(Sc + src0 + it); pr[u] = __ldcg(Pc + src0 + it); }
            }
            if (nsplit > 1) cluster.sync(); else __syncthreads();
#pragma unroll
            for (int u = 0; u < PER; ++u) {
                const int it = r0 + u * nw_all + gw;
                if (it >= nmove) continue;
                if (lane < CHUNKS) {
                    reinterpret_cast<uint4*>(Kc + (size_t)(dst0 + it) * D)[lane] = kr[u];
                    reinterpret_cast<uint4*>(Vc + (size_t)(dst0 + it) * D)[lane] = vr[u];
                }
                if (lane == 0) { Sc[dst0 + it] = sr[u]; Pc[dst0 + it] = pr[u]; }
            }
        }
    }
    if (rank == 0 && tid == 0) cv.n_seen[unit] = N + 1;
}

static size_t decode_mma_smem_bytes_ns(int G, int D, int c, int split, int stages) {
    const size_t ring = (size_t)kMmaWarps * stages * 2 * kBlk * D * 2;
    return ring + sizeof(float) * ((size_t)G * mma_rows_cap(c, split) + (kMmaWarps + 1) * 2 * G + kMaxSplit * 2 * G +
                                   (size_t)split * G * D + (size_t)mma_rows_cap(c, split) + 2) + 4 * (size_t)D * 2 + 16 +
           16 + (size_t)(G + 2) * D * 2;
}

size_t decode_mma_smem_bytes(int G, int D, int c, int split) { return decode_mma_smem_bytes_ns(G, D, c, split, kMmaStages); }

static int decode_sm_count() {
    static int sm_count[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    dev &= 63;
    if (sm_count[dev] == 0) cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev);
    return std::max(sm_count[dev], 1);
}

template <int D, int G, int NS, bool ROPE>
static cudaError_t launch_decode_mma_nsr(const CacheView& cv, const void* q, const void* k, const void* v, void* out,
                                        const ActiveMask& active, int split, int inputs_final, cudaStream_t stream) {
    auto kern = decode_mma_kernel<D, G, kMmaWarps, NS, ROPE>;
    const int rows_cap = mma_rows_cap(cv.c, split);
    size_t smem = decode_mma_smem_bytes_ns(G, D, cv.c, split, NS);
    static size_t smem_set[64] = {};  // per device: the opt-in limit only ever needs raising
    int dev = 0;
    cudaGetDevice(&dev);
    dev &= 63;
    const int sms = decode_sm_count();
    // When the whole grid fits at w = ceil(CTAs / SMs) thread blocks per SM, ask for just enough shared memory that
    // no SM can take more than w: the block scheduler otherwise packs some SMs to their limit and leaves others idle,
    // and the streaming rate of an SM does not grow in proportion to the blocks it hosts.
    {
        constexpr size_t kSmemPerSm = 227 * 1024, kReserved = 1024;  // per-block reservation of the runtime
        const long ncta = (long)split * cv.Hkv * cv.B;
        const long w = (ncta + sms - 1) / sms;
        if (w >= 1 && (size_t)(w + 1) * (smem + kReserved) <= kSmemPerSm)
            smem = std::max(smem, kSmemPerSm / (size_t)(w + 1) + 1 - kReserved + 1024);
    }
    if (smem > smem_set[dev]) {
        const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        smem_set[dev] = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(split, cv.Hkv, cv.B);
    cfg.blockDim = dim3(kMmaWarps * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = split;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // the kernel orders itself with griddepcontrol.wait
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    using T = __nv_bfloat16;
    return cudaLaunchKernelEx(&cfg, kern, cv, reinterpret_cast<const T*>(q), reinterpret_cast<const T*>(k),
                              reinterpret_cast<const T*>(v), reinterpret_cast<T*>(out), active, rows_cap, inputs_final);
}

template <int D, int G, int NS>
static cudaError_t launch_decode_mma_ns(const CacheView& cv, const void* q, const void* k, const void* v, void* out,
                                        const ActiveMask& active, int split, int inputs_final, cudaStream_t stream) {
    return cv.rope_cos ? launch_decode_mma_nsr<D, G, NS, true>(cv, q, k, v, out, active, split, inputs_final, stream)
                       : launch_decode_mma_nsr<D, G, NS, false>(cv, q, k, v, out, active, split, inputs_final, stream);
}

// A thread block that has an SM to itself keeps three tiles per warp in flight instead of two (when they fit): one
// block of four warps per SM is otherwise short of bytes in flight.
template <int D, int G>
static cudaError_t launch_decode_mma_t(const CacheView& cv, const void* q, const void* k, const void* v, void* out,
                                       const ActiveMask& active, int split, int inputs_final, cudaStream_t stream) {
    const long ncta = (long)split * cv.Hkv * cv.B;
    if (ncta <= decode_sm_count() && decode_mma_smem_bytes_ns(G, D, cv.c, split, 3) <= 227 * 1024)
        return launch_decode_mma_ns<D, G, 3>(cv, q, k, v, out, active, split, inputs_final, stream);
    return launch_decode_mma_ns<D, G, kMmaStages>(cv, q, k, v, out, active, split, inputs_final, stream);
}

template <int D>
static cudaError_t launch_decode_mma_g(const CacheView& cv, const void* q, const void* k, const void* v, void* out,
                                       const ActiveMask& active, int split, int inputs_final, cudaStream_t stream) {
    switch (cv.Hq / cv.Hkv) {
        case 1: return launch_decode_mma_t<D, 1>(cv, q, k, v, out, active, split, inputs_final, stream);
        case 2: return launch_decode_mma_t<D, 2>(cv, q, k, v, out, active, split, inputs_final, stream);
        case 4: return launch_decode_mma_t<D, 4>(cv, q, k, v, out, active, split, inputs_final, stream);
        case 8: return launch_decode_mma_t<D, 8>(cv, q, k, v, out, active, split, inputs_final, stream);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_decode_mma(const CacheView& cv, const void* q, const void* k, const void* v, void* out,
                              const ActiveMask& active, int split, int inputs_final, cudaStream_t stream) {
    if (cv.d == 64) return launch_decode_mma_g<64>(cv, q, k, v, out, active, split, inputs_final, stream);
    if (cv.d == 128) return launch_decode_mma_g<128>(cv, q, k, v, out, active, split, inputs_final, stream);
    return cudaErrorInvalidValue;
}

}  // namespace treekv
