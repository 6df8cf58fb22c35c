// Chunked-prefill attention of TreeKV on the 5th-generation tensor cores, 256 query rows per CTA.
//
// Same computation and the same two passes as prefill_tc.cu (Section 3.1 of the paper applied to a chunk; the
// column sums feed Algorithm 1's score update), organised for large grids: a CTA owns two adjacent tiles of 128
// query rows ("sub-tiles") of one unit and streams every K / V tile once for both.  What limits the 128-row
// kernel is the shared-memory it can give to loads in flight against the latency of a tile load; here the same
// bytes in flight feed twice the tensor-core work.
//   pass A  S_s = Q_s K^T for s = 0, 1 (lane = query): running row max and sum -> log-sum-exp per query.
//   pass B  S_s^T = K Q_s^T (lane = key): P_s^T = exp2(S_s^T * scale - lse[query]) is already normalised, its row
//           sums are the sub-tile's column sums, and O_s^T += V^T P_s^T.
// Warp roles: warp 0 issues TMA, warp 1 issues MMA and owns the tensor-memory allocation, warps 2-9 are the
// softmax group of sub-tile 0 and warps 10-17 that of sub-tile 1 (inside a group a warp owns one tensor-memory
// lane quarter and one half of a tile's 128 columns).  Tensor memory: pass A double-buffers S per sub-tile (four
// buffers of 128 columns); pass B holds S_s^T in buffers 0, 1 and O_s^T in buffers 2, 3.  Shared memory: two Q
// tiles, a ring of three K / V tiles, one P^T tile per sub-tile.  All waits are bounded mbarrier waits; a wait
// that gives up sets an error word and the CTA drains to its exit, where tensor memory is released.
#include <algorithm>
#include <type_traits>

#include "prefill_tc_common.cuh"

namespace treekv {

namespace {

using namespace tc;

constexpr int kRing = 3;       // K / V tiles in flight

enum Bar { Q_FULL = 0, RING_FULL = 1, RING_EMPTY = 4, S_FULL = 7, S_FREE = 11, P_FULL = 15, P_FREE = 17, O_FULL = 19,
           X_STATS = 20, X_FREE = 21, X_RECV = 22, N_BARS = 23 };  // X_*: signalled by the other CTA of a key-split pair

}  // namespace

template <int G, int KS>
__global__ void __launch_bounds__(kThreads, 1)
prefill_tc2_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmKin,
                   const __grid_constant__ CUtensorMap tmVin, ChunkDirect cd, CacheView cv, PrefillScratch ps,
                   __nv_bfloat16* __restrict__ out, ChunkLens lens, int chunk_stride, int pairs_per_unit,
                   int n_whole_clusters) {
    constexpr int TOK = 128 / G;  // tokens per sub-tile
    // KS == 1: grid (tile pairs, units).  KS == 2: a 1-D grid of two-CTA clusters over the call's items (unit, tile
    // pair) in order: the CTAs of the first n_whole_clusters clusters take one whole item each (they exchange nothing
    // and never synchronise with each other), every later cluster splits one item's key tiles between its CTAs - the
    // items of a last, partial wave, which then fills the machine and is about half as long.
    int unit, qt2, ks = 0;
    bool split = false;
    if constexpr (KS == 1) {
        unit = blockIdx.y; qt2 = blockIdx.x;
    } else {
        const int cid = (int)(blockIdx.x >> 1), rk = (int)(blockIdx.x & 1);
        split = cid >= n_whole_clusters;
        const int item = split ? 2 * n_whole_clusters + (cid - n_whole_clusters) : 2 * cid + rk;
        unit = item / pairs_per_unit; qt2 = item % pairs_per_unit;
        ks = split ? rk : 0;
        if (unit >= cv.B * cv.Hkv) return;  // the odd CTA of the last whole-item cluster
    }
    const int b = unit / cv.Hkv, kh = unit % cv.Hkv;
    const int m = lens.m[b];
    const int t0c = qt2 * 2 * TOK;  // first token of the CTA
    if (t0c >= m) return;  // uniform over a splitting cluster
    const int t1c = min(t0c + 2 * TOK, m);
    const int N = cv.n_seen[unit];
    const UnitState st = unit_state(N, cv);
    const KeyTiles kt = key_tiles(st, st.L + t1c, cd.k != nullptr);
    const int NT = kt.NT;
    const int n = st.L + m;
    // this CTA's key tiles [jb, jb + nt): all of them, or its half (rank 0 the first, larger one: never empty)
    const int jb = (split && ks == 1) ? (NT + 1) / 2 : 0;
    const int nt = split ? (ks == 0 ? (NT + 1) / 2 : NT - (NT + 1) / 2) : NT;

    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const uint32_t base = smem_addr_u32(smem_raw);
    const uint32_t sQ = base, sRing = base + 2 * kSlot, sP = base + (2 + kRing) * kSlot;
    unsigned char* p_area = smem_raw + (2 + kRing) * kSlot;
    float* lse = reinterpret_cast<float*>(smem_raw + (4 + kRing) * kSlot);  // [2][128] minus log-sum-exp of the query rows
    float* xch = lse + 256;                                                   // [2][128] column sums, upper -> lower column half
    uint64_t* bars = reinterpret_cast<uint64_t*>(xch + 256);                 // [N_BARS]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + N_BARS);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t bar0 = smem_addr_u32(bars);
    auto bar = [&](int idx) { return bar0 + 8u * (uint32_t)idx; };

    if (tid == 0) {
        mbar_init(bar(Q_FULL), 1);
        for (int s = 0; s < kRing; ++s) { mbar_init(bar(RING_FULL + s), 1); mbar_init(bar(RING_EMPTY + s), 1); }
        for (int s = 0; s < 4; ++s) { mbar_init(bar(S_FULL + s), 1); mbar_init(bar(S_FREE + s), 8); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar(P_FULL + s), 8); mbar_init(bar(P_FREE + s), 1); }
        mbar_init(bar(O_FULL), 1);
        mbar_init(bar(X_STATS), 8); mbar_init(bar(X_FREE), 1); mbar_init(bar(X_RECV), 16);
        mbar_fence_init();
        if (base & 1023u) atomicOr(&cv.stats->error, 32u);  // the tiles' swizzle needs a 1024-byte aligned base
    }
    if (warp == 1) { tmem_alloc(smem_addr_u32(tmem_slot), kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    // both CTAs of a pair are running and their barriers are initialised before either signals the other
    if (KS > 1 && split) cluster_sync_all();

    bool ok = true;
    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            mbar_arrive_expect_tx(bar(Q_FULL), 2 * kSlot);
#pragma unroll
            for (int s = 0; s < 2; ++s) {  // a sub-tile that starts past the last token row of the tensor reads zeros
                tma_load_3d(sQ + s * kSlot, &tmQ, 0, kh * G, b * chunk_stride + t0c + s * TOK, bar(Q_FULL));
                tma_load_3d(sQ + s * kSlot + kHalf, &tmQ, 64, kh * G, b * chunk_stride + t0c + s * TOK, bar(Q_FULL));
            }
            int ld = 0;
            auto load_tile = [&](const CUtensorMap* mp, const CUtensorMap* mp_in, int j) {
                int lam0, row0, valid;
                const bool from_chunk = tile_of(kt, jb + j, lam0, row0, valid);
                const int slot = ld % kRing;
                if (!mbar_wait(bar(RING_EMPTY + slot), ((ld / kRing) & 1) ^ 1)) { ok = false; return; }
                const uint32_t dst = sRing + slot * kSlot;
                mbar_arrive_expect_tx(bar(RING_FULL + slot), kSlot);
                if (from_chunk) {  // 128 tokens of the caller's tensor
                    tma_load_3d(dst, mp_in, 0, kh, b * chunk_stride + row0, bar(RING_FULL + slot));
                    tma_load_3d(dst + kHalf, mp_in, 64, kh, b * chunk_stride + row0, bar(RING_FULL + slot));
                } else {
                    const int grow = unit * cv.R + row0;
                    tma_load_2d(dst, mp, 0, grow, bar(RING_FULL + slot));
                    tma_load_2d(dst + kHalf, mp, 64, grow, bar(RING_FULL + slot));
                }
                ++ld;
            };
            // pass A: K tiles in order.  Pass B, in the order the MMA warp consumes them: K_0 | K_1 V_0 | K_2 V_1 | ...
            for (int j = 0; j < nt && ok; ++j) load_tile(&tmK, &tmKin, j);
            if (ok && nt > 0) load_tile(&tmK, &tmKin, 0);
            for (int j = 0; j < nt && ok; ++j) {
                if (j + 1 < nt) load_tile(&tmK, &tmKin, j + 1);
                if (ok) load_tile(&tmV, &tmVin, j);
            }
            if (!ok) atomicOr(&cv.stats->error, 4u);
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0) {
            constexpr uint32_t idesc_kk = umma_idesc_bf16(128, 128, 0, 0);  // both operands K-major (rows x channels)
            constexpr uint32_t idesc_pv = umma_idesc_bf16(128, 128, 1, 1);  // V^T and P^T: MN-major
            ok = mbar_wait(bar(Q_FULL), 0);
            tc_fence_after();
            int use0 = 0, use1 = 0, use2 = 0, use3 = 0;  // times each S buffer has been handed to the softmax warps
            auto s_free_wait = [&](int buf) {
                const int u = buf == 0 ? use0 : buf == 1 ? use1 : buf == 2 ? use2 : use3;
                return mbar_wait(bar(S_FREE + buf), (u & 1) ^ 1);
            };
            auto s_used = [&](int buf) { if (buf == 0) ++use0; else if (buf == 1) ++use1; else if (buf == 2) ++use2; else ++use3; };
            int ld = 0;  // ring entries consumed so far, in the producer's order
            auto ring_wait = [&](int& slot) {
                slot = ld % kRing;
                const bool r = mbar_wait(bar(RING_FULL + slot), (ld / kRing) & 1);
                ++ld;
                return r;
            };
            // ---- pass A: S_s = Q_s K_j^T into buffer 2 s + (j & 1)
            for (int j = 0; j < nt && ok; ++j) {
                int slot;
                if (!(ok = ring_wait(slot))) break;
                const uint32_t sK = sRing + slot * kSlot;
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    const int buf = 2 * s + (j & 1);
                    if (!(ok = s_free_wait(buf))) break;
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint32_t off = (kk >> 2) * kHalf + (kk & 3) * 32;
                        umma_bf16(tmem + buf * 128, umma_desc_sw128(sQ + s * kSlot + off, 16, 1024),
                                  umma_desc_sw128(sK + off, 16, 1024), idesc_kk, kk > 0);
                    }
                    umma_commit(bar(S_FULL + buf));
                    s_used(buf);
                }
                if (!ok) break;
                umma_commit(bar(RING_EMPTY + slot));
            }
            // ---- pass B: S_s^T(j+1) = K_{j+1} Q_s^T is issued before O_s^T += V_j^T P_s^T(j), so a group finds its
            //      next logits ready when it has finished a tile; S_s^T lives in buffer s, O_s^T in buffer 2 + s
            auto issue_st = [&](int j) {
                int slot;
                if (!(ok = ring_wait(slot))) return;
                const uint32_t sK = sRing + slot * kSlot;
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    if (!(ok = s_free_wait(s))) return;
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint32_t off = (kk >> 2) * kHalf + (kk & 3) * 32;
                        umma_bf16(tmem + s * 128, umma_desc_sw128(sK + off, 16, 1024),
                                  umma_desc_sw128(sQ + s * kSlot + off, 16, 1024), idesc_kk, kk > 0);
                    }
                    umma_commit(bar(S_FULL + s));
                    s_used(s);
                }
                umma_commit(bar(RING_EMPTY + slot));
                (void)j;
            };
            if (ok && nt > 0) issue_st(0);
            for (int pj = 0; pj < nt && ok; ++pj) {
                if (pj + 1 < nt) { issue_st(pj + 1); if (!ok) break; }
                int slot;
                if (!(ok = ring_wait(slot))) break;
                const uint32_t sV = sRing + slot * kSlot;
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    if (!(ok = mbar_wait(bar(P_FULL + s), pj & 1))) break;
                    tc_fence_after();
                    const uint32_t sPT = sP + s * kSlot;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {  // 16 keys per step: 16 rows of 128 bytes
                        umma_bf16(tmem + (2 + s) * 128, umma_desc_sw128(sV + kk * 2048, kHalf, 1024),
                                  umma_desc_sw128(sPT + kk * 2048, kHalf, 1024), idesc_pv, (pj > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(bar(P_FREE + s));
                }
                if (!ok) break;
                umma_commit(bar(RING_EMPTY + slot));
            }
            if (ok) umma_commit(bar(O_FULL));
            else atomicOr(&cv.stats->error, 8u);
        }
    } else {
        // ================= softmax warps =================
        const int sw = warp - 2;               // 0..15
        const int sub = sw >> 3;               // the group's sub-tile
        const int half = (sw >> 2) & 1;        // this warp handles columns [64*half, 64*half + 64) of a tile
        const int quarter = warp & 3;          // tensor-memory lanes [32*quarter, +32) belong to this warp
        const int row = quarter * 32 + lane;   // pass A: query row; pass B: key of the tile; epilogue: channel
        const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
        const float sc2 = kLog2e * rsqrtf((float)kD);
        const int t0 = t0c + sub * TOK;        // the sub-tile's tokens [t0, t1); empty when t0 >= m
        const int t1 = min(t0 + TOK, m);
        const bool sub_live = t0 < m;
        float* nlse = lse + sub * 128;
        // running (max, sum) of pass A per (sub-tile, column half), [4][128] each; they borrow the P^T area
        float* part_m = reinterpret_cast<float*>(p_area);
        float* part_l = part_m + 512;
        uint32_t va[32], vb[32];  // two chunks of 32 columns: the next one is in flight while this one is used
        if (cd.k) append_own_tokens(cv, cd, unit, b, kh, chunk_stride, st, N, t0, t1, tid - 64 - sub * 256, 256);
        // ---- pass A: row statistics of the sub-tile over all key tiles
        {
            const int tq = max(t0c, min(t0 + row / G, t1 - 1));  // rows past the chunk repeat a real row: finite, unused
            float mrun = -INFINITY, lrun = 0.f;
            for (int j = 0; j < nt && ok; ++j) {
                const int buf = 2 * sub + (j & 1);
                const uint32_t tmSg = tmem + buf * 128 + lane_off;
                if (!mbar_wait(bar(S_FULL + buf), (j >> 1) & 1)) { ok = false; break; }
                tc_fence_after();
                int lam0, row0, valid;
                tile_of(kt, jb + j, lam0, row0, valid);
                const int limit = max(0, min(valid, kt.L + tq - lam0 + 1));  // columns [0, limit) are visible to this row
                const bool full = __all_sync(0xffffffffu, limit >= 128);
                auto stats32 = [&](const uint32_t (&v)[32], int cg) {
                    if (full) {
                        float cmax = __uint_as_float(v[0]);
#pragma unroll
                        for (int e = 1; e < 32; ++e) cmax = fmaxf(cmax, __uint_as_float(v[e]));
                        const float mnew = fmaxf(mrun, cmax * sc2);
                        float s0 = 0.f, s1 = 0.f;
#pragma unroll
                        for (int e = 0; e < 32; e += 2) {
                            s0 += ex2(fmaf(__uint_as_float(v[e]), sc2, -mnew));
                            s1 += ex2(fmaf(__uint_as_float(v[e + 1]), sc2, -mnew));
                        }
                        lrun = lrun * ex2(mrun - mnew) + (s0 + s1);
                        mrun = mnew;
                    } else {
                        float x[32];
                        float cmax = -INFINITY;
#pragma unroll
                        for (int e = 0; e < 32; ++e) {
                            x[e] = (cg * 32 + e < limit) ? __uint_as_float(v[e]) * sc2 : -INFINITY;
                            cmax = fmaxf(cmax, x[e]);
                        }
                        if (cmax > -INFINITY) {
                            const float mnew = fmaxf(mrun, cmax);
                            float sacc = 0.f;
#pragma unroll
                            for (int e = 0; e < 32; ++e) sacc += ex2(x[e] - mnew);
                            lrun = lrun * ex2(mrun - mnew) + sacc;
                            mrun = mnew;
                        }
                    }
                };
                tmem_ld32(tmSg + 64 * half, va);
                tmem_ld_wait_for(va);
                tmem_ld32(tmSg + 64 * half + 32, vb);
                stats32(va, 2 * half);
                tmem_ld_wait_for(vb);
                tc_fence_before();  // last read of this S buffer: hand it back before the arithmetic on it
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(S_FREE + buf));
                stats32(vb, 2 * half + 1);
            }
            part_m[(sub * 2 + half) * 128 + row] = mrun;
            part_l[(sub * 2 + half) * 128 + row] = lrun;
        }
        // all softmax warps: the partial statistics are complete, and nobody reads a pass-A buffer any more (two
        // of them become the O^T accumulators)
        asm volatile("bar.sync 1, 512;" ::: "memory");
        if (half == 0) {
            const float m0 = part_m[(sub * 2) * 128 + row], m1 = part_m[(sub * 2 + 1) * 128 + row];
            float M = fmaxf(m0, m1);
            float l = (m0 == -INFINITY ? 0.f : part_l[(sub * 2) * 128 + row] * ex2(m0 - M)) +
                      (m1 == -INFINITY ? 0.f : part_l[(sub * 2 + 1) * 128 + row] * ex2(m1 - M));
            if (KS > 1 && split) {
                // the other half of the keys: hand over this half's (max, sum), take the other's, combine - rank 0's
                // term first on both sides, so the two CTAs normalise with the same log-sum-exp bit for bit
                float* xstat = part_m + 1024;  // [2][128] x (max, sum), written by the other CTA
                const uint32_t peer = (uint32_t)(ks ^ 1);
                st_remote_v2(map_to_cta(smem_addr_u32(xstat + 2 * (sub * 128 + row)), peer), M, l);
                fence_cluster();
                __syncwarp();
                if (lane == 0) mbar_arrive_remote(map_to_cta(bar(X_STATS), peer));
                if (!mbar_wait_cluster(bar(X_STATS), 0)) ok = false;
                const float2 o = *reinterpret_cast<const float2*>(xstat + 2 * (sub * 128 + row));
                const float Mx = fmaxf(M, o.x);
                const float la = M == -INFINITY ? 0.f : l * ex2(M - Mx), lb = o.x == -INFINITY ? 0.f : o.y * ex2(o.x - Mx);
                l = ks == 0 ? la + lb : lb + la;
                M = Mx;
            }
            nlse[row] = -(M + log2f(l));
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");  // lse[] is complete; the P^T area is free for pass B
        // ---- pass B: probabilities, column sums, P^T for the tensor cores
        const int rmax = sub_live ? G * (t1 - t0) : 0;  // query columns [rmax, 128) are padding
        // observation window (one-shot prefill): only the last ps.window tokens of the chunk add to the column sums
        const int rwin = ps.window > 0 ? max(0, G * (m - ps.window - t0)) : 0;
        float* part = ps.colsum + ((size_t)unit * ps.QT + 2 * qt2 + sub) * ps.n_max;
        const int fills_a = sub == 0 ? (nt + 1) / 2 : nt / 2;  // times pass A filled barrier pair `sub` (buffers 0 and 1)
        float* xrow = xch + sub * 128;
        for (int j = 0; j < nt && ok; ++j) {
            const uint32_t tmSg = tmem + sub * 128 + lane_off;
            if (!mbar_wait(bar(S_FULL + sub), (fills_a + j) & 1)) { ok = false; break; }
            tc_fence_after();
            int lam0, row0, valid;
            tile_of(kt, jb + j, lam0, row0, valid);
            const bool kvalid = row < valid;
            const int lam = lam0 + row;
            const int rmin = kvalid ? max(0, G * (lam - kt.L - t0)) : 128;  // first query column that sees this key
            const bool full = __all_sync(0xffffffffu, rmin == 0) && rmax == 128 && rwin == 0;
            float colsum = 0.f;
            unsigned char* prow = p_area + sub * kSlot + row * 128;
            auto probs32 = [&](auto full_tag, auto first_tag, const uint32_t (&v)[32], int cg) {
                constexpr bool kFull = decltype(full_tag)::value;    // every (key, query) pair of the warp's rows is visible
                constexpr bool kFirst = decltype(first_tag)::value;  // first chunk of the tile: the P^T buffer may still be read
                uint4 pk[4];
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {  // 8 query columns -> one 16-byte chunk of the P^T row
                    float p[8];
#pragma unroll
                    for (int h4 = 0; h4 < 2; ++h4) {
                        const float4 l4 = *reinterpret_cast<const float4*>(nlse + cg * 32 + q4 * 8 + h4 * 4);
                        const float ls[4] = {l4.x, l4.y, l4.z, l4.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float pe = ex2(fmaf(__uint_as_float(v[q4 * 8 + h4 * 4 + e]), sc2, ls[e]));
                            if constexpr (kFull) {
                                p[h4 * 4 + e] = pe;
                            } else {
                                const int r = cg * 32 + q4 * 8 + h4 * 4 + e;
                                p[h4 * 4 + e] = (r >= rmin && r < rmax) ? pe : 0.f;
                            }
                        }
                    }
                    if constexpr (kFull) {
                        colsum += ((p[0] + p[1]) + (p[2] + p[3])) + ((p[4] + p[5]) + (p[6] + p[7]));
                    } else {
                        const int r0 = cg * 32 + q4 * 8;  // columns below rwin belong to queries outside the window
                        float w[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) w[e] = (r0 + e >= rwin) ? p[e] : 0.f;
                        colsum += ((w[0] + w[1]) + (w[2] + w[3])) + ((w[4] + w[5]) + (w[6] + w[7]));
                    }
                    __nv_bfloat162 t2;
                    t2 = __floats2bfloat162_rn(p[0], p[1]); pk[q4].x = *reinterpret_cast<uint32_t*>(&t2);
                    t2 = __floats2bfloat162_rn(p[2], p[3]); pk[q4].y = *reinterpret_cast<uint32_t*>(&t2);
                    t2 = __floats2bfloat162_rn(p[4], p[5]); pk[q4].z = *reinterpret_cast<uint32_t*>(&t2);
                    t2 = __floats2bfloat162_rn(p[6], p[7]); pk[q4].w = *reinterpret_cast<uint32_t*>(&t2);
                }
                if constexpr (kFirst) {
                    // the O^T MMA of the previous tile must have read the P^T buffer; it has had the time of the first
                    // loads and of this chunk's arithmetic to finish
                    if (!mbar_wait(bar(P_FREE + sub), (j & 1) ^ 1)) { ok = false; }
                }
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    const int cidx = cg * 4 + q4;  // 16-byte chunk of the 128-query row: half = cidx / 8
                    *reinterpret_cast<uint4*>(prow + (cidx >> 3) * kHalf + (((cidx & 7) ^ (row & 7)) << 4)) = pk[q4];
                }
            };
            tmem_ld32(tmSg + 64 * half, va);
            tmem_ld_wait_for(va);
            tmem_ld32(tmSg + 64 * half + 32, vb);
            if (full) probs32(std::true_type{}, std::true_type{}, va, 2 * half); else probs32(std::false_type{}, std::true_type{}, va, 2 * half);
            tmem_ld_wait_for(vb);
            tc_fence_before();  // last read of this S^T buffer
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(S_FREE + sub));
            if (full) probs32(std::true_type{}, std::false_type{}, vb, 2 * half + 1); else probs32(std::false_type{}, std::false_type{}, vb, 2 * half + 1);
            // the key's column sum = lower half + upper half, added in that order.  The warp of the upper half hands
            // its sum over through shared memory (named barrier of the two warps); it can only write the slot again
            // after this tile's P^T has been consumed, which needs the lower half's arrival below.
            const int pair_bar = 2 + sub * 4 + quarter;
            if (half == 1) {
                xrow[row] = colsum;
                asm volatile("bar.arrive %0, 64;" ::"r"(pair_bar) : "memory");
            } else {
                asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
                if (kvalid && sub_live) part[lam] = colsum + xrow[row];
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(P_FULL + sub));
        }
        // keys this CTA's queries cannot see contribute nothing
        if (sub_live && ks == 0)
            for (int lam = kt.nvis + (tid - 64 - sub * 256); lam < n; lam += 256) part[lam] = 0.f;
        // ---- epilogue: O_s^T (lane = channel, column = query row) -> out[token][head][channel]
        if (ok && mbar_wait(bar(O_FULL), 0)) {
            tc_fence_after();
            if (KS == 1 || !split) {
                // 64 query columns per warp, staged through the sub-tile's idle P^T buffer so that whole rows are
                // written; the four warps (lane quarters) of a column half synchronise on a barrier of their own
                unsigned char* stage = p_area + sub * kSlot;
#pragma unroll 1
                for (int cg = 2 * half; cg < 2 * half + 2; ++cg) {
                    tmem_ld32(tmem + (2 + sub) * 128 + lane_off + cg * 32, va);
                    tmem_ld_wait_for(va);
#pragma unroll
                    for (int e = 0; e < 32; ++e) stage_put(stage, cg * 32 + e, row, __uint_as_float(va[e]));
                }
                asm volatile("bar.sync %0, 128;" ::"r"(10 + sub * 2 + half) : "memory");
                stage_flush<G>(stage, out, (size_t)b * chunk_stride + t0, cv.Hq, kh, 64 * half, 64, rmax, quarter * 32 + lane, 128);
            } else {
                // Every MMA of this CTA has completed, so its ring is idle: tell the other CTA, which stages there the
                // partial O^T of the sub-tile this CTA finishes.  A warp takes 32 query columns of its lane quarter:
                // first of the other CTA's sub-tile (sent), then of its own (summed with what was received).
                const uint32_t peer = (uint32_t)(ks ^ 1);
                const int cg = sw >> 2;  // query columns [32 cg, 32 cg + 32)
                const uint32_t stage = sRing + (uint32_t)((cg * 4 + quarter) * 32 * 32 * 4);  // [8 groups of 4 columns][32 lanes][4]
                if (sw == 0 && lane == 0) mbar_arrive_remote(map_to_cta(bar(X_FREE), peer));
                if (mbar_wait_cluster(bar(X_FREE), 0)) {
                    tmem_ld32(tmem + (2 + (ks ^ 1)) * 128 + lane_off + cg * 32, va);
                    tmem_ld_wait_for(va);
                    const uint32_t dst = map_to_cta(stage, peer) + (uint32_t)lane * 16u;
#pragma unroll
                    for (int v4 = 0; v4 < 8; ++v4) {
                        // a CTA without key tiles never wrote its accumulators: its partial is zero
                        const float x0 = nt > 0 ? __uint_as_float(va[4 * v4]) : 0.f, x1 = nt > 0 ? __uint_as_float(va[4 * v4 + 1]) : 0.f;
                        const float x2 = nt > 0 ? __uint_as_float(va[4 * v4 + 2]) : 0.f, x3 = nt > 0 ? __uint_as_float(va[4 * v4 + 3]) : 0.f;
                        st_remote_v4(dst + (uint32_t)v4 * 512u, x0, x1, x2, x3);
                    }
                    fence_cluster();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_remote(map_to_cta(bar(X_RECV), peer));
                } else {
                    ok = false;
                }
                if (ok && mbar_wait_cluster(bar(X_RECV), 0)) {
                    tmem_ld32(tmem + (2 + ks) * 128 + lane_off + cg * 32, va);
                    tmem_ld_wait_for(va);
                    const int t0o = t0c + ks * TOK;                     // this CTA finishes sub-tile ks
                    const int rmaxo = t0o < m ? G * (min(t0o + TOK, m) - t0o) : 0;
                    const float* rcv = reinterpret_cast<const float*>(smem_raw + (stage - base)) + lane * 4;
                    unsigned char* ostage = p_area;  // rows are put together in the idle P^T area, see the one-CTA case
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const float mine = nt > 0 ? __uint_as_float(va[e]) : 0.f, theirs = rcv[(e >> 2) * 128 + (e & 3)];
                        stage_put(ostage, cg * 32 + e, row, ks == 0 ? mine + theirs : theirs + mine);
                    }
                    asm volatile("bar.sync %0, 128;" ::"r"(10 + cg) : "memory");
                    stage_flush<G>(ostage, out, (size_t)b * chunk_stride + t0o, cv.Hq, kh, cg * 32, 32, rmaxo, quarter * 32 + lane, 128);
                } else {
                    ok = false;
                }
                if (!ok) atomicOr(&cv.stats->error, 16u);
            }
            tc_fence_before();
        } else {
            atomicOr(&cv.stats->error, 16u);
        }
    }
    __syncthreads();
    // neither CTA of a splitting pair exits while the other may still write into its shared memory or signal its barriers
    if (KS > 1 && split) cluster_sync_all();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

size_t prefill_tc2_smem_bytes() { return (size_t)(4 + kRing) * kSlot + 512 * sizeof(float) + N_BARS * 8 + 16; }

template <int G, int KS>
static cudaError_t launch_prefill_tc2_t(const CacheView& cv, const PrefillScratch& ps, const CUtensorMap& tmQ,
                                        const CUtensorMap& tmK, const CUtensorMap& tmV, const ChunkTensors& ct, void* out,
                                        const ChunkLens& lens, int chunk_stride, int max_m, int n_whole_clusters,
                                        cudaStream_t stream) {
    auto kern = prefill_tc2_kernel<G, KS>;
    const size_t smem = prefill_tc2_smem_bytes();
    static bool smem_set[64] = {};  // per device: the opt-in is needed once
    int dev = 0;
    cudaGetDevice(&dev);
    dev &= 63;
    if (!smem_set[dev]) {
        const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        smem_set[dev] = true;
    }
    const ChunkDirect cd = {reinterpret_cast<const __nv_bfloat16*>(ct.k), reinterpret_cast<const __nv_bfloat16*>(ct.v)};
    const int pairs = (max_m * G + 2 * kQTileRows - 1) / (2 * kQTileRows), units = cv.B * cv.Hkv;
    cudaLaunchConfig_t cfg = {};
    if (KS == 1) {
        cfg.gridDim = dim3(pairs, units);
    } else {  // whole-item clusters first (two items each, the last one possibly with an idle CTA), then one cluster per split item
        const long items = (long)pairs * units;
        const long whole_items = std::min<long>(2L * n_whole_clusters, items);
        cfg.gridDim = dim3((unsigned)(2 * (n_whole_clusters + (items - whole_items))));
    }
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = KS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = KS > 1 ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, tmQ, tmK, tmV, ct.k ? ct.tmK : tmK, ct.k ? ct.tmV : tmV, cd, cv, ps,
                              reinterpret_cast<__nv_bfloat16*>(out), lens, chunk_stride, pairs, n_whole_clusters);
}

// n_whole_clusters < 0: one CTA per tile pair.  Otherwise clusters of two CTAs: the first n_whole_clusters take two tile
// pairs each (one per CTA), every remaining tile pair gets a cluster that splits its key tiles.
cudaError_t launch_prefill_tc2(const CacheView& cv, const PrefillScratch& ps, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                               const CUtensorMap& tmV, const ChunkTensors& ct, void* out, const ChunkLens& lens,
                               int chunk_stride, int max_m, int n_whole_clusters, cudaStream_t stream) {
    if (cv.d != kD) return cudaErrorInvalidValue;
#define TREEKV_TC2_CASE(g)                                                                                                    \
    case g:                                                                                                                   \
        return n_whole_clusters >= 0                                                                                          \
                   ? launch_prefill_tc2_t<g, 2>(cv, ps, tmQ, tmK, tmV, ct, out, lens, chunk_stride, max_m, n_whole_clusters, stream) \
                   : launch_prefill_tc2_t<g, 1>(cv, ps, tmQ, tmK, tmV, ct, out, lens, chunk_stride, max_m, 0, stream);
    switch (cv.Hq / cv.Hkv) {
        TREEKV_TC2_CASE(1)
        TREEKV_TC2_CASE(2)
        TREEKV_TC2_CASE(4)
        TREEKV_TC2_CASE(8)
    }
#undef TREEKV_TC2_CASE
    return cudaErrorInvalidValue;
}

}  // namespace treekv
