// Chunked-prefill attention of TreeKV on the 5th-generation tensor cores (bf16, head_dim 128).
//
// What it computes (Section 3.1 of the paper applied to a chunk): for a tile of 128 query rows (row = token * G
// + head-in-group) of one unit (sequence, KV head), out = softmax(q K^T / sqrt(d)) V over every cached row and
// the chunk rows up to the query's own, and the tile's column sums of that probability matrix, which the score
// update adds to S (Algorithm 1: S <- S + a, for all steps of the chunk at once).
//
// How: two passes over the key tiles, both on tcgen05.mma with TMA-fed, 128-byte-swizzled shared-memory tiles
// and accumulators in tensor memory.
//   pass A  S = Q K^T (tensor-memory lane = query): running row max and sum -> log-sum-exp per query.
//   pass B  S^T = K Q^T (lane = key): P^T = exp2(S^T * scale - lse[query]) is already normalised, so its row
//           sums over the queries ARE the column sums (one register add per element, no cross-lane reduction),
//           and O^T += V^T P^T accumulates the output with no rescaling.  P^T goes to shared memory as the
//           MN-major B operand; V is consumed as the MN-major A operand straight from its row-major tile.
// Same three contractions and two exponentials per element as "attention, then recompute against the final
// log-sum-exp", with the probabilities used for the output and for the scores being the same numbers.
//
// Warp roles: warp 0 issues TMA, warp 1 issues MMA and owns the tensor-memory allocation, warps 2-17 are two
// groups of eight softmax warps; inside a group a warp owns one tensor-memory lane quarter and one half of a
// tile's 128 columns.  Group g takes the key tiles of parity g and owns P^T buffer g, so the two groups
// alternate tiles and overlap each other's latency.  The S / S^T accumulators are three tensor-memory buffers
// used round-robin by tile index, so the MMA warp can start a tile's logits while both groups are still reading
// theirs.  All waits are bounded mbarrier waits; a wait that gives up sets an error word and the CTA drains to
// its exit, where tensor memory is released.
#include <type_traits>

#include "prefill_tc_common.cuh"

namespace treekv {

namespace {

using namespace tc;

constexpr int kRing = 4;       // K / V tiles in flight
constexpr int kTcThreads = tc::kThreads;

constexpr int kSBufs = 3;     // S / S^T accumulators in tensor memory, used round-robin by tile index
enum Bar { Q_FULL = 0, RING_FULL = 1, RING_EMPTY = 5, S_FULL = 9, S_FREE = 12, P_FULL = 15, P_FREE = 17, O_FULL = 19, N_BARS = 20 };

}  // namespace

template <int G>
__global__ void __launch_bounds__(kTcThreads, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmKin,
                  const __grid_constant__ CUtensorMap tmVin, ChunkDirect cd, CacheView cv, PrefillScratch ps,
                  __nv_bfloat16* __restrict__ out, ChunkLens lens, int chunk_stride) {
    constexpr int TOK = 128 / G;
    const int unit = blockIdx.y, qt = blockIdx.x;
    const int b = unit / cv.Hkv, kh = unit % cv.Hkv;
    const int m = lens.m[b];
    const int t0 = qt * TOK;
    if (t0 >= m) return;
    const int t1 = min(t0 + TOK, m);
    const int N = cv.n_seen[unit];
    const UnitState st = unit_state(N, cv);
    const KeyTiles kt = key_tiles(st, st.L + t1, cd.k != nullptr);
    const int NT = kt.NT;
    const int n = st.L + m;

    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t bars[N_BARS];
    __shared__ uint32_t tmem_slot;
    const uint32_t base = (smem_addr_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_addr_u32(smem_raw));
    const uint32_t sQ = base, sRing = base + kSlot, sP = base + (1 + kRing) * kSlot;
    float* lse = reinterpret_cast<float*>(base_ptr + (3 + kRing) * kSlot);  // [128] minus log-sum-exp of the query rows

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t bar0 = smem_addr_u32(&bars[0]);
    auto bar = [&](int idx) { return bar0 + 8u * (uint32_t)idx; };

    if (tid == 0) {
        mbar_init(bar(Q_FULL), 1);
        for (int s = 0; s < kRing; ++s) { mbar_init(bar(RING_FULL + s), 1); mbar_init(bar(RING_EMPTY + s), 1); }
        for (int s = 0; s < kSBufs; ++s) { mbar_init(bar(S_FULL + s), 1); mbar_init(bar(S_FREE + s), 8); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar(P_FULL + s), 8); mbar_init(bar(P_FREE + s), 1); }
        mbar_init(bar(O_FULL), 1);
        mbar_fence_init();
    }
    if (warp == 1) { tmem_alloc(smem_addr_u32(&tmem_slot), kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const uint32_t tmS = tmem, tmO = tmem + 128 * kSBufs;  // S / S^T buffers at columns 0, 128, 256; O^T at 384

    bool ok = true;
    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            mbar_arrive_expect_tx(bar(Q_FULL), kSlot);
            tma_load_3d(sQ, &tmQ, 0, kh * G, b * chunk_stride + t0, bar(Q_FULL));
            tma_load_3d(sQ + kHalf, &tmQ, 64, kh * G, b * chunk_stride + t0, bar(Q_FULL));
            int ld = 0;
            auto load_tile = [&](const CUtensorMap* mp, const CUtensorMap* mp_in, int j) {
                int lam0, row0, valid;
                const bool from_chunk = tile_of(kt, j, lam0, row0, valid);
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
            // pass A: K tiles in order.  Pass B: the same order in which the MMA warp consumes them - K runs three
            // tiles ahead of V (K_0 K_1 K_2 | V_0 K_3 | V_1 K_4 | ...), so a K tile is requested as soon as the S^T
            // two tiles back has executed and its load latency hides behind two tiles of work.
            for (int j = 0; j < NT && ok; ++j) load_tile(&tmK, &tmKin, j);
            for (int j = 0; j < 3 && j < NT && ok; ++j) load_tile(&tmK, &tmKin, j);
            for (int j = 0; j < NT && ok; ++j) {
                load_tile(&tmV, &tmVin, j);
                if (ok && j + 3 < NT) load_tile(&tmK, &tmKin, j + 3);
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
            int use[kSBufs] = {0, 0, 0};  // times each S buffer has been handed to the softmax warps (both passes)
            // ---- pass A: S = Q K^T
            for (int j = 0; j < NT && ok; ++j) {
                const int ld = j, slot = ld % kRing, buf = j % kSBufs;
                ok = mbar_wait(bar(RING_FULL + slot), (ld / kRing) & 1) && mbar_wait(bar(S_FREE + buf), (use[buf] & 1) ^ 1);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sK = sRing + slot * kSlot;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t off = (kk >> 2) * kHalf + (kk & 3) * 32;
                    umma_bf16(tmS + buf * 128, umma_desc_sw128(sQ + off, 16, 1024), umma_desc_sw128(sK + off, 16, 1024),
                              idesc_kk, kk > 0);
                }
                umma_commit(bar(RING_EMPTY + slot));
                umma_commit(bar(S_FULL + buf));
                ++use[buf];
            }
            // ---- pass B: S^T_j = K_j Q^T runs two tiles ahead of O^T_j += V_j^T P_j^T, so that the group that
            //      owns buffer j & 1 finds S^T_{j+2} ready when it finishes tile j (its buffer is free as soon as
            //      it has read tile j into registers, long before P_j^T is complete)
            auto issue_st = [&](int j) {
                const int ld = NT + (j < 3 ? j : 2 * j - 2), slot = ld % kRing, buf = j % kSBufs;  // see the producer's load order
                ok = mbar_wait(bar(RING_FULL + slot), (ld / kRing) & 1) && mbar_wait(bar(S_FREE + buf), (use[buf] & 1) ^ 1);
                if (!ok) return;
                tc_fence_after();
                const uint32_t sK = sRing + slot * kSlot;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t off = (kk >> 2) * kHalf + (kk & 3) * 32;
                    umma_bf16(tmS + buf * 128, umma_desc_sw128(sK + off, 16, 1024), umma_desc_sw128(sQ + off, 16, 1024),
                              idesc_kk, kk > 0);
                }
                umma_commit(bar(RING_EMPTY + slot));
                umma_commit(bar(S_FULL + buf));
                ++use[buf];
            };
            for (int j = 0; j < 2 && j < NT && ok; ++j) issue_st(j);
            for (int pj = 0; pj < NT && ok; ++pj) {
                if (pj + 2 < NT) { issue_st(pj + 2); if (!ok) break; }
                const int pbuf = pj & 1;
                const int ld = NT + min(3, NT) + pj + min(pj, max(0, NT - 3)), slot = ld % kRing;
                ok = mbar_wait(bar(P_FULL + pbuf), (pj >> 1) & 1) && mbar_wait(bar(RING_FULL + slot), (ld / kRing) & 1);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sV = sRing + slot * kSlot, sPT = sP + pbuf * kSlot;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {  // 16 keys per step: 16 rows of 128 bytes
                    umma_bf16(tmO, umma_desc_sw128(sV + kk * 2048, kHalf, 1024), umma_desc_sw128(sPT + kk * 2048, kHalf, 1024),
                              idesc_pv, (pj > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(bar(RING_EMPTY + slot));
                umma_commit(bar(P_FREE + pbuf));
            }
            if (ok) umma_commit(bar(O_FULL));
            else atomicOr(&cv.stats->error, 8u);
        }
    } else {
        // ================= softmax warps =================
        const int sw = warp - 2;               // 0..15
        const int grp = sw >> 3;               // group 0: warps 2-9, group 1: warps 10-17; group g owns tiles j = g (mod 2)
        const int half = (sw >> 2) & 1;        // this warp handles columns [64*half, 64*half + 64) of a tile
        const int quarter = warp & 3;          // tensor-memory lanes [32*quarter, +32) belong to this warp
        const int row = quarter * 32 + lane;   // pass A: query row; pass B: key of the tile; epilogue: channel
        const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
        const float sc2 = kLog2e * rsqrtf((float)kD);
        float* nlse = lse;                     // [128] minus the log2-domain log-sum-exp of every query row
        // running (max, sum) of pass A per (group, column half), [4][128] each; they borrow the P^T area, which
        // pass A does not use
        float* part_m = reinterpret_cast<float*>(base_ptr + (1 + kRing) * kSlot);
        float* part_l = part_m + 512;
        float* xch = lse + 128;                // [2][128] column sums handed from the upper to the lower column half
        uint32_t va[32], vb[32];  // two chunks of 32 columns: the next one is in flight while this one is used
        if (cd.k) append_own_tokens(cv, cd, unit, b, kh, chunk_stride, st, N, t0, t1, tid - 64, 512);
        // ---- pass A: row statistics over this group's tiles
        {
            const int tq = min(t0 + row / G, t1 - 1);  // rows past the chunk repeat the last real row: finite, unused
            float mrun = -INFINITY, lrun = 0.f;
            for (int j = grp; j < NT && ok; j += 2) {
                const int buf = j % kSBufs;  // the buffer's fill number in this pass is j / kSBufs
                const uint32_t tmSg = tmS + buf * 128 + lane_off;
                if (!mbar_wait(bar(S_FULL + buf), (j / kSBufs) & 1)) { ok = false; break; }
                tc_fence_after();
                int lam0, row0, valid;
                tile_of(kt, j, lam0, row0, valid);
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
            part_m[(grp * 2 + half) * 128 + row] = mrun;
            part_l[(grp * 2 + half) * 128 + row] = lrun;
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");  // all softmax warps: the partial statistics are complete
        if (sw < 4) {
            float M = -INFINITY;
#pragma unroll
            for (int u = 0; u < 4; ++u) M = fmaxf(M, part_m[u * 128 + row]);
            float l = 0.f;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float mu = part_m[u * 128 + row];
                if (mu != -INFINITY) l += part_l[u * 128 + row] * ex2(mu - M);
            }
            nlse[row] = -(M + log2f(l));
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");  // nlse[] is complete
        // ---- pass B: probabilities, column sums, P^T for the tensor cores
        const int rmax = G * (t1 - t0);  // query columns [rmax, 128) are padding
        // observation window (one-shot prefill): only the last ps.window tokens of the chunk add to the column sums
        const int rwin = ps.window > 0 ? max(0, G * (m - ps.window - t0)) : 0;
        float* part = ps.colsum + ((size_t)unit * ps.QT + qt) * ps.n_max;
        int puse = 0;  // times this group's P^T buffer has been filled
        for (int j = grp; j < NT && ok; j += 2) {
            const int buf = j % kSBufs;
            const uint32_t tmSg = tmS + buf * 128 + lane_off;
            const int fills_a = (NT + kSBufs - 1 - buf) / kSBufs;  // times pass A filled this buffer
            if (!mbar_wait(bar(S_FULL + buf), (fills_a + j / kSBufs) & 1)) { ok = false; break; }
            tc_fence_after();
            int lam0, row0, valid;
            tile_of(kt, j, lam0, row0, valid);
            const bool kvalid = row < valid;
            const int lam = lam0 + row;
            const int rmin = kvalid ? max(0, G * (lam - kt.L - t0)) : 128;  // first query column that sees this key
            const bool full = __all_sync(0xffffffffu, rmin == 0) && rmax == 128 && rwin == 0;
            float colsum = 0.f;
            unsigned char* prow = base_ptr + (1 + kRing) * kSlot + grp * kSlot + row * 128;
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
                    // the O^T MMA of this group's previous tile must have read the P^T buffer; it has had the time of
                    // the first loads and of this chunk's arithmetic to finish
                    if (!mbar_wait(bar(P_FREE + grp), (puse & 1) ^ 1)) { ok = false; }
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
            if (lane == 0) mbar_arrive(bar(S_FREE + buf));
            if (full) probs32(std::true_type{}, std::false_type{}, vb, 2 * half + 1); else probs32(std::false_type{}, std::false_type{}, vb, 2 * half + 1);
            // the key's column sum = lower half + upper half, added in that order.  The warp of the upper half hands
            // its sum over through shared memory (named barrier of the two warps); it can only write the slot again
            // after this tile's P^T has been consumed, which needs the lower half's arrival below.
            const int pair_bar = 2 + grp * 4 + quarter;
            if (half == 1) {
                xch[grp * 128 + row] = colsum;
                asm volatile("bar.arrive %0, 64;" ::"r"(pair_bar) : "memory");
            } else {
                asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
                if (kvalid) part[lam] = colsum + xch[grp * 128 + row];
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(P_FULL + grp));
            ++puse;
        }
        // keys this tile's queries cannot see contribute nothing
        for (int lam = kt.nvis + (tid - 64); lam < n; lam += 512) part[lam] = 0.f;
        // ---- epilogue: O^T (lane = channel, column = query row) -> out[token][head][channel], staged through the idle
        //      P^T area so that whole rows are written; the four warps (lane quarters) that share 32 query columns
        //      synchronise on a barrier of their own
        if (ok && mbar_wait(bar(O_FULL), 0)) {
            tc_fence_after();
            const int cg = sw >> 2;  // one chunk of 32 query columns per warp
            unsigned char* stage = base_ptr + (1 + kRing) * kSlot;
            tmem_ld32(tmO + lane_off + cg * 32, va);
            tmem_ld_wait_for(va);
#pragma unroll
            for (int e = 0; e < 32; ++e) stage_put(stage, cg * 32 + e, row, __uint_as_float(va[e]));
            asm volatile("bar.sync %0, 128;" ::"r"(10 + cg) : "memory");
            stage_flush<G>(stage, out, (size_t)b * chunk_stride + t0, cv.Hq, kh, cg * 32, 32, rmax, quarter * 32 + lane, 128);
            tc_fence_before();
        } else {
            atomicOr(&cv.stats->error, 16u);
        }
    }
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

size_t prefill_tc_smem_bytes() { return 1024 + (size_t)(3 + kRing) * kSlot + (128 + 256) * sizeof(float); }

template <int G>
static cudaError_t launch_prefill_tc_t(const CacheView& cv, const PrefillScratch& ps, const CUtensorMap& tmQ,
                                       const CUtensorMap& tmK, const CUtensorMap& tmV, const ChunkTensors& ct, void* out,
                                       const ChunkLens& lens, int chunk_stride, int max_m, cudaStream_t stream) {
    auto kern = prefill_tc_kernel<G>;
    const size_t smem = prefill_tc_smem_bytes();
    static bool smem_set[64] = {};  // per device: the opt-in is needed once
    int dev = 0;
    cudaGetDevice(&dev);
    dev &= 63;
    if (!smem_set[dev]) {
        const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        smem_set[dev] = true;
    }
    dim3 grid((max_m * G + kQTileRows - 1) / kQTileRows, cv.B * cv.Hkv);
    const ChunkDirect cd = {reinterpret_cast<const __nv_bfloat16*>(ct.k), reinterpret_cast<const __nv_bfloat16*>(ct.v)};
    kern<<<grid, kTcThreads, smem, stream>>>(tmQ, tmK, tmV, ct.k ? ct.tmK : tmK, ct.k ? ct.tmV : tmV, cd, cv, ps,
                                             reinterpret_cast<__nv_bfloat16*>(out), lens, chunk_stride);
    return cudaGetLastError();
}

cudaError_t launch_prefill_tc(const CacheView& cv, const PrefillScratch& ps, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                              const CUtensorMap& tmV, const ChunkTensors& ct, void* out, const ChunkLens& lens,
                              int chunk_stride, int max_m, cudaStream_t stream) {
    if (cv.d != kD) return cudaErrorInvalidValue;
    switch (cv.Hq / cv.Hkv) {
        case 1: return launch_prefill_tc_t<1>(cv, ps, tmQ, tmK, tmV, ct, out, lens, chunk_stride, max_m, stream);
        case 2: return launch_prefill_tc_t<2>(cv, ps, tmQ, tmK, tmV, ct, out, lens, chunk_stride, max_m, stream);
        case 4: return launch_prefill_tc_t<4>(cv, ps, tmQ, tmK, tmV, ct, out, lens, chunk_stride, max_m, stream);
        case 8: return launch_prefill_tc_t<8>(cv, ps, tmQ, tmK, tmV, ct, out, lens, chunk_stride, max_m, stream);
    }
    return cudaErrorInvalidValue;
}

}  // namespace treekv
