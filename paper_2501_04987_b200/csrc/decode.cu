// Decode step of TreeKV (Algorithm 1, one loop iteration; attention of Section 3.1) as ONE kernel launch.
//
// A thread-block cluster of `split` CTAs owns one unit (sequence, KV head).  Each CTA streams its share of
// the c+1 live rows of K with 128-bit loads, keeps the logits of all G query heads of the group in shared
// memory, and the cluster agrees on the softmax statistics through distributed shared memory.  Every CTA
// then turns its logits into normalised probabilities, adds their group mean to S, streams its share of V
// and the cluster sums the partial outputs.  Finally CTA 0 plays Algorithm 1's eviction branch: compare the
// averaged scores of rows (2i, 2i+1), move the survivor to row i, advance the token count.  K and V are read
// exactly once per step; nothing but the survivor row is ever moved.
#include <cooperative_groups.h>

#include "common.cuh"
#include "simt_attend.cuh"

namespace cg = cooperative_groups;

namespace treekv {

template <typename T, int D, int G, int U>
__global__ void __launch_bounds__(kDecodeThreads)
decode_kernel(CacheView cv, const T* __restrict__ q, const T* __restrict__ k_in, const T* __restrict__ v_in,
              T* __restrict__ out, ActiveMask active, int rows_cap) {
    constexpr int VEC = Elem<T>::kVec;
    constexpr int LPR = D / VEC;   // lanes per row
    constexpr int CHUNKS = D * (int)sizeof(T) / 16;
    static_assert(LPR >= 1 && LPR <= 32 && (32 % LPR) == 0, "row must map onto a warp");

    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int nsplit = (int)cluster.num_blocks();
    const int kh = blockIdx.y, b = blockIdx.z;
    // Programmatic dependent launch: the next kernel in the stream may be scheduled while this one runs, and nothing
    // below the wait touches memory before the previous kernel's writes are complete and visible.  Every block waits,
    // also one of an inactive sequence.
    pdl_trigger();
    pdl_wait();
    if (!active.test(b)) return;  // the whole cluster shares b

    const int unit = b * cv.Hkv + kh;
    const int N = cv.n_seen[unit];
    const UnitState st = unit_state(N, cv);
    const int n = st.L + 1;  // live rows including the token appended by this step
    const int i_cyc = st.i;
    const int per = (n + nsplit - 1) / nsplit;
    const int lo = min(rank * per, n), hi = min(lo + per, n);
    const int nrows = hi - lo;

    T* Kc = reinterpret_cast<T*>(cv.K) + (size_t)unit * cv.R * D;
    T* Vc = reinterpret_cast<T*>(cv.V) + (size_t)unit * cv.R * D;
    float* Sc = cv.S + (size_t)unit * cv.R;
    int32_t* Pc = cv.pos + (size_t)unit * cv.R;
    const T* k_new = k_in + (size_t)unit * D;
    const T* v_new = v_in + (size_t)unit * D;
    const int new_row = st.L + i_cyc;  // physical row of the appended token

    extern __shared__ __align__(16) float smem[];
    float* sl = smem;                          // [G][rows_cap] logits -> probabilities
    float* red = sl + (size_t)G * rows_cap;    // [kDecodeWarps][G]
    float* cl_stats = red + kDecodeWarps * G;  // [2G] this CTA's (max, sum), read by the cluster
    float* o_part = cl_stats + 2 * G;          // [G][D] this CTA's partial output, read by the cluster
    float* o_warp = o_part + G * D;            // [kDecodeWarps][G][D]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR;

    // ---- append (Algorithm 1: K <- K u {k}, V <- V u {v}).  This step itself reads the new token from
    //      k_in / v_in, so the slab row is not read back before the cluster barrier below.
    if (hi == n && nrows > 0 && warp == 0) {
        for (int e = lane; e < CHUNKS; e += 32) {
            reinterpret_cast<uint4*>(Kc + (size_t)new_row * D)[e] = ld_plain(reinterpret_cast<const uint4*>(k_new) + e);
            reinterpret_cast<uint4*>(Vc + (size_t)new_row * D)[e] = ld_plain(reinterpret_cast<const uint4*>(v_new) + e);
        }
    }

    // ---- q of the group, this lane's channel slice, pre-scaled by log2(e)/sqrt(d)
    float qr[G][VEC];
    {
        const float scale = kLog2e * rsqrtf((float)D);
#pragma unroll
        for (int h = 0; h < G; ++h) {
            const uint4 u = ld_plain(reinterpret_cast<const uint4*>(q + ((size_t)b * cv.Hq + kh * G + h) * D) + sub);
            Elem<T>::unpack(u, qr[h]);
            if (cv.rope_cos) rope_apply<T, D>(qr[h], n - 1, sub, cv.rope_cos, cv.rope_sin);  // the query sits in the last slot
#pragma unroll
            for (int e = 0; e < VEC; ++e) qr[h][e] *= scale;
        }
    }

    // ---- K phase: logits (in log2 units) of this CTA's rows
    float mx[G];
    k_phase<T, D, G, U>(Kc, lo, hi, st, n - 1, k_new, qr, sl, rows_cap, mx, cv.rope_cos, cv.rope_sin);
    block_reduce<G>(mx, red, true);  // includes the barrier that publishes sl

    // ---- e = 2^(s - max), local sum
    float sum[G];
#pragma unroll
    for (int h = 0; h < G; ++h) sum[h] = 0.f;
    for (int j = tid; j < nrows; j += kDecodeThreads) {
#pragma unroll
        for (int h = 0; h < G; ++h) {
            const float e = exp2f(sl[h * rows_cap + j] - mx[h]);
            sl[h * rows_cap + j] = e;
            sum[h] += e;
        }
    }
    block_reduce<G>(sum, red, false);
    if (tid < G) { cl_stats[tid] = mx[tid]; cl_stats[G + tid] = sum[tid]; }

    cluster.sync();  // (A) every CTA's statistics are visible

    // ---- global softmax statistics through distributed shared memory; factor that normalises this CTA's e
    float fac[G];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        float M = -INFINITY;
        for (int r = 0; r < nsplit; ++r) M = fmaxf(M, cluster.map_shared_rank(cl_stats, r)[h]);
        float Lsum = 0.f;
        for (int r = 0; r < nsplit; ++r) {
            const float* rs = cluster.map_shared_rank(cl_stats, r);
            const float mr = rs[h];
            Lsum += (mr == -INFINITY) ? 0.f : rs[G + h] * exp2f(mr - M);
        }
        fac[h] = (mx[h] == -INFINITY) ? 0.f : exp2f(mx[h] - M) / Lsum;
    }

    // ---- normalised probabilities; score update (Algorithm 1: S <- (S u {0}) + a, group mean)
    for (int j = tid; j < nrows; j += kDecodeThreads) {
        float ps = 0.f;
#pragma unroll
        for (int h = 0; h < G; ++h) {
            const float p = sl[h * rows_cap + j] * fac[h];
            sl[h * rows_cap + j] = p;
            ps += p;
        }
        const int lam = lo + j;
        const int ph = phys_row(lam, st);
        const float s_old = (lam == n - 1) ? 0.f : Sc[ph];
        Sc[ph] = s_old + ps * (1.0f / G);
        if (lam == n - 1) Pc[ph] = N;
    }
    __syncthreads();

    // ---- V phase: o = sum_j p_j v_j over this CTA's rows
    v_phase<T, D, G, U>(Vc, lo, hi, st, n - 1, v_new, sl, rows_cap, o_warp, o_part);

    cluster.sync();  // (B) partial outputs, the appended row and every S update of the unit are complete

    if (rank == 0) {
        for (int t = tid; t < G * D; t += kDecodeThreads) {
            float r = 0.f;
            for (int rr = 0; rr < nsplit; ++rr) r += cluster.map_shared_rank(o_part, rr)[t];
            out[((size_t)b * cv.Hq + kh * G) * D + t] = Elem<T>::from_float(r);
        }
        // ---- Algorithm 1, "length > c" branch: scope {idx, idx+1} = physical rows (a + i, a + i + 1), survivor to row a
        if (warp == 0) {
            const int N1 = N + 1;
            if (N1 > cv.c) {
                const int l = st.a + i_cyc, r = l + 1;
                int evict_right = 0;
                if (lane == 0) {
                    bool near_tie = false;
                    const int w0 = cv.w0[unit];
                    evict_right = pair_evicts_right(__ldcg(Sc + l), score_count(N1, __ldcg(Pc + l), w0), __ldcg(Sc + r),
                                                    score_count(N1, __ldcg(Pc + r), w0), cv.rule, &near_tie) ? 1 : 0;
                    if (near_tie) atomicAdd(&cv.stats->near_ties, 1ull);
                }
                evict_right = __shfl_sync(0xffffffffu, evict_right, 0);
                const int src = evict_right ? l : r, dst = st.a;
                if (src != dst) {
                    for (int e = lane; e < CHUNKS; e += 32) {
                        const uint4 kk = __ldcg(reinterpret_cast<const uint4*>(Kc + (size_t)src * D) + e);
                        const uint4 vv = __ldcg(reinterpret_cast<const uint4*>(Vc + (size_t)src * D) + e);
                        reinterpret_cast<uint4*>(Kc + (size_t)dst * D)[e] = kk;
                        reinterpret_cast<uint4*>(Vc + (size_t)dst * D)[e] = vv;
                    }
                    if (lane == 0) { Sc[dst] = __ldcg(Sc + src); Pc[dst] = __ldcg(Pc + src); }
                }
            }
        }
    }
    cluster.sync();  // (C) keep shared memory alive until CTA 0 has read it; the survivor's move is complete
    // ---- end of a cycle with a protected recent window: the nr rows behind the last pair move down next to the
    //      middle region (see common.cuh), in rounds of "read into registers / cluster barrier / write"
    if (N + 1 > cv.c && cv.nr > 0 && i_cyc == cv.cm - 1) {
        constexpr int PER = 4;
        const int src0 = cv.ns + 2 * cv.cm, dst0 = cv.ns + cv.cm, nmove = cv.nr;
        const int gw = rank * kDecodeWarps + warp, nw_all = nsplit * kDecodeWarps;
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
            cluster.sync();
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

size_t decode_smem_bytes(int G, int D, int c, int split) {
    const int rows_cap = (c + 1 + split - 1) / split;
    return sizeof(float) * ((size_t)G * rows_cap + kDecodeWarps * G + 2 * G + (size_t)G * D + (size_t)kDecodeWarps * G * D);
}

template <typename T, int D, int G>
static cudaError_t launch_decode_t(const CacheView& cv, const void* q, const void* k, const void* v, void* out,
                                   const ActiveMask& active, int split, cudaStream_t stream) {
    constexpr int U = 4;
    auto kern = decode_kernel<T, D, G, U>;
    const int rows_cap = (cv.c + 1 + split - 1) / split;
    const size_t smem = decode_smem_bytes(G, D, cv.c, split);
    static size_t smem_set[64] = {};  // per device: the opt-in limit only ever needs raising
    int dev = 0;
    cudaGetDevice(&dev);
    dev &= 63;
    if (smem > smem_set[dev]) {
        const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        smem_set[dev] = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(split, cv.Hkv, cv.B);
    cfg.blockDim = dim3(kDecodeThreads);
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
    return cudaLaunchKernelEx(&cfg, kern, cv, reinterpret_cast<const T*>(q), reinterpret_cast<const T*>(k),
                              reinterpret_cast<const T*>(v), reinterpret_cast<T*>(out), active, rows_cap);
}

template <typename T, int D>
static cudaError_t launch_decode_g(const CacheView& cv, const void* q, const void* k, const void* v, void* out,
                                   const ActiveMask& active, int split, cudaStream_t stream) {
    switch (cv.Hq / cv.Hkv) {
        case 1: return launch_decode_t<T, D, 1>(cv, q, k, v, out, active, split, stream);
        case 2: return launch_decode_t<T, D, 2>(cv, q, k, v, out, active, split, stream);
        case 4: return launch_decode_t<T, D, 4>(cv, q, k, v, out, active, split, stream);
        case 8: return launch_decode_t<T, D, 8>(cv, q, k, v, out, active, split, stream);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_decode(const CacheView& cv, treekv_dtype dt, const void* q, const void* k, const void* v, void* out,
                          const ActiveMask& active, int split, cudaStream_t stream) {
    if (dt == TREEKV_F32) {
        if (cv.d == 64) return launch_decode_g<float, 64>(cv, q, k, v, out, active, split, stream);
        if (cv.d == 128) return launch_decode_g<float, 128>(cv, q, k, v, out, active, split, stream);
    } else {
        if (cv.d == 64) return launch_decode_g<__nv_bfloat16, 64>(cv, q, k, v, out, active, split, stream);
        if (cv.d == 128) return launch_decode_g<__nv_bfloat16, 128>(cv, q, k, v, out, active, split, stream);
    }
    return cudaErrorInvalidValue;
}

}  // namespace treekv
