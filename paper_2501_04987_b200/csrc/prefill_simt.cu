// Chunked-prefill attention on CUDA cores: the path for fp32 and for shapes the tensor-core kernel does not
// cover.  One CTA owns one tile of 128 query rows (row = token * G + head-in-group) of one unit and walks its
// tokens in order; each token is a decode-style pass over the rows it may see (every cached row and chunk
// rows up to itself), with exact softmax (Section 3.1).  The tile's column sums of the probability matrix are
// kept in shared memory in a fixed order and written once, as the tile's slice of the partial column sums.
#include "common.cuh"
#include "simt_attend.cuh"

namespace treekv {

template <typename T, int D, int G, int U>
__global__ void __launch_bounds__(kDecodeThreads)
prefill_simt_kernel(CacheView cv, PrefillScratch ps, const T* __restrict__ q, T* __restrict__ out, ChunkLens lens,
                    int chunk_stride) {
    constexpr int VEC = Elem<T>::kVec;
    constexpr int LPR = D / VEC;
    constexpr int TOK = kQTileRows / G;  // tokens per tile
    const int unit = blockIdx.y;
    const int b = unit / cv.Hkv, kh = unit % cv.Hkv;
    const int m = lens.m[b];
    const int t0 = blockIdx.x * TOK;
    if (t0 >= m) return;
    const int t1 = min(t0 + TOK, m);
    const int N = cv.n_seen[unit];
    const UnitState st = unit_state(N, cv);
    const int n = st.L + m;
    const int rows_cap = ps.n_max;
    const int wstart = ps.window > 0 ? m - ps.window : 0;  // one-shot prefill: only the observation window scores

    const T* Kc = reinterpret_cast<const T*>(cv.K) + (size_t)unit * cv.R * D;
    const T* Vc = reinterpret_cast<const T*>(cv.V) + (size_t)unit * cv.R * D;

    extern __shared__ __align__(16) float smem[];
    float* sl = smem;                           // [G][n_max]
    float* col = sl + (size_t)G * rows_cap;     // [n_max]
    float* red = col + rows_cap;                // [kDecodeWarps][G]
    float* o_part = red + kDecodeWarps * G;     // [G][D]
    float* o_warp = o_part + G * D;             // [kDecodeWarps][G][D]

    const int tid = threadIdx.x, lane = tid & 31;
    const int sub = lane % LPR;
    for (int j = tid; j < n; j += kDecodeThreads) col[j] = 0.f;

    for (int t = t0; t < t1; ++t) {
        const int n_vis = st.L + t + 1;  // cached rows, then chunk rows 0..t
        float qr[G][VEC];
        const float scale = kLog2e * rsqrtf((float)D);
#pragma unroll
        for (int h = 0; h < G; ++h) {
            const uint4 u = ld_plain(reinterpret_cast<const uint4*>(
                                         q + (((size_t)b * chunk_stride + t) * cv.Hq + kh * G + h) * D) + sub);
            Elem<T>::unpack(u, qr[h]);
            if (cv.rope_cos) rope_apply<T, D>(qr[h], n_vis - 1, sub, cv.rope_cos, cv.rope_sin);  // the row's own slot
#pragma unroll
            for (int e = 0; e < VEC; ++e) qr[h][e] *= scale;
        }
        float mx[G];
        k_phase<T, D, G, U>(Kc, 0, n_vis, st, -1, nullptr, qr, sl, rows_cap, mx, cv.rope_cos, cv.rope_sin);
        block_reduce<G>(mx, red, true);
        float sum[G];
#pragma unroll
        for (int h = 0; h < G; ++h) sum[h] = 0.f;
        for (int j = tid; j < n_vis; j += kDecodeThreads) {
#pragma unroll
            for (int h = 0; h < G; ++h) {
                const float e = exp2f(sl[h * rows_cap + j] - mx[h]);
                sl[h * rows_cap + j] = e;
                sum[h] += e;
            }
        }
        block_reduce<G>(sum, red, false);
        for (int j = tid; j < n_vis; j += kDecodeThreads) {
            float psum = 0.f;
#pragma unroll
            for (int h = 0; h < G; ++h) {
                const float p = sl[h * rows_cap + j] / sum[h];
                sl[h * rows_cap + j] = p;
                psum += p;
            }
            if (t >= wstart) col[j] += psum;  // same thread owns column j for every token: fixed summation order
        }
        __syncthreads();
        v_phase<T, D, G, U>(Vc, 0, n_vis, st, -1, nullptr, sl, rows_cap, o_warp, o_part);
        __syncthreads();
        for (int e = tid; e < G * D; e += kDecodeThreads)
            out[(((size_t)b * chunk_stride + t) * cv.Hq + kh * G) * D + e] = Elem<T>::from_float(o_part[e]);
        __syncthreads();
    }
    float* dst = ps.colsum + ((size_t)unit * ps.QT + blockIdx.x) * ps.n_max;
    for (int j = tid; j < n; j += kDecodeThreads) dst[j] = col[j];
}

size_t prefill_simt_smem_bytes(int G, int D, int n_max) {
    return sizeof(float) * ((size_t)G * n_max + n_max + kDecodeWarps * G + (size_t)G * D + (size_t)kDecodeWarps * G * D);
}

template <typename T, int D, int G>
static cudaError_t launch_prefill_simt_t(const CacheView& cv, const PrefillScratch& ps, const void* q, void* out,
                                         const ChunkLens& lens, int chunk_stride, int max_m, cudaStream_t stream) {
    auto kern = prefill_simt_kernel<T, D, G, 4>;
    const size_t smem = prefill_simt_smem_bytes(G, D, ps.n_max);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid((max_m * G + kQTileRows - 1) / kQTileRows, cv.B * cv.Hkv);
    kern<<<grid, kDecodeThreads, smem, stream>>>(cv, ps, reinterpret_cast<const T*>(q), reinterpret_cast<T*>(out), lens,
                                                 chunk_stride);
    return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t launch_prefill_simt_g(const CacheView& cv, const PrefillScratch& ps, const void* q, void* out,
                                         const ChunkLens& lens, int chunk_stride, int max_m, cudaStream_t stream) {
    switch (cv.Hq / cv.Hkv) {
        case 1: return launch_prefill_simt_t<T, D, 1>(cv, ps, q, out, lens, chunk_stride, max_m, stream);
        case 2: return launch_prefill_simt_t<T, D, 2>(cv, ps, q, out, lens, chunk_stride, max_m, stream);
        case 4: return launch_prefill_simt_t<T, D, 4>(cv, ps, q, out, lens, chunk_stride, max_m, stream);
        case 8: return launch_prefill_simt_t<T, D, 8>(cv, ps, q, out, lens, chunk_stride, max_m, stream);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_prefill_simt(const CacheView& cv, treekv_dtype dt, const PrefillScratch& ps, const void* q, void* out,
                                const ChunkLens& lens, int chunk_stride, int max_m, cudaStream_t stream) {
    if (dt == TREEKV_F32) {
        if (cv.d == 64) return launch_prefill_simt_g<float, 64>(cv, ps, q, out, lens, chunk_stride, max_m, stream);
        if (cv.d == 128) return launch_prefill_simt_g<float, 128>(cv, ps, q, out, lens, chunk_stride, max_m, stream);
    } else {
        if (cv.d == 64) return launch_prefill_simt_g<__nv_bfloat16, 64>(cv, ps, q, out, lens, chunk_stride, max_m, stream);
        if (cv.d == 128) return launch_prefill_simt_g<__nv_bfloat16, 128>(cv, ps, q, out, lens, chunk_stride, max_m, stream);
    }
    return cudaErrorInvalidValue;
}

}  // namespace treekv
