// CUDA-core building blocks of attention over cache rows (Section 3.1 of the TreeKV paper), shared by the
// decode kernel and by the CUDA-core prefill kernel: a row of d elements is spread over LPR lanes with one
// 128-bit load each, a warp covers RPW rows per load instruction and keeps U loads in flight.
#pragma once

#include "common.cuh"

namespace treekv {

constexpr int kDecodeThreads = 256;
constexpr int kDecodeWarps = kDecodeThreads / 32;

// Block-wide max or sum of N values per thread; result in every thread.  Contains two barriers.
template <int N>
__device__ inline void block_reduce(float (&v)[N], float* scratch /*[kDecodeWarps][N]*/, bool is_max) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int h = 0; h < N; ++h) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float x = __shfl_xor_sync(0xffffffffu, v[h], o);
            v[h] = is_max ? fmaxf(v[h], x) : v[h] + x;
        }
    }
    __syncthreads();  // scratch may still be read from a previous use
    if (lane == 0) {
#pragma unroll
        for (int h = 0; h < N; ++h) scratch[warp * N + h] = v[h];
    }
    __syncthreads();
#pragma unroll
    for (int h = 0; h < N; ++h) {
        float r = scratch[h];
        for (int w = 1; w < kDecodeWarps; ++w) r = is_max ? fmaxf(r, scratch[w * N + h]) : r + scratch[w * N + h];
        v[h] = r;
    }
}

// Logits s[h][lam - lo] = q_h . K[row(lam)] for live indices lam in [lo, hi), all G heads of the group, written
// to sl[h * rows_cap + (lam - lo)]; per-thread running maxima in mx.  qr holds this lane's slice of q, already
// scaled.  Live index `special` (or -1) is read from special_row with plain loads instead of from the slab.
template <typename T, int D, int G, int U>
__device__ inline void k_phase(const T* Kc, int lo, int hi, const UnitState& st, int special, const T* special_row,
                               const float (&qr)[G][Elem<T>::kVec], float* sl, int rows_cap, float (&mx)[G],
                               const float* rope_cos = nullptr, const float* rope_sin = nullptr) {
    constexpr int VEC = Elem<T>::kVec;
    constexpr int LPR = D / VEC;
    constexpr int RPW = 32 / LPR;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane % LPR, rsub = lane / LPR;
#pragma unroll
    for (int h = 0; h < G; ++h) mx[h] = -INFINITY;
    for (int base = lo + warp * RPW * U; base < hi; base += kDecodeWarps * RPW * U) {
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int lam = base + u * RPW + rsub;
            raw[u] = make_uint4(0, 0, 0, 0);
            if (lam < hi) {
                if (lam == special) raw[u] = ld_plain(reinterpret_cast<const uint4*>(special_row) + sub);
                else raw[u] = ld_stream(reinterpret_cast<const uint4*>(Kc + (size_t)phys_row(lam, st) * D) + sub);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int lam = base + u * RPW + rsub;
            float f[VEC];
            Elem<T>::unpack(raw[u], f);
            // in-cache positions: the key in cache slot lam is encoded at position lam
            if (rope_cos) rope_apply<T, D>(f, min(lam, hi - 1), sub, rope_cos, rope_sin);
#pragma unroll
            for (int h = 0; h < G; ++h) {
                float a = 0.f;
#pragma unroll
                for (int e = 0; e < VEC; ++e) a = fmaf(qr[h][e], f[e], a);
#pragma unroll
                for (int o = LPR / 2; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
                if (lam < hi) {
                    mx[h] = fmaxf(mx[h], a);
                    if (sub == 0) sl[h * rows_cap + (lam - lo)] = a;
                }
            }
        }
    }
}

// o_part[h][:] = sum over lam in [lo, hi) of p[h][lam - lo] * V[row(lam)], p read from sl.  o_warp is
// [kDecodeWarps][G][D] scratch.  Contains one barrier; o_part is complete for the threads that wrote it only
// after the caller's next barrier.
template <typename T, int D, int G, int U>
__device__ inline void v_phase(const T* Vc, int lo, int hi, const UnitState& st, int special, const T* special_row,
                               const float* sl, int rows_cap, float* o_warp, float* o_part) {
    constexpr int VEC = Elem<T>::kVec;
    constexpr int LPR = D / VEC;
    constexpr int RPW = 32 / LPR;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR, rsub = lane / LPR;
    float acc[G][VEC];
#pragma unroll
    for (int h = 0; h < G; ++h)
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc[h][e] = 0.f;
    for (int base = lo + warp * RPW * U; base < hi; base += kDecodeWarps * RPW * U) {
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int lam = base + u * RPW + rsub;
            raw[u] = make_uint4(0, 0, 0, 0);
            if (lam < hi) {
                if (lam == special) raw[u] = ld_plain(reinterpret_cast<const uint4*>(special_row) + sub);
                else raw[u] = ld_stream(reinterpret_cast<const uint4*>(Vc + (size_t)phys_row(lam, st) * D) + sub);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int lam = base + u * RPW + rsub;
            if (lam < hi) {
                float f[VEC];
                Elem<T>::unpack(raw[u], f);
#pragma unroll
                for (int h = 0; h < G; ++h) {
                    const float p = sl[h * rows_cap + (lam - lo)];
#pragma unroll
                    for (int e = 0; e < VEC; ++e) acc[h][e] = fmaf(p, f[e], acc[h][e]);
                }
            }
        }
    }
    // rows handled by lanes holding the same channel slice
#pragma unroll
    for (int h = 0; h < G; ++h)
#pragma unroll
        for (int e = 0; e < VEC; ++e)
#pragma unroll
            for (int o = 16; o >= LPR; o >>= 1) acc[h][e] += __shfl_xor_sync(0xffffffffu, acc[h][e], o);
    if (rsub == 0) {
#pragma unroll
        for (int h = 0; h < G; ++h)
#pragma unroll
            for (int e = 0; e < VEC; ++e) o_warp[(warp * G + h) * D + sub * VEC + e] = acc[h][e];
    }
    __syncthreads();
    for (int t = tid; t < G * D; t += kDecodeThreads) {
        float r = 0.f;
        for (int w = 0; w < kDecodeWarps; ++w) r += o_warp[w * G * D + t];
        o_part[t] = r;
    }
}

}  // namespace treekv
