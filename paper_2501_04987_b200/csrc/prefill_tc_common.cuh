// Pieces shared by the two tensor-core prefill kernels (one / two 128-row query tiles per thread block): tile
// geometry in shared memory, the walk over a unit's key tiles in cycle coordinates, and the one-instruction exp2.
#pragma once

#include "common.cuh"
#include "tma.cuh"

namespace treekv {
namespace tc {

constexpr int kSlot = 32768;   // one tile: [2 halves of 64 channels or 64 queries][128 rows][128 bytes]
constexpr int kHalf = 16384;
constexpr uint32_t kTmemCols = 512;
constexpr int kD = 128;
constexpr int kThreads = 576;  // TMA warp, MMA warp, 2 groups x 8 softmax warps

// Where a thread block's keys come from.  Cached tokens are two row segments of the unit's slab (live indices [0, a)
// at row = index, [a, L) at row = index + i).  The chunk's own tokens are either rows of the slab behind them (an
// append kernel ran first), or - "direct" - read from the caller's k / v tensors in tiles of 128 tokens, in which
// case the attention kernel also appends its own tokens to the slab and no append kernel runs.
struct KeyTiles {
    int i;     // cycle position
    int a;     // split point (protected initial tokens + i)
    int L;     // cached rows before the chunk
    int nvis;  // live indices [0, nvis) are visible to at least one query of this thread block
    int nA;    // tiles over the first segment [0, a)
    int nB;    // tiles over the second segment: [a, L) when direct, [a, nvis) otherwise
    int NT;    // all tiles
    bool direct;
};
__device__ inline KeyTiles key_tiles(const UnitState& st, int nvis, bool direct) {
    KeyTiles kt;
    kt.i = st.i; kt.a = st.a; kt.L = st.L; kt.nvis = nvis; kt.direct = direct;
    kt.nA = (st.a + 127) / 128;
    kt.nB = ((direct ? st.L : nvis) - st.a + 127) / 128;
    kt.NT = kt.nA + kt.nB + (direct ? (nvis - st.L + 127) / 128 : 0);
    return kt;
}
// key tile j: first live index, first row (of the slab, or token of the chunk when the result is true), rows that exist
__device__ inline bool tile_of(const KeyTiles& kt, int j, int& lam0, int& row0, int& valid) {
    if (j < kt.nA) { lam0 = j * 128; row0 = lam0; valid = min(128, kt.a - lam0); return false; }
    if (j < kt.nA + kt.nB) {
        lam0 = kt.a + (j - kt.nA) * 128; row0 = lam0 + kt.i; valid = min(128, (kt.direct ? kt.L : kt.nvis) - lam0);
        return false;
    }
    row0 = (j - kt.nA - kt.nB) * 128; lam0 = kt.L + row0; valid = min(128, kt.nvis - lam0);
    return true;
}

// The chunk's k and v as the caller passed them ([batch][chunk_stride][n_kv_heads][128] bf16) when the kernel reads
// its chunk tiles from there (tensor maps over the same memory: channels x heads x tokens, box 64 x 1 x 128);
// k == nullptr: the chunk's rows are already in the slab.
struct ChunkDirect {
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
};

// Direct mode: the thread block appends the tokens [t0, t1) of its own query rows to the unit's slab (Algorithm 1's
// append: k, v, stream position, S = 0) - rows no thread block reads during this kernel.  `nthr` threads with
// index `t` in [0, nthr) take part.
__device__ inline void append_own_tokens(const CacheView& cv, const ChunkDirect& cd, int unit, int b, int kh, int chunk_stride,
                                         const UnitState& st, int N, int t0, int t1, int t, int nthr) {
    const int ntok = t1 - t0;
    if (ntok <= 0) return;
    const size_t rbase = (size_t)unit * cv.R + st.L + st.i + t0;
    const size_t src0 = (((size_t)b * chunk_stride + t0) * cv.Hkv + kh) * (kD / 8);  // in 16-byte pieces
    const size_t sstride = (size_t)cv.Hkv * (kD / 8);
    const uint4* ks = reinterpret_cast<const uint4*>(cd.k);
    const uint4* vs = reinterpret_cast<const uint4*>(cd.v);
    uint4* kd = reinterpret_cast<uint4*>(cv.K) + rbase * (kD / 8);
    uint4* vd = reinterpret_cast<uint4*>(cv.V) + rbase * (kD / 8);
    for (int idx = t; idx < ntok * (kD / 8); idx += nthr) {
        const int r = idx / (kD / 8), e = idx % (kD / 8);
        kd[idx] = ks[src0 + r * sstride + e];
        vd[idx] = vs[src0 + r * sstride + e];
    }
    for (int r = t; r < ntok; r += nthr) {
        cv.pos[rbase + r] = N + t0 + r;
        cv.S[rbase + r] = 0.f;
    }
}

// 2^x on the special-function unit, one instruction (inputs here are <= ~0; results below 2^-126 flush to zero)
__device__ inline float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}


// Output staging.  O^T leaves tensor memory with a thread holding one channel of 32 query rows; written to `out` like
// that, a warp store covers 64 bytes of one row.  Instead the rows are put together in shared memory - [128 query
// rows][256 bytes], the 16-byte pieces of row r XOR-swizzled by (r & 15) so that both the 2-byte puts (a warp: 32
// consecutive channels of one row) and the 16-byte gets (a quarter warp: 8 pieces of one row) are conflict-free -
// and go out as whole 256-byte rows.
__device__ inline void stage_put(unsigned char* stage, int r, int ch, float x) {
    *reinterpret_cast<__nv_bfloat16*>(stage + r * 256 + ((((ch >> 3) ^ (r & 15)) << 4) | ((ch & 7) << 1))) =
        __float2bfloat16_rn(x);
}
// rows [r0, r0 + nrows) of the staged tile (those below rmax) -> out[token][head][channel]; row r is token r / G,
// head r % G of the tile whose first token has index tok0 in the call's tensor; threads t of nthr take part
template <int G>
__device__ inline void stage_flush(const unsigned char* stage, __nv_bfloat16* __restrict__ out, size_t tok0, int Hq, int kh,
                                   int r0, int nrows, int rmax, int t, int nthr) {
    for (int idx = t; idx < nrows * 16; idx += nthr) {
        const int r = r0 + (idx >> 4), c16 = idx & 15;
        if (r < rmax) {
            const uint4 v = *reinterpret_cast<const uint4*>(stage + r * 256 + ((c16 ^ (r & 15)) << 4));
            *reinterpret_cast<uint4*>(out + ((tok0 + r / G) * Hq + kh * G + (r % G)) * kD + c16 * 8) = v;
        }
    }
}

}  // namespace tc
}  // namespace treekv
