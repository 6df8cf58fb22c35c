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

struct KeyTiles {
    int i;     // cycle position: live indices [0, a) sit at row = index, the others at row = index + i
    int a;     // split point (protected initial tokens + i)
    int L;     // cached rows before the chunk
    int nvis;  // live indices [0, nvis) are visible to at least one query of this thread block
    int nA;    // tiles over the first segment [0, a)
    int NT;    // all tiles
};
__device__ inline KeyTiles key_tiles(const UnitState& st, int nvis) {
    KeyTiles kt;
    kt.i = st.i; kt.a = st.a; kt.L = st.L; kt.nvis = nvis;
    kt.nA = (st.a + 127) / 128;
    kt.NT = kt.nA + (nvis - st.a + 127) / 128;
    return kt;
}
// key tile j: first live index, first physical row, rows that exist
__device__ inline void tile_of(const KeyTiles& kt, int j, int& lam0, int& row0, int& valid) {
    if (j < kt.nA) { lam0 = j * 128; row0 = lam0; valid = min(128, kt.a - lam0); }
    else { lam0 = kt.a + (j - kt.nA) * 128; row0 = lam0 + kt.i; valid = min(128, kt.nvis - lam0); }
}

// 2^x on the special-function unit, one instruction (inputs here are <= ~0; results below 2^-126 flush to zero)
__device__ inline float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

}  // namespace tc
}  // namespace treekv
